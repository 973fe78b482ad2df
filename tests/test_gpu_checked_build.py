"""The checked build of the library (the same sources with -DTTF_DEBUG: every global store whose index a kernel
computes is preceded by a range test that records and skips, never traps) runs the parity cases with a clean
status, and its reporting path works: with the test hook lowering every limit by a few elements, valid indices at
the end of the arrays are reported (TTF_ERR_BOUNDS) and skipped, all accesses still in bounds; the next call is
clean again.  The library path is fixed when it is first loaded, so the case runs in a process of its own."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASE = r"""
import numpy as np, torch
import paper_2605_07355_b200 as P
from paper_2605_07355_b200 import clips
from tests.parity import check_clip, to_device
from tests.test_gpu_parity import corr_clip

assert P.LIB_PATH.endswith("libttf_b200_checked.so")
assert P.ttf_debug_set_check_slack(0) == 0                       # this build has the checks
shapes = [(4, 8, 8, 64, 1, "bf16"), (5, 6, 7, 256, 1, "bf16"), (6, 5, 6, 264, 0, "bf16"), (4, 6, 7, 520, 2, "bf16"),
          (33, 2, 3, 64, 1, "bf16"), (5, 3, 7, 40, 1, "f32"), (3, 4, 4, 33, 3, "f32"), (40, 7, 9, 512, 1, "bf16")]
for which in (1, 2):                                              # warp-level and tcgen05 matching
    P.ttf_set_match_kernel(which)
    for (F, H, W, C, r, dt) in shapes:
        X = corr_clip(F, H, W, C, seed=F + H + W + C + r, dtype=dt)
        check_clip(X, r, 0.7)
        check_clip(X, r, 0.5, order=1, pos_base=3)
        assert P.ttf_last_device_status() == 0, (which, F, H, W, C, r, dt)
P.ttf_set_match_kernel(0)
s = clips.CONFIGS["vl2b_cal"]
check_clip(clips.make_clip(s), s.r, s.t)
assert P.ttf_last_device_status() == 0

# the reporting path: limits lowered by 5 elements, so the last tokens' results are reported and not written
X = corr_clip(6, 5, 4, 64, seed=9, dtype="bf16")
Xd = to_device(X)
for which in (1, 2):
    P.ttf_set_match_kernel(which)
    assert P.ttf_debug_set_check_slack(5) == 0
    P.ttf_query(Xd, 1, 0.7)
    assert P.ttf_last_device_status() == P.TTF_ERR_BOUNDS, which
    assert P.ttf_debug_set_check_slack(0) == 0
    check_clip(X, 1, 0.7)                                         # the first kernel of a call clears the word
    assert P.ttf_last_device_status() == 0
print("checked build ok")
"""


def test_checked_build_passes_parity_and_reports_through_the_status_word():
    from paper_2605_07355_b200 import build as B
    lib = B.build(checked=True)
    env = dict(os.environ, TTF_B200_LIB=lib)
    out = subprocess.run([sys.executable, "-c", CASE], env=env, cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "checked build ok" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]
