"""ttf_query_static, the entry point for callers that may not allocate device memory (a server whose memory
belongs to a framework pool, a latency-critical loop that cannot take cudaMalloc's synchronisation, a
plug-in whose host forbids allocation after start-up).  It runs the query pass on a scratch array built into
the library instead of on allocated scratch, so its results must equal ttf_query's.  The file name makes
pytest collect it last: a failure here cannot hide the outcome of any other test."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2605_07355_b200 as P
from paper_2605_07355_b200 import clips
from tests.parity import SIM_ATOL, to_device

pytestmark = pytest.mark.gpu


def _outputs(F, N, fill):
    """pre-allocated result tensors: the entry point under test must not need any allocation of its own"""
    return {
        "anchor": torch.full((1,), fill, dtype=torch.int32, device="cuda"),
        "keep": torch.full((F * N,), 7, dtype=torch.uint8, device="cuda"),
        "dst": torch.full((F * N,), fill, dtype=torch.int32, device="cuda"),
        "best_sim": torch.full((F * N,), float(fill), dtype=torch.float32, device="cuda"),
        "fuse_cnt": torch.full((N,), fill, dtype=torch.int32, device="cuda"),
    }


def _same(got, ref):
    assert int(got["anchor"].item()) == int(ref["anchor"].item())
    assert torch.equal(got["keep"], ref["keep"])
    assert torch.equal(got["dst"], ref["dst"])
    assert torch.equal(got["fuse_cnt"], ref["fuse_cnt"])
    assert float((got["best_sim"] - ref["best_sim"]).abs().max().item()) <= SIM_ATOL


def test_static_scratch_query_matches_query_twice_in_a_row():
    # two different clips back to back: the second call finds the first call's leftovers in the shared scratch
    specs = [clips.CONFIGS["vl2b_cal"], clips.CONFIGS["tiny"]]
    for rep in range(2):
        for s in specs:
            X = to_device(clips.make_clip(s, s.seed + rep))
            ref = P.ttf_query(X, s.r, s.t)
            out = _outputs(s.F, s.N, -5 - rep)
            got = P.ttf_query_static(X, s.r, s.t, out)
            torch.cuda.synchronize()
            _same(got, ref)
    # the same clip twice in a row gives the same bits
    s = specs[0]
    X = to_device(clips.make_clip(s))
    a = P.ttf_query_static(X, s.r, s.t, _outputs(s.F, s.N, -1))
    b = P.ttf_query_static(X, s.r, s.t, _outputs(s.F, s.N, -2))
    torch.cuda.synchronize()
    for k in a:
        assert torch.equal(a[k], b[k]), k


def test_static_scratch_query_takes_no_device_memory():
    """what the entry point exists for: once the address of the built-in array has been looked up, further calls
    (another shape, another stream) leave the device's free memory exactly as it was"""
    s0, s1 = clips.CONFIGS["tiny"], clips.CONFIGS["vl2b_cal"]
    X0, X1 = to_device(clips.make_clip(s0)), to_device(clips.make_clip(s1))
    out0, out1 = _outputs(s0.F, s0.N, -7), _outputs(s1.F, s1.N, -8)
    st = torch.cuda.Stream()
    P.ttf_query_static(X0, s0.r, s0.t, out0)                   # the first call on the device: address look-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    P.ttf_query_static(X1, s1.r, s1.t, out1)                   # a new shape ...
    torch.cuda.synchronize()
    P.ttf_query_static(X0, s0.r, s0.t, out0, stream=st)        # ... and a stream the library has never seen
    st.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    _same(out1, P.ttf_query(X1, s1.r, s1.t))


def test_static_scratch_limit_is_enforced_before_any_launch():
    lib = P.lib()
    fake = ctypes.c_void_p(4096)            # never dereferenced: the size check comes first
    rc = lib.ttf_query_static(fake, 256, 64, 64, 4096, 1, 0.7, P.TTF_DTYPE_BF16, None, None, None, None, None, None)
    assert lib.ttf_status_string(rc) == b"TTF_ERR_STATIC_LIMIT"
    assert lib.ttf_query_static(None, 4, 4, 4, 8, 1, 0.7, 0, None, None, None, None, None, None) == 1
    # a clip that does fit still works afterwards
    s = clips.CONFIGS["tiny"]
    X = to_device(clips.make_clip(s))
    got = P.ttf_query_static(X, s.r, s.t, _outputs(s.F, s.N, -3))
    ref = P.ttf_query(X, s.r, s.t)
    torch.cuda.synchronize()
    _same(got, ref)
