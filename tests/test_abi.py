"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol include/ttf.h declares,
and rejects invalid arguments before any CUDA call."""
import ctypes
import os
import re

import pytest

import paper_2605_07355_b200 as P
from paper_2605_07355_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return P.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ttf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*|int)\s+(ttf_\w+)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert "ttf_compress" in names and "ttf_query" in names and len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(P.EXPORTS)


def test_checked_build_exports_the_same_symbols_and_only_it_takes_the_slack_hook(lib):
    from paper_2605_07355_b200 import build as B
    checked = ctypes.CDLL(B.build(checked=True))
    for n in declared_symbols():
        assert hasattr(checked, n), n
    assert lib.ttf_debug_set_check_slack(3) == 2                  # TTF_ERR_UNSUPPORTED: no checks in the normal build
    assert checked.ttf_debug_set_check_slack(-1) == 1
    assert checked.ttf_debug_set_check_slack(3) == 0 and checked.ttf_debug_set_check_slack(0) == 0
    checked.ttf_status_string.restype = ctypes.c_char_p
    assert checked.ttf_status_string(7) == b"TTF_ERR_BOUNDS"


def test_status_strings(lib):
    assert lib.ttf_status_string(0) == b"TTF_OK"
    assert lib.ttf_status_string(1) == b"TTF_ERR_INVALID_ARG"
    assert lib.ttf_status_string(99) == b"TTF_ERR_UNKNOWN"


def test_workspace_bytes_and_validation(lib):
    n = P.ttf_workspace_bytes(32, 16, 16, 4096, 1, P.TTF_DTYPE_BF16)
    assert n % 256 == 0 and n > 32 * 4096 * 4
    assert P.ttf_workspace_bytes(64, 32, 32, 4096, 2, P.TTF_DTYPE_BF16) > n
    sz = ctypes.c_size_t(0)
    bad = [(0, 4, 4, 8, 1, 0), (4, 0, 4, 8, 1, 0), (4, 4, 4, 0, 1, 0), (4, 4, 4, 8, -1, 0), (4, 4, 4, 8, 1, 7)]
    for args in bad:
        assert lib.ttf_workspace_bytes(*args, ctypes.byref(sz)) == 1
    assert lib.ttf_workspace_bytes(1 << 16, 1 << 8, 1 << 8, 8, 1, 0, ctypes.byref(sz)) == 2     # F*H*W >= 2^31
    assert lib.ttf_workspace_bytes(4, 4, 4, 8, 1, 0, None) == 1


def test_null_and_nonfinite_arguments_are_rejected_before_any_launch(lib):
    fake = ctypes.c_void_p(4096)        # never dereferenced: validation fails first
    f = lib.ttf_compress
    assert f(None, 4, 4, 4, 8, 1, 0.7, 0, fake, fake, fake, None) == 1
    assert f(fake, 4, 4, 4, 8, 1, 0.7, 0, None, fake, fake, None) == 1
    assert f(fake, 4, 4, 4, 8, 1, float("nan"), 0, fake, fake, fake, None) == 1
    assert f(fake, 4, 4, 4, 8, 1, float("inf"), 0, fake, fake, fake, None) == 1
    assert f(fake, 4, 4, 4, 8, -1, 0.7, 0, fake, fake, fake, None) == 1
    assert f(fake, 4, 4, 4, 8, 1, 0.7, 3, fake, fake, fake, None) == 1
    assert lib.ttf_compress_ws(fake, 4, 4, 4, 8, 1, 0.7, 0, fake, fake, fake, None, 0, None) == 3
    assert lib.ttf_compress_ws(fake, 4, 4, 4, 8, 1, 0.7, 0, fake, fake, fake, ctypes.c_void_p(4096 + 8), 1 << 30, None) == 3
    assert lib.ttf_query(None, 4, 4, 4, 8, 1, 0.7, 0, None, None, None, None, None, None) == 1
    assert lib.ttf_compress_host(None, 4, 4, 4, 8, 1, 0.7, 0, fake, fake, fake) == 1
    from paper_2605_07355_b200.binding import TTFOptions
    opt = lambda *a: ctypes.byref(TTFOptions(*a))
    ex = lib.ttf_compress_ex
    assert ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(4, 0, 0, 0), fake, fake, fake, None) == 1      # unknown anchor rule
    assert ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(3, 4, 0, 0), fake, fake, fake, None) == 1      # explicit frame >= F
    assert ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(0, 0, 2, 0), fake, fake, fake, None) == 1      # unknown order
    assert ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(0, 0, 0, -1), fake, fake, fake, None) == 1     # negative position base
    assert ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(0, 0, 0, 2**31 - 2), fake, fake, fake, None) == 1   # positions overflow
    assert ex(None, 4, 4, 4, 8, 1, 0.7, 0, None, fake, fake, fake, None) == 1
    assert lib.ttf_query_ex(fake, 4, 4, 4, 8, 1, 0.7, 0, opt(3, -1, 0, 0), None, None, None, None, None, None) == 1
    arr = (ctypes.c_void_p * 2)(4096, 8192)
    assert lib.ttf_compress_batch_ex(arr, 2, 4, 4, 4, 8, 1, 0.7, 0, opt(0, 0, 0, 0), None, arr, arr, None) == 1


def test_batch_and_variant_entry_points_validate_before_any_cuda_call(lib):
    fake = ctypes.c_void_p(4096)
    arr = (ctypes.c_void_p * 2)(4096, 8192)
    hole = (ctypes.c_void_p * 2)(4096, None)
    counts = (ctypes.c_int * 2)()
    f = lib.ttf_compress_batch
    assert f(None, 2, 4, 4, 4, 8, 1, 0.7, 0, arr, arr, arr, None) == 1
    assert f(arr, 0, 4, 4, 4, 8, 1, 0.7, 0, arr, arr, arr, None) == 1
    assert f(hole, 2, 4, 4, 4, 8, 1, 0.7, 0, arr, arr, arr, None) == 1          # a NULL clip inside the batch
    assert f(arr, 2, 4, 4, 4, 0, 1, 0.7, 0, arr, arr, arr, None) == 1
    assert f(arr, 2, 4, 4, 4, 8, 1, float("nan"), 0, arr, arr, arr, None) == 1
    h = lib.ttf_compress_host_batch
    assert h(arr, 0, 4, 4, 4, 8, 1, 0.7, 0, arr, ctypes.cast(counts, ctypes.c_void_p), arr) == 1
    assert h(arr, 2, 4, 4, 4, 8, 1, 0.7, 0, hole, ctypes.cast(counts, ctypes.c_void_p), arr) == 1
    assert h(arr, 2, 4, 4, 4, 8, 1, 0.7, 0, arr, None, arr) == 1
    assert h(arr, 2, 4, 4, 4, 8, -1, 0.7, 0, arr, ctypes.cast(counts, ctypes.c_void_p), arr) == 1
    assert lib.ttf_compress_mean(None, 4, 4, 4, 8, 1, 0.7, 0, fake, fake, fake, None) == 1
    assert lib.ttf_compress_mean(fake, 4, 4, 4, 8, 1, 0.7, 2, fake, fake, fake, None) == 1
    ms = (ctypes.c_double * 5)()
    assert lib.ttf_profile_stages(arr, 2, 4, 4, 4, 8, 1, 0.7, 0, arr, arr, arr, 0, ms, 5, None) == 1   # reps < 1
    assert lib.ttf_profile_stages(arr, 2, 4, 4, 4, 8, 1, 0.7, 0, arr, arr, arr, 1, None, 5, None) == 1
    assert lib.ttf_stats(None, fake, fake, 4, 4, 4, 0.7, 1e-4, fake, None) == 1
    assert lib.ttf_stats(fake, fake, fake, 4, 4, 4, 0.7, -1.0, fake, None) == 1                  # negative band
    assert lib.ttf_stats(fake, fake, fake, 4, 4, 4, float("nan"), 1e-4, fake, None) == 1
    assert lib.ttf_stats(fake, fake, fake, 0, 4, 4, 0.7, 1e-4, fake, None) == 1
    one = ctypes.c_double()
    assert lib.ttf_profile_read_floor(arr, 2, ctypes.c_size_t(24), 1, ctypes.byref(one), None) == 1     # not a multiple of 16
    assert lib.ttf_profile_read_floor(hole, 2, ctypes.c_size_t(32), 1, ctypes.byref(one), None) == 1
    assert lib.ttf_profile_read_floor(arr, 2, ctypes.c_size_t(32), 0, ctypes.byref(one), None) == 1
    assert lib.ttf_set_schedule(9) == 1 and lib.ttf_set_schedule(-2) == 1
    assert lib.ttf_set_schedule(-1) == 0         # TTF_SCHEDULE_PIPELINED
    assert lib.ttf_set_schedule(0) == 0


def test_decode_alignment_helper():
    assert P.ttf_decode_pos(2703, 57, 0) == 2760 and P.ttf_decode_pos(2703, 57, 4) == 2764


def test_flop_counter_reproduces_table3():
    """The paper's Table 3 prints 18 / 164 / 456 MFLOPS for r = 0 / 1 / 2 (F=32, N=256); 2(F-1)N(2r+1)^2 C
    gives those figures for C = 1152 (456 is 25 x the rounded per-candidate figure)."""
    from paper_2605_07355_b200 import accounting as A
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "table3_mflops.txt")) if l[0].isdigit()]
    got = {int(r): A.matching_flops_nominal(32, 256, 1152, int(r)) / 1e6 for r, _, _ in rows}
    for r, _, printed in rows:
        assert abs(got[int(r)] - float(printed)) / float(printed) < 0.02
    assert abs(got[1] / 1e3 - 0.16) < 0.01                  # abstract: about 0.16 GFLOPs
    assert A.window_pairs(16, 16, 1) == 2116 and A.window_pairs(32, 32, 2) == 23716
    assert A.matching_flops(32, 16, 16, 1152, 1) < A.matching_flops_nominal(32, 256, 1152, 1)
    assert A.pass_bytes(32, 256, 4096, 2, 2703) == 32 * 256 * 4096 * 2 + 2703 * 8192 + 2703 * 12 + 4


def test_dynamic_shared_memory_limits_are_recorded_per_function_and_device(lib):
    """a function attribute set in one device's context says nothing about another device"""
    import ctypes
    need = lib.ttf_debug_func_attr_needed
    need.restype = ctypes.c_int
    need.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t]
    key_a, key_b = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x2000)
    assert need(key_a, 0, 65536) == 1            # first launch of a on device 0: set it
    assert need(key_a, 0, 65536) == 0            # already set there
    assert need(key_a, 1, 65536) == 1            # device 1 has its own context
    assert need(key_b, 0, 65536) == 1            # another function
    assert need(key_a, 0, 32768) == 0            # a smaller request is covered
    assert need(key_a, 0, 131072) == 1           # a larger one is not
    assert need(key_a, 1, 65536) == 0


def test_status_entry_points_validate(lib):
    import ctypes
    assert lib.ttf_last_device_status(None, None) == 1
    assert lib.ttf_workspace_status(None, None, None) == 1
    assert lib.ttf_debug_set_wait(0, 0) == 1 and lib.ttf_debug_set_wait(8, 8) == 1 and lib.ttf_debug_set_wait(8, 2048) == 1
    assert lib.ttf_debug_set_wait(1 << 18, 0) == 0
    assert lib.ttf_status_string(5) == b"TTF_ERR_TIMEOUT" and lib.ttf_status_string(6) == b"TTF_ERR_STATIC_LIMIT"
