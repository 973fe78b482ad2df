"""The give-up path of the bounded device waits, driven without a fault or a hang: a test hook makes every copy
barrier expect 16 bytes more than its copy delivers and lowers the poll limit, so the data lands, the barrier never
completes, the waiting lane runs out of polls, stops and sets the error word."""
import numpy as np
import pytest
import torch

import paper_2605_07355_b200 as P
from paper_2605_07355_b200 import binding as B
from tests.parity import check_clip, to_device
from tests.test_gpu_parity import corr_clip

pytestmark = pytest.mark.gpu


def test_copy_wait_runs_out_then_the_next_call_is_clean():
    X = corr_clip(6, 6, 7, 256, seed=77, dtype="bf16")
    Xd = to_device(X)
    st = torch.cuda.Stream()
    ref = P.ttf_compress(Xd, 1, 0.7, stream=st)
    assert P.ttf_last_device_status(st) == B.TTF_OK
    L = int(ref[1].item())
    assert L > 6 * 7
    P.ttf_debug_set_wait(32, 16)
    try:
        toks, cnt, pos = P.ttf_compress(Xd, 1, 0.7, stream=st)
        assert P.ttf_last_device_status(st) == B.TTF_ERR_TIMEOUT        # synchronises the stream
        assert int(cnt.item()) == -1
        # a batch reports through the caller's stream
        outs = P.ttf_compress_batch([Xd, Xd, Xd], 1, 0.7, stream=st)
        assert P.ttf_last_device_status(st) == B.TTF_ERR_TIMEOUT
        assert all(int(c.item()) == -1 for c in outs[1])
    finally:
        P.ttf_debug_set_wait()
    # the same stream, hence the same scratch block: nothing of the failed calls is left
    toks, cnt, pos = P.ttf_compress(Xd, 1, 0.7, stream=st)
    assert P.ttf_last_device_status(st) == B.TTF_OK
    assert int(cnt.item()) == L
    assert torch.equal(toks[:L], ref[0][:L]) and torch.equal(pos[:L], ref[2][:L])
    outs = P.ttf_compress_batch([Xd, Xd, Xd], 1, 0.7, stream=st)
    assert P.ttf_last_device_status(st) == B.TTF_OK
    assert all(int(c.item()) == L for c in outs[1])
    with torch.cuda.stream(st):
        check_clip(X, 1, 0.7, stream=st)                                 # and it still equals the oracle


@pytest.mark.parametrize("C", [256, 2048])
def test_tensor_core_pipeline_gives_up_and_recovers(C):
    """the tcgen05 matching kernel under the same hook: its copy barriers never complete, so its MMA issuer, its
    epilogue warps and then its producer run out of polls; the CTAs (alone for C = 256, in clusters of 8 for
    C = 2048) still meet at their barriers, free their tensor memory and return; the query reports the time-out
    and the next call is clean"""
    X = corr_clip(6, 6, 7, C, seed=79, dtype="bf16")
    Xd = to_device(X)
    st = torch.cuda.Stream()
    P.ttf_set_match_kernel(2)
    try:
        ref = P.ttf_query(Xd, 1, 0.7, stream=st)
        assert P.ttf_last_device_status(st) == B.TTF_OK
        P.ttf_debug_set_wait(32, 16)
        try:
            P.ttf_query(Xd, 1, 0.7, stream=st)
            assert P.ttf_last_device_status(st) == B.TTF_ERR_TIMEOUT
            _, cnt, _ = P.ttf_compress(Xd, 1, 0.7, stream=st)
            assert P.ttf_last_device_status(st) == B.TTF_ERR_TIMEOUT and int(cnt.item()) == -1
        finally:
            P.ttf_debug_set_wait()
        again = P.ttf_query(Xd, 1, 0.7, stream=st)
        assert P.ttf_last_device_status(st) == B.TTF_OK
        for k in ref:
            assert torch.equal(ref[k], again[k]), k
        with torch.cuda.stream(st):
            check_clip(X, 1, 0.7, stream=st)
    finally:
        P.ttf_set_match_kernel(0)


def test_status_of_caller_owned_and_built_in_scratch():
    X = corr_clip(4, 5, 5, 128, seed=78, dtype="bf16")
    Xd = to_device(X)
    nbytes = P.ttf_workspace_bytes(4, 5, 5, 128, 1, 1)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    P.ttf_debug_set_wait(32, 16)
    try:
        _, cnt, _ = P.ttf_compress(Xd, 1, 0.7, workspace=ws)
        assert P.ttf_workspace_status(ws) == B.TTF_ERR_TIMEOUT and int(cnt.item()) == -1
    finally:
        P.ttf_debug_set_wait()
    _, cnt, _ = P.ttf_compress(Xd, 1, 0.7, workspace=ws)
    assert P.ttf_workspace_status(ws) == B.TTF_OK and int(cnt.item()) > 0
    out = {"keep": torch.empty(100, dtype=torch.uint8, device="cuda")}
    P.ttf_query_static(Xd, 1, 0.7, out)
    assert P.ttf_workspace_status(None) == B.TTF_OK
    assert P.ttf_last_device_status(torch.cuda.Stream()) == B.TTF_OK      # a stream the library has never seen
