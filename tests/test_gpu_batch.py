"""GPU parity of the batch entry points (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips
import paper_2605_07355_b200 as P
from tests.parity import check_clip, to_device, to_bits
from tests.test_gpu_parity import corr_clip

pytestmark = pytest.mark.gpu


def assert_same_as_single(Xs, r, t, outs):
    """every clip of a batch must give exactly what ttf_compress gives for it alone"""
    toks, cnts, poss = outs
    for j, X in enumerate(Xs):
        a = P.ttf_compress(X, r, t)
        torch.cuda.synchronize()
        L = int(a[1].item())
        assert int(cnts[j].item()) == L, (j, int(cnts[j].item()), L)
        assert torch.equal(toks[j][:L], a[0][:L]) and torch.equal(poss[j][:L], a[2][:L]), j


def test_batch_on_library_streams_matches_single_calls_and_oracle():
    s = clips.CONFIGS["vl2b_cal"]
    Xn = [clips.make_clip(s, s.seed + j) for j in range(11)]         # 11 clips over 8 streams: ragged last round
    Xs = [to_device(x) for x in Xn]
    outs = P.ttf_compress_batch(Xs, s.r, s.t)
    torch.cuda.synchronize()
    assert_same_as_single(Xs, s.r, s.t, outs)
    R = O.compress(Xn[3], s.r, s.t)
    q = P.ttf_query(Xs[3], s.r, s.t)
    forced = O.compress(Xn[3], s.r, s.t, anchor_frame=int(q["anchor"].item()), forced_keep=q["keep"].cpu().numpy())
    in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(s.t)) < 1e-4
    assert not ((q["keep"].cpu().numpy() != R.keep) & ~in_band).any()
    L = int(outs[1][3].item())
    assert L == forced.count
    assert (outs[2][3][:L].cpu().numpy() == forced.pos).all() and (to_bits(outs[0][3][:L]) == forced.tokens).all()


def test_batch_small_and_fp32_and_stream_order():
    Xs = [to_device(corr_clip(3, 4, 5, 40, seed=31 + j, dtype="f32")) for j in range(3)]
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        outs = P.ttf_compress_batch(Xs, 1, 0.7, stream=st)
        first = outs[1][0] + 0                   # ordered after the batch on the caller's stream
    st.synchronize()
    assert_same_as_single(Xs, 1, 0.7, outs)
    assert int(first.item()) == int(outs[1][0].item())
    one = P.ttf_compress_batch(Xs[:1], 1, 0.7)
    torch.cuda.synchronize()
    assert_same_as_single(Xs[:1], 1, 0.7, one)
    with pytest.raises(ValueError):
        P.ttf_compress_batch([Xs[0], Xs[1][:2]], 1, 0.7)


SHAPES = [(1, 4, 4, 32, 1), (2, 3, 5, 40, 1), (6, 5, 6, 264, 0), (17, 3, 3, 72, 1), (33, 2, 3, 64, 1),
          (9, 4, 6, 1032, 1), (40, 7, 9, 512, 2)]


@pytest.mark.parametrize("kernel", [1, 2])
@pytest.mark.parametrize("shape", SHAPES)
def test_batch_chains_small_shapes(shape, kernel):
    """seven clips over one, two and three lanes: clips of a lane form a chain on two scratch blocks in which the
    sweep of a clip runs beside the gather of the clip before it; both matching kernels"""
    F, H, W, C, r = shape
    Xs = [to_device(corr_clip(F, H, W, C, seed=sum(shape) + j, dtype="bf16")) for j in range(7)]
    P.ttf_set_match_kernel(kernel)
    try:
        ref = [P.ttf_compress(x, r, 0.6) for x in Xs]
        torch.cuda.synchronize()
        for lanes in (1, 2, 3):
            P.ttf_set_schedule(lanes)
            for rep in range(2):
                toks, cnts, poss = P.ttf_compress_batch(Xs, r, 0.6)
            torch.cuda.synchronize()
            assert P.ttf_last_device_status() == 0
            for j in range(len(Xs)):
                L = int(ref[j][1].item())
                assert int(cnts[j].item()) == L, (lanes, j)
                assert torch.equal(toks[j][:L], ref[j][0][:L]) and torch.equal(poss[j][:L], ref[j][2][:L])
        check_clip(to_bits(Xs[3]).reshape(F, H, W, C), r, 0.6)
    finally:
        P.ttf_set_schedule(0)
        P.ttf_set_match_kernel(0)


def test_batch_with_options_matches_single_calls():
    Xs = [to_device(corr_clip(5, 6, 6, 128, seed=400 + j, dtype="bf16")) for j in range(5)]
    for kw in (dict(anchor_mode=1), dict(anchor_mode=2, order=1), dict(anchor_mode=3, anchor_frame=2, pos_base=99), dict(order=1)):
        toks, cnts, poss = P.ttf_compress_batch(Xs, 1, 0.6, **kw)
        torch.cuda.synchronize()
        for j, x in enumerate(Xs):
            a = P.ttf_compress(x, 1, 0.6, **kw)
            torch.cuda.synchronize()
            L = int(a[1].item())
            assert int(cnts[j].item()) == L
            assert torch.equal(toks[j][:L], a[0][:L]) and torch.equal(poss[j][:L], a[2][:L])


def test_host_batch_matches_device_calls():
    s = clips.CONFIGS["tiny_cal"]
    Xn = [clips.make_clip(s, s.seed + j) for j in range(5)]           # more clips than staging slots
    host = [torch.from_numpy(x).pin_memory() for x in Xn]
    toks, Ls, poss = P.ttf_compress_host_batch(host, s.r, s.t)
    for j, x in enumerate(Xn):
        a = P.ttf_compress(to_device(x), s.r, s.t)
        torch.cuda.synchronize()
        L = int(a[1].item())
        assert Ls[j] == L and torch.equal(toks[j], a[0][:L].cpu()) and torch.equal(poss[j], a[2][:L].cpu())
    one_t, one_L, one_p = P.ttf_compress_host(host[2], s.r, s.t)
    assert one_L == Ls[2] and torch.equal(one_t, toks[2]) and torch.equal(one_p, poss[2])


def test_bench_configuration_full_size_against_oracle():
    """the launch configuration the benchmark times: 16 clips of the 8B shape through one ttf_compress_batch call,
    every clip checked against the oracle (decisions outside the threshold band exact, the rest bit for bit)"""
    s = clips.CONFIGS["vl8b_cal"]
    n = 16
    Xn = [clips.make_clip(s, s.seed + j) for j in range(n)]
    Xs = [to_device(x) for x in Xn]
    for rep in range(2):                                               # second round: scratch reuse across calls
        toks, cnts, poss = P.ttf_compress_batch(Xs, s.r, s.t)
    torch.cuda.synchronize()
    rhos = []
    for j in range(n):
        R = O.compress(Xn[j], s.r, s.t)
        q = P.ttf_query(Xs[j], s.r, s.t)
        keep = q["keep"].cpu().numpy()
        assert int(q["anchor"].item()) == R.anchor
        in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(s.t)) < 1e-4
        assert not ((keep != R.keep) & ~in_band).any()
        forced = O.compress(Xn[j], s.r, s.t, anchor_frame=R.anchor, forced_keep=keep)
        L = int(cnts[j].item())
        assert L == forced.count
        assert (poss[j][:L].cpu().numpy() == forced.pos).all()
        assert (to_bits(toks[j][:L]) == forced.tokens).all()
        rhos.append(1.0 - L / s.tokens)
    assert abs(float(np.mean(rhos)) - 0.67) < 0.03
    # the benchmark replays the call from a CUDA graph: the replayed batch must write the same bytes
    st = torch.cuda.Stream()
    gt = [torch.zeros_like(x) for x in toks]
    gc = [torch.zeros_like(x) for x in cnts]
    gp = [torch.zeros_like(x) for x in poss]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        P.ttf_compress_batch(Xs, s.r, s.t, gt, gc, gp, stream=st)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    for j in range(n):
        L = int(cnts[j].item())
        assert int(gc[j].item()) == L
        assert torch.equal(gt[j][:L], toks[j][:L]) and torch.equal(gp[j][:L], poss[j][:L])


def test_host_batch_fp32_and_single_clip():
    Xn = [corr_clip(4, 3, 5, 24, seed=70 + j, dtype="f32") for j in range(3)]
    host = [torch.from_numpy(x) for x in Xn]                              # pageable memory works too
    toks, Ls, poss = P.ttf_compress_host_batch(host, 1, 0.6)
    for j, x in enumerate(Xn):
        R = O.compress(x, 1, 0.6)
        q = P.ttf_query(to_device(x), 1, 0.6)
        forced = O.compress(x, 1, 0.6, anchor_frame=int(q["anchor"].item()), forced_keep=q["keep"].cpu().numpy())
        assert Ls[j] == forced.count
        assert (toks[j].numpy() == forced.tokens).all() and (poss[j].numpy() == forced.pos).all()
    one = P.ttf_compress_host_batch(host[:1], 1, 0.6)
    assert one[1][0] == Ls[0] and torch.equal(one[0][0], toks[0])


@pytest.mark.parametrize("name", ["long", "long_cal"])
def test_long_video_batch_of_eight_against_oracle(name):
    """the long-video configuration at full size: 8 clips of F=128 frames in one ttf_compress_batch call; `long`
    is the configuration text word for word (per-clip noise level, Poisson scene cuts), `long_cal` the anchored
    variant the throughput runs use"""
    s = clips.CONFIGS[name]
    n = 8
    Xs, refs = [], []
    for j in range(n):
        Xn = clips.make_clip(s, s.seed + j)
        refs.append((Xn, O.compress(Xn, s.r, s.t)))
        Xs.append(to_device(Xn))
    toks, cnts, poss = P.ttf_compress_batch(Xs, s.r, s.t)
    torch.cuda.synchronize()
    for j, (Xn, R) in enumerate(refs):
        q = P.ttf_query(Xs[j], s.r, s.t)
        keep = q["keep"].cpu().numpy()
        assert int(q["anchor"].item()) == R.anchor
        in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(s.t)) < 1e-4
        assert not ((keep != R.keep) & ~in_band).any()
        forced = O.compress(Xn, s.r, s.t, anchor_frame=R.anchor, forced_keep=keep)
        L = int(cnts[j].item())
        assert L == forced.count
        assert (poss[j][:L].cpu().numpy() == forced.pos).all()
        assert (to_bits(toks[j][:L]) == forced.tokens).all()


def test_multi_block_scratch_after_another_shape_on_the_same_stream():
    """the per-stream scratch cache is reused with another layout: blocks of the batch land on old data"""
    st = torch.cuda.Stream()
    big = to_device(clips.make_clip(clips.CONFIGS["vl2b_cal"]))
    small = [to_device(corr_clip(4, 5, 5, 128, seed=200 + j, dtype="bf16")) for j in range(6)]
    ref = [P.ttf_compress(x, 1, 0.7) for x in small]
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        P.ttf_compress(big, 1, 0.7, stream=st)                     # fills the stream's scratch with its arrays
        toks, cnts, poss = P.ttf_compress_batch(small, 1, 0.7, stream=st)
    st.synchronize()
    for j in range(len(small)):
        L = int(ref[j][1].item())
        assert int(cnts[j].item()) == L
        assert torch.equal(toks[j][:L], ref[j][0][:L]) and torch.equal(poss[j][:L], ref[j][2][:L])


@pytest.mark.parametrize("match_kernel", [1, 2])
def test_pipelined_schedule_gives_the_same_results(match_kernel):
    """ttf_set_schedule(TTF_SCHEDULE_PIPELINED): two lanes in opposite phases, L2 eviction hints on the matching
    pass and the gather; scheduling and cache policy only, so every clip must come out bit for bit as from
    ttf_compress, and equal to the oracle (8B-shaped clips, seven of them: several turns per lane and a ragged
    end; then small fp32 clips, which take the kernels without hints)"""
    s = clips.CONFIGS["vl8b_cal"]
    Xn = [clips.make_clip(s, s.seed + j) for j in range(7)]
    Xs = [to_device(x) for x in Xn]
    P.ttf_set_match_kernel(match_kernel)
    P.ttf_set_schedule(P.TTF_SCHEDULE_PIPELINED)
    try:
        for _ in range(2):                       # the second call finds the scratch blocks as the first left them
            outs = P.ttf_compress_batch(Xs, s.r, s.t)
            torch.cuda.synchronize()
            assert P.ttf_last_device_status() == P.TTF_OK
            assert_same_as_single(Xs, s.r, s.t, outs)
        R = O.compress(Xn[5], s.r, s.t)
        q = P.ttf_query(Xs[5], s.r, s.t)
        keep = q["keep"].cpu().numpy()
        assert int(q["anchor"].item()) == R.anchor
        in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(s.t)) < 1e-4
        assert not ((keep != R.keep) & ~in_band).any()
        forced = O.compress(Xn[5], s.r, s.t, anchor_frame=R.anchor, forced_keep=keep)
        L = int(outs[1][5].item())
        assert L == forced.count
        assert (outs[2][5][:L].cpu().numpy() == forced.pos).all() and (to_bits(outs[0][5][:L]) == forced.tokens).all()
        small = [to_device(corr_clip(5, 4, 5, 40, seed=77 + j, dtype="f32")) for j in range(5)]
        outs = P.ttf_compress_batch(small, 1, 0.7)
        torch.cuda.synchronize()
        assert_same_as_single(small, 1, 0.7, outs)
        first = P.ttf_compress_batch(Xs[:4], s.r, s.t, anchor_mode=P.TTF_ANCHOR_FIRST)   # fixed anchor: ordinary lanes
        torch.cuda.synchronize()
        for j in range(4):
            a = P.ttf_compress(Xs[j], s.r, s.t, anchor_mode=P.TTF_ANCHOR_FIRST)
            torch.cuda.synchronize()
            L = int(a[1].item())
            assert int(first[1][j].item()) == L and torch.equal(first[0][j][:L], a[0][:L])
    finally:
        P.ttf_set_schedule(0)
        P.ttf_set_match_kernel(0)
