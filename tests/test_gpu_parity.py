"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded clips."""
import numpy as np
import pytest
import torch

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips
import paper_2605_07355_b200 as P
from tests.parity import check_clip, to_device, to_bits

pytestmark = pytest.mark.gpu


def corr_clip(F, H, W, C, seed, dtype="f32", sigma=0.5):
    rng = np.random.default_rng(seed)
    base = rng.standard_normal((H, W, C))
    X = base[None] + sigma * rng.standard_normal((F, H, W, C)) * np.exp(0.7 * rng.standard_normal((F, H, W, 1)))
    X = X.astype(np.float32)
    return X if dtype == "f32" else clips.f32_to_bf16_bits(X)


@pytest.mark.parametrize("name", ["tiny", "tiny_cal"])
def test_tiny_config(name):
    s = clips.CONFIGS[name]
    rep = check_clip(clips.make_clip(s), s.r, s.t)
    assert 0.2 < rep["rho"] < 0.75


SHAPES = [
    # F, H, W, C, r
    (1, 4, 4, 32, 1), (2, 3, 5, 40, 1), (3, 7, 5, 33, 1), (5, 1, 9, 24, 1), (4, 9, 1, 16, 2),
    (3, 2, 2, 7, 1), (6, 5, 6, 264, 0), (4, 6, 7, 520, 2), (3, 4, 4, 64, 5), (17, 3, 3, 72, 1),
    (33, 2, 3, 8, 1), (4, 5, 5, 1, 1), (2, 1, 1, 16, 1), (9, 4, 6, 1032, 1),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_small_shapes(shape, dtype):
    F, H, W, C, r = shape
    X = corr_clip(F, H, W, C, seed=sum(shape), dtype=dtype)
    for t in (0.7, 0.5):
        check_clip(X, r, t)


@pytest.mark.parametrize("t", [-2.0, 0.0, 0.7, 1.0, 2.0])
def test_threshold_range(t):
    X = corr_clip(4, 6, 5, 48, seed=3, dtype="bf16")
    rep = check_clip(X, 1, t)
    if t >= 1.0:
        assert rep["count"] == 4 * 30
    if t < -1.0:
        assert rep["count"] == 30


def test_identical_frames_and_zero_tokens():
    X = np.repeat(corr_clip(1, 5, 4, 64, seed=8), 4, axis=0)
    rep = check_clip(X, 1, 0.7)
    assert rep["count"] == 20 and rep["anchor"] == 0
    Z = corr_clip(3, 4, 4, 32, seed=9)
    Z[1, 2, 1] = 0.0
    Z[0, 0, 0] = 0.0
    check_clip(Z, 1, 0.0)
    check_clip(np.zeros((3, 3, 3, 16), np.float32), 1, 0.5)


@pytest.mark.parametrize("mode,frame", [(1, 0), (2, 0), (3, 0), (3, 2), (3, 4)])
def test_fixed_anchor_rules(mode, frame):
    """first / last / explicit anchors (the paper's Table 1 variants)"""
    for dtype, shape in (("bf16", (5, 6, 7, 256)), ("f32", (5, 4, 5, 40))):
        X = corr_clip(*shape, seed=21 + mode + frame, dtype=dtype)
        rep = check_clip(X, 1, 0.7, anchor_mode=mode, anchor_frame=frame)
        assert rep["anchor"] == {1: 0, 2: shape[0] - 1, 3: frame}[mode]
    with pytest.raises(P.TTFError):
        P.ttf_query(to_device(X), 1, 0.7, anchor_mode=3, anchor_frame=5)


@pytest.mark.parametrize("dtype,C", [("bf16", 128), ("f32", 24), ("bf16", 33)])
def test_natural_order_and_position_base(dtype, C):
    """options of the _ex entry points: ascending flat order, positions offset by a base, with every anchor rule"""
    X = corr_clip(6, 5, 7, C, seed=300 + C, dtype=dtype)
    for mode, frame in ((0, 0), (1, 0), (2, 0), (3, 3)):
        for order, base in ((1, 0), (0, 777), (1, 12345)):
            rep = check_clip(X, 1, 0.6, anchor_mode=mode, anchor_frame=frame, order=order, pos_base=base)
            assert rep["count"] > 35


def test_misaligned_base_pointer_takes_scalar_path():
    F, H, W, C = 3, 4, 5, 64
    X = corr_clip(F, H, W, C, seed=12, dtype="bf16")
    buf = torch.zeros(F * H * W * C + 8, dtype=torch.bfloat16, device="cuda")
    view = buf[1:1 + F * H * W * C].view(F, H, W, C)          # 2 bytes off a 16-byte boundary
    view.copy_(to_device(X))
    assert view.data_ptr() % 16 != 0
    R = O.compress(X, 1, 0.7)
    toks, cnt, pos = P.ttf_compress(view, 1, 0.7)
    torch.cuda.synchronize()
    L = int(cnt.item())
    forced = R
    assert L == forced.count
    assert (pos[:L].cpu().numpy() == forced.pos).all() and (to_bits(toks[:L]) == forced.tokens).all()


@pytest.mark.parametrize("name", ["vl2b", "vl2b_cal", "vl8b", "vl8b_cal"])
def test_paper_shaped_clips(name):
    s = clips.CONFIGS[name]
    X = clips.make_clip(s)
    ts = (0.60, 0.70, 0.80) if name.startswith("vl8b") else (s.t,)
    for t in ts:
        rep = check_clip(X, s.r, t)
        print(name, t, rep)
    if name.endswith("_cal"):
        assert abs(check_clip(X, s.r, 0.70)["rho"] - 0.67) < 0.02


@pytest.mark.parametrize("name", ["wide", "wide_cal"])
def test_wide_search_clip(name):
    """F=64, 32x32, r=2: the configuration text word for word (shifts in {-2..2}^2, outlier tokens) and the
    anchored variant the throughput runs use"""
    s = clips.CONFIGS[name]
    rep = check_clip(clips.make_clip(s), s.r, s.t)
    print(name, rep)


def test_long_clip_batch_on_streams():
    """clips of the long-video batch processed concurrently on separate streams"""
    s = clips.CONFIGS["long_cal"]
    n = 3
    Xs = [clips.make_clip(s, s.seed + j) for j in range(n)]
    Rs = [O.compress(X, s.r, s.t) for X in Xs]
    Xd = [to_device(X) for X in Xs]
    streams = [torch.cuda.Stream() for _ in range(n)]
    outs = []
    torch.cuda.synchronize()
    for rep in range(2):
        outs = []
        for X, st in zip(Xd, streams):
            with torch.cuda.stream(st):
                outs.append(P.ttf_compress(X, s.r, s.t, stream=st))
    torch.cuda.synchronize()
    for X, R, (toks, cnt, pos) in zip(Xs, Rs, outs):
        q = P.ttf_query(to_device(X), s.r, s.t)
        keep = q["keep"].cpu().numpy()
        forced = O.compress(X, s.r, s.t, anchor_frame=int(q["anchor"].item()), forced_keep=keep)
        in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(s.t)) < 1e-4
        assert not ((keep != R.keep) & ~in_band).any()
        L = int(cnt.item())
        assert L == forced.count
        assert (pos[:L].cpu().numpy() == forced.pos).all() and (to_bits(toks[:L]) == forced.tokens).all()


def test_deterministic_and_canary():
    s = clips.CONFIGS["vl2b_cal"]
    X = to_device(clips.make_clip(s))
    n = s.tokens
    runs = []
    for _ in range(3):
        toks = torch.full((n + 4, s.C), -7.0, dtype=torch.bfloat16, device="cuda")
        pos = torch.full((n + 4, 3), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((2,), -7, dtype=torch.int32, device="cuda")
        P.ttf_compress(X, s.r, s.t, out_tokens=toks, out_count=cnt, out_pos_thw=pos)
        torch.cuda.synchronize()
        L = int(cnt[0].item())
        assert int(cnt[1].item()) == -7
        assert (toks[L:] == -7.0).all() and (pos[L:] == -7).all()       # nothing written past L'
        runs.append((L, to_bits(toks[:L]).copy(), pos[:L].cpu().numpy().copy()))
    for L, tk, ps in runs[1:]:
        assert L == runs[0][0] and (tk == runs[0][1]).all() and (ps == runs[0][2]).all()
    qa = P.ttf_query(X, s.r, s.t)
    qb = P.ttf_query(X, s.r, s.t)
    torch.cuda.synchronize()
    for k in qa:
        assert torch.equal(qa[k], qb[k]), k


def test_caller_workspace_and_host_entry_point():
    s = clips.CONFIGS["tiny_cal"]
    Xn = clips.make_clip(s)
    X = to_device(Xn)
    nbytes = P.ttf_workspace_bytes(s.F, s.H, s.W, s.C, s.r, P.TTF_DTYPE_F32)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    a = P.ttf_compress(X, s.r, s.t, workspace=ws)
    b = P.ttf_compress(X, s.r, s.t)
    torch.cuda.synchronize()
    L = int(a[1].item())
    assert L == int(b[1].item()) and torch.equal(a[0][:L], b[0][:L]) and torch.equal(a[2][:L], b[2][:L])
    with pytest.raises(P.TTFError):
        P.ttf_compress(X, s.r, s.t, workspace=ws[: nbytes // 2])
    host = torch.from_numpy(Xn).pin_memory()
    toks, Lh, pos = P.ttf_compress_host(host, s.r, s.t)
    assert Lh == L and torch.equal(toks, a[0][:L].cpu()) and torch.equal(pos, a[2][:L].cpu())


def test_many_frames_uses_prescanned_prefix():
    # more frames than the gather kernel scans in shared memory
    F, H, W, C = 2100, 2, 2, 8
    X = corr_clip(F, H, W, C, seed=77, dtype="bf16", sigma=0.8)
    rep = check_clip(X, 1, 0.7)
    assert 4 < rep["count"] < F * 4


@pytest.mark.parametrize("dtype,C", [("bf16", 256), ("f32", 40)])
def test_non_finite_tokens_are_kept(dtype, C):
    """a NaN similarity keeps the token (the gate is evaluated as !(s_hat > t)); other tokens are unaffected"""
    F, H, W = 5, 6, 7
    N = H * W
    Xf = corr_clip(F, H, W, C, seed=91, dtype="f32")
    Xf[0, 1, 1, 5] = np.nan            # a source token
    Xf[2, 3, 3, 7] = np.nan            # a token of the anchor frame (frame 2 below)
    Xf[4, 2, 2, 0] = np.inf            # an infinite source token: its norm is infinite, the cosine NaN
    X = Xf if dtype == "f32" else clips.f32_to_bf16_bits(Xf)
    Xd = to_device(X)
    R = O.compress(X, 1, 0.6, anchor_frame=2)
    q = P.ttf_query(Xd, 1, 0.6, anchor_mode=3, anchor_frame=2)
    toks, cnt, pos = P.ttf_compress(Xd, 1, 0.6, anchor_mode=3, anchor_frame=2)
    torch.cuda.synchronize()
    keep = q["keep"].cpu().numpy()
    sim = q["best_sim"].cpu().numpy()
    assert keep[0 * N + 1 * W + 1] == 1 and keep[4 * N + 2 * W + 2] == 1
    assert np.isnan(sim[0 * N + 1 * W + 1]) and np.isnan(R.s_hat[0 * N + 1 * W + 1])
    finite = np.isfinite(R.s_hat)
    assert (np.isfinite(sim) == finite).all()
    assert np.abs(sim[finite] - R.s_hat[finite]).max() <= 2e-5
    in_band = finite & (np.abs(R.s_hat.astype(np.float32) - np.float32(0.6)) < 1e-4)
    assert not ((keep != R.keep) & ~in_band).any()
    forced = O.compress(X, 1, 0.6, anchor_frame=2, forced_keep=keep)
    L = int(cnt.item())
    assert L == forced.count and (pos[:L].cpu().numpy() == forced.pos).all()
    bits = (lambda v: v.view(np.uint32)) if dtype == "f32" else (lambda v: v)     # NaN rows compare by bit pattern
    assert (bits(to_bits(toks[:L])) == bits(np.ascontiguousarray(forced.tokens))).all()
