"""Pins for the CPU oracle: each test checks it against something the paper or the mathematics fixes
(invariants, closed forms, special cases that reduce to a numpy / scipy routine, brute force on tiny grids),
never against the CUDA path.  A dropped term, a wrong sign, a transposed index or a wrong border rule in
oracle/ttf_oracle.c fails at least one of them."""
import numpy as np
import pytest
from scipy.spatial.distance import cdist

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips


def rand_clip(F, H, W, C, seed, dtype="f32"):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((F, H, W, C)).astype(np.float32)
    return X if dtype == "f32" else clips.f32_to_bf16_bits(X)


def corr_clip(F, H, W, C, seed, sigma=0.5):
    """frames = one scene + noise, so similarities spread around typical thresholds"""
    rng = np.random.default_rng(seed)
    base = rng.standard_normal((H, W, C))
    X = base[None] + sigma * rng.standard_normal((F, H, W, C)) * np.exp(0.7 * rng.standard_normal((F, H, W, 1)))
    return X.astype(np.float32)


# ---- Eq. (gating), Eq. (mask), Eq. (xprime_stack): counting invariants -------------------------------------
@pytest.mark.parametrize("shape", [(4, 8, 8, 64), (5, 3, 7, 33), (2, 1, 5, 8), (3, 6, 1, 16), (1, 4, 4, 8)])
@pytest.mark.parametrize("r", [0, 1, 2])
def test_kept_plus_fused_is_FN(shape, r):
    F, H, W, C = shape
    N = H * W
    X = corr_clip(F, H, W, C, seed=11 + r)
    R = O.compress(X, r, 0.70)
    fused = int((R.keep == 0).sum())
    P = int(R.keep.sum()) - N
    assert R.count == N + P
    assert R.count + fused == F * N
    assert int(R.fuse_cnt.sum()) == fused
    assert R.keep.reshape(F, N)[R.anchor].all()
    assert abs(R.rho - (1.0 - (N + P) / (F * N))) < 1e-15
    assert R.tokens.shape == (R.count, C) and R.pos.shape == (R.count, 3)


def test_threshold_extremes():
    X = corr_clip(4, 5, 6, 32, seed=3)
    F, N = 4, 30
    assert O.compress(X, 1, 1.001).count == F * N          # cosine never exceeds 1: nothing is fused
    assert O.compress(X, 1, -1.001).count == N             # cosine always above -1: every source token fused
    R = O.compress(X, 1, -1.001)
    assert (R.keep.reshape(F, N).sum(axis=1) == np.where(np.arange(F) == R.anchor, N, 0)).all()


def test_gate_is_strict_at_equality():
    # identical frames: every best match has cosine exactly 1 (in fp32); Eq. (gating) keeps s_hat <= t
    X = np.repeat(rand_clip(1, 4, 4, 16, seed=5), 3, axis=0)
    assert O.compress(X, 1, 1.0).count == 3 * 16
    assert O.compress(X, 1, np.nextafter(np.float32(1.0), np.float32(0.0))).count == 16


def test_identical_frames_collapse_to_anchor():
    X = np.repeat(rand_clip(1, 6, 5, 24, seed=7), 4, axis=0)
    R = O.compress(X, 1, 0.70)
    N = 30
    assert R.anchor == 0                                   # all frame cosines tie: the lowest frame wins
    assert R.count == N
    assert (R.dst.reshape(4, N) == np.arange(N)[None]).all()
    assert np.allclose(R.s_hat, 1.0, atol=1e-12)
    assert (R.tokens == X[0].reshape(N, -1)).all()
    assert (R.fuse_cnt == 3).all()


# ---- scale invariance of the cosine ----------------------------------------------------------------------
def test_uniform_power_of_two_scale_changes_nothing():
    X = corr_clip(4, 6, 6, 32, seed=9)
    R1, R2 = O.compress(X, 1, 0.70), O.compress(X * np.float32(8.0), 1, 0.70)
    assert R1.anchor == R2.anchor and R1.count == R2.count
    assert (R1.keep == R2.keep).all() and (R1.dst == R2.dst).all() and (R1.pos == R2.pos).all()
    assert (R1.s_hat == R2.s_hat).all()                    # exact: powers of two commute with rounding
    assert (R2.tokens == R1.tokens * np.float32(8.0)).all()


def test_per_token_scale_leaves_matching_unchanged():
    X = corr_clip(4, 6, 6, 32, seed=10).astype(np.float64)
    rng = np.random.default_rng(1)
    scale = np.exp(0.5 * rng.standard_normal((4, 6, 6, 1)))
    Xs = (X * scale).astype(np.float32)
    # the rescaled clip is re-rounded to fp32, so compare in tolerance; the anchor is pinned because the
    # anchor rule averages raw tokens and is not scale-free
    a = 2
    s1, d1, _ = O.match(X.astype(np.float32), 1, a)
    s2, d2, _ = O.match(Xs, 1, a)
    assert np.abs(s1 - s2).max() < 1e-6
    assert (d1 == d2).all()


# ---- Eq. (pi): a radius that covers the grid is an all-pairs search ------------------------------------------
@pytest.mark.parametrize("H,W", [(4, 4), (3, 6), (1, 5), (6, 2)])
def test_full_radius_equals_all_pairs_search_scipy(H, W):
    F, C, a = 3, 20, 1
    X = corr_clip(F, H, W, C, seed=H * 10 + W)
    N = H * W
    s_hat, dst, _ = O.match(X, max(H, W) - 1, a)
    Xd = X.reshape(F, N, C).astype(np.float64)
    for k in range(F):
        if k == a:
            continue
        sim = 1.0 - cdist(Xd[k], Xd[a], metric="cosine")          # [N source, N anchor]
        assert np.abs(sim.max(axis=1) - s_hat.reshape(F, N)[k]).max() < 1e-12
        assert (sim.argmax(axis=1) == dst.reshape(F, N)[k]).all()
    g_s, g_d = O.match_global(X, a)
    assert np.abs(g_s - s_hat).max() < 1e-15 and (g_d == dst).all()


@pytest.mark.parametrize("H,W,r", [(5, 7, 1), (4, 4, 2), (1, 6, 1), (6, 1, 2), (2, 2, 1), (1, 1, 1), (3, 3, 0)])
def test_window_is_grid_intersection(H, W, r):
    """clip-and-mask (Eq. pi plus the duplicate rule) must equal a search over the in-grid window"""
    F, C, a = 3, 12, 0
    X = corr_clip(F, H, W, C, seed=100 + H * W + r)
    N = H * W
    s_hat, dst, second = O.match(X, r, a)
    Xd = X.reshape(F, N, C).astype(np.float64)
    for k in range(1, F):
        sim = 1.0 - cdist(Xd[k], Xd[a], metric="cosine")
        for i in range(N):
            y, x = divmod(i, W)
            cand = [yy * W + xx for yy in range(max(0, y - r), min(H, y + r + 1))
                    for xx in range(max(0, x - r), min(W, x + r + 1))]
            vals = sim[i, cand]
            f = k * N + i
            assert abs(vals.max() - s_hat[f]) < 1e-12
            assert cand[int(vals.argmax())] == dst[f]
            yd, xd = divmod(int(dst[f]), W)
            assert abs(yd - y) <= r and abs(xd - x) <= r
            if len(cand) > 1:
                assert abs(np.sort(vals)[-2] - second[f]) < 1e-12
            else:
                assert second[f] == -np.inf


# ---- planted shift: closed form for dst -------------------------------------------------------------------
@pytest.mark.parametrize("dy,dx", [(0, 0), (1, 0), (0, -1), (-1, 1), (1, 1)])
def test_planted_shift_closed_form(dy, dx):
    H, W, C = 6, 7, 48
    base = rand_clip(1, H, W, C, seed=21)[0]
    X = np.stack([base, np.roll(base, (dy, dx), axis=(0, 1))])   # frame 1, cell (y,x) = base cell (y-dy, x-dx)
    s_hat, dst, _ = O.match(X, 1, a=0)
    for y in range(H):
        for x in range(W):
            f = H * W + y * W + x
            ys, xs = y - dy, x - dx
            if 0 <= ys < H and 0 <= xs < W:
                assert dst[f] == ys * W + xs
                assert abs(s_hat[f] - 1.0) < 1e-12
            else:                                                  # wrapped content: not in the window
                assert s_hat[f] < 0.9
    R = O.compress(X, 1, 0.70, anchor_frame=0)
    wrapped = H * W - (H - abs(dy)) * (W - abs(dx))
    assert R.count == H * W + wrapped


# ---- Eq. (auto_anchor) ------------------------------------------------------------------------------------
def test_anchor_frame_equal_to_clip_mean_wins_with_cosine_one():
    F, H, W, C = 5, 3, 4, 16
    X = rand_clip(F, H, W, C, seed=31).astype(np.float64)
    j = 3
    others = [k for k in range(F) if k != j]
    X[j] = X[others].mean(axis=0)          # then the global mean token equals frame j's mean token
    a, cos = O.anchor(X.astype(np.float32))
    assert a == j
    assert abs(cos[j] - 1.0) < 1e-6        # inputs are re-rounded to fp32
    assert (np.delete(cos, j) < 0.999).all()


def test_anchor_cosines_match_numpy_and_ignore_mean_normalisation():
    F, H, W, C = 6, 4, 5, 40
    X = corr_clip(F, H, W, C, seed=33)
    a, cos = O.anchor(X)
    Xd = X.reshape(F, H * W, C).astype(np.float64)
    m = Xd.sum(axis=1)                     # un-normalised sums: 1/N and 1/(FN) cancel in the cosine
    g = m.sum(axis=0)
    ref = 1.0 - cdist(m, g[None], metric="cosine")[:, 0]
    assert np.abs(ref - cos).max() < 1e-12
    assert a == int(ref.argmax())


def test_single_frame_clip():
    X = rand_clip(1, 3, 3, 8, seed=2)
    R = O.compress(X, 1, 0.70)
    assert R.anchor == 0 and R.count == 9 and (R.index == np.arange(9)).all()


# ---- Eq. (compress_pos): survivors keep their coordinates, anchor rows first ------------------------------
@pytest.mark.parametrize("anchor_frame", [None, 0, 2, 3])
def test_positions_and_order(anchor_frame):
    F, H, W, C = 4, 5, 6, 32
    N = H * W
    X = corr_clip(F, H, W, C, seed=41)
    R = O.compress(X, 1, 0.70, anchor_frame=anchor_frame)
    a = R.anchor if anchor_frame is None else anchor_frame
    assert (R.index[:N] == a * N + np.arange(N)).all()
    src = R.index[N:]
    assert (np.diff(src) > 0).all() and not np.isin(src // N, [a]).any()
    assert set(src.tolist()) == set(np.flatnonzero(R.keep.reshape(F, N) & (np.arange(F)[:, None] != a)).tolist())
    k, i = R.index // N, R.index % N
    assert (R.pos[:, 0] == k).all() and (R.pos[:, 1] == i // W).all() and (R.pos[:, 2] == i % W).all()
    assert (R.tokens == X.reshape(F * N, C)[R.index]).all()
    assert 0 < len(src) < (F - 1) * N       # the case exercises both outcomes of the gate


def test_natural_order_and_position_base():
    """the other reading of "ordered index set" (ascending flat index) and a constant position offset"""
    F, H, W, C = 5, 4, 6, 16
    N = H * W
    X = corr_clip(F, H, W, C, seed=71)
    for a in (0, 2, 4):
        R = O.compress(X, 1, 0.6, anchor_frame=a)
        Rn = O.compress(X, 1, 0.6, anchor_frame=a, natural=True)
        assert Rn.count == R.count and (Rn.keep == R.keep).all()
        assert (np.diff(Rn.index) > 0).all()                                 # strictly ascending flat index
        assert sorted(Rn.index.tolist()) == sorted(R.index.tolist())         # the same tokens, another order
        assert (Rn.index == np.flatnonzero(R.keep)).all()                    # = every retained token, numpy's own scan
        assert (Rn.tokens == X.reshape(F * N, C)[Rn.index]).all()
        k, i = Rn.index // N, Rn.index % N
        assert (Rn.pos == np.stack([k, i // W, i % W], axis=1)).all()
        if a == 0:                                                           # anchor first = natural when a = 0
            assert (Rn.index == R.index).all() and (Rn.pos == R.pos).all() and (Rn.tokens == R.tokens).all()
        Rb = O.compress(X, 1, 0.6, anchor_frame=a, pos_base=1000)
        assert (Rb.pos == R.pos + 1000).all() and (Rb.tokens == R.tokens).all() and (Rb.index == R.index).all()


def test_forced_keep_drives_compaction():
    X = corr_clip(3, 4, 4, 16, seed=43)
    R = O.compress(X, 1, 0.70)
    forced = R.keep.copy()
    flip = int(np.flatnonzero(forced == 0)[0])
    forced[flip] = 1
    R2 = O.compress(X, 1, 0.70, forced_keep=forced)
    assert R2.count == R.count + 1 and flip in R2.index.tolist()


# ---- monotonicity -----------------------------------------------------------------------------------------
def test_rho_monotone_in_t_and_r():
    X = corr_clip(5, 6, 6, 32, seed=51)
    a = 2
    rho_t = [O.compress(X, 1, t, anchor_frame=a).rho for t in (0.3, 0.5, 0.6, 0.7, 0.8, 0.9)]
    assert all(x >= y for x, y in zip(rho_t, rho_t[1:])) and rho_t[0] > rho_t[-1]
    s = [O.match(X, r, a)[0] for r in (0, 1, 2, 5)]
    for lo, hi in zip(s, s[1:]):
        assert (hi >= lo).all()             # a larger window can only raise the best similarity
    rho_r = [O.compress(X, r, 0.7, anchor_frame=a).rho for r in (0, 1, 2, 5)]
    assert all(x <= y for x, y in zip(rho_r, rho_r[1:]))


# ---- degenerate tokens ------------------------------------------------------------------------------------
def test_zero_token_has_similarity_zero():
    X = corr_clip(3, 4, 4, 16, seed=61)
    X[1, 2, 2] = 0.0
    f = 1 * 16 + 2 * 4 + 2
    s_hat, _, _ = O.match(X, 1, 0)
    assert s_hat[f] == 0.0
    assert O.compress(X, 1, 0.0, anchor_frame=0).keep[f] == 1      # 0 <= t keeps
    assert O.compress(X, 1, -0.5, anchor_frame=0).keep[f] == 0


def test_exact_tie_takes_lowest_anchor_index():
    H, W, C = 3, 3, 8
    X = np.ones((2, H, W, C), dtype=np.float32)                     # all candidates tie at cosine 1
    _, dst, _ = O.match(X, 1, 0)
    for i in range(H * W):
        y, x = divmod(i, W)
        assert dst[H * W + i] == max(0, y - 1) * W + max(0, x - 1)


# ---- bf16 inputs are widened exactly ----------------------------------------------------------------------
def test_bf16_bits_equal_their_fp32_widening():
    Xb = rand_clip(3, 4, 4, 16, seed=71, dtype="bf16")
    Xf = clips.bf16_bits_to_f32(Xb)
    Rb, Rf = O.compress(Xb, 1, 0.70), O.compress(Xf, 1, 0.70)
    assert (Rb.s_hat == Rf.s_hat).all() and (Rb.keep == Rf.keep).all() and Rb.anchor == Rf.anchor
    assert Rb.tokens.dtype == np.uint16 and (clips.bf16_bits_to_f32(Rb.tokens) == Rf.tokens).all()


# ---- Eqs. (Lpre), (decode_pos) ----------------------------------------------------------------------------
def test_decode_alignment():
    assert O.decode_pos(2703, 57, 0) == 2703 + 57
    assert O.decode_pos(2703, 57, 9) == 2703 + 57 + 9


# ---- Discussion D4: restoration through dst ----------------------------------------------------------------
def test_restore_inverts_compaction():
    F, H, W, C = 4, 5, 4, 16
    N = H * W
    X = corr_clip(F, H, W, C, seed=81)
    R = O.compress(X, 1, 0.70)
    full, idx = O.restore(R.tokens, R.keep, R.dst, F, N, R.anchor)
    Xf = X.reshape(F * N, C)
    kept = R.keep.astype(bool)
    assert (full[kept] == Xf[kept]).all()                               # retained tokens come back unchanged
    fused = np.flatnonzero(~kept)
    assert (full[fused] == Xf[R.anchor * N + R.dst[fused]]).all()       # fused ones become their anchor match
    assert (idx[fused] == R.dst[fused]).all() and (idx[R.anchor * N:(R.anchor + 1) * N] == np.arange(N)).all()
    assert sorted(idx[kept].tolist()) == list(range(R.count))           # a bijection onto the compressed rows
    # nothing fused: restoration is the identity
    R2 = O.compress(X, 1, 1.5)
    full2, idx2 = O.restore(R2.tokens, R2.keep, R2.dst, F, N, R2.anchor)
    assert (full2 == Xf).all()
    # everything fused with identical frames: every frame becomes the anchor frame
    Xi = np.repeat(X[:1], 3, axis=0)
    R3 = O.compress(Xi, 1, 0.7)
    full3, _ = O.restore(R3.tokens, R3.keep, R3.dst, 3, N, R3.anchor)
    assert (full3.reshape(3, N, C) == Xi.reshape(3, N, C)).all()


def test_fuse_count_is_a_bincount_of_the_fused_destinations():
    """the bookkeeping of identity replacement written with numpy's own counting routine"""
    for seed, r, t in [(91, 1, 0.70), (92, 2, 0.5), (93, 0, 0.3)]:
        F, H, W, C = 6, 5, 7, 32
        N = H * W
        R = O.compress(corr_clip(F, H, W, C, seed=seed), r, t)
        src = np.ones(F * N, dtype=bool)
        src[R.anchor * N:(R.anchor + 1) * N] = False
        fused = src & (R.keep == 0)
        assert fused.any()
        assert (R.fuse_cnt == np.bincount(R.dst[fused], minlength=N)).all()
        assert (O.fuse_count(R.keep, R.dst, F, N, R.anchor) == R.fuse_cnt).all()


# ---- Discussion D1: distribution of the best similarities ---------------------------------------------------
@pytest.mark.parametrize("bins", [1, 7, 64, 200])
def test_sim_histogram_matches_numpy(bins):
    F, H, W, C = 5, 6, 5, 24
    N = H * W
    X = corr_clip(F, H, W, C, seed=83)
    R = O.compress(X, 1, 0.70)
    s = R.s_hat.astype(np.float32)
    h = O.sim_histogram(s, F, N, R.anchor, bins)
    src = np.delete(s.reshape(F, N), R.anchor, axis=0).ravel()
    ref, _ = np.histogram(src.astype(np.float64), bins=bins, range=(-1.0, 1.0))
    assert h.sum() == (F - 1) * N
    # numpy's bins are half-open like the definition except that its last bin is closed, which the clamp reproduces
    assert (h.astype(np.int64) == ref).all()
    # values exactly on bin edges, where a wrong rounding direction or a wrong clamp would show
    edges = np.array([-1.0, -0.5, 0.0, 0.25, 0.5, 1.0, 1.5, -1.5], dtype=np.float32)
    he = O.sim_histogram(np.concatenate([np.ones(8, np.float32), edges]), 2, 8, 0, 4)      # frame 0 is the anchor
    # four bins of width 0.5: {-1.5 (clamped), -1} | {-0.5} | {0, 0.25} | {0.5, 1 (closed end), 1.5 (clamped)}
    assert he.tolist() == [2, 1, 2, 3]
    s2 = s.copy(); s2[N * ((R.anchor + 1) % F)] = np.nan
    assert O.sim_histogram(s2, F, N, R.anchor, bins).sum() == (F - 1) * N - 1


# ---- Discussion D3: streaming segment with a rolling anchor ---------------------------------------------------
def test_segment_emits_only_new_preserved_tokens():
    F, H, W, C = 4, 4, 5, 16
    N = H * W
    X = corr_clip(F, H, W, C, seed=85)
    toks, pos, P = O.compress_segment(X, 1, 0.70, frame_base=9)
    R = O.compress(X, 1, 0.70, anchor_frame=0)
    assert P == R.count - N and (toks == R.tokens[N:]).all()
    assert (pos[:, 0] == R.pos[N:, 0] + 8).all() and (pos[:, 1:] == R.pos[N:, 1:]).all()
    assert pos[:, 0].min() >= 9                                          # frame 1 of the segment is video frame 9
    t_all, p_all, P_all = O.compress_segment(X, 1, 1.5, frame_base=0)    # nothing fused: all new frames, in order
    assert P_all == (F - 1) * N and (t_all == X[1:].reshape(-1, C)).all()
    assert O.compress_segment(np.repeat(X[:1], 3, axis=0), 1, 0.7, 5)[2] == 0


# ---- mean fusion (the averaging alternative that Sec. 3, Threshold Gating, rules out; optional mode only) --------
def test_mean_fuse_hand_example():
    # F = 2 frames, N = 2 cells, C = 1; frame 0 is the anchor.  Both source tokens are fused into cell 0.
    X = np.array([[[[1.0], [10.0]]], [[[3.0], [5.0]]]], np.float32)           # [F=2, H=1, W=2, C=1]
    keep = np.array([1, 1, 0, 0], np.uint8)
    dst = np.array([0, 1, 0, 0], np.int32)
    out = O.fuse_mean(X, keep, dst, 0)
    assert out.tolist() == [[3.0], [10.0]]                                    # (1 + 3 + 5) / 3 and 10 / 1
    keep[3] = 1                                                               # a retained token contributes nothing
    assert O.fuse_mean(X, keep, dst, 0).tolist() == [[2.0], [10.0]]
    dst[2] = 1                                                                # ... and dst picks the receiving cell
    assert O.fuse_mean(X, keep, dst, 0).tolist() == [[1.0], [6.5]]


def test_mean_fuse_without_fusion_and_with_identical_frames_is_the_anchor_frame():
    X = corr_clip(4, 5, 4, 24, seed=41)
    R = O.compress(X, 1, 2.0)                                                 # t > 1: nothing is fused
    assert (O.fuse_mean(X, R.keep, R.dst, R.anchor) == X[R.anchor].reshape(20, 24).astype(np.float64)).all()
    Y = np.repeat(X[:1], 5, axis=0)                                           # identical frames: every mean is the row
    R = O.compress(Y, 1, 0.7)
    assert R.count == 20
    assert (O.fuse_mean(Y, R.keep, R.dst, R.anchor) == Y[0].reshape(20, 24).astype(np.float64)).all()


@pytest.mark.parametrize("seed,r", [(51, 0), (52, 1), (53, 2)])
def test_mean_fuse_conserves_the_absorbed_mass_and_matches_numpy(seed, r):
    F, H, W, C = 6, 5, 6, 40
    N = H * W
    X = corr_clip(F, H, W, C, seed=seed)
    R = O.compress(X, r, 0.6)
    assert 0 < (R.keep == 0).sum() < (F - 1) * N
    out = O.fuse_mean(X, R.keep, R.dst, R.anchor)
    flat = X.reshape(F * N, C).astype(np.float64)
    fused = R.keep == 0
    # the size-weighted means add up to everything that was absorbed: the anchor frame plus the fused tokens
    total = (out * (1 + R.fuse_cnt)[:, None]).sum(axis=0)
    assert np.allclose(total, flat[R.anchor * N:(R.anchor + 1) * N].sum(axis=0) + flat[fused].sum(axis=0), rtol=0, atol=1e-9)
    # numpy's own scatter-add over the same (keep, dst)
    acc = flat[R.anchor * N:(R.anchor + 1) * N].copy()
    np.add.at(acc, R.dst[fused], flat[fused])
    assert np.allclose(out, acc / (1 + np.bincount(R.dst[fused], minlength=N))[:, None], rtol=0, atol=1e-12)


def test_bf16_rounding_helper_is_round_to_nearest_even():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(50000).astype(np.float32)
    u = x.view(np.uint32)
    rne = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    assert (O.round_to_bf16_bits(x.astype(np.float64)) == rne).all()
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -1.0 - 3 * 2.0 ** -8])
    assert O.round_to_bf16_bits(ties).tolist() == [0x3F80, 0x3F82, 0xBF82]


def test_stats_reduction_ratio_closed_forms_and_count_identity():
    """Sec. 3 (after Eq. Lpre): rho = 1 - (N + P) / (F N).  Identical frames fuse every source token: P = 0 and
    rho = 1 - 1/F exactly; a threshold nothing exceeds keeps everything: rho = 0; on a generic clip N + P equals the
    length of the compressed sequence the compaction step returns, and the band count equals a vectorised count."""
    rng = np.random.default_rng(5)
    F, H, W, C = 6, 3, 4, 16
    N = H * W
    frame = rng.standard_normal((H, W, C)).astype(np.float32)
    X = np.broadcast_to(frame, (F, H, W, C)).copy()
    R = O.compress(X, 1, 0.7)
    P, fused, band, rho = O.stats(R.s_hat.astype(np.float32), R.keep, F, N, R.anchor, 0.7, 1e-4)
    assert (P, fused) == (0, (F - 1) * N) and rho == 1.0 - 1.0 / F
    R = O.compress(X, 1, 2.0)
    P, fused, band, rho = O.stats(R.s_hat.astype(np.float32), R.keep, F, N, R.anchor, 2.0, 1e-4)
    assert (P, fused, band) == ((F - 1) * N, 0, 0) and rho == 0.0
    X = rng.standard_normal((F, H, W, C)).astype(np.float32) * 0.6 + frame
    R = O.compress(X, 1, 0.6)
    s32 = R.s_hat.astype(np.float32)
    P, fused, band, rho = O.stats(s32, R.keep, F, N, R.anchor, 0.6, 0.05)
    assert N + P == R.count and P + fused == (F - 1) * N and 0 < P < (F - 1) * N
    src = np.arange(F) != R.anchor
    want = int((np.abs(s32.reshape(F, N)[src].astype(np.float64) - float(np.float32(0.6))) < float(np.float32(0.05))).sum())
    assert band == want and band > 0
    assert abs(rho - (1.0 - R.count / (F * N))) < 1e-15
