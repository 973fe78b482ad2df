"""GPU parity of the extensions from the paper's Discussion: streaming segment (D3), TTF-R restoration (D4) and
the best-similarity histogram (D1), each against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips
import paper_2605_07355_b200 as P
from tests.parity import to_device, to_bits
from tests.test_gpu_parity import corr_clip

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,dtype", [((4, 6, 5, 64), "bf16"), ((5, 3, 7, 40), "f32"), ((3, 4, 4, 33), "bf16"),
                                         ((32, 16, 16, 256), "bf16")])
def test_restore_matches_oracle(shape, dtype):
    F, H, W, C = shape
    N = H * W
    X = corr_clip(F, H, W, C, seed=91 + C, dtype=dtype)
    Xd = to_device(X)
    q = P.ttf_query(Xd, 1, 0.7)
    toks, cnt, pos = P.ttf_compress(Xd, 1, 0.7)
    torch.cuda.synchronize()
    L = int(cnt.item())
    full, idx = P.ttf_restore(toks[:L].contiguous(), F, H, W, q["anchor"], q["keep"], q["dst"])
    torch.cuda.synchronize()
    keep, dst, a = q["keep"].cpu().numpy(), q["dst"].cpu().numpy(), int(q["anchor"].item())
    ref_full, ref_idx = O.restore(to_bits(toks[:L]), keep, dst, F, N, a)
    assert (idx.cpu().numpy() == ref_idx).all()
    assert (to_bits(full) == ref_full).all()
    Xf = X.reshape(F * N, C)
    assert (to_bits(full)[keep.astype(bool)] == Xf[keep.astype(bool)]).all()
    # a payload that is not the tokens (e.g. hidden states), odd row size
    payload = torch.arange(L * 3, dtype=torch.float32, device="cuda").reshape(L, 3)
    full2, _ = P.ttf_restore(payload, F, H, W, q["anchor"], q["keep"], q["dst"])
    assert (full2.cpu().numpy() == payload.cpu().numpy()[ref_idx]).all()


@pytest.mark.parametrize("offset", [0, 1, 3, 13])
def test_restore_flag_counts_from_any_alignment(offset):
    """The index step counts the flags of earlier frames 16 per load between an unaligned head and tail: odd N,
    many frames, the flag array at every kind of offset from a 16-byte boundary, non-0/1 flag values."""
    F, H, W, C = 45, 5, 7, 16
    N = H * W
    X = corr_clip(F, H, W, C, seed=123, dtype="f32")
    q = P.ttf_query(to_device(X), 1, 0.6)
    toks, cnt, _ = P.ttf_compress(to_device(X), 1, 0.6)
    torch.cuda.synchronize()
    L = int(cnt.item())
    buf = torch.zeros(F * N + 32, dtype=torch.uint8, device="cuda")
    keep_view = buf[offset:offset + F * N]
    keep_view.copy_(q["keep"].view(-1) * 255)                        # any non-zero value is a set flag
    full, idx = P.ttf_restore(toks[:L].contiguous(), F, H, W, q["anchor"], keep_view, q["dst"])
    torch.cuda.synchronize()
    keep, dst, a = q["keep"].cpu().numpy(), q["dst"].cpu().numpy(), int(q["anchor"].item())
    ref_full, ref_idx = O.restore(to_bits(toks[:L]), keep, dst, F, N, a)
    assert (idx.cpu().numpy() == ref_idx).all()
    assert (to_bits(full) == ref_full).all()


@pytest.mark.parametrize("bins", [1, 16, 100])
def test_histogram_matches_oracle(bins):
    s = clips.CONFIGS["vl2b_cal"]
    Xd = to_device(clips.make_clip(s))
    q = P.ttf_query(Xd, s.r, s.t)
    hist = P.ttf_sim_histogram(q["best_sim"], q["anchor"], s.F, s.H, s.W, bins)
    torch.cuda.synchronize()
    sim = q["best_sim"].cpu().numpy()
    a = int(q["anchor"].item())
    ref = O.sim_histogram(sim, s.F, s.N, a, bins).astype(np.int64)
    got = hist.cpu().numpy().view(np.uint32).astype(np.int64)
    assert got.sum() == (s.F - 1) * s.N
    # the oracle bins in double, the kernel in fp32: a similarity within 1e-6 of a bin edge may land on either
    # side of it.  Such values are counted per edge; every other value must be in the oracle's bin.
    src = np.delete(sim.reshape(s.F, s.N), a, axis=0).ravel().astype(np.float64)
    x = (src + 1.0) / 2.0 * bins
    e = np.rint(x)
    near = (np.abs(x - e) * 2.0 / bins < 1e-6) & (e >= 1) & (e <= bins - 1)
    slack = np.bincount(e[near].astype(np.int64), minlength=bins + 1)      # slack[j]: values near the edge below bin j
    print(f"bins={bins}: {int(near.sum())} similarities within 1e-6 of a bin edge")
    assert (np.abs(got - ref) <= slack[:bins] + slack[1:bins + 1]).all()


@pytest.mark.parametrize("shape,dtype", [((4, 6, 5, 64), "bf16"), ((5, 3, 7, 40), "f32"), ((9, 16, 16, 512), "bf16")])
def test_segment_matches_oracle(shape, dtype):
    F, H, W, C = shape
    N = H * W
    X = corr_clip(F, H, W, C, seed=95 + C, dtype=dtype)
    Xd = to_device(X)
    toks, cnt, pos = P.ttf_compress_segment(Xd, 1, 0.7, frame_base=17)
    q = P.ttf_query(Xd, 1, 0.7, anchor_mode=P.TTF_ANCHOR_FIRST)
    torch.cuda.synchronize()
    keep = q["keep"].cpu().numpy()
    R = O.compress(X, 1, 0.7, anchor_frame=0)
    in_band = np.abs(R.s_hat.astype(np.float32) - np.float32(0.7)) < 1e-4
    assert not ((keep != R.keep) & ~in_band).any()
    ref_t, ref_p, ref_P = O.compress_segment(X, 1, 0.7, 17, forced_keep=keep)
    Pn = int(cnt.item())
    assert Pn == ref_P == int(keep.sum()) - N
    assert (pos[:Pn].cpu().numpy() == ref_p).all() and (to_bits(toks[:Pn]) == ref_t).all()
    assert Pn == 0 or int(pos[:Pn, 0].min().item()) >= 17


@pytest.mark.parametrize("name,band", [("tiny_cal", 1e-2), ("vl2b_cal", 1e-3)])
def test_stats_match_oracle(name, band):
    """ttf_stats on the GPU's own query outputs equals the oracle's counts exactly (integers), rho follows."""
    s = clips.CONFIGS[name]
    X = clips.make_clip(s)
    F, H, W = s.F, s.H, s.W
    N = H * W
    q = P.ttf_query(to_device(X), s.r, s.t)
    st = P.ttf_stats(q["best_sim"], q["keep"], q["anchor"], F, H, W, s.t, band)
    torch.cuda.synchronize()
    a = int(q["anchor"].item())
    Pn, fused, in_band, rho = O.stats(q["best_sim"].cpu().numpy(), q["keep"].cpu().numpy(), F, N, a, s.t, band)
    assert st.tolist() == [Pn, fused, in_band]
    assert in_band > 0 and Pn + fused == (F - 1) * N
    assert P.ttf_reduction_ratio(int(st[0]), F, N) == rho
    toks, cnt, pos = P.ttf_compress(to_device(X), s.r, s.t)
    assert int(cnt.item()) == N + Pn                                  # L' = N + P (Eq. Lpre)
