"""Element-by-element comparison of the CUDA library (through its C ABI) with the CPU oracle.

Tolerances:
  * anchor index, dst, keep, fuse counts, L', positions, token rows: bit-exact, except
      - keep may differ only where the oracle's fp32-rounded similarity lies within BAND of t,
      - dst may differ only where the oracle's best and second-best similarity are within BAND;
    such tokens are counted and reported.  After these in-band decisions are accepted (the oracle re-runs its
    gate-to-compaction steps with the GPU's decisions forced), everything downstream must match exactly.
  * best similarity: |gpu - oracle| <= SIM_ATOL (fp32 accumulation of C products against fp64).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import ttf_oracle as O
import paper_2605_07355_b200 as P

BAND = 1e-4
SIM_ATOL = 2e-5
ANCHOR_MARGIN = 1e-5


def to_device(X: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy clip (float32, or uint16 bf16 bit patterns) -> torch tensor with the same bits"""
    if X.dtype == np.float32:
        return torch.from_numpy(np.ascontiguousarray(X)).to(device)
    return torch.from_numpy(np.ascontiguousarray(X).view(np.int16)).view(torch.bfloat16).to(device)


def to_bits(t: torch.Tensor) -> np.ndarray:
    """device tensor -> numpy with the same bits (bf16 -> uint16)"""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def check_clip(X: np.ndarray, r: int, t: float, *, stream=None, workspace=None, oracle=None,
               require_anchor=True, anchor_mode: int = 0, anchor_frame: int = 0, order: int = 0,
               pos_base: int = 0) -> dict:
    """Runs ttf_query and ttf_compress on X and compares with the oracle.  Returns a small report."""
    F, H, W, C = X.shape
    N = H * W
    fixed = {0: None, 1: 0, 2: F - 1, 3: anchor_frame}[anchor_mode]       # first / last / explicit anchors
    R = oracle if oracle is not None else O.compress(X, r, t, anchor_frame=fixed)
    Xd = to_device(X)

    kw = dict(stream=stream, workspace=workspace, anchor_mode=anchor_mode, anchor_frame=anchor_frame)
    q = P.ttf_query(Xd, r, t, **kw)
    toks, cnt, pos = P.ttf_compress(Xd, r, t, order=order, pos_base=pos_base, **kw)
    torch.cuda.synchronize()

    a_gpu = int(q["anchor"].item())
    cos_sorted = np.sort(R.anchor_cos)
    margin = float(cos_sorted[-1] - cos_sorted[-2]) if F > 1 else float("inf")
    if fixed is not None:
        assert a_gpu == fixed, f"anchor {a_gpu} != requested {fixed}"
    elif a_gpu != R.anchor:
        assert not require_anchor or margin < ANCHOR_MARGIN, f"anchor {a_gpu} != oracle {R.anchor} (margin {margin:.3g})"
        R = O.compress(X, r, t, anchor_frame=a_gpu)

    sim = q["best_sim"].cpu().numpy()
    dst = q["dst"].cpu().numpy()
    keep = q["keep"].cpu().numpy()
    fuse = q["fuse_cnt"].cpu().numpy()

    finite = np.isfinite(R.s_hat)
    err = float(np.abs(sim[finite].astype(np.float64) - R.s_hat[finite]).max()) if finite.any() else 0.0
    assert err <= SIM_ATOL, f"best similarity differs by {err:.3g}"

    in_band = np.abs(R.s_hat.astype(np.float32).astype(np.float64) - np.float64(np.float32(t))) < BAND
    bad_keep = (keep != R.keep) & ~in_band
    assert not bad_keep.any(), f"{int(bad_keep.sum())} keep decisions differ outside the band"
    tie_band = (R.s_hat - R.second) < BAND
    bad_dst = (dst != R.dst) & ~tie_band
    assert not bad_dst.any(), f"{int(bad_dst.sum())} dst differ outside the tie band"

    # everything downstream of the accepted decisions is exact
    forced = O.compress(X, r, t, anchor_frame=a_gpu, forced_keep=keep, natural=bool(order), pos_base=pos_base)
    assert (fuse == O.fuse_count(keep, dst, F, N, a_gpu)).all(), "fuse counts differ"
    L = int(cnt.item())
    assert L == forced.count, f"count {L} != {forced.count}"
    assert L == int(keep.sum()), "count != number of retained tokens"
    assert (pos[:L].cpu().numpy() == forced.pos).all(), "positions differ"
    assert (to_bits(toks[:L]) == forced.tokens).all(), "token rows differ"
    return {"anchor": a_gpu, "anchor_margin": margin, "count": L, "rho": 1.0 - L / (F * N),
            "band": int(in_band.sum()), "keep_flips": int((keep != R.keep).sum()),
            "dst_flips": int((dst != R.dst).sum()), "sim_err": err}
