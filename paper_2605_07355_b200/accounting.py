"""Algorithmic bytes and flops of the TTF pass (host arithmetic only; used by the benchmark's roofline).

"Algorithmic" = what the method must move or compute for one clip, independent of how kernels are organised:
the pass has to read X once and write X', P' and L' (Eqs. xprime_stack, compress_pos, Lpre).
"""
from __future__ import annotations


def window_pairs(H: int, W: int, r: int) -> int:
    """sum over cells of |J(i)|: candidates left by clipping (Eq. pi) and duplicate masking."""
    ny = sum(min(H - 1, y + r) - max(0, y - r) + 1 for y in range(H))
    nx = sum(min(W - 1, x + r) - max(0, x - r) + 1 for x in range(W))
    return ny * nx


def matching_flops_nominal(F: int, N: int, C: int, r: int) -> int:
    """The paper's count of the matching overhead: 2 (F-1) N (2r+1)^2 C (cost term O((2r+1)^2 FNC); Table 3)."""
    return 2 * (F - 1) * N * (2 * r + 1) ** 2 * C


def matching_flops(F: int, H: int, W: int, C: int, r: int) -> int:
    """Multiply-adds actually needed (border cells have fewer candidates), as flops."""
    return 2 * (F - 1) * window_pairs(H, W, r) * C


def pass_bytes(F: int, N: int, C: int, itemsize: int, count: int) -> int:
    """B_min: read X once; write X' (count rows), P' (count x 3 int32) and L'."""
    return F * N * C * itemsize + count * C * itemsize + count * 12 + 4


def kernel_bytes(kind: str, F: int, N: int, C: int, itemsize: int, count: int) -> int:
    """Algorithmic bytes of one launch of each kernel kind."""
    X = F * N * C * itemsize
    if kind == "norm_sum":          # reads X; writes the frame sums (the norms only on the CUDA-core path)
        return X + F * C * 4
    if kind == "frame_stats":       # reads the frame sums
        return F * C * 4
    if kind == "match":             # reads X (sources + anchor frame once); writes s_hat, dst, keep
        return X + F * N * 9
    if kind == "compact":           # reads the retained rows, writes them with their positions
        return 2 * count * C * itemsize + count * 12 + F * N + 4
    raise KeyError(kind)


def pipeline_dram_bytes_model(F: int, N: int, C: int, itemsize: int, count: int, lanes, fixed_anchor: bool = False) -> int:
    """DRAM bytes one clip moves in the pipeline as scheduled (confirmed with the profiler's DRAM counters over a
    whole step: 93.8 / 153.4 / 172.7 MB per 8B-shaped clip for 1 / 2 / 8 clips in flight, 113.7 MB with a fixed
    anchor).  With one clip in flight the matching pass and the gather find the clip in L2, so it is read once; with
    two or more in flight the clips displace one another, and the second pass over X (which only the automatic anchor
    of Eq. auto_anchor needs) and the gather's rows come from DRAM again.  Output rows, positions and the small
    per-token arrays are written once either way."""
    X = F * N * C * itemsize
    rows = count * C * itemsize
    small = F * N * 9 + count * 12 + 4
    if lanes == "2, pipelined":         # X once, the kept rows for the gather again, the output (measured: 133 MB,
        return X + 2 * rows + small     # the model's 114 MB plus what the matching pass still misses)
    if lanes <= 1:
        return X + rows + small
    return (1 if fixed_anchor else 2) * X + 2 * rows + small


def csrc_hash() -> str:
    """Hash of the CUDA sources and the C header the library is built from: ties stored profiler counters to the
    kernels they were taken on."""
    import glob
    import hashlib
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    files = sorted(glob.glob(os.path.join(here, "csrc", "*.cu")) + glob.glob(os.path.join(here, "csrc", "*.cuh")))
    files.append(os.path.join(os.path.dirname(here), "include", "ttf.h"))
    h = hashlib.sha256()
    for f in files:
        h.update(os.path.basename(f).encode())
        h.update(open(f, "rb").read())
    return h.hexdigest()[:16]
