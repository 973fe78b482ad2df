"""ctypes front end of the CPU oracle (oracle/ttf_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this module; the CUDA
library never does.  This file only marshals arrays: every step of the method is in the C file, which
follows Sec. 3 of the paper (anchor rule, local-window matching, threshold gate, compaction, positions).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ttf_oracle.c")
_LIB = os.path.join(_HERE, "libttf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, so double arithmetic stays in source order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_int, c_sz, vp = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
        lib.ttf_oracle_threads.restype = c_int
        lib.ttf_oracle_anchor.restype = c_int
        lib.ttf_oracle_anchor.argtypes = [vp, c_int, c_int, c_int, vp]
        lib.ttf_oracle_match.restype = None
        lib.ttf_oracle_match.argtypes = [vp, c_int, c_int, c_int, c_int, c_int, c_int, vp, vp, vp]
        lib.ttf_oracle_match_global.restype = None
        lib.ttf_oracle_match_global.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp]
        lib.ttf_oracle_gate.restype = None
        lib.ttf_oracle_gate.argtypes = [vp, c_int, c_int, c_int, ctypes.c_float, vp]
        lib.ttf_oracle_fuse_count.restype = None
        lib.ttf_oracle_fuse_count.argtypes = [vp, vp, c_int, c_int, c_int, vp]
        lib.ttf_oracle_compact.restype = c_int
        lib.ttf_oracle_compact.argtypes = [vp, c_sz, vp, c_int, c_int, c_int, c_int, c_int, c_int, vp, vp, vp]
        lib.ttf_oracle_restore.restype = None
        lib.ttf_oracle_restore.argtypes = [vp, c_sz, vp, vp, c_int, c_int, c_int, vp, vp]
        lib.ttf_oracle_sim_histogram.restype = None
        lib.ttf_oracle_sim_histogram.argtypes = [vp, c_int, c_int, c_int, c_int, vp]
        lib.ttf_oracle_fuse_mean.restype = None
        lib.ttf_oracle_fuse_mean.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp, vp]
        lib.ttf_oracle_decode_pos.restype = ctypes.c_longlong
        lib.ttf_oracle_decode_pos.argtypes = [ctypes.c_longlong] * 3
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().ttf_oracle_threads())


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _widen(X: np.ndarray) -> np.ndarray:
    """fp32 view of the clip: fp32 as is, bf16 bit patterns (uint16) widened exactly (16-bit shift)."""
    if X.dtype == np.float32:
        return np.ascontiguousarray(X)
    if X.dtype == np.uint16:
        return (np.ascontiguousarray(X).astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise TypeError("clip must be float32 or uint16 (bf16 bit patterns)")


def _shape(X: np.ndarray):
    if X.ndim != 4:
        raise ValueError("clip must be [F, H, W, C]")
    return X.shape


def anchor(X: np.ndarray):
    """Eq. (auto_anchor): returns (a*, cos[F])."""
    F, H, W, C = _shape(X)
    Xf = _widen(X)
    cos = np.empty(F, dtype=np.float64)
    a = _load().ttf_oracle_anchor(_ptr(Xf), F, H * W, C, _ptr(cos))
    return int(a), cos


def match(X: np.ndarray, r: int, a: int):
    """Eqs. (pi), (argmax), (dst): returns (s_hat[F*N] f64, dst[F*N] i32, second[F*N] f64)."""
    F, H, W, C = _shape(X)
    Xf = _widen(X)
    n = F * H * W
    s_hat = np.empty(n, dtype=np.float64)
    dst = np.empty(n, dtype=np.int32)
    second = np.empty(n, dtype=np.float64)
    _load().ttf_oracle_match(_ptr(Xf), F, H, W, C, int(r), int(a), _ptr(s_hat), _ptr(dst), _ptr(second))
    return s_hat, dst, second


def match_global(X: np.ndarray, a: int):
    """Best cosine over ALL anchor tokens (all-pairs search); cross-check only."""
    F, H, W, C = _shape(X)
    Xf = _widen(X)
    n = F * H * W
    s_hat = np.empty(n, dtype=np.float64)
    dst = np.empty(n, dtype=np.int32)
    _load().ttf_oracle_match_global(_ptr(Xf), F, H * W, C, int(a), _ptr(s_hat), _ptr(dst))
    return s_hat, dst


def gate(s_hat: np.ndarray, F: int, N: int, a: int, t: float) -> np.ndarray:
    """Eqs. (gating), (mask): keep[F*N] uint8."""
    s_hat = np.ascontiguousarray(s_hat, dtype=np.float64)
    keep = np.empty(F * N, dtype=np.uint8)
    _load().ttf_oracle_gate(_ptr(s_hat), F, N, int(a), float(t), _ptr(keep))
    return keep


def fuse_count(keep: np.ndarray, dst: np.ndarray, F: int, N: int, a: int) -> np.ndarray:
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    dst = np.ascontiguousarray(dst, dtype=np.int32)
    out = np.empty(N, dtype=np.int32)
    _load().ttf_oracle_fuse_count(_ptr(keep), _ptr(dst), F, N, int(a), _ptr(out))
    return out


def compact(X: np.ndarray, keep: np.ndarray, a: int, natural: bool = False, pos_base: int = 0):
    """Eqs. (xprime_stack), (compress_pos): returns (tokens[L', C] same dtype as X, pos[L', 3] i32,
    index[L'] i32 flat source index of each output row, L').  natural: ascending flat index instead of the anchor
    block first; pos_base: added to all three coordinates."""
    F, H, W, C = _shape(X)
    Xc = np.ascontiguousarray(X)
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    n = F * H * W
    tokens = np.empty((n, C), dtype=X.dtype)
    pos = np.empty((n, 3), dtype=np.int32)
    index = np.empty(n, dtype=np.int32)
    L = _load().ttf_oracle_compact(_ptr(Xc), C * X.dtype.itemsize, _ptr(keep), F, H, W, int(a),
                                   1 if natural else 0, int(pos_base), _ptr(tokens), _ptr(pos), _ptr(index))
    return tokens[:L], pos[:L], index[:L], int(L)


def restore(compressed: np.ndarray, keep: np.ndarray, dst: np.ndarray, F: int, N: int, a: int):
    """Discussion D4 (TTF-R): returns (full[F*N, ...], row_index[F*N])."""
    comp = np.ascontiguousarray(compressed)
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    dst = np.ascontiguousarray(dst, dtype=np.int32)
    row_bytes = comp[0].size * comp.itemsize
    full = np.empty((F * N,) + comp.shape[1:], dtype=comp.dtype)
    idx = np.empty(F * N, dtype=np.int32)
    _load().ttf_oracle_restore(_ptr(comp), row_bytes, _ptr(keep), _ptr(dst), F, N, int(a), _ptr(idx), _ptr(full))
    return full, idx


def sim_histogram(s_hat_f32: np.ndarray, F: int, N: int, a: int, bins: int) -> np.ndarray:
    """Discussion D1: histogram of the best similarities of the source tokens over [-1, 1]."""
    s = np.ascontiguousarray(s_hat_f32, dtype=np.float32)
    hist = np.empty(bins, dtype=np.uint32)
    _load().ttf_oracle_sim_histogram(_ptr(s), F, N, int(a), int(bins), _ptr(hist))
    return hist


def stats(s_hat_f32: np.ndarray, keep: np.ndarray, F: int, N: int, a: int, t: float, band: float):
    """Sec. 3, after Eq. Lpre: rho = 1 - (N + P) / (F N).  Returns (P, fused, in_band, rho) over the source tokens:
    P preserved, fused = (F-1) N - P, in_band = |s_hat - t| < band on the stored fp32 similarities and the fp32
    threshold, compared in double.  Plain loops, one token at a time."""
    s = np.asarray(s_hat_f32, dtype=np.float32).reshape(F, N)
    kp = np.asarray(keep).reshape(F, N)
    tt = float(np.float32(t))
    bb = float(np.float32(band))
    P = fused = in_band = 0
    for k in range(F):
        if k == a:
            continue
        for i in range(N):
            if kp[k, i]:
                P += 1
            else:
                fused += 1
            if abs(float(s[k, i]) - tt) < bb:
                in_band += 1
    return P, fused, in_band, 1.0 - (N + P) / (F * N)


def compress_segment(X: np.ndarray, r: int, t: float, frame_base: int, forced_keep: Optional[np.ndarray] = None):
    """Discussion D3 (rolling anchor): frame 0 is the anchor of the segment and is not emitted; returns
    (tokens[P, C], pos[P, 3] with the frame coordinate frame_base + k - 1, P)."""
    F, H, W, C = _shape(X)
    N = H * W
    R = compress(X, r, t, anchor_frame=0, forced_keep=forced_keep)
    pos = R.pos[N:].copy()
    pos[:, 0] += frame_base - 1
    return R.tokens[N:], pos, R.count - N


def fuse_mean(X: np.ndarray, keep: np.ndarray, dst: np.ndarray, a: int) -> np.ndarray:
    """Mean fusion (NOT the paper's method, which replaces a fused token by its anchor token unchanged): [N, C]
    f64, row j = mean of anchor token j and of the source tokens fused into it."""
    F, H, W, C = _shape(X)
    Xf = _widen(X)
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    dst = np.ascontiguousarray(dst, dtype=np.int32)
    out = np.empty((H * W, C), dtype=np.float64)
    _load().ttf_oracle_fuse_mean(_ptr(Xf), F, H * W, C, int(a), _ptr(keep), _ptr(dst), _ptr(out))
    return out


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit patterns (uint16), round to nearest, ties to even, in one rounding."""
    x = np.asarray(x, dtype=np.float64)
    down = (x.astype(np.float32).view(np.uint32) & np.uint32(0xFFFF0000))          # a bf16 value near x
    cand = np.stack([down - np.uint32(0x10000), down, down + np.uint32(0x10000)])     # its neighbours
    vals = cand.view(np.float32).astype(np.float64)
    err = np.abs(vals - x[None])
    err = np.where(np.isfinite(vals), err, np.inf)
    even = ((cand >> np.uint32(16)) & np.uint32(1)) == 0
    nearest = err == err.min(axis=0)[None]
    best = np.argmin(np.where(nearest, np.where(even, 0, 1), 2), axis=0)             # ties: the even pattern
    out = np.take_along_axis(cand, best[None], axis=0)[0]
    return (out >> np.uint32(16)).astype(np.uint16)


def decode_pos(L_prime: int, T: int, l: int) -> int:
    """Eqs. (Lpre), (decode_pos)."""
    return int(_load().ttf_oracle_decode_pos(L_prime, T, l))


@dataclass
class OracleResult:
    anchor: int
    anchor_cos: np.ndarray      # [F] f64
    s_hat: np.ndarray           # [F*N] f64
    dst: np.ndarray             # [F*N] i32
    second: np.ndarray          # [F*N] f64 runner-up similarity
    keep: np.ndarray            # [F*N] u8
    fuse_cnt: np.ndarray        # [N] i32
    tokens: np.ndarray          # [L', C]
    pos: np.ndarray             # [L', 3] i32
    index: np.ndarray           # [L'] i32
    count: int                  # L' = N + P

    @property
    def rho(self) -> float:
        return 1.0 - self.count / float(self.keep.size)


def compress(X: np.ndarray, r: int, t: float, anchor_frame: Optional[int] = None,
             forced_keep: Optional[np.ndarray] = None, natural: bool = False, pos_base: int = 0) -> OracleResult:
    """The whole pass in the paper's order.  ``anchor_frame`` overrides the anchor rule (first / last /
    explicit anchors of Table 1); ``forced_keep`` replaces the gate's decisions (used after near-threshold
    differences have been accepted, so that counts, positions and rows can still be compared exactly)."""
    F, H, W, C = _shape(X)
    N = H * W
    a_auto, cos = anchor(X)
    a = a_auto if anchor_frame is None else int(anchor_frame)
    s_hat, dst, second = match(X, r, a)
    keep = gate(s_hat, F, N, a, t) if forced_keep is None else np.ascontiguousarray(forced_keep, dtype=np.uint8).reshape(-1)
    fc = fuse_count(keep, dst, F, N, a)
    tokens, pos, index, L = compact(X, keep, a, natural=natural, pos_base=pos_base)
    return OracleResult(a, cos, s_hat, dst, second, keep, fc, tokens, pos, index, L)
