"""Thin Python binding of libttf_b200.so: argument marshalling only.

Function names and argument order follow include/ttf.h.  Tensors are torch tensors (device memory and
streams come from PyTorch); every step of the pass runs in the library's CUDA kernels.  There is no CPU
fallback: if the shared library is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("TTF_B200_LIB") or os.path.join(_HERE, "libttf_b200.so")

TTF_DTYPE_F32, TTF_DTYPE_BF16 = 0, 1
TTF_OK = 0

EXPORTS = [
    "ttf_status_string", "ttf_last_cuda_error", "ttf_workspace_bytes", "ttf_compress", "ttf_compress_ws",
    "ttf_query", "ttf_query_ws", "ttf_compress_host", "ttf_release", "ttf_profile_begin", "ttf_profile_end",
    "ttf_query_static", "ttf_compress_ex", "ttf_query_ex", "ttf_compress_segment", "ttf_restore",
    "ttf_sim_histogram", "ttf_stats", "ttf_compress_batch", "ttf_compress_batch_ex", "ttf_profile_stages", "ttf_profile_read_floor", "ttf_compress_mean", "ttf_compress_host_batch",
    "ttf_set_schedule", "ttf_set_match_kernel", "ttf_last_device_status", "ttf_workspace_status", "ttf_debug_set_wait", "ttf_debug_func_attr_needed", "ttf_debug_set_check_slack",
]
TTF_ERR_TIMEOUT, TTF_ERR_STATIC_LIMIT, TTF_ERR_BOUNDS = 5, 6, 7
TTF_ANCHOR_AUTO, TTF_ANCHOR_FIRST, TTF_ANCHOR_LAST, TTF_ANCHOR_EXPLICIT = 0, 1, 2, 3
TTF_ORDER_ANCHOR_FIRST, TTF_ORDER_NATURAL = 0, 1
TTF_SCHEDULE_PIPELINED = -1


class TTFOptions(ctypes.Structure):
    """ttf_options of include/ttf.h"""
    _fields_ = [("anchor_mode", ctypes.c_int), ("anchor_frame", ctypes.c_int), ("order", ctypes.c_int),
                ("pos_base", ctypes.c_int)]


def _options(anchor_mode: int, anchor_frame: int, order: int, pos_base: int):
    """NULL when everything is at its default, else a ttf_options by reference"""
    if not (anchor_mode or anchor_frame or order or pos_base):
        return None
    return ctypes.byref(TTFOptions(int(anchor_mode), int(anchor_frame), int(order), int(pos_base)))

TTF_STATIC_SCRATCH_BYTES = 8 << 20
KERNEL_KINDS = ["norm_sum", "frame_stats", "match", "compact", "fuse_count"]

_lib = None


class TTFError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib().ttf_status_string(status).decode()
        extra = f" (cudaError {lib().ttf_last_cuda_error()})" if name == "TTF_ERR_CUDA" else ""
        super().__init__(f"{where}: {name}{extra}")


def lib() -> ctypes.CDLL:
    """Loads the C-ABI library (built by paper_2605_07355_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2605_07355_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        i, f, vp, sz = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
        shape = [i, i, i, i, i]                       # F, H, W, C, r
        L.ttf_status_string.restype = ctypes.c_char_p
        L.ttf_status_string.argtypes = [i]
        L.ttf_last_cuda_error.restype = i
        L.ttf_last_cuda_error.argtypes = []
        L.ttf_workspace_bytes.restype = i
        L.ttf_workspace_bytes.argtypes = shape + [i, ctypes.POINTER(sz)]
        L.ttf_compress.restype = i
        L.ttf_compress.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp]
        L.ttf_compress_batch.restype = i
        L.ttf_compress_batch.argtypes = [vp, i] + shape + [f, i, vp, vp, vp, vp]
        L.ttf_profile_stages.restype = i
        L.ttf_profile_stages.argtypes = [vp, i] + shape + [f, i, vp, vp, vp, i, ctypes.POINTER(ctypes.c_double), i, vp]
        L.ttf_last_device_status.restype = i
        L.ttf_last_device_status.argtypes = [vp, ctypes.POINTER(i)]
        L.ttf_workspace_status.restype = i
        L.ttf_workspace_status.argtypes = [vp, vp, ctypes.POINTER(i)]
        L.ttf_debug_set_check_slack.restype = i
        L.ttf_debug_set_check_slack.argtypes = [i]
        L.ttf_debug_set_wait.restype = i
        L.ttf_debug_set_wait.argtypes = [i, i]
        L.ttf_debug_func_attr_needed.restype = i
        L.ttf_debug_func_attr_needed.argtypes = [vp, i, sz]
        L.ttf_set_match_kernel.restype = i
        L.ttf_set_match_kernel.argtypes = [i]
        L.ttf_set_schedule.restype = i
        L.ttf_set_schedule.argtypes = [i]
        L.ttf_compress_mean.restype = i
        L.ttf_compress_mean.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp]
        L.ttf_compress_host_batch.restype = i
        L.ttf_compress_host_batch.argtypes = [vp, i] + shape + [f, i, vp, vp, vp]
        L.ttf_compress_ws.restype = i
        L.ttf_compress_ws.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, sz, vp]
        L.ttf_query.restype = i
        L.ttf_query.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, vp, vp]
        L.ttf_query_ws.restype = i
        L.ttf_query_ws.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, vp, vp, sz, vp]
        L.ttf_compress_ex.restype = i
        L.ttf_compress_ex.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, vp]
        L.ttf_compress_batch_ex.restype = i
        L.ttf_compress_batch_ex.argtypes = [vp, i] + shape + [f, i, vp, vp, vp, vp, vp]
        L.ttf_query_ex.restype = i
        L.ttf_query_ex.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, vp, vp, vp]
        L.ttf_compress_segment.restype = i
        L.ttf_compress_segment.argtypes = [vp] + shape + [f, i, i, vp, vp, vp, vp]
        L.ttf_restore.restype = i
        L.ttf_restore.argtypes = [vp, sz, i, i, i, vp, vp, vp, vp, vp, vp]
        L.ttf_profile_read_floor.restype = i
        L.ttf_profile_read_floor.argtypes = [vp, i, ctypes.c_size_t, i, vp, vp]
        L.ttf_stats.restype = i
        L.ttf_stats.argtypes = [vp, vp, vp, i, i, i, ctypes.c_float, ctypes.c_float, vp, vp]
        L.ttf_sim_histogram.restype = i
        L.ttf_sim_histogram.argtypes = [vp, vp, i, i, i, i, vp, vp]
        L.ttf_query_static.restype = i
        L.ttf_query_static.argtypes = [vp] + shape + [f, i, vp, vp, vp, vp, vp, vp]
        L.ttf_compress_host.restype = i
        L.ttf_compress_host.argtypes = [vp] + shape + [f, i, vp, vp, vp]
        L.ttf_release.restype = i
        L.ttf_release.argtypes = []
        L.ttf_profile_begin.restype = i
        L.ttf_profile_begin.argtypes = []
        L.ttf_profile_end.restype = i
        L.ttf_profile_end.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong), i]
        _lib = L
    return _lib


def _dtype_code(x: torch.Tensor) -> int:
    if x.dtype == torch.float32:
        return TTF_DTYPE_F32
    if x.dtype == torch.bfloat16:
        return TTF_DTYPE_BF16
    raise TypeError(f"features must be float32 or bfloat16, got {x.dtype}")


def _check_features(x: torch.Tensor, device: str):
    if x.dim() != 4:
        raise ValueError("features must be [F, H, W, C]")
    if not x.is_contiguous():
        raise ValueError("features must be contiguous")
    if device == "cuda" and not x.is_cuda:
        raise ValueError("features must be a CUDA tensor")
    if device == "cpu" and x.is_cuda:
        raise ValueError("features must be a host tensor")
    return tuple(int(v) for v in x.shape)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def ttf_workspace_bytes(F: int, H: int, W: int, C: int, r: int, dtype: int) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().ttf_workspace_bytes(F, H, W, C, r, dtype, ctypes.byref(n))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_workspace_bytes")
    return int(n.value)


def ttf_compress(features: torch.Tensor, r: int, t: float, out_tokens: Optional[torch.Tensor] = None,
                 out_count: Optional[torch.Tensor] = None, out_pos_thw: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None, stream=None,
                 anchor_mode: int = 0, anchor_frame: int = 0, order: int = 0, pos_base: int = 0):
    """ttf_compress / ttf_compress_ws (ttf_compress_ex when any option is given).  Returns (out_tokens [F*H*W, C], out_count int32[1],
    out_pos_thw int32 [F*H*W, 3]); only the first out_count rows are defined.  Does not synchronise."""
    F, H, W, C = _check_features(features, "cuda")
    dev = features.device
    n = F * H * W
    if out_tokens is None:
        out_tokens = torch.empty((n, C), dtype=features.dtype, device=dev)
    if out_count is None:
        out_count = torch.empty(1, dtype=torch.int32, device=dev)
    if out_pos_thw is None:
        out_pos_thw = torch.empty((n, 3), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        sp = _stream_ptr(stream)
        opt = _options(anchor_mode, anchor_frame, order, pos_base)
        if opt is not None:
            if workspace is not None:
                raise ValueError("the entry point with options uses the library's own scratch")
            rc = lib().ttf_compress_ex(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features), opt,
                                       _p(out_tokens), _p(out_count), _p(out_pos_thw), sp)
        elif workspace is None:
            rc = lib().ttf_compress(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features),
                                    _p(out_tokens), _p(out_count), _p(out_pos_thw), sp)
        else:
            rc = lib().ttf_compress_ws(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features),
                                       _p(out_tokens), _p(out_count), _p(out_pos_thw),
                                       _p(workspace), workspace.numel() * workspace.element_size(), sp)
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress")
    return out_tokens, out_count, out_pos_thw


def ttf_profile_stages(features, r: int, t: float, out_tokens, out_count, out_pos_thw, reps: int = 10, stream=None) -> dict:
    """ttf_profile_stages: milliseconds per launch of each kernel of the pass at steady state, by kernel kind."""
    feats = list(features)
    F, H, W, C = _check_features(feats[0], "cuda")
    B = len(feats)
    arr = lambda ts: (ctypes.c_void_p * B)(*[t_.data_ptr() for t_ in ts])
    n = len(KERNEL_KINDS)
    ms = (ctypes.c_double * n)()
    with torch.cuda.device(feats[0].device):
        rc = lib().ttf_profile_stages(arr(feats), B, F, H, W, C, int(r), float(t), _dtype_code(feats[0]),
                                      arr(out_tokens), arr(out_count), arr(out_pos_thw), int(reps), ms, n,
                                      _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_profile_stages")
    return {k: float(ms[i]) for i, k in enumerate(KERNEL_KINDS[:4])}


def ttf_profile_read_floor(buffers, reps: int = 10, stream=None) -> float:
    """ttf_profile_read_floor: ms per launch of a plain read kernel over each of `buffers` (same size, contiguous)."""
    nbytes = buffers[0].numel() * buffers[0].element_size()
    ptrs = (ctypes.c_void_p * len(buffers))(*[b.data_ptr() for b in buffers])
    ms = ctypes.c_double(0.0)
    with torch.cuda.device(buffers[0].device):
        rc = lib().ttf_profile_read_floor(ptrs, len(buffers), ctypes.c_size_t(nbytes), int(reps), ctypes.byref(ms),
                                          _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_profile_read_floor")
    return ms.value


def ttf_last_device_status(stream=None) -> int:
    """ttf_last_device_status: synchronises the stream; TTF_OK or TTF_ERR_TIMEOUT for the last call on it."""
    v = ctypes.c_int(0)
    rc = lib().ttf_last_device_status(_stream_ptr(stream), ctypes.byref(v))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_last_device_status")
    return int(v.value)


def ttf_workspace_status(workspace: Optional[torch.Tensor], stream=None) -> int:
    """ttf_workspace_status: the same for caller-owned scratch (None = the array of ttf_query_static)."""
    v = ctypes.c_int(0)
    rc = lib().ttf_workspace_status(_p(workspace), _stream_ptr(stream), ctypes.byref(v))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_workspace_status")
    return int(v.value)


def ttf_debug_set_wait(poll_limit: int = 1 << 18, tx_extra_bytes: int = 0) -> None:
    """ttf_debug_set_wait (test hook): poll limit of the bounded waits and extra bytes announced to copy barriers."""
    rc = lib().ttf_debug_set_wait(int(poll_limit), int(tx_extra_bytes))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_debug_set_wait")


def ttf_debug_set_check_slack(slack: int = 0) -> int:
    """ttf_debug_set_check_slack: returns the status (TTF_ERR_UNSUPPORTED = 2 from the normal build)."""
    return int(lib().ttf_debug_set_check_slack(int(slack)))


def ttf_set_match_kernel(which: int = 0) -> None:
    """ttf_set_match_kernel: 0 automatic, 1 warp-level MMA kernel, 2 tcgen05 kernel."""
    rc = lib().ttf_set_match_kernel(int(which))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_set_match_kernel")


def ttf_set_schedule(clips_in_flight: int = 0) -> None:
    """ttf_set_schedule: clips of a batch in flight (0 = automatic, 1 to 8, or TTF_SCHEDULE_PIPELINED = -1: two
    lanes in opposite phases with the matching pass served by L2)."""
    rc = lib().ttf_set_schedule(int(clips_in_flight))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_set_schedule")


def ttf_compress_mean(features: torch.Tensor, r: int, t: float, stream=None):
    """ttf_compress_mean: ttf_compress with the anchor rows replaced by the means of the tokens fused into them
    (not the paper's method).  Returns (out_tokens, out_count, out_pos_thw).  Does not synchronise."""
    F, H, W, C = _check_features(features, "cuda")
    dev = features.device
    n = F * H * W
    out_tokens = torch.empty((n, C), dtype=features.dtype, device=dev)
    out_count = torch.empty(1, dtype=torch.int32, device=dev)
    out_pos_thw = torch.empty((n, 3), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ttf_compress_mean(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features),
                                     _p(out_tokens), _p(out_count), _p(out_pos_thw), _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress_mean")
    return out_tokens, out_count, out_pos_thw


def ttf_compress_batch(features, r: int, t: float, out_tokens=None, out_count=None, out_pos_thw=None, stream=None,
                       anchor_mode: int = 0, anchor_frame: int = 0, order: int = 0, pos_base: int = 0):
    """ttf_compress_batch (ttf_compress_batch_ex when any option is given): `features` is a sequence of [F, H, W, C]
    device tensors of one shape and dtype.
    Returns three lists (out_tokens, out_count, out_pos_thw), one entry per clip, as ttf_compress does for one
    clip.  Does not synchronise."""
    feats = list(features)
    if not feats:
        raise ValueError("empty batch")
    F, H, W, C = _check_features(feats[0], "cuda")
    dev, dt = feats[0].device, feats[0].dtype
    for x in feats[1:]:
        if _check_features(x, "cuda") != (F, H, W, C) or x.dtype != dt or x.device != dev:
            raise ValueError("all clips of a batch must have the same shape, dtype and device")
    n, B = F * H * W, len(feats)
    if out_tokens is None:
        out_tokens = [torch.empty((n, C), dtype=dt, device=dev) for _ in range(B)]
    if out_count is None:
        out_count = [torch.empty(1, dtype=torch.int32, device=dev) for _ in range(B)]
    if out_pos_thw is None:
        out_pos_thw = [torch.empty((n, 3), dtype=torch.int32, device=dev) for _ in range(B)]
    if not (len(out_tokens) == len(out_count) == len(out_pos_thw) == B):
        raise ValueError("one output of each kind per clip")
    arr = lambda ts: (ctypes.c_void_p * B)(*[t_.data_ptr() for t_ in ts])
    opt = _options(anchor_mode, anchor_frame, order, pos_base)
    with torch.cuda.device(dev):
        if opt is None:
            rc = lib().ttf_compress_batch(arr(feats), B, F, H, W, C, int(r), float(t), _dtype_code(feats[0]),
                                          arr(out_tokens), arr(out_count), arr(out_pos_thw), _stream_ptr(stream))
        else:
            rc = lib().ttf_compress_batch_ex(arr(feats), B, F, H, W, C, int(r), float(t), _dtype_code(feats[0]), opt,
                                             arr(out_tokens), arr(out_count), arr(out_pos_thw), _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress_batch")
    return out_tokens, out_count, out_pos_thw


def ttf_query(features: torch.Tensor, r: int, t: float, workspace: Optional[torch.Tensor] = None, stream=None,
              want=("anchor", "keep", "dst", "best_sim", "fuse_cnt"), anchor_mode: int = 0,
              anchor_frame: int = 0) -> dict:
    """ttf_query / ttf_query_ws (ttf_query_ex when an anchor rule other than auto is given).  Returns the requested device tensors.  Does not synchronise."""
    F, H, W, C = _check_features(features, "cuda")
    dev = features.device
    n = F * H * W
    out = {
        "anchor": torch.empty(1, dtype=torch.int32, device=dev) if "anchor" in want else None,
        "keep": torch.empty(n, dtype=torch.uint8, device=dev) if "keep" in want else None,
        "dst": torch.empty(n, dtype=torch.int32, device=dev) if "dst" in want else None,
        "best_sim": torch.empty(n, dtype=torch.float32, device=dev) if "best_sim" in want else None,
        "fuse_cnt": torch.empty(H * W, dtype=torch.int32, device=dev) if "fuse_cnt" in want else None,
    }
    args = [_p(features), F, H, W, C, int(r), float(t), _dtype_code(features), _p(out["anchor"]), _p(out["keep"]),
            _p(out["dst"]), _p(out["best_sim"]), _p(out["fuse_cnt"])]
    with torch.cuda.device(dev):
        sp = _stream_ptr(stream)
        opt = _options(anchor_mode, anchor_frame, 0, 0)
        if opt is not None:
            if workspace is not None:
                raise ValueError("the entry point with options uses the library's own scratch")
            rc = lib().ttf_query_ex(*args[:8], opt, *args[8:], sp)
        elif workspace is None:
            rc = lib().ttf_query(*args, sp)
        else:
            rc = lib().ttf_query_ws(*args, _p(workspace), workspace.numel() * workspace.element_size(), sp)
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_query")
    return {k: v for k, v in out.items() if v is not None}


def ttf_query_static(features: torch.Tensor, r: int, t: float, out: dict, stream=None) -> dict:
    """ttf_query_static: the query pass on the library's built-in scratch array; allocates nothing.

    For callers that may not allocate: ``out`` must already hold the tensors to fill (any of "anchor" int32[1],
    "keep" uint8[F*H*W], "dst" int32[F*H*W], "best_sim" float32[F*H*W], "fuse_cnt" int32[H*W]); this wrapper
    creates none.  Calls that can overlap on the GPU share the scratch and race; keep them on one stream.
    Raises TTFError(TTF_ERR_STATIC_LIMIT) when the clip needs more than TTF_STATIC_SCRATCH_BYTES."""
    F, H, W, C = _check_features(features, "cuda")
    args = [_p(features), F, H, W, C, int(r), float(t), _dtype_code(features), _p(out.get("anchor")),
            _p(out.get("keep")), _p(out.get("dst")), _p(out.get("best_sim")), _p(out.get("fuse_cnt"))]
    with torch.cuda.device(features.device):
        rc = lib().ttf_query_static(*args, _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_query_static")
    return out


def ttf_compress_segment(features: torch.Tensor, r: int, t: float, frame_base: int, stream=None):
    """ttf_compress_segment: frame 0 is the rolling anchor, frames 1.. are compressed against it; returns
    (out_tokens [(F-1)*H*W, C], out_count int32[1] = P, out_pos_thw [(F-1)*H*W, 3])."""
    F, H, W, C = _check_features(features, "cuda")
    dev = features.device
    n = max(1, (F - 1) * H * W)
    out_tokens = torch.empty((n, C), dtype=features.dtype, device=dev)
    out_count = torch.empty(1, dtype=torch.int32, device=dev)
    out_pos = torch.empty((n, 3), dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ttf_compress_segment(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features),
                                        int(frame_base), _p(out_tokens), _p(out_count), _p(out_pos), _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress_segment")
    return out_tokens, out_count, out_pos


def ttf_restore(compressed: torch.Tensor, F: int, H: int, W: int, anchor: torch.Tensor, keep: torch.Tensor,
                dst: torch.Tensor, stream=None):
    """ttf_restore: returns (out_full [F*H*W, ...row shape], row_index int32 [F*H*W])."""
    if not compressed.is_contiguous():
        raise ValueError("compressed must be contiguous")
    dev = compressed.device
    row_bytes = compressed[0].numel() * compressed.element_size()
    out = torch.empty((F * H * W,) + tuple(compressed.shape[1:]), dtype=compressed.dtype, device=dev)
    idx = torch.empty(F * H * W, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ttf_restore(_p(compressed), row_bytes, F, H, W, _p(anchor), _p(keep), _p(dst), _p(out), _p(idx),
                               _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_restore")
    return out, idx


def ttf_sim_histogram(best_sim: torch.Tensor, anchor: torch.Tensor, F: int, H: int, W: int, bins: int, stream=None):
    """ttf_sim_histogram: uint32 counts [bins] (returned as an int32 tensor with the same bits)."""
    dev = best_sim.device
    hist = torch.empty(bins, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ttf_sim_histogram(_p(best_sim), _p(anchor), F, H, W, int(bins), _p(hist), _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_sim_histogram")
    return hist


def ttf_stats(best_sim: torch.Tensor, keep: torch.Tensor, anchor: torch.Tensor, F: int, H: int, W: int, t: float,
              band: float = 1e-4, stream=None) -> torch.Tensor:
    """ttf_stats: int64 [3] on the device = (P preserved, fused, in-band source tokens).  Does not synchronise."""
    dev = best_sim.device
    out = torch.empty(3, dtype=torch.int64, device=dev)
    with torch.cuda.device(dev):
        rc = lib().ttf_stats(_p(best_sim), _p(keep), _p(anchor), F, H, W, float(t), float(band), _p(out), _stream_ptr(stream))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_stats")
    return out


def ttf_reduction_ratio(P_count: int, F: int, N: int) -> float:
    """rho = 1 - (N + P) / (F N)  (Sec. 3, after Eq. Lpre); the header's inline helper, restated for Python callers."""
    return 1.0 - (N + P_count) / (F * N)


def ttf_compress_host(features: torch.Tensor, r: int, t: float, out_tokens: Optional[torch.Tensor] = None,
                      out_pos_thw: Optional[torch.Tensor] = None, device: Optional[int] = None):
    """ttf_compress_host: HOST tensors in and out (pinned memory recommended).  Returns
    (out_tokens[:L'], L', out_pos_thw[:L']); synchronous."""
    F, H, W, C = _check_features(features, "cpu")
    n = F * H * W
    if out_tokens is None:
        out_tokens = torch.empty((n, C), dtype=features.dtype)
    if out_pos_thw is None:
        out_pos_thw = torch.empty((n, 3), dtype=torch.int32)
    cnt = ctypes.c_int(0)
    with torch.cuda.device(torch.cuda.current_device() if device is None else device):
        rc = lib().ttf_compress_host(_p(features), F, H, W, C, int(r), float(t), _dtype_code(features),
                                     _p(out_tokens), ctypes.cast(ctypes.byref(cnt), ctypes.c_void_p), _p(out_pos_thw))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress_host")
    L = int(cnt.value)
    return out_tokens[:L], L, out_pos_thw[:L]


def ttf_compress_host_batch(features, r: int, t: float, out_tokens=None, out_pos_thw=None, device: Optional[int] = None):
    """ttf_compress_host_batch: a sequence of HOST clips of one shape (pinned memory recommended) through the
    pipelined copy-in / pass / copy-out path.  Returns (list of out_tokens[:L'], list of L', list of
    out_pos_thw[:L']); synchronous."""
    feats = list(features)
    if not feats:
        raise ValueError("empty batch")
    F, H, W, C = _check_features(feats[0], "cpu")
    for x in feats[1:]:
        if _check_features(x, "cpu") != (F, H, W, C) or x.dtype != feats[0].dtype:
            raise ValueError("all clips of a batch must have the same shape and dtype")
    n, B = F * H * W, len(feats)
    if out_tokens is None:
        out_tokens = [torch.empty((n, C), dtype=feats[0].dtype) for _ in range(B)]
    if out_pos_thw is None:
        out_pos_thw = [torch.empty((n, 3), dtype=torch.int32) for _ in range(B)]
    if len(out_tokens) != B or len(out_pos_thw) != B:
        raise ValueError("one output of each kind per clip")
    arr = lambda ts: (ctypes.c_void_p * B)(*[t_.data_ptr() for t_ in ts])
    counts = (ctypes.c_int * B)()
    with torch.cuda.device(torch.cuda.current_device() if device is None else device):
        rc = lib().ttf_compress_host_batch(arr(feats), B, F, H, W, C, int(r), float(t), _dtype_code(feats[0]),
                                           arr(out_tokens), ctypes.cast(counts, ctypes.c_void_p), arr(out_pos_thw))
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_compress_host_batch")
    Ls = [int(c) for c in counts]
    return [o[:L] for o, L in zip(out_tokens, Ls)], Ls, [o[:L] for o, L in zip(out_pos_thw, Ls)]


def ttf_release() -> None:
    rc = lib().ttf_release()
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_release")


def ttf_profile_begin() -> None:
    rc = lib().ttf_profile_begin()
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_profile_begin")


def ttf_profile_end() -> dict:
    """Returns {kernel kind: (total device ms, launches)} for the launches since ttf_profile_begin."""
    n = len(KERNEL_KINDS)
    ms = (ctypes.c_double * n)()
    cnt = (ctypes.c_longlong * n)()
    rc = lib().ttf_profile_end(ms, cnt, n)
    if rc != TTF_OK:
        raise TTFError(rc, "ttf_profile_end")
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(KERNEL_KINDS)}


def ttf_decode_pos(L_prime: int, T: int, l: int) -> int:
    """Eqs. (Lpre), (decode_pos): the inline helper of ttf.h."""
    return int(L_prime) + int(T) + int(l)
