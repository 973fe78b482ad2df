"""GPU parity of the optional mean fusion (ttf_compress_mean; not the paper's method) against the oracle.

Tolerances: fp32 clips |gpu - oracle| <= 1e-5 * max(|oracle|, rms of the output row) (fp32 accumulation of at
most (F-1)(2r+1)^2 + 1 terms against fp64); bf16 clips within 1 bf16 ulp of the oracle's fp64 mean rounded once
(the fp32 sum can sit on the other side of a rounding boundary).  Everything else of the call must equal
ttf_compress bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ttf_oracle as O
from paper_2605_07355_b200 import clips
import paper_2605_07355_b200 as P
from tests.parity import to_device, to_bits
from tests.test_gpu_parity import corr_clip

pytestmark = pytest.mark.gpu


def ordered(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> integers whose order and spacing are those of the values (ulp distance)"""
    s = bits.astype(np.int32)
    mag = s & 0x7FFF
    return np.where(s & 0x8000, -mag, mag)


def check_mean(X: np.ndarray, r: int, t: float) -> int:
    F, H, W, C = X.shape
    N = H * W
    Xd = to_device(X)
    q = P.ttf_query(Xd, r, t)
    ref = P.ttf_compress(Xd, r, t)
    toks, cnt, pos = P.ttf_compress_mean(Xd, r, t)
    torch.cuda.synchronize()
    L = int(cnt.item())
    assert L == int(ref[1].item())
    assert torch.equal(pos[:L], ref[2][:L])
    assert torch.equal(toks[N:L], ref[0][N:L])                     # preserved source rows: bit copies as before
    a = int(q["anchor"].item())
    keep, dst = q["keep"].cpu().numpy(), q["dst"].cpu().numpy()
    want = O.fuse_mean(X, keep, dst, a)                            # fp64, from the decisions the GPU took
    got = to_bits(toks[:N])
    if X.dtype == np.float32:
        scale = np.maximum(np.abs(want), np.sqrt((want ** 2).mean(axis=1, keepdims=True)))
        bad = np.abs(got.astype(np.float64) - want) > 1e-5 * scale + 1e-30
        assert not bad.any(), f"{int(bad.sum())} fp32 means off by more than 1e-5 relative"
    else:
        ulp = np.abs(ordered(got) - ordered(O.round_to_bf16_bits(want)))
        assert ulp.max() <= 1, f"bf16 means off by {int(ulp.max())} ulp"
    again = P.ttf_compress_mean(Xd, r, t)
    torch.cuda.synchronize()
    assert torch.equal(again[0][:L], toks[:L])                     # reproducible bit for bit
    return int((keep == 0).sum())


SHAPES = [(1, 4, 4, 32, 1), (2, 3, 5, 40, 1), (3, 7, 5, 33, 1), (4, 9, 1, 16, 2), (3, 2, 2, 7, 1),
          (6, 5, 6, 264, 0), (4, 6, 7, 520, 2), (17, 3, 3, 72, 1), (9, 4, 6, 1032, 1), (3, 4, 4, 64, 5)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_mean_fuse_small_shapes(shape, dtype):
    F, H, W, C, r = shape
    X = corr_clip(F, H, W, C, seed=sum(shape) + 1, dtype=dtype)
    for t in (0.7, 0.4):
        check_mean(X, r, t)


def test_mean_fuse_extremes():
    X = corr_clip(6, 5, 4, 48, seed=4, dtype="bf16")
    assert check_mean(X, 1, 2.0) == 0                              # nothing fused: the anchor rows themselves
    Xd = to_device(X)
    assert torch.equal(P.ttf_compress_mean(Xd, 1, 2.0)[0][:20], P.ttf_compress(Xd, 1, 2.0)[0][:20])
    assert check_mean(X, 1, -2.0) == 5 * 20                        # every source token fused
    assert check_mean(corr_clip(300, 2, 3, 16, seed=6, dtype="f32", sigma=0.2), 1, 0.3) > 256   # several list rounds


@pytest.mark.parametrize("name", ["tiny_cal", "vl2b_cal"])
def test_mean_fuse_paper_shaped(name):
    s = clips.CONFIGS[name]
    fused = check_mean(clips.make_clip(s), s.r, s.t)
    assert fused > 0.4 * s.tokens


def test_mean_fuse_misaligned_base_pointer_takes_scalar_path():
    F, H, W, C = 4, 4, 5, 64
    X = corr_clip(F, H, W, C, seed=15, dtype="bf16")
    buf = torch.zeros(F * H * W * C + 8, dtype=torch.bfloat16, device="cuda")
    view = buf[1:1 + F * H * W * C].view(F, H, W, C)                  # 2 bytes off a 16-byte boundary
    view.copy_(to_device(X))
    assert view.data_ptr() % 16 != 0
    a = P.ttf_compress_mean(view, 1, 0.6)
    b = P.ttf_compress_mean(to_device(X), 1, 0.6)
    torch.cuda.synchronize()
    L = int(a[1].item())
    assert L == int(b[1].item()) and torch.equal(a[0][:L], b[0][:L]) and torch.equal(a[2][:L], b[2][:L])
