// Pointwise Matching with Local Window Search and Threshold Gating (Eqs. pi, argmax, dst, gating, mask).
//
// Work is grouped by grid cell: all F tokens at cell i share the same candidate set
//   J(i) = { y'*W + x' : |y'-y_i| <= r, |x'-x_i| <= r, inside the grid },
// which is what clipping the offsets (Eq. pi) and masking the duplicates leaves.  Candidates are visited in
// ascending anchor index and the running maximum is replaced only on a strictly larger similarity, so equal
// candidates resolve to the lowest anchor index.  keep = !(s_hat > t): a token is fused only when its best
// similarity exceeds t strictly (Eq. gating keeps s_hat <= t); a NaN similarity keeps the token.
//
// k_match_generic is the reference CUDA-core kernel: any dtype, any radius, any C.  One CTA per
// (cell, chunk of frames), one warp per source token, lanes stride over the channels with 16-byte loads when
// rows allow it, fp32 FMA accumulation, fixed-order warp reduction.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kMatchWarps = 8;

template <typename T, int V>
__global__ void __launch_bounds__(kMatchWarps * 32)
k_match_generic(const T* __restrict__ X, int F, int H, int W, int C, int r, float t, int fchunk, int nslice,
                const int* __restrict__ hdr, const float* __restrict__ ssq,
                float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep,
                int* __restrict__ cnt)
{
    const int N = H * W;
    const int i = blockIdx.x % N;
    const int chunk = blockIdx.x / N;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int a = hdr[HDR_ANCHOR];
    const int y = i / W, x = i - y * W;
    const size_t FN = (size_t)F * N;
    const int y_lo = max(0, y - r), y_hi = min(H - 1, y + r);
    const int x_lo = max(0, x - r), x_hi = min(W - 1, x + r);
    const int k_end = min(F, (chunk + 1) * fchunk);
    const T* Xa = X + (size_t)a * N * C;

    for (int k = chunk * fchunk + w; k < k_end; k += kMatchWarps) {
        const size_t f = (size_t)k * N + i;
        if (k == a) {                       // anchor tokens are always retained (Eq. mask)
            if (lane == 0) { shat[f] = 1.0f; dst[f] = i; keep[f] = 1; }
            continue;
        }
        const T* xs = X + f * C;
        const float rs = inv_norm(ssq, nslice, FN, f);
        float best = -INFINITY;
        int best_j = -1;
        for (int yy = y_lo; yy <= y_hi; ++yy) {
            for (int xx = x_lo; xx <= x_hi; ++xx) {
                const int j = yy * W + xx;
                const T* xa = Xa + (size_t)j * C;
                float acc0 = 0.f, acc1 = 0.f;
                int c = lane * V;
                for (; c + 32 * V < C; c += 64 * V) {
                    float u0[V], v0[V], u1[V], v1[V];
                    Loader<T, V>::load(xs + c, u0);
                    Loader<T, V>::load(xa + c, v0);
                    Loader<T, V>::load(xs + c + 32 * V, u1);
                    Loader<T, V>::load(xa + c + 32 * V, v1);
#pragma unroll
                    for (int v = 0; v < V; ++v) { acc0 = fmaf(u0[v], v0[v], acc0); acc1 = fmaf(u1[v], v1[v], acc1); }
                }
                if (c < C) {
                    float u0[V], v0[V];
                    Loader<T, V>::load(xs + c, u0);
                    Loader<T, V>::load(xa + c, v0);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc0 = fmaf(u0[v], v0[v], acc0);
                }
                const float dot = warp_sum(acc0 + acc1);
                const float s = dot * rs * inv_norm(ssq, nslice, FN, (size_t)a * N + j);
                if (s > best || best_j < 0) { best = s; best_j = j; }
            }
        }
        if (lane == 0) {
            const unsigned char kp = !(best > t);
            shat[f] = best; dst[f] = best_j; keep[f] = kp;
            if (kp) atomicAdd(&cnt[k], 1);   // integer count: order-independent
        }
    }
}

template <typename T, int V>
static cudaError_t launch_generic_t(const Problem& p, const Scratch& s, float* shat, int* dst,
                                    unsigned char* keep, cudaStream_t st) {
    // enough CTAs to fill the GPU a few times over: split the frames into chunks when the grid is small
    int fchunk = p.F;
    const long long want = 4LL * sm_count();
    if ((long long)p.N < want) {
        long long chunks = (want + p.N - 1) / p.N;
        fchunk = (int)((p.F + chunks - 1) / chunks);
        if (fchunk < kMatchWarps) fchunk = kMatchWarps;
    }
    const long long nchunk = (p.F + fchunk - 1) / fchunk;
    k_match_generic<T, V><<<(unsigned)(nchunk * p.N), kMatchWarps * 32, 0, st>>>(
        reinterpret_cast<const T*>(p.X), p.F, p.H, p.W, p.C, p.r, p.t, fchunk, p.nslice, s.hdr, s.ssq,
        shat, dst, keep, s.cnt);
    return cudaGetLastError();
}

cudaError_t launch_match(const Problem& p, const Scratch& s, float* shat, int* dst, unsigned char* keep,
                         cudaStream_t st) {
    if (p.dtype == 0) return p.vec ? launch_generic_t<float, 4>(p, s, shat, dst, keep, st)
                                   : launch_generic_t<float, 1>(p, s, shat, dst, keep, st);
    return p.vec ? launch_generic_t<bf16_t, 8>(p, s, shat, dst, keep, st)
                 : launch_generic_t<bf16_t, 1>(p, s, shat, dst, keep, st);
}

}  // namespace ttf
