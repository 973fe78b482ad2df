// Anchor Frame Selection (Eq. auto_anchor) and per-token norms.
//
// k_norm_sum streams X once: a CTA owns (frame k, channel slice q) where a slice is 32 lanes x one 16-byte
// load; warp w walks the tokens i = w, w+8, ... of the frame.  Each lane keeps the running channel sums of
// its channels (the frame sum S_k = N * mean token of frame k) and every token's squared norm restricted to
// the slice is reduced over the warp and stored as a partial (the full norm is the sum over slices, taken in
// slice order by the consumers).  All reductions have a fixed order, so results are reproducible.
//
// k_anchor_pick computes g = sum_k S_k (= F*N times the global mean token), the cosine of every S_k to g
// (the factors 1/N and 1/(FN) of Eq. auto_anchor cancel in a cosine) and the arg max, lowest frame on ties.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kNormWarps = 8;
constexpr int kNormUnroll = 4;

template <typename T, int V>
__global__ void __launch_bounds__(kNormWarps * 32)
k_norm_sum(const T* __restrict__ X, int F, int N, int C, int nslice,
           float* __restrict__ S, float* __restrict__ ssq, int* __restrict__ cnt)
{
    const int k = blockIdx.x / nslice;
    const int q = blockIdx.x - k * nslice;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int c0 = (q * 32 + lane) * V;
    const bool active = c0 < C;                 // C is a multiple of V on the vector path
    const size_t FN = (size_t)F * N;
    const T* base = X + (size_t)k * N * C + c0;

    float col[V];
#pragma unroll
    for (int v = 0; v < V; ++v) col[v] = 0.f;

    for (int i0 = w; i0 < N; i0 += kNormWarps * kNormUnroll) {
        float x[kNormUnroll][V];
#pragma unroll
        for (int u = 0; u < kNormUnroll; ++u) {
            const int i = i0 + u * kNormWarps;
            if (active && i < N) {
                Loader<T, V>::load(base + (size_t)i * C, x[u]);
            } else {
#pragma unroll
                for (int v = 0; v < V; ++v) x[u][v] = 0.f;
            }
        }
#pragma unroll
        for (int u = 0; u < kNormUnroll; ++u) {
            float ss = 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) { ss = fmaf(x[u][v], x[u][v], ss); col[v] += x[u][v]; }
            ss = warp_sum(ss);
            const int i = i0 + u * kNormWarps;
            if (lane == 0 && i < N) ssq[(size_t)q * FN + (size_t)k * N + i] = ss;
        }
    }

    __shared__ float sm[kNormWarps][32 * V];
#pragma unroll
    for (int v = 0; v < V; ++v) sm[w][lane * V + v] = col[v];
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * V; idx += kNormWarps * 32) {
        const int c = q * 32 * V + idx;
        if (c < C) {
            float s = 0.f;
#pragma unroll
            for (int ww = 0; ww < kNormWarps; ++ww) s += sm[ww][idx];
            S[(size_t)k * C + c] = s;
        }
    }
    if (q == 0 && threadIdx.x == 0) cnt[k] = 0;   // survivor counters start at zero for the matching kernel
}

template <typename T, int V>
static cudaError_t launch_norm_sum_t(const Problem& p, const Scratch& s, cudaStream_t st) {
    const long long blocks = (long long)p.F * p.nslice;
    k_norm_sum<T, V><<<(unsigned)blocks, kNormWarps * 32, 0, st>>>(
        reinterpret_cast<const T*>(p.X), p.F, p.N, p.C, p.nslice, s.S, s.ssq, s.cnt);
    return cudaGetLastError();
}

cudaError_t launch_norm_sum(const Problem& p, const Scratch& s, cudaStream_t st) {
    if (p.dtype == 0) return p.vec ? launch_norm_sum_t<float, 4>(p, s, st) : launch_norm_sum_t<float, 1>(p, s, st);
    return p.vec ? launch_norm_sum_t<bf16_t, 8>(p, s, st) : launch_norm_sum_t<bf16_t, 1>(p, s, st);
}

// ---------------------------------------------------------------------------------------------------------
constexpr int kPickThreads = 1024;

__global__ void __launch_bounds__(kPickThreads)
k_anchor_pick(const float* __restrict__ S, int F, int C, float* __restrict__ g, float* __restrict__ fcos,
              int* __restrict__ hdr, int* __restrict__ out_anchor, int mode, int arg)
{
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    __shared__ float s_gg[kPickThreads / 32];
    __shared__ float s_best[kPickThreads / 32];
    __shared__ int s_idx[kPickThreads / 32];

    if (mode != 0) {   // fixed anchors of Table 1 (first / last) or an explicit frame
        if (tid == 0) {
            int a = mode == 1 ? 0 : (mode == 2 ? F - 1 : arg);
            hdr[HDR_ANCHOR] = a;
            if (out_anchor) *out_anchor = a;
        }
        return;
    }

    // g[c] = sum_k S[k][c], frames in ascending order; |g|^2 reduced in a fixed order
    float gg = 0.f;
    for (int c = tid; c < C; c += kPickThreads) {
        float a = 0.f;
        for (int k = 0; k < F; ++k) a += S[(size_t)k * C + c];
        g[c] = a;
        gg = fmaf(a, a, gg);
    }
    gg = warp_sum(gg);
    if (lane == 0) s_gg[w] = gg;
    __syncthreads();                     // also makes g[] visible to the whole block
    float gnorm2 = 0.f;
    for (int ww = 0; ww < kPickThreads / 32; ++ww) gnorm2 += s_gg[ww];
    const float ginv = 1.0f / fmaxf(sqrtf(gnorm2), kNormFloor);

    // cosine of every frame sum to g: one warp per frame
    for (int k = w; k < F; k += kPickThreads / 32) {
        const float* Sk = S + (size_t)k * C;
        float d = 0.f, qq = 0.f;
        for (int c = lane; c < C; c += 32) {
            const float v = Sk[c];
            d = fmaf(v, g[c], d);
            qq = fmaf(v, v, qq);
        }
        d = warp_sum(d);
        qq = warp_sum(qq);
        if (lane == 0) fcos[k] = d * ginv * (1.0f / fmaxf(sqrtf(qq), kNormFloor));
    }
    __syncthreads();

    // arg max over frames, lowest frame on ties
    float best = -INFINITY;
    int idx = 0x7fffffff;
    for (int k = tid; k < F; k += kPickThreads) {
        const float v = fcos[k];
        if (v > best || idx == 0x7fffffff) { best = v; idx = k; }   // ascending k per thread: first max stays
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (oi != 0x7fffffff && (idx == 0x7fffffff || ob > best || (ob == best && oi < idx))) { best = ob; idx = oi; }
    }
    if (lane == 0) { s_best[w] = best; s_idx[w] = idx; }
    __syncthreads();
    if (tid == 0) {
        float b = s_best[0];
        int bi = s_idx[0];
        for (int ww = 1; ww < kPickThreads / 32; ++ww) {
            const float ob = s_best[ww];
            const int oi = s_idx[ww];
            if (oi != 0x7fffffff && (bi == 0x7fffffff || ob > b || (ob == b && oi < bi))) { b = ob; bi = oi; }
        }
        hdr[HDR_ANCHOR] = bi;
        if (out_anchor) *out_anchor = bi;
    }
}

cudaError_t launch_anchor_pick(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    k_anchor_pick<<<1, kPickThreads, 0, st>>>(s.S, p.F, p.C, s.g, s.fcos, s.hdr, out_anchor, p.anchor_mode,
                                              p.anchor_arg);
    return cudaGetLastError();
}

}  // namespace ttf
