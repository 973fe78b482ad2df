// Extensions the paper sketches in its Discussion: TTF-R restoration through dst(k,i) (D4) and the empirical
// distribution of the best-match similarities that an adaptive threshold would look at (D1).
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kXThreads = 256;

// Row of the compressed sequence that stands for token (k,i): its own row if it was retained (anchor rows are
// rows 0..N-1, preserved source tokens follow in ascending flat order, Eq. xprime_stack), else the anchor row
// dst(k,i) it was fused into (Eq. dst).  One CTA per frame.
__global__ void __launch_bounds__(kXThreads)
k_restore_index(const int* __restrict__ anchor, const unsigned char* __restrict__ keep, const int* __restrict__ dst,
                int F, int N, int* __restrict__ row_index)
{
    __shared__ int s_warp[kXThreads / 32];
    __shared__ int s_base;
    const int k = blockIdx.x, tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int a = *anchor;
    if (k == a) {
        for (int i = tid; i < N; i += kXThreads) row_index[(size_t)k * N + i] = i;
        return;
    }
    // preserved source tokens in the frames before this one (the anchor frame does not count)
    int c = 0;
    const size_t before = (size_t)k * N;
    for (size_t f = tid; f < before; f += kXThreads) c += (f / N != (size_t)a && keep[f]) ? 1 : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) s_warp[w] = c;
    __syncthreads();
    if (tid == 0) { int b = 0; for (int ww = 0; ww < kXThreads / 32; ++ww) b += s_warp[ww]; s_base = b; }
    __syncthreads();
    int run = N + s_base;
    for (int i0 = 0; i0 < N; i0 += kXThreads) {
        const int i = i0 + tid;
        const bool kp = i < N && keep[before + i];
        const unsigned m = __ballot_sync(0xffffffffu, kp);
        __syncthreads();
        if (lane == 0) s_warp[w] = __popc(m);
        __syncthreads();
        int off = 0, total = 0;
        for (int ww = 0; ww < kXThreads / 32; ++ww) { if (ww < w) off += s_warp[ww]; total += s_warp[ww]; }
        if (i < N) row_index[before + i] = kp ? run + off + __popc(m & ((1u << lane) - 1)) : dst[before + i];
        run += total;
    }
}

template <typename U>
__global__ void __launch_bounds__(kXThreads)
k_restore_copy(const unsigned char* __restrict__ comp, size_t row_bytes, long long rows,
               const int* __restrict__ row_index, unsigned char* __restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * (kXThreads / 32) + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * (kXThreads / 32);
    const int units = (int)(row_bytes / sizeof(U));
    for (long long f = gw; f < rows; f += nw) {
        const U* src = reinterpret_cast<const U*>(comp + (size_t)row_index[f] * row_bytes);
        U* d = reinterpret_cast<U*>(out + (size_t)f * row_bytes);
        for (int u = lane; u < units; u += 32) d[u] = src[u];
    }
}

cudaError_t launch_restore(const void* comp, size_t row_bytes, int F, int N, const int* anchor,
                           const unsigned char* keep, const int* dst, void* out_full, int* row_index,
                           cudaStream_t st) {
    k_restore_index<<<F, kXThreads, 0, st>>>(anchor, keep, dst, F, N, row_index);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long rows = (long long)F * N;
    long long blocks = (rows + kXThreads / 32 - 1) / (kXThreads / 32);
    if (blocks > 8LL * sm_count()) blocks = 8LL * sm_count();
    const unsigned char* c = reinterpret_cast<const unsigned char*>(comp);
    unsigned char* o = reinterpret_cast<unsigned char*>(out_full);
    const uintptr_t al = reinterpret_cast<uintptr_t>(comp) | reinterpret_cast<uintptr_t>(out_full) | row_bytes;
    if (al % 16 == 0) k_restore_copy<uint4><<<(unsigned)blocks, kXThreads, 0, st>>>(c, row_bytes, rows, row_index, o);
    else if (al % 4 == 0) k_restore_copy<uint32_t><<<(unsigned)blocks, kXThreads, 0, st>>>(c, row_bytes, rows, row_index, o);
    else if (al % 2 == 0) k_restore_copy<uint16_t><<<(unsigned)blocks, kXThreads, 0, st>>>(c, row_bytes, rows, row_index, o);
    else k_restore_copy<unsigned char><<<(unsigned)blocks, kXThreads, 0, st>>>(c, row_bytes, rows, row_index, o);
    return cudaGetLastError();
}

// Histogram of the best-match similarities of the source tokens over `bins` equal bins of [-1, 1]
// (bin = floor((s + 1) / 2 * bins), clamped; NaN is not counted).  Integer atomics: order-independent.
__global__ void __launch_bounds__(kXThreads)
k_sim_histogram(const float* __restrict__ sim, const int* __restrict__ anchor, int N, long long total, int bins,
                unsigned int* __restrict__ hist)
{
    const int a = *anchor;
    const long long stride = (long long)gridDim.x * kXThreads;
    for (long long f = (long long)blockIdx.x * kXThreads + threadIdx.x; f < total; f += stride) {
        if (f / N == a) continue;
        const float s = sim[f];
        if (!(s == s)) continue;
        int b = (int)floorf((s + 1.0f) * 0.5f * (float)bins);
        b = b < 0 ? 0 : (b >= bins ? bins - 1 : b);
        atomicAdd(&hist[b], 1u);
    }
}

cudaError_t launch_sim_histogram(const float* sim, const int* anchor, int F, int N, int bins, unsigned int* hist,
                                 cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(hist, 0, sizeof(unsigned int) * (size_t)bins, st);
    if (e != cudaSuccess) return e;
    const long long total = (long long)F * N;
    long long blocks = (total + kXThreads - 1) / kXThreads;
    if (blocks > 4LL * sm_count()) blocks = 4LL * sm_count();
    k_sim_histogram<<<(unsigned)blocks, kXThreads, 0, st>>>(sim, anchor, N, total, bins, hist);
    return cudaGetLastError();
}

}  // namespace ttf
