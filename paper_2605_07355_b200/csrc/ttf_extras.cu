// Extensions the paper sketches in its Discussion: TTF-R restoration through dst(k,i) (D4) and the empirical
// distribution of the best-match similarities that an adaptive threshold would look at (D1).
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kXThreads = 256;

// Number of non-zero flags in keep[lo, hi): bytes up to the first 16-byte boundary, 16 flags per load from there,
// bytes again at the end.  Every thread of the CTA takes part; the caller adds the per-thread counts up.
__device__ __forceinline__ int count_flags(const unsigned char* __restrict__ keep, size_t lo, size_t hi, int tid) {
    if (lo >= hi) return 0;
    int c = 0;
    const uintptr_t base = reinterpret_cast<uintptr_t>(keep);
    size_t head = lo + ((16 - ((base + lo) & 15)) & 15);          // first index whose address is 16-byte aligned
    if (head > hi) head = hi;
    const size_t nvec = (hi - head) / 16, tail = head + nvec * 16;
    for (size_t f = lo + tid; f < head; f += kXThreads) c += keep[f] ? 1 : 0;
    const uint4* v = reinterpret_cast<const uint4*>(keep + head);
    for (size_t u = tid; u < nvec; u += kXThreads) {
        const uint4 q = __ldg(v + u);
        // a flag is any non-zero byte: fold each byte's bits into its lowest one
        unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            unsigned b = w[e];
            b |= b >> 4; b |= b >> 2; b |= b >> 1;
            c += __popc(b & 0x01010101u);
        }
    }
    for (size_t f = tail + tid; f < hi; f += kXThreads) c += keep[f] ? 1 : 0;
    return c;
}

// Row of the compressed sequence that stands for token (k,i): its own row if it was retained (anchor rows are
// rows 0..N-1, preserved source tokens follow in ascending flat order, Eq. xprime_stack), else the anchor row
// dst(k,i) it was fused into (Eq. dst).  One CTA per frame; it counts the flags of the frames before its own
// (16 per load, at most F N bytes, from L2 after the first CTA has touched them).
__global__ void __launch_bounds__(kXThreads)
k_restore_index(const int* __restrict__ anchor, const unsigned char* __restrict__ keep, const int* __restrict__ dst,
                int F, int N, int* __restrict__ row_index)
{
    __shared__ int s_warp[kXThreads / 32];
    __shared__ int s_base;
    pdl_launch_dependents();                     // the copy kernel may start its set-up; it waits before it reads row_index
    const int k = blockIdx.x, tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int a = *anchor;
    if (k == a) {
        for (int i = tid; i < N; i += kXThreads) row_index[(size_t)k * N + i] = i;
        return;
    }
    // preserved source tokens in the frames before this one (the anchor frame does not count)
    const size_t before = (size_t)k * N;
    int c = count_flags(keep, 0, before, tid);
    if (a < k) c -= count_flags(keep, (size_t)a * N, (size_t)(a + 1) * N, tid);
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

// One warp per output row; a lane keeps up to eight loads in flight before it stores them, so a row of 8 KB moves
// in two rounds.  Rows of retained tokens are read once (consecutive tokens sit in consecutive compressed rows);
// the N anchor rows are read again and again and stay in L2.
template <typename U>
__global__ void __launch_bounds__(kXThreads)
k_restore_copy(const unsigned char* __restrict__ comp, size_t row_bytes, long long rows,
               const int* __restrict__ row_index, unsigned char* __restrict__ out)
{
    constexpr int kInFlight = 8;
    const int lane = threadIdx.x & 31;
    const long long gw = (long long)blockIdx.x * (kXThreads / 32) + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * (kXThreads / 32);
    const int units = (int)(row_bytes / sizeof(U));
    pdl_wait();                                  // row_index is complete
    for (long long f = gw; f < rows; f += nw) {
        const U* src = reinterpret_cast<const U*>(comp + (size_t)__ldcg(row_index + f) * row_bytes);
        U* d = reinterpret_cast<U*>(out + (size_t)f * row_bytes);
        int u = lane;
        for (; u + (kInFlight - 1) * 32 < units; u += kInFlight * 32) {
            U v[kInFlight];
#pragma unroll
            for (int e = 0; e < kInFlight; ++e) v[e] = src[u + e * 32];
#pragma unroll
            for (int e = 0; e < kInFlight; ++e) d[u + e * 32] = v[e];
        }
        for (; u < units; u += 32) d[u] = src[u];
    }
}

template <typename U>
static cudaError_t launch_restore_copy(const unsigned char* c, size_t row_bytes, long long rows, const int* row_index,
                                       unsigned char* o, cudaStream_t st) {
    long long blocks = (rows + kXThreads / 32 - 1) / (kXThreads / 32);
    if (blocks > 8LL * sm_count()) blocks = 8LL * sm_count();
    return launch_pdl(k_restore_copy<U>, dim3((unsigned)blocks), dim3(kXThreads), st, c, row_bytes, rows, row_index, o);
}

cudaError_t launch_restore(const void* comp, size_t row_bytes, int F, int N, const int* anchor,
                           const unsigned char* keep, const int* dst, void* out_full, int* row_index,
                           cudaStream_t st) {
    k_restore_index<<<F, kXThreads, 0, st>>>(anchor, keep, dst, F, N, row_index);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long rows = (long long)F * N;
    const unsigned char* c = reinterpret_cast<const unsigned char*>(comp);
    unsigned char* o = reinterpret_cast<unsigned char*>(out_full);
    const uintptr_t al = reinterpret_cast<uintptr_t>(comp) | reinterpret_cast<uintptr_t>(out_full) | row_bytes;
    if (al % 16 == 0) return launch_restore_copy<uint4>(c, row_bytes, rows, row_index, o, st);
    if (al % 4 == 0) return launch_restore_copy<uint32_t>(c, row_bytes, rows, row_index, o, st);
    if (al % 2 == 0) return launch_restore_copy<uint16_t>(c, row_bytes, rows, row_index, o, st);
    return launch_restore_copy<unsigned char>(c, row_bytes, rows, row_index, o, st);
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

// Counts behind the reduction ratio rho = 1 - (N + P) / (F N) (Sec. 3, after Eq. Lpre) and the number of source
// tokens whose best similarity lies within `band` of the threshold (the decisions rounding could flip).
// out[0] = P (preserved source tokens), out[1] = fused source tokens, out[2] = in-band source tokens.  The band test
// is taken in double on the stored fp32 values, so the counts are exact functions of the arrays.  Integer atomics.
__global__ void __launch_bounds__(kXThreads)
k_stats(const float* __restrict__ sim, const unsigned char* __restrict__ keep, const int* __restrict__ anchor, int N,
        long long total, float t, float band, unsigned long long* __restrict__ out)
{
    __shared__ int s_part[3][kXThreads / 32];
    const int a = *anchor;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int c[3] = {0, 0, 0};
    const long long stride = (long long)gridDim.x * kXThreads;
    for (long long f = (long long)blockIdx.x * kXThreads + threadIdx.x; f < total; f += stride) {
        if (f / N == a) continue;
        const bool kp = keep[f] != 0;
        c[0] += kp ? 1 : 0;
        c[1] += kp ? 0 : 1;
        c[2] += fabs((double)sim[f] - (double)t) < (double)band ? 1 : 0;
    }
#pragma unroll
    for (int q = 0; q < 3; ++q) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c[q] += __shfl_xor_sync(0xffffffffu, c[q], o);
        if (lane == 0) s_part[q][w] = c[q];
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        unsigned long long v = 0;
        for (int ww = 0; ww < kXThreads / 32; ++ww) v += (unsigned long long)s_part[threadIdx.x][ww];
        if (v) atomicAdd(out + threadIdx.x, v);
    }
}

cudaError_t launch_stats(const float* sim, const unsigned char* keep, const int* anchor, int F, int N, float t, float band,
                         long long* out, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(out, 0, 3 * sizeof(long long), st);
    if (e != cudaSuccess) return e;
    const long long total = (long long)F * N;
    long long blocks = (total + kXThreads - 1) / kXThreads;
    if (blocks > 2LL * sm_count()) blocks = 2LL * sm_count();
    k_stats<<<(unsigned)blocks, kXThreads, 0, st>>>(sim, keep, anchor, N, total, t, band,
                                                   reinterpret_cast<unsigned long long*>(out));
    return cudaGetLastError();
}

// Measurement aid: the plainest kernel that reads a buffer once (fully coalesced, eight 16-byte loads in flight per
// thread, eight CTAs of 256 threads per SM, launched like the kernels of the pass).  What a launch of this kind
// takes on one clip is the floor for any kernel that must read that clip: ramp-up and tail of a launch that lasts
// some 10 us are a visible share of it, so it is well below the copy rate of large buffers.
__global__ void __launch_bounds__(kXThreads)
k_read_floor(const uint4* __restrict__ buf, long long n16, unsigned* __restrict__ sink)
{
    pdl_launch_dependents();
    pdl_wait();
    unsigned acc = 0;
    const long long stride = (long long)gridDim.x * kXThreads * 8;
    for (long long i0 = (long long)blockIdx.x * kXThreads * 8 + threadIdx.x; i0 < n16; i0 += stride) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = i0 + u * kXThreads < n16 ? __ldcs(buf + i0 + u * kXThreads) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc += v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    if (acc == 0x9e3779b9u && sink) *sink = acc;       // keeps the loads alive; practically never true
}

cudaError_t launch_read_floor(const void* buf, size_t bytes, unsigned* sink, cudaStream_t st) {
    return launch_pdl(k_read_floor, dim3((unsigned)(8 * sm_count())), dim3(kXThreads), st,
                      reinterpret_cast<const uint4*>(buf), (long long)(bytes / 16), sink);
}

}  // namespace ttf
