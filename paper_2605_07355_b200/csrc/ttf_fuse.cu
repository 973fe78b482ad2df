// Optional mean fusion.  NOT the paper's method: Sec. 3 (Threshold Gating) replaces a fused token by its anchor
// token unchanged and rules out any convex combination of features.  This is the averaging alternative, offered
// as a separate entry point: after the ordinary pass, anchor row j of the compressed sequence is overwritten with
//     ( x_{a,j} + sum of the source tokens (k,i) with keep(k,i) = 0 and dst(k,i) = j ) / ( 1 + fuse_cnt_j ).
//
// The reduction is gather-side and segmented by anchor cell: the CTAs of cell j visit the (F-1) x |window| tokens
// that can point to j in ascending flat order k*N + i, keep those that do, and add their rows in that order in
// fp32, starting from the anchor token.  No atomics: the result does not depend on scheduling.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kFuseThreads = 256;
constexpr int kFuseWarps = kFuseThreads / 32;

// fp32 -> storage type, round to nearest even
template <typename T> struct Narrow;
template <> struct Narrow<float> {
    static __device__ __forceinline__ float from(float v) { return v; }
};
template <> struct Narrow<bf16_t> {
    static __device__ __forceinline__ bf16_t from(float v) {
        uint32_t u = __float_as_uint(v);
        bf16_t o;
        if ((u & 0x7fffffffu) > 0x7f800000u) { o.bits = (uint16_t)((u >> 16) | 0x40u); return o; }   // NaN stays NaN
        u += 0x7fffu + ((u >> 16) & 1u);
        o.bits = (uint16_t)(u >> 16);
        return o;
    }
};

template <typename T, int V> struct Storer;
template <> struct Storer<float, 4> {
    static __device__ __forceinline__ void store(float* p, const float (&x)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};
template <> struct Storer<float, 1> {
    static __device__ __forceinline__ void store(float* p, const float (&x)[1]) { p[0] = x[0]; }
};
template <> struct Storer<bf16_t, 8> {
    static __device__ __forceinline__ void store(bf16_t* p, const float (&x)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            w[e] = (uint32_t)Narrow<bf16_t>::from(x[2 * e]).bits | ((uint32_t)Narrow<bf16_t>::from(x[2 * e + 1]).bits << 16);
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};
template <> struct Storer<bf16_t, 1> {
    static __device__ __forceinline__ void store(bf16_t* p, const float (&x)[1]) { p[0] = Narrow<bf16_t>::from(x[0]); }
};

// CTA = (anchor cell j, slice of kFuseThreads * V channels).  Candidates are taken kFuseThreads at a time in
// ascending flat order; the ones fused into j are packed, in that order, into a list in shared memory (ballot +
// prefix over the warps), then every thread adds the listed rows to its V channels.
template <typename T, int V>
__global__ void __launch_bounds__(kFuseThreads)
k_fuse_mean(const T* __restrict__ X, int F, int H, int W, int C, int r, const int* __restrict__ hdr,
            const unsigned char* __restrict__ keep, const int* __restrict__ dst, T* __restrict__ out_tokens, int nslices)
{
    using L = Loader<T, V>;
    __shared__ int s_list[kFuseThreads];
    __shared__ int s_warp[kFuseWarps];
    const int N = H * W;
    const int j = blockIdx.x / nslices, slice = blockIdx.x - j * nslices;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int a = hdr[HDR_ANCHOR];
    const int y = j / W, x = j - y * W;
    const int y_lo = max(0, y - r), y_hi = min(H - 1, y + r);
    const int x_lo = max(0, x - r), x_hi = min(W - 1, x + r);
    const int nx = x_hi - x_lo + 1, wsz = (y_hi - y_lo + 1) * nx;       // window ∩ grid, ascending cell index
    const long long ncand = (long long)(F - 1) * wsz;
    const int c0 = (slice * kFuseThreads + tid) * V;
    const bool on = c0 < C;

    float acc[V];
    if (on) L::load(X + ((size_t)a * N + j) * C + c0, acc);             // the anchor token is the first term
    else {
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
    }
    int members = 1;
    for (long long q0 = 0; q0 < ncand; q0 += kFuseThreads) {
        const long long q = q0 + tid;
        int f = -1;
        if (q < ncand) {
            const int kk = (int)(q / wsz), e = (int)(q - (long long)kk * wsz);
            const int k = kk < a ? kk : kk + 1;                          // source frames only
            const int cell = (y_lo + e / nx) * W + x_lo + e % nx;
            const int cand = k * N + cell;
            if (!keep[cand] && dst[cand] == j) f = cand;
        }
        const unsigned m = __ballot_sync(0xffffffffu, f >= 0);
        if (lane == 0) s_warp[w] = __popc(m);
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int ww = 0; ww < kFuseWarps; ++ww) { const int c = s_warp[ww]; if (ww < w) before += c; total += c; }
        if (f >= 0) s_list[before + __popc(m & ((1u << lane) - 1u))] = f;
        __syncthreads();
        if (on) {
            int e = 0;
            for (; e + 4 <= total; e += 4) {                             // four rows in flight, added in list order
                typename L::Raw raw[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) raw[u] = L::load_raw(X + (size_t)s_list[e + u] * C + c0);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float v[V];
                    L::unpack(raw[u], v);
#pragma unroll
                    for (int c = 0; c < V; ++c) acc[c] += v[c];
                }
            }
            for (; e < total; ++e) {
                float v[V];
                L::load(X + (size_t)s_list[e] * C + c0, v);
#pragma unroll
                for (int c = 0; c < V; ++c) acc[c] += v[c];
            }
        }
        members += total;
        __syncthreads();                                                 // the list is rebuilt by the next round
    }
    if (on) {
        const float denom = (float)members;
#pragma unroll
        for (int c = 0; c < V; ++c) acc[c] = acc[c] / denom;
        Storer<T, V>::store(out_tokens + (size_t)j * C + c0, acc);
    }
}

template <typename T, int V>
static cudaError_t launch_fuse_mean_t(const Problem& p, const Scratch& s, void* out_tokens, cudaStream_t st) {
    const int per = kFuseThreads * V;
    const int nslices = (p.C + per - 1) / per;
    const long long blocks = (long long)p.N * nslices;
    if (blocks >= (1LL << 31)) return cudaErrorInvalidConfiguration;
    k_fuse_mean<T, V><<<(unsigned)blocks, kFuseThreads, 0, st>>>(
        reinterpret_cast<const T*>(p.X), p.F, p.H, p.W, p.C, p.r, s.hdr, s.keep, s.dst,
        reinterpret_cast<T*>(out_tokens), nslices);
    return cudaGetLastError();
}

// Overwrites rows [0, N) of out_tokens (the anchor block of the compressed sequence) with the means; reads the
// anchor, keep and dst that the pass left in the scratch block.
cudaError_t launch_fuse_mean(const Problem& p, const Scratch& s, void* out_tokens, cudaStream_t st) {
    const bool vec = p.vec && reinterpret_cast<uintptr_t>(out_tokens) % 16 == 0;
    if (p.dtype == 0) return vec ? launch_fuse_mean_t<float, 4>(p, s, out_tokens, st) : launch_fuse_mean_t<float, 1>(p, s, out_tokens, st);
    return vec ? launch_fuse_mean_t<bf16_t, 8>(p, s, out_tokens, st) : launch_fuse_mean_t<bf16_t, 1>(p, s, out_tokens, st);
}

}  // namespace ttf
