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
constexpr int kFuseCand = 2;                 // candidates a thread tests per round (512 per CTA: one round for F <= 57 at r = 1)
constexpr int kRows = 8;                     // rows a thread has in flight

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

// CTA = (anchor cell j, slice of kFuseThreads * V channels): small CTAs, so that all of them are resident at once
// (a 32-frame 16 x 16 clip of 4096 bf16 channels makes 2048 of them, 14 per SM) and the time of the kernel is the
// time of one CTA rather than a sum over waves.  Candidates are taken kFuseCand per thread and round in ascending
// flat order; the ones fused into j are packed, in that order, into a list in shared memory (prefix sum over the
// CTA), then every thread adds the listed rows to its V channels, kRows loads in flight.
template <typename T, int V>
__global__ void __launch_bounds__(kFuseThreads)
k_fuse_mean(const T* __restrict__ X, int F, int H, int W, int C, int r, const int* __restrict__ hdr,
            const unsigned char* __restrict__ keep, const int* __restrict__ dst, T* __restrict__ out_tokens, int nslices)
{
    using L = Loader<T, V>;
    constexpr int kRound = kFuseCand * kFuseThreads;
    __shared__ int s_list[kRound];
    __shared__ int s_cnt[kFuseCand][kFuseWarps];
    const int N = H * W;
    const int j = blockIdx.x / nslices, slice = blockIdx.x - j * nslices;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    pdl_launch_dependents();
    pdl_wait();                                  // the gather has written the anchor rows this kernel overwrites
    const int a = __ldcg(hdr + HDR_ANCHOR);
    const int y = j / W, x = j - y * W;
    const int y_lo = max(0, y - r), y_hi = min(H - 1, y + r);
    const int x_lo = max(0, x - r), x_hi = min(W - 1, x + r);
    const int nx = x_hi - x_lo + 1, wsz = (y_hi - y_lo + 1) * nx;       // window ∩ grid, ascending cell index
    const int ncand = (F - 1) * wsz;                                    // < 2^31: checked by the host
    const int c0 = (slice * kFuseThreads + tid) * V;
    const bool on = c0 < C;

    float acc[V];
    if (on) L::load(X + ((size_t)a * N + j) * C + c0, acc);             // the anchor token is the first term
    else {
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
    }
    int members = 1;
    for (int q0 = 0; q0 < ncand; q0 += kRound) {
        int f[kFuseCand], kp[kFuseCand], d[kFuseCand];
        // all loads first and unconditional (a candidate index beyond the end is clamped to the last one and ignored
        // below), so that they are in flight together; neighbouring lanes test neighbouring candidates, so that one
        // load instruction touches few sectors
#pragma unroll
        for (int h = 0; h < kFuseCand; ++h) {                            // thread t tests q0 + h kFuseThreads + t
            const int q = min(q0 + h * kFuseThreads + tid, ncand - 1);
            const int kk = (int)((unsigned)q / (unsigned)wsz), e = q - kk * wsz;
            const int k = kk < a ? kk : kk + 1;                          // source frames only
            const int ey = (int)((unsigned)e / (unsigned)nx);
            f[h] = k * N + (y_lo + ey) * W + x_lo + (e - ey * nx);
            kp[h] = __ldcg(keep + f[h]);
            d[h] = __ldcg(dst + f[h]);
        }
        unsigned m[kFuseCand];
#pragma unroll
        for (int h = 0; h < kFuseCand; ++h) {
            const bool hit = q0 + h * kFuseThreads + tid < ncand && !kp[h] && d[h] == j;
            m[h] = __ballot_sync(0xffffffffu, hit);
            if (!hit) f[h] = -1;
            if (lane == 0) s_cnt[h][w] = __popc(m[h]);
        }
        __syncthreads();
        int total = 0;                                                   // list position: ascending q = (h, warp, lane)
        const unsigned lt = (1u << lane) - 1u;
#pragma unroll
        for (int h = 0; h < kFuseCand; ++h) {
#pragma unroll
            for (int ww = 0; ww < kFuseWarps; ++ww) {
                if (ww == w && f[h] >= 0) s_list[total + __popc(m[h] & lt)] = f[h];
                total += s_cnt[h][ww];
            }
        }
        __syncthreads();
        if (on) {
            for (int e = 0; e < total; e += kRows) {                     // kRows rows in flight, added in list order
                typename L::Raw raw[kRows];
#pragma unroll
                for (int u = 0; u < kRows; ++u)                          // (beyond the end: the last row again, not added)
                    raw[u] = L::load_raw(X + (size_t)s_list[min(e + u, total - 1)] * C + c0);
#pragma unroll
                for (int u = 0; u < kRows; ++u) {
                    float v[V];
                    L::unpack(raw[u], v);
                    const bool in = e + u < total;
#pragma unroll
                    for (int c2 = 0; c2 < V; ++c2) acc[c2] = in ? acc[c2] + v[c2] : acc[c2];
                }
            }
        }
        members += total;
        __syncthreads();                                                 // the list is rebuilt by the next round
    }
    if (on) {
        const float denom = (float)members;
#pragma unroll
        for (int c2 = 0; c2 < V; ++c2) acc[c2] = acc[c2] / denom;
        Storer<T, V>::store(out_tokens + (size_t)j * C + c0, acc);
    }
}

template <typename T, int V>
static cudaError_t launch_fuse_mean_t(const Problem& p, const Scratch& s, void* out_tokens, cudaStream_t st) {
    const int per = kFuseThreads * V;
    const int nslices = (p.C + per - 1) / per;
    const long long blocks = (long long)p.N * nslices;
    if (blocks >= (1LL << 31) || (long long)p.F * (2 * p.r + 1) * (2 * p.r + 1) >= (1LL << 31) - kFuseCand * kFuseThreads)
        return cudaErrorInvalidConfiguration;
    return launch_pdl(k_fuse_mean<T, V>, dim3((unsigned)blocks), dim3(kFuseThreads), st,
                      reinterpret_cast<const T*>(p.X), p.F, p.H, p.W, p.C, p.r, (const int*)s.hdr,
                      (const unsigned char*)s.keep, (const int*)s.dst, reinterpret_cast<T*>(out_tokens), nslices);
}

// Overwrites rows [0, N) of out_tokens (the anchor block of the compressed sequence) with the means; reads the
// anchor, keep and dst that the pass left in the scratch block.
cudaError_t launch_fuse_mean(const Problem& p, const Scratch& s, void* out_tokens, cudaStream_t st) {
    const bool vec = p.vec && reinterpret_cast<uintptr_t>(out_tokens) % 16 == 0;
    if (p.dtype == 0) return vec ? launch_fuse_mean_t<float, 4>(p, s, out_tokens, st) : launch_fuse_mean_t<float, 1>(p, s, out_tokens, st);
    return vec ? launch_fuse_mean_t<bf16_t, 8>(p, s, out_tokens, st) : launch_fuse_mean_t<bf16_t, 1>(p, s, out_tokens, st);
}

}  // namespace ttf
