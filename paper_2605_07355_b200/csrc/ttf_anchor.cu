// Anchor Frame Selection (Eq. auto_anchor) and per-token norms: one streaming sweep over X plus a small
// statistics kernel whose last CTA takes the arg max (resolve_anchor).
//
// k_norm_sum.  A CTA owns (frame k, channel slice q); a slice is LS = 32 lanes x one 16-byte load (512 bytes
// of every token row; the CTAs of neighbouring slices run side by side, so DRAM sees whole rows).  The
// 256 / LS row groups (warps) of a CTA walk the tokens of the frame interleaved, eight tokens per thread in
// flight and the next eight prefetched.  A thread keeps running sums of its channels; the row groups are combined through
// shared memory in a fixed order and give the frame sum S_k[slice] (= N x mean token of frame k) directly.
// The squared norm of every token restricted to one warp's 32 lanes is reduced with a 9-shuffle fold and
// stored as a partial (consumers add the partials in plane order).
//
// k_frame_stats.  One CTA per 128-channel slice forms g[slice] = sum_k S_k[slice] and the slice's shares of
// <S_k, g>, |S_k|^2 and |g|^2 (the factors 1/N and 1/(FN) of Eq. auto_anchor cancel in a cosine).  Every order
// of summation is fixed, so the result is reproducible.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kNormWarps = 8;
constexpr int kNormThreads = kNormWarps * 32;
constexpr int kBatch = 8;            // tokens per thread in flight (times two with the prefetch)

// Sum of v[u] over the warp for u = 0..7 with 9 shuffles.  On return the lanes with (lane & 3) == 0 hold the
// total of token u = 4*bit4 + 2*bit3 + bit2 of their lane index.
__device__ __forceinline__ float fold8(float (&v)[8], int lane) {
    {
        const bool up = lane & 16;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float send = up ? v[j] : v[j + 4];
            const float keep = up ? v[j + 4] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
    }
    {
        const bool up = lane & 8;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float send = up ? v[j] : v[j + 2];
            const float keep = up ? v[j + 2] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
    }
    {
        const bool up = lane & 4;
        const float send = up ? v[0] : v[1];
        const float keep = up ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    float r = v[0];
    r += __shfl_xor_sync(0xffffffffu, r, 2);
    r += __shfl_xor_sync(0xffffffffu, r, 1);
    return r;
}

// LS: lanes across a slice (32 or 64); RG = 256 / LS row groups walk the tokens interleaved.
// NORMS: also store the per-token partial squared norms (only the CUDA-core matching kernel reads them).
template <typename T, int V, int LS, bool NORMS>
__global__ void __launch_bounds__(kNormThreads)
k_norm_sum(const T* __restrict__ X, int F, int N, int C, int nq,
           float* __restrict__ S, float* __restrict__ ssq, int* __restrict__ cnt, int* __restrict__ hdr,
           int chain)
{
    using L = Loader<T, V>;
    constexpr int RG = kNormThreads / LS;
    constexpr int WPS = LS / 32;                    // warps across a slice = norm planes per slice
    pdl_launch_dependents();
    // This kernel may be scheduled while the kernel before it in the stream still runs.  Normally that kernel may be
    // anything (the previous call's gather, which shares the scratch, or an upstream kernel that still writes X), so
    // nothing is read or written before the wait.  Inside a chain of clips of one batch the predecessor is known: the
    // gather of the previous clip, which works on another scratch block and another clip; then the sweep runs beside
    // it, and one CTA waits for it before it exits, so that "this sweep has completed" still implies "everything
    // before it has completed" for the kernels that follow.  (One CTA, not all: a CTA that waits keeps its place on
    // the SM, and the CTAs of the sweep that have not started yet need those places.)
    if (!chain) pdl_wait();
    trace_mark(hdr, 0, false);
    if (chain) trace_mark(hdr, 15, false);
    const int k = blockIdx.x / nq, q = blockIdx.x - k * nq;
    const int tid = threadIdx.x, lane = tid & 31;
    const int ls = tid & (LS - 1), rg = tid / LS;
    const int wcol = ls >> 5;
    const size_t FN = (size_t)F * N;
    const int c0 = (q * LS + ls) * V;
    const bool active = c0 < C;                     // C is a multiple of V on the vector path
    const T* base = X + (size_t)k * N * C + c0;
    float* plane = ssq + (size_t)(q * WPS + wcol) * FN + (size_t)k * N;

    __shared__ float sm[RG][LS * V];
    float col[V];
#pragma unroll
    for (int v = 0; v < V; ++v) col[v] = 0.f;

    // thread's tokens: rg, rg + RG, rg + 2 RG, ...; a batch is kBatch of them
    typename L::Raw cur[kBatch], nxt[kBatch];
    auto load_batch = [&](typename L::Raw (&d)[kBatch], int i0) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = i0 + u * RG;
            d[u] = (active && i < N) ? L::load_raw_cg(base + (size_t)i * C) : L::zero();
        }
    };
    if (rg < N) load_batch(cur, rg);
    for (int i0 = rg; i0 < N; i0 += RG * kBatch) {
        if (i0 + RG * kBatch < N) load_batch(nxt, i0 + RG * kBatch);
        float ss[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            float x[V];
            L::unpack(cur[u], x);
            float s = 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (NORMS) s = fmaf(x[v], x[v], s);
                col[v] += x[v];
            }
            ss[u] = s;
        }
        if (NORMS) {
#pragma unroll
            for (int h = 0; h < kBatch / 8; ++h) {
                float part[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) part[e] = ss[h * 8 + e];
                const float tot = fold8(part, lane);
                const int u = h * 8 + ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
                if ((lane & 3) == 0 && i0 + u * RG < N) plane[i0 + u * RG] = tot;
            }
        }
#pragma unroll
        for (int uu = 0; uu < kBatch; ++uu) cur[uu] = nxt[uu];
    }

#pragma unroll
    for (int v = 0; v < V; ++v) sm[rg][ls * V + v] = col[v];
    __syncthreads();
    for (int idx = tid; idx < LS * V; idx += kNormThreads) {
        const int c = q * LS * V + idx;
        if (c < C) {
            float s = 0.f;
#pragma unroll
            for (int r2 = 0; r2 < RG; ++r2) s += sm[r2][idx];
            if (in_bounds(hdr, 1, (long long)k * C + c, (long long)F * C)) S[(size_t)k * C + c] = s;
        }
    }
    if (q == 0 && tid == 0) cnt[k] = 0;             // survivor counters start at zero for the matching kernel
    if (blockIdx.x == 0 && tid == 0) hdr[HDR_ERROR] = 0;   // the error word reports on this call only
    if (chain && blockIdx.x == 0) pdl_wait();
    trace_mark(hdr, 0, true);
}

template <typename T, int V>
static cudaError_t launch_sum_t(const Problem& p, const Scratch& s, cudaStream_t st) {
    const T* X = reinterpret_cast<const T*>(p.X);
    const unsigned blocks = (unsigned)((long long)p.F * p.nq);
    const dim3 g(blocks), b(kNormThreads);
    if (!needs_sweep_norms(p))
        return launch_ex(true, 0, k_norm_sum<T, V, 32, false>, g, b, st, X, p.F, p.N, p.C, p.nq, s.S,
                         s.ssq, s.cnt, s.hdr, p.chain);
    return launch_ex(true, 0, k_norm_sum<T, V, 32, true>, g, b, st, X, p.F, p.N, p.C, p.nq, s.S, s.ssq,
                     s.cnt, s.hdr, p.chain);
}

// ---------------------------------------------------------------------------------------------------------
constexpr int kStatFB = 4;           // frames per thread held in registers (8 warps x 4 = 32 frames)

template <int V> __device__ __forceinline__ void load_f32(const float* p, float (&x)[V]);
template <> __device__ __forceinline__ void load_f32<4>(const float* p, float (&x)[4]) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
}
template <> __device__ __forceinline__ void load_f32<1>(const float* p, float (&x)[1]) { x[0] = __ldcg(p); }

// A CTA owns a slice of kStatSub*32*V channels: warp = frame row (frames w, w+8, ...), lane = V channels in each
// of the kStatSub sub-slices.  V = 4 when C is a multiple of 4 (16-byte loads of the fp32 frame sums), else 1.
constexpr int kStatSub = 1;

template <int V>
__global__ void __launch_bounds__(kNormThreads)
k_frame_stats(const float* S, int F, int C, int nsl, float* Dp, float* Qp, float* Gp, int* hdr, int* out_anchor)
{
    pdl_launch_dependents();
    trace_mark(hdr, 1, false);
    pdl_wait();                                      // the sweep's frame sums are complete and visible
    trace_mark(hdr, 4, false);
    const int q = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    constexpr int NV = kStatSub * V;                 // channels per lane
    __shared__ float s_gp[kNormWarps][32 * NV];
    int c0[kStatSub];
    bool on[kStatSub];
#pragma unroll
    for (int sb = 0; sb < kStatSub; ++sb) {
        c0[sb] = ((q * kStatSub + sb) * 32 + lane) * V;
        on[sb] = c0[sb] < C;                         // C % V == 0
    }
    const bool resident = F <= kNormWarps * kStatFB; // this thread's frame sums all stay in registers

    auto load_frames = [&](int kb, float (&acc)[kStatFB][NV]) {
#pragma unroll
        for (int jj = 0; jj < kStatFB; ++jj) {
            const int kk = kb + jj * kNormWarps;
#pragma unroll
            for (int sb = 0; sb < kStatSub; ++sb) {
                float x[V];
                if (on[sb] && kk < F) load_f32<V>(S + (size_t)kk * C + c0[sb], x);
                else {
#pragma unroll
                    for (int v = 0; v < V; ++v) x[v] = 0.f;
                }
#pragma unroll
                for (int v = 0; v < V; ++v) acc[jj][sb * V + v] = x[v];
            }
        }
    };

    float acc[kStatFB][NV];
    float gacc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) gacc[v] = 0.f;
    for (int kb = w; kb < F; kb += kNormWarps * kStatFB) {
        load_frames(kb, acc);
#pragma unroll
        for (int jj = 0; jj < kStatFB; ++jj)
#pragma unroll
            for (int v = 0; v < NV; ++v) gacc[v] += acc[jj][v];
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) s_gp[w][lane * NV + v] = gacc[v];
    __syncthreads();
    float gl[NV];                                    // g[c] = sum_k S_k[c], warps combined in warp order
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        float g = 0.f;
#pragma unroll
        for (int ww = 0; ww < kNormWarps; ++ww) g += s_gp[ww][lane * NV + v];
        gl[v] = g;
    }
    for (int kb = w; kb < F; kb += kNormWarps * kStatFB) {     // trip count is uniform inside a warp
        if (!resident) load_frames(kb, acc);
#pragma unroll
        for (int jj = 0; jj < kStatFB; ++jj) {
            const int kk = kb + jj * kNormWarps;
            float d = 0.f, qq = 0.f;
#pragma unroll
            for (int v = 0; v < NV; ++v) { d = fmaf(acc[jj][v], gl[v], d); qq = fmaf(acc[jj][v], acc[jj][v], qq); }
            d = warp_sum(d);
            qq = warp_sum(qq);
            if (lane < kStatReplicas && kk < F) {             // every lane holds the sums: one lane per replica
                Dp[((size_t)lane * nsl + q) * F + kk] = d;
                Qp[((size_t)lane * nsl + q) * F + kk] = qq;
            }
        }
    }
    if (w == 0) {
        float gg = 0.f;
#pragma unroll
        for (int v = 0; v < NV; ++v) gg = fmaf(gl[v], gl[v], gg);
        gg = warp_sum(gg);
        if (lane < kStatReplicas) Gp[(size_t)lane * nsl + q] = gg;
    }

    // The CTA that finishes last takes the arg max over the frames (Eq. auto_anchor) for the whole clip, so that the
    // CTAs of the matching kernel only read one word instead of each repeating the search while they hold most of an
    // SM.  The arrival counter is left at zero for the next call.
    __shared__ int s_last;
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        s_last = atomicAdd(hdr + HDR_DONE_ALL, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (s_last) {
        __threadfence();
        AnchorSrc src;
        src.Dp = Dp; src.Qp = Qp; src.Gp = Gp; src.nsl = nsl; src.fixed = -1; src.from_hdr = 0; src.hdr = hdr;
        src.out_anchor = out_anchor;
        const int a = resolve_anchor(src, F);
        if (tid == 0) {
            hdr[HDR_ANCHOR] = a;
            if (out_anchor) *out_anchor = a;
            hdr[HDR_DONE_ALL] = 0;
        }
    }
    trace_mark(hdr, 1, true);
}

// ---------------------------------------------------------------------------------------------------------
// The same statistics as ONE thread-block cluster of 8 CTAs, for clips of at most 4096 channels and 256 frames (the
// frame sums of 32 / 64 / 128 frames at 4 / 2 / 1 slices of 128 channels per CTA stay in registers; longer clips are
// fetched a second time for the second step).  A grid of
// independent CTAs has to go through global memory, a fence and an arrival counter before one of them can take
// the arg max, which is five to six dependent round trips after the sweep; here every CTA fetches all of its
// frame sums in one round trip, the per-frame shares of <S_k, g>, |S_k|^2 and |g|^2 go to rank 0 through
// distributed shared memory, and rank 0 takes the arg max after one cluster barrier (7.2 -> 4.8 us per launch on
// the 8B-shaped clip, 42.1 -> 37.7 us per clip with one clip in flight).  Every order of summation is fixed
// (slices inside a CTA, then ranks), so the result is reproducible; it may differ in the last bits from the grid
// kernel's, which adds the same terms in another fixed order.
constexpr int kStatCluster = 8;

__device__ __forceinline__ uint32_t stat_cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void stat_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void stat_st_cluster(const float* local, uint32_t rank, float v) {
    uint32_t remote;
    const uint32_t l = static_cast<uint32_t>(__cvta_generic_to_shared(local));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(l), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

constexpr int kStatClusterMaxF = 256;     // frames the cluster kernel takes (shares of all frames live in shared memory)

template <int SL>     // slices of 128 channels per CTA; FB = 16 / SL frames per thread and chunk (warp w owns frames w, w + 8, ...)
__global__ void __launch_bounds__(kNormThreads)
k_frame_stats_cluster(const float* S, int F, int C, int nsl, int* hdr, int* out_anchor)
{
    constexpr int FB = 16 / SL;
    constexpr int CHUNK = kNormWarps * FB;           // frames per chunk: 32 / 64 / 128
    __shared__ float4 s_g[SL][kNormWarps][32];
    __shared__ float s_D[kStatClusterMaxF], s_Q[kStatClusterMaxF], s_G;
    __shared__ float s_x[kStatCluster - 1][2 * kStatClusterMaxF + 1];      // what the other ranks send (rank 0 only)
    __shared__ float s_best[kNormWarps];
    __shared__ int s_idx[kNormWarps];
    pdl_launch_dependents();
    trace_mark(hdr, 1, false);
    pdl_wait();                                      // the sweep's frame sums are complete and visible
    trace_mark(hdr, 4, false);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int rank = (int)stat_cluster_rank();
    const bool one_chunk = F <= CHUNK;               // then the frame sums stay in registers for the second step

    // the frame sums of one chunk of frames: one round trip
    float4 v[SL][FB];
    auto load_chunk = [&](int k0) {
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) {
            const int q = rank + sl * kStatCluster;
            const int c0 = (q * 32 + lane) * 4;
#pragma unroll
            for (int jj = 0; jj < FB; ++jj) {
                const int kk = k0 + w + jj * kNormWarps;
                v[sl][jj] = (q < nsl && c0 < C && kk < F) ? __ldcg(reinterpret_cast<const float4*>(S + (size_t)kk * C + c0))
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    };
    // step 1: g[c] = sum_k S_k[c] over all frames (chunks in order, then the warps in warp order)
    float4 gacc[SL];
#pragma unroll
    for (int sl = 0; sl < SL; ++sl) gacc[sl] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = 0; k0 < F; k0 += CHUNK) {
        load_chunk(k0);
#pragma unroll
        for (int sl = 0; sl < SL; ++sl)
#pragma unroll
            for (int jj = 0; jj < FB; ++jj) {
                gacc[sl].x += v[sl][jj].x; gacc[sl].y += v[sl][jj].y; gacc[sl].z += v[sl][jj].z; gacc[sl].w += v[sl][jj].w;
            }
    }
#pragma unroll
    for (int sl = 0; sl < SL; ++sl) s_g[sl][w][lane] = gacc[sl];
    __syncthreads();
    float4 gl[SL];
#pragma unroll
    for (int sl = 0; sl < SL; ++sl) {
        float4 g = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int ww = 0; ww < kNormWarps; ++ww) { const float4 t = s_g[sl][ww][lane]; g.x += t.x; g.y += t.y; g.z += t.z; g.w += t.w; }
        gl[sl] = g;
    }
    // step 2: this CTA's shares of <S_k, g> and |S_k|^2 for every frame, slices in order
    for (int k0 = 0; k0 < F; k0 += CHUNK) {
        if (!one_chunk) load_chunk(k0);              // (a second round trip per chunk for clips of several chunks)
#pragma unroll
        for (int jj = 0; jj < FB; ++jj) {
            float d = 0.f, qq = 0.f;
#pragma unroll
            for (int sl = 0; sl < SL; ++sl) {
                const float4 x = v[sl][jj], g = gl[sl];
                d = fmaf(x.x, g.x, d); d = fmaf(x.y, g.y, d); d = fmaf(x.z, g.z, d); d = fmaf(x.w, g.w, d);
                qq = fmaf(x.x, x.x, qq); qq = fmaf(x.y, x.y, qq); qq = fmaf(x.z, x.z, qq); qq = fmaf(x.w, x.w, qq);
            }
            d = warp_sum(d);
            qq = warp_sum(qq);
            const int kk = k0 + w + jj * kNormWarps;
            if (lane == 0 && kk < F) { s_D[kk] = d; s_Q[kk] = qq; }
        }
    }
    if (w == 0) {
        float gg = 0.f;
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) {
            const float4 g = gl[sl];
            gg = fmaf(g.x, g.x, gg); gg = fmaf(g.y, g.y, gg); gg = fmaf(g.z, g.z, gg); gg = fmaf(g.w, g.w, gg);
        }
        gg = warp_sum(gg);
        if (lane == 0) s_G = gg;
    }
    __syncthreads();
    if (rank > 0) {                                  // hand the shares to rank 0
        for (int i = tid; i < 2 * F + 1; i += kNormThreads)
            stat_st_cluster(&s_x[rank - 1][i], 0, i < F ? s_D[i] : (i < 2 * F ? s_Q[i - F] : s_G));
    }
    __syncthreads();
    stat_cluster_sync();
    if (rank == 0) {
        // Eq. (auto_anchor): a* = arg max_k <S_k, g> / (|S_k| |g|), lowest frame on ties; ranks added in rank order
        float best = -INFINITY;
        int idx = 0x7fffffff;
        if (tid < F) {                               // F <= kStatClusterMaxF = the CTA's 256 threads
            float D = s_D[tid], Q = s_Q[tid], G = s_G;
            for (int r = 0; r < kStatCluster - 1; ++r) { D += s_x[r][tid]; Q += s_x[r][F + tid]; G += s_x[r][2 * F]; }
            best = D * (1.0f / fmaxf(sqrtf(G), kNormFloor)) * (1.0f / fmaxf(sqrtf(Q), kNormFloor));
            idx = tid;
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
            for (int ww = 1; ww < kNormWarps; ++ww)
                if (s_idx[ww] != 0x7fffffff && (idx == 0x7fffffff || s_best[ww] > best || (s_best[ww] == best && s_idx[ww] < idx))) {
                    best = s_best[ww]; idx = s_idx[ww];
                }
            hdr[HDR_ANCHOR] = idx;
            if (out_anchor) *out_anchor = idx;
        }
    }
    trace_mark(hdr, 1, true);
}

template <int SL>
static cudaError_t launch_stats_cluster_t(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kStatCluster); cfg.blockDim = dim3(kNormThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kStatCluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, k_frame_stats_cluster<SL>, (const float*)s.S, p.F, p.C, p.nsl, s.hdr, out_anchor);
}

// What the sweep leaves behind besides its sums, for calls that need no sweep (a fixed anchor and a matching kernel
// that takes the token norms itself): survivor counters at zero, error word cleared.
__global__ void __launch_bounds__(256)
k_begin_call(int F, int* __restrict__ cnt, int* __restrict__ hdr)
{
    pdl_launch_dependents();
    pdl_wait();                                      // the previous call's gather may still read the counters
    for (int k = threadIdx.x; k < F; k += 256) cnt[k] = 0;
    if (threadIdx.x == 0) hdr[HDR_ERROR] = 0;
}

cudaError_t launch_norm_sum(const Problem& p, const Scratch& s, cudaStream_t st) {
    if (p.anchor_mode != 0 && !needs_sweep_norms(p))           // Eq. (auto_anchor) is not evaluated: no pass over X
        return launch_ex(true, 0, k_begin_call, dim3(1), dim3(256), st, p.F, s.cnt, s.hdr);
    if (p.dtype == 0) return p.vec ? launch_sum_t<float, 4>(p, s, st) : launch_sum_t<float, 1>(p, s, st);
    return p.vec ? launch_sum_t<bf16_t, 8>(p, s, st) : launch_sum_t<bf16_t, 1>(p, s, st);
}

cudaError_t launch_frame_stats(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    if (p.anchor_mode != 0) return cudaSuccess;                // fixed anchors need no statistics
    // The single-cluster kernel is the shorter one (4.9 against 7.2 us on a 32-frame clip of 4096 channels) and takes
    // the call whenever it can, with one exception that was measured: short clips with four or more clips in flight.
    // A cluster starts only when eight CTA slots of one GPC are free at the same moment, and on a GPU that is full of
    // other clips' kernels that wait costs more than the kernel saves (8B-shaped clip, eight in flight: 30.3 us per
    // clip with the cluster kernel, 29.8 with the grid kernel; two in flight: 33.9 against 35.0; 128-frame clip, eight
    // in flight: 107.9 against 110.1, the grid kernel's time grows with F).
    const bool crowded = p.overlapped >= 4 && p.F <= 32;
    if (!crowded && p.C % 4 == 0 && p.nsl <= 4 * kStatCluster && p.F <= kStatClusterMaxF) {
        const int sl = (p.nsl + kStatCluster - 1) / kStatCluster;          // slices per CTA: 1 .. 4
        if (sl <= 1) return launch_stats_cluster_t<1>(p, s, out_anchor, st);
        if (sl <= 2) return launch_stats_cluster_t<2>(p, s, out_anchor, st);
        return launch_stats_cluster_t<4>(p, s, out_anchor, st);
    }
    if (p.C % 4 == 0)
        return launch_pdl(k_frame_stats<4>, dim3(p.nsl), dim3(kNormThreads), st, (const float*)s.S, p.F, p.C, p.nsl,
                          s.Dp, s.Qp, s.Gp, s.hdr, out_anchor);
    return launch_pdl(k_frame_stats<1>, dim3(p.nsl), dim3(kNormThreads), st, (const float*)s.S, p.F, p.C, p.nsl,
                      s.Dp, s.Qp, s.Gp, s.hdr, out_anchor);
}

}  // namespace ttf
