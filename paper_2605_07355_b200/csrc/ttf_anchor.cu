// Anchor Frame Selection (Eq. auto_anchor) and per-token norms: one streaming sweep over X plus a small
// reduction kernel.
//
// k_norm_sum.  A CTA owns (frame k, token group tg) and reads whole token rows: thread t loads the 16-byte
// chunks t, t+256, ... of a row, so a CTA streams a contiguous piece of X (a batch of 4 rows = 4 x C
// elements), the next batch being prefetched while the current one is reduced.  Every thread keeps running
// sums of its own channels (no cross-thread reduction: the token-group partial of the frame sum
// S_k = N x mean token of frame k goes straight to memory) and its share of each token's squared norm, which
// is reduced over the warp with a shuffle fold and stored as one partial per (warp, token); consumers add the
// partials in a fixed order.
//
// k_anchor_pick.  One CTA per 32-channel slice adds the token-group partials into S_k[slice] (registers), forms
// g[slice] = sum_k S_k[slice] and the slice's shares of <S_k, g>, |S_k|^2, |g|^2.  The slices count
// themselves; the last one adds the shares in slice order, takes the cosines (the factors 1/N and 1/(FN) of
// Eq. auto_anchor cancel in a cosine) and the arg max (lowest frame on ties) and resets the counter.  Which
// CTA is last never changes the order of a sum, so the result is reproducible.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kNormWarps = 8;
constexpr int kNormThreads = kNormWarps * 32;
constexpr int kMaxTG = 16;           // token groups per frame (partial frame sums kept per group)
#ifndef TTF_ROWBATCH
#define TTF_ROWBATCH 4
#endif
#ifndef TTF_NORM_MINBLOCKS
#define TTF_NORM_MINBLOCKS 2
#endif
constexpr int kRowBatch = TTF_ROWBATCH;   // rows in flight per step (times two with the prefetch): 2 or 4

// Sum of v[u] over the warp for u = 0..3 with 6 shuffles; lanes with (lane & 7) == 0 hold the total of token
// u = 2*bit4 + bit3 of their lane index.
template <int NV> __device__ __forceinline__ float fold4(float (&v)[NV], int lane) {
    static_assert(NV >= 4, "fold4 needs four values");
    {
        const bool up = lane & 16;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float send = up ? v[j] : v[j + 2];
            const float keep = up ? v[j + 2] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
    }
    {
        const bool up = lane & 8;
        const float send = up ? v[0] : v[1];
        const float keep = up ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    float r = v[0];
    r += __shfl_xor_sync(0xffffffffu, r, 4);
    r += __shfl_xor_sync(0xffffffffu, r, 2);
    r += __shfl_xor_sync(0xffffffffu, r, 1);
    return r;
}

template <int V> __device__ __forceinline__ void store_f32(float* p, const float (&x)[V]) {
    if constexpr (V == 1) { p[0] = x[0]; }
    else {
#pragma unroll
        for (int h = 0; h < V / 4; ++h)
            reinterpret_cast<float4*>(p)[h] = make_float4(x[4 * h], x[4 * h + 1], x[4 * h + 2], x[4 * h + 3]);
    }
}

// CPT: 16-byte chunks per thread per row (column blocks of 256*CPT chunks are walked one after the other)
template <typename T, int V, int CPT>
__global__ void __launch_bounds__(kNormThreads, TTF_NORM_MINBLOCKS)
k_norm_sum(const T* __restrict__ X, int F, int N, int C, int TG, int ncb,
           float* __restrict__ Sp, float* __restrict__ ssq, int* __restrict__ cnt, int* __restrict__ hdr)
{
    using L = Loader<T, V>;
    pdl_launch_dependents();
    // This kernel may be scheduled while the previous call's gather still runs (it shares the scratch) or
    // while an upstream kernel still writes X: nothing is read or written before the wait.
    pdl_wait();
    trace_mark(hdr, 0, false);
    const int k = blockIdx.x / TG, tg = blockIdx.x - k * TG;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const size_t FN = (size_t)F * N;
    const int i_begin = (int)((long long)N * tg / TG), i_end = (int)((long long)N * (tg + 1) / TG);
    const T* frame = X + (size_t)k * N * C;

    for (int cb = 0; cb < ncb; ++cb) {
        int c0[CPT];
        bool on[CPT];
#pragma unroll
        for (int j = 0; j < CPT; ++j) {
            c0[j] = ((cb * CPT + j) * kNormThreads + tid) * V;
            on[j] = c0[j] < C;                       // C is a multiple of V on the vector path
        }
        float col[CPT][V];
#pragma unroll
        for (int j = 0; j < CPT; ++j)
#pragma unroll
            for (int v = 0; v < V; ++v) col[j][v] = 0.f;

        typename L::Raw cur[kRowBatch][CPT], nxt[kRowBatch][CPT];
        auto load_batch = [&](typename L::Raw (&d)[kRowBatch][CPT], int i0) {
#pragma unroll
            for (int u = 0; u < kRowBatch; ++u)
#pragma unroll
                for (int j = 0; j < CPT; ++j)
                    d[u][j] = (on[j] && i0 + u < i_end) ? L::load_raw_cg(frame + (size_t)(i0 + u) * C + c0[j]) : L::zero();
        };
        if (i_begin < i_end) load_batch(cur, i_begin);
        for (int i0 = i_begin; i0 < i_end; i0 += kRowBatch) {
            if (i0 + kRowBatch < i_end) load_batch(nxt, i0 + kRowBatch);
            float ss[kRowBatch];
#pragma unroll
            for (int u = 0; u < kRowBatch; ++u) {
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < CPT; ++j) {
                    float x[V];
                    L::unpack(cur[u][j], x);
#pragma unroll
                    for (int v = 0; v < V; ++v) { s = fmaf(x[v], x[v], s); col[j][v] += x[v]; }
                }
                ss[u] = s;
            }
            float tot;
            int u;
            if constexpr (kRowBatch == 4) {
                tot = fold4<kRowBatch>(ss, lane);
                u = ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1);
            } else {
                const bool up = lane & 16;
                tot = (up ? ss[1] : ss[0]) + __shfl_xor_sync(0xffffffffu, up ? ss[0] : ss[1], 16);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
                u = (lane >> 4) & 1;
            }
            if ((lane & (kRowBatch == 4 ? 7 : 15)) == 0 && i0 + u < i_end) ssq[(size_t)(cb * kNormWarps + w) * FN + (size_t)k * N + i0 + u] = tot;
#pragma unroll
            for (int uu = 0; uu < kRowBatch; ++uu)
#pragma unroll
                for (int j = 0; j < CPT; ++j) cur[uu][j] = nxt[uu][j];
        }
#pragma unroll
        for (int j = 0; j < CPT; ++j)
            if (on[j]) store_f32<V>(Sp + ((size_t)tg * F + k) * C + c0[j], col[j]);
    }
    if (tg == 0 && tid == 0) cnt[k] = 0;            // survivor counters start at zero for the matching kernel
    trace_mark(hdr, 0, true);
}

int norm_token_groups(const Problem& p) {
    // shape-only rule (the order of every sum must not depend on the device): F * TG close to, and not above,
    // 296 CTAs (two per SM on a 148-SM part), at least 8 rows per CTA, at most kMaxTG groups
    long long tg = 296 / p.F;
    if (tg > p.N / 8) tg = p.N / 8;
    if (tg > kMaxTG) tg = kMaxTG;
    if (tg < 1) tg = 1;
    return (int)tg;
}

template <typename T, int V>
static cudaError_t launch_sum_t(const Problem& p, const Scratch& s, cudaStream_t st) {
    const int TG = norm_token_groups(p);
    const unsigned blocks = (unsigned)((long long)p.F * TG);
    const T* X = reinterpret_cast<const T*>(p.X);
    if (p.cpt == 1)
        return launch_pdl(k_norm_sum<T, V, 1>, dim3(blocks), dim3(kNormThreads), st, X, p.F, p.N, p.C, TG, p.ncb,
                          s.Sp, s.ssq, s.cnt, s.hdr);
    return launch_pdl(k_norm_sum<T, V, 2>, dim3(blocks), dim3(kNormThreads), st, X, p.F, p.N, p.C, TG, p.ncb,
                      s.Sp, s.ssq, s.cnt, s.hdr);
}

// ---------------------------------------------------------------------------------------------------------
constexpr int kPickFB = 2;           // frames per thread held in registers
constexpr int kPickLanes = 8;        // threads across a slice (each V channels); 32 frame rows per CTA

struct PickArgs {
    const float* Sp;    // [TG, F, C]
    float* Dp;          // [nsl, F] slice shares of <S_k, g>
    float* Qp;          // [nsl, F] slice shares of |S_k|^2
    float* Gp;          // [nsl]    slice shares of |g|^2
    float* fcos;        // [F]
    int* hdr;
    int* out_anchor;    // optional user copy of a*
    int mode, arg;      // anchor rule: 0 auto, 1 first, 2 last, 3 explicit frame `arg`
};

template <int V> __device__ __forceinline__ void load_f32(const float* p, float (&x)[V]);
template <> __device__ __forceinline__ void load_f32<4>(const float* p, float (&x)[4]) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
}
template <> __device__ __forceinline__ void load_f32<1>(const float* p, float (&x)[1]) { x[0] = __ldcg(p); }

// A CTA owns a slice of 8*V channels: thread = (frame row 0..31, lane 0..7 with V channels).
// V = 4 when C is a multiple of 4 (16-byte loads of the fp32 partial sums), else 1.
template <int V>
__global__ void __launch_bounds__(kNormThreads)
k_anchor_pick(int F, int C, int TG, int nsl, PickArgs A)
{
    pdl_launch_dependents();
    const int q = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int cl = tid & (kPickLanes - 1), row = tid / kPickLanes;
    __shared__ float s_gp[kNormThreads / kPickLanes][kPickLanes * V];
    __shared__ float s_red[kNormWarps];
    __shared__ int s_redi[kNormWarps];
    __shared__ int s_flag;

    trace_mark(A.hdr, 1, false);
    pdl_wait();                                      // the sweep's partial sums are complete and visible
    trace_mark(A.hdr, 4, false);
    if (A.mode != 0) {                               // fixed anchors of Table 1 (first / last) or an explicit frame
        if (q == 0 && tid == 0) {
            const int a = A.mode == 1 ? 0 : (A.mode == 2 ? F - 1 : A.arg);
            A.hdr[HDR_ANCHOR] = a;
            if (A.out_anchor) *A.out_anchor = a;
        }
        return;
    }

    const int c0 = (q * kPickLanes + cl) * V;
    const bool active = c0 < C;                      // C % V == 0
    constexpr int kRows = kNormThreads / kPickLanes; // 32
    const bool resident = F <= kRows * kPickFB;      // all frame sums of this thread stay in registers

    // S_k[c] = sum over token groups (ascending), for the frames row, row+16, ... of this thread
    auto frame_sums = [&](int kb, float (&acc)[kPickFB][V]) {
#pragma unroll
        for (int jj = 0; jj < kPickFB; ++jj)
#pragma unroll
            for (int v = 0; v < V; ++v) acc[jj][v] = 0.f;
#pragma unroll
        for (int t2 = 0; t2 < kMaxTG; ++t2) {       // all loads of the batch are independent and issued together
#pragma unroll
            for (int jj = 0; jj < kPickFB; ++jj) {
                const int kk = kb + jj * kRows;
                if (active && kk < F && t2 < TG) {
                    float x[V];
                    load_f32<V>(A.Sp + ((size_t)t2 * F + kk) * C + c0, x);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[jj][v] += x[v];
                }
            }
        }
    };

    float acc[kPickFB][V];
    float gacc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) gacc[v] = 0.f;
    // trip counts are the same for every thread (the shuffles below need whole warps); frames past F add zeros
    for (int kb0 = 0; kb0 < F; kb0 += kRows * kPickFB) {
        const int kb = kb0 + row;
        frame_sums(kb, acc);
#pragma unroll
        for (int jj = 0; jj < kPickFB; ++jj)
#pragma unroll
            for (int v = 0; v < V; ++v) gacc[v] += acc[jj][v];      // frames past F contributed zeros
    }
#pragma unroll
    for (int v = 0; v < V; ++v) s_gp[row][cl * V + v] = gacc[v];
    __syncthreads();
    float gl[V];                                     // g[c] = sum_k S_k[c], rows combined in row order
#pragma unroll
    for (int v = 0; v < V; ++v) {
        float g = 0.f;
#pragma unroll
        for (int rr = 0; rr < kRows; ++rr) g += s_gp[rr][cl * V + v];
        gl[v] = g;
    }
    for (int kb0 = 0; kb0 < F; kb0 += kRows * kPickFB) {
        const int kb = kb0 + row;
        if (!resident) frame_sums(kb, acc);
#pragma unroll
        for (int jj = 0; jj < kPickFB; ++jj) {
            const int kk = kb + jj * kRows;
            float d = 0.f, qq = 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) { d = fmaf(acc[jj][v], gl[v], d); qq = fmaf(acc[jj][v], acc[jj][v], qq); }
#pragma unroll
            for (int o = kPickLanes / 2; o > 0; o >>= 1) {
                d += __shfl_xor_sync(0xffffffffu, d, o);
                qq += __shfl_xor_sync(0xffffffffu, qq, o);
            }
            if (cl == 0 && kk < F) { A.Dp[(size_t)q * F + kk] = d; A.Qp[(size_t)q * F + kk] = qq; }
        }
    }
    if (w == 0) {
        float gg = 0.f;
        if (row == 0) {
#pragma unroll
            for (int v = 0; v < V; ++v) gg = fmaf(gl[v], gl[v], gg);
        }
        gg = warp_sum(gg);                           // the lanes of rows 1..3 add zeros
        if (lane == 0) A.Gp[q] = gg;
    }

    // ---- last slice: cosines and arg max ---------------------------------------------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = (atomicAdd(&A.hdr[HDR_DONE_ALL], 1) == nsl - 1);
    __syncthreads();
    trace_mark(A.hdr, 4, true);
    if (!s_flag) return;
    __threadfence();

    if (w == 0) {
        float gg = 0.f;
        for (int qq = lane; qq < nsl; qq += 32) gg += __ldcg(A.Gp + qq);
        gg = warp_sum(gg);
        if (lane == 0) s_red[0] = 1.0f / fmaxf(sqrtf(gg), kNormFloor);
    }
    __syncthreads();
    const float ginv = s_red[0];
    __syncthreads();
    // thread = (frame, part): part p of 8 adds slices p, p+8, ...; the 8 parts are combined by shuffles
    float best = -INFINITY;
    int idx = 0x7fffffff;
    for (int kb = 0; kb < F; kb += kNormThreads / 8) {
        const int kk = kb + (tid >> 3), part = tid & 7;
        float d = 0.f, s2 = 0.f;
        if (kk < F) {
#pragma unroll 16
            for (int qq = part; qq < nsl; qq += 8) {
                d += __ldcg(A.Dp + (size_t)qq * F + kk);
                s2 += __ldcg(A.Qp + (size_t)qq * F + kk);
            }
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
            d += __shfl_xor_sync(0xffffffffu, d, o);
            s2 += __shfl_xor_sync(0xffffffffu, s2, o);
        }
        if (kk < F && part == 0) {
            const float v = d * ginv * (1.0f / fmaxf(sqrtf(s2), kNormFloor));
            A.fcos[kk] = v;
            if (v > best || idx == 0x7fffffff) { best = v; idx = kk; }   // ascending kk per thread: first max stays
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (oi != 0x7fffffff && (idx == 0x7fffffff || ob > best || (ob == best && oi < idx))) { best = ob; idx = oi; }
    }
    if (lane == 0) { s_red[w] = best; s_redi[w] = idx; }
    __syncthreads();
    if (tid == 0) {
        float b = s_red[0];
        int bi = s_redi[0];
        for (int ww = 1; ww < kNormWarps; ++ww) {
            const float ob = s_red[ww];
            const int oi = s_redi[ww];
            if (oi != 0x7fffffff && (bi == 0x7fffffff || ob > b || (ob == b && oi < bi))) { b = ob; bi = oi; }
        }
        A.hdr[HDR_ANCHOR] = bi;
        if (A.out_anchor) *A.out_anchor = bi;
        A.hdr[HDR_DONE_ALL] = 0;                     // ready for the next call
    }
    trace_mark(A.hdr, 1, true);
}

cudaError_t launch_norm_anchor(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    cudaError_t e;
    if (p.dtype == 0) e = p.vec ? launch_sum_t<float, 4>(p, s, st) : launch_sum_t<float, 1>(p, s, st);
    else e = p.vec ? launch_sum_t<bf16_t, 8>(p, s, st) : launch_sum_t<bf16_t, 1>(p, s, st);
    if (e != cudaSuccess) return e;
    PickArgs A;
    A.Sp = s.Sp; A.Dp = s.Dp; A.Qp = s.Qp; A.Gp = s.Gp; A.fcos = s.fcos; A.hdr = s.hdr;
    A.out_anchor = out_anchor; A.mode = p.anchor_mode; A.arg = p.anchor_arg;
    const int TG = norm_token_groups(p);
    const bool fixed = p.anchor_mode != 0;
    if (p.C % 4 == 0)
        return launch_pdl(k_anchor_pick<4>, dim3(fixed ? 1 : p.nsl), dim3(kNormThreads), st, p.F, p.C, TG, p.nsl, A);
    return launch_pdl(k_anchor_pick<1>, dim3(fixed ? 1 : p.nsl), dim3(kNormThreads), st, p.F, p.C, TG, p.nsl, A);
}

}  // namespace ttf
