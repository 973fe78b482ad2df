// Anchor Frame Selection (Eq. auto_anchor) and per-token norms, in one sweep over X and one launch.
//
// Streaming part.  A CTA owns (frame k, token group tg, channel slice q); a slice is 32 lanes x one 16-byte
// load.  Warp w walks its tokens eight at a time (eight independent 16-byte loads per lane in flight, the next
// eight prefetched before the current ones are reduced).  Each lane keeps running channel sums of its
// channels (they add up to the frame sum S_k = N x the mean token of frame k); the eight squared norms of a
// batch, restricted to the slice, are reduced over the warp with a 9-shuffle fold and stored as partials
// (consumers add the slices in slice order).
//
// Anchor part, without a second launch.  CTAs count themselves per slice; the last CTA of slice q adds the
// token-group partials into S[:, slice], forms g[slice] = sum_k S_k[slice] and the slice's share of
// <S_k, g>, |S_k|^2 and |g|^2.  Slices count themselves too; the last one adds the shares in slice order,
// takes the cosines (the 1/N and 1/(FN) of Eq. auto_anchor cancel in a cosine) and the arg max (lowest frame
// on ties), and resets the counters for the next call.  Which CTA happens to be last never changes a sum's
// order, so results are reproducible.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kNormWarps = 8;
constexpr int kNormThreads = kNormWarps * 32;
constexpr int kBatch = 8;            // tokens per warp per step

// Sum of v[u] over the warp for u = 0..7 with 9 shuffles.  On return the lanes with (lane & 3) == 0 hold the
// total of token u = 4*bit4 + 2*bit3 + bit2 of their lane index (all four lanes of a quad hold it).
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

// V consecutive fp32 values written earlier in this kernel (possibly by another CTA): L2-coherent loads
template <int V> __device__ __forceinline__ void load_f32(const float* p, float (&x)[V]);
template <> __device__ __forceinline__ void load_f32<8>(const float* p, float (&x)[8]) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p)), b = __ldcg(reinterpret_cast<const float4*>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <> __device__ __forceinline__ void load_f32<4>(const float* p, float (&x)[4]) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(p));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
}
template <> __device__ __forceinline__ void load_f32<1>(const float* p, float (&x)[1]) { x[0] = __ldcg(p); }
template <int V> __device__ __forceinline__ void store_f32(float* p, const float (&x)[V]) {
    if constexpr (V == 1) { p[0] = x[0]; }
    else {
#pragma unroll
        for (int h = 0; h < V / 4; ++h)
            reinterpret_cast<float4*>(p)[h] = make_float4(x[4 * h], x[4 * h + 1], x[4 * h + 2], x[4 * h + 3]);
    }
}

struct AnchorArgs {
    float* Sp;          // [TG, F, C] token-group partial frame sums
    float* S;           // [F, C]
    float* ssq;         // [nslice, F*N]
    float* Dp;          // [nslice, F] slice shares of <S_k, g>
    float* Qp;          // [nslice, F] slice shares of |S_k|^2
    float* Gp;          // [nslice]    slice shares of |g|^2
    float* fcos;        // [F]
    int* cnt;           // [F] survivor counters, zeroed here for the matching kernel
    int* hdr;           // header words
    int* done_slice;    // [nslice] arrival counters (zero on entry, zero again on exit)
    int* out_anchor;    // optional user copy of a*
    int mode, arg;      // anchor rule: 0 auto, 1 first, 2 last, 3 explicit frame `arg`
};

template <typename T, int V>
__global__ void __launch_bounds__(kNormThreads)
k_norm_anchor(const T* __restrict__ X, int F, int N, int C, int nslice, int TG, AnchorArgs A)
{
    using L = Loader<T, V>;
    const int q = blockIdx.x % nslice;
    const int tg = (blockIdx.x / nslice) % TG;
    const int k = blockIdx.x / (nslice * TG);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c0 = (q * 32 + lane) * V;
    const bool active = c0 < C;                 // C is a multiple of V on the vector path
    const size_t FN = (size_t)F * N;
    const int i_begin = (int)((long long)N * tg / TG), i_end = (int)((long long)N * (tg + 1) / TG);
    const T* base = X + (size_t)k * N * C + c0;

    __shared__ float sm[kNormWarps][32 * V];
    __shared__ float s_g[32 * V];
    __shared__ float s_red[kNormWarps];
    __shared__ int s_redi[kNormWarps];
    __shared__ int s_flag;

    float col[V];
#pragma unroll
    for (int v = 0; v < V; ++v) col[v] = 0.f;

    typename L::Raw cur[kBatch], nxt[kBatch];
    auto load_batch = [&](typename L::Raw (&dst)[kBatch], int i0) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int i = i0 + u;
            dst[u] = (active && i < i_end) ? L::load_raw(base + (size_t)i * C) : L::zero();
        }
    };

    int i0 = i_begin + w * kBatch;
    if (i0 < i_end) load_batch(cur, i0);
    for (; i0 < i_end; i0 += kNormWarps * kBatch) {
        const int inext = i0 + kNormWarps * kBatch;
        if (inext < i_end) load_batch(nxt, inext);
        float ss[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            float x[V];
            L::unpack(cur[u], x);
            float s = 0.f;
#pragma unroll
            for (int v = 0; v < V; ++v) { s = fmaf(x[v], x[v], s); col[v] += x[v]; }
            ss[u] = s;
        }
        const float tot = fold8(ss, lane);
        const int u = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
        if ((lane & 3) == 0 && i0 + u < i_end) A.ssq[(size_t)q * FN + (size_t)k * N + i0 + u] = tot;
#pragma unroll
        for (int uu = 0; uu < kBatch; ++uu) cur[uu] = nxt[uu];
    }

#pragma unroll
    for (int v = 0; v < V; ++v) sm[w][lane * V + v] = col[v];
    __syncthreads();
    for (int idx = tid; idx < 32 * V; idx += kNormThreads) {
        const int c = q * 32 * V + idx;
        if (c < C) {
            float s = 0.f;
#pragma unroll
            for (int ww = 0; ww < kNormWarps; ++ww) s += sm[ww][idx];
            A.Sp[((size_t)tg * F + k) * C + c] = s;
        }
    }
    if (q == 0 && tg == 0 && tid == 0) A.cnt[k] = 0;

    if (A.mode != 0) {                          // fixed anchors of Table 1 (first / last) or an explicit frame
        if (blockIdx.x == 0 && tid == 0) {
            const int a = A.mode == 1 ? 0 : (A.mode == 2 ? F - 1 : A.arg);
            A.hdr[HDR_ANCHOR] = a;
            if (A.out_anchor) *A.out_anchor = a;
        }
        return;
    }

    // ---- last CTA of this slice: frame sums, g and the slice's share of the cosine terms -----------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = (atomicAdd(&A.done_slice[q], 1) == F * TG - 1);
    __syncthreads();
    if (!s_flag) return;
    __threadfence();

    // warp w owns frames w, w+8, ...; lane owns the same V channels as in the sweep.  Four frames per warp are
    // in flight at a time.  The frame sums are written to S and read back by the thread that wrote them.
    constexpr int FB = 4;
    float gacc[V];
#pragma unroll
    for (int v = 0; v < V; ++v) gacc[v] = 0.f;
    for (int kb = w; kb < F; kb += kNormWarps * FB) {
        float acc[FB][V];
#pragma unroll
        for (int jj = 0; jj < FB; ++jj)
#pragma unroll
            for (int v = 0; v < V; ++v) acc[jj][v] = 0.f;
        for (int t2 = 0; t2 < TG; ++t2) {
#pragma unroll
            for (int jj = 0; jj < FB; ++jj) {
                const int kk = kb + jj * kNormWarps;
                if (active && kk < F) {
                    float x[V];
                    load_f32<V>(A.Sp + ((size_t)t2 * F + kk) * C + c0, x);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc[jj][v] += x[v];
                }
            }
        }
#pragma unroll
        for (int jj = 0; jj < FB; ++jj) {
            const int kk = kb + jj * kNormWarps;
            if (active && kk < F) {
                store_f32<V>(A.S + (size_t)kk * C + c0, acc[jj]);
#pragma unroll
                for (int v = 0; v < V; ++v) gacc[v] += acc[jj][v];
            }
        }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) sm[w][lane * V + v] = gacc[v];
    __syncthreads();
    for (int idx = tid; idx < 32 * V; idx += kNormThreads) {
        float g = 0.f;
#pragma unroll
        for (int ww = 0; ww < kNormWarps; ++ww) g += sm[ww][idx];
        s_g[idx] = g;                       // channels past C hold 0
    }
    __syncthreads();
    float gl[V];
#pragma unroll
    for (int v = 0; v < V; ++v) gl[v] = s_g[lane * V + v];
    for (int kb = w; kb < F; kb += kNormWarps * FB) {
        float d[FB], qq[FB];
#pragma unroll
        for (int jj = 0; jj < FB; ++jj) {
            const int kk = kb + jj * kNormWarps;
            d[jj] = 0.f; qq[jj] = 0.f;
            if (active && kk < F) {
                float x[V];
                load_f32<V>(A.S + (size_t)kk * C + c0, x);
#pragma unroll
                for (int v = 0; v < V; ++v) { d[jj] = fmaf(x[v], gl[v], d[jj]); qq[jj] = fmaf(x[v], x[v], qq[jj]); }
            }
        }
#pragma unroll
        for (int jj = 0; jj < FB; ++jj) {
            const int kk = kb + jj * kNormWarps;
            const float ds = warp_sum(d[jj]), qs = warp_sum(qq[jj]);
            if (lane == 0 && kk < F) { A.Dp[(size_t)q * F + kk] = ds; A.Qp[(size_t)q * F + kk] = qs; }
        }
    }
    if (w == 0) {
        float gg = 0.f;
#pragma unroll
        for (int v = 0; v < V; ++v) gg = fmaf(gl[v], gl[v], gg);
        gg = warp_sum(gg);
        if (lane == 0) A.Gp[q] = gg;
    }

    // ---- last slice: cosines and arg max ---------------------------------------------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag = (atomicAdd(&A.hdr[HDR_DONE_ALL], 1) == nslice - 1);
    __syncthreads();
    if (!s_flag) return;
    __threadfence();

    if (w == 0) {
        float gg = 0.f;
        for (int qq = lane; qq < nslice; qq += 32) gg += __ldcg(A.Gp + qq);
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
        if (kk < F)
            for (int qq = part; qq < nslice; qq += 8) {
                d += __ldcg(A.Dp + (size_t)qq * F + kk);
                s2 += __ldcg(A.Qp + (size_t)qq * F + kk);
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
        A.hdr[HDR_DONE_ALL] = 0;
    }
    for (int qq = tid; qq < nslice; qq += kNormThreads) A.done_slice[qq] = 0;
}

int norm_token_groups(const Problem& p) {
    // shape-only rule (the summation order must not depend on the device): enough CTAs to load-balance
    // 148 SMs, at least 64 tokens per CTA
    int tg = 1;
    while (tg < 8 && (long long)p.F * p.nslice * tg < 1024 && p.N / (tg * 2) >= 64) tg *= 2;
    return tg;
}

template <typename T, int V>
static cudaError_t launch_t(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    const int TG = norm_token_groups(p);
    AnchorArgs A;
    A.Sp = s.Sp; A.S = s.S; A.ssq = s.ssq; A.Dp = s.Dp; A.Qp = s.Qp; A.Gp = s.Gp; A.fcos = s.fcos;
    A.cnt = s.cnt; A.hdr = s.hdr; A.done_slice = s.done_slice; A.out_anchor = out_anchor;
    A.mode = p.anchor_mode; A.arg = p.anchor_arg;
    const long long blocks = (long long)p.F * p.nslice * TG;
    k_norm_anchor<T, V><<<(unsigned)blocks, kNormThreads, 0, st>>>(
        reinterpret_cast<const T*>(p.X), p.F, p.N, p.C, p.nslice, TG, A);
    return cudaGetLastError();
}

cudaError_t launch_norm_anchor(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st) {
    if (p.dtype == 0) return p.vec ? launch_t<float, 4>(p, s, out_anchor, st) : launch_t<float, 1>(p, s, out_anchor, st);
    return p.vec ? launch_t<bf16_t, 8>(p, s, out_anchor, st) : launch_t<bf16_t, 1>(p, s, out_anchor, st);
}

}  // namespace ttf
