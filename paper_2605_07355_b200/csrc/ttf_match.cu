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
#include "ttf_match_mma.cuh"

namespace ttf {

constexpr int kMatchWarps = 8;

template <typename T, int V>
__global__ void __launch_bounds__(kMatchWarps * 32)
k_match_generic(const T* __restrict__ X, int F, int H, int W, int C, int r, float t, int fchunk, int nslice,
                AnchorSrc asrc, const float* __restrict__ ssq,
                float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep,
                int* __restrict__ cnt)
{
    pdl_launch_dependents();
    pdl_wait();                                  // norms and the frame statistics are complete
    const int N = H * W;
    const int i = blockIdx.x % N;
    const int chunk = blockIdx.x / N;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int a = resolve_anchor(asrc, F);
    if (blockIdx.x == 0 && threadIdx.x == 0 && !asrc.from_hdr) {
        asrc.hdr[HDR_ANCHOR] = a;                // the gather reads it from here
        if (asrc.out_anchor) *asrc.out_anchor = a;
    }
    const int y = i / W, x = i - y * W;
    const size_t FN = (size_t)F * N;
    const int y_lo = max(0, y - r), y_hi = min(H - 1, y + r);
    const int x_lo = max(0, x - r), x_hi = min(W - 1, x + r);
    const int k_end = min(F, (chunk + 1) * fchunk);
    const T* Xa = X + (size_t)a * N * C;

    for (int k = chunk * fchunk + w; k < k_end; k += kMatchWarps) {
        const size_t f = (size_t)k * N + i;
        if (k == a) {                       // anchor tokens are always retained (Eq. mask)
            if (lane == 0 && in_bounds(asrc.hdr, 2, (long long)f, (long long)FN)) { shat[f] = 1.0f; dst[f] = i; keep[f] = 1; }
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
        if (lane == 0 && in_bounds(asrc.hdr, 2, (long long)f, (long long)FN)) {
            const unsigned char kp = !(best > t);
            shat[f] = best; dst[f] = best_j; keep[f] = kp;
            if (kp) atomicAdd(&cnt[k], 1);   // integer count: order-independent
        }
    }
}


// Prologue of the stand-alone kernels: anchor arg max (every CTA for itself), then the CTA's one unit.
template <int MT, int NT, bool GRAM, int ST>
__device__ __forceinline__ void match_mma_body(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t,
                                               const AnchorSrc& asrc, const float* ssq, int nslice,
                                               float* __restrict__ shat, int* __restrict__ dst,
                                               unsigned char* __restrict__ keep, int* __restrict__ cnt,
                                               int stream_once)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    const int N = H * W;
    const int i = blockIdx.x % N;
    const int k0 = (blockIdx.x / N) * 16 * MT;
    // No griddepcontrol.launch_dependents at the start: the next kernel of the stream is the gather, whose CTAs would
    // become resident at once (all CTAs of this grid start together) and then sit out this whole kernel in their wait,
    // each holding 64 KB of shared memory and a CTA slot that the kernels of other clips could use (8B-shaped clip,
    // eight clips in flight: 29.8 us per clip with the trigger here, 29.4 - 29.5 without).  The unit triggers after
    // its main loop instead, so that the gather's launch overlaps the epilogue.
    trace_mark(asrc.hdr, 2, false);
    // Everything upstream is complete after this wait: the frame statistics, and also whatever produced X (an
    // earlier kernel of the caller may still be writing X while this CTA is already resident, so X is not read
    // before the wait either).
    pdl_wait();
    trace_mark(asrc.hdr, 5, false);
    auto anchor_fn = [&]() -> int {              // runs while the first source rows are in flight
        const int a = resolve_anchor(asrc, F);
        if (blockIdx.x == 0 && threadIdx.x == 0 && !asrc.from_hdr) {
            asrc.hdr[HDR_ANCHOR] = a;            // the gather reads it from here
            if (asrc.out_anchor) *asrc.out_anchor = a;
        }
        trace_mark(asrc.hdr, 4, true);
        return a;
    };
    match_mma_unit<MT, NT, GRAM, ST>(X, F, H, W, C, r, t, anchor_fn, i, k0, ssq, nslice, shat, dst, keep, cnt, asrc.hdr, dyn_smem, stream_once);
    trace_mark(asrc.hdr, 2, true);
}

// r <= 1: 32 frames per CTA, norms from Gram diagonals, 96 registers (see TTF_MMA_BOUNDS)
template <int MT, int NT>
__global__ void TTF_MMA_BOUNDS
k_match_mma(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t, AnchorSrc asrc,
            float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt,
            int stream_once)
{
    match_mma_body<MT, NT, true, kMmaStagesDefault>(X, F, H, W, C, r, t, asrc, nullptr, 0, shat, dst, keep, cnt, stream_once);
}

// r = 2: the 25 candidate rows of a cell are as much data as 25 source rows, so a CTA takes 64 frames per cell to
// amortise them (2.6 -> 1.4 times |X| of operand traffic); norms come from the sweep, which frees the registers
// of the Gram accumulators for the 64 x 32 tile of dot products.
constexpr int kWideMT = 4;           // 64 frames per CTA
constexpr int kWideStages = 2;       // cp.async stages per warp (the 64 x 32 accumulator tile leaves no room for more)
__global__ void __launch_bounds__(kMmaWarps * 32, 2)
k_match_mma_wide(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t, AnchorSrc asrc,
                 const float* __restrict__ ssq, int nslice,
                 float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt)
{
    match_mma_body<kWideMT, 4, false, kWideStages>(X, F, H, W, C, r, t, asrc, ssq, nslice, shat, dst, keep, cnt, 0);
}

template <int MT, int NT>
static cudaError_t launch_mma_t(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                                unsigned char* keep, cudaStream_t st) {
    const long long chunks = (p.F + 16 * MT - 1) / (16 * MT);
    constexpr size_t smem = sizeof(uint4) * kMmaWarps * kMmaStagesDefault * (2 * MT + NT) * 32;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_match_mma<MT, NT>), smem);
    if (e != cudaSuccess) return e;
    return launch_ex(true, smem, k_match_mma<MT, NT>, dim3((unsigned)(chunks * p.N)),
                     dim3(kMmaWarps * 32), st, reinterpret_cast<const bf16_t*>(p.X), p.F, p.H, p.W, p.C, p.r, p.t,
                     make_anchor_src(p, s, out_anchor), shat, dst, keep, s.cnt, p.stream_once);
}

static cudaError_t launch_mma_wide(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                                   unsigned char* keep, cudaStream_t st) {
    constexpr size_t smem = sizeof(uint4) * kMmaWarps * kWideStages * (2 * kWideMT + 4) * 32;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_match_mma_wide), smem);
    if (e != cudaSuccess) return e;
    const long long chunks = (p.F + 16 * kWideMT - 1) / (16 * kWideMT);
    return launch_ex(true, smem, k_match_mma_wide, dim3((unsigned)(chunks * p.N)), dim3(kMmaWarps * 32),
                     st, reinterpret_cast<const bf16_t*>(p.X), p.F, p.H, p.W, p.C, p.r, p.t,
                     make_anchor_src(p, s, out_anchor), (const float*)s.ssq, p.nslice, shat, dst, keep, s.cnt);
}

template <typename T, int V>
static cudaError_t launch_generic_t(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
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
    return launch_pdl(k_match_generic<T, V>, dim3((unsigned)(nchunk * p.N)), dim3(kMatchWarps * 32), st,
                      reinterpret_cast<const T*>(p.X), p.F, p.H, p.W, p.C, p.r, p.t, fchunk, p.nslice,
                      make_anchor_src(p, s, out_anchor), (const float*)s.ssq, shat, dst, keep, s.cnt);
}

cudaError_t launch_match(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                         unsigned char* keep, cudaStream_t st) {
    if (p.dtype == 0) return p.vec ? launch_generic_t<float, 4>(p, s, out_anchor, shat, dst, keep, st)
                                   : launch_generic_t<float, 1>(p, s, out_anchor, shat, dst, keep, st);
    if (p.use_tc) return launch_match_tc(p, s, out_anchor, shat, dst, keep, st);
    if (uses_mma_match(p)) {
        if (p.r == 0) return launch_mma_t<2, 1>(p, s, out_anchor, shat, dst, keep, st);
        if (p.r == 1) return launch_mma_t<2, 2>(p, s, out_anchor, shat, dst, keep, st);
        return launch_mma_wide(p, s, out_anchor, shat, dst, keep, st);
    }
    return p.vec ? launch_generic_t<bf16_t, 8>(p, s, out_anchor, shat, dst, keep, st)
                 : launch_generic_t<bf16_t, 1>(p, s, out_anchor, shat, dst, keep, st);
}

}  // namespace ttf
