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

// ---------------------------------------------------------------------------------------------------------
// bf16 fast path.  Per grid cell the work is a small dense contraction: the F source rows at that cell times
// the (2r+1)^2 candidate anchor rows, over C channels.  At 9 to 25 multiply-adds per loaded element the plain
// fp32 pipes, not memory, bound the per-token formulation, so the products go through the warp-level bf16
// MMA (m16n8k16, fp32 accumulate: bf16 products are exact in fp32).  M = frames (16 per tile), N = candidates
// (8 per tile), K = channels.
//
// No cross-thread staging: a dot product does not care about the order of its terms, so the K index of a
// fragment may be any fixed permutation of the channels as long as A and B use the same one.  Each lane fetches
// 16 contiguous bytes (8 channels) of "its" row (frame g / g+8 for A, candidate g for B; g = lane/4) at
// 16-byte column lane%4 of a 64-byte block and uses them as its fragment elements of two consecutive MMA
// steps.  The fetch is a cp.async into a lane-private shared-memory slot (coalesced in 64-byte runs per row,
// zero-filled past the row end and for absent candidates), several blocks ahead of the MMAs, so that the bytes
// in flight are bounded by shared memory rather than by registers; the measured floor of this kernel is the
// per-SM L2 read bandwidth (about 72 GB/s per SM), not latency.
//
// The 8 warps of a CTA take interleaved 64-byte blocks of the rows (split K) and their partial products are
// summed through shared memory in warp order, so the result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int kMmaWarps = 8;
#ifndef TTF_MMA_STAGES
#define TTF_MMA_STAGES 3
#endif
#ifndef TTF_MMA_MAXREG
#define TTF_MMA_MAXREG 96
#endif
constexpr int kMmaStagesDefault = TTF_MMA_STAGES; // cp.async stages per warp (stages - 1 blocks in flight)

// One pipeline stage of a warp: the 16-byte fragment pieces of its 64-byte block, (2 MT + NT) per lane.  The
// pieces travel global -> shared with cp.async (no registers are tied up while they are in flight, so a warp
// keeps several stages outstanding); every lane copies into and later reads back its own 16-byte slots.
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src, bool valid) {
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(dst_smem));
    const int bytes = valid ? 16 : 0;            // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// slot layout of a stage: [(2 MT + NT) pieces][32 lanes] x 16 bytes
template <int MT, int NT>
__device__ __forceinline__ void mma_issue_stage(uint4* slot, const uint4* const (&arow)[MT][2],
                                                const uint4* const (&brow)[NT], const bool (&bvalid)[NT],
                                                int idx, int units, int lane) {
    const bool ok = idx < units;
    const int safe = ok ? idx : 0;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) cp_async16(slot + (mt * 2 + h) * 32 + lane, arow[mt][h] + safe, ok);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) cp_async16(slot + (2 * MT + nt) * 32 + lane, brow[nt] + safe, ok && bvalid[nt]);
}

// Consumes one landed stage of a warp: dot products of every source row with every candidate row and, when
// GRAM, the squared norms of all rows: the Gram tile of a 16-row tile with itself has the squared norms on its
// diagonal, so two extra MMAs per tile (columns = rows 0..7, then rows 8..15) give them on the tensor pipe from
// fragments that are in registers anyway.  Fragments are read from the lane's slots tile by tile.
template <int MT, int NT, bool GRAM>
__device__ __forceinline__ void mma_consume_stage(const uint4* slot, int lane, float (&acc)[MT][NT][4],
                                                  float (&accn)[GRAM ? MT : 1][2][4], float (&accb)[GRAM ? NT : 1][4]) {
    uint4 b[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) b[nt] = slot[(2 * MT + nt) * 32 + lane];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const uint4 a0 = slot[(mt * 2 + 0) * 32 + lane], a1 = slot[(mt * 2 + 1) * 32 + lane];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            mma_bf16_16816(acc[mt][nt], a0.x, a1.x, a0.y, a1.y, b[nt].x, b[nt].y);
            mma_bf16_16816(acc[mt][nt], a0.z, a1.z, a0.w, a1.w, b[nt].z, b[nt].w);
        }
        if constexpr (GRAM) {
            mma_bf16_16816(accn[mt][0], a0.x, a1.x, a0.y, a1.y, a0.x, a0.y);
            mma_bf16_16816(accn[mt][0], a0.z, a1.z, a0.w, a1.w, a0.z, a0.w);
            mma_bf16_16816(accn[mt][1], a0.x, a1.x, a0.y, a1.y, a1.x, a1.y);
            mma_bf16_16816(accn[mt][1], a0.z, a1.z, a0.w, a1.w, a1.z, a1.w);
        }
    }
    if constexpr (GRAM) {
        // candidate rows: rows of the Gram tile = slots of the tile pair (even, odd), columns = slots of tile nt
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const uint4 lo = b[nt & ~1];
            const uint4 hi = (nt | 1) < NT ? b[(nt | 1) < NT ? (nt | 1) : nt] : make_uint4(0, 0, 0, 0);
            mma_bf16_16816(accb[nt], lo.x, hi.x, lo.y, hi.y, b[nt].x, b[nt].y);
            mma_bf16_16816(accb[nt], lo.z, hi.z, lo.w, hi.w, b[nt].z, b[nt].w);
        }
    }
}

// 96 registers and 3 stages (74 KB) per CTA: two of these CTAs leave room on an SM for a CTA of the next clip's
// sweep, which is what lets clips on different streams overlap (measured: 31.6 vs 33.3 us per clip, 4 streams)
#define TTF_MMA_BOUNDS __maxnreg__(TTF_MMA_MAXREG)
// GRAM: token norms from Gram-diagonal MMAs (else from the sweep's partial squared norms); ST: cp.async stages.
template <int MT, int NT, bool GRAM, int ST>
__device__ __forceinline__ void match_mma_body(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t,
                                               const AnchorSrc& asrc, const float* ssq, int nslice,
                                               float* __restrict__ shat, int* __restrict__ dst,
                                               unsigned char* __restrict__ keep, int* __restrict__ cnt)
{
    constexpr int kMmaStages = ST;
    constexpr int FR = 16 * MT;      // frames per CTA
    constexpr int NC = 8 * NT;       // candidate slots per CTA (>= (2r+1)^2)
    constexpr int PIECES = 2 * MT + NT;
    // ring[warp][stage][piece][lane]; after the main loop the same memory holds the per-warp partial products
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    uint4* ring = reinterpret_cast<uint4*>(dyn_smem);
    float (*s_part)[FR][NC] = reinterpret_cast<float (*)[FR][NC]>(dyn_smem);
    static_assert(sizeof(float) * kMmaWarps * FR * NC <= sizeof(uint4) * kMmaWarps * kMmaStages * PIECES * 32,
                  "partial products must fit the ring");
    __shared__ float s_dot[FR][NC];
    __shared__ float s_na[GRAM ? kMmaWarps : 1][FR];   // partial squared norms of the source rows, per warp
    __shared__ float s_nb[GRAM ? kMmaWarps : 1][NC];   // ... of the candidate rows
    __shared__ float s_rs[FR];
    __shared__ float s_ra[NC];
    __shared__ int s_j[NC];

    const int N = H * W;
    const int i = blockIdx.x % N;
    const int k0 = (blockIdx.x / N) * FR;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = lane >> 2, tig = lane & 3;
    pdl_launch_dependents();
    trace_mark(asrc.hdr, 2, false);
#ifdef TTF_WARM
    {   // rehearsal: run the anchor search once on whatever the buffers hold, only to have its code fetched
        const int warm = resolve_anchor(asrc, F);
        if (warm == 0x7ffffffe) asrc.hdr[kHdrInts - 1] = warm;
        __syncthreads();
    }
#endif
    pdl_wait();                                  // the frame statistics are complete (X itself is an input)
    trace_mark(asrc.hdr, 5, false);
    const int a = resolve_anchor(asrc, F);
    if (blockIdx.x == 0 && tid == 0 && !asrc.from_hdr) {
        asrc.hdr[HDR_ANCHOR] = a;                // the gather reads it from here
        if (asrc.out_anchor) *asrc.out_anchor = a;
    }
    trace_mark(asrc.hdr, 4, true);
    const int y = i / W, x = i - y * W;
    const int side = 2 * r + 1, ncand = side * side;
    const int units = C / 8;                     // 16-byte units per row

    // candidate c = (dy + r) * side + (dx + r): ascending c is ascending anchor index among in-grid cells
    auto cand_index = [&](int c) -> int {
        if (c >= ncand) return -1;
        const int yy = y + c / side - r, xx = x + c % side - r;
        return (yy >= 0 && yy < H && xx >= 0 && xx < W) ? yy * W + xx : -1;
    };

    if (tid < NC) s_j[tid] = cand_index(tid);
    if constexpr (!GRAM) {                       // inverse norms from the sweep's partials
        const size_t FN = (size_t)F * N;
        for (int q = tid; q < FR + NC; q += kMmaWarps * 32) {
            if (q < FR) { const int k = k0 + q; s_rs[q] = k < F ? inv_norm(ssq, nslice, FN, (size_t)k * N + i) : 0.f; }
            else { const int j = cand_index(q - FR); s_ra[q - FR] = j >= 0 ? inv_norm(ssq, nslice, FN, (size_t)a * N + j) : 0.f; }
        }
    }

    const uint4* arow[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = min(F - 1, k0 + mt * 16 + h * 8 + g);    // rows past the clip repeat the last frame
            arow[mt][h] = reinterpret_cast<const uint4*>(X + ((size_t)k * N + i) * C);
        }
    const uint4* brow[NT];
    bool bvalid[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int j = cand_index(nt * 8 + g);
        bvalid[nt] = j >= 0;
        brow[nt] = reinterpret_cast<const uint4*>(X + ((size_t)a * N + (j >= 0 ? j : 0)) * C);
    }

    float acc[MT][NT][4], accn[GRAM ? MT : 1][2][4], accb[GRAM ? NT : 1][4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) acc[mt][nt][q] = 0.f;
#pragma unroll
        for (int mt = 0; mt < (GRAM ? MT : 1); ++mt) { accn[mt][0][q] = 0.f; accn[mt][1][q] = 0.f; }
#pragma unroll
        for (int nt = 0; nt < (GRAM ? NT : 1); ++nt) accb[nt][q] = 0.f;
    }

    // split K: warp w takes 64-byte blocks w, w + 8, ...; kMmaStages - 1 blocks are in flight per warp
    const int nblk = (units + 3) / 4;
    uint4* wring = ring + (size_t)w * kMmaStages * PIECES * 32;
    const int nmine = nblk > w ? (nblk - w + kMmaWarps - 1) / kMmaWarps : 0;      // blocks of this warp
#pragma unroll
    for (int st = 0; st < kMmaStages - 1; ++st) {
        if (st < nmine)
            mma_issue_stage<MT, NT>(wring + st * PIECES * 32, arow, brow, bvalid, (w + st * kMmaWarps) * 4 + tig, units, lane);
        cp_async_commit();
    }
    for (int b = 0; b < nmine; ++b) {
        const int nb = b + kMmaStages - 1;
        if (nb < nmine)
            mma_issue_stage<MT, NT>(wring + (nb % kMmaStages) * PIECES * 32, arow, brow, bvalid,
                                    (w + nb * kMmaWarps) * 4 + tig, units, lane);
        cp_async_commit();
        cp_async_wait<kMmaStages - 1>();         // block b has landed (each lane waits for its own copies)
        mma_consume_stage<MT, NT, GRAM>(wring + (b % kMmaStages) * PIECES * 32, lane, acc, accn, accb);
    }
    cp_async_wait<0>();
    __syncthreads();                             // every warp is done with its ring: reuse it for the partials

    // accumulator fragment: c0,c1 = (frame g, candidates 2*tig, 2*tig+1); c2,c3 = (frame g+8, same candidates)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            s_part[w][mt * 16 + g][nt * 8 + 2 * tig] = acc[mt][nt][0];
            s_part[w][mt * 16 + g][nt * 8 + 2 * tig + 1] = acc[mt][nt][1];
            s_part[w][mt * 16 + g + 8][nt * 8 + 2 * tig] = acc[mt][nt][2];
            s_part[w][mt * 16 + g + 8][nt * 8 + 2 * tig + 1] = acc[mt][nt][3];
        }
    // Gram diagonals: the lane with tig == g / 2 holds entry (g, g) in c0 / c1 and (g + 8, g) in c2 / c3
    if (GRAM && tig == (g >> 1)) {
        const bool odd = g & 1;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            s_na[w][mt * 16 + g] = odd ? accn[mt][0][1] : accn[mt][0][0];          // frame g against column g
            s_na[w][mt * 16 + 8 + g] = odd ? accn[mt][1][3] : accn[mt][1][2];      // frame g + 8 against column g
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)                  // slot nt*8 + g is row g of an even tile, row g + 8 of an odd one
            s_nb[w][nt * 8 + g] = (nt & 1) ? (odd ? accb[nt][3] : accb[nt][2]) : (odd ? accb[nt][1] : accb[nt][0]);
    }
    __syncthreads();
    for (int idx = tid; idx < FR * NC; idx += kMmaWarps * 32) {
        float d = 0.f;
#pragma unroll
        for (int ww = 0; ww < kMmaWarps; ++ww) d += (&s_part[ww][0][0])[idx];
        (&s_dot[0][0])[idx] = d;
    }
    if (GRAM && tid < FR + NC) {                         // 1 / max(||x||, floor), warps added in warp order
        float n2 = 0.f;
#pragma unroll
        for (int ww = 0; ww < kMmaWarps; ++ww) n2 += tid < FR ? s_na[ww][tid] : s_nb[ww][tid - FR];
        const float rinv = 1.0f / fmaxf(sqrtf(n2), kNormFloor);
        if (tid < FR) s_rs[tid] = rinv; else s_ra[tid - FR] = rinv;
    }
    __syncthreads();

    if (tid < FR) {
        const int k = k0 + tid;
        if (k < F) {
            const size_t f = (size_t)k * N + i;
            if (k == a) {                           // anchor tokens are always retained (Eq. mask)
                shat[f] = 1.0f; dst[f] = i; keep[f] = 1;
            } else {
                const float rs = s_rs[tid];
                float best = -INFINITY;
                int best_j = -1;
                for (int c = 0; c < ncand; ++c) {
                    const int j = s_j[c];
                    if (j < 0) continue;
                    const float s = s_dot[tid][c] * rs * s_ra[c];
                    if (s > best || best_j < 0) { best = s; best_j = j; }
                }
                const unsigned char kp = !(best > t);
                shat[f] = best; dst[f] = best_j; keep[f] = kp;
                if (kp) atomicAdd(&cnt[k], 1);
            }
        }
    }
    trace_mark(asrc.hdr, 2, true);
}

// r <= 1: 32 frames per CTA, norms from Gram diagonals, 96 registers (see TTF_MMA_BOUNDS)
template <int MT, int NT>
__global__ void TTF_MMA_BOUNDS
k_match_mma(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t, AnchorSrc asrc,
            float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt)
{
    match_mma_body<MT, NT, true, kMmaStagesDefault>(X, F, H, W, C, r, t, asrc, nullptr, 0, shat, dst, keep, cnt);
}

// r = 2: the 25 candidate rows of a cell are as much data as 25 source rows, so a CTA takes 64 frames per cell to
// amortise them (2.6 -> 1.4 times |X| of operand traffic); norms come from the sweep, which frees the registers
// of the Gram accumulators for the 64 x 32 tile of dot products.
#ifndef TTF_WIDE_MT
#define TTF_WIDE_MT 4
#endif
#ifndef TTF_WIDE_STAGES
#define TTF_WIDE_STAGES 2
#endif
constexpr int kWideMT = TTF_WIDE_MT;
constexpr int kWideStages = TTF_WIDE_STAGES;
__global__ void __launch_bounds__(kMmaWarps * 32, 2)
k_match_mma_wide(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t, AnchorSrc asrc,
                 const float* __restrict__ ssq, int nslice,
                 float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt)
{
    match_mma_body<kWideMT, 4, false, kWideStages>(X, F, H, W, C, r, t, asrc, ssq, nslice, shat, dst, keep, cnt);
}

template <int MT, int NT>
static cudaError_t launch_mma_t(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                                unsigned char* keep, cudaStream_t st) {
    const long long chunks = (p.F + 16 * MT - 1) / (16 * MT);
    constexpr size_t smem = sizeof(uint4) * kMmaWarps * kMmaStagesDefault * (2 * MT + NT) * 32;
    static bool configured = false;              // per instantiation; the attribute belongs to the function
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(k_match_mma<MT, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(chunks * p.N)); cfg.blockDim = dim3(kMmaWarps * 32);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_match_mma<MT, NT>, reinterpret_cast<const bf16_t*>(p.X), p.F, p.H, p.W, p.C,
                              p.r, p.t, make_anchor_src(p, s, out_anchor), shat, dst, keep, s.cnt);
}

static cudaError_t launch_mma_wide(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                                   unsigned char* keep, cudaStream_t st) {
    constexpr size_t smem = sizeof(uint4) * kMmaWarps * kWideStages * (2 * kWideMT + 4) * 32;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(k_match_mma_wide, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const long long chunks = (p.F + 16 * kWideMT - 1) / (16 * kWideMT);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(chunks * p.N)); cfg.blockDim = dim3(kMmaWarps * 32);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_match_mma_wide, reinterpret_cast<const bf16_t*>(p.X), p.F, p.H, p.W, p.C, p.r,
                              p.t, make_anchor_src(p, s, out_anchor), (const float*)s.ssq, p.nslice, shat, dst, keep,
                              s.cnt);
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
    if (uses_mma_match(p)) {
        if (p.r == 0) return launch_mma_t<2, 1>(p, s, out_anchor, shat, dst, keep, st);
        if (p.r == 1) return launch_mma_t<2, 2>(p, s, out_anchor, shat, dst, keep, st);
        return launch_mma_wide(p, s, out_anchor, shat, dst, keep, st);
    }
    return p.vec ? launch_generic_t<bf16_t, 8>(p, s, out_anchor, shat, dst, keep, st)
                 : launch_generic_t<bf16_t, 1>(p, s, out_anchor, shat, dst, keep, st);
}

}  // namespace ttf
