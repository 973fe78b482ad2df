// bf16 windowed matching on the warp-level tensor-core MMA: the unit of work shared by the stand-alone matching
// kernels.
#pragma once

#include "ttf_internal.cuh"

namespace ttf {

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
constexpr int kMmaStagesDefault = 3; // cp.async stages per warp (stages - 1 blocks in flight)
constexpr int kMmaMaxReg = 96;       // registers per thread of the r <= 1 kernel (see TTF_MMA_BOUNDS)

// One pipeline stage of a warp: the 16-byte fragment pieces of its 64-byte block, (2 MT + NT) per lane.  The
// pieces travel global -> shared with cp.async (no registers are tied up while they are in flight, so a warp
// keeps several stages outstanding); every lane copies into and later reads back its own 16-byte slots.
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src, bool valid) {
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(dst_smem));
    const int bytes = valid ? 16 : 0;            // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
// the same copy with an L2 cache policy (createpolicy) on the line it reads
__device__ __forceinline__ void cp_async16_hint(void* dst_smem, const void* src, bool valid, unsigned long long policy) {
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(dst_smem));
    const int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;" ::"r"(d), "l"(src), "r"(bytes), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// slot layout of a stage: [(2 MT + NT) pieces][32 lanes] x 16 bytes.  DO_A / DO_B: copy the pieces of the source
// rows / of the candidate rows (the prologue copies them at different times, see match_mma_unit)
template <int MT, int NT, bool DO_A = true, bool DO_B = true>
__device__ __forceinline__ void mma_issue_stage(uint4* slot, const uint4* const (&arow)[MT][2],
                                                const uint4* const (&brow)[NT], const bool (&bvalid)[NT],
                                                int idx, int units, int lane, int stream_once) {
    const bool ok = idx < units;
    const int safe = ok ? idx : 0;
    if constexpr (DO_A) {
        // a source row is read by this CTA alone: where the next clip streams into L2 meanwhile, its lines go first
        if (stream_once) {
            const unsigned long long once = l2_evict_first_policy();
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) cp_async16_hint(slot + (mt * 2 + h) * 32 + lane, arow[mt][h] + safe, ok, once);
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) cp_async16(slot + (mt * 2 + h) * 32 + lane, arow[mt][h] + safe, ok);
        }
    }
    if constexpr (DO_B) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) cp_async16(slot + (2 * MT + nt) * 32 + lane, brow[nt] + safe, ok && bvalid[nt]);
    }
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
#define TTF_MMA_BOUNDS __maxnreg__(kMmaMaxReg)
// GRAM: token norms from Gram-diagonal MMAs (else from the sweep's partial squared norms); ST: cp.async stages.
//
// One unit of work: cell i, frames k0 .. k0 + 16 MT - 1.  Called by all threads of a CTA of kMmaWarps warps;
// `dyn_smem` is at least kMmaWarps * ST * (2 MT + NT) * 512 bytes, 128-byte aligned.  A CTA that runs several
// units in a row must put a __syncthreads() between them.
// The anchor frame comes from `anchor_fn()`, which every thread calls once, AFTER the copies of the source rows
// of the first ST - 1 stages have been issued: the source rows do not depend on the anchor, so the loads that the
// anchor arg max waits for overlap their flight.  X must be readable when the unit is entered.
template <int MT, int NT, bool GRAM, int ST, typename AnchorFn>
__device__ __forceinline__ void match_mma_unit(const bf16_t* __restrict__ X, int F, int H, int W, int C, int r, float t,
                                               AnchorFn anchor_fn, int i, int k0, const float* ssq, int nslice,
                                               float* __restrict__ shat, int* __restrict__ dst,
                                               unsigned char* __restrict__ keep, int* __restrict__ cnt,
                                               int* hdr, unsigned char* dyn_smem, int stream_once)
{
    constexpr int kMmaStages = ST;
    constexpr int FR = 16 * MT;      // frames per CTA
    constexpr int NC = 8 * NT;       // candidate slots per CTA (>= (2r+1)^2)
    constexpr int PIECES = 2 * MT + NT;
    // ring[warp][stage][piece][lane]; after the main loop the same memory holds the per-warp partial products
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
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = lane >> 2, tig = lane & 3;
    const int y = i / W, x = i - y * W;
    const int side = 2 * r + 1, ncand = side * side;
    const int units = C / 8;                     // 16-byte units per row

    // candidate c = (dy + r) * side + (dx + r): ascending c is ascending anchor index among in-grid cells
    auto cand_index = [&](int c) -> int {
        if (c >= ncand) return -1;
        const int yy = y + c / side - r, xx = x + c % side - r;
        return (yy >= 0 && yy < H && xx >= 0 && xx < W) ? yy * W + xx : -1;
    };

    const uint4* arow[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = min(F - 1, k0 + mt * 16 + h * 8 + g);    // rows past the clip repeat the last frame
            arow[mt][h] = reinterpret_cast<const uint4*>(X + ((size_t)k * N + i) * C);
        }
    // split K: warp w takes 64-byte blocks w, w + 8, ...; kMmaStages - 1 blocks are in flight per warp
    const int nblk = (units + 3) / 4;
    uint4* wring = ring + (size_t)w * kMmaStages * PIECES * 32;
    const int nmine = nblk > w ? (nblk - w + kMmaWarps - 1) / kMmaWarps : 0;      // blocks of this warp
    const uint4* brow[NT];
    bool bvalid[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { brow[nt] = nullptr; bvalid[nt] = false; }

    // source rows of the first stages: one copy group, in flight while the anchor is found
#pragma unroll
    for (int st = 0; st < kMmaStages - 1; ++st)
        if (st < nmine)
            mma_issue_stage<MT, NT, true, false>(wring + st * PIECES * 32, arow, brow, bvalid,
                                                 (w + st * kMmaWarps) * 4 + tig, units, lane, stream_once);
    cp_async_commit();

    const int a = anchor_fn();

    if (tid < NC) s_j[tid] = cand_index(tid);
    if constexpr (!GRAM) {                       // inverse norms from the sweep's partials
        const size_t FN = (size_t)F * N;
        for (int q = tid; q < FR + NC; q += kMmaWarps * 32) {
            if (q < FR) { const int k = k0 + q; s_rs[q] = k < F ? inv_norm(ssq, nslice, FN, (size_t)k * N + i) : 0.f; }
            else { const int j = cand_index(q - FR); s_ra[q - FR] = j >= 0 ? inv_norm(ssq, nslice, FN, (size_t)a * N + j) : 0.f; }
        }
    }
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

    // candidate rows of the first stages, one copy group per stage.  Groups so far: the source-row group, then
    // these; the main loop adds one group per block, so "all but the newest ST - 1" still means "block b landed".
#pragma unroll
    for (int st = 0; st < kMmaStages - 1; ++st) {
        if (st < nmine)
            mma_issue_stage<MT, NT, false, true>(wring + st * PIECES * 32, arow, brow, bvalid,
                                                 (w + st * kMmaWarps) * 4 + tig, units, lane, stream_once);
        cp_async_commit();
    }
    for (int b = 0; b < nmine; ++b) {
        const int nb = b + kMmaStages - 1;
        if (nb < nmine)
            mma_issue_stage<MT, NT>(wring + (nb % kMmaStages) * PIECES * 32, arow, brow, bvalid,
                                    (w + nb * kMmaWarps) * 4 + tig, units, lane, stream_once);
        cp_async_commit();
        cp_async_wait<kMmaStages - 1>();         // block b has landed (each lane waits for its own copies)
        mma_consume_stage<MT, NT, GRAM>(wring + (b % kMmaStages) * PIECES * 32, lane, acc, accn, accb);
    }
    cp_async_wait<0>();
    pdl_launch_dependents();                     // (here rather than at the start: see match_mma_body)
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
        if (k < F && in_bounds(hdr, 2, (long long)k * N + i, (long long)F * N)) {
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
}


}  // namespace ttf
