// Token Compression and Positional Alignment (Eqs. xprime_stack, mask, compress_pos, Lpre), plus the
// bookkeeping of identity replacement (how many source tokens each anchor cell absorbed).
//
// The output position of a preserved source token is N plus the number of preserved source tokens before it
// in flat (k, i) order.  That exclusive prefix is taken in two levels: the per-frame survivor counts written
// by the matching kernel are scanned by every warp for itself (shuffles; a pre-scanned array for very long
// clips), and inside a frame the rank is a population count over the frame's keep flags.  The gather is then
// driven from the OUTPUT side: one warp per output row finds the source row by rank/select and copies it
// with all of its 16-byte loads in flight at once, so the work per warp is the same no matter how unevenly
// the survivors are spread over the frames.  No warp ever waits for another one.
#include "ttf_internal.cuh"
#include "ttf_async.cuh"
#include "ttf_gather.cuh"

namespace ttf {

// exclusive scan of the effective per-frame counts (anchor frame counts as 0) for clips with more frames
// than fit the shared-memory scan of the gather kernel
__global__ void __launch_bounds__(1024)
k_frame_prefix(const int* __restrict__ cnt, const int* __restrict__ hdr, int F, int* __restrict__ prefix)
{
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int a = hdr[HDR_ANCHOR];
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < F; base += 1024) {
        const int k = base + tid;
        int v = (k < F && k != a) ? cnt[k] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        if (lane == 31) s_warp[w] = incl;
        __syncthreads();
        if (w == 0) {
            int x = s_warp[lane], xi = x;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int n = __shfl_up_sync(0xffffffffu, xi, o);
                if (lane >= o) xi += n;
            }
            s_warp[lane] = xi - x;       // exclusive over warps
        }
        __syncthreads();
        const int carry = s_carry;
        if (k < F) prefix[k] = carry + s_warp[w] + incl - v;
        __syncthreads();
        if (tid == 1023) s_carry = carry + s_warp[w] + incl;
        __syncthreads();
    }
    if (tid == 0) prefix[F] = s_carry;
}

// COPY_BYTES: 16 when rows are 16-byte aligned multiples of 16 bytes, else the element size (2 or 4)
template <int COPY_BYTES> struct CopyUnit;
template <> struct CopyUnit<16> { using type = uint4; };
template <> struct CopyUnit<4> { using type = uint32_t; };
template <> struct CopyUnit<2> { using type = uint16_t; };

#ifndef TTF_COPY_UNROLL
#define TTF_COPY_UNROLL 8
#endif
constexpr int kCopyUnroll = TTF_COPY_UNROLL;   // 16-byte units in flight per lane (two steps for an 8 KB row)
// Gather with bulk asynchronous copies, for rows that are 16-byte aligned multiples of 16 bytes: a warp finds the
// source row of its output row as above, then one lane moves the row global -> shared -> global with two bulk
// copies per piece of at most kBulkPiece bytes, so no data passes through registers.
#ifndef TTF_BULK_PIECE
#define TTF_BULK_PIECE 8192
#endif
constexpr int kBulkPiece = TTF_BULK_PIECE;

__global__ void __launch_bounds__(kCopyWarps * 32)
k_compact_bulk(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
               const int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
               const unsigned char* __restrict__ keep, const int* __restrict__ dst,
               unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
               int* __restrict__ fuse_cnt, int ncopy_blocks, int NA, int t_off)
{
    extern __shared__ __align__(128) unsigned char stage[];     // [kCopyWarps][kBulkPiece]
    __shared__ uint64_t bar[kCopyWarps];
    const int N = H * W;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    pdl_launch_dependents();                     // the next call's sweep may be scheduled; it waits for this grid
    trace_mark(const_cast<int*>(hdr), 3, false);
    if (lane == 0) { mbar_init(&bar[w], 1); mbar_init_fence(); }
    __syncwarp();
    pdl_wait();                                  // keep flags and survivor counts are complete
    trace_mark(const_cast<int*>(hdr), 6, false);
    const int a = __ldcg(hdr + HDR_ANCHOR);
    if ((int)blockIdx.x >= ncopy_blocks) {       // bookkeeping CTAs: tokens fused into each anchor cell
        fuse_count_cta(F, H, W, r, a, keep, dst, fuse_cnt, (int)blockIdx.x - ncopy_blocks, (int)gridDim.x - ncopy_blocks);
        return;
    }
    const int gw = blockIdx.x * kCopyWarps + w;
    const int nw = ncopy_blocks * kCopyWarps;
    if (gw == 0) {                               // L' = N + P (Eq. Lpre)
        int kk, bb;
        const int P = find_frame(cnt, gprefix, F, a, lane, -1, kk, bb);
        if (lane == 0) *out_count = __ldcg(hdr + HDR_ERROR) ? -1 : NA + P;
    }
    unsigned char* buf = stage + (size_t)w * kBulkPiece;
    const int pieces = (int)((row_bytes + kBulkPiece - 1) / kBulkPiece);
    uint32_t phase = 0;
    bool gave_up = false;
    for (int j = gw; ; j += nw) {
        int f;
        if (j < NA) f = a * N + j;               // anchor rows first (Eq. xprime_stack)
        else {
            int k, before;
            find_frame(cnt, gprefix, F, a, lane, j - NA, k, before);
            if (k < 0) break;                    // past the last output row
            const int i = select_in_frame(keep + (size_t)k * N, N, j - NA - before, lane);
            if (i < 0) break;                    // cannot happen when cnt matches keep
            f = k * N + i;
        }
        if (lane < 3) {                          // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
            const int k = f / N, i = f - k * N, yy = i / W;
            out_pos[(size_t)j * 3 + lane] = lane == 0 ? k + t_off : (lane == 1 ? yy : i - yy * W);
        }
        if (lane == 0 && !gave_up) {
            for (int pc = 0; pc < pieces; ++pc) {
                const size_t off = (size_t)pc * kBulkPiece;
                const uint32_t bytes = (uint32_t)(row_bytes - off < (size_t)kBulkPiece ? row_bytes - off : kBulkPiece);
                bulk_wait_read<0>();             // the previous store has finished reading the buffer
                mbar_arrive_expect_tx(&bar[w], bytes);
                bulk_load(buf, X + (size_t)f * row_bytes + off, bytes, &bar[w]);
                if (!mbar_wait(&bar[w], phase & 1)) { gave_up = true; break; }
                ++phase;
                bulk_store(out_tokens + (size_t)j * row_bytes + off, buf, bytes);
                bulk_commit();
            }
        }
        __syncwarp();
    }
    if (lane == 0) {
        bulk_wait<0>();                          // all rows of this warp are in global memory
        if (gave_up) atomicExch(const_cast<int*>(hdr) + HDR_ERROR, 1);
    }
    trace_mark(const_cast<int*>(hdr), 3, true);
}

template <int COPY_BYTES>
__global__ void __launch_bounds__(kCopyWarps * 32)
k_compact(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
          const int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
          const unsigned char* __restrict__ keep, const int* __restrict__ dst,
          unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
          int* __restrict__ fuse_cnt, int ncopy_blocks, int NA, int t_off)
{
    using U = typename CopyUnit<COPY_BYTES>::type;
    const int N = H * W;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    pdl_launch_dependents();                     // the next call's sweep may be scheduled; it waits for this grid
    trace_mark(const_cast<int*>(hdr), 3, false);
    pdl_wait();                                  // keep flags, dst and survivor counts are complete
    trace_mark(const_cast<int*>(hdr), 6, false);
    const int a = __ldcg(hdr + HDR_ANCHOR);

    // ---- bookkeeping CTAs: tokens fused into each anchor cell ------------------------------------------------
    if ((int)blockIdx.x >= ncopy_blocks) {
        fuse_count_cta(F, H, W, r, a, keep, dst, fuse_cnt, (int)blockIdx.x - ncopy_blocks, (int)gridDim.x - ncopy_blocks);
        return;
    }

    // ---- output-driven gather, one warp per output row, no block-level synchronisation -----------------------
    // frame search: the frame that holds the e-th preserved source token (flat order, anchor frame skipped)
    // and the number of preserved tokens before that frame.  Returns the total P when e is past the end.
    const int gw = blockIdx.x * kCopyWarps + w;            // global warp index
    const int nw = ncopy_blocks * kCopyWarps;
    if (gw == 0) {                                         // L' = N + P (Eq. Lpre)
        int kk, bb;
        const int P = find_frame(cnt, gprefix, F, a, lane, -1, kk, bb);
        // a bounded wait of an earlier kernel of this call gave up: report instead of a plausible count
        if (lane == 0) *out_count = __ldcg(hdr + HDR_ERROR) ? -1 : NA + P;
    }
    const int upr = (int)(row_bytes / COPY_BYTES);         // copy units per row
    for (int j = gw; ; j += nw) {
        int f;
        if (j < NA) f = a * N + j;                         // anchor rows first (Eq. xprime_stack)
        else {
            int k, before;
            find_frame(cnt, gprefix, F, a, lane, j - NA, k, before);
            if (k < 0) break;                              // past the last output row
            const int i = select_in_frame(keep + (size_t)k * N, N, j - NA - before, lane);
            if (i < 0) break;                              // cannot happen when cnt matches keep
            f = k * N + i;
        }
        if (lane < 3) {                                    // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
            const int k = f / N, i = f - k * N, yy = i / W;
            out_pos[(size_t)j * 3 + lane] = lane == 0 ? k + t_off : (lane == 1 ? yy : i - yy * W);
        }
        const U* src = reinterpret_cast<const U*>(X + (size_t)f * row_bytes);
        U* dsto = reinterpret_cast<U*>(out_tokens + (size_t)j * row_bytes);
        for (int u0 = lane; u0 < upr; u0 += 32 * kCopyUnroll) {
            U v[kCopyUnroll];
#pragma unroll
            for (int q = 0; q < kCopyUnroll; ++q) if (u0 + q * 32 < upr) v[q] = __ldcs(src + u0 + q * 32);
#pragma unroll
            for (int q = 0; q < kCopyUnroll; ++q) if (u0 + q * 32 < upr) __stcs(dsto + u0 + q * 32, v[q]);
        }
    }
    trace_mark(const_cast<int*>(hdr), 3, true);
}

cudaError_t launch_fuse_count(const Problem& p, const Scratch& s, const int* dst, const unsigned char* keep,
                              int* fuse_cnt, cudaStream_t st) {
    // bookkeeping only: the same kernel with zero copy CTAs
    const int nb = (p.N + kCopyWarps - 1) / kCopyWarps;
    k_compact<4><<<nb < 1024 ? nb : 1024, kCopyWarps * 32, 0, st>>>(
        nullptr, 0, p.F, p.H, p.W, p.r, s.hdr, s.cnt, s.prefix, keep, dst, nullptr, nullptr, nullptr,
        fuse_cnt, 0, p.N, 0);
    return cudaGetLastError();
}

cudaError_t launch_compact(const Problem& p, const Scratch& s, void* out_tokens, int* out_pos, int* out_count,
                           cudaStream_t st) {
    const size_t esize = p.dtype == 0 ? 4 : 2;
    const size_t row_bytes = (size_t)p.C * esize;
    const bool vec = p.vec && (reinterpret_cast<uintptr_t>(out_tokens) % 16 == 0);
    if (p.F > kWarpPrefixMaxF) {
        k_frame_prefix<<<1, 1024, 0, st>>>(s.cnt, s.hdr, p.F, s.prefix);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    // enough warps for one output row each at the usual two-thirds removal (a warp loops when there are more)
    const long long want = ((long long)p.F * p.N / 3 + p.N + kCopyWarps - 1) / kCopyWarps;
    const int ncopy = (int)(want < 3LL * sm_count() ? (want < 1 ? 1 : want) : 3LL * sm_count());
    int nfuse = (p.N + kCopyWarps - 1) / kCopyWarps;
    if (nfuse > sm_count()) nfuse = sm_count();
    const int grid = ncopy + nfuse;
    const unsigned char* X = reinterpret_cast<const unsigned char*>(p.X);
    unsigned char* out = reinterpret_cast<unsigned char*>(out_tokens);
    const dim3 g(grid), b(kCopyWarps * 32);
    const int NA = p.emit_anchor ? p.N : 0;      // a streaming segment does not emit its rolling anchor again
    // the pre-scanned prefix of very long clips is read through plain loads: order that case by the stream
    const bool pdl = p.F <= kWarpPrefixMaxF;
    if (vec) {
        static bool configured = false;          // the attribute belongs to the function, set it once
        const size_t smem = (size_t)kCopyWarps * kBulkPiece;
        if (!configured) {
            cudaError_t e = cudaFuncSetAttribute(k_compact_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            configured = true;
        }
        return launch_ex(pdl, smem, k_compact_bulk, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r,
                         (const int*)s.hdr, (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep,
                         (const int*)s.dst, out, out_pos, out_count, s.fuse_cnt, ncopy, NA, p.pos_t_offset);
    }
    if (esize == 4)
        return launch_pdl_if(pdl, k_compact<4>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                          (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                          out, out_pos, out_count, s.fuse_cnt, ncopy, NA, p.pos_t_offset);
    return launch_pdl_if(pdl, k_compact<2>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                      (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                      out, out_pos, out_count, s.fuse_cnt, ncopy, NA, p.pos_t_offset);
}

}  // namespace ttf
