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
k_frame_prefix(const int* __restrict__ cnt, const int* __restrict__ hdr, int F, int acnt, int* __restrict__ prefix)
{
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int a = hdr[HDR_ANCHOR];
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < F; base += 1024) {
        const int k = base + tid;
        int v = k < F ? (k == a ? acnt : cnt[k]) : 0;
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

constexpr int kCopyUnroll = 8;       // 16-byte units in flight per lane of the element-wise gather (two steps for an 8 KB row)

// Gather with bulk asynchronous copies, for rows that are 16-byte aligned multiples of 16 bytes: a warp finds the
// source row of its output row by rank/select (frame search over the survivor counts, then a select inside that
// frame's keep flags), then one lane moves the row global -> shared -> global with two bulk copies per piece of at
// most kBulkPiece bytes, so no data passes through registers.  One row per warp at a time and 24 warps per SM:
// measured against variants in which a warp owns a contiguous range of rows, finds it with fewer dependent loads
// and keeps two to four rows in flight through a ring of slots, this plain form was the fastest (11.7 against
// 14.9 - 16.5 us on the 8B-shaped clip): the copies of a clip are one short burst that is bounded by what an SM can
// take in and put out per cycle, and what counts is how early the first copy of every warp is on its way.
// Every wait is bounded; a warp whose wait runs out stops copying, raises the error word and writes L' = -1.
constexpr int kBulkPiece = 8192;     // bytes per staging slot; longer rows go in pieces

__global__ void __launch_bounds__(kCopyWarps * 32)
k_compact_bulk(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
               int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
               const unsigned char* __restrict__ keep, const int* __restrict__ dst,
               unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
               int* __restrict__ fuse_cnt, int ncopy_blocks, int NA, int acnt, int t_off, int pos_base,
               int late_trigger, int wait_limit, int tx_extra, int stream_once)
{
    extern __shared__ __align__(128) unsigned char stage[];     // [kCopyWarps][kBulkPiece]
    __shared__ uint64_t bar[kCopyWarps];
    const int N = H * W;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    // The next kernel of the stream may be scheduled once every CTA has said so (or has exited).  Normally that is
    // said at once: the next kernel waits for this grid before it touches anything, and meanwhile its CTAs are set
    // up.  When the next kernel is the sweep of the next clip of a batch, which runs beside this gather without
    // waiting, it is said only after the wait below: the sweep must not start while the matching kernel still
    // needs this clip in L2.
    if (!late_trigger) pdl_launch_dependents();
    trace_mark(hdr, 3, false);
    if (lane == 0) { mbar_init(&bar[w], 1); mbar_init_fence(); }
    __syncwarp();
    pdl_wait();                                  // keep flags, dst and survivor counts are complete
    if (late_trigger) pdl_launch_dependents();
    trace_mark(hdr, 6, false);
    const int a = __ldcg(hdr + HDR_ANCHOR);
    if ((int)blockIdx.x >= ncopy_blocks) {       // bookkeeping CTAs: tokens fused into each anchor cell
        fuse_count_cta(F, H, W, r, a, keep, dst, fuse_cnt, (int)blockIdx.x - ncopy_blocks, (int)gridDim.x - ncopy_blocks);
        return;
    }
    const int gw = blockIdx.x * kCopyWarps + w;
    const int nw = ncopy_blocks * kCopyWarps;
    int Lp = 0;
    if (gw == 0) {                               // L' = N + P (Eq. Lpre)
        int kk, bb;
        Lp = NA + find_frame(cnt, gprefix, F, a, acnt, lane, -1, kk, bb);
        if (lane == 0) *reinterpret_cast<volatile int*>(out_count) = Lp;
    }
    unsigned char* buf = stage + (size_t)w * kBulkPiece;
    const int pieces = (int)((row_bytes + kBulkPiece - 1) / kBulkPiece);
    uint32_t phase = 0;
    bool gave_up = false;
    // pipelined schedule: neither the rows read here nor the rows written are needed in L2 again, while the clip
    // that is being matched and the one streaming in are: their lines are the first to go
    const unsigned long long once = l2_evict_first_policy();
    for (int j = gw; ; j += nw) {
        int f;
        if (j < NA) f = a * N + j;               // anchor rows first (Eq. xprime_stack)
        else {
            int k, before;
            find_frame(cnt, gprefix, F, a, acnt, lane, j - NA, k, before);
            if (k < 0) break;                    // past the last output row
            const int i = select_in_frame(keep + (size_t)k * N, N, j - NA - before, lane);
            if (i < 0) break;                    // cannot happen when cnt matches keep
            f = k * N + i;
        }
        // (checked build: the output row and the source row both lie inside their F N rows)
        const bool row_ok = in_bounds(hdr, 4, j, (long long)F * N) && in_bounds(hdr, 4, f, (long long)F * N);
        if (lane < 3 && row_ok) {                // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
            const int k = f / N, i = f - k * N, yy = i / W;
            out_pos[(size_t)j * 3 + lane] = pos_base + (lane == 0 ? k + t_off : (lane == 1 ? yy : i - yy * W));
        }
        if (lane == 0 && !gave_up && row_ok) {
            for (int pc = 0; pc < pieces; ++pc) {
                const size_t off = (size_t)pc * kBulkPiece;
                const uint32_t bytes = (uint32_t)(row_bytes - off < (size_t)kBulkPiece ? row_bytes - off : kBulkPiece);
                bulk_wait_read<0>();             // the previous store has finished reading the buffer
                mbar_arrive_expect_tx(&bar[w], bytes + (uint32_t)tx_extra);
                if (stream_once) bulk_load_hint(buf, X + (size_t)f * row_bytes + off, bytes, &bar[w], once);
                else bulk_load(buf, X + (size_t)f * row_bytes + off, bytes, &bar[w]);
                if (!mbar_wait(&bar[w], phase & 1, wait_limit)) {
                    mbar_wait(&bar[w], phase & 1, wait_limit);   // one more bounded chance for the copy to land
                    gave_up = true;
                    break;
                }
                ++phase;
                if (stream_once) bulk_store_hint(out_tokens + (size_t)j * row_bytes + off, buf, bytes, once);
                else bulk_store(out_tokens + (size_t)j * row_bytes + off, buf, bytes);
                bulk_commit();
            }
        }
        __syncwarp();
    }
    if (lane == 0) {
        bulk_wait<0>();                          // all rows of this warp are in global memory
        // L', or -1 if a wait of this call gave up.  Warp 0 has published L' above and looks at the error word now; a
        // warp that gave up raises the error word first and writes -1 afterwards.  Whichever order the two run in, -1
        // is what stays: either the -1 lands after L', or warp 0 sees the error word and writes -1 itself.
        if (gave_up) {
            atomicExch(hdr + HDR_ERROR, 1);
            __threadfence();
            *reinterpret_cast<volatile int*>(out_count) = -1;
        }
        if (gw == 0) {
            __threadfence();
            if (atomicAdd(hdr + HDR_ERROR, 0)) *reinterpret_cast<volatile int*>(out_count) = -1;
        }
    }
    trace_mark(hdr, 3, true);
}

template <int COPY_BYTES>
__global__ void __launch_bounds__(kCopyWarps * 32)
k_compact(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
          const int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
          const unsigned char* __restrict__ keep, const int* __restrict__ dst,
          unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
          int* __restrict__ fuse_cnt, int ncopy_blocks, int NA, int acnt, int t_off, int pos_base, int late_trigger)
{
    using U = typename CopyUnit<COPY_BYTES>::type;
    const int N = H * W;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    trace_mark(const_cast<int*>(hdr), 3, false);
    if (!late_trigger) pdl_launch_dependents();  // (see k_compact_bulk)
    pdl_wait();                                  // keep flags, dst and survivor counts are complete
    if (late_trigger) pdl_launch_dependents();
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
        const int P = find_frame(cnt, gprefix, F, a, acnt, lane, -1, kk, bb);
        // a bounded wait of an earlier kernel of this call gave up: report instead of a plausible count
        if (lane == 0) *out_count = __ldcg(hdr + HDR_ERROR) ? -1 : NA + P;
    }
    const int upr = (int)(row_bytes / COPY_BYTES);         // copy units per row
    for (int j = gw; ; j += nw) {
        int f;
        if (j < NA) f = a * N + j;                         // anchor rows first (Eq. xprime_stack)
        else {
            int k, before;
            find_frame(cnt, gprefix, F, a, acnt, lane, j - NA, k, before);
            if (k < 0) break;                              // past the last output row
            const int i = select_in_frame(keep + (size_t)k * N, N, j - NA - before, lane);
            if (i < 0) break;                              // cannot happen when cnt matches keep
            f = k * N + i;
        }
        const bool row_ok = in_bounds(const_cast<int*>(hdr), 4, j, (long long)F * N) &&
                            in_bounds(const_cast<int*>(hdr), 4, f, (long long)F * N);     // (checked build)
        if (!row_ok) continue;
        if (lane < 3) {                                    // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
            const int k = f / N, i = f - k * N, yy = i / W;
            out_pos[(size_t)j * 3 + lane] = pos_base + (lane == 0 ? k + t_off : (lane == 1 ? yy : i - yy * W));
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
        fuse_cnt, 0, p.N, 0, 0, 0, 0);
    return cudaGetLastError();
}

cudaError_t launch_compact(const Problem& p, const Scratch& s, void* out_tokens, int* out_pos, int* out_count,
                           cudaStream_t st) {
    const size_t esize = p.dtype == 0 ? 4 : 2;
    const size_t row_bytes = (size_t)p.C * esize;
    const bool vec = p.vec && (reinterpret_cast<uintptr_t>(out_tokens) % 16 == 0);
    // rows emitted as the anchor block / tokens the anchor frame adds to the flat walk: (N, 0) in the paper's order
    // (Eq. xprime_stack), (0, N) in natural order, (0, 0) for a streaming segment, which does not emit its anchor
    const int NA = (p.emit_anchor && !p.natural_order) ? p.N : 0;
    const int acnt = (p.emit_anchor && p.natural_order) ? p.N : 0;
    if (p.F > kWarpPrefixMaxF) {
        k_frame_prefix<<<1, 1024, 0, st>>>(s.cnt, s.hdr, p.F, acnt, s.prefix);
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
    // the pre-scanned prefix of very long clips is read through plain loads: order that case by the stream
    const bool pdl = p.F <= kWarpPrefixMaxF;
    if (vec) {
        const size_t smem = (size_t)kCopyWarps * kBulkPiece;
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_compact_bulk), smem);
        if (e != cudaSuccess) return e;
        return launch_ex(pdl, smem, k_compact_bulk, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, s.hdr,
                         (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst, out,
                         out_pos, out_count, s.fuse_cnt, ncopy, NA, acnt, p.pos_t_offset, p.pos_base, p.chain_next,
                         wait_poll_limit(), wait_tx_extra(), p.stream_once);
    }
    if (esize == 4)
        return launch_pdl_if(pdl, k_compact<4>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                          (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                          out, out_pos, out_count, s.fuse_cnt, ncopy, NA, acnt, p.pos_t_offset, p.pos_base, p.chain_next);
    return launch_pdl_if(pdl, k_compact<2>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                      (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                      out, out_pos, out_count, s.fuse_cnt, ncopy, NA, acnt, p.pos_t_offset, p.pos_base, p.chain_next);
}

}  // namespace ttf
