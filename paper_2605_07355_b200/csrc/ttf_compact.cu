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

constexpr int kCopyUnroll = 8;       // 16-byte units in flight per lane of the element-wise gather (two steps for an 8 KB row)

// Gather with bulk asynchronous copies, for rows that are 16-byte aligned multiples of 16 bytes.
//
// A warp owns a contiguous range of output rows.  It finds the source row of its first row by rank/select (frame
// search over the survivor counts, then a select inside that frame's keep flags) and from there on walks the keep
// flags in flat order, 128 at a time, so the search is paid once per range and not once per row.  The rows then
// move global -> shared -> global as bulk copies (no data passes through registers) through a ring of kBulkLanes
// staging slots per warp, each with its own mbarrier, driven by one lane: the loads run kBulkLanes rows ahead of
// the stores.  Every wait is bounded; a warp whose wait runs out stops copying and sets the error word.  L' (or -1 after a give-up) is written by the warp that
// finishes last, when every copy of the grid has completed or has been given up.
constexpr int kBulkWarps = 2;        // warps per CTA
constexpr int kBulkLanes = 4;        // staging slots (rows in flight) per warp
constexpr int kBulkPiece = 8192;     // bytes per staging slot; longer rows go in pieces

__global__ void __launch_bounds__(kBulkWarps * 32)
k_compact_bulk(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
               int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
               const unsigned char* __restrict__ keep, const int* __restrict__ dst,
               unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
               int* __restrict__ fuse_cnt, int ncopy_blocks, int NA, int t_off, int l2_mode, int wait_limit, int tx_extra)
{
    extern __shared__ __align__(128) unsigned char stage[];     // [kBulkWarps][kBulkLanes][kBulkPiece]
    __shared__ uint64_t bar[kBulkWarps][kBulkLanes];
    __shared__ int s_src[kBulkWarps][32];
    const int N = H * W;
    const long long FN = (long long)F * N;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    pdl_launch_dependents();                     // the next kernel of the stream may be scheduled
    if (lane < kBulkLanes) mbar_init(&bar[w][lane], 1);
    mbar_init_fence();
    __syncwarp();
    pdl_wait();                                  // keep flags, dst and survivor counts are complete
    const int a = __ldcg(hdr + HDR_ANCHOR);
    if ((int)blockIdx.x >= ncopy_blocks) {       // bookkeeping CTAs: tokens fused into each anchor cell
        fuse_count_cta(F, H, W, r, a, keep, dst, fuse_cnt, (int)blockIdx.x - ncopy_blocks, (int)gridDim.x - ncopy_blocks);
        return;
    }
    const int gw = blockIdx.x * kBulkWarps + w;
    const int nw = ncopy_blocks * kBulkWarps;
    int kk, bb;
    const int P = find_frame(cnt, gprefix, F, a, lane, -1, kk, bb);
    const int Lp = NA + P;                       // L' = N + P (Eq. Lpre)
    const int R = (Lp + nw - 1) / nw;            // rows per warp
    const long long j0 = (long long)gw * R;
    long long j1 = j0 + R < (long long)Lp ? j0 + R : (long long)Lp;

    unsigned char* wbuf = stage + (size_t)w * kBulkLanes * kBulkPiece;   // this warp's ring of slots
    const int pieces = (int)((row_bytes + kBulkPiece - 1) / kBulkPiece);
    const uint64_t pol = l2_policy(0);           // rows are read, and written, for the last time: evict-first
    uint32_t phase = 0;                          // bit s: parity the next wait on slot s expects
    bool gave_up = false;

    long long f_next = FN;                       // next flat index whose keep flag has not been looked at
    if (j0 < j1 && j1 > NA) {                    // the range holds source rows: locate the first one
        const int e0 = (int)((j0 > NA ? j0 : (long long)NA) - NA);
        int k, before;
        find_frame(cnt, gprefix, F, a, lane, e0, k, before);
        const int i = k >= 0 ? select_in_frame(keep + (size_t)k * N, N, e0 - before, lane) : -1;
        if (i >= 0) f_next = (long long)k * N + i;
    }
    for (long long jc = j0; jc < j1; jc += 32) {
        const int n = (int)(j1 - jc < 32 ? j1 - jc : 32);
        const int na = jc >= NA ? 0 : (int)(NA - jc < n ? NA - jc : n);     // anchor rows first (Eq. xprime_stack)
        if (lane < na) s_src[w][lane] = a * N + (int)jc + lane;
        const int m = n - na;
        int got = 0;
        while (got < m && f_next < FN) {
            if (f_next / N == a) { f_next = (long long)(a + 1) * N; continue; }
            unsigned char fl[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {        // 128 flags in flight, then consumed 32 at a time
                const long long f = f_next + q * 32 + lane;
                fl[q] = (f < FN && f / N != a) ? __ldcg(keep + f) : (unsigned char)0;
            }
            bool full = false;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (full) continue;
                const unsigned mask = __ballot_sync(0xffffffffu, fl[q] != 0);
                const int c = __popc(mask);
                const int rank = got + __popc(mask & ((1u << lane) - 1u));
                if (fl[q] && rank < m) s_src[w][na + rank] = (int)(f_next + q * 32 + lane);
                if (got + c >= m) {              // the range's last row of this chunk lies in this group of 32
                    f_next += q * 32 + (int)__fns(mask, 0, m - got) + 1;
                    got = m; full = true;
                } else got += c;
            }
            if (!full) f_next += 128;
        }
        const int rows = na + got;               // = n unless the counts and the flags disagree
        __syncwarp();
        // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos), three ints per row, written as one contiguous run
        for (int idx = lane; idx < 3 * rows; idx += 32) {
            const int q = idx / 3, comp = idx - 3 * q;
            const int f = s_src[w][q], k = f / N, i = f - k * N, yy = i / W;
            out_pos[(size_t)jc * 3 + idx] = comp == 0 ? k + t_off : (comp == 1 ? yy : i - yy * W);
        }
        if (lane == 0 && !gave_up) {
            // one lane drives the warp's ring of kBulkLanes slots: loads run ahead of the stores by that many items
            // (item = one piece of one row), so the latency of a load is paid once per ring, not once per row
            const int items = rows * pieces;
            auto issue = [&](int it) {
                const int q = it / pieces, pc = it - q * pieces, slot = it % kBulkLanes;
                const size_t off = (size_t)pc * kBulkPiece;
                const uint32_t bytes = (uint32_t)(row_bytes - off < (size_t)kBulkPiece ? row_bytes - off : kBulkPiece);
                const unsigned char* src = X + (size_t)s_src[w][q] * row_bytes + off;
                mbar_arrive_expect_tx(&bar[w][slot], bytes + (uint32_t)tx_extra);
                if (l2_mode) bulk_load_hint(wbuf + (size_t)slot * kBulkPiece, src, bytes, &bar[w][slot], pol);
                else bulk_load(wbuf + (size_t)slot * kBulkPiece, src, bytes, &bar[w][slot]);
            };
            bulk_wait_read<0>();                 // the previous chunk's stores have finished reading the slots
            for (int it = 0; it < items && it < kBulkLanes; ++it) issue(it);
            for (int it = 0; it < items; ++it) {
                const int q = it / pieces, pc = it - q * pieces, slot = it % kBulkLanes;
                const size_t off = (size_t)pc * kBulkPiece;
                const uint32_t bytes = (uint32_t)(row_bytes - off < (size_t)kBulkPiece ? row_bytes - off : kBulkPiece);
                if (!mbar_wait(&bar[w][slot], (phase >> slot) & 1, wait_limit)) {
                    // give the copies in flight one more bounded chance to land before the ring is abandoned
                    for (int u = it; u < items && u < it + kBulkLanes; ++u)
                        mbar_wait(&bar[w][u % kBulkLanes], (phase >> (u % kBulkLanes)) & 1, wait_limit);
                    gave_up = true;
                    break;
                }
                phase ^= 1u << slot;
                unsigned char* out = out_tokens + (size_t)(jc + q) * row_bytes + off;
                if (l2_mode) bulk_store_hint(out, wbuf + (size_t)slot * kBulkPiece, bytes, pol);
                else bulk_store(out, wbuf + (size_t)slot * kBulkPiece, bytes);
                bulk_commit();
                if (it + kBulkLanes < items) {
                    bulk_wait_read<0>();         // the store just issued has finished reading the slot
                    issue(it + kBulkLanes);
                }
            }
        }
        __syncwarp();                            // s_src is rewritten by the next chunk
    }
    if (lane == 0) {                             // the warp that arrives last publishes L'
        bulk_wait<0>();                          // all rows of this warp are in global memory
        if (gave_up) atomicExch(hdr + HDR_ERROR, 1);
        __threadfence();
        if (atomicAdd(hdr + HDR_GATHER_DONE, 1) == nw - 1) {
            __threadfence();
            *out_count = atomicAdd(hdr + HDR_ERROR, 0) ? -1 : Lp;
            hdr[HDR_GATHER_DONE] = 0;            // left at zero for the next call
        }
    }
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
        const size_t smem = (size_t)kBulkWarps * kBulkLanes * kBulkPiece;
        cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_compact_bulk), smem);
        if (e != cudaSuccess) return e;
        // three CTAs of 64 KB per SM; a warp takes ceil(L' / warps) rows
        const int nbulk = 3 * sm_count();
        int nf = (p.N + kBulkWarps - 1) / kBulkWarps;
        if (nf > sm_count()) nf = sm_count();
        return launch_ex(pdl, smem, k_compact_bulk, dim3(nbulk + nf), dim3(kBulkWarps * 32), st, X, row_bytes, p.F, p.H,
                         p.W, p.r, s.hdr, (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep,
                         (const int*)s.dst, out, out_pos, out_count, s.fuse_cnt, nbulk, NA, p.pos_t_offset, p.l2_mode,
                         wait_poll_limit(), wait_tx_extra());
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
