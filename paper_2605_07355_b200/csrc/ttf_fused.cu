// The whole pass of one clip in ONE cooperative launch (bf16 clips with 16-byte aligned rows, r <= 1, at most
// kResolveMaxF frames): frame-sum sweep (Eq. auto_anchor) -> frame statistics -> anchor arg max + windowed
// matching + gate (Eqs. pi, argmax, dst, gating, mask) -> compaction with positions (Eqs. xprime_stack,
// compress_pos, Lpre).  The phases are separated by grid-wide barriers instead of kernel boundaries, so a clip
// pays no launch gaps, and the kernel is persistent (a fixed number of CTAs per SM that loop over units of
// work), so that the kernels of clips on other streams stay resident beside it and their phases overlap: the
// HBM-bound sweep of one clip runs under the L2-bound matching of another.
//
// Every barrier wait is bounded: a CTA that does not see the others arrive within kBarrierPolls polls sets
// the error word of the scratch header and carries on without waiting again; the call then reports
// out_count = -1.  The launch is cooperative, so all CTAs of the grid are resident whenever any of them is.
#include "ttf_internal.cuh"
#include "ttf_async.cuh"
#include "ttf_match_mma.cuh"
#include "ttf_gather.cuh"

#include <cstdlib>

namespace ttf {

constexpr int kFusedThreads = 256;
constexpr int kFusedWarps = kFusedThreads / 32;
constexpr int kBarrierPolls = 1 << 21;     // about a second of polling before a barrier gives up
constexpr int kSweepBatch = 8;             // 16-byte loads per thread in flight, and as many prefetched

static_assert(kFusedWarps == kMmaWarps && kFusedWarps == kCopyWarps, "phases share the CTA shape");

constexpr int kFusedMaxClips = kFusedBatchMax;   // clips of one launch (their pointers travel as kernel arguments)

// One clip: shape, options and the device pointers of its scratch block and outputs.
struct FusedArgs {
    const bf16_t* X;
    int F, H, W, C, r;
    float t;
    int N;
    int nq;              // 512-byte channel slices per row (sweep)
    int nsplit;          // token ranges per (frame, slice): sweep units = F * nq * nsplit
    int nsl;             // 128-channel slices of the frame statistics
    int anchor_fixed;    // >= 0: first / last / explicit anchor, no statistics
    int NA;              // anchor rows emitted in front (N, or 0 for a streaming segment)
    int t_off;           // added to the frame coordinate of every position
    int do_gather;       // 0: query (no compaction)
    int* hdr;
    int* cnt;            // [F]
    float* S;            // [nsplit][F][C]
    float* Dp;
    float* Qp;
    float* Gp;
    float* shat;
    int* dst;
    unsigned char* keep;
    int* fuse_cnt;       // may be NULL
    int* out_anchor;     // may be NULL
    unsigned char* out_tokens;
    int* out_pos;
    int* out_count;
};

struct ClipIO { const bf16_t* X; unsigned char* out_tokens; int* out_pos; int* out_count; };

// A launch: `nclips` clips of one shape.  `clip0` describes clip 0; clip n uses the scratch block `ws_stride`
// bytes further on per clip and its own io[n].  The CTAs form `ngroups` groups (CTA b belongs to group
// b % ngroups); group g runs the clips g, g + ngroups, ... one after the other, each as the four phases below
// separated by barriers among the CTAs of the group.  With two groups the HBM-bound sweep of one clip runs under
// the L2-bound matching and gather of the previous one: the sweeps take turns in clip order (a group starts the
// sweep of clip n only when the sweep of clip n - 1 is complete), which keeps the two groups half a clip apart.
// Control words (in the header of scratch block 0, zero between launches): HDR_BAR + g barrier arrivals of group
// g, HDR_SWEEP CTAs that completed a sweep, HDR_EXIT CTAs done, HDR_ERROR a bounded wait gave up.
struct BatchArgs {
    FusedArgs clip0;
    int nclips, ngroups;
    long long ws_stride;
    ClipIO io[kFusedMaxClips];
};

// ---- grid barrier ------------------------------------------------------------------------------------------
__device__ __forceinline__ int ld_acquire(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait until *counter >= target; false if it gave up (and then the error word is set).  Thread 0 only.
__device__ __forceinline__ bool wait_count(const int* counter, int target, int* err) {
    int polls = 0;
    while (ld_acquire(counter) < target) {
        if (++polls > kBarrierPolls || ((polls & 255) == 0 && ld_acquire(err) != 0)) {
            atomicExch(err, 1);
            return false;
        }
        __nanosleep(64);
    }
    return true;
}

// Barrier among the CTAs that count on `counter`: returns when `target` arrivals have been counted (the counter
// only grows during a launch).  `dead` is CTA-uniform: once a wait has given up, later barriers only arrive.
__device__ __forceinline__ void group_barrier(int* counter, int* err, int target, bool& dead) {
    __shared__ int s_dead;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(counter, 1);
        int gave_up = dead ? 1 : 0;
        if (!gave_up && !wait_count(counter, target, err)) gave_up = 1;
        __threadfence();
        s_dead = gave_up;
    }
    __syncthreads();
    dead = s_dead != 0;
}

// ---- phase 1: frame sums -----------------------------------------------------------------------------------
// Unit u = (frame k, 256-channel slice q, token range part): the sum over the tokens [i_lo, i_hi) of frame k of
// the channels of slice q, written to S[part][k][slice].  Warp w takes the tokens i_lo + w, i_lo + w + 8, ... of a
// unit in batches of kSweepBatch per thread; the warps' sums are combined in warp order.  A CTA walks its units
// u = rank, rank + size, ... as one stream of batches: the loads of the next batch (of the same or of the next
// unit) are in flight while the current one is added up and, at the end of a unit, combined and stored.
struct SweepCursor {
    int u, k, q, i_lo, i_hi, i0;        // unit, its frame / slice / token range, first token of the current batch
};

__device__ __forceinline__ void sweep_phase(const FusedArgs& A, int rank, int size, float (*sm)[kFusedWarps][256]) {
    using L = Loader<bf16_t, 8>;
    const int tid = threadIdx.x, lane = tid & 31, rg = tid >> 5;
    const int per = (A.N + A.nsplit - 1) / A.nsplit;
    const int units = A.F * A.nq * A.nsplit;
    constexpr int kStep = kFusedWarps * kSweepBatch;         // tokens of one batch over all warps

    auto open_unit = [&](SweepCursor& c, int u) {
        c.u = u;
        if (u >= units) return;
        const int part = u % A.nsplit, kq = u / A.nsplit;
        c.k = kq / A.nq; c.q = kq - c.k * A.nq;
        c.i_lo = part * per; c.i_hi = min(A.N, c.i_lo + per); c.i0 = c.i_lo;
    };
    auto advance = [&](SweepCursor& c) {                     // next batch: same unit, or the first of the next one
        c.i0 += kStep;
        if (c.i0 >= c.i_hi) open_unit(c, c.u + size);
    };
    auto load_batch = [&](typename L::Raw (&d)[kSweepBatch], const SweepCursor& c) {
        const int c0 = (c.q * 32 + lane) * 8;
        const bool active = c0 < A.C;
        const bf16_t* base = A.X + (size_t)c.k * A.N * A.C + c0;
#pragma unroll
        for (int e = 0; e < kSweepBatch; ++e) {
            const int i = c.i0 + rg + e * kFusedWarps;
            d[e] = (active && i < c.i_hi) ? L::load_raw_cg(base + (size_t)i * A.C) : L::zero();
        }
    };

    SweepCursor cur_c, nxt_c;
    open_unit(cur_c, rank);
    if (cur_c.u >= units) return;
    typename L::Raw cur[kSweepBatch], nxt[kSweepBatch];
    load_batch(cur, cur_c);
    float col[8];
#pragma unroll
    for (int v = 0; v < 8; ++v) col[v] = 0.f;
    int parity = 0;
    while (true) {
        nxt_c = cur_c;
        advance(nxt_c);
        const bool more = nxt_c.u < units;
        if (more) load_batch(nxt, nxt_c);
#pragma unroll
        for (int e = 0; e < kSweepBatch; ++e) {
            float x[8];
            L::unpack(cur[e], x);
#pragma unroll
            for (int v = 0; v < 8; ++v) col[v] += x[v];
        }
        if (nxt_c.u != cur_c.u) {                            // last batch of the unit: combine the warps
#pragma unroll
            for (int v = 0; v < 8; ++v) { sm[parity][rg][lane * 8 + v] = col[v]; col[v] = 0.f; }
            __syncthreads();                                 // (the buffer of the unit before last is free by now)
            const int c = cur_c.q * 256 + tid;
            if (c < A.C) {
                float t = 0.f;
#pragma unroll
                for (int r2 = 0; r2 < kFusedWarps; ++r2) t += sm[parity][r2][tid];
                const int part = cur_c.u % A.nsplit;
                A.S[((size_t)part * A.F + cur_c.k) * A.C + c] = t;
            }
            parity ^= 1;
        }
        if (!more) break;
        cur_c = nxt_c;
#pragma unroll
        for (int e = 0; e < kSweepBatch; ++e) cur[e] = nxt[e];
    }
    __syncthreads();
}

// ---- phase 2: frame statistics -----------------------------------------------------------------------------
// Unit q: the 128-channel slice q of g = sum_k S_k and its shares of <S_k, g>, |S_k|^2, |g|^2 (the factors 1/N and
// 1/(FN) of Eq. auto_anchor cancel in a cosine).  S_k is the sum of the sweep's token-range parts in part order.
// Warp w holds the frames w, w + 8, ... (four at a time, all of their loads in flight together).
constexpr int kStatFrames = 4;
__device__ __forceinline__ void stats_unit(const float* S, int nsplit, int F, int C, int nsl, int q,
                                           float* Dp, float* Qp, float* Gp, float (*s_gp)[128]) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int c0 = (q * 32 + lane) * 4;
    const bool on = c0 < C;
    auto frame_sums = [&](int kb, float (&x)[kStatFrames][4]) {
        float4 v[kStatFrames][kFusedMaxSplit];
#pragma unroll
        for (int jj = 0; jj < kStatFrames; ++jj)
#pragma unroll
            for (int p = 0; p < kFusedMaxSplit; ++p) {
                const int kk = kb + jj * kFusedWarps;
                v[jj][p] = (on && kk < F && p < nsplit)
                               ? __ldcg(reinterpret_cast<const float4*>(S + ((size_t)p * F + kk) * C + c0))
                               : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
        for (int jj = 0; jj < kStatFrames; ++jj) {
            x[jj][0] = x[jj][1] = x[jj][2] = x[jj][3] = 0.f;
#pragma unroll
            for (int p = 0; p < kFusedMaxSplit; ++p) {
                x[jj][0] += v[jj][p].x; x[jj][1] += v[jj][p].y; x[jj][2] += v[jj][p].z; x[jj][3] += v[jj][p].w;
            }
        }
    };
    const bool resident = F <= kFusedWarps * kStatFrames;    // this thread's frame sums all stay in registers
    float x[kStatFrames][4];
    float gacc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int kb = w; kb < F; kb += kFusedWarps * kStatFrames) {
        frame_sums(kb, x);
#pragma unroll
        for (int jj = 0; jj < kStatFrames; ++jj)
#pragma unroll
            for (int v = 0; v < 4; ++v) gacc[v] += x[jj][v];
    }
#pragma unroll
    for (int v = 0; v < 4; ++v) s_gp[w][lane * 4 + v] = gacc[v];
    __syncthreads();
    float gl[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        float g = 0.f;
#pragma unroll
        for (int ww = 0; ww < kFusedWarps; ++ww) g += s_gp[ww][lane * 4 + v];
        gl[v] = g;
    }
    for (int kb = w; kb < F; kb += kFusedWarps * kStatFrames) {      // trip count is uniform inside a warp
        if (!resident) frame_sums(kb, x);
        float d[kStatFrames], qq[kStatFrames];
#pragma unroll
        for (int jj = 0; jj < kStatFrames; ++jj) {
            d[jj] = 0.f; qq[jj] = 0.f;
#pragma unroll
            for (int v = 0; v < 4; ++v) { d[jj] = fmaf(x[jj][v], gl[v], d[jj]); qq[jj] = fmaf(x[jj][v], x[jj][v], qq[jj]); }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
            for (int jj = 0; jj < kStatFrames; ++jj) {
                d[jj] += __shfl_xor_sync(0xffffffffu, d[jj], o);
                qq[jj] += __shfl_xor_sync(0xffffffffu, qq[jj], o);
            }
#pragma unroll
        for (int jj = 0; jj < kStatFrames; ++jj) {
            const int kk = kb + jj * kFusedWarps;
            if (lane < kStatReplicas && kk < F) {            // every lane holds the sums: one lane per replica
                Dp[((size_t)lane * nsl + q) * F + kk] = d[jj];
                Qp[((size_t)lane * nsl + q) * F + kk] = qq[jj];
            }
        }
    }
    if (w == 0) {
        float gg = 0.f;
#pragma unroll
        for (int v = 0; v < 4; ++v) gg = fmaf(gl[v], gl[v], gg);
        gg = warp_sum(gg);
        if (lane < kStatReplicas) Gp[(size_t)lane * nsl + q] = gg;
    }
    __syncthreads();
}

// Tokens fused into each anchor cell j (the bookkeeping side of identity replacement) for r <= 1: one warp per
// cell, lane = source frame, the nine (keep, dst) pairs of a lane loaded together.  Integer, order-free.
__device__ __forceinline__ void fuse_count_warp(const FusedArgs& A, int a, int j, int lane) {
    const int y = j / A.W, x = j - y * A.W;
    int c = 0;
    for (int kb = 0; kb < A.F; kb += 32) {
        const int k = kb + lane;
        unsigned char kp[9];
        int ds[9];
#pragma unroll
        for (int e = 0; e < 9; ++e) {
            const int yy = y + e / 3 - 1, xx = x + e % 3 - 1;
            const bool in = k < A.F && k != a && e / 3 - 1 >= -A.r && e / 3 - 1 <= A.r && e % 3 - 1 >= -A.r &&
                            e % 3 - 1 <= A.r && yy >= 0 && yy < A.H && xx >= 0 && xx < A.W;
            const size_t f = (size_t)k * A.N + yy * A.W + xx;
            kp[e] = in ? __ldcg(A.keep + f) : (unsigned char)1;
            ds[e] = in ? __ldcg(A.dst + f) : -1;
        }
#pragma unroll
        for (int e = 0; e < 9; ++e) c += (!kp[e] && ds[e] == j) ? 1 : 0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0) A.fuse_cnt[j] = c;
}

// ---- phase 4: gather ---------------------------------------------------------------------------------------
// One warp per output row, rows interleaved over all warps of the grid: rank/select finds the source row, two
// bulk copies move it global -> shared -> global.  Returns false when a bulk-copy wait gave up.
__device__ __forceinline__ bool gather_rows(const FusedArgs& A, int a, int gw, int nw, unsigned char* buf,
                                            uint64_t* bar, uint32_t& phase) {
    const int lane = threadIdx.x & 31;
    const int N = A.N;
    const size_t row_bytes = (size_t)A.C * 2;
    const unsigned char* X = reinterpret_cast<const unsigned char*>(A.X);
    const int pieces = (int)((row_bytes + 8191) / 8192);
    bool gave_up = false;
    for (int j = gw; ; j += nw) {
        int f;
        if (j < A.NA) f = a * N + j;                 // anchor rows first (Eq. xprime_stack)
        else {
            int k, before;
            find_frame(A.cnt, nullptr, A.F, a, lane, j - A.NA, k, before);
            if (k < 0) break;                        // past the last output row
            const int i = select_in_frame(A.keep + (size_t)k * N, N, j - A.NA - before, lane);
            if (i < 0) break;
            f = k * N + i;
        }
        if (lane < 3) {                              // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
            const int k = f / N, i = f - k * N, yy = i / A.W;
            A.out_pos[(size_t)j * 3 + lane] = lane == 0 ? k + A.t_off : (lane == 1 ? yy : i - yy * A.W);
        }
        if (lane == 0 && !gave_up) {
            for (int pc = 0; pc < pieces; ++pc) {
                const size_t off = (size_t)pc * 8192;
                const uint32_t bytes = (uint32_t)(row_bytes - off < (size_t)8192 ? row_bytes - off : 8192);
                bulk_wait_read<0>();                 // the previous store has finished reading the buffer
                mbar_arrive_expect_tx(bar, bytes);
                bulk_load(buf, X + (size_t)f * row_bytes + off, bytes, bar);
                if (!mbar_wait(bar, phase & 1)) { gave_up = true; break; }
                ++phase;
                bulk_store(A.out_tokens + (size_t)j * row_bytes + off, buf, bytes);
                bulk_commit();
            }
        }
        __syncwarp();
    }
    if (lane == 0) bulk_wait<0>();                   // all rows of this warp are in global memory
    return !gave_up;
}

template <typename T>
__device__ __forceinline__ void shift_ptr(T*& p, long long off) {
    p = reinterpret_cast<T*>(reinterpret_cast<char*>(p) + off);
}

template <int NT>
__global__ void __launch_bounds__(kFusedThreads, 2)
k_ttf_fused(const __grid_constant__ BatchArgs B)
{
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ uint64_t bar[kFusedWarps];
    __shared__ float s_stat[kFusedWarps][128];
    __shared__ int s_ok;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int group = blockIdx.x % B.ngroups, rank = blockIdx.x / B.ngroups;
    const int size = (gridDim.x - group + B.ngroups - 1) / B.ngroups;      // CTAs of this group
    int* const ctl = B.clip0.hdr;
    int* const err = ctl + HDR_ERROR;
    int* const gbar = ctl + HDR_BAR + group;
    bool dead = false;
    int arrivals = 0;
    uint32_t phase = 0;

    if (lane == 0) { mbar_init(&bar[w], 1); mbar_init_fence(); }

    for (int n = group; n < B.nclips; n += B.ngroups) {
        FusedArgs A = B.clip0;
        {
            const long long off = (long long)n * B.ws_stride;
            shift_ptr(A.hdr, off); shift_ptr(A.cnt, off); shift_ptr(A.S, off);
            shift_ptr(A.Dp, off); shift_ptr(A.Qp, off); shift_ptr(A.Gp, off);
            if (B.nclips > 1) {                          // (a single clip may write these to user buffers)
                shift_ptr(A.shat, off); shift_ptr(A.dst, off); shift_ptr(A.keep, off);
                if (A.fuse_cnt) shift_ptr(A.fuse_cnt, off);
            }
            A.X = B.io[n].X; A.out_tokens = B.io[n].out_tokens; A.out_pos = B.io[n].out_pos; A.out_count = B.io[n].out_count;
        }
        if (rank == 0) for (int k = tid; k < A.F; k += kFusedThreads) A.cnt[k] = 0;

        // ---- phase 1 + 2: Anchor Frame Selection (Eq. auto_anchor) -----------------------------------------
        if (A.anchor_fixed < 0) {
            if (B.ngroups > 1 && n > 0) {                // the sweeps take turns in clip order
                if (tid == 0) s_ok = (dead || !wait_count(ctl + HDR_SWEEP, n * (int)(gridDim.x / B.ngroups), err)) ? 0 : 1;
                __syncthreads();
                if (!s_ok) dead = true;
            }
            trace_mark(A.hdr, 0, false);
            sweep_phase(A, rank, size, reinterpret_cast<float (*)[kFusedWarps][256]>(dyn_smem));
            trace_mark(A.hdr, 0, true);
            if (B.ngroups > 1 && tid == 0) { __threadfence(); atomicAdd(ctl + HDR_SWEEP, 1); }
            group_barrier(gbar, err, arrivals += size, dead);
            trace_mark(A.hdr, 1, false);
            for (int q = rank; q < A.nsl; q += size) stats_unit(A.S, A.nsplit, A.F, A.C, A.nsl, q, A.Dp, A.Qp, A.Gp, s_stat);
            trace_mark(A.hdr, 1, true);
        }
        group_barrier(gbar, err, arrivals += size, dead);    // also orders the cleared survivor counters
        trace_mark(A.hdr, 4, false);

        // ---- phase 3: Pointwise Matching with Local Window Search and Threshold Gating -----------------------
        AnchorSrc asrc;
        asrc.Dp = A.Dp; asrc.Qp = A.Qp; asrc.Gp = A.Gp; asrc.nsl = A.nsl; asrc.fixed = A.anchor_fixed;
        asrc.from_hdr = 0; asrc.hdr = A.hdr; asrc.out_anchor = A.out_anchor;
        const int a = resolve_anchor(asrc, A.F);
        if (rank == 0 && tid == 0) {
            A.hdr[HDR_ANCHOR] = a;
            if (A.out_anchor) *A.out_anchor = a;
        }
        trace_mark(A.hdr, 2, false);
        {
            const int chunks = (A.F + 31) / 32;
            const int units = A.N * chunks;
            for (int u = rank; u < units; u += size) {
                const int i = u % A.N, k0 = (u / A.N) * 32;
                match_mma_unit<2, NT, true, kMmaStagesDefault>(A.X, A.F, A.H, A.W, A.C, A.r, A.t, [a]() { return a; }, i, k0, nullptr, 0,
                                                              A.shat, A.dst, A.keep, A.cnt, dyn_smem);
                __syncthreads();
            }
        }
        trace_mark(A.hdr, 2, true);
        group_barrier(gbar, err, arrivals += size, dead);
        trace_mark(A.hdr, 3, false);

        // ---- phase 4: Token Compression and Positional Alignment ---------------------------------------------
        const int gw = rank * kFusedWarps + w, nw = size * kFusedWarps;
        if (A.do_gather) {
            if (gw == 0) {                               // L' = N + P (Eq. Lpre)
                int kk, bb;
                const int P = find_frame(A.cnt, nullptr, A.F, a, lane, -1, kk, bb);
                if (lane == 0) *A.out_count = (dead || ld_acquire(err)) ? -1 : A.NA + P;
            }
            if (A.fuse_cnt) {                            // the last N warps of the group take one anchor cell each first
                for (int j = nw - 1 - gw; j < A.N; j += nw) fuse_count_warp(A, a, j, lane);
            }
            if (!gather_rows(A, a, gw, nw, dyn_smem + (size_t)w * 8192, &bar[w], phase) && lane == 0)
                atomicExch(err, 1);
        } else if (A.fuse_cnt) {
            for (int j = gw; j < A.N; j += nw) fuse_count_warp(A, a, j, lane);
        }
        trace_mark(A.hdr, 3, true);
        __syncthreads();                                 // the staging buffers are free for the next clip's phases
    }

    // ---- leave the control words at zero for the next launch (the last CTA out resets them) ------------------
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(ctl + HDR_EXIT, 1) == (int)gridDim.x - 1) {
            if (B.clip0.do_gather && ld_acquire(err))
                for (int n = 0; n < B.nclips; ++n) *B.io[n].out_count = -1;
            ctl[HDR_BAR] = 0; ctl[HDR_BAR + 1] = 0; ctl[HDR_SWEEP] = 0; ctl[HDR_EXIT] = 0;
            __threadfence();
        }
    }
}

// ------------------------------------------------------------------------------------------------------------
bool fused_eligible(const Problem& p) {
    return p.dtype == 1 && p.vec && p.r <= 1 && p.F <= kResolveMaxF && p.C % 8 == 0;
}

static int g_fused_cps = 0;   // CTAs per SM of the fused kernel; 0 = not yet decided
void set_fused_ctas_per_sm(int n) { g_fused_cps = n < 1 ? 1 : (n > 2 ? 2 : n); }

template <int NT>
static cudaError_t launch_fused_t(const BatchArgs& B, int grid, cudaStream_t st) {
    constexpr size_t ring = sizeof(uint4) * kMmaWarps * kMmaStagesDefault * (2 * 2 + NT) * 32;
    constexpr size_t smem = ring > (size_t)kFusedWarps * 8192 ? ring : (size_t)kFusedWarps * 8192;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(k_ttf_fused<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_ttf_fused<NT>, B);
}

int fused_grid() {
    if (g_fused_cps == 0) {
        const char* e = getenv("TTF_FUSED_CTAS_PER_SM");
        set_fused_ctas_per_sm(e ? atoi(e) : 2);
    }
    return sm_count() * g_fused_cps;
}

// Token ranges per (frame, slice) so that the sweep units spread evenly over the grid: the smallest of 1, 2, 4
// that wastes less than a tenth of a round (else the best of the three).
int fused_sweep_split(const Problem& p, int grid) {
    const long long base = (long long)p.F * p.nq;
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= kFusedMaxSplit; s *= 2) {
        if (s > 1 && p.N / s < 8) break;
        const long long units = base * s;
        const long long rounds = (units + grid - 1) / grid;
        const double eff = (double)units / (double)(rounds * grid);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
        if (eff >= 0.9) break;
    }
    return best;
}

static void fill_clip(const Problem& p, const Scratch& s, int grid_per_group, FusedArgs* A) {
    A->X = reinterpret_cast<const bf16_t*>(p.X);
    A->F = p.F; A->H = p.H; A->W = p.W; A->C = p.C; A->r = p.r; A->t = p.t; A->N = p.N;
    A->nq = p.nq;
    A->nsplit = fused_sweep_split(p, grid_per_group);
    A->nsl = p.nsl;
    A->anchor_fixed = p.anchor_mode == 0 ? -1 : (p.anchor_mode == 1 ? 0 : (p.anchor_mode == 2 ? p.F - 1 : p.anchor_arg));
    A->NA = p.emit_anchor ? p.N : 0;
    A->t_off = p.pos_t_offset;
    A->hdr = s.hdr; A->cnt = s.cnt; A->S = s.S; A->Dp = s.Dp; A->Qp = s.Qp; A->Gp = s.Gp;
}

cudaError_t launch_fused(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                         unsigned char* keep, int* fuse_cnt, void* out_tokens, int* out_pos, int* out_count,
                         cudaStream_t st) {
    BatchArgs B;
    const int grid = fused_grid();
    fill_clip(p, s, grid, &B.clip0);
    FusedArgs& A = B.clip0;
    A.do_gather = out_tokens != nullptr;
    A.shat = shat; A.dst = dst; A.keep = keep; A.fuse_cnt = fuse_cnt; A.out_anchor = out_anchor;
    A.out_tokens = reinterpret_cast<unsigned char*>(out_tokens); A.out_pos = out_pos; A.out_count = out_count;
    B.nclips = 1; B.ngroups = 1; B.ws_stride = 0;
    B.io[0] = {A.X, A.out_tokens, A.out_pos, A.out_count};
    return p.r == 0 ? launch_fused_t<1>(B, grid, st) : launch_fused_t<2>(B, grid, st);
}

// `nclips` <= kFusedMaxClips clips of the shape of `p`; scratch block n = `s` shifted by n * ws_stride bytes.
cudaError_t launch_fused_batch(const Problem& p, const Scratch& s, long long ws_stride, int nclips,
                               const void* const* X, void* const* out_tokens, int* const* out_pos,
                               int* const* out_count, cudaStream_t st) {
    BatchArgs B;
    const int ngroups = nclips > 1 ? 2 : 1;
    const int grid = ngroups == 2 ? 2 * sm_count() : fused_grid();
    fill_clip(p, s, grid / ngroups, &B.clip0);
    FusedArgs& A = B.clip0;
    A.do_gather = 1;
    A.shat = s.shat; A.dst = s.dst; A.keep = s.keep; A.fuse_cnt = s.fuse_cnt; A.out_anchor = nullptr;
    A.out_tokens = nullptr; A.out_pos = nullptr; A.out_count = nullptr;
    B.nclips = nclips; B.ngroups = ngroups; B.ws_stride = ws_stride;
    for (int n = 0; n < nclips; ++n)
        B.io[n] = {reinterpret_cast<const bf16_t*>(X[n]), reinterpret_cast<unsigned char*>(out_tokens[n]), out_pos[n],
                   out_count[n]};
    return p.r == 0 ? launch_fused_t<1>(B, grid, st) : launch_fused_t<2>(B, grid, st);
}

}  // namespace ttf
