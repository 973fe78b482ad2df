// Pointwise Matching with Local Window Search and Threshold Gating (Eqs. pi, argmax, dst, gating, mask) for bf16
// clips on the fifth-generation tensor cores: TMA tensor tiles -> shared memory -> tcgen05.mma -> tensor memory.
//
// All tokens of a grid cell share their candidate set, and neighbouring cells share most of it, so the unit of
// work is a TILE of 128 source rows = 32 frames x a strip of 4 cells of one grid row, against the
// (2r+1) x (4+2r) anchor cells around the strip (18 for r = 1): one dense contraction
//     D[128 x NB] = A[128 x C] . B[NB x C]^T,     NB = 16 / 32 / 48 >= (2r+1)(4+2r),
// of which every source row uses its own (2r+1)^2 columns.  Operand traffic is (128 + 18) / 128 = 1.14 x |X| for
// r = 1 instead of 41 / 32 when every cell fetches its own 9 candidates.
//
//   A tile:  box (64 channels, 4 cells, 1 row, 32 frames) of X viewed as [F, H, W, C]; row m = 4 * frame + cell.
//   B tile:  box (64 channels, 4 + 2r cells, 2r + 1 rows, 1 frame) at frame a*, starting r cells up and left of the
//            strip; cells outside the grid arrive as zeros and are left out of the arg max (window clipped to the
//            grid, Eq. pi, with the duplicates of the clipping masked).
//   Both arrive with the 128-byte swizzle, which is the K-major operand layout of tcgen05.mma; a pipeline stage is
//   64 channels (4 MMAs of K = 16).  fp32 accumulation in tensor memory; bf16 products are exact in fp32.
//
// The channel range of a tile is cut into `pieces` consecutive parts, one CTA each, so that a small clip still gives
// about two CTAs per SM.  The CTAs of a tile form a thread-block cluster: when their pipelines have drained, ranks
// > 0 write their partial sums into rank 0's shared memory (distributed shared memory, two cluster barriers) and
// rank 0 adds them in rank order, so the result does not depend on scheduling.
// Token norms are taken from the tiles themselves: while the pipeline runs, every epilogue thread adds up the squares
// of "its" source row (and the first NCAND threads those of a candidate row) as the stages pass through shared memory.
// Warp roles: 0 TMA producer, 1 tensor-memory owner and MMA issuer, 2-5 epilogue (one tensor-memory lane = one
// source row per thread).
//
// Every mbarrier wait is bounded; a wait that runs out sets the error word of the call, the CTA stops feeding its
// pipeline, waits (bounded again) for the copies it has in flight, frees its tensor memory and returns.
#include <cuda.h>

#include "ttf_internal.cuh"
#include "ttf_async.cuh"

#include <map>
#include <mutex>

namespace ttf {

constexpr int kTcWB = 4;                 // cells per strip
constexpr int kTcFR = 32;                // frames per tile
constexpr int kTcM = kTcWB * kTcFR;      // 128 source rows = tensor-memory lanes
constexpr int kTcKC = 64;                // channels per stage (128 bytes: one swizzle row)
constexpr int kTcABytes = kTcM * 128;    // 16 KB
constexpr int kTcThreads = 192;

// ---- PTX wrappers -----------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_4d(void* dst_smem, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3),
          "r"(smem_u32(bar))
        : "memory");
}
// the same copy with an L2 cache policy (createpolicy) on the lines it reads
__device__ __forceinline__ void tma_load_4d_hint(void* dst_smem, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
        ::"r"(smem_u32(dst_smem)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3),
          "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tensormap_prefetch(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// whole warp: allocates `cols` (a power of two >= 32) columns of tensor memory, base address -> *dst_smem
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem desc] . B[smem desc]^T, issued by one thread
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// the barrier receives one arrival when every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 16 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void epilogue_bar_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// K-major operand tile with the 128-byte swizzle: rows of 128 bytes, groups of 8 rows 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);          // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset (not used by swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                               // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}
// bf16 x bf16 -> fp32, A and B K-major, M = 128, N = NB
__host__ __device__ constexpr uint32_t idesc_bf16(int NB) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NB >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
}

// ---- the kernel -------------------------------------------------------------------------------------------
template <int R> struct TcShape {
    static constexpr int SIDE = 2 * R + 1;
    static constexpr int BW = kTcWB + 2 * R;              // candidate cells per window row
    static constexpr int NCAND = SIDE * BW;               // rows the B box delivers
    static constexpr int NB = (NCAND + 15) / 16 * 16;     // MMA N
    static constexpr int BBYTES = NB * 128;
    static constexpr int BBOX = NCAND * 128;              // bytes one B box copy delivers
    static constexpr int STAGE = kTcABytes + BBYTES;
    static constexpr int STAGES = 4;                      // two CTAs per SM with room left for CTAs of other kernels
    static constexpr int TMEM_COLS = NB <= 32 ? 32 : 64;
    static constexpr int WIN = SIDE * SIDE;               // candidates of one source row
};

// ---- thread-block clusters: the CTAs of one tile exchange their partial sums through distributed shared memory
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// all threads of all CTAs of the cluster; writes before it are visible to every CTA of the cluster after it
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f32(uint32_t local_smem_addr, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_smem_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// sum of squares of the 8 bf16 values of a 16-byte piece
__device__ __forceinline__ float ssq8(const uint4& v, float acc) {
    float x;
    x = bf16_lo(v.x); acc = fmaf(x, x, acc); x = bf16_hi(v.x); acc = fmaf(x, x, acc);
    x = bf16_lo(v.y); acc = fmaf(x, x, acc); x = bf16_hi(v.y); acc = fmaf(x, x, acc);
    x = bf16_lo(v.z); acc = fmaf(x, x, acc); x = bf16_hi(v.z); acc = fmaf(x, x, acc);
    x = bf16_lo(v.w); acc = fmaf(x, x, acc); x = bf16_hi(v.w); acc = fmaf(x, x, acc);
    return acc;
}

template <int R>
__global__ void __launch_bounds__(kTcThreads)
k_match_tc(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
           int F, int H, int W, int C, float t, AnchorSrc asrc, int pieces,
           float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt,
           int wait_limit, int tx_extra, int stream_once)
{
    using S = TcShape<R>;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ uint64_t bar_full[S::STAGES], bar_empty[S::STAGES], bar_acc;
    __shared__ uint32_t s_tmem;
    __shared__ int s_err;
    __shared__ float s_nb[S::NCAND];                       // 1 / norm of the candidate rows
    __shared__ float s_nbp[S::NCAND * 8];                  // ... per 16-byte piece column, before they are added up

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = H * W;
    const int xs_n = (W + kTcWB - 1) / kTcWB;
    const int tile = blockIdx.x / pieces;
    const int piece = pieces > 1 ? (int)cluster_rank() : 0;        // = blockIdx.x % pieces
    const int kg = tile / (H * xs_n), rem = tile - kg * (H * xs_n);
    const int y = rem / xs_n, x0 = (rem - y * xs_n) * kTcWB;
    const int k0 = kg * kTcFR;
    const int nst_all = (C + kTcKC - 1) / kTcKC;
    const int st0 = (int)((long long)nst_all * piece / pieces), st1 = (int)((long long)nst_all * (piece + 1) / pieces);
    const int nst = st1 - st0;

    // 1024-byte aligned stage ring (the swizzle pattern is a function of the shared-memory address)
    const uint32_t dyn_base = (smem_u32(dyn_raw) + 1023u) & ~1023u;
    unsigned char* dyn = dyn_raw + (dyn_base - smem_u32(dyn_raw));

    pdl_launch_dependents();
    trace_mark(asrc.hdr, 2, false);
    if (tid == 0) {
        // a stage is full when its two copies have landed, and free again when the MMAs that read it have completed
        // and each of the four epilogue warps has taken its share of the norms from it
        for (int s = 0; s < S::STAGES; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 5); }
        mbar_init(&bar_acc, 1);
        mbar_init_fence();
        s_err = 0;
        tensormap_prefetch(&mapA);
        tensormap_prefetch(&mapB);
    }
    // the B rows beyond the box (NCAND .. NB-1) are never written by a copy: zero them once
    for (int i = tid; i < S::STAGES * (S::BBYTES - S::BBOX) / 16; i += kTcThreads) {
        const int s = i / ((S::BBYTES - S::BBOX) / 16), o = i - s * ((S::BBYTES - S::BBOX) / 16);
        reinterpret_cast<uint4*>(dyn + (size_t)s * S::STAGE + kTcABytes + S::BBOX)[o] = make_uint4(0, 0, 0, 0);
    }
    fence_async_smem();
    if (warp == 1) tmem_alloc(&s_tmem, S::TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;

    // everything upstream (the anchor, and whatever produced X) is complete after this wait
    trace_mark(asrc.hdr, 11, false); trace_mark(asrc.hdr, 11, true);     // set-up done
    pdl_wait();
    trace_mark(asrc.hdr, 5, false);
    const int a = asrc.fixed >= 0 ? asrc.fixed : __ldcg(asrc.hdr + HDR_ANCHOR);
    if (blockIdx.x == 0 && tid == 0 && asrc.fixed >= 0) {
        asrc.hdr[HDR_ANCHOR] = a;                // the gather reads it from here
        if (asrc.out_anchor) *asrc.out_anchor = a;
    }

    // epilogue-thread state that outlives the role code
    const int q = warp & 3;                                // tensor-memory lane quadrant an epilogue warp may read
    const int m = q * 32 + lane;                           // source row of an epilogue thread: 4 * frame + cell
    const int et = (warp - 2) * 32 + lane;                 // 0..127 among the epilogue threads
    float win[S::WIN];                                     // this row's window of dot products
    float na = 0.f, nb = 0.f;                              // squared norm of source row m / of candidate row et

    if (warp == 0) {
        // ---- producer: one lane issues the tile copies of every stage ----------------------------------------
        if (lane == 0) {
            int issued = 0;
            const uint64_t once = l2_evict_first_policy();
            for (int it = 0; it < nst; ++it) {
                const int s = it % S::STAGES;
                if (it >= S::STAGES && !mbar_wait(&bar_empty[s], ((it / S::STAGES) & 1) ^ 1, wait_limit)) { atomicExch(&s_err, 1); break; }
                if (*(volatile int*)&s_err) break;
                unsigned char* sa = dyn + (size_t)s * S::STAGE;
                const int c0 = (st0 + it) * kTcKC;
                mbar_arrive_expect_tx(&bar_full[s], kTcABytes + S::BBOX + (uint32_t)tx_extra);   // (extra: test hook only)
                // source rows are read by this tile alone: in a schedule that streams the next clip into L2 meanwhile,
                // their lines are the ones to give up first (the candidate rows are shared with neighbouring tiles)
                if (stream_once) tma_load_4d_hint(sa, &mapA, c0, x0, y, k0, &bar_full[s], once);
                else tma_load_4d(sa, &mapA, c0, x0, y, k0, &bar_full[s]);
                tma_load_4d(sa + kTcABytes, &mapB, c0, x0 - R, y - R, a, &bar_full[s]);
                issued = it + 1;
            }
            trace_mark_any(asrc.hdr, 12, false); trace_mark_any(asrc.hdr, 12, true);   // all copies issued
            if (*(volatile int*)&s_err) {
                // copies already issued still land in this CTA's shared memory: wait (bounded) for the stages that
                // nobody consumed before the CTA is allowed to exit
                for (int it = issued > S::STAGES ? issued - S::STAGES : 0; it < issued; ++it)
                    mbar_wait(&bar_full[it % S::STAGES], (it / S::STAGES) & 1, wait_limit);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one lane, four K = 16 steps per stage -----------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(S::NB);
            for (int it = 0; it < nst; ++it) {
                const int s = it % S::STAGES;
                if (!mbar_wait(&bar_full[s], (it / S::STAGES) & 1, wait_limit)) { atomicExch(&s_err, 1); break; }
                tc_fence_after();
                const uint32_t sa = dyn_base + (uint32_t)s * S::STAGE;
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + kTcABytes);
#pragma unroll
                for (int k = 0; k < kTcKC / 16; ++k)       // 32 bytes further along K inside the swizzle row
                    umma_bf16(tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, it > 0 || k > 0);
                umma_commit(&bar_empty[s]);                // one of the five arrivals that free the stage
            }
            umma_commit(&bar_acc);                         // accumulator complete (also arrives after a give-up)
        }
    } else {
        // ---- epilogue warps, part 1: while the pipeline runs, the squared norms of the rows that pass through
        // shared memory (source row m by every thread, candidate row et by the first NCAND threads).  A row is 128
        // bytes per stage; its 16-byte pieces sit at (piece ^ (row & 7)) (the 128-byte swizzle), and a sum of
        // squares does not care in which order it meets them ---------------------------------------------------
        bool ok = true;
        constexpr int NP = S::NCAND * 8;                   // (candidate row, 16-byte piece column) pairs
        constexpr int PP = (NP + 127) / 128;               // pairs per epilogue thread
        float na8[8], nbq[PP];                             // one running sum per piece column: eight short chains
#pragma unroll
        for (int c = 0; c < 8; ++c) na8[c] = 0.f;
#pragma unroll
        for (int u = 0; u < PP; ++u) nbq[u] = 0.f;
        for (int it = 0; it < nst; ++it) {
            const int s = it % S::STAGES;
            if (!mbar_wait(&bar_full[s], (it / S::STAGES) & 1, wait_limit)) { atomicExch(&s_err, 1); ok = false; break; }
            const unsigned char* sa = dyn + (size_t)s * S::STAGE;
            const uint4* rowa = reinterpret_cast<const uint4*>(sa + (size_t)m * 128);
            uint4 va[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) va[c] = rowa[c ^ (m & 7)];
            uint4 vb[PP];
#pragma unroll
            for (int u = 0; u < PP; ++u) {
                const int pr = et + u * 128, row = pr >> 3, pc = pr & 7;
                vb[u] = pr < NP ? reinterpret_cast<const uint4*>(sa + kTcABytes + (size_t)row * 128)[pc ^ (row & 7)]
                                : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) na8[c] = ssq8(va[c], na8[c]);
#pragma unroll
            for (int u = 0; u < PP; ++u) nbq[u] = ssq8(vb[u], nbq[u]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_empty[s]);
        }
        na = ((na8[0] + na8[1]) + (na8[2] + na8[3])) + ((na8[4] + na8[5]) + (na8[6] + na8[7]));
#pragma unroll
        for (int u = 0; u < PP; ++u) if (et + u * 128 < NP) s_nbp[et + u * 128] = nbq[u];
        epilogue_bar_sync();
        if (et < S::NCAND) {
            const float* pp = s_nbp + et * 8;
            nb = ((pp[0] + pp[1]) + (pp[2] + pp[3])) + ((pp[4] + pp[5]) + (pp[6] + pp[7]));
        }
        if (et == 0) { trace_mark_any(asrc.hdr, 13, false); trace_mark_any(asrc.hdr, 13, true); }   // norms done
        // ---- part 2: the accumulator ---------------------------------------------------------------------------
        if (ok) ok = mbar_wait(&bar_acc, 0, wait_limit);
        if (!ok) atomicExch(&s_err, 1);
        if (et == 0) { trace_mark_any(asrc.hdr, 14, false); trace_mark_any(asrc.hdr, 14, true); }   // accumulator complete
        tc_fence_after();
        float d[S::NB];
        if (ok) {
#pragma unroll
            for (int c = 0; c < S::NB / 16; ++c) {
                float v[16];
                tmem_ld16(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 16), v);
#pragma unroll
                for (int i = 0; i < 16; ++i) d[c * 16 + i] = v[i];
            }
        } else {
#pragma unroll
            for (int i = 0; i < S::NB; ++i) d[i] = 0.f;
        }
        // this row's window: candidate (dy, ddx) is column (dy + R) * BW + dx + ddx + R of the tile
        const int dx = m & 3;
#pragma unroll
        for (int wy = 0; wy < S::SIDE; ++wy)
#pragma unroll
            for (int wx = 0; wx < S::SIDE; ++wx) {
                const int n0 = wy * S::BW + wx;
                win[wy * S::SIDE + wx] = dx == 0 ? d[n0] : (dx == 1 ? d[n0 + 1] : (dx == 2 ? d[n0 + 2] : d[n0 + 3]));
            }
    }

    // ---- split K: the CTAs of a tile form a cluster; ranks > 0 hand their partial sums to rank 0 through its
    // shared memory (the stage ring, idle by then) and rank 0 adds them in rank order ----------------------------
    constexpr int XROW = (S::WIN + 1) * kTcM + S::NCAND;   // floats one rank sends: window sums, row norms, candidate norms
    if (pieces > 1) {
        __syncwarp();
        cluster_sync_all();                                // every CTA of the tile is past its pipeline: rank 0's ring is idle
        if (warp >= 2 && piece > 0) {
            const uint32_t base = dyn_base + (uint32_t)(piece - 1) * XROW * 4;
#pragma unroll
            for (int c = 0; c < S::WIN; ++c) st_cluster_f32(base + (uint32_t)(c * kTcM + m) * 4, 0, win[c]);
            st_cluster_f32(base + (uint32_t)(S::WIN * kTcM + m) * 4, 0, na);
            if (et < S::NCAND) st_cluster_f32(base + (uint32_t)((S::WIN + 1) * kTcM + et) * 4, 0, nb);
        }
        __syncwarp();
        cluster_sync_all();
        if (warp >= 2 && piece == 0) {
            const float* xin = reinterpret_cast<const float*>(dyn);
            for (int p = 1; p < pieces; ++p) {             // rank order
                const float* xp = xin + (size_t)(p - 1) * XROW;
#pragma unroll
                for (int c = 0; c < S::WIN; ++c) win[c] += xp[c * kTcM + m];
                na += xp[S::WIN * kTcM + m];
                if (et < S::NCAND) nb += xp[(S::WIN + 1) * kTcM + et];
            }
        }
    }

    if (warp >= 2 && piece == 0) {
        // ---- epilogue, part 3 (rank 0 of the tile): cosine, arg max over the window clipped to the grid, gate --
        if (et < S::NCAND) s_nb[et] = 1.0f / fmaxf(sqrtf(nb), kNormFloor);     // once per candidate row, not once per use
        epilogue_bar_sync();
        const int kl = m >> 2, dx = m & 3;
        const int k = k0 + kl, x = x0 + dx;
        if (k < F && x < W && in_bounds(asrc.hdr, 3, (long long)k * N + (long long)y * W + x, (long long)F * N)) {
            const size_t f = (size_t)k * N + (size_t)y * W + x;
            if (k == a) {                                  // anchor tokens are always retained (Eq. mask)
                shat[f] = 1.0f; dst[f] = y * W + x; keep[f] = 1;
            } else {
                const float rs = 1.0f / fmaxf(sqrtf(na), kNormFloor);
                float best = -INFINITY;
                int best_j = -1;
#pragma unroll
                for (int wy = 0; wy < S::SIDE; ++wy)
#pragma unroll
                    for (int wx = 0; wx < S::SIDE; ++wx) {     // ascending anchor index among in-grid cells
                        const int yy = y + wy - R, xx = x + wx - R;
                        if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                        const float sim = win[wy * S::SIDE + wx] * rs * s_nb[wy * S::BW + dx + wx];
                        if (sim > best || best_j < 0) { best = sim; best_j = yy * W + xx; }
                    }
                const unsigned char kp = !(best > t);
                shat[f] = best; dst[f] = best_j; keep[f] = kp;
                if (kp) atomicAdd(&cnt[k], 1);
            }
        }
    }

    // ---- teardown: every role is done with tensor memory before its owner frees it --------------------------
    tc_fence_before();
    __syncthreads();
    trace_mark(asrc.hdr, 2, true);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, S::TMEM_COLS);
    }
    if (tid == 0 && s_err) atomicExch(asrc.hdr + HDR_ERROR, 1);
}

// ---- host side: tensor maps and launch ------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static std::mutex mu;
    static EncodeTiledFn fn = nullptr;
    std::lock_guard<std::mutex> lk(mu);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// X viewed as [F, H, W, C] (C innermost), one box of (64, bw, bh, bf) elements, 128-byte swizzle, zeros outside
static bool make_map(CUtensorMap* m, const void* X, int F, int H, int W, int C, int bw, int bh, int bf) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)F};
    const cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    const cuuint32_t box[4] = {(cuuint32_t)kTcKC, (cuuint32_t)bw, (cuuint32_t)bh, (cuuint32_t)bf};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(X), dims, strides, box, estr,
               // (256-byte L2 promotion: the next stage reads the next 128 bytes of the same rows; 5 - 9 % faster than 128)
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_match_eligible(const Problem& p) {
    if (p.dtype != 1 || !p.vec || p.r > 2 || p.C < kTcKC) return false;
    return (long long)tc_match_tiles(p) * 8 < (1LL << 31);
}

size_t tc_match_tiles(const Problem& p) {
    return (size_t)((p.F + kTcFR - 1) / kTcFR) * p.H * ((p.W + kTcWB - 1) / kTcWB);
}

// CTAs (= cluster size) per tile: the largest power of two that still fits the GPU in one wave of two CTAs per SM,
// at most 8 (4 for r = 2, whose exchange rows are longer) and at least 4 stages each.  (One CTA per SM with a ring
// twice as deep measured the same alone, 18.8 against 19.2 us on a cold 8B-shaped clip, and slower with other clips'
// kernels beside it, 34.0 against 32.2 us per clip.)
int tc_match_pieces(const Problem& p) {
    const long long tiles = (long long)tc_match_tiles(p);
    const int nst = (p.C + kTcKC - 1) / kTcKC;
    const int cap = p.r == 2 ? 4 : 8;
    int pieces = 1;
    while (pieces * 2 <= cap && tiles * (pieces * 2) <= 2LL * sm_count() && nst / (pieces * 2) >= 4) pieces *= 2;
    return pieces;
}

template <int R>
static cudaError_t launch_tc_t(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                               unsigned char* keep, cudaStream_t st) {
    using S = TcShape<R>;
    static_assert((size_t)7 * ((S::WIN + 1) * kTcM + S::NCAND) * 4 <= (size_t)S::STAGES * S::STAGE || R == 2, "exchange rows must fit the ring");
    static_assert((size_t)3 * ((S::WIN + 1) * kTcM + S::NCAND) * 4 <= (size_t)S::STAGES * S::STAGE, "exchange rows must fit the ring");
    CUtensorMap mapA, mapB;
    if (!make_map(&mapA, p.X, p.F, p.H, p.W, p.C, kTcWB, 1, kTcFR) ||
        !make_map(&mapB, p.X, p.F, p.H, p.W, p.C, S::BW, S::SIDE, 1))
        return cudaErrorInvalidValue;
    const size_t smem = (size_t)S::STAGES * S::STAGE + 1024;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_match_tc<R>), smem);
    if (e != cudaSuccess) return e;
    const int pieces = tc_match_pieces(p);
    const long long tiles = (long long)tc_match_tiles(p);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * pieces)); cfg.blockDim = dim3(kTcThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    int n = 1;
    if (pieces > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)pieces; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr; cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, k_match_tc<R>, mapA, mapB, p.F, p.H, p.W, p.C, p.t, make_anchor_src(p, s, out_anchor),
                              pieces, shat, dst, keep, s.cnt, wait_poll_limit(), wait_tx_extra(), p.stream_once);
}

cudaError_t launch_match_tc(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                            unsigned char* keep, cudaStream_t st) {
    if (p.r == 0) return launch_tc_t<0>(p, s, out_anchor, shat, dst, keep, st);
    if (p.r == 1) return launch_tc_t<1>(p, s, out_anchor, shat, dst, keep, st);
    return launch_tc_t<2>(p, s, out_anchor, shat, dst, keep, st);
}

}  // namespace ttf
