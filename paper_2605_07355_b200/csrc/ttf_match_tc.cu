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
// The channel range of a tile is cut into `pieces` consecutive parts, one CTA each, so that a clip gives at least
// two CTAs per SM; the partial sums of a tile go through global memory and are added in piece order by whichever
// CTA of the tile arrives last (an arrival counter per tile), so the result does not depend on scheduling.
// Token norms come from the sweep's partial squared norms.  Warp roles: 0 TMA producer, 1 tensor-memory owner and
// MMA issuer, 2-5 epilogue (one tensor-memory lane = one source row per thread).
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
    static constexpr int STAGES = R == 2 ? 4 : 5;
    static constexpr int TMEM_COLS = NB <= 32 ? 32 : 64;
    static constexpr int WIN = SIDE * SIDE;               // candidates of one source row
};

template <int R>
__global__ void __launch_bounds__(kTcThreads)
k_match_tc(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
           int F, int H, int W, int C, float t, AnchorSrc asrc, const float* __restrict__ ssq, int nslice,
           int pieces, float* __restrict__ part, int* __restrict__ tile_cnt,
           float* __restrict__ shat, int* __restrict__ dst, unsigned char* __restrict__ keep, int* __restrict__ cnt,
           int wait_limit)
{
    using S = TcShape<R>;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ uint64_t bar_full[S::STAGES], bar_empty[S::STAGES], bar_acc;
    __shared__ uint32_t s_tmem;
    __shared__ int s_err, s_last;
    __shared__ float s_ra[S::NCAND];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = H * W;
    const int xs_n = (W + kTcWB - 1) / kTcWB;
    const int tile = blockIdx.x / pieces, piece = blockIdx.x - tile * pieces;
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
    if (tid == 0) {
        for (int s = 0; s < S::STAGES; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_acc, 1);
        mbar_init_fence();
        s_err = 0; s_last = 0;
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

    // everything upstream (the sweep's norms, the anchor, and whatever produced X) is complete after this wait
    pdl_wait();
    const int a = asrc.fixed >= 0 ? asrc.fixed : __ldcg(asrc.hdr + HDR_ANCHOR);
    if (blockIdx.x == 0 && tid == 0 && asrc.fixed >= 0) {
        asrc.hdr[HDR_ANCHOR] = a;                // the gather reads it from here
        if (asrc.out_anchor) *asrc.out_anchor = a;
    }

    if (warp == 0) {
        // ---- producer: one lane issues the tile copies of every stage ----------------------------------------
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < nst; ++it) {
                const int s = it % S::STAGES;
                if (it >= S::STAGES && !mbar_wait(&bar_empty[s], ((it / S::STAGES) & 1) ^ 1, wait_limit)) { atomicExch(&s_err, 1); break; }
                if (*(volatile int*)&s_err) break;
                unsigned char* sa = dyn + (size_t)s * S::STAGE;
                const int c0 = (st0 + it) * kTcKC;
                mbar_arrive_expect_tx(&bar_full[s], kTcABytes + S::BBOX);
                tma_load_4d(sa, &mapA, c0, x0, y, k0, &bar_full[s]);
                tma_load_4d(sa + kTcABytes, &mapB, c0, x0 - R, y - R, a, &bar_full[s]);
                issued = it + 1;
            }
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
            bool ok = true;
            for (int it = 0; it < nst && ok; ++it) {
                const int s = it % S::STAGES;
                if (!mbar_wait(&bar_full[s], (it / S::STAGES) & 1, wait_limit)) { atomicExch(&s_err, 1); ok = false; break; }
                tc_fence_after();
                const uint32_t sa = dyn_base + (uint32_t)s * S::STAGE;
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sa + kTcABytes);
#pragma unroll
                for (int k = 0; k < kTcKC / 16; ++k)       // 32 bytes further along K inside the swizzle row
                    umma_bf16(tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc, it > 0 || k > 0);
                umma_commit(&bar_empty[s]);                // the stage is free once these MMAs have read it
            }
            umma_commit(&bar_acc);                         // accumulator complete (also arrives after a give-up)
        }
    } else {
        // ---- epilogue: thread = source row m = 4 * frame + cell ----------------------------------------------
        const int q = warp & 3;                            // tensor-memory lane quadrant this warp may read
        const int m = q * 32 + lane;
        const int et = (warp - 2) * 32 + lane;             // 0..127 among the epilogue threads
        const int kl = m >> 2, dx = m & 3;
        const int k = k0 + kl, x = x0 + dx;
        const bool row_ok = k < F && x < W;
        const size_t FN = (size_t)F * N;
        const size_t f = (size_t)(row_ok ? k : 0) * N + (size_t)y * W + (row_ok ? x : 0);
        // inverse norms (independent of the accumulator: fetched while the pipeline runs)
        const float rs = row_ok ? inv_norm(ssq, nslice, FN, f) : 0.f;
        if (et < S::NCAND) {
            const int yy = y - R + et / S::BW, xx = x0 - R + et % S::BW;
            s_ra[et] = (yy >= 0 && yy < H && xx >= 0 && xx < W) ? inv_norm(ssq, nslice, FN, (size_t)a * N + (size_t)yy * W + xx) : 0.f;
        }
        bool ok = mbar_wait(&bar_acc, 0, wait_limit);
        if (!ok) atomicExch(&s_err, 1);
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
        float win[S::WIN];
#pragma unroll
        for (int wy = 0; wy < S::SIDE; ++wy)
#pragma unroll
            for (int wx = 0; wx < S::SIDE; ++wx) {
                const int n0 = wy * S::BW + wx;
                win[wy * S::SIDE + wx] = dx == 0 ? d[n0] : (dx == 1 ? d[n0 + 1] : (dx == 2 ? d[n0 + 2] : d[n0 + 3]));
            }
        bool last = true;
        if (pieces > 1) {
            // partial sums of this piece: [tile][piece][candidate][row], rows contiguous across the threads
            float* mine = part + ((size_t)blockIdx.x * S::WIN) * kTcM + m;
#pragma unroll
            for (int c = 0; c < S::WIN; ++c) __stcg(mine + (size_t)c * kTcM, win[c]);
            __threadfence();
            epilogue_bar_sync();
            if (et == 0) s_last = atomicAdd(tile_cnt + tile, 1) == pieces - 1;
            epilogue_bar_sync();
            last = s_last != 0;
            if (last) {
                __threadfence();
                const float* all = part + ((size_t)tile * pieces * S::WIN) * kTcM + m;
#pragma unroll
                for (int c = 0; c < S::WIN; ++c) {
                    float sum = 0.f;
                    for (int p = 0; p < pieces; ++p) sum += __ldcg(all + ((size_t)p * S::WIN + c) * kTcM);   // piece order
                    win[c] = sum;
                }
                if (et == 0) tile_cnt[tile] = 0;           // left at zero for the next call
            }
        } else {
            epilogue_bar_sync();                           // s_ra is complete
        }
        if (last && row_ok) {
            if (k == a) {                                  // anchor tokens are always retained (Eq. mask)
                shat[f] = 1.0f; dst[f] = y * W + x; keep[f] = 1;
            } else {
                float best = -INFINITY;
                int best_j = -1;
#pragma unroll
                for (int wy = 0; wy < S::SIDE; ++wy)
#pragma unroll
                    for (int wx = 0; wx < S::SIDE; ++wx) {     // ascending anchor index among in-grid cells
                        const int yy = y + wy - R, xx = x + wx - R;
                        if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
                        const float s = win[wy * S::SIDE + wx] * rs * s_ra[wy * S::BW + dx + wx];
                        if (s > best || best_j < 0) { best = s; best_j = yy * W + xx; }
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
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tc_match_eligible(const Problem& p) {
    if (p.dtype != 1 || !p.vec || p.r > 2 || p.C < kTcKC) return false;
    const long long tiles = (long long)((p.F + kTcFR - 1) / kTcFR) * p.H * ((p.W + kTcWB - 1) / kTcWB);
    return tiles * 8 < (1LL << 31);
}

// CTAs per tile: enough that a clip gives every SM two CTAs, at most 8 and at least 4 stages each
int tc_match_pieces(const Problem& p) {
    const long long tiles = (long long)((p.F + kTcFR - 1) / kTcFR) * p.H * ((p.W + kTcWB - 1) / kTcWB);
    const int nst = (p.C + kTcKC - 1) / kTcKC;
    long long want = (2LL * sm_count() + tiles - 1) / tiles;
    if (want > 8) want = 8;
    if (want > nst / 4) want = nst / 4;
    return want < 1 ? 1 : (int)want;
}

size_t tc_match_part_floats(const Problem& p) {
    const long long tiles = (long long)((p.F + kTcFR - 1) / kTcFR) * p.H * ((p.W + kTcWB - 1) / kTcWB);
    const int pieces = tc_match_pieces(p);
    const int win = (2 * p.r + 1) * (2 * p.r + 1);
    return pieces > 1 ? (size_t)tiles * pieces * win * kTcM : 0;
}

size_t tc_match_tiles(const Problem& p) {
    return (size_t)((p.F + kTcFR - 1) / kTcFR) * p.H * ((p.W + kTcWB - 1) / kTcWB);
}

template <int R>
static cudaError_t launch_tc_t(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                               unsigned char* keep, cudaStream_t st) {
    using S = TcShape<R>;
    CUtensorMap mapA, mapB;
    if (!make_map(&mapA, p.X, p.F, p.H, p.W, p.C, kTcWB, 1, kTcFR) ||
        !make_map(&mapB, p.X, p.F, p.H, p.W, p.C, S::BW, S::SIDE, 1))
        return cudaErrorInvalidValue;
    const size_t smem = (size_t)S::STAGES * S::STAGE + 1024;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(k_match_tc<R>), smem);
    if (e != cudaSuccess) return e;
    const int pieces = tc_match_pieces(p);
    const long long tiles = (long long)tc_match_tiles(p);
    return launch_ex(true, smem, k_match_tc<R>, dim3((unsigned)(tiles * pieces)), dim3(kTcThreads), st, mapA, mapB,
                     p.F, p.H, p.W, p.C, p.t, make_anchor_src(p, s, out_anchor), (const float*)s.ssq, p.nslice, pieces,
                     s.tc_part, s.tc_cnt, shat, dst, keep, s.cnt, wait_poll_limit());
}

cudaError_t launch_match_tc(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                            unsigned char* keep, cudaStream_t st) {
    if (p.r == 0) return launch_tc_t<0>(p, s, out_anchor, shat, dst, keep, st);
    if (p.r == 1) return launch_tc_t<1>(p, s, out_anchor, shat, dst, keep, st);
    return launch_tc_t<2>(p, s, out_anchor, shat, dst, keep, st);
}

}  // namespace ttf
