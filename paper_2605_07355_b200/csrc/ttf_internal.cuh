// Shared declarations of the TTF kernels: scratch layout, launch entry points, small device helpers.
// Paper references are to arXiv 2605.07355, Sec. 3.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

namespace ttf {

constexpr float kNormFloor = 1e-12f;   // norms are floored here before dividing (zero token -> similarity 0)
constexpr int kWarpPrefixMaxF = 1024;  // frame counts up to this are scanned by each warp of the gather itself
constexpr int kHdrInts = 128;
constexpr int kStatReplicas = 16;      // copies of the frame statistics, so that the CTAs that read them at the
                                       // same moment do not all queue on the same few cache lines

// header words of the scratch block
enum { HDR_ANCHOR = 0,          // anchor frame a*
       HDR_DONE_ALL = 1,        // arrival counter of the statistics CTAs (zero between calls)
       HDR_ERROR = 2,           // 1: a bounded wait of this call gave up; 2: a checked build caught an index outside its
                                // array (cleared by the first kernel of every call)
       HDR_CHECK_SLACK = 8,     // checked build: every limit is lowered by this much (test hook; zero otherwise)
       HDR_CHECK_SITE = 9,      // checked build: kernel site, index (clamped to 31 bits) and limit of the first index
       HDR_CHECK_INDEX = 10,    // that was out of range
       HDR_CHECK_LIMIT = 11 };

// Problem description handed to every launcher.
struct Problem {
    const void* X;      // [F, N, C]
    int F, H, W, C, r;
    float t;
    int dtype;          // 0 fp32, 1 bf16
    int N;              // H * W
    int vec;            // 1 when rows are 16-byte aligned and a multiple of 16 bytes long, else 0
    int lanes_elems;    // channels one lane loads at once: 16 B worth when vec, else 1
    int ls;             // norm sweep: lanes across a channel slice (32: one warp)
    int nq;             // norm sweep: channel slices per row, ceil(C / (ls * lanes_elems))
    int nslice;         // planes of partial squared norms: one per warp across a slice, nq * ls / 32
    int nsl;            // frame statistics: channel slices (128 channels when C % 4 == 0, else 32)
    int anchor_mode;    // 0 auto (Eq. auto_anchor), 1 first, 2 last, 3 explicit
    int anchor_arg;     // explicit anchor frame
    int emit_anchor;    // 1: X' starts with the N anchor rows (Eq. xprime_stack); 0: streaming segment, sources only
    int pos_t_offset;   // added to the frame coordinate of every emitted position
    int pos_base;       // added to all three coordinates of every emitted position
    int natural_order;  // 1: all retained tokens in ascending flat index (the anchor rows where they fall)
    int use_tc;         // 1: the matching step runs on tcgen05 (ttf_match_tc.cu)
    int chain;          // 1: the kernel before this call's sweep in the stream is the gather of the library's previous
                        // clip, which works on another scratch block: the sweep may run beside it
    int chain_next;     // 1: the kernel after this call's gather is such a sweep
    int overlapped;     // clips whose kernels run beside one another: the lanes of a batch (0 or 1: this call runs alone)
    int stream_once;    // 1: the matching kernel marks the lines of the source rows it reads as the first to leave L2
                        // (the pipelined schedule: the next clip streams into L2 while this one is matched)
};

// Device pointers carved out of one scratch allocation.
struct Scratch {
    int* hdr;           // [kHdrInts]  anchor frame, arrival counter of the anchor-pick slices
    int* cnt;           // [F]   preserved tokens per source frame (Eq. gating summed over a frame)
    int* prefix;        // [F+1] exclusive scan of cnt, only used when F > kWarpPrefixMaxF
    float* S;           // [F, C] per-frame channel sums
    float* Dp;          // [kStatReplicas][nsl, F] per-slice share of <S_k, g>
    float* Qp;          // [kStatReplicas][nsl, F] per-slice share of |S_k|^2
    float* Gp;          // [kStatReplicas][nsl]    per-slice share of |g|^2
    float* ssq;         // [nslice, F*N] partial squared norms (one plane per warp and column block)
    float* shat;        // [F*N] best similarity (Eq. argmax)
    int* dst;           // [F*N] best anchor cell (Eq. dst)
    unsigned char* keep;// [F*N] retention mask (Eq. mask)
    int* fuse_cnt;      // [N]   tokens fused into each anchor cell
    size_t bytes;       // total, multiple of 256
};

// Where a kernel gets the anchor frame a* from.
struct AnchorSrc {
    const float* Dp;    // [kStatReplicas][nsl, F] slice shares of <S_k, g>
    const float* Qp;    // [kStatReplicas][nsl, F] slice shares of |S_k|^2
    const float* Gp;    // [kStatReplicas][nsl]    slice shares of |g|^2
    int nsl;
    int fixed;          // >= 0: the anchor is this frame (first / last / explicit rule)
    int from_hdr;       // 1: an earlier kernel left it in hdr[HDR_ANCHOR]
    int* hdr;
    int* out_anchor;    // optional user copy
};

inline AnchorSrc make_anchor_src(const Problem& p, const Scratch& s, int* out_anchor);

// bf16 clips with 16-byte aligned rows and r <= 2 take the tensor-core matching kernel, which also derives the
// token norms itself; everything else takes the CUDA-core kernel, which reads the norms of the sweep.
inline bool uses_mma_match(const Problem& p) {
    return p.dtype == 1 && p.vec && p.r <= 2 && (long long)p.N * ((p.F + 15) / 16) < (1LL << 31);
}

// The sweep stores per-token partial squared norms only for the kernels that read them.
inline bool needs_sweep_norms(const Problem& p) { return !p.use_tc && (!uses_mma_match(p) || p.r == 2); }

// tcgen05 matching (ttf_match_tc.cu)
bool tc_match_eligible(const Problem& p);
int tc_match_pieces(const Problem& p);
size_t tc_match_tiles(const Problem& p);
cudaError_t launch_match_tc(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                            unsigned char* keep, cudaStream_t st);

// Fills the offsets (base may be NULL to only compute `bytes`).
void carve_scratch(const Problem& p, void* base, Scratch* s);

// Kernel launchers (each enqueues on `st` and returns the launch error, if any).
cudaError_t launch_norm_sum(const Problem& p, const Scratch& s, cudaStream_t st);
cudaError_t launch_frame_stats(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st);
cudaError_t launch_match(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                         unsigned char* keep, cudaStream_t st);
cudaError_t launch_fuse_count(const Problem& p, const Scratch& s, const int* dst, const unsigned char* keep,
                              int* fuse_cnt, cudaStream_t st);
cudaError_t launch_compact(const Problem& p, const Scratch& s, void* out_tokens, int* out_pos, int* out_count,
                           cudaStream_t st);

cudaError_t launch_restore(const void* comp, size_t row_bytes, int F, int N, const int* anchor,
                           const unsigned char* keep, const int* dst, void* out_full, int* row_index,
                           cudaStream_t st);
cudaError_t launch_sim_histogram(const float* sim, const int* anchor, int F, int N, int bins, unsigned int* hist,
                                 cudaStream_t st);
cudaError_t launch_read_floor(const void* buf, size_t bytes, unsigned* sink, cudaStream_t st);
cudaError_t launch_stats(const float* sim, const unsigned char* keep, const int* anchor, int F, int N, float t, float band,
                         long long* out, cudaStream_t st);

// Optional mean fusion (ttf_fuse.cu; not the paper's method): overwrites the anchor block of out_tokens.
cudaError_t launch_fuse_mean(const Problem& p, const Scratch& s, void* out_tokens, cudaStream_t st);

int sm_count();   // SMs of the current device (cached per device)

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to a function in the context of ONE device: set it the first
// time `func` is launched on the current device (and again if a larger size is asked for).
cudaError_t ensure_dynamic_smem(const void* func, size_t bytes);

// Bounded waits: polls of an mbarrier before a waiter gives up, and extra bytes announced to it (always 0 outside
// the test that makes a wait run out; see ttf_debug_set_wait).
int wait_poll_limit();
int wait_tx_extra();

inline AnchorSrc make_anchor_src(const Problem& p, const Scratch& s, int* out_anchor) {
    AnchorSrc a;
    a.Dp = s.Dp; a.Qp = s.Qp; a.Gp = s.Gp; a.nsl = p.nsl; a.hdr = s.hdr; a.out_anchor = out_anchor;
    a.fixed = p.anchor_mode == 0 ? -1 : (p.anchor_mode == 1 ? 0 : (p.anchor_mode == 2 ? p.F - 1 : p.anchor_arg));
    a.from_hdr = p.anchor_mode == 0 ? 1 : 0;     // the statistics kernel's last CTA left the arg max there
    return a;
}

// Launch with programmatic dependent launch: the kernel may be scheduled while the previous kernel of the
// stream drains; it must execute pdl_wait() before it touches anything an earlier kernel wrote, and every
// kernel launched this way executes pdl_wait() on all paths so that completion stays transitive.
// Because such a kernel is already alive while its predecessor still writes, whatever the predecessor
// produces is NOT read-only data for it: it must be read with L2-coherent loads (__ldcg), never through the
// non-coherent / L1 path that `const __restrict__` pointers and __ldg select.  Only X is truly read-only.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_ex(bool pdl, size_t smem, void (*kernel)(KArgs...), dim3 grid, dim3 block,
                             cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    int n = 0;
    if (pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr; cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_if(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st,
                                 Args... args) {
    return launch_ex(pdl, 0, kernel, grid, block, st, args...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
    return launch_pdl_if(true, kernel, grid, block, st, args...);
}

// ---------------------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------------------
#ifdef __CUDACC__

// griddepcontrol: wait = all kernels this one depends on have completed and their writes are visible (a no-op
// for a normally launched kernel); launch_dependents = the next kernel of the stream may be scheduled.
// L2 cache policy for data that is read once more and then dead: its lines are evicted before any others
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Development aid (compiled out unless the library is built with -DTTF_TRACE): earliest / latest time at which
// any CTA passed a mark, in nanoseconds of the global timer, kept in header words 16..111 of the scratch block
// (mark id < 24; two 64-bit words each: ~earliest, latest).  trace_mark is called by thread 0 of a CTA,
// trace_mark_any by whichever single thread reaches the point.
#ifdef TTF_TRACE
__device__ __forceinline__ void trace_mark_any(int* hdr, int id, bool end) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    unsigned long long* s = reinterpret_cast<unsigned long long*>(hdr + 16) + id * 2 + (end ? 1 : 0);
    atomicMax(s, end ? t : ~t);
}
__device__ __forceinline__ void trace_mark(int* hdr, int id, bool end) {
    if (threadIdx.x == 0) trace_mark_any(hdr, id, end);
}
// mean of a duration over the threads that report it: word 0 of the mark = sum of nanoseconds, word 1 = reports
__device__ __forceinline__ unsigned long long trace_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void trace_acc(int* hdr, int id, unsigned long long ns) {
    unsigned long long* s = reinterpret_cast<unsigned long long*>(hdr + 16) + id * 2;
    atomicAdd(s, ns);
    atomicAdd(s + 1, 1ull);
}
#else
__device__ __forceinline__ void trace_mark_any(int*, int, bool) {}
__device__ __forceinline__ void trace_mark(int*, int, bool) {}
__device__ __forceinline__ unsigned long long trace_now() { return 0; }
__device__ __forceinline__ void trace_acc(int*, int, unsigned long long) {}
#endif

// Checked build (-DTTF_DEBUG): every global store whose index a kernel computes is guarded by in_bounds().  An
// index outside [0, limit) raises the status word of the call's scratch to 2, leaves (site, index, limit) of the first
// offender in the header, and the caller skips the access: nothing traps, the context stays usable, and the host
// reads TTF_ERR_BOUNDS.  In the normal build the test is the constant true and disappears.
// Sites: 1 sweep, 2 warp-level / CUDA-core matching, 3 tcgen05 matching, 4 gather rows, 5 gather positions.
#ifdef TTF_DEBUG
__device__ __forceinline__ bool in_bounds(int* hdr, int site, long long idx, long long limit) {
    limit -= __ldcg(hdr + HDR_CHECK_SLACK);
    if (idx >= 0 && idx < limit) return true;
    if (atomicCAS(hdr + HDR_ERROR, 0, 2) == 0) {
        hdr[HDR_CHECK_SITE] = site;
        hdr[HDR_CHECK_INDEX] = (int)(idx < 0 ? -1 : (idx > 0x7fffffffLL ? 0x7fffffffLL : idx));
        hdr[HDR_CHECK_LIMIT] = (int)(limit > 0x7fffffffLL ? 0x7fffffffLL : limit);
    }
    return false;
}
#else
__device__ __forceinline__ bool in_bounds(int*, int, long long, long long) { return true; }
#endif

struct bf16_t { uint16_t bits; };   // storage type only: all arithmetic is on the widened fp32 value

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Loads V consecutive channels starting at p (p is 16-byte aligned when V > 1) and widens them to fp32.
template <typename T, int V> struct Loader;
// load_raw fetches the bits (so that several loads can be in flight before any is unpacked), unpack widens.
template <> struct Loader<float, 4> {
    using Raw = float4;
    static __device__ __forceinline__ Raw load_raw(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ Raw load_raw_cg(const float* p) { return __ldcg(reinterpret_cast<const float4*>(p)); }
    static __device__ __forceinline__ Raw zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&x)[4]) { x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
    static __device__ __forceinline__ void load(const float* p, float (&x)[4]) { unpack(load_raw(p), x); }
};
template <> struct Loader<float, 1> {
    using Raw = float;
    static __device__ __forceinline__ Raw load_raw(const float* p) { return __ldg(p); }
    static __device__ __forceinline__ Raw load_raw_cg(const float* p) { return __ldcg(p); }
    static __device__ __forceinline__ Raw zero() { return 0.f; }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&x)[1]) { x[0] = v; }
    static __device__ __forceinline__ void load(const float* p, float (&x)[1]) { x[0] = __ldg(p); }
};
template <> struct Loader<bf16_t, 8> {
    using Raw = uint4;
    static __device__ __forceinline__ Raw load_raw(const bf16_t* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
    static __device__ __forceinline__ Raw load_raw_cg(const bf16_t* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }
    static __device__ __forceinline__ Raw zero() { return make_uint4(0, 0, 0, 0); }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&x)[8]) {
        x[0] = bf16_lo(v.x); x[1] = bf16_hi(v.x); x[2] = bf16_lo(v.y); x[3] = bf16_hi(v.y);
        x[4] = bf16_lo(v.z); x[5] = bf16_hi(v.z); x[6] = bf16_lo(v.w); x[7] = bf16_hi(v.w);
    }
    static __device__ __forceinline__ void load(const bf16_t* p, float (&x)[8]) { unpack(load_raw(p), x); }
};
template <> struct Loader<bf16_t, 1> {
    using Raw = float;
    static __device__ __forceinline__ Raw load_raw(const bf16_t* p) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    static __device__ __forceinline__ Raw load_raw_cg(const bf16_t* p) {
        return __uint_as_float(static_cast<uint32_t>(__ldcg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    static __device__ __forceinline__ Raw zero() { return 0.f; }
    static __device__ __forceinline__ void unpack(const Raw& v, float (&x)[1]) { x[0] = v; }
    static __device__ __forceinline__ void load(const bf16_t* p, float (&x)[1]) { x[0] = load_raw(p); }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Anchor Frame Selection, last step (Eq. auto_anchor): a* = arg max_k <S_k, g> / (|S_k| |g|), lowest frame on
// ties, from the per-slice shares written by k_frame_stats; the shares are added in slice order.  Called by
// all threads of a CTA (any block size that is a multiple of 32, at most 1024); returns the same value to all.
__device__ __forceinline__ int resolve_anchor(const AnchorSrc& src, int F) {
    if (src.fixed >= 0) return src.fixed;
    if (src.from_hdr) return __ldcg(src.hdr + HDR_ANCHOR);
    __shared__ float s_d[32][33], s_q[32][33];        // [warp][frame of the chunk]
    __shared__ int s_anchor;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5, nw = blockDim.x >> 5;
    const int rep = blockIdx.x % kStatReplicas;       // identical copies: which one is read does not matter
    const float* Dp = src.Dp + (size_t)rep * src.nsl * F;
    const float* Qp = src.Qp + (size_t)rep * src.nsl * F;
    const float* Gp = src.Gp + (size_t)rep * src.nsl;
    float ginv = 0.f;
    if (w == 0) {
        float gg = 0.f;
        for (int q = lane; q < src.nsl; q += 32) gg += __ldcg(Gp + q);
        gg = warp_sum(gg);
        ginv = 1.0f / fmaxf(sqrtf(gg), kNormFloor);
    }
    float best = -INFINITY;
    int idx = 0x7fffffff;
    for (int kb = 0; kb < F; kb += 32) {              // lane = frame: loads are coalesced over the frames
        const int kk = kb + lane;
        float d = 0.f, s2 = 0.f;
        if (kk < F) {
#pragma unroll 4
            for (int q = w; q < src.nsl; q += nw) {   // warp w adds the slices w, w + nw, ...
                d += __ldcg(Dp + (size_t)q * F + kk);
                s2 += __ldcg(Qp + (size_t)q * F + kk);
            }
        }
        s_d[w][lane] = d; s_q[w][lane] = s2;
        __syncthreads();
        if (w == 0 && kk < F) {                       // warps combined in warp order
            float dd = 0.f, qq = 0.f;
            for (int ww = 0; ww < nw; ++ww) { dd += s_d[ww][lane]; qq += s_q[ww][lane]; }
            const float v = dd * ginv * (1.0f / fmaxf(sqrtf(qq), kNormFloor));
            if (v > best || idx == 0x7fffffff) { best = v; idx = kk; }   // ascending kk per lane: first max stays
        }
        __syncthreads();
    }
    if (w == 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (oi != 0x7fffffff && (idx == 0x7fffffff || ob > best || (ob == best && oi < idx))) { best = ob; idx = oi; }
        }
        if (lane == 0) s_anchor = idx;
    }
    __syncthreads();
    return s_anchor;
}

// 1 / max(||x||, floor) from the per-slice partial squared norms of token f, summed in slice order
__device__ __forceinline__ float inv_norm(const float* __restrict__ ssq, int nslice, size_t FN, size_t f) {
    float s = 0.f;
    for (int q = 0; q < nslice; ++q) s += __ldcg(ssq + (size_t)q * FN + f);
    return 1.0f / fmaxf(sqrtf(s), kNormFloor);
}

#endif  // __CUDACC__

}  // namespace ttf
