// Shared declarations of the TTF kernels: scratch layout, launch entry points, small device helpers.
// Paper references are to arXiv 2605.07355, Sec. 3.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

namespace ttf {

constexpr float kNormFloor = 1e-12f;   // norms are floored here before dividing (zero token -> similarity 0)
constexpr int kWarpPrefixMaxF = 1024;  // frame counts up to this are scanned by each warp of the gather itself
constexpr int kHdrInts = 64;

// header words of the scratch block
enum { HDR_ANCHOR = 0, HDR_DONE_ALL = 1 };

// Problem description handed to every launcher.
struct Problem {
    const void* X;      // [F, N, C]
    int F, H, W, C, r;
    float t;
    int dtype;          // 0 fp32, 1 bf16
    int N;              // H * W
    int vec;            // 1 when rows are 16-byte aligned and a multiple of 16 bytes long, else 0
    int lanes_elems;    // channels one lane loads at once: 16 B worth when vec, else 1
    int cpt;            // norm sweep: chunks of lanes_elems channels per thread per row (1 or 2)
    int ncb;            // norm sweep: column blocks of 256 * cpt chunks per row
    int nslice;         // planes of partial squared norms: 8 warps x ncb
    int nsl;            // anchor pick: channel slices (32 channels when C % 4 == 0, else 8)
    int anchor_mode;    // 0 auto (Eq. auto_anchor), 1 first, 2 last, 3 explicit
    int anchor_arg;     // explicit anchor frame
};

// Device pointers carved out of one scratch allocation.
struct Scratch {
    int* hdr;           // [kHdrInts]  anchor frame, arrival counter of the anchor-pick slices
    int* cnt;           // [F]   preserved tokens per source frame (Eq. gating summed over a frame)
    int* prefix;        // [F+1] exclusive scan of cnt, only used when F > kWarpPrefixMaxF
    float* fcos;        // [F]   cosine of each frame mean to the global mean (Eq. auto_anchor)
    float* Sp;          // [TG, F, C] per-frame channel sums of each token group
    float* Dp;          // [nsl, F] per-slice share of <S_k, g>
    float* Qp;          // [nsl, F] per-slice share of |S_k|^2
    float* Gp;          // [nsl]    per-slice share of |g|^2
    float* ssq;         // [nslice, F*N] partial squared norms (one plane per warp and column block)
    float* shat;        // [F*N] best similarity (Eq. argmax)
    int* dst;           // [F*N] best anchor cell (Eq. dst)
    unsigned char* keep;// [F*N] retention mask (Eq. mask)
    int* fuse_cnt;      // [N]   tokens fused into each anchor cell
    size_t bytes;       // total, multiple of 256
};

// Fills the offsets (base may be NULL to only compute `bytes`).
void carve_scratch(const Problem& p, void* base, Scratch* s);

// Kernel launchers (each enqueues on `st` and returns the launch error, if any).
int norm_token_groups(const Problem& p);   // token groups per frame of the norm/anchor sweep (shape-only rule)
cudaError_t launch_norm_anchor(const Problem& p, const Scratch& s, int* out_anchor, cudaStream_t st);
cudaError_t launch_match(const Problem& p, const Scratch& s, float* shat, int* dst, unsigned char* keep,
                         cudaStream_t st);
cudaError_t launch_fuse_count(const Problem& p, const Scratch& s, const int* dst, const unsigned char* keep,
                              int* fuse_cnt, cudaStream_t st);
cudaError_t launch_compact(const Problem& p, const Scratch& s, void* out_tokens, int* out_pos, int* out_count,
                           cudaStream_t st);

int sm_count();   // SMs of the current device (cached per device)

// Launch with programmatic dependent launch: the kernel may be scheduled while the previous kernel of the
// stream drains; it must execute pdl_wait() before it touches anything an earlier kernel wrote, and every
// kernel launched this way executes pdl_wait() on all paths so that completion stays transitive.
// Because such a kernel is already alive while its predecessor still writes, whatever the predecessor
// produces is NOT read-only data for it: it must be read with L2-coherent loads (__ldcg), never through the
// non-coherent / L1 path that `const __restrict__` pointers and __ldg select.  Only X is truly read-only.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_if(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st,
                                 Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
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
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Development aid (compiled out unless TTF_TRACE is defined): earliest start / latest end of every kernel of
// a call in nanoseconds of the global timer, kept in header words 16..47 of the scratch block.
#ifdef TTF_TRACE
__device__ __forceinline__ void trace_mark(int* hdr, int id, bool end) {
    if (threadIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        unsigned long long* s = reinterpret_cast<unsigned long long*>(hdr + 16) + id * 2 + (end ? 1 : 0);
        atomicMax(s, end ? t : ~t);
    }
}
#else
__device__ __forceinline__ void trace_mark(int*, int, bool) {}
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

// 1 / max(||x||, floor) from the per-slice partial squared norms of token f, summed in slice order
__device__ __forceinline__ float inv_norm(const float* __restrict__ ssq, int nslice, size_t FN, size_t f) {
    float s = 0.f;
    for (int q = 0; q < nslice; ++q) s += __ldcg(ssq + (size_t)q * FN + f);
    return 1.0f / fmaxf(sqrtf(s), kNormFloor);
}

#endif  // __CUDACC__

}  // namespace ttf
