// Token Compression and Positional Alignment (Eqs. xprime_stack, mask, compress_pos, Lpre), plus the
// bookkeeping of identity replacement (how many source tokens each anchor cell absorbed).
//
// The output position of a preserved source token is N plus the number of preserved source tokens before it
// in flat (k, i) order.  That exclusive prefix is taken in two levels: the per-frame survivor counts written
// by the matching kernel are scanned by every CTA (shared memory, or a pre-scanned array for very long
// clips), and inside a frame the rank is a population count over the frame's keep flags.  The gather is then
// driven from the OUTPUT side: every CTA owns an equal, contiguous range of output rows, finds their source
// rows by rank/select and copies them, so the bytes per CTA are the same no matter how unevenly the
// survivors are spread over the frames.  No CTA ever waits for another one.
#include "ttf_internal.cuh"

namespace ttf {

constexpr int kCopyWarps = 8;

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

constexpr int kRowsPerPass = 32;     // output rows whose sources a CTA resolves before copying them
constexpr int kCopyUnroll = 8;       // copy units in flight per thread

// Cell index of the n-th (0-based) retained token of one frame: a warp-wide rank/select over the keep flags.
// All lanes must call with the same arguments; returns -1 if the frame holds fewer than n+1 retained tokens.
__device__ __forceinline__ int select_in_frame(const unsigned char* __restrict__ kf, int N, int n, int lane) {
    for (int b = 0; b < N; b += 256) {                     // 8 cells per lane, 256 per step
        const int c0 = b + lane * 8;
        unsigned bits = 0;
        if (c0 + 8 <= N && ((reinterpret_cast<uintptr_t>(kf + c0) & 7) == 0)) {
            const uint2 v = __ldcg(reinterpret_cast<const uint2*>(kf + c0));
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                bits |= ((v.x >> (8 * e)) & 0xffu) ? (1u << e) : 0u;
                bits |= ((v.y >> (8 * e)) & 0xffu) ? (1u << (4 + e)) : 0u;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) bits |= (c0 + e < N && __ldcg(kf + c0 + e) != 0) ? (1u << e) : 0u;
        }
        const int mine = __popc(bits);
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (n < total) {
            const int excl = incl - mine;
            const bool here = n >= excl && n < incl;       // exactly one lane
            const int cell = here ? c0 + (int)__fns(bits, 0, n - excl + 1) : 0;
            const unsigned who = __ballot_sync(0xffffffffu, here);
            return __shfl_sync(0xffffffffu, cell, __ffs(who) - 1);
        }
        n -= total;
    }
    return -1;
}

template <int COPY_BYTES>
__global__ void __launch_bounds__(kCopyWarps * 32)
k_compact(const unsigned char* __restrict__ X, size_t row_bytes, int F, int H, int W, int r,
          const int* __restrict__ hdr, const int* __restrict__ cnt, const int* __restrict__ gprefix,
          const unsigned char* __restrict__ keep, const int* __restrict__ dst,
          unsigned char* __restrict__ out_tokens, int* __restrict__ out_pos, int* __restrict__ out_count,
          int* __restrict__ fuse_cnt, int ncopy_blocks)
{
    using U = typename CopyUnit<COPY_BYTES>::type;
    const int N = H * W;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    pdl_wait();                                  // keep flags, dst and survivor counts are complete
    const int a = __ldcg(hdr + HDR_ANCHOR);

    // ---- bookkeeping CTAs: tokens fused into each anchor cell (gather-side, integer, fixed order) --------
    if ((int)blockIdx.x >= ncopy_blocks) {
        if (fuse_cnt == nullptr) return;
        const int nb = gridDim.x - ncopy_blocks;
        for (int j = ((int)blockIdx.x - ncopy_blocks) * kCopyWarps + w; j < N; j += nb * kCopyWarps) {
            const int y = j / W, x = j - y * W;
            int c = 0;
            for (int k = lane; k < F; k += 32) {
                if (k == a) continue;
                for (int yy = max(0, y - r); yy <= min(H - 1, y + r); ++yy)
                    for (int xx = max(0, x - r); xx <= min(W - 1, x + r); ++xx) {
                        const size_t f = (size_t)k * N + yy * W + xx;
                        c += (!__ldcg(keep + f) && __ldcg(dst + f) == j) ? 1 : 0;
                    }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            if (lane == 0) fuse_cnt[j] = c;
        }
        return;
    }

    // ---- exclusive prefix of preserved tokens per frame ------------------------------------------------
    __shared__ int s_pre[kSmemPrefixMaxF + 1];
    __shared__ int s_warp[kCopyWarps];
    __shared__ int s_src[kRowsPerPass];
    const int* pre;
    if (F <= kSmemPrefixMaxF) {
        // each thread scans a contiguous run of frames, runs are combined over the block in thread order
        const int per = (F + kCopyWarps * 32 - 1) / (kCopyWarps * 32);
        const int k0 = tid * per;
        int sum = 0;
        for (int k = k0; k < min(F, k0 + per); ++k) sum += (k != a) ? __ldcg(cnt + k) : 0;
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        if (lane == 31) s_warp[w] = incl;
        __syncthreads();
        int woff = 0;
        for (int ww = 0; ww < w; ++ww) woff += s_warp[ww];
        int run = woff + incl - sum;
        for (int k = k0; k < min(F, k0 + per); ++k) { s_pre[k] = run; run += (k != a) ? __ldcg(cnt + k) : 0; }
        if (tid == kCopyWarps * 32 - 1) s_pre[F] = woff + incl;
        __syncthreads();
        pre = s_pre;
    } else {
        pre = gprefix;
    }
    const int P = pre[F];
    const int L = N + P;                                   // L' = N + P (Eq. Lpre)
    if (blockIdx.x == 0 && tid == 0) { *out_count = L; }

    // ---- output-driven gather: this CTA owns a contiguous, balanced range of output rows ------------------
    const int j_begin = (int)((long long)L * blockIdx.x / ncopy_blocks);
    const int j_end = (int)((long long)L * (blockIdx.x + 1) / ncopy_blocks);
    const int upr = (int)(row_bytes / COPY_BYTES);         // copy units per row
    for (int jb = j_begin; jb < j_end; jb += kRowsPerPass) {
        const int rows = min(kRowsPerPass, j_end - jb);
        __syncthreads();                                   // previous pass has finished with s_src
        // a) source token of every output row of the pass: one warp per row
        for (int rr = w; rr < rows; rr += kCopyWarps) {
            const int j = jb + rr;
            int f;
            if (j < N) f = a * N + j;                      // anchor rows first (Eq. xprime_stack)
            else {
                const int e = j - N;
                int lo = 0, hi = F;                        // largest k with pre[k] <= e
                while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (pre[mid] <= e) lo = mid; else hi = mid; }
                const int i = select_in_frame(keep + (size_t)lo * N, N, e - pre[lo], lane);
                f = i < 0 ? -1 : lo * N + i;               // -1 cannot happen when cnt matches keep
            }
            if (lane == 0) s_src[rr] = f;
            if (lane < 3 && f >= 0) {                      // p_{k,i} = (k, y_i, x_i)  (Eq. compress_pos)
                const int k = f / N, i = f - k * N, yy = i / W;
                out_pos[(size_t)j * 3 + lane] = lane == 0 ? k : (lane == 1 ? yy : i - yy * W);
            }
        }
        __syncthreads();
        // b) copy: consecutive threads move consecutive 16-byte units, several rows in flight per thread
        const long long total = (long long)rows * upr;
        for (long long base = tid; base < total; base += (long long)kCopyWarps * 32 * kCopyUnroll) {
            U v[kCopyUnroll];
            long long o[kCopyUnroll];
#pragma unroll
            for (int q = 0; q < kCopyUnroll; ++q) {
                const long long u = base + (long long)q * kCopyWarps * 32;
                o[q] = -1;
                if (u < total) {
                    const int rr = (int)(u / upr);
                    const int off = (int)(u - (long long)rr * upr);
                    const int f = s_src[rr];
                    if (f >= 0) {
                        v[q] = __ldcs(reinterpret_cast<const U*>(X + (size_t)f * row_bytes) + off);
                        o[q] = (long long)(jb + rr) * upr + off;
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < kCopyUnroll; ++q)
                if (o[q] >= 0) __stcs(reinterpret_cast<U*>(out_tokens) + o[q], v[q]);
        }
    }
}

cudaError_t launch_fuse_count(const Problem& p, const Scratch& s, const int* dst, const unsigned char* keep,
                              int* fuse_cnt, cudaStream_t st) {
    // bookkeeping only: the same kernel with zero copy CTAs
    const int nb = (p.N + kCopyWarps - 1) / kCopyWarps;
    k_compact<4><<<nb < 1024 ? nb : 1024, kCopyWarps * 32, 0, st>>>(
        nullptr, 0, p.F, p.H, p.W, p.r, s.hdr, s.cnt, s.prefix, keep, dst, nullptr, nullptr, nullptr,
        fuse_cnt, 0);
    return cudaGetLastError();
}

cudaError_t launch_compact(const Problem& p, const Scratch& s, void* out_tokens, int* out_pos, int* out_count,
                           cudaStream_t st) {
    const size_t esize = p.dtype == 0 ? 4 : 2;
    const size_t row_bytes = (size_t)p.C * esize;
    const bool vec = p.vec && (reinterpret_cast<uintptr_t>(out_tokens) % 16 == 0);
    if (p.F > kSmemPrefixMaxF) {
        k_frame_prefix<<<1, 1024, 0, st>>>(s.cnt, s.hdr, p.F, s.prefix);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int ncopy = 2 * sm_count();
    int nfuse = (p.N + kCopyWarps - 1) / kCopyWarps;
    if (nfuse > sm_count()) nfuse = sm_count();
    const int grid = ncopy + nfuse;
    const unsigned char* X = reinterpret_cast<const unsigned char*>(p.X);
    unsigned char* out = reinterpret_cast<unsigned char*>(out_tokens);
    const dim3 g(grid), b(kCopyWarps * 32);
    // the pre-scanned prefix of very long clips is read through plain loads: order that case by the stream
    const bool pdl = p.F <= kSmemPrefixMaxF;
    if (vec)
        return launch_pdl_if(pdl, k_compact<16>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                          (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                          out, out_pos, out_count, s.fuse_cnt, ncopy);
    if (esize == 4)
        return launch_pdl_if(pdl, k_compact<4>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                          (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                          out, out_pos, out_count, s.fuse_cnt, ncopy);
    return launch_pdl_if(pdl, k_compact<2>, g, b, st, X, row_bytes, p.F, p.H, p.W, p.r, (const int*)s.hdr,
                      (const int*)s.cnt, (const int*)s.prefix, (const unsigned char*)s.keep, (const int*)s.dst,
                      out, out_pos, out_count, s.fuse_cnt, ncopy);
}

}  // namespace ttf
