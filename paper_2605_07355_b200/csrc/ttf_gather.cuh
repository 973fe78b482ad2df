// Rank/select helpers of the output-driven gather and the fuse-count bookkeeping, shared by the stand-alone
// compaction kernels.
#pragma once

#include "ttf_internal.cuh"

namespace ttf {

constexpr int kCopyWarps = 8;
constexpr int kScanChunks = 4;       // frame counts per lane fetched at once by the warp-level frame search

// Tokens fused into each anchor cell j: |{(k,i): k != a, keep = 0, dst = j}|, gather-side (every cell looks at
// the (2r+1)^2 x (F-1) tokens that can point to it), integer, order-free.  Run by whole CTAs: block `b` of `nb`,
// one warp per cell (any number of warps per CTA).  The lanes split the (frame, window cell) pairs of the cell and fetch both flags of four
// pairs at a time without testing one before loading the other, so the loads of a lane overlap instead of
// forming a chain of dependent round trips.
__device__ __forceinline__ void fuse_count_cta(int F, int H, int W, int r, int a, const unsigned char* keep,
                                               const int* dst, int* fuse_cnt, int b, int nb) {
    if (fuse_cnt == nullptr) return;
    const int N = H * W;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, warps = blockDim.x >> 5;
    for (int j = b * warps + w; j < N; j += nb * warps) {
        const int y = j / W, x = j - y * W;
        const int y_lo = max(0, y - r), x_lo = max(0, x - r);
        const int nx = min(W - 1, x + r) - x_lo + 1, wsz = (min(H - 1, y + r) - y_lo + 1) * nx;
        const long long pairs = (long long)F * wsz;
        int c = 0;
        for (long long q0 = lane; q0 < pairs; q0 += 4 * 32) {
            unsigned char kp[4];
            int ds[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long q = q0 + u * 32;
                const int k = (int)(q / wsz), e = (int)(q - (long long)k * wsz);
                const bool in = q < pairs && k != a;
                const size_t f = (size_t)k * N + (y_lo + e / nx) * W + x_lo + e % nx;
                kp[u] = in ? __ldcg(keep + f) : (unsigned char)1;
                ds[u] = in ? __ldcg(dst + f) : -1;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) c += (!kp[u] && ds[u] == j) ? 1 : 0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0) fuse_cnt[j] = c;
    }
}

// Frame search of the gather: the frame that holds the e-th token of the flat walk and the number of walked tokens
// before that frame.  The walk visits the preserved tokens of the source frames in flat order; the anchor frame
// contributes `acnt` tokens: 0 when its rows are emitted as a block of their own (Eq. xprime_stack), N in natural
// order (all of its tokens are retained, Eq. mask).  Returns the total; k_out = -1 when e is past the end (e < 0
// asks for the total only).  All lanes of a warp call it with the same arguments.
__device__ __forceinline__ int find_frame(const int* __restrict__ cnt, const int* __restrict__ gprefix, int F, int a,
                                          int acnt, int lane, int e, int& k_out, int& before) {
    int running = 0;
    k_out = -1; before = 0;
    if (F > kWarpPrefixMaxF) {                         // pre-scanned prefix: binary search
        int lo = 0, hi = F;
        const int P = __ldcg(gprefix + F);
        if (e < P) {
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (__ldcg(gprefix + mid) <= e) lo = mid; else hi = mid; }
            k_out = lo; before = __ldcg(gprefix + lo);
        }
        return P;
    }
    for (int base = 0; base < F; base += 32 * kScanChunks) {
        int c[kScanChunks];
#pragma unroll
        for (int q = 0; q < kScanChunks; ++q) {
            const int k = base + q * 32 + lane;
            c[q] = k < F ? (k == a ? acnt : __ldcg(cnt + k)) : 0;
        }
#pragma unroll
        for (int q = 0; q < kScanChunks; ++q) {
            int incl = c[q];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const int total = __shfl_sync(0xffffffffu, incl, 31);
            if (k_out < 0 && e < running + total) {
                const unsigned m = __ballot_sync(0xffffffffu, running + incl > e);
                const int l = __ffs(m) - 1;
                k_out = base + q * 32 + l;
                before = running + __shfl_sync(0xffffffffu, incl - c[q], l);
            }
            running += total;
        }
        if (k_out >= 0 && e >= 0) break;               // e < 0 asks for the total only
    }
    return running;
}


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

}  // namespace ttf
