/*
 * CPU oracle for Temporal Token Fusion (TTF, arXiv 2605.07355), Sec. 3.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the method computes; it is what
 * the CUDA library is checked against and what the CPU baseline times.  It shares no code, header, table or
 * helper with the CUDA path, and the CUDA path never calls it.  Every function takes the paper's steps in
 * the paper's order and notation, with all floating-point arithmetic in double (inputs are fp32 values;
 * bf16 inputs are widened exactly by the caller).  The only parallelism is an OpenMP loop over frames.
 *
 * Notation (Sec. 3, Problem Setup): X in R^{FN x C}, frames k in [0,F), cells i in [0,N), N = H*W,
 * (y_i, x_i) = (i / W, i mod W); a is the anchor frame; every other frame is a source frame.
 *
 * Readings of points the paper leaves open (each is also pinned or exercised by a test):
 *   - gate at equality: keep = 1[s_hat <= t] (Eq. gating), so a token is fused only when s_hat > t strictly;
 *     the comparison is taken after rounding s_hat to fp32, the precision the CUDA path decides in;
 *     a NaN similarity keeps the token.
 *   - which border duplicate is masked: offsets are visited in lexicographic (dy, dx) order and a candidate
 *     whose clipped index pi was already produced by an earlier offset gets -inf (the first one survives).
 *   - exact ties between distinct candidates, and between frames in the anchor rule: the first maximum in
 *     visiting order wins, i.e. the lowest anchor index / lowest frame.
 *   - zero vectors: norms are floored at 1e-12 before dividing, so a zero token has similarity 0 to all.
 *   - order of X': the N anchor rows first, then preserved source rows by ascending flat index k*N + i.
 *
 * Pins (tests/test_oracle_pins.py): kept + fused = FN; t > 1 keeps everything and t < -1 fuses every source
 * token; identical frames collapse to the anchor; uniform and per-token rescaling; a radius that covers the
 * grid equals an all-pairs search done with scipy's cdist; a planted integer shift gives dst in closed form;
 * a frame equal to the clip mean wins the anchor rule with cosine 1; clip-and-mask equals window-intersect-
 * grid; rho is monotone in t and in r; survivors keep their (k, y, x) in ascending order.
 * Mean fusion (ttf_oracle_fuse_mean, not the paper's method) is pinned by: nothing fused or identical frames give
 * the anchor rows back; the weighted means add up to the sum of all absorbed tokens; numpy's own accumulation.
 * Parity unpinned: nothing computed here; what cannot be pinned is accuracy on real video, which needs the
 * paper's datasets and weights and is not computed by this file at all.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define TTF_ORACLE_NORM_FLOOR 1e-12

int ttf_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* cos(u, v) = u.v / (|u| |v|), Sec. 3 (definition under Eq. auto_anchor), for double vectors */
static double cos_dd(const double* u, const double* v, int C) {
    double uv = 0.0, uu = 0.0, vv = 0.0;
    for (int c = 0; c < C; ++c) { uv += u[c] * v[c]; uu += u[c] * u[c]; vv += v[c] * v[c]; }
    double nu = sqrt(uu), nv = sqrt(vv);
    if (nu < TTF_ORACLE_NORM_FLOOR) nu = TTF_ORACLE_NORM_FLOOR;
    if (nv < TTF_ORACLE_NORM_FLOOR) nv = TTF_ORACLE_NORM_FLOOR;
    return uv / (nu * nv);
}

/* the same for two fp32 token rows */
static double cos_ff(const float* u, const float* v, int C) {
    double uv = 0.0, uu = 0.0, vv = 0.0;
    for (int c = 0; c < C; ++c) {
        double a = (double)u[c], b = (double)v[c];
        uv += a * b; uu += a * a; vv += b * b;
    }
    double nu = sqrt(uu), nv = sqrt(vv);
    if (nu < TTF_ORACLE_NORM_FLOOR) nu = TTF_ORACLE_NORM_FLOOR;
    if (nv < TTF_ORACLE_NORM_FLOOR) nv = TTF_ORACLE_NORM_FLOOR;
    return uv / (nu * nv);
}

/*
 * Anchor Frame Selection, Eq. (auto_anchor):
 *   a* = argmax_k cos( (1/N) sum_i x_{k,i} ,  (1/(FN)) sum_{k',i} x_{k',i} ).
 * cos_out[k] receives the cosine of frame k.  Returns a*.
 */
int ttf_oracle_anchor(const float* X, int F, int N, int C, double* cos_out) {
    double* m = (double*)calloc((size_t)F * C, sizeof(double));   /* m_k = spatial mean of frame k */
    double* g = (double*)calloc((size_t)C, sizeof(double));       /* global mean token            */
    for (int k = 0; k < F; ++k) {
        for (int i = 0; i < N; ++i) {
            const float* x = X + ((size_t)k * N + i) * C;
            for (int c = 0; c < C; ++c) m[(size_t)k * C + c] += (double)x[c];
        }
        for (int c = 0; c < C; ++c) {
            g[c] += m[(size_t)k * C + c];
            m[(size_t)k * C + c] /= (double)N;
        }
    }
    for (int c = 0; c < C; ++c) g[c] /= ((double)F * (double)N);
    int a = 0;
    double best = -INFINITY;
    for (int k = 0; k < F; ++k) {
        double ck = cos_dd(m + (size_t)k * C, g, C);
        if (cos_out) cos_out[k] = ck;
        if (ck > best) { best = ck; a = k; }
    }
    free(m); free(g);
    return a;
}

/* integer projection onto [lo, hi], Eq. (proj) */
static int proj(int z, int lo, int hi) { return z < lo ? lo : (z > hi ? hi : z); }

/* flat anchor-frame index for offset (dy, dx), Eq. (pi) */
static int pi_index(int i, int dy, int dx, int H, int W) {
    int y = i / W, x = i % W;
    return proj(y + dy, 0, H - 1) * W + proj(x + dx, 0, W - 1);
}

/*
 * Pointwise Matching with Local Window Search, Eqs. (pi), (argmax), (dst).
 * For every source frame k != a and cell i: the (2r+1)^2 offsets are visited in lexicographic order; a
 * candidate whose clipped index repeats an earlier one is masked with -inf; s_hat is the largest remaining
 * cosine, dst the anchor index that attains it, second the runner-up (-inf if there is only one candidate).
 * Rows of frame a receive s_hat = 1, dst = i, second = -inf.
 */
void ttf_oracle_match(const float* X, int F, int H, int W, int C, int r, int a,
                      double* s_hat, int* dst, double* second) {
    const int N = H * W;
    const int side = 2 * r + 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int k = 0; k < F; ++k) {
        int* seen = (int*)malloc(sizeof(int) * (size_t)side * side);
        for (int i = 0; i < N; ++i) {
            size_t f = (size_t)k * N + i;
            if (k == a) { s_hat[f] = 1.0; dst[f] = i; if (second) second[f] = -INFINITY; continue; }
            const float* xs = X + f * C;
            double best = -INFINITY, runner = -INFINITY;
            int best_j = -1, nseen = 0;
            for (int dy = -r; dy <= r; ++dy) {
                for (int dx = -r; dx <= r; ++dx) {
                    int j = pi_index(i, dy, dx, H, W);
                    int dup = 0;
                    for (int q = 0; q < nseen; ++q) if (seen[q] == j) { dup = 1; break; }
                    seen[nseen++] = j;
                    double s = dup ? -INFINITY : cos_ff(xs, X + ((size_t)a * N + j) * C, C);
                    if (dup) continue;
                    if (s > best || best_j < 0) { runner = best; best = s; best_j = j; }
                    else if (s > runner) runner = s;
                }
            }
            s_hat[f] = best; dst[f] = best_j; if (second) second[f] = runner;
        }
        free(seen);
    }
}

/*
 * All-pairs search against the anchor frame (the global matching the paper contrasts TTF with, Sec. 1-2):
 * best cosine over all N anchor tokens.  Used only as a cross-check for r >= max(H, W) - 1.
 */
void ttf_oracle_match_global(const float* X, int F, int N, int C, int a, double* s_hat, int* dst) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int k = 0; k < F; ++k) {
        for (int i = 0; i < N; ++i) {
            size_t f = (size_t)k * N + i;
            if (k == a) { s_hat[f] = 1.0; dst[f] = i; continue; }
            double best = -INFINITY; int best_j = -1;
            for (int j = 0; j < N; ++j) {
                double s = cos_ff(X + f * C, X + ((size_t)a * N + j) * C, C);
                if (s > best || best_j < 0) { best = s; best_j = j; }
            }
            s_hat[f] = best; dst[f] = best_j;
        }
    }
}

/*
 * Threshold Gating, Eq. (gating), and the retention mask, Eq. (mask):
 *   m_{k,i} = 1 for k = a, else 1[s_hat_{k,i} <= t]   (evaluated as !(s_hat > t) on fp32-rounded values).
 */
void ttf_oracle_gate(const double* s_hat, int F, int N, int a, float t, uint8_t* keep) {
    for (int k = 0; k < F; ++k)
        for (int i = 0; i < N; ++i) {
            size_t f = (size_t)k * N + i;
            keep[f] = (k == a) ? 1 : (uint8_t)(!((float)s_hat[f] > t));
        }
}

/* fused tokens per anchor cell: |{(k,i): k != a, m_{k,i} = 0, dst(k,i) = j}|  (bookkeeping of Eq. dst) */
void ttf_oracle_fuse_count(const uint8_t* keep, const int* dst, int F, int N, int a, int* fuse_cnt) {
    for (int j = 0; j < N; ++j) fuse_cnt[j] = 0;
    for (int k = 0; k < F; ++k) {
        if (k == a) continue;
        for (int i = 0; i < N; ++i) {
            size_t f = (size_t)k * N + i;
            if (!keep[f]) fuse_cnt[dst[f]] += 1;
        }
    }
}

/*
 * Compressed sequence and positions, Eqs. (xprime_stack), (compress_pos): gather the rows of X and of
 * P = {(k, y_i, x_i)} with m_{k,i} = 1, anchor rows first, then source rows by ascending flat index.
 * Rows are copied byte for byte (row_bytes = C * element size).  index_out[j] = flat index of output row j.
 * Returns L' = N + P (Eq. Lpre).  Any of out_tokens / out_pos / index_out may be NULL.
 * natural != 0 gives the other reading of "ordered index set": one pass in ascending flat index, the anchor rows
 * where they fall.  pos_base is added to all three coordinates (the offset at which a prompt places its visual
 * tokens).
 */
int ttf_oracle_compact(const void* Xbytes, size_t row_bytes, const uint8_t* keep, int F, int H, int W, int a,
                       int natural, int pos_base, void* out_tokens, int* out_pos, int* index_out) {
    const int N = H * W;
    int L = 0;
    for (int pass = natural ? 1 : 0; pass < 2; ++pass) {
        for (int k = 0; k < F; ++k) {
            /* paper's order: pass 0 = the anchor frame, pass 1 = the source frames; natural: one pass over all */
            if (!natural && (pass == 0) != (k == a)) continue;
            for (int i = 0; i < N; ++i) {
                size_t f = (size_t)k * N + i;
                if (!keep[f]) continue;
                if (out_tokens)
                    memcpy((char*)out_tokens + (size_t)L * row_bytes, (const char*)Xbytes + f * row_bytes, row_bytes);
                if (out_pos) {
                    out_pos[3 * L + 0] = pos_base + k; out_pos[3 * L + 1] = pos_base + i / W; out_pos[3 * L + 2] = pos_base + i % W;
                }
                if (index_out) index_out[L] = (int)f;
                ++L;
            }
        }
    }
    return L;
}

/*
 * TTF-R restoration (Discussion D4): the row of the compressed sequence that stands for token (k,i) is its own
 * row if m_{k,i} = 1 (anchor rows 0..N-1, then preserved source tokens in ascending flat order), else the anchor
 * row dst(k,i).  Fills row_index[F*N] and, if out_full is given, copies the rows (row_bytes each).
 */
void ttf_oracle_restore(const void* compressed, size_t row_bytes, const uint8_t* keep, const int* dst,
                        int F, int N, int a, int* row_index, void* out_full) {
    int next = N;                                   /* next preserved source row */
    for (int k = 0; k < F; ++k)
        for (int i = 0; i < N; ++i) {
            size_t f = (size_t)k * N + i;
            int row;
            if (k == a) row = i;
            else if (keep[f]) row = next++;
            else row = dst[f];
            row_index[f] = row;
            if (out_full)
                memcpy((char*)out_full + f * row_bytes, (const char*)compressed + (size_t)row * row_bytes, row_bytes);
        }
}

/*
 * Distribution of the best-match similarities of the source tokens (Discussion D1): counts over `bins` equal
 * bins of [-1, 1]: bin = floor((s + 1) / 2 * bins), clamped to [0, bins - 1]; NaN skipped.  Plain double.
 */
void ttf_oracle_sim_histogram(const float* s_hat, int F, int N, int a, int bins, unsigned int* hist) {
    for (int b = 0; b < bins; ++b) hist[b] = 0;
    for (int k = 0; k < F; ++k) {
        if (k == a) continue;
        for (int i = 0; i < N; ++i) {
            double s = (double)s_hat[(size_t)k * N + i];
            if (!(s == s)) continue;
            double x = floor((s + 1.0) / 2.0 * (double)bins);
            int b = x < 0.0 ? 0 : (x >= (double)bins ? bins - 1 : (int)x);
            hist[b] += 1;
        }
    }
}

/* Cache-aware Decode Alignment, Eqs. (Lpre), (decode_pos): pos_dec(l) = L' + T + l */
/*
 * Mean fusion.  NOT the paper's method: Sec. 3 (Threshold Gating) states that a fused token is replaced by its
 * anchor token unchanged, with no convex combination of features.  This is the averaging alternative the paper
 * contrasts itself with, written out as its plain definition so that the optional mean-fuse mode of the CUDA
 * library has something to be checked against: anchor cell j receives the arithmetic mean of its own token and
 * of every source token fused into it,
 *     out_j = ( x_{a,j} + sum_{(k,i): keep(k,i) = 0, dst(k,i) = j} x_{k,i} ) / ( 1 + fuse_cnt_j ),
 * in double.  out is [N, C].
 */
void ttf_oracle_fuse_mean(const float* X, int F, int N, int C, int a, const uint8_t* keep, const int* dst,
                          double* out) {
    int* members = (int*)malloc(sizeof(int) * (size_t)N);
    for (int j = 0; j < N; ++j) {
        members[j] = 1;
        for (int c = 0; c < C; ++c) out[(size_t)j * C + c] = (double)X[((size_t)a * N + j) * C + c];
    }
    for (int k = 0; k < F; ++k) {
        if (k == a) continue;
        for (int i = 0; i < N; ++i) {
            const size_t f = (size_t)k * N + i;
            if (keep[f]) continue;
            const int j = dst[f];
            members[j] += 1;
            for (int c = 0; c < C; ++c) out[(size_t)j * C + c] += (double)X[f * C + c];
        }
    }
    for (int j = 0; j < N; ++j)
        for (int c = 0; c < C; ++c) out[(size_t)j * C + c] /= (double)members[j];
    free(members);
}

long long ttf_oracle_decode_pos(long long L_prime, long long T, long long l) { return L_prime + T + l; }
