/*
 * ttf.h : C ABI of the B200 Temporal Token Fusion library (libttf_b200.so).
 *
 * The library implements the pre-LLM pass of Temporal Token Fusion (arXiv 2605.07355, Sec. 3) for one clip
 * of visual tokens X[F, H, W, C] on one sm_100a GPU:
 *
 *   anchor frame a* (Eq. auto_anchor)  ->  best cosine match of every source token inside the
 *   (2r+1) x (2r+1) window of the anchor grid (Eqs. pi, argmax, dst)  ->  gate keep = 1[s_hat <= t]
 *   (Eq. gating)  ->  compressed sequence X' = N anchor rows followed by the P preserved source rows
 *   (Eq. xprime_stack) with their original (k, y, x) position triples (Eqs. mask, compress_pos) and the
 *   compressed length L' = N + P that prefill and decoding use as position base (Eqs. Lpre, decode_pos).
 *
 * Fusion is the paper's identity replacement (Sec. 3, Threshold Gating): a fused token is dropped and the
 * anchor row dst(k,i) stands for it unchanged; output rows are bit copies of input rows.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer on the current CUDA device unless its name ends in _host.
 *   - The caller owns every buffer.  The library never frees caller memory and writes at most
 *     F*H*W rows into out_tokens / out_pos_thw (the worst case, nothing fused).
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as an opaque pointer; NULL = legacy default
 *     stream) and return without synchronising, except the *_host entry point.
 *   - features: contiguous [F, H, W, C], C fastest, row = one token; dtype selects fp32 or bf16.
 *     Any C >= 1 is accepted; rows whose byte length is a multiple of 16 with a 16-byte aligned base take
 *     the vectorised kernels, everything else a scalar path with identical results.
 *   - r >= 0 is the search radius (window side 2r+1); t is any finite float (not restricted to (0,1)).
 *   - Return value: a ttf_status.  Host-detectable problems (NULL pointer, non-positive size, negative r,
 *     non-finite t, unknown dtype, F*H*W*C overflow, workspace too small or misaligned) are reported
 *     before anything is launched, and nothing is written.  CUDA launch failures return TTF_ERR_CUDA.
 *   - Similarities are computed in fp32 (bf16 products are exact in fp32; fp32 accumulation); norms are
 *     floored at 1e-12, so an all-zero token has similarity 0 to everything.  A token is fused iff
 *     s_hat > t strictly; equal candidates resolve to the lowest anchor index, equal anchor cosines to the
 *     lowest frame.
 *   - Results are deterministic: no floating-point atomics, every reduction has a fixed order.
 *   - The library has no CPU fallback: without a CUDA device every compute entry point fails.
 */
#ifndef TTF_B200_H_
#define TTF_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { TTF_DTYPE_F32 = 0, TTF_DTYPE_BF16 = 1 } ttf_dtype;

typedef enum {
    TTF_OK = 0,
    TTF_ERR_INVALID_ARG = 1,   /* NULL pointer, size < 1, r < 0, non-finite t, unknown dtype or option       */
    TTF_ERR_UNSUPPORTED = 2,   /* sizes beyond int32 indexing (F*H*W >= 2^31 or F*H*W*C*itemsize >= 2^46)    */
    TTF_ERR_WORKSPACE = 3,     /* caller workspace NULL, smaller than ttf_workspace_bytes or not 256-aligned */
    TTF_ERR_CUDA = 4,          /* a CUDA runtime call failed (see ttf_last_cuda_error)                       */
    TTF_ERR_TIMEOUT = 5,       /* device status only: a kernel gave up on one of its bounded waits           */
    TTF_ERR_STATIC_LIMIT = 6,  /* ttf_query_static: the clip needs more scratch than TTF_STATIC_SCRATCH_BYTES */
    TTF_ERR_BOUNDS = 7         /* device status only, checked build: a kernel computed an index outside its array */
} ttf_status;

/* anchor rule: Eq. (auto_anchor), or the fixed first / last frame anchors compared in Table 1 and ablation A2,
 * or an explicit frame (e.g. the rolling anchor of a streaming segment, Sec. 5 D3) */
typedef enum { TTF_ANCHOR_AUTO = 0, TTF_ANCHOR_FIRST = 1, TTF_ANCHOR_LAST = 2, TTF_ANCHOR_EXPLICIT = 3 } ttf_anchor_mode;

/* order of the compressed sequence: the paper's (anchor-frame rows precede the preserved source rows, Eq.
 * xprime_stack), or every retained token in ascending flat index k*N + i (the anchor rows where they fall) */
typedef enum { TTF_ORDER_ANCHOR_FIRST = 0, TTF_ORDER_NATURAL = 1 } ttf_order;

/* Options of the _ex entry points; a NULL pointer means all zero: the automatic anchor, the paper's order, raw
 * (k, y, x) positions. */
typedef struct {
    int anchor_mode;   /* a ttf_anchor_mode                                                                      */
    int anchor_frame;  /* the frame of TTF_ANCHOR_EXPLICIT, in [0, F); ignored otherwise                         */
    int order;         /* a ttf_order                                                                            */
    int pos_base;      /* >= 0, added to all three coordinates of every emitted position (e.g. the index of the  */
                       /* first visual token in the prompt, as multimodal rotary embeddings count it)            */
} ttf_options;

typedef struct CUstream_st* ttf_stream_t;      /* same type as cudaStream_t */

/* Human-readable name of a ttf_status. Never NULL. */
const char* ttf_status_string(int status);

/* cudaError_t of the most recent failing CUDA call made by this library on the calling thread (0 if none). */
int ttf_last_cuda_error(void);

/*
 * Device-side status of the most recent call of this library on `stream` (the paper has no counterpart).  The only
 * waits inside the kernels are waits of a warp for its own asynchronous copies; each is bounded, and a warp whose
 * wait runs out stops copying and sets an error word in the call's scratch, which the first kernel of every call
 * clears.  ttf_last_device_status synchronises `stream`, reads the error word(s) of the last call enqueued on it (for
 * a batch call: of every clip of the batch) and stores TTF_OK or TTF_ERR_TIMEOUT (in the checked build also
 * TTF_ERR_BOUNDS) in *host_status.  ttf_compress also
 * reports the condition as out_count = -1; the query entry points have no other channel than this one.  The return
 * value is the status of the status query itself.  ttf_workspace_status is the same for calls that ran on
 * caller-owned scratch (`workspace` as passed to the _ws entry point; NULL = the built-in array of ttf_query_static).
 */
int ttf_last_device_status(ttf_stream_t stream, int* host_status);
int ttf_workspace_status(const void* workspace, ttf_stream_t stream, int* host_status);

/*
 * Test hooks (the paper has no counterpart; not for production use).
 * ttf_debug_set_wait: poll_limit = polls of a barrier before a waiting warp gives up (default 2^18); tx_extra_bytes
 * (a multiple of 16, normally 0) is added to the byte count every copy barrier is told to expect, so that with a
 * non-zero value the data lands but the barrier never completes and every bounded wait runs out: the give-up path
 * can be exercised without a fault or a hang.  Process-wide.
 * ttf_debug_func_attr_needed: the per-(function, device) table behind the kernels' dynamic shared memory limits;
 * returns 1 when (key, device) had not been recorded with at least `bytes` before, and records it.
 * ttf_debug_set_check_slack: only in the checked build of the library (the same sources compiled with -DTTF_DEBUG:
 * every global store whose index a kernel computes is preceded by a range test; an index outside its array is
 * recorded, the store is skipped, nothing traps, and the device status becomes TTF_ERR_BOUNDS).  `slack` >= 0 lowers
 * every limit of those tests by that many elements, so that valid indices at the end of an array are reported and
 * skipped: the reporting path can be exercised with all accesses still in bounds.  The normal build returns
 * TTF_ERR_UNSUPPORTED.
 */
int ttf_debug_set_wait(int poll_limit, int tx_extra_bytes);
int ttf_debug_func_attr_needed(const void* key, int device, size_t bytes);
int ttf_debug_set_check_slack(int slack);

/*
 * Scratch bytes one call needs for a clip of this shape (per-token inverse norms, per-frame channel sums,
 * anchor cosines, s_hat / dst / keep, per-frame survivor counts).  Sec. 3 has no counterpart: this is
 * bookkeeping of the implementation.  The result is a multiple of 256.
 */
int ttf_workspace_bytes(int F, int H, int W, int C, int r, int dtype, size_t* bytes);

/*
 * The whole pass for one clip (Sec. 3; Fig. 1): anchor selection, windowed matching, gating, compaction and
 * positional alignment.
 *   out_tokens   [capacity F*H*W rows, C] same dtype as features; rows [0, N) are the anchor frame's tokens,
 *                rows [N, N+P) the preserved source tokens in ascending flat index k*N + i (Eq. xprime_stack).
 *   out_count    one int32: L' = N + P (Eq. Lpre).  pos_dec(l) = L' + T + l (Eq. decode_pos) is
 *                ttf_decode_pos below.  -1 reports that a kernel gave up on one of its (bounded) internal
 *                waits, which does not happen on a healthy device; the other outputs are then undefined
 *                (see ttf_last_device_status).  It is written last, when every copy has completed.
 *   out_pos_thw  [capacity F*H*W, 3] int32; row j = (k, y, x) of output row j (Eq. compress_pos).
 * Rows beyond L' are not written.  Scratch comes from a cache the library keeps per (device, stream),
 * allocated with cudaMalloc on first use and grown when a larger clip arrives; two calls on the same stream
 * are ordered by the stream, calls on different streams use different scratch.
 */
int ttf_compress(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream);

/*
 * A batch of clips of one shape in one call (the long-video workload: the clips of a request processed
 * concurrently; Sec. 3 treats every clip independently, so this is scheduling only and each clip's results are
 * exactly those of ttf_compress).  features, out_tokens, out_count and out_pos_thw are HOST arrays of nclips
 * DEVICE pointers, read before the call returns.  The clips are spread round-robin over up to eight streams ("lanes")
 * that the library keeps per device; these fork from `stream` and join it again through events, so the call is
 * asynchronous, ordered on `stream` like any other, and can be captured in a CUDA graph.  The kernels of one clip
 * leave much of the GPU idle while they ramp up and drain; with several clips in flight those gaps are filled
 * (ttf_set_schedule sets the number of lanes).  Within a lane the clips form a chain on two scratch blocks used in
 * turn: the sweep of a clip runs beside the gather of the clip before it.  The streams, their events and the scratch are created by
 * the first call on a device: make that call outside any stream capture.
 */
int ttf_compress_batch(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                       int dtype, void* const* out_tokens, int* const* out_count, int* const* out_pos_thw,
                       ttf_stream_t stream);

/*
 * Kernel of the matching step for bf16 clips with r <= 2 and 16-byte aligned rows (the paper has no counterpart; the
 * results are the same within the stated tolerance): 0 automatic (the faster of the two as measured: the tcgen05
 * kernel for r = 2 and for clips with at least about 300 tiles of 32 frames x 4 cells, else the warp-level kernel);
 * 1 the warp-level tensor-core MMA kernel (one cell x 32 frames per CTA, token norms from Gram-tile diagonals); 2 the
 * tcgen05 kernel (strips of 4 cells x 32 frames as TMA tiles, accumulators in tensor memory, token norms taken from
 * the tiles in shared memory; needs C >= 64).  Process-wide; takes effect with the next call.
 */
int ttf_set_match_kernel(int which);

/*
 * Schedule of ttf_compress_batch (the paper has no counterpart).  clips_in_flight bounds how many clips of a batch run
 * concurrently (lanes): 0 = automatic, 1 to 8, or TTF_SCHEDULE_PIPELINED.  Eq. (auto_anchor) needs all of X before any token can be matched,
 * so X is read twice; with few clips in flight the second read finds the clip in L2 but the kernels of one clip leave
 * much of the GPU idle while they ramp up and drain, with many the gaps are filled but the clips displace one another
 * in L2.  Results do not depend on it.  Process-wide; takes effect with the next call.
 *
 * TTF_SCHEDULE_PIPELINED (batches of three or more clips with the automatic anchor; other batches run as with 0): two
 * lanes in opposite phases, so that one clip is matched out of L2 while the next one streams in; the matching kernel
 * and the gather mark the lines they are done with as the first to leave L2.  On the 8B-shaped clip this takes the DRAM
 * traffic of a clip from 170 MB to 133 MB (the matching pass is served by L2 for the most part), but the sweep, the
 * matching kernel and the gather slow one another down when they share the SMs and the pass is slower than with
 * eight clips in flight (32.6 against 29.8 us per clip), which is why it is not the default.
 */
#define TTF_SCHEDULE_PIPELINED (-1)
int ttf_set_schedule(int clips_in_flight);

/* Same, with caller-owned scratch: `workspace` must be 256-byte aligned device memory of at least
 * ttf_workspace_bytes(...) bytes that no other in-flight call uses.  Allocates nothing. */
int ttf_compress_ws(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                    void* out_tokens, int* out_count, int* out_pos_thw,
                    void* workspace, size_t workspace_bytes, ttf_stream_t stream);

/*
 * Query: the pass stopped before compaction (Sec. 3, Anchor Frame Selection to Threshold Gating).
 * Any output pointer may be NULL.
 *   out_anchor    one int32: a* (Eq. auto_anchor)
 *   out_keep      [F*H*W] uint8: retention mask m_{k,i} (Eq. mask); the anchor frame is all 1
 *   out_dst       [F*H*W] int32: dst(k,i), anchor-frame cell index in [0, N) (Eq. dst); i for anchor rows
 *   out_best_sim  [F*H*W] fp32: s_hat_{k,i} (Eq. argmax); 1 for anchor rows
 *   out_fuse_cnt  [H*W] int32: number of source tokens fused into each anchor cell
 *                 (|{(k,i): m_{k,i} = 0, dst(k,i) = j}|, the bookkeeping side of identity replacement)
 */
int ttf_query(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
              int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
              int* out_fuse_cnt, ttf_stream_t stream);

int ttf_query_ws(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                 int* out_fuse_cnt, void* workspace, size_t workspace_bytes, ttf_stream_t stream);

/*
 * ttf_compress / ttf_query / ttf_compress_batch with options (Table 1 rows "first", "last", "auto" and ablation A2 for
 * the anchor rule; Eqs. xprime_stack and compress_pos for order and positions).  With a fixed anchor the frame-mean
 * cosines of Eq. (auto_anchor) are not evaluated.  In natural order row j of out_tokens is the j-th retained token in
 * ascending flat index, anchor rows included (the two orders coincide when the anchor is frame 0).  Positions are
 * (pos_base + k, pos_base + y, pos_base + x).  The query outputs do not depend on order or pos_base.  Everything
 * else is as in the plain entry points (scratch from the per-stream cache).
 */
int ttf_compress_ex(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                    const ttf_options* options,
                    void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream);
int ttf_query_ex(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 const ttf_options* options,
                 int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                 int* out_fuse_cnt, ttf_stream_t stream);
int ttf_compress_batch_ex(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                          int dtype, const ttf_options* options,
                          void* const* out_tokens, int* const* out_count, int* const* out_pos_thw, ttf_stream_t stream);

/*
 * ttf_compress with MEAN fusion.  This is NOT the paper's method: Sec. 3 (Threshold Gating) replaces a fused token
 * by its anchor token unchanged and states that there is no convex combination of features.  This entry point is
 * the averaging alternative for callers who want to compare the two: everything is as in ttf_compress (same
 * anchor, matches, gate, order, positions, L'), except that anchor row j of out_tokens holds
 *     ( x_{a,j} + sum of the source tokens (k,i) with keep(k,i) = 0 and dst(k,i) = j ) / ( 1 + fuse_cnt_j ),
 * accumulated in fp32 in ascending flat order k*N + i starting from the anchor token, divided once, and rounded to
 * the clip's dtype (bf16: round to nearest even).  The reduction is segmented by anchor cell and uses no atomics,
 * so results are reproducible bit for bit.  Preserved source rows are bit copies as before.
 */
int ttf_compress_mean(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                      void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream);

/*
 * Streaming segment (Discussion D3: the last frame of each segment serves as a rolling anchor; new frames are
 * compressed against it and appended to the KV cache).  features = [F, H, W, C] whose frame 0 is the rolling
 * anchor, i.e. the last frame of the previous segment, which the consumer already holds; frames 1..F-1 are the
 * new ones and are matched against frame 0.  Only the preserved new tokens are emitted (no anchor rows):
 * out_count = P, rows in ascending flat order, positions (frame_base + k - 1, y, x) so that frame 1 of the
 * segment carries the video frame index frame_base.  Capacity (F-1)*H*W rows.  Otherwise as ttf_compress.
 */
int ttf_compress_segment(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                         int frame_base, void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream);

/*
 * TTF-R restoration (Discussion D4: a restoration step reconstructs the full spatio-temporal layout through
 * the mapping dst(k,i), Eq. dst).  `compressed` holds one row of row_bytes bytes per token of the compressed
 * sequence, in the order ttf_compress emits (any payload: the tokens themselves or what a model computed for
 * them).  out_full [F*H*W rows] receives, for token (k,i), its own compressed row if it was retained, else the
 * anchor row dst(k,i) it was fused into.  anchor (one device int), keep and dst are ttf_query's outputs.
 * row_index [F*H*W] int32 is written with the source row of every token (scratch and result).
 */
int ttf_restore(const void* compressed, size_t row_bytes, int F, int H, int W, const int* anchor,
                const unsigned char* keep, const int* dst, void* out_full, int* row_index, ttf_stream_t stream);

/*
 * The statistic an adaptive threshold would be calibrated on (Discussion D1: the empirical distribution of the
 * best-match similarities of the current clip; the paper gives no rule for choosing t from it, so only the
 * distribution is computed).  out_hist [bins] uint32: counts of best_sim over the source tokens (anchor frame
 * excluded, NaN skipped) in `bins` equal bins of [-1, 1]: bin = floor((s + 1) / 2 * bins), clamped to the range.
 */
int ttf_sim_histogram(const float* best_sim, const int* anchor, int F, int H, int W, int bins,
                      unsigned int* out_hist, ttf_stream_t stream);

/*
 * The counts behind the reduction ratio (Sec. 3, after Eq. Lpre: rho = 1 - (N + P) / (F N)) from ttf_query's
 * outputs.  out_stats [3] (device, 64-bit): [0] = P, the preserved source tokens (so L' = N + P, Eq. Lpre);
 * [1] = the fused source tokens, (F-1) N - P; [2] = the source tokens whose best similarity lies within `band` of t
 * (|best_sim - t| < band, evaluated in double on the stored fp32 values; NaN never counts): the decisions that a
 * different rounding of the similarity could flip.  The anchor frame is excluded from all three.  band >= 0.
 * ttf_reduction_ratio below turns P into rho on the host.
 */
int ttf_stats(const float* best_sim, const unsigned char* keep, const int* anchor, int F, int H, int W, float t,
              float band, long long* out_stats, ttf_stream_t stream);

/* rho = 1 - (N + P) / (F N)  (Sec. 3, after Eq. Lpre).  Host arithmetic; N = H * W. */
static inline double ttf_reduction_ratio(long long P, int F, int N) {
    return 1.0 - ((double)N + (double)P) / ((double)F * (double)N);
}

/*
 * The same pass for callers whose tensors live in HOST memory (all four pointers are host pointers; pinned
 * memory makes the copies asynchronous).  Copies features to the device, runs ttf_compress, copies L' and the
 * first L' rows of tokens and positions back, and returns after synchronising.  Device staging buffers are
 * cached per device and reused; calls from several host threads are serialised.  out_count_host receives L'.
 */
int ttf_compress_host(const void* features_host, int F, int H, int W, int C, int r, float t, int dtype,
                      void* out_tokens_host, int* out_count_host, int* out_pos_thw_host);

/*
 * ttf_compress_host for a batch of clips of one shape: features_host, out_tokens_host and out_pos_thw_host are
 * arrays of nclips HOST pointers (pinned memory makes the copies asynchronous and lets them overlap), and
 * out_count_host is an array of nclips ints that receives each clip's L'.  The clips go through two sets of
 * device staging buffers: while clip n runs and its results are copied back, clip n + 1 is already being copied
 * in, so the link to the host is busy in both directions.  Returns after everything has arrived.
 */
int ttf_compress_host_batch(const void* const* features_host, int nclips, int F, int H, int W, int C, int r, float t,
                            int dtype, void* const* out_tokens_host, int* out_count_host,
                            int* const* out_pos_thw_host);

/*
 * ttf_query for callers that must not allocate device memory.  (The paper has no counterpart: this entry
 * point exists for the needs of the host program, not of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits or too costly -- a serving loop whose memory
 * was handed over in full to a framework's pool at start-up, a latency-critical thread that cannot afford
 * the device-wide synchronisation an allocation implies, a plug-in running under a host that forbids
 * allocations after initialisation.  ttf_query allocates scratch on first use per stream and ttf_query_ws
 * needs a buffer the caller had to get from somewhere; this variant needs neither.
 *
 * How: its scratch is a fixed array of TTF_STATIC_SCRATCH_BYTES (8 MiB) that is part of the library image,
 * so every GPU on which the library is used holds those 8 MiB until the process exits, whether or not this
 * function is ever called.  Arguments, outputs and results are exactly those of ttf_query.
 *   - A clip whose scratch need (the unaligned-layout figure ttf_workspace_bytes reports is an upper bound;
 *     the 8B-shaped clip F=32, 16x16, C=4096 bf16 needs about 3 MiB) exceeds the array is rejected with
 *     TTF_ERR_STATIC_LIMIT before anything is launched.
 *   - The first call on each device looks up the array's device address (a CUDA runtime query, no
 *     allocation); make that first call outside any stream capture.  Later calls only enqueue work:
 *     a small memset of the control words, then the kernels.
 *   - All calls on a device share the one array and it keeps whatever the previous call left in it.  Calls
 *     on the same stream are ordered and safe.  Two calls that can overlap on the GPU (different streams,
 *     no event between them) race on the scratch and give undefined results: serialise them.
 * No cudaMalloc, cudaFree or other allocating routine is called on any path of this function.
 */
#define TTF_STATIC_SCRATCH_BYTES (8u << 20)
int ttf_query_static(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                     int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                     int* out_fuse_cnt, ttf_stream_t stream);

/*
 * Per-kernel timing (the paper has no counterpart; it reports no profile of the pass).  Between
 * ttf_profile_begin and ttf_profile_end every kernel this library launches is bracketed by two CUDA events
 * on its own stream.  ttf_profile_end waits for those events and returns, per kernel kind, the summed
 * device time in milliseconds and the number of launches; `kinds` is the length of both arrays
 * (TTF_KERNEL_KINDS covers all).  Kinds: 0 frame-sum (and norm) sweep, 1 frame statistics of the anchor rule,
 * 2 windowed match + gate (its prologue takes the anchor arg max), 3 compaction gather (with the frame-count
 * prefix of clips longer than 1024 frames), 4 fuse-count bookkeeping of ttf_query.  Profiling is process-wide
 * and meant for benchmarks; leave it off otherwise.
 */
#define TTF_KERNEL_KINDS 5
int ttf_profile_begin(void);
int ttf_profile_end(double* total_ms, long long* launches, int kinds);

/*
 * Steady-state duration of each kernel of the pass (no counterpart in the paper).  For `reps` rounds, each of the
 * four kernels (kinds 0..3 above) is launched back to back for all `nclips` clips of the batch, each clip on its
 * own scratch block, with one pair of CUDA events around the group; ms_per_launch[kind] = group time / nclips,
 * averaged over the rounds.  With a batch larger than L2 every launch finds its clip cold in HBM, which is how a
 * kernel runs when several clips are in flight.  Arguments as ttf_compress_batch; the outputs are those of the
 * pass.  Synchronises `stream`.
 */
int ttf_profile_stages(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                       int dtype, void* const* out_tokens, int* const* out_count, int* const* out_pos_thw,
                       int reps, double* ms_per_launch, int kinds, ttf_stream_t stream);

/*
 * Measurement aid (no counterpart in the paper): the time of the plainest kernel that reads a buffer once (fully
 * coalesced 16-byte loads, eight in flight per thread, launched like the kernels of the pass), launched back to back
 * over `nbuffers` device buffers of `bytes` bytes each (16-byte aligned, a multiple of 16), `reps` rounds after one
 * warm-up round; *ms_per_launch = time / launches.  With buffers that are together larger than L2 every launch reads
 * from HBM: this is the floor for any kernel that has to read one clip in one launch, and for clips of some 10 us
 * of HBM time it lies well below the copy rate of large buffers.  Synchronises `stream`.
 */
int ttf_profile_read_floor(const void* const* buffers, int nbuffers, size_t bytes, int reps, double* ms_per_launch,
                           ttf_stream_t stream);

/* Frees every cached scratch / staging buffer of the calling process (all devices).  Synchronises. */
int ttf_release(void);

/* Eqs. (Lpre), (decode_pos): position of the l-th generated token after a prefill of L' visual tokens
 * and T text tokens. */
static inline long long ttf_decode_pos(long long L_prime, long long T, long long l) { return L_prime + T + l; }

#ifdef __cplusplus
}
#endif
#endif /* TTF_B200_H_ */
