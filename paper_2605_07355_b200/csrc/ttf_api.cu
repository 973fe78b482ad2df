// C ABI of libttf_b200.so: argument validation, scratch management and the launch sequence of one clip.
// Declarations and the contract of every entry point are in include/ttf.h.
#include "../../include/ttf.h"
#include "ttf_internal.cuh"

#include <nvtx3/nvToolsExt.h>

#include <atomic>
#include <cmath>
#include <cstdlib>
#include <map>
#include <mutex>
#include <utility>
#include <vector>

namespace ttf {

static thread_local int tl_cuda_error = 0;

static int cuda_fail(cudaError_t e) {
    tl_cuda_error = (int)e;
    return TTF_ERR_CUDA;
}

int sm_count() {
    static std::mutex mu;
    static std::map<int, int> cache;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    std::lock_guard<std::mutex> lk(mu);
    auto it = cache.find(dev);
    if (it != cache.end()) return it->second;
    int n = 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
    cache[dev] = n;
    return n;
}

// ---- per-(function, device) record of the dynamic shared memory limit that has been set ------------------
struct FuncAttrTable {
    std::mutex mu;
    std::map<std::pair<const void*, int>, size_t> set;
    // true when (func, dev) has not been given at least `bytes` yet; records it
    bool needs(const void* func, int dev, size_t bytes) {
        std::lock_guard<std::mutex> lk(mu);
        size_t& have = set[std::make_pair(func, dev)];
        if (have >= bytes) return false;
        have = bytes;
        return true;
    }
    void forget(const void* func, int dev) {
        std::lock_guard<std::mutex> lk(mu);
        set.erase(std::make_pair(func, dev));
    }
};
static FuncAttrTable g_func_attr;

cudaError_t ensure_dynamic_smem(const void* func, size_t bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!g_func_attr.needs(func, dev, bytes)) return cudaSuccess;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) g_func_attr.forget(func, dev);
    return e;
}

static std::atomic<int> g_wait_limit{1 << 18};
static std::atomic<int> g_wait_tx_extra{0};
int wait_poll_limit() { return g_wait_limit.load(); }
int wait_tx_extra() { return g_wait_tx_extra.load(); }

// ---- optional per-kernel timing: CUDA events recorded around every launch while profiling is on ---------
enum { PK_NORM_SUM = 0, PK_FRAME_STATS = 1, PK_MATCH = 2, PK_COMPACT = 3, PK_FUSE_COUNT = 4, PK_KINDS = 5 };
struct ProfRecord { int kind; cudaEvent_t a, b; };
static std::mutex g_prof_mu;
static std::atomic<bool> g_prof_on{false};
static std::vector<ProfRecord> g_prof;

static const char* const kKindNames[PK_KINDS] = {"ttf sweep", "ttf frame statistics", "ttf matching", "ttf gather",
                                                 "ttf fuse count"};

// One scope per kernel launch: an NVTX range on the host side of the launch (a no-op unless a tool that listens is
// attached) and, while profiling is on, a pair of CUDA events around it.
struct ProfScope {
    cudaStream_t st; int kind; cudaEvent_t a = nullptr, b = nullptr; bool on;
    struct Range { Range(int k) { nvtxRangePushA(kKindNames[k]); } ~Range() { nvtxRangePop(); } } range;
    ProfScope(cudaStream_t s, int k) : st(s), kind(k), on(g_prof_on), range(k) {
        if (!on) return;
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { on = false; return; }
        cudaEventRecord(a, st);
    }
    ~ProfScope() {
        if (!on) return;
        cudaEventRecord(b, st);
        std::lock_guard<std::mutex> lk(g_prof_mu);
        g_prof.push_back({kind, a, b});
    }
};

// Schedule of a batch: clips in flight (ttf_set_schedule)
static std::atomic<int> g_sched_lanes{0};        // 0: automatic
static std::atomic<int> g_match_kernel{0};       // ttf_set_match_kernel: 0 automatic, 1 warp-level MMA, 2 tcgen05

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

void carve_scratch(const Problem& p, void* base, Scratch* s) {
    size_t off = 0;
    char* b = reinterpret_cast<char*>(base);
    auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return b ? (void*)(b + o) : nullptr; };
    const size_t FN = (size_t)p.F * p.N;
    s->hdr = (int*)take(sizeof(int) * kHdrInts);      // control words first: one small memset clears them
    s->cnt = (int*)take(sizeof(int) * p.F);
    s->prefix = (int*)take(sizeof(int) * ((size_t)p.F + 1));
    s->S = (float*)take(sizeof(float) * (size_t)p.F * p.C);
    s->Dp = (float*)take(sizeof(float) * (size_t)kStatReplicas * p.nsl * p.F);
    s->Qp = (float*)take(sizeof(float) * (size_t)kStatReplicas * p.nsl * p.F);
    s->Gp = (float*)take(sizeof(float) * (size_t)kStatReplicas * p.nsl);
    s->ssq = (float*)take(sizeof(float) * (size_t)p.nslice * FN);
    s->shat = (float*)take(sizeof(float) * FN);
    s->dst = (int*)take(sizeof(int) * FN);
    s->keep = (unsigned char*)take(FN);
    s->fuse_cnt = (int*)take(sizeof(int) * p.N);
    s->bytes = off;
}

// Validates the shape arguments and fills the derived fields.  Pointers are checked by the callers.
static int make_problem(const void* X, int F, int H, int W, int C, int r, float t, int dtype, Problem* p) {
    if (F < 1 || H < 1 || W < 1 || C < 1 || r < 0) return TTF_ERR_INVALID_ARG;
    if (dtype != TTF_DTYPE_F32 && dtype != TTF_DTYPE_BF16) return TTF_ERR_INVALID_ARG;
    if (!std::isfinite(t)) return TTF_ERR_INVALID_ARG;
    const long long N = (long long)H * W;
    const long long FN = N * F;
    if (N >= (1LL << 31) || FN >= (1LL << 31)) return TTF_ERR_UNSUPPORTED;
    const long long esize = dtype == TTF_DTYPE_F32 ? 4 : 2;
    if ((double)FN * (double)C * (double)esize >= (double)(1LL << 46)) return TTF_ERR_UNSUPPORTED;
    p->X = X; p->F = F; p->H = H; p->W = W; p->C = C; p->r = r; p->t = t; p->dtype = dtype;
    p->N = (int)N;
    const long long row_bytes = (long long)C * esize;
    p->vec = (row_bytes % 16 == 0) && (reinterpret_cast<uintptr_t>(X) % 16 == 0);
    p->lanes_elems = p->vec ? (int)(16 / esize) : 1;
    // norm sweep: one warp (32 lanes x 16 bytes) across a channel slice; measured faster than 64-lane slices
    // (11.8 vs 13.5 us on the 8B-shaped clip: twice the CTAs, half the dependent batches per thread)
    const long long chunks = ((long long)C + p->lanes_elems - 1) / p->lanes_elems;
    p->ls = 32;
    p->nq = (int)((chunks + p->ls - 1) / p->ls);
    p->nslice = p->nq * (p->ls / 32);
    if ((long long)F * p->nq >= (1LL << 31)) return TTF_ERR_UNSUPPORTED;
    p->nsl = C % 4 == 0 ? (C + 127) / 128 : (C + 31) / 32;
    p->anchor_mode = 0; p->anchor_arg = 0; p->emit_anchor = 1; p->pos_t_offset = 0; p->pos_base = 0; p->natural_order = 0;
    // Matching kernel: on request, else by measurement: the tcgen05 kernel where a clip has enough tiles to fill the
    // GPU without cutting their channel range (long clips: 112 against 115 us; the 5 x 5 window: 218 against 303 us
    // per clip), the warp-level MMA kernel for the short 16 x 16 clips (30 against 32 us on the 8B-shaped clip).
    p->use_tc = 0;
    const int which = g_match_kernel.load();
    if (tc_match_eligible(*p)) p->use_tc = which == 2 || (which == 0 && (r == 2 || tc_match_pieces(*p) == 1)) ? 1 : 0;
    p->chain = 0; p->chain_next = 0; p->overlapped = 0; p->stream_once = 0;
    return TTF_OK;
}

// ---- scratch cache: one block per (device, stream), grown on demand -------------------------------------
struct CacheEntry {
    void* ptr = nullptr; size_t bytes = 0;
    std::vector<const int*> status_words;        // header blocks the most recent call on this stream used
};
static std::mutex g_mu;
static std::map<std::pair<int, cudaStream_t>, CacheEntry> g_scratch;

static int cached_scratch(size_t bytes, cudaStream_t st, void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    std::lock_guard<std::mutex> lk(g_mu);
    CacheEntry& ce = g_scratch[std::make_pair(dev, st)];
    if (ce.bytes < bytes) {
        if (ce.ptr) {
            // earlier calls on this stream may still read the old block
            e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) return cuda_fail(e);
            cudaFree(ce.ptr);
            ce.ptr = nullptr; ce.bytes = 0;
            ce.status_words.clear();
        }
        e = cudaMalloc(&ce.ptr, bytes);
        if (e != cudaSuccess) { ce.ptr = nullptr; return cuda_fail(e); }
        ce.bytes = bytes;
        // the arrival counters must start at zero; the kernels leave them at zero after every call
        e = cudaMemsetAsync(ce.ptr, 0, bytes, st);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    *out = ce.ptr;
    ce.status_words.assign(1, reinterpret_cast<const int*>(ce.ptr));
    return TTF_OK;
}

static int check_ws(const Problem& p, void* ws, size_t ws_bytes, Scratch* s) {
    carve_scratch(p, nullptr, s);
    if (!ws || ws_bytes < s->bytes || reinterpret_cast<uintptr_t>(ws) % 256 != 0) return TTF_ERR_WORKSPACE;
    carve_scratch(p, ws, s);
    return TTF_OK;
}

// Scratch that is not the library's own may hold anything: clear the control words (stream-ordered).
static int clear_control(const Problem&, void* ws, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(ws, 0, sizeof(int) * kHdrInts, st);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

// The control words of `n` scratch blocks `stride` bytes apart.  A cached allocation that is reused with another
// clip shape holds old data where the new layout has its control words; block 0 of the cache is kept clean by the
// kernels themselves, the further blocks of a multi-clip layout are cleared before use.
static int clear_control_blocks(void* ws, size_t stride, int n, cudaStream_t st) {
    cudaError_t e = cudaMemset2DAsync(ws, stride, 0, sizeof(int) * kHdrInts, (size_t)n, st);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

// Checked build: the slack by which every index limit of the next calls is lowered (test hook, normally zero).
#ifdef TTF_DEBUG
static std::atomic<int> g_check_slack{0};
__global__ void k_set_word(int* word, int value) { *word = value; }
#endif

// steps shared by compress and query: norms + frame sums, anchor, matching + gate
static int run_front(const Problem& p, const Scratch& s, int* out_anchor, float* shat, int* dst,
                     unsigned char* keep, cudaStream_t st) {
    cudaError_t e;
#ifdef TTF_DEBUG
    k_set_word<<<1, 1, 0, st>>>(s.hdr + HDR_CHECK_SLACK, g_check_slack.load());
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
#endif
    { ProfScope ps(st, PK_NORM_SUM); e = launch_norm_sum(p, s, st); }
    if (e != cudaSuccess) return cuda_fail(e);
    if (p.anchor_mode == 0) {
        ProfScope ps(st, PK_FRAME_STATS);
        e = launch_frame_stats(p, s, out_anchor, st);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    { ProfScope ps(st, PK_MATCH); e = launch_match(p, s, out_anchor, shat, dst, keep, st); }
    if (e != cudaSuccess) return cuda_fail(e);
    return TTF_OK;
}

static int compress_impl(const Problem& p, void* ws, void* out_tokens, int* out_count, int* out_pos,
                         cudaStream_t st) {
    Scratch s;
    carve_scratch(p, ws, &s);
    int rc = run_front(p, s, nullptr, s.shat, s.dst, s.keep, st);
    if (rc != TTF_OK) return rc;
    cudaError_t e;
    { ProfScope ps(st, PK_COMPACT); e = launch_compact(p, s, out_tokens, out_pos, out_count, st); }
    if (e != cudaSuccess) return cuda_fail(e);
    return TTF_OK;
}

static int query_impl(const Problem& p, void* ws, int* out_anchor, unsigned char* out_keep, int* out_dst,
                      float* out_sim, int* out_fuse, cudaStream_t st) {
    Scratch s;
    carve_scratch(p, ws, &s);
    float* shat = out_sim ? out_sim : s.shat;
    int* dst = out_dst ? out_dst : s.dst;
    unsigned char* keep = out_keep ? out_keep : s.keep;
    int rc = run_front(p, s, out_anchor, shat, dst, keep, st);
    if (rc != TTF_OK) return rc;
    if (out_fuse) {
        cudaError_t e;
        { ProfScope ps(st, PK_FUSE_COUNT); e = launch_fuse_count(p, s, dst, keep, out_fuse, st); }
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return TTF_OK;
}

// ---- host-buffer entry point: staging buffers per device -------------------------------------------------
struct Staging {
    void* feat = nullptr; size_t feat_bytes = 0;
    void* tok = nullptr; size_t tok_bytes = 0;
    int* pos = nullptr; size_t pos_bytes = 0;
    int* count = nullptr;
    cudaStream_t stream = nullptr;
};
static std::map<int, Staging> g_staging;

static cudaError_t grow(void** p, size_t* have, size_t want) {
    if (*have >= want) return cudaSuccess;
    if (*p) cudaFree(*p);
    *p = nullptr; *have = 0;
    cudaError_t e = cudaMalloc(p, want);
    if (e == cudaSuccess) *have = want;
    return e;
}

// ---- scratch of ttf_query_static: part of the library image, one copy per GPU that loads it --------------
// In host code `g_static_scratch` is only a handle for the runtime's symbol calls, never a device address;
// static_scratch_address() asks the runtime for the address once per device and caches it.
static __device__ __align__(256) unsigned char g_static_scratch[TTF_STATIC_SCRATCH_BYTES];
constexpr int kMaxStaticDevices = 64;
static void* g_static_addr[kMaxStaticDevices] = {};
static std::mutex g_static_mu;

static int static_scratch_address(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxStaticDevices) return TTF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);     // `dev` is current: the address is this device's copy
        if (e != cudaSuccess) return cuda_fail(e);
        if (!p || reinterpret_cast<uintptr_t>(p) % 256 != 0) return TTF_ERR_WORKSPACE;
        g_static_addr[dev] = p;
    }
    *out = g_static_addr[dev];
    return TTF_OK;
}

}  // namespace ttf

using namespace ttf;

extern "C" {

const char* ttf_status_string(int status) {
    switch (status) {
        case TTF_OK: return "TTF_OK";
        case TTF_ERR_INVALID_ARG: return "TTF_ERR_INVALID_ARG";
        case TTF_ERR_UNSUPPORTED: return "TTF_ERR_UNSUPPORTED";
        case TTF_ERR_WORKSPACE: return "TTF_ERR_WORKSPACE";
        case TTF_ERR_CUDA: return "TTF_ERR_CUDA";
        case TTF_ERR_TIMEOUT: return "TTF_ERR_TIMEOUT";
        case TTF_ERR_STATIC_LIMIT: return "TTF_ERR_STATIC_LIMIT";
        case TTF_ERR_BOUNDS: return "TTF_ERR_BOUNDS";
        default: return "TTF_ERR_UNKNOWN";
    }
}

int ttf_last_cuda_error(void) { return tl_cuda_error; }

static int read_status_words(const std::vector<const int*>& words, int* host_status) {
    *host_status = TTF_OK;
    for (const int* hdr : words) {
        int v = 0;
        cudaError_t e = cudaMemcpy(&v, hdr + HDR_ERROR, sizeof(int), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(e);
        if (v == 2) *host_status = TTF_ERR_BOUNDS;                   // (checked build only)
        else if (v && *host_status == TTF_OK) *host_status = TTF_ERR_TIMEOUT;
    }
    return TTF_OK;
}

int ttf_last_device_status(ttf_stream_t stream, int* host_status) {
    if (!host_status) return TTF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    std::vector<const int*> words;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_scratch.find(std::make_pair(dev, st));
        if (it != g_scratch.end()) words = it->second.status_words;
    }
    return read_status_words(words, host_status);     // no call of the library on this stream yet: TTF_OK
}

int ttf_workspace_status(const void* workspace, ttf_stream_t stream, int* host_status) {
    if (!host_status) return TTF_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e);
    void* ws = const_cast<void*>(workspace);
    if (!ws) {                                   // NULL: the built-in array of ttf_query_static
        int rc = static_scratch_address(&ws);
        if (rc != TTF_OK) return rc;
    }
    return read_status_words(std::vector<const int*>(1, reinterpret_cast<const int*>(ws)), host_status);
}

#ifdef TTF_TRACE
// trace builds only: copies the trace marks (48 64-bit words) of scratch block `block` of the last call on `stream`
// to host memory and clears them; returns the number of blocks that call used
int ttf_trace_read(ttf_stream_t stream, int block, unsigned long long* host_out) {
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_scratch.find(std::make_pair(dev, (cudaStream_t)stream));
    if (it == g_scratch.end()) return 0;
    const int n = (int)it->second.status_words.size();
    if (block >= 0 && block < n) {
        const int* hdr = it->second.status_words[block];
        cudaMemcpy(host_out, hdr + 16, 384, cudaMemcpyDeviceToHost);
        cudaMemset(const_cast<int*>(hdr) + 16, 0, 384);
    }
    return n;
}
#endif

int ttf_debug_set_wait(int poll_limit, int tx_extra_bytes) {
    if (poll_limit < 1 || tx_extra_bytes < 0 || tx_extra_bytes % 16 != 0 || tx_extra_bytes > 1024) return TTF_ERR_INVALID_ARG;
    g_wait_limit.store(poll_limit);
    g_wait_tx_extra.store(tx_extra_bytes);
    return TTF_OK;
}

int ttf_debug_func_attr_needed(const void* key, int device, size_t bytes) {
    return g_func_attr.needs(key, device, bytes) ? 1 : 0;
}

int ttf_workspace_bytes(int F, int H, int W, int C, int r, int dtype, size_t* bytes) {
    if (!bytes) return TTF_ERR_INVALID_ARG;
    Problem p;
    // the scalar layout (one channel per lane) is the larger one: size for it so that the same scratch
    // serves a clip whatever the alignment of its base pointer
    int rc = make_problem(reinterpret_cast<const void*>(uintptr_t(1)), F, H, W, C, r, 0.f, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    size_t need = s.bytes;
    rc = make_problem(reinterpret_cast<const void*>(uintptr_t(256)), F, H, W, C, r, 0.f, dtype, &p);
    if (rc != TTF_OK) return rc;
    carve_scratch(p, nullptr, &s);
    if (s.bytes > need) need = s.bytes;
    *bytes = need;
    return TTF_OK;
}

int ttf_compress_ws(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                    void* out_tokens, int* out_count, int* out_pos_thw,
                    void* workspace, size_t workspace_bytes, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    rc = check_ws(p, workspace, workspace_bytes, &s);
    if (rc != TTF_OK) return rc;
    rc = clear_control(p, workspace, (cudaStream_t)stream);
    if (rc != TTF_OK) return rc;
    return compress_impl(p, workspace, out_tokens, out_count, out_pos_thw, (cudaStream_t)stream);
}

int ttf_compress(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    return compress_impl(p, ws, out_tokens, out_count, out_pos_thw, (cudaStream_t)stream);
}

int ttf_query_ws(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                 int* out_fuse_cnt, void* workspace, size_t workspace_bytes, ttf_stream_t stream) {
    if (!features) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    rc = check_ws(p, workspace, workspace_bytes, &s);
    if (rc != TTF_OK) return rc;
    rc = clear_control(p, workspace, (cudaStream_t)stream);
    if (rc != TTF_OK) return rc;
    return query_impl(p, workspace, out_anchor, out_keep, out_dst, out_best_sim, out_fuse_cnt,
                      (cudaStream_t)stream);
}

int ttf_query(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
              int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
              int* out_fuse_cnt, ttf_stream_t stream) {
    if (!features) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    return query_impl(p, ws, out_anchor, out_keep, out_dst, out_best_sim, out_fuse_cnt, (cudaStream_t)stream);
}

static int set_anchor_rule(Problem* p, int anchor_mode, int anchor_frame) {
    if (anchor_mode < TTF_ANCHOR_AUTO || anchor_mode > TTF_ANCHOR_EXPLICIT) return TTF_ERR_INVALID_ARG;
    if (anchor_mode == TTF_ANCHOR_EXPLICIT && (anchor_frame < 0 || anchor_frame >= p->F)) return TTF_ERR_INVALID_ARG;
    p->anchor_mode = anchor_mode;
    p->anchor_arg = anchor_mode == TTF_ANCHOR_EXPLICIT ? anchor_frame : 0;
    return TTF_OK;
}

static int set_output_options(Problem* p, int order, int pos_base) {
    if (order != TTF_ORDER_ANCHOR_FIRST && order != TTF_ORDER_NATURAL) return TTF_ERR_INVALID_ARG;
    // positions stay inside int32: the largest coordinate is max(F, H, W) - 1 + pos_base
    const long long top = (long long)(p->F > p->H ? (p->F > p->W ? p->F : p->W) : (p->H > p->W ? p->H : p->W)) + pos_base;
    if (pos_base < 0 || top >= (1LL << 31)) return TTF_ERR_INVALID_ARG;
    p->natural_order = order == TTF_ORDER_NATURAL ? 1 : 0;
    p->pos_base = pos_base;
    return TTF_OK;
}

static int apply_options(Problem* p, const ttf_options* opt) {
    if (!opt) return TTF_OK;
    int rc = set_anchor_rule(p, opt->anchor_mode, opt->anchor_frame);
    if (rc == TTF_OK) rc = set_output_options(p, opt->order, opt->pos_base);
    return rc;
}

int ttf_compress_ex(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                    const ttf_options* options,
                    void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc == TTF_OK) rc = apply_options(&p, options);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    return compress_impl(p, ws, out_tokens, out_count, out_pos_thw, (cudaStream_t)stream);
}

int ttf_query_ex(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                 const ttf_options* options,
                 int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                 int* out_fuse_cnt, ttf_stream_t stream) {
    if (!features) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc == TTF_OK) rc = apply_options(&p, options);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    return query_impl(p, ws, out_anchor, out_keep, out_dst, out_best_sim, out_fuse_cnt, (cudaStream_t)stream);
}

int ttf_compress_mean(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                      void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    rc = compress_impl(p, ws, out_tokens, out_count, out_pos_thw, (cudaStream_t)stream);
    if (rc != TTF_OK) return rc;
    carve_scratch(p, ws, &s);
    cudaError_t e = launch_fuse_mean(p, s, out_tokens, (cudaStream_t)stream);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

// ---- batches on the library's own streams -----------------------------------------------------------------
// The clips of a batch are independent, and the kernels of one clip leave most of the GPU idle while they ramp up
// and drain, so a batch is spread round-robin over kBatchStreams internal streams per device that fork from the
// caller's stream and join it again (events only: the call stays asynchronous and can be captured in a graph).
constexpr int kBatchStreams = 8;
constexpr int kMatchedRing = 4;                  // events "clip n has been matched" of the pipelined schedule, used in turn
struct BatchLanes {
    cudaStream_t s[kBatchStreams] = {}; cudaEvent_t fork = nullptr; cudaEvent_t join[kBatchStreams] = {};
    cudaEvent_t matched[kMatchedRing] = {};
    bool ok = false;
};
static std::map<int, BatchLanes> g_lanes;
static std::mutex g_lane_mu;                     // the fork / join events are shared: one batch is enqueued at a time

static int batch_lanes(BatchLanes** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    std::lock_guard<std::mutex> lk(g_mu);
    BatchLanes& L = g_lanes[dev];
    if (!L.ok) {
        e = cudaEventCreateWithFlags(&L.fork, cudaEventDisableTiming);
        for (int i = 0; i < kBatchStreams && e == cudaSuccess; ++i) {
            e = cudaStreamCreateWithFlags(&L.s[i], cudaStreamNonBlocking);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&L.join[i], cudaEventDisableTiming);
        }
        for (int i = 0; i < kMatchedRing && e == cudaSuccess; ++i)
            e = cudaEventCreateWithFlags(&L.matched[i], cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(e);
        L.ok = true;
    }
    *out = &L;
    return TTF_OK;
}

// The clips of a lane form a chain on the lane's stream: sweep, statistics, matching, gather, next sweep, ... with two
// scratch blocks used in turn, so that the sweep of a clip can run beside the gather of the clip before it.
static int batch_on_streams(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                            int dtype, const ttf_options* options,
                            void* const* out_tokens, int* const* out_count, int* const* out_pos_thw, cudaStream_t st) {
    std::lock_guard<std::mutex> enqueue(g_lane_mu);
    BatchLanes* L = nullptr;
    int rc = batch_lanes(&L);
    if (rc != TTF_OK) return rc;
    std::vector<Problem> ps(nclips);
    size_t stride = 0;
    for (int n = 0; n < nclips; ++n) {
        rc = make_problem(features[n], F, H, W, C, r, t, dtype, &ps[n]);
        if (rc == TTF_OK) rc = apply_options(&ps[n], options);
        if (rc != TTF_OK) return rc;
        Scratch s;
        carve_scratch(ps[n], nullptr, &s);
        if (s.bytes > stride) stride = s.bytes;
    }
    int want = g_sched_lanes.load();
    // Pipelined schedule (TTF_SCHEDULE_PIPELINED, automatic anchor only).  Eq. (auto_anchor) forces two passes over X;
    // the second is free only while the clip is still in L2, which holds one 8B-shaped clip and most of a second.
    // Two lanes in opposite phases: the matching kernels of consecutive clips are ordered one after the other, and a
    // lane's next sweep starts when its previous clip has been matched (the chain below), so at any time one clip is
    // matched out of L2 while the next one streams in.  The matching kernel marks the source rows it has read, and
    // the gather what it reads and writes, as the first lines to leave L2; without that the incoming clip displaces
    // exactly the rows that are still to be matched (they are the oldest lines).
    const bool pipelined = want == TTF_SCHEDULE_PIPELINED && nclips >= 3 && ps[0].anchor_mode == 0;
    if (pipelined) want = 2;
    if (want < 1 || want > kBatchStreams) want = kBatchStreams;      // automatic: measured best for every clip shape so far
    const int lanes = nclips < want ? nclips : want;
    std::vector<void*> ws(lanes, nullptr);
    for (int i = 0; i < lanes; ++i) {            // (may allocate: before the fork, outside the event bracket)
        rc = cached_scratch(2 * stride, L->s[i], &ws[i]);
        if (rc != TTF_OK) return rc;
    }
    cudaError_t e = cudaEventRecord(L->fork, st);
    for (int i = 0; i < lanes && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(L->s[i], L->fork, 0);
    if (e != cudaSuccess) return cuda_fail(e);
    int first_rc = TTF_OK;
    std::vector<const int*> words;
    for (int n = 0; n < nclips && first_rc == TTF_OK; ++n) {
        const int lane = n % lanes, turn = n / lanes;
        void* block = (char*)ws[lane] + (size_t)(turn & 1) * stride;
        ps[n].overlapped = lanes;
        ps[n].stream_once = pipelined ? 1 : 0;
        ps[n].chain = turn > 0 ? 1 : 0;          // the lane's previous kernel is the gather of its previous clip
        if (turn < 2) {
            // the block may hold anything (another shape's data, or a failed call's counters): clear its control words
            first_rc = clear_control(ps[n], block, L->s[lane]);
            words.push_back(reinterpret_cast<const int*>(block));
            if (first_rc != TTF_OK) break;
            if (turn == 1) ps[n].chain = 0;      // (the memset sits between the gather and this sweep)
        }
        // (the lane's next clip, if there is one, is at turn + 1; its sweep is chained from turn 2 on)
        ps[n].chain_next = (n + lanes < nclips && turn + 1 >= 2) ? 1 : 0;
        if (!pipelined) {
            first_rc = compress_impl(ps[n], block, out_tokens[n], out_count[n], out_pos_thw[n], L->s[lane]);
            continue;
        }
        // the same kernels as compress_impl, with the matching kernel ordered after that of the clip before (which
        // ran in the other lane)
        Scratch sc;
        carve_scratch(ps[n], block, &sc);
        cudaStream_t ls = L->s[lane];
        { ProfScope pr(ls, PK_NORM_SUM); e = launch_norm_sum(ps[n], sc, ls); }
        if (e == cudaSuccess) { ProfScope pr(ls, PK_FRAME_STATS); e = launch_frame_stats(ps[n], sc, nullptr, ls); }
        if (e == cudaSuccess && n > 0) e = cudaStreamWaitEvent(ls, L->matched[(n - 1) % kMatchedRing], 0);
        if (e == cudaSuccess) { ProfScope pr(ls, PK_MATCH); e = launch_match(ps[n], sc, nullptr, sc.shat, sc.dst, sc.keep, ls); }
        if (e == cudaSuccess) e = cudaEventRecord(L->matched[n % kMatchedRing], ls);
        if (e == cudaSuccess) { ProfScope pr(ls, PK_COMPACT); e = launch_compact(ps[n], sc, out_tokens[n], out_pos_thw[n], out_count[n], ls); }
        if (e != cudaSuccess) first_rc = cuda_fail(e);
    }
    {   // the caller asks about the batch through its own stream: point it at the lanes' error words
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) {
            std::lock_guard<std::mutex> lk(g_mu);
            g_scratch[std::make_pair(dev, st)].status_words = words;
        }
    }
    // always join, also after a failed launch, so that the caller's stream (or capture) is whole again
    for (int i = 0; i < lanes; ++i) {
        cudaError_t e2 = cudaEventRecord(L->join[i], L->s[i]);
        if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(st, L->join[i], 0);
        if (e2 != cudaSuccess && e == cudaSuccess) e = e2;
    }
    if (first_rc != TTF_OK) return first_rc;
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_set_match_kernel(int which) {
    if (which < 0 || which > 2) return TTF_ERR_INVALID_ARG;
    g_match_kernel.store(which);
    return TTF_OK;
}

int ttf_set_schedule(int clips_in_flight) {
    if (clips_in_flight < TTF_SCHEDULE_PIPELINED || clips_in_flight > kBatchStreams) return TTF_ERR_INVALID_ARG;
    g_sched_lanes.store(clips_in_flight);
    return TTF_OK;
}

int ttf_compress_batch(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                       int dtype, void* const* out_tokens, int* const* out_count, int* const* out_pos_thw,
                       ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw || nclips < 1) return TTF_ERR_INVALID_ARG;
    for (int n = 0; n < nclips; ++n)
        if (!features[n] || !out_tokens[n] || !out_count[n] || !out_pos_thw[n]) return TTF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    Problem p;
    int rc = make_problem(features[0], F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    return batch_on_streams(features, nclips, F, H, W, C, r, t, dtype, nullptr, out_tokens, out_count, out_pos_thw, st);
}

int ttf_compress_batch_ex(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                          int dtype, const ttf_options* options,
                          void* const* out_tokens, int* const* out_count, int* const* out_pos_thw, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw || nclips < 1) return TTF_ERR_INVALID_ARG;
    for (int n = 0; n < nclips; ++n)
        if (!features[n] || !out_tokens[n] || !out_count[n] || !out_pos_thw[n]) return TTF_ERR_INVALID_ARG;
    return batch_on_streams(features, nclips, F, H, W, C, r, t, dtype, options, out_tokens, out_count, out_pos_thw,
                            (cudaStream_t)stream);
}

int ttf_compress_segment(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                         int frame_base, void* out_tokens, int* out_count, int* out_pos_thw, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc == TTF_OK) rc = set_anchor_rule(&p, TTF_ANCHOR_FIRST, 0);
    if (rc != TTF_OK) return rc;
    p.emit_anchor = 0;
    p.pos_t_offset = frame_base - 1;             // frame 1 of the segment is frame `frame_base` of the video
    Scratch s;
    carve_scratch(p, nullptr, &s);
    void* ws = nullptr;
    rc = cached_scratch(s.bytes, (cudaStream_t)stream, &ws);
    if (rc != TTF_OK) return rc;
    return compress_impl(p, ws, out_tokens, out_count, out_pos_thw, (cudaStream_t)stream);
}

int ttf_restore(const void* compressed, size_t row_bytes, int F, int H, int W, const int* anchor,
                const unsigned char* keep, const int* dst, void* out_full, int* row_index, ttf_stream_t stream) {
    if (!compressed || !anchor || !keep || !dst || !out_full || !row_index) return TTF_ERR_INVALID_ARG;
    if (F < 1 || H < 1 || W < 1 || row_bytes < 1) return TTF_ERR_INVALID_ARG;
    if ((long long)F * H * W >= (1LL << 31)) return TTF_ERR_UNSUPPORTED;
    cudaError_t e = launch_restore(compressed, row_bytes, F, H * W, anchor, keep, dst, out_full, row_index,
                                   (cudaStream_t)stream);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_sim_histogram(const float* best_sim, const int* anchor, int F, int H, int W, int bins,
                      unsigned int* out_hist, ttf_stream_t stream) {
    if (!best_sim || !anchor || !out_hist || F < 1 || H < 1 || W < 1 || bins < 1) return TTF_ERR_INVALID_ARG;
    if ((long long)F * H * W >= (1LL << 31)) return TTF_ERR_UNSUPPORTED;
    cudaError_t e = launch_sim_histogram(best_sim, anchor, F, H * W, bins, out_hist, (cudaStream_t)stream);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_debug_set_check_slack(int slack) {
#ifdef TTF_DEBUG
    if (slack < 0) return TTF_ERR_INVALID_ARG;
    g_check_slack.store(slack);
    return TTF_OK;
#else
    (void)slack;
    return TTF_ERR_UNSUPPORTED;                  // this build carries no index checks
#endif
}

int ttf_stats(const float* best_sim, const unsigned char* keep, const int* anchor, int F, int H, int W, float t,
              float band, long long* out_stats, ttf_stream_t stream) {
    if (!best_sim || !keep || !anchor || !out_stats || F < 1 || H < 1 || W < 1 || !(band >= 0.0f) || !(t == t))
        return TTF_ERR_INVALID_ARG;
    if ((long long)F * H * W >= (1LL << 31)) return TTF_ERR_UNSUPPORTED;
    cudaError_t e = launch_stats(best_sim, keep, anchor, F, H * W, t, band, out_stats, (cudaStream_t)stream);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_query_static(const void* features, int F, int H, int W, int C, int r, float t, int dtype,
                     int* out_anchor, unsigned char* out_keep, int* out_dst, float* out_best_sim,
                     int* out_fuse_cnt, ttf_stream_t stream) {
    if (!features) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(features, F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    Scratch s;
    carve_scratch(p, nullptr, &s);
    if (s.bytes > (size_t)TTF_STATIC_SCRATCH_BYTES) return TTF_ERR_STATIC_LIMIT;
    void* ws = nullptr;
    rc = static_scratch_address(&ws);
    if (rc != TTF_OK) return rc;
    // the array still holds the previous call's state: the control words must start at zero
    rc = clear_control(p, ws, (cudaStream_t)stream);
    if (rc != TTF_OK) return rc;
    return query_impl(p, ws, out_anchor, out_keep, out_dst, out_best_sim, out_fuse_cnt, (cudaStream_t)stream);
}

int ttf_compress_host(const void* features_host, int F, int H, int W, int C, int r, float t, int dtype,
                      void* out_tokens_host, int* out_count_host, int* out_pos_thw_host) {
    if (!features_host || !out_tokens_host || !out_count_host || !out_pos_thw_host) return TTF_ERR_INVALID_ARG;
    Problem p;
    // the staging copy is always 256-byte aligned: validate with an aligned stand-in pointer
    int rc = make_problem(reinterpret_cast<const void*>(uintptr_t(256)), F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    const size_t esize = dtype == TTF_DTYPE_F32 ? 4 : 2;
    const size_t FN = (size_t)p.F * p.N;
    const size_t row_bytes = (size_t)C * esize;

    // one host call at a time per process: the staging buffers and their stream are shared, and a second call with a
    // larger clip would free buffers the first still uses
    static std::mutex host_call_mu;
    std::lock_guard<std::mutex> whole_call(host_call_mu);
    std::unique_lock<std::mutex> lk(g_mu);
    Staging& sg = g_staging[dev];
    if (!sg.stream) {
        e = cudaStreamCreateWithFlags(&sg.stream, cudaStreamNonBlocking);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (!sg.count) {
        e = cudaMalloc((void**)&sg.count, 256);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    e = grow(&sg.feat, &sg.feat_bytes, FN * row_bytes);
    if (e == cudaSuccess) e = grow(&sg.tok, &sg.tok_bytes, FN * row_bytes);
    if (e == cudaSuccess) e = grow((void**)&sg.pos, &sg.pos_bytes, FN * 3 * sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e);
    Staging local = sg;
    lk.unlock();

    cudaStream_t st = local.stream;
    e = cudaMemcpyAsync(local.feat, features_host, FN * row_bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e);
    rc = ttf_compress(local.feat, F, H, W, C, r, t, dtype, local.tok, local.count, local.pos, st);
    if (rc != TTF_OK) return rc;
    e = cudaMemcpyAsync(out_count_host, local.count, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    const size_t L = (size_t)*out_count_host;
    if (L > FN) return TTF_ERR_CUDA;
    e = cudaMemcpyAsync(out_tokens_host, local.tok, L * row_bytes, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_pos_thw_host, local.pos, L * 3 * sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e);
    return TTF_OK;
}

// ---- host-buffer batch: copies in, kernels and copies out of consecutive clips overlap ----------------------
struct HostPipe {
    struct Slot { void* feat = nullptr; void* tok = nullptr; int* pos = nullptr; int* count = nullptr;
                  cudaEvent_t loaded = nullptr, computed = nullptr, drained = nullptr; } slot[2];
    size_t row_cap = 0, rows_cap = 0;            // capacity of the slot buffers: bytes per row, rows
    cudaStream_t up = nullptr, run = nullptr, down = nullptr;
    int* count_host = nullptr;                   // pinned, one int per slot
    bool ok = false;
};
static std::map<int, HostPipe> g_pipes;
static std::mutex g_pipe_mu;                     // one host batch at a time per process

static cudaError_t pipe_prepare(HostPipe& hp, size_t FN, size_t row_bytes) {
    cudaError_t e = cudaSuccess;
    if (!hp.ok) {
        e = cudaStreamCreateWithFlags(&hp.up, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&hp.run, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&hp.down, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaHostAlloc((void**)&hp.count_host, 2 * sizeof(int), cudaHostAllocDefault);
        for (auto& sl : hp.slot) {
            if (e == cudaSuccess) e = cudaMalloc((void**)&sl.count, 256);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sl.loaded, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sl.computed, cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&sl.drained, cudaEventDisableTiming);
        }
        if (e != cudaSuccess) return e;
        hp.ok = true;
    }
    if (hp.rows_cap * hp.row_cap < FN * row_bytes || hp.rows_cap < FN) {
        e = cudaDeviceSynchronize();
        for (auto& sl : hp.slot) {
            if (sl.feat) cudaFree(sl.feat);
            if (sl.tok) cudaFree(sl.tok);
            if (sl.pos) cudaFree(sl.pos);
            sl.feat = sl.tok = nullptr; sl.pos = nullptr;
            if (e == cudaSuccess) e = cudaMalloc(&sl.feat, FN * row_bytes);
            if (e == cudaSuccess) e = cudaMalloc(&sl.tok, FN * row_bytes);
            if (e == cudaSuccess) e = cudaMalloc((void**)&sl.pos, FN * 3 * sizeof(int));
        }
        if (e != cudaSuccess) { hp.rows_cap = hp.row_cap = 0; return e; }
        hp.rows_cap = FN; hp.row_cap = row_bytes;
    }
    return cudaSuccess;
}

int ttf_compress_host_batch(const void* const* features_host, int nclips, int F, int H, int W, int C, int r, float t,
                            int dtype, void* const* out_tokens_host, int* out_count_host,
                            int* const* out_pos_thw_host) {
    if (!features_host || !out_tokens_host || !out_count_host || !out_pos_thw_host || nclips < 1) return TTF_ERR_INVALID_ARG;
    for (int n = 0; n < nclips; ++n)
        if (!features_host[n] || !out_tokens_host[n] || !out_pos_thw_host[n]) return TTF_ERR_INVALID_ARG;
    Problem p;
    int rc = make_problem(reinterpret_cast<const void*>(uintptr_t(256)), F, H, W, C, r, t, dtype, &p);
    if (rc != TTF_OK) return rc;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    const size_t esize = dtype == TTF_DTYPE_F32 ? 4 : 2;
    const size_t FN = (size_t)p.F * p.N, row_bytes = (size_t)C * esize;

    std::lock_guard<std::mutex> lk(g_pipe_mu);
    HostPipe& hp = g_pipes[dev];
    e = pipe_prepare(hp, FN, row_bytes);
    if (e != cudaSuccess) return cuda_fail(e);

    auto load_and_run = [&](int n) -> int {      // copy clip n in and run the pass on it, all asynchronous
        HostPipe::Slot& sl = hp.slot[n & 1];
        cudaError_t e2 = cudaSuccess;
        if (n >= 2) e2 = cudaStreamWaitEvent(hp.up, sl.drained, 0);          // the slot's last results have left
        if (e2 == cudaSuccess) e2 = cudaMemcpyAsync(sl.feat, features_host[n], FN * row_bytes, cudaMemcpyHostToDevice, hp.up);
        if (e2 == cudaSuccess) e2 = cudaEventRecord(sl.loaded, hp.up);
        if (e2 == cudaSuccess) e2 = cudaStreamWaitEvent(hp.run, sl.loaded, 0);
        if (e2 != cudaSuccess) return cuda_fail(e2);
        int rc2 = ttf_compress(sl.feat, F, H, W, C, r, t, dtype, sl.tok, sl.count, sl.pos, (ttf_stream_t)hp.run);
        if (rc2 != TTF_OK) return rc2;
        e2 = cudaEventRecord(sl.computed, hp.run);
        return e2 == cudaSuccess ? TTF_OK : cuda_fail(e2);
    };

    rc = load_and_run(0);
    for (int n = 0; n < nclips && rc == TTF_OK; ++n) {
        if (n + 1 < nclips) rc = load_and_run(n + 1);                        // next clip travels while this one drains
        if (rc != TTF_OK) break;
        HostPipe::Slot& sl = hp.slot[n & 1];
        e = cudaStreamWaitEvent(hp.down, sl.computed, 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(hp.count_host + (n & 1), sl.count, sizeof(int), cudaMemcpyDeviceToHost, hp.down);
        if (e == cudaSuccess) e = cudaStreamSynchronize(hp.down);            // L' sizes the copies back
        if (e != cudaSuccess) { rc = cuda_fail(e); break; }
        const int Lp = hp.count_host[n & 1];
        out_count_host[n] = Lp;
        if (Lp < 0 || (size_t)Lp > FN) { rc = TTF_ERR_CUDA; break; }
        e = cudaMemcpyAsync(out_tokens_host[n], sl.tok, (size_t)Lp * row_bytes, cudaMemcpyDeviceToHost, hp.down);
        if (e == cudaSuccess) e = cudaMemcpyAsync(out_pos_thw_host[n], sl.pos, (size_t)Lp * 3 * sizeof(int), cudaMemcpyDeviceToHost, hp.down);
        if (e == cudaSuccess) e = cudaEventRecord(sl.drained, hp.down);
        if (e != cudaSuccess) { rc = cuda_fail(e); break; }
    }
    // nothing of this call stays in flight, whatever happened
    cudaError_t e1 = cudaStreamSynchronize(hp.up), e2 = cudaStreamSynchronize(hp.run), e3 = cudaStreamSynchronize(hp.down);
    if (rc != TTF_OK) return rc;
    if (e1 != cudaSuccess) return cuda_fail(e1);
    if (e2 != cudaSuccess) return cuda_fail(e2);
    if (e3 != cudaSuccess) return cuda_fail(e3);
    return TTF_OK;
}

int ttf_profile_begin(void) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    for (auto& r : g_prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    g_prof.clear();
    g_prof_on = true;
    return TTF_OK;
}

int ttf_profile_end(double* total_ms, long long* launches, int kinds) {
    if (!total_ms || !launches || kinds < 1) return TTF_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = false;
    for (int k = 0; k < kinds; ++k) { total_ms[k] = 0.0; launches[k] = 0; }
    cudaError_t first = cudaSuccess;
    for (auto& r : g_prof) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(r.b);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.a, r.b);
        if (e != cudaSuccess && first == cudaSuccess) first = e;
        if (e == cudaSuccess && r.kind < kinds) { total_ms[r.kind] += ms; launches[r.kind] += 1; }
        cudaEventDestroy(r.a); cudaEventDestroy(r.b);
    }
    g_prof.clear();
    return first == cudaSuccess ? TTF_OK : cuda_fail(first);
}

int ttf_profile_stages(const void* const* features, int nclips, int F, int H, int W, int C, int r, float t,
                       int dtype, void* const* out_tokens, int* const* out_count, int* const* out_pos_thw,
                       int reps, double* ms_per_launch, int kinds, ttf_stream_t stream) {
    if (!features || !out_tokens || !out_count || !out_pos_thw || !ms_per_launch || nclips < 1 || reps < 1 ||
        kinds < 4) return TTF_ERR_INVALID_ARG;
    for (int n = 0; n < nclips; ++n)
        if (!features[n] || !out_tokens[n] || !out_count[n] || !out_pos_thw[n]) return TTF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<Problem> ps(nclips);
    int want = g_sched_lanes.load();             // the kernels a batch call of these clips would launch
    if (want < 1 || want > kBatchStreams) want = kBatchStreams;
    for (int n = 0; n < nclips; ++n) {
        int rc = make_problem(features[n], F, H, W, C, r, t, dtype, &ps[n]);
        if (rc != TTF_OK) return rc;
        ps[n].overlapped = nclips < want ? nclips : want;
    }
    Scratch s0;
    carve_scratch(ps[0], nullptr, &s0);
    size_t stride = s0.bytes;
    for (int n = 1; n < nclips; ++n) {           // (the layout depends on the alignment of the clip)
        Scratch sn;
        carve_scratch(ps[n], nullptr, &sn);
        if (sn.bytes > stride) stride = sn.bytes;
    }
    void* ws = nullptr;
    int rc = cached_scratch(stride * nclips, st, &ws);
    if (rc != TTF_OK) return rc;
    rc = clear_control_blocks(ws, stride, nclips, st);
    if (rc != TTF_OK) return rc;
    cudaEvent_t ev[5];
    for (auto& e : ev) if (cudaEventCreate(&e) != cudaSuccess) return cuda_fail(cudaGetLastError());
    for (int k = 0; k < kinds; ++k) ms_per_launch[k] = 0.0;
    cudaError_t e = cudaSuccess;
    for (int rep = 0; rep < reps && e == cudaSuccess; ++rep) {
        for (int stage = 0; stage < 4 && e == cudaSuccess; ++stage) {
            cudaEventRecord(ev[stage], st);
            for (int n = 0; n < nclips && e == cudaSuccess; ++n) {
                Scratch s;
                carve_scratch(ps[n], (char*)ws + stride * n, &s);
                if (stage == 0) e = launch_norm_sum(ps[n], s, st);
                else if (stage == 1) e = launch_frame_stats(ps[n], s, nullptr, st);
                else if (stage == 2) e = launch_match(ps[n], s, nullptr, s.shat, s.dst, s.keep, st);
                else e = launch_compact(ps[n], s, out_tokens[n], out_pos_thw[n], out_count[n], st);
            }
        }
        cudaEventRecord(ev[4], st);
        if (e == cudaSuccess) e = cudaEventSynchronize(ev[4]);
        for (int stage = 0; stage < 4 && e == cudaSuccess; ++stage) {
            float ms = 0.f;
            e = cudaEventElapsedTime(&ms, ev[stage], ev[stage + 1]);
            ms_per_launch[stage] += ms / (double)nclips / (double)reps;
        }
    }
    for (auto& x : ev) cudaEventDestroy(x);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_profile_read_floor(const void* const* buffers, int nbuffers, size_t bytes, int reps, double* ms_per_launch,
                           ttf_stream_t stream) {
    if (!buffers || nbuffers < 1 || bytes < 16 || bytes % 16 != 0 || reps < 1 || !ms_per_launch) return TTF_ERR_INVALID_ARG;
    for (int n = 0; n < nbuffers; ++n)
        if (!buffers[n] || reinterpret_cast<uintptr_t>(buffers[n]) % 16 != 0) return TTF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return cuda_fail(cudaGetLastError());
    cudaError_t e = cudaSuccess;
    for (int n = 0; n < nbuffers && e == cudaSuccess; ++n) e = launch_read_floor(buffers[n], bytes, nullptr, st);   // warm-up
    cudaEventRecord(e0, st);
    for (int rep = 0; rep < reps && e == cudaSuccess; ++rep)
        for (int n = 0; n < nbuffers && e == cudaSuccess; ++n) e = launch_read_floor(buffers[n], bytes, nullptr, st);
    cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    *ms_per_launch = (double)ms / ((double)reps * (double)nbuffers);
    return e == cudaSuccess ? TTF_OK : cuda_fail(e);
}

int ttf_release(void) {
    std::lock_guard<std::mutex> lk(g_mu);
    int cur = 0;
    cudaGetDevice(&cur);
    cudaError_t first = cudaSuccess;
    for (auto& kv : g_scratch) {
        cudaSetDevice(kv.first.first);
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess && first == cudaSuccess) first = e;
        if (kv.second.ptr) cudaFree(kv.second.ptr);
    }
    g_scratch.clear();
    for (auto& kv : g_staging) {
        cudaSetDevice(kv.first);
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess && first == cudaSuccess) first = e;
        Staging& s = kv.second;
        if (s.feat) cudaFree(s.feat);
        if (s.tok) cudaFree(s.tok);
        if (s.pos) cudaFree(s.pos);
        if (s.count) cudaFree(s.count);
        if (s.stream) cudaStreamDestroy(s.stream);
    }
    g_staging.clear();
    for (auto& kv : g_pipes) {
        cudaSetDevice(kv.first);
        HostPipe& hp = kv.second;
        cudaDeviceSynchronize();
        for (auto& sl : hp.slot) {
            if (sl.feat) cudaFree(sl.feat);
            if (sl.tok) cudaFree(sl.tok);
            if (sl.pos) cudaFree(sl.pos);
            if (sl.count) cudaFree(sl.count);
            if (sl.loaded) cudaEventDestroy(sl.loaded);
            if (sl.computed) cudaEventDestroy(sl.computed);
            if (sl.drained) cudaEventDestroy(sl.drained);
        }
        if (hp.count_host) cudaFreeHost(hp.count_host);
        if (hp.up) cudaStreamDestroy(hp.up);
        if (hp.run) cudaStreamDestroy(hp.run);
        if (hp.down) cudaStreamDestroy(hp.down);
    }
    g_pipes.clear();
    for (auto& kv : g_lanes) {
        cudaSetDevice(kv.first);
        BatchLanes& L = kv.second;
        for (int i = 0; i < kBatchStreams; ++i) {
            if (L.s[i]) { cudaStreamSynchronize(L.s[i]); cudaStreamDestroy(L.s[i]); }
            if (L.join[i]) cudaEventDestroy(L.join[i]);
        }
        if (L.fork) cudaEventDestroy(L.fork);
    }
    g_lanes.clear();
    cudaSetDevice(cur);
    return first == cudaSuccess ? TTF_OK : cuda_fail(first);
}

}  // extern "C"
