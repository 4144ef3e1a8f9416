// C ABI of libdynakv: context management, argument checks, and the call sequences that
// string the kernels together.  No arithmetic of the method lives here.
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"

using namespace dkv;

namespace dkv {
// tensor-core distance GEMM path (assign_tc.cu)
bool tc_assign_supported(const Tables& t, long long n, int M);
size_t tc_assign_scratch_bytes(const Tables& t, long long n, int M);
bool tc_assign_begin(const Tables& t, const void* K, long long n, int M, void* scratch, cudaStream_t s, long long* launches);
void launch_assign_tc(const Tables& t, const void* K, long long n, int M, const float* C, int* assign, void* scratch,
                      cudaStream_t s, long long* launches);
}  // namespace dkv

static thread_local char g_err[256] = "";

struct dynakv_ctx {
    dynakv_config cfg;
    cudaStream_t stream;
    Tables t;
    std::vector<void*> allocs;
    std::vector<void*> host_allocs;   // pinned host memory (the page pool of the two-tier mode)
    bool tier = false;
    TierState ts;
    bool built = false;
    long long n_prefill = 0;
    int M0 = 0;
    long long launches = 0;
    // build trace
    int* trace_assign = nullptr;   // [T][U][n]
    int* trace_picks = nullptr;    // [U][M0]
    // graph loop
    int* step_ctr = nullptr;          // device: step index of the captured loop
    int* step_lim = nullptr;          // device: number of steps of the loop in flight
    static constexpr int N_GRAPHS = 4;            // captured loops of 8, 4, 2 and 1 iterations
    cudaGraphExec_t graph_exec[N_GRAPHS] = {nullptr, nullptr, nullptr, nullptr};
    const void** loop_args = nullptr; // device: [4] q, k, v, out arrays of the loop in flight (read by the captured kernels)
    int g_budget = -1;
    long long graph_nodes = 0;        // kernel launches per captured iteration
    // staging for dynakv_step_host
    float* st_q = nullptr; void* st_k = nullptr; void* st_v = nullptr; float* st_out = nullptr;
    cudaStream_t copy_stream = nullptr;      // carries the result copy of a host step past the step's append / split
    cudaEvent_t ev_attended = nullptr;
    // the front half of a host step as one executable graph (per token budget): three copy-in nodes and the kernels up
    // to the attention output
    cudaGraphExec_t host_exec = nullptr;
    cudaGraph_t host_graph = nullptr;            // kept: its node handles name the copy nodes in later updates
    cudaGraphNode_t host_nodes[3] = {nullptr, nullptr, nullptr};    // copy nodes: q, k, v
    const void* host_ptrs[3] = {nullptr, nullptr, nullptr};         // the host addresses the nodes hold now
    int host_budget = -1;
    long long host_launches = 0;
    // dynakv_decode_loop_host: two sets of device staging arrays for chunks of steps, a stream for the copies in and
    // one for the copies out, and the events that order them against the loop
    static constexpr int HOST_CHUNK = 32;
    char* hl_q[2] = {nullptr, nullptr}; char* hl_k[2] = {nullptr, nullptr}; char* hl_v[2] = {nullptr, nullptr};
    char* hl_out[2] = {nullptr, nullptr};
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    // optional per-kernel event timing (off inside graph capture)
    bool timing = false;
    struct Span { int kc; cudaEvent_t e0, e1; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> event_pool;
    double kc_ms[KC_COUNT] = {0};
    long long kc_n[KC_COUNT] = {0};
};

// Scope that brackets one kernel launch with events when timing is on.
struct TimeScope {
    dynakv_ctx* c; bool on; dynakv_ctx::Span sp;
    TimeScope(dynakv_ctx* c_, int kc, bool allowed = true) : c(c_), on(c_->timing && allowed) {
        if (!on) return;
        sp.kc = kc;
        for (cudaEvent_t* e : {&sp.e0, &sp.e1}) {
            if (!c->event_pool.empty()) { *e = c->event_pool.back(); c->event_pool.pop_back(); }
            else cudaEventCreate(e);
        }
        cudaEventRecord(sp.e0, c->stream);
    }
    ~TimeScope() {
        if (!on) return;
        cudaEventRecord(sp.e1, c->stream);
        c->spans.push_back(sp);
    }
};

#define CK(call)                                                                                   \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess) {                                                                   \
            snprintf(g_err, sizeof(g_err), "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
            return DYNAKV_ERR_CUDA;                                                                \
        }                                                                                          \
    } while (0)

template <typename T>
static int dev_alloc(dynakv_ctx* c, T** p, size_t count, bool zero = false) {
    void* q = nullptr;
    size_t bytes = sizeof(T) * (count ? count : 1);
    cudaError_t e = cudaMalloc(&q, bytes);
    if (e != cudaSuccess) {
        snprintf(g_err, sizeof(g_err), "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
        cudaGetLastError();
        return DYNAKV_ERR_NOMEM;
    }
    c->allocs.push_back(q);
    if (zero) cudaMemsetAsync(q, 0, bytes, c->stream);
    *p = reinterpret_cast<T*>(q);
    return DYNAKV_OK;
}

#define ALLOC(ptr, count, zero)                                    \
    do {                                                           \
        int rc_ = dev_alloc(c, &(ptr), (size_t)(count), zero);     \
        if (rc_ != DYNAKV_OK) { dynakv_destroy(c); return rc_; }   \
    } while (0)

// inside build_index a failed allocation must not tear the caller's context down
#define ALLOC_B(ptr, count, zero)                                  \
    do {                                                           \
        int rc_ = dev_alloc(c, &(ptr), (size_t)(count), zero);     \
        if (rc_ != DYNAKV_OK) return rc_;                          \
    } while (0)

static size_t kv_bytes(const dynakv_config& cfg) { return cfg.kv_dtype == DYNAKV_F32 ? 4 : 2; }

extern "C" const char* dynakv_last_error(void) { return g_err; }

extern "C" int dynakv_create(const dynakv_config* cfg, void* cuda_stream, dynakv_ctx** out) {
    if (!cfg || !out) return DYNAKV_ERR_ARG;
    *out = nullptr;
    if (cfg->n_units < 1 || cfg->gqa_group < 1 || cfg->gqa_group > MAX_G) return DYNAKV_ERR_ARG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return DYNAKV_ERR_ARG;
    if (cfg->kv_dtype != DYNAKV_F32 && cfg->kv_dtype != DYNAKV_BF16 && cfg->kv_dtype != DYNAKV_FP8) return DYNAKV_ERR_ARG;
    if (cfg->kv_dtype == DYNAKV_FP8 && cfg->head_dim != 128) return DYNAKV_ERR_ARG;
    if (cfg->max_tokens < 1 || cfg->max_clusters < 1 || cfg->max_clusters > 4096) return DYNAKV_ERR_ARG;
    if (cfg->kmeans_iters < 1 || cfg->split_iters < 1) return DYNAKV_ERR_ARG;
    if (cfg->init_mode != DYNAKV_INIT_KMEANSPP && cfg->init_mode != DYNAKV_INIT_RANDOM) return DYNAKV_ERR_ARG;
    if (cfg->update_mode < DYNAKV_MODE_ADAPTIVE || cfg->update_mode > DYNAKV_MODE_DELAYED) return DYNAKV_ERR_ARG;
    if (cfg->update_mode == DYNAKV_MODE_DELAYED && cfg->buf_max < 1) return DYNAKV_ERR_ARG;
    if (cfg->update_mode == DYNAKV_MODE_LOCAL && cfg->local_max < 2) return DYNAKV_ERR_ARG;
    if (cfg->tier != 0 && cfg->tier != 1) return DYNAKV_ERR_ARG;
    if (cfg->tier && (cfg->cache_pages < 1 || cfg->cache_pages >= (1 << 20) || cfg->n_units > 65535)) return DYNAKV_ERR_ARG;
    dynakv_ctx* c = new (std::nothrow) dynakv_ctx();
    if (!c) return DYNAKV_ERR_NOMEM;
    c->cfg = *cfg;
    c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    Tables& t = c->t;
    memset(&t, 0, sizeof(t));
    t.U = cfg->n_units; t.G = cfg->gqa_group; t.d = cfg->head_dim;
    t.fp8 = cfg->kv_dtype == DYNAKV_FP8 ? 1 : 0;
    t.kv_dtype = t.fp8 ? DYNAKV_BF16 : cfg->kv_dtype;
    t.max_tokens = cfg->max_tokens; t.max_clusters = cfg->max_clusters;
    t.update_mode = cfg->update_mode; t.local_max = cfg->local_max;
    t.det_sums = cfg->det_sums ? 1 : 0;
    t.buf_max = cfg->buf_max;
    const int full_pages = (cfg->max_tokens + PAGE - 1) / PAGE;
    int slack = full_pages / 8; if (slack < 64) slack = 64;
    t.P = full_pages + cfg->max_clusters + slack;
    t.W = (PAGE / ENTRY_ROWS) * t.P;
    if (t.W >= (1 << 19)) {          // the selection packs a work-list position and a cluster count into one word
        snprintf(g_err, sizeof(g_err), "max_tokens too large: a unit's work list would have %d entries (limit %d)", t.W, (1 << 19) - 1);
        delete c;
        return DYNAKV_ERR_ARG;
    }
    t.n_splits_attn = 8;
    {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            snprintf(g_err, sizeof(g_err), "no usable CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
            delete c;
            return DYNAKV_ERR_CUDA;
        }
        t.n_attn_ctas = 2 * sms;
        t.attn_pf_in_smem = cfg->n_units <= 1024 ? 1 : 0;
    }
    const size_t U = t.U, P = t.P, Mx = t.max_clusters, d = t.d;
    const size_t page_elems = U * P * PAGE * d;
    if (t.fp8 && !cfg->tier) {
        ALLOC(t.k8, page_elems, false); ALLOC(t.v8, page_elems, false);
        ALLOC(t.k8e, U * P * PAGE, true); ALLOC(t.v8e, U * P * PAGE, true);
    }
    if (cfg->tier) {
        // two tiers: the page pool is pinned host memory the device reads and writes in place; device memory holds the
        // frame cache only
        c->tier = true;
        memset(&c->ts, 0, sizeof(c->ts));
        const size_t elem = t.fp8 ? 1 : kv_bytes(*cfg);
        void* pool[4] = {nullptr, nullptr, nullptr, nullptr};          // K rows, V rows; FP8: K and V scale exponents
        for (int i = 0; i < (t.fp8 ? 4 : 2); i++) {
            const size_t bytes = i < 2 ? page_elems * elem : U * P * PAGE;
            void* h = nullptr;
            cudaError_t e = cudaHostAlloc(&h, bytes, cudaHostAllocMapped | cudaHostAllocPortable);
            if (e == cudaSuccess) { c->host_allocs.push_back(h); e = cudaHostGetDevicePointer(&pool[i], h, 0); }
            if (e != cudaSuccess) {
                snprintf(g_err, sizeof(g_err), "pinned host allocation of %zu bytes for the page pool failed: %s", bytes, cudaGetErrorString(e));
                cudaGetLastError();
                dynakv_destroy(c);
                return DYNAKV_ERR_NOMEM;
            }
            if (i >= 2) memset(h, 0, bytes);
        }
        if (t.fp8) {
            t.k8 = (unsigned char*)pool[0]; t.v8 = (unsigned char*)pool[1]; t.k8e = (signed char*)pool[2]; t.v8e = (signed char*)pool[3];
            t.kpages = nullptr; t.vpages = nullptr;
        } else { t.kpages = pool[0]; t.vpages = pool[1]; }
        TierState& ts = c->ts;
        ts.Fc = cfg->cache_pages;
        const size_t Fc = ts.Fc;
        char *ka, *va;
        ALLOC(ka, U * Fc * PAGE * d * elem, true); ALLOC(va, U * Fc * PAGE * d * elem, true);
        ts.kcache = ka; ts.vcache = va;
        if (t.fp8) { ALLOC(ts.kecache, U * Fc * PAGE, true); ALLOC(ts.vecache, U * Fc * PAGE, true); }
        ALLOC(ts.cl_fr_head, U * Mx, false); ALLOC(ts.cl_fr_tail, U * Mx, false);
        ALLOC(ts.cl_snap, U * Mx * 4, true);
        ALLOC(ts.cl_lru, U * Mx, false);
        ALLOC(ts.page_frame, U * P, false);
        ALLOC(ts.frame_page, U * Fc, false); ALLOC(ts.frame_next, U * Fc, false);
        ALLOC(ts.fr_free, U * Fc, false); ALLOC(ts.fr_free_cnt, U, false);
        ALLOC(ts.miss_list, U * Mx, false);
        ALLOC(ts.jobs, U * (Fc + Mx), false); ALLOC(ts.n_jobs, U, false);
        ALLOC(ts.clock, U, false);
        ALLOC(ts.counters, TIER_COUNTERS, false);
        ALLOC(t.cl_ver, U * Mx, false);
        launch_tier_init(t, ts, c->stream, &c->launches);
    } else if (cfg->kv_dtype == DYNAKV_F32) {
        float *a, *b; ALLOC(a, page_elems, false); ALLOC(b, page_elems, false); t.kpages = a; t.vpages = b;
    } else if (t.fp8) {
        // FP8 storage: the rows live in their one-byte form only; whoever re-reads keys (the splits' 2-means, the exact
        // statistics, export) decodes them, which is exact
        t.kpages = nullptr; t.vpages = nullptr;
    } else {
        __nv_bfloat16 *a, *b; ALLOC(a, page_elems, false); ALLOC(b, page_elems, false); t.kpages = a; t.vpages = b;
    }
    ALLOC(t.page_tok, U * P * PAGE, false);
    ALLOC(t.page_next, U * P, false);
    ALLOC(t.free_stack, U * P, false);
    ALLOC(t.cl_r, U * Mx * d, true);
    ALLOC(t.cl_M2, U * Mx, true);
    ALLOC(t.cl_n, U * Mx, true);
    ALLOC(t.cl_head, U * Mx, true);
    ALLOC(t.cl_tail, U * Mx, true);
    ALLOC(t.cl_flags, U * Mx, true);
    ALLOC(t.cl_buf, U * Mx, true);
    ALLOC(t.u_N, U, true); ALLOC(t.u_M, U, true); ALLOC(t.u_Mlive, U, true); ALLOC(t.u_tau, U, true);
    ALLOC(t.u_page_top, U, true); ALLOC(t.u_free_cnt, U, true);
    ALLOC(t.tok_cluster, U * (size_t)t.max_tokens, false);
    ALLOC(t.scores, U * Mx, true);
    ALLOC(t.dists, U * Mx, true);
    ALLOC(t.u_scan, U, true); ALLOC(t.u_last, U, true);
    ALLOC(t.sel_ids, U * Mx, true);
    ALLOC(t.sel_n, U, true); ALLOC(t.sel_tokens, U, true);
    ALLOC(t.work, U * (size_t)t.W, false);
    ALLOC(t.n_work, U, true);
    {
        size_t recs = U * (size_t)t.n_splits_attn;
        if (recs < 2 * (size_t)t.n_attn_ctas) recs = 2 * (size_t)t.n_attn_ctas;
        ALLOC(t.part, recs * (t.G * (d + 2) + 16), false);
    }
    ALLOC(t.work_prefix, U + 1, true);
    ALLOC(t.unit_arrive, U, true);
    ALLOC(t.plan_counter, 2, true);
    ALLOC(t.tail_sync, 4, true);
    ALLOC(t.tail_queue, 2 * U, true);
    ALLOC(t.front_done, U, true);
    ALLOC(t.trig_n, U, true);
    ALLOC(t.trig_list, U * Mx, false);
    if (t.kv_dtype == DYNAKV_BF16 && attn_tma_prepare(t) != 0) {
        snprintf(g_err, sizeof(g_err), "cannot reserve shared memory for the gather-attention kernel: %s", cudaGetErrorString(cudaGetLastError()));
        dynakv_destroy(c);
        return DYNAKV_ERR_CUDA;
    }
    ALLOC(t.sp_label, U * (size_t)t.max_tokens, false);
    ALLOC(t.sp_pos, U * 2 * (size_t)t.max_tokens, false);
    ALLOC(t.status, 1, true);
    ALLOC(t.counters, 8, true);
    ALLOC(t.check_rec, 2, true);
    ALLOC(c->step_ctr, 1, true);
    ALLOC(c->step_lim, 1, true);
    ALLOC(c->loop_args, 4, true);
    ALLOC(c->st_q, U * t.G * d, false);
    ALLOC(c->st_out, U * t.G * d, false);
    {
        char *a, *b; ALLOC(a, U * d * kv_bytes(*cfg), false); ALLOC(b, U * d * kv_bytes(*cfg), false);
        c->st_k = a; c->st_v = b;
    }
    CK(cudaStreamSynchronize(c->stream));
    *out = c;
    return DYNAKV_OK;
}

extern "C" void dynakv_destroy(dynakv_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    if (c->copy_stream) { cudaStreamSynchronize(c->copy_stream); cudaStreamDestroy(c->copy_stream); }
    if (c->ev_attended) cudaEventDestroy(c->ev_attended);
    for (cudaStream_t s : {c->in_stream, c->out_stream}) if (s) { cudaStreamSynchronize(s); cudaStreamDestroy(s); }
    for (int i = 0; i < 2; i++) for (cudaEvent_t e : {c->ev_in[i], c->ev_done[i], c->ev_out[i]}) if (e) cudaEventDestroy(e);
    if (c->host_exec) cudaGraphExecDestroy(c->host_exec);
    if (c->host_graph) cudaGraphDestroy(c->host_graph);
    for (cudaGraphExec_t g : c->graph_exec) if (g) cudaGraphExecDestroy(g);
    for (auto& sp : c->spans) { cudaEventDestroy(sp.e0); cudaEventDestroy(sp.e1); }
    for (cudaEvent_t e : c->event_pool) cudaEventDestroy(e);
    for (void* p : c->allocs) cudaFree(p);
    for (void* p : c->host_allocs) cudaFreeHost(p);
    delete c;
}

static int build_index_impl(dynakv_ctx* c, const void* K, const void* V, int64_t n, int32_t d, int32_t n_clusters,
                            uint64_t seed, const float* q_ref, int64_t n_ref, int32_t ref_budget) {
    if (!c || !K || !V) return DYNAKV_ERR_ARG;
    if (c->built) return DYNAKV_ERR_STATE;
    Tables& t = c->t;
    if (d != t.d || n_clusters < 1 || n_clusters > t.max_clusters || n < n_clusters || n > t.max_tokens) return DYNAKV_ERR_ARG;
    const int M = n_clusters, T = c->cfg.kmeans_iters;
    const size_t U = t.U;
    BuildScratch b;
    memset(&b, 0, sizeof(b));
    const size_t mark = c->allocs.size();
    ALLOC_B(b.C, U * M * d, false);
    ALLOC_B(b.sums, U * M * d * (t.det_sums ? 2 : 1), false);      // 64-bit sums in the order-independent mode
    ALLOC_B(b.counts, U * M, false);
    ALLOC_B(b.cursor, U * M, false);
    ALLOC_B(b.picks, U * M, false);
    if (!t.det_sums) {
        ALLOC_B(b.upd_offset, U * M, false); ALLOC_B(b.upd_cursor, U * M, false); ALLOC_B(b.upd_order, U * (size_t)n, false);
    }
    if (c->cfg.init_mode == DYNAKV_INIT_KMEANSPP) ALLOC_B(b.D2, U * (size_t)n, false);
    int* assign_buf = nullptr;
    if (c->cfg.trace) { ALLOC_B(c->trace_assign, (size_t)T * U * n, false); }
    else ALLOC_B(assign_buf, U * (size_t)n, false);
    if (t.fp8) {
        // FP8 mode: the rows are rounded to the storage grid first; everything below works on the rounded copies
        __nv_bfloat16 *kq, *vq;
        ALLOC_B(kq, U * (size_t)n * d, false); ALLOC_B(vq, U * (size_t)n * d, false);
        launch_fp8_round_rows(K, kq, (long long)U * n, c->stream, &c->launches);
        launch_fp8_round_rows(V, vq, (long long)U * n, c->stream, &c->launches);
        K = kq; V = vq;
    }
    bool use_tc = c->cfg.assign_mode == 0 && tc_assign_supported(t, n, M);
    void* tc_scratch = nullptr;
    if (use_tc) { char* p; ALLOC_B(p, tc_assign_scratch_bytes(t, n, M), false); tc_scratch = p; }
    // fp16 copy of the keys; falls back to the fp32 kernel when a key is out of fp16 range
    if (use_tc) { TimeScope ts(c, KC_INIT); use_tc = tc_assign_begin(t, K, n, M, tc_scratch, c->stream, &c->launches); }

    { TimeScope ts(c, KC_INIT); launch_init_centres(t, K, n, M, seed, c->cfg.init_mode, b, c->stream, &c->launches); }
    for (int it = 0; it < T; it++) {
        b.assign = c->cfg.trace ? c->trace_assign + (size_t)it * U * n : assign_buf;
        {
            TimeScope ts(c, KC_ASSIGN);
            if (use_tc) launch_assign_tc(t, K, n, M, b.C, b.assign, tc_scratch, c->stream, &c->launches);
            else launch_assign_f32(t, K, n, M, b.C, b.assign, c->stream, &c->launches);
        }
        { TimeScope ts(c, KC_UPDATE); launch_update(t, K, n, M, b.assign, b, c->stream, &c->launches); }
    }
    { TimeScope ts(c, KC_FINALIZE); launch_finalize(t, K, V, n, M, b, c->cfg.split_var_factor, c->stream, &c->launches); }
    if (q_ref && n_ref > 0) {
        // Correlation-aware placement (Section 5.1): the reference queries are run through the scoring and the
        // selection on the index as it stands, every pair of clusters retrieved together is counted, a placement
        // order is derived from the counts, and the pages are laid out once more in that order.  Counters and status
        // word are put back afterwards: the reference queries are not decode steps.
        unsigned int* f = nullptr; int* order = nullptr;
        ALLOC_B(f, U * (size_t)M * M, true);
        ALLOC_B(order, U * M, false);
        unsigned long long cnt_save[8]; unsigned int st_save = 0;
        CK(cudaStreamSynchronize(c->stream));
        CK(cudaMemcpy(cnt_save, t.counters, sizeof(cnt_save), cudaMemcpyDeviceToHost));
        CK(cudaMemcpy(&st_save, t.status, sizeof(st_save), cudaMemcpyDeviceToHost));
        t.M_floor = M;
        const long long qs = (long long)t.U * t.G * t.d * 4;
        for (int64_t r = 0; r < n_ref; r++) {
            launch_front(t, StepPtr{(const char*)q_ref + r * qs, 0, nullptr}, StepPtr{nullptr, 0, nullptr}, 1, 0, c->stream, &c->launches);
            launch_select(t, ref_budget, nullptr, c->stream, &c->launches);
            launch_pair_count(t, M, f, c->stream, &c->launches);
        }
        launch_place_order(t, M, f, order, c->stream, &c->launches);
        { TimeScope ts(c, KC_FINALIZE); launch_finalize(t, K, V, n, M, b, c->cfg.split_var_factor, c->stream, &c->launches, order); }
        CK(cudaStreamSynchronize(c->stream));
        CK(cudaMemcpy(t.counters, cnt_save, sizeof(cnt_save), cudaMemcpyHostToDevice));
        CK(cudaMemcpy(t.status, &st_save, sizeof(st_save), cudaMemcpyHostToDevice));
    }
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    // keep the picks for the trace; free the rest of the build scratch
    if (c->cfg.trace) c->trace_picks = b.picks;
    std::vector<void*> keep;
    for (size_t i = mark; i < c->allocs.size(); i++) {
        void* p = c->allocs[i];
        if (c->cfg.trace && (p == (void*)c->trace_assign || p == (void*)b.picks)) keep.push_back(p);
        else cudaFree(p);
    }
    c->allocs.resize(mark);
    for (void* p : keep) c->allocs.push_back(p);
    c->built = true; c->n_prefill = n; c->M0 = M;
    t.M_floor = M;
    return DYNAKV_OK;
}

static void enqueue_front(dynakv_ctx* c, StepPtr q, StepPtr k, int has_q, int has_k, bool timed) {
    TimeScope ts(c, KC_FRONT, timed);
    launch_front(c->t, q, k, has_q, has_k, c->stream, &c->launches);
}

// gather attention -> combine, on work lists already written by a selection
static void enqueue_attend(dynakv_ctx* c, StepPtr q, StepPtrW out, bool timed);

// select -> gather attention -> combine, on scores already written by the front pass
static void enqueue_retrieve(dynakv_ctx* c, StepPtr q, int budget, StepPtrW out, int* sel_ids, bool timed) {
    { TimeScope ts(c, KC_SELECT, timed); launch_select(c->t, budget, sel_ids, c->stream, &c->launches); }
    // two tiers: bring the selected clusters into the frame cache and point the gather list at the frames
    if (c->tier) { TimeScope ts(c, KC_TIER, timed); launch_tier_resolve_fetch(c->t, c->ts, c->stream, &c->launches); }
    enqueue_attend(c, q, out, timed);
}

// The tables the attention kernels read rows through: the page pool, or in the two-tier mode the frame cache.
static Tables attn_tables(const dynakv_ctx* c) {
    Tables a = c->t;
    if (c->tier) {
        if (a.fp8) { a.k8 = (unsigned char*)c->ts.kcache; a.v8 = (unsigned char*)c->ts.vcache; a.k8e = c->ts.kecache; a.v8e = c->ts.vecache; }
        else { a.kpages = c->ts.kcache; a.vpages = c->ts.vcache; }
        a.P = c->ts.Fc;
    }
    return a;
}

static void enqueue_attend(dynakv_ctx* c, StepPtr q, StepPtrW out, bool timed) {
    const Tables at = attn_tables(c);
    if (c->t.kv_dtype == DYNAKV_BF16 && c->cfg.attn_mode == 0) {
        // gather, attend and combine in one persistent kernel
        TimeScope ts(c, KC_ATTN, timed);
        launch_gather_attn_tma(at, q, out, c->stream, &c->launches);
    } else {
        { TimeScope ts(c, KC_ATTN, timed); launch_gather_attn_v1(at, q, c->stream, &c->launches); }
        { TimeScope ts(c, KC_COMBINE, timed); launch_attn_combine(at, out, c->stream, &c->launches); }
    }
}

static void enqueue_append_apply(dynakv_ctx* c, StepPtr k, StepPtr v, bool timed) {
    TimeScope ts(c, KC_APPEND, timed);
    launch_append_apply(c->t, k, v, c->stream, &c->launches);
}

static const NextFront kNoNextFront = {0, StepPtr{nullptr, 0, nullptr}, StepPtr{nullptr, 0, nullptr}, nullptr};

// One iteration of a captured loop in three launches.  The centroid pass of step t + 1 is part of the tail kernel
// of step t (every unit's block runs it as soon as the unit's own append is done), so an iteration starts at the
// selection; the pass of step 0 is launched once ahead of the loop.  The tail kernel's last block advances the
// device-side step index that all kernels of the loop read.
static void enqueue_loop_iteration(dynakv_ctx* c, StepPtr q, StepPtr k, StepPtr v, int budget, StepPtrW out) {
    enqueue_retrieve(c, q, budget, out, nullptr, false);
    launch_append_split(c->t, c->cfg.split_size_factor, c->cfg.split_var_factor > 0.f ? 1 : 0, c->cfg.split_min_size,
                        c->cfg.split_iters, 1, k, v, c->step_ctr, NextFront{1, q, k, c->step_lim}, c->stream, &c->launches);
}


extern "C" int dynakv_build_index(dynakv_ctx* c, const void* K, const void* V, int64_t n, int32_t d,
                                  int32_t n_clusters, uint64_t seed) {
    return build_index_impl(c, K, V, n, d, n_clusters, seed, nullptr, 0, 0);
}

extern "C" int dynakv_build_index_placed(dynakv_ctx* c, const void* K, const void* V, int64_t n, int32_t d,
                                         int32_t n_clusters, uint64_t seed, const float* q_ref, int64_t n_ref,
                                         int32_t token_budget) {
    if (!q_ref || n_ref < 1 || token_budget < 0) return DYNAKV_ERR_ARG;
    return build_index_impl(c, K, V, n, d, n_clusters, seed, q_ref, n_ref, token_budget);
}

extern "C" int dynakv_decode_step(dynakv_ctx* c, const float* q, int32_t token_budget, float* out, int32_t* selected_ids) {
    if (!c || !q || !out || token_budget < 0) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    enqueue_front(c, StepPtr{q, 0, nullptr}, StepPtr{nullptr, 0, nullptr}, 1, 0, true);
    enqueue_retrieve(c, StepPtr{q, 0, nullptr}, token_budget, StepPtrW{out, 0, nullptr}, selected_ids, true);
    CK(cudaGetLastError());
    return DYNAKV_OK;
}

extern "C" int dynakv_append(dynakv_ctx* c, const void* k, const void* v) {
    if (!c || !k || !v) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    enqueue_front(c, StepPtr{nullptr, 0, nullptr}, StepPtr{k, 0, nullptr}, 0, 1, true);
    enqueue_append_apply(c, StepPtr{k, 0, nullptr}, StepPtr{v, 0, nullptr}, true);
    CK(cudaGetLastError());
    return DYNAKV_OK;
}

static void enqueue_split(dynakv_ctx* c, bool timed = true) {
    TimeScope ts(c, KC_SPLIT, timed);
    launch_split_check(c->t, c->cfg.split_size_factor, c->cfg.split_var_factor > 0.f ? 1 : 0, c->cfg.split_min_size,
                       c->cfg.split_iters, c->stream, &c->launches);
}

extern "C" int dynakv_split_check(dynakv_ctx* c) {
    if (!c) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    enqueue_split(c);
    CK(cudaGetLastError());
    return DYNAKV_OK;
}

extern "C" int dynakv_decode_loop(dynakv_ctx* c, const float* q_steps, const void* k_steps, const void* v_steps,
                                  int64_t n_steps, int32_t token_budget, float* out_steps) {
    if (!c || !q_steps || !k_steps || !v_steps || !out_steps || n_steps < 0 || n_steps > 0x7fffffff || token_budget < 0) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    if (c->stream == nullptr || c->stream == cudaStreamLegacy) {
        snprintf(g_err, sizeof(g_err), "dynakv_decode_loop captures a CUDA graph and needs a context created on a non-default stream");
        return DYNAKV_ERR_STATE;
    }
    const Tables& t = c->t;
    const long long qs = (long long)t.U * t.G * t.d * 4, ks = (long long)t.U * t.d * (long long)kv_bytes(c->cfg);
    // The loop is captured once per token budget as graphs of 8, 4, 2 and 1 iterations.  The captured kernels read
    // the caller's arrays through c->loop_args (stored by the pass that opens the loop), so the same graphs serve
    // every later call whatever arrays it passes.
    if (!c->graph_exec[0] || c->g_budget != token_budget) {
        for (cudaGraphExec_t& g : c->graph_exec) if (g) { cudaGraphExecDestroy(g); g = nullptr; }
        const StepPtr gq{nullptr, qs, c->step_ctr, c->loop_args + 0}, gk{nullptr, ks, c->step_ctr, c->loop_args + 1},
                      gv{nullptr, ks, c->step_ctr, c->loop_args + 2};
        const StepPtrW go{nullptr, qs, c->step_ctr, (void* const*)(c->loop_args + 3)};
        for (int which = 0; which < dynakv_ctx::N_GRAPHS; which++) {
            const int reps = 8 >> which;
            cudaGraph_t graph = nullptr;
            long long before = c->launches;
            CK(cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
            for (int r = 0; r < reps; r++) enqueue_loop_iteration(c, gq, gk, gv, token_budget, go);
            cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
            c->graph_nodes = (c->launches - before) / reps;
            c->launches = before;
            if (e == cudaSuccess && graph) {
                e = cudaGraphInstantiate(&c->graph_exec[which], graph, 0);
                cudaGraphDestroy(graph);
                // send the executable graph to the device now, not inside the first timed launch
                if (e == cudaSuccess) e = cudaGraphUpload(c->graph_exec[which], c->stream);
            }
            if (e != cudaSuccess) {
                for (cudaGraphExec_t& g : c->graph_exec) if (g) { cudaGraphExecDestroy(g); g = nullptr; }
                snprintf(g_err, sizeof(g_err), "graph capture / instantiate failed: %s", cudaGetErrorString(e));
                cudaGetLastError();
                return DYNAKV_ERR_CUDA;
            }
        }
        c->g_budget = token_budget;
    }
    if (n_steps == 0) return DYNAKV_OK;
    {
        // step 0's centroid pass opens the loop (step index, hand-over words, the caller's arrays); every later
        // pass rides in the tail kernel of the step before it
        LoopBegin lb;
        lb.on = 1; lb.step_ctr = c->step_ctr; lb.step_lim = c->step_lim; lb.n_steps = (int)n_steps; lb.args = c->loop_args;
        lb.q = q_steps; lb.k = k_steps; lb.v = v_steps; lb.out = out_steps;
        launch_front(c->t, StepPtr{q_steps, qs, nullptr}, StepPtr{k_steps, ks, nullptr}, 1, 1, c->stream, &c->launches, &lb);
    }
    int64_t left = n_steps;
    for (int which = 0; which < dynakv_ctx::N_GRAPHS; which++) {
        const int reps = 8 >> which;
        for (; left >= reps; left -= reps) CK(cudaGraphLaunch(c->graph_exec[which], c->stream));
    }
    c->launches += c->graph_nodes * n_steps;
    return DYNAKV_OK;
}

extern "C" int dynakv_step_host(dynakv_ctx* c, const float* q_host, const void* k_host, const void* v_host,
                                int32_t token_budget, float* out_host) {
    if (!c || !q_host || !k_host || !v_host || !out_host || token_budget < 0) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    const Tables& t = c->t;
    const size_t qb = (size_t)t.U * t.G * t.d * 4, kb = (size_t)t.U * t.d * kv_bytes(c->cfg);
    // The result depends on the attention kernel only: its copy back runs on a second stream beside the step's
    // append and split check, and the call returns when the result is on the host.  Whatever is called next on
    // the context is ordered behind the append and split check by the context's stream.
    if (!c->copy_stream) {
        CK(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
        CK(cudaEventCreateWithFlags(&c->ev_attended, cudaEventDisableTiming));
    }
    const StepPtr q{c->st_q, 0, nullptr}, k{c->st_k, 0, nullptr}, v{c->st_v, 0, nullptr};
    const bool can_graph = !c->timing && c->stream != nullptr && c->stream != cudaStreamLegacy;
    if (can_graph) {
        // ---- the three copies in and the kernels up to the attention output as ONE graph launch.  Captured once per
        // budget; a later call with other host arrays only rewrites the copy nodes' addresses.
        const void* now[3] = {q_host, k_host, v_host};
        if (!c->host_exec || c->host_budget != token_budget) {
            if (c->host_exec) { cudaGraphExecDestroy(c->host_exec); c->host_exec = nullptr; }
            if (c->host_graph) { cudaGraphDestroy(c->host_graph); c->host_graph = nullptr; }
            cudaGraph_t graph = nullptr;
            const long long before = c->launches;
            CK(cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
            cudaMemcpyAsync(c->st_q, q_host, qb, cudaMemcpyHostToDevice, c->stream);
            cudaMemcpyAsync(c->st_k, k_host, kb, cudaMemcpyHostToDevice, c->stream);
            cudaMemcpyAsync(c->st_v, v_host, kb, cudaMemcpyHostToDevice, c->stream);
            enqueue_front(c, q, k, 1, 1, false);
            enqueue_retrieve(c, q, token_budget, StepPtrW{c->st_out, 0, nullptr}, nullptr, false);
            cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
            c->host_launches = c->launches - before;
            c->launches = before;
            if (e == cudaSuccess && graph) e = cudaGraphInstantiate(&c->host_exec, graph, 0);
            if (e == cudaSuccess) {
                // find the three copy nodes by the device staging buffer they write
                size_t nn = 0;
                cudaGraphGetNodes(graph, nullptr, &nn);
                std::vector<cudaGraphNode_t> nodes(nn);
                cudaGraphGetNodes(graph, nodes.data(), &nn);
                for (int i = 0; i < 3; i++) c->host_nodes[i] = nullptr;
                for (cudaGraphNode_t nd : nodes) {
                    cudaGraphNodeType ty;
                    if (cudaGraphNodeGetType(nd, &ty) != cudaSuccess || ty != cudaGraphNodeTypeMemcpy) continue;
                    cudaMemcpy3DParms mp;
                    if (cudaGraphMemcpyNodeGetParams(nd, &mp) != cudaSuccess) continue;
                    if (mp.dstPtr.ptr == (void*)c->st_q) c->host_nodes[0] = nd;
                    else if (mp.dstPtr.ptr == c->st_k) c->host_nodes[1] = nd;
                    else if (mp.dstPtr.ptr == c->st_v) c->host_nodes[2] = nd;
                }
                if (!c->host_nodes[0] || !c->host_nodes[1] || !c->host_nodes[2]) e = cudaErrorUnknown;
            }
            if (e != cudaSuccess) {
                if (graph) cudaGraphDestroy(graph);
                if (c->host_exec) { cudaGraphExecDestroy(c->host_exec); c->host_exec = nullptr; }
                snprintf(g_err, sizeof(g_err), "host-step graph capture / instantiate failed: %s", cudaGetErrorString(e));
                cudaGetLastError();
                return DYNAKV_ERR_CUDA;
            }
            c->host_graph = graph;
            cudaGraphUpload(c->host_exec, c->stream);
            c->host_budget = token_budget;
            for (int i = 0; i < 3; i++) c->host_ptrs[i] = now[i];
        }
        const size_t bytes[3] = {qb, kb, kb};
        void* const dev[3] = {c->st_q, c->st_k, c->st_v};
        for (int i = 0; i < 3; i++) {
            if (c->host_ptrs[i] == now[i]) continue;
            CK(cudaGraphExecMemcpyNodeSetParams1D(c->host_exec, c->host_nodes[i], dev[i], now[i], bytes[i], cudaMemcpyHostToDevice));
            c->host_ptrs[i] = now[i];
        }
        CK(cudaGraphLaunch(c->host_exec, c->stream));
        c->launches += c->host_launches;
    } else {
        CK(cudaMemcpyAsync(c->st_q, q_host, qb, cudaMemcpyHostToDevice, c->stream));
        CK(cudaMemcpyAsync(c->st_k, k_host, kb, cudaMemcpyHostToDevice, c->stream));
        CK(cudaMemcpyAsync(c->st_v, v_host, kb, cudaMemcpyHostToDevice, c->stream));
        enqueue_front(c, q, k, 1, 1, true);
        enqueue_retrieve(c, q, token_budget, StepPtrW{c->st_out, 0, nullptr}, nullptr, true);
    }
    CK(cudaEventRecord(c->ev_attended, c->stream));
    CK(cudaStreamWaitEvent(c->copy_stream, c->ev_attended, 0));
    CK(cudaMemcpyAsync(out_host, c->st_out, qb, cudaMemcpyDeviceToHost, c->copy_stream));
    {
        TimeScope ts(c, KC_SPLIT, true);
        launch_append_split(c->t, c->cfg.split_size_factor, c->cfg.split_var_factor > 0.f ? 1 : 0, c->cfg.split_min_size,
                            c->cfg.split_iters, 1, k, v, nullptr, kNoNextFront, c->stream, &c->launches);
    }
    CK(cudaStreamSynchronize(c->copy_stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_decode_loop_host(dynakv_ctx* c, const float* q_host, const void* k_host, const void* v_host,
                                       int64_t n_steps, int32_t token_budget, float* out_host) {
    if (!c || !q_host || !k_host || !v_host || !out_host || n_steps < 0 || token_budget < 0) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    const Tables& t = c->t;
    const size_t qs = (size_t)t.U * t.G * t.d * 4, ks = (size_t)t.U * t.d * kv_bytes(c->cfg);
    constexpr int CH = dynakv_ctx::HOST_CHUNK;
    if (!c->in_stream) {
        // first call: staging arrays (kept until destroy), streams, events
        for (int b = 0; b < 2; b++) {
            ALLOC_B(c->hl_q[b], CH * qs, false); ALLOC_B(c->hl_k[b], CH * ks, false); ALLOC_B(c->hl_v[b], CH * ks, false);
            ALLOC_B(c->hl_out[b], CH * qs, false);
        }
        CK(cudaStreamCreateWithFlags(&c->in_stream, cudaStreamNonBlocking));
        CK(cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; b++)
            for (cudaEvent_t* e : {&c->ev_in[b], &c->ev_done[b], &c->ev_out[b]}) CK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
    }
    // Chunks of up to CH steps: chunk i + 1 is copied in and chunk i - 1 copied out while the loop runs chunk i.
    // The first chunk's copy in and the last chunk's copy out have nothing to hide behind, so the chunks start at
    // 4 steps and double up to CH, and halve again towards the end of the call.
    // whatever ran on the context's stream before must be complete before its inputs are overwritten
    CK(cudaEventRecord(c->ev_done[0], c->stream)); CK(cudaEventRecord(c->ev_done[1], c->stream));
    CK(cudaEventRecord(c->ev_out[0], c->out_stream)); CK(cudaEventRecord(c->ev_out[1], c->out_stream));
    int64_t s0 = 0;
    for (int64_t i = 0; s0 < n_steps; i++) {
        const int b = (int)(i & 1);
        const int64_t left = n_steps - s0;
        int64_t nb = i < 3 ? (int64_t)4 << i : CH;
        if (nb > CH) nb = CH;
        if (nb > (left + 1) / 2) nb = (left + 1) / 2 > 4 ? (left + 1) / 2 : 4;
        if (nb > left) nb = left;
        // copy in: the staging set is free once the loop over the chunk that used it before has finished
        CK(cudaStreamWaitEvent(c->in_stream, c->ev_done[b], 0));
        CK(cudaMemcpyAsync(c->hl_q[b], (const char*)q_host + s0 * qs, nb * qs, cudaMemcpyHostToDevice, c->in_stream));
        CK(cudaMemcpyAsync(c->hl_k[b], (const char*)k_host + s0 * ks, nb * ks, cudaMemcpyHostToDevice, c->in_stream));
        CK(cudaMemcpyAsync(c->hl_v[b], (const char*)v_host + s0 * ks, nb * ks, cudaMemcpyHostToDevice, c->in_stream));
        CK(cudaEventRecord(c->ev_in[b], c->in_stream));
        // the loop: needs the chunk's inputs, and its output set copied out (two chunks ago)
        CK(cudaStreamWaitEvent(c->stream, c->ev_in[b], 0));
        CK(cudaStreamWaitEvent(c->stream, c->ev_out[b], 0));
        int rc = dynakv_decode_loop(c, (const float*)c->hl_q[b], c->hl_k[b], c->hl_v[b], nb, token_budget, (float*)c->hl_out[b]);
        if (rc != DYNAKV_OK) return rc;
        CK(cudaEventRecord(c->ev_done[b], c->stream));
        // copy out
        CK(cudaStreamWaitEvent(c->out_stream, c->ev_done[b], 0));
        CK(cudaMemcpyAsync((char*)out_host + s0 * qs, c->hl_out[b], nb * qs, cudaMemcpyDeviceToHost, c->out_stream));
        CK(cudaEventRecord(c->ev_out[b], c->out_stream));
        s0 += nb;
    }
    CK(cudaStreamSynchronize(c->out_stream));
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

__global__ void k_sum_status(Tables t, long long* out) {
    // out[0] tokens selected, out[1] clusters selected, out[2] pages in use
    long long a = 0, b = 0, p = 0;
    for (int u = threadIdx.x; u < t.U; u += blockDim.x) {
        a += t.sel_tokens[u]; b += t.sel_n[u]; p += t.u_page_top[u] - t.u_free_cnt[u];
    }
    atomicAdd((unsigned long long*)&out[0], (unsigned long long)a);
    atomicAdd((unsigned long long*)&out[1], (unsigned long long)b);
    atomicAdd((unsigned long long*)&out[2], (unsigned long long)p);
}

extern "C" int dynakv_get_status(dynakv_ctx* c, dynakv_status* host_out) {
    if (!c || !host_out) return DYNAKV_ERR_ARG;
    memset(host_out, 0, sizeof(*host_out));
    unsigned long long cnt[8];
    CK(cudaMemsetAsync(c->t.counters + 4, 0, 3 * sizeof(unsigned long long), c->stream));
    if (c->built) { k_sum_status<<<1, 256, 0, c->stream>>>(c->t, (long long*)(c->t.counters + 4)); c->launches++; }
    CK(cudaMemcpyAsync(&host_out->error_bits, c->t.status, sizeof(unsigned int), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(cnt, c->t.counters, sizeof(cnt), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(&host_out->bounds_site, c->t.check_rec, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    host_out->n_appended = (int64_t)cnt[CNT_APPENDED];
    host_out->n_splits = (int64_t)cnt[CNT_SPLITS];
    host_out->assign_rechecked = (int64_t)cnt[CNT_RECHECKED];
    host_out->tokens_attended_total = (int64_t)cnt[CNT_TOKENS_ATTENDED];
    host_out->clusters_selected_total = (int64_t)cnt[CNT_CLUSTERS_SELECTED];
    host_out->tokens_selected = (int64_t)cnt[4];
    host_out->clusters_selected = (int64_t)cnt[5];
    host_out->pages_in_use = (int64_t)cnt[6];
    return DYNAKV_OK;
}

extern "C" int dynakv_export_state(dynakv_ctx* c, int32_t* tok_cluster, float* centroids, int32_t* counts, float* M2,
                                   int32_t* n_tokens, int32_t* n_ids, float* tau) {
    if (!c) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    const Tables& t = c->t;
    const size_t U = t.U, Mx = t.max_clusters;
    cudaStream_t s = c->stream;
    if (tok_cluster) CK(cudaMemcpyAsync(tok_cluster, t.tok_cluster, sizeof(int) * U * t.max_tokens, cudaMemcpyDeviceToHost, s));
    if (centroids) CK(cudaMemcpyAsync(centroids, t.cl_r, sizeof(float) * U * Mx * t.d, cudaMemcpyDeviceToHost, s));
    if (counts) CK(cudaMemcpyAsync(counts, t.cl_n, sizeof(int) * U * Mx, cudaMemcpyDeviceToHost, s));
    if (M2) CK(cudaMemcpyAsync(M2, t.cl_M2, sizeof(float) * U * Mx, cudaMemcpyDeviceToHost, s));
    if (n_tokens) CK(cudaMemcpyAsync(n_tokens, t.u_N, sizeof(int) * U, cudaMemcpyDeviceToHost, s));
    if (n_ids) CK(cudaMemcpyAsync(n_ids, t.u_M, sizeof(int) * U, cudaMemcpyDeviceToHost, s));
    if (tau) CK(cudaMemcpyAsync(tau, t.u_tau, sizeof(float) * U, cudaMemcpyDeviceToHost, s));
    CK(cudaStreamSynchronize(s));
    return DYNAKV_OK;
}

extern "C" int dynakv_export_kv(dynakv_ctx* c, void* K_out, void* V_out, int64_t n) {
    if (!c || !K_out || !V_out || n < 1 || n > c->t.max_tokens) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    launch_export_rows(c->t, K_out, V_out, n, c->stream, &c->launches);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_import_state(dynakv_ctx* c, const void* K, const void* V, int64_t n, const int32_t* tok_cluster,
                                   const int32_t* n_ids, const float* tau, int32_t n_build_clusters) {
    if (!c || !K || !V || !tok_cluster || !n_ids || !tau) return DYNAKV_ERR_ARG;
    if (c->built) return DYNAKV_ERR_STATE;
    Tables& t = c->t;
    if (n < 1 || n > t.max_tokens || n_build_clusters < 1 || n_build_clusters > t.max_clusters) return DYNAKV_ERR_ARG;
    const size_t U = t.U;
    int M = 0, Mmin = t.max_clusters;
    for (size_t u = 0; u < U; u++) {
        if (n_ids[u] < 1 || n_ids[u] > t.max_clusters) return DYNAKV_ERR_ARG;
        M = n_ids[u] > M ? n_ids[u] : M;
        Mmin = n_ids[u] < Mmin ? n_ids[u] : Mmin;
    }
    if (n_build_clusters > Mmin) return DYNAKV_ERR_ARG;
    const int d = t.d;
    BuildScratch b;
    memset(&b, 0, sizeof(b));
    const size_t mark = c->allocs.size();
    int* ids_dev = nullptr; float* tau_dev = nullptr;
    ALLOC_B(b.C, U * M * d, true);
    ALLOC_B(b.sums, U * M * d * (t.det_sums ? 2 : 1), false);      // 64-bit sums in the order-independent mode
    ALLOC_B(b.counts, U * M, false);
    ALLOC_B(b.cursor, U * M, false);
    ALLOC_B(ids_dev, U, false);
    ALLOC_B(tau_dev, U, false);
    b.assign = const_cast<int*>(tok_cluster);
    if (t.fp8) {
        __nv_bfloat16 *kq, *vq;
        ALLOC_B(kq, U * (size_t)n * d, false); ALLOC_B(vq, U * (size_t)n * d, false);
        launch_fp8_round_rows(K, kq, (long long)U * n, c->stream, &c->launches);
        launch_fp8_round_rows(V, vq, (long long)U * n, c->stream, &c->launches);
        K = kq; V = vq;
    }
    CK(cudaMemcpyAsync(ids_dev, n_ids, sizeof(int) * U, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(tau_dev, tau, sizeof(float) * U, cudaMemcpyHostToDevice, c->stream));
    // representatives = member means (Eq. 4), then the layout and the exact statistics, as at the end of a build
    launch_update(t, K, n, M, b.assign, b, c->stream, &c->launches);
    launch_finalize(t, K, V, n, M, b, c->cfg.split_var_factor, c->stream, &c->launches);
    launch_import_units(t, ids_dev, tau_dev, c->stream, &c->launches);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    for (size_t i = mark; i < c->allocs.size(); i++) cudaFree(c->allocs[i]);
    c->allocs.resize(mark);
    c->built = true; c->n_prefill = n; c->M0 = n_build_clusters;
    t.M_floor = n_build_clusters;
    return DYNAKV_OK;
}

extern "C" int dynakv_get_selection(dynakv_ctx* c, int32_t* n_selected, int32_t* tokens_selected) {
    if (!c) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    if (n_selected) CK(cudaMemcpyAsync(n_selected, c->t.sel_n, sizeof(int) * c->t.U, cudaMemcpyDeviceToHost, c->stream));
    if (tokens_selected) CK(cudaMemcpyAsync(tokens_selected, c->t.sel_tokens, sizeof(int) * c->t.U, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_get_work_list(dynakv_ctx* c, int32_t* n_entries, int32_t* entries, int64_t entries_per_unit) {
    if (!c || !n_entries) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    const Tables& t = c->t;
    if (entries && entries_per_unit < t.W) return DYNAKV_ERR_ARG;
    CK(cudaMemcpyAsync(n_entries, t.n_work, sizeof(int) * t.U, cudaMemcpyDeviceToHost, c->stream));
    if (entries)
        CK(cudaMemcpy2DAsync(entries, (size_t)entries_per_unit * 8, t.work, (size_t)t.W * 8, (size_t)t.W * 8, t.U,
                             cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_get_tier_stats(dynakv_ctx* c, dynakv_tier_stats* out) {
    if (!c || !out) return DYNAKV_ERR_ARG;
    if (!c->tier) return DYNAKV_ERR_STATE;
    unsigned long long cnt[TIER_COUNTERS];
    std::vector<int> free_cnt(c->t.U);
    CK(cudaMemcpyAsync(cnt, c->ts.counters, sizeof(cnt), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(free_cnt.data(), c->ts.fr_free_cnt, sizeof(int) * c->t.U, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    out->pages_fetched = (int64_t)cnt[TIER_PAGES_FETCHED];
    out->clusters_hit = (int64_t)cnt[TIER_HITS];
    out->clusters_fetched = (int64_t)cnt[TIER_FETCHED];
    out->clusters_refreshed = (int64_t)cnt[TIER_REFRESHED];
    out->clusters_evicted = (int64_t)cnt[TIER_EVICTED];
    out->copies_dropped_stale = (int64_t)cnt[TIER_STALE];
    out->rows_fetched = (int64_t)cnt[TIER_ROWS];
    out->frames_total = (int64_t)c->t.U * c->ts.Fc;
    out->frames_in_use = out->frames_total;
    for (int f : free_cnt) out->frames_in_use -= f;
    return DYNAKV_OK;
}

extern "C" int dynakv_work_list_capacity(dynakv_ctx* c) { return c ? c->t.W : DYNAKV_ERR_ARG; }

extern "C" int dynakv_get_build_trace(dynakv_ctx* c, int32_t* picks, int32_t* assign) {
    if (!c) return DYNAKV_ERR_ARG;
    if (!c->built || !c->cfg.trace) return DYNAKV_ERR_STATE;
    const size_t U = c->t.U;
    if (picks) CK(cudaMemcpyAsync(picks, c->trace_picks, sizeof(int) * U * c->M0, cudaMemcpyDeviceToHost, c->stream));
    if (assign) CK(cudaMemcpyAsync(assign, c->trace_assign, sizeof(int) * (size_t)c->cfg.kmeans_iters * U * c->n_prefill,
                                   cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_selftest_wait_expiry(dynakv_ctx* c, int32_t* gave_up) {
    if (!c || !gave_up) return DYNAKV_ERR_ARG;
    int* flag = reinterpret_cast<int*>(c->t.plan_counter);      // a scratch word that is zero between calls
    launch_selftest_wait_expiry(c->t, flag, c->stream, &c->launches);
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(gave_up, flag, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemsetAsync(flag, 0, sizeof(int), c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return DYNAKV_OK;
}

extern "C" int dynakv_time_gather_attention(dynakv_ctx* c, const float* q, float* out, int32_t reps, float* ms_per_launch) {
    if (!c || !q || !out || !ms_per_launch || reps < 1) return DYNAKV_ERR_ARG;
    if (!c->built) return DYNAKV_ERR_STATE;
    if (c->t.kv_dtype != DYNAKV_BF16 || c->cfg.attn_mode != 0) return DYNAKV_ERR_ARG;
    cudaEvent_t e0, e1;
    CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1));
    const StepPtr qp{q, 0, nullptr};
    const StepPtrW op{out, 0, nullptr};
    const Tables at = attn_tables(c);
    launch_gather_attn_plain(at, qp, op, c->stream, &c->launches);       // one untimed launch first
    CK(cudaEventRecord(e0, c->stream));
    for (int i = 0; i < reps; i++) launch_gather_attn_plain(at, qp, op, c->stream, &c->launches);
    CK(cudaEventRecord(e1, c->stream));
    CK(cudaGetLastError());
    CK(cudaEventSynchronize(e1));
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, e0, e1));
    *ms_per_launch = ms / (float)reps;
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    return DYNAKV_OK;
}

extern "C" int dynakv_set_timing(dynakv_ctx* c, int32_t on) {
    if (!c) return DYNAKV_ERR_ARG;
    c->timing = on != 0;
    return DYNAKV_OK;
}

extern "C" int dynakv_get_kernel_times(dynakv_ctx* c, double* ms_total, int64_t* launches, int32_t reset) {
    if (!c || !ms_total || !launches) return DYNAKV_ERR_ARG;
    CK(cudaStreamSynchronize(c->stream));
    for (auto& sp : c->spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.e0, sp.e1) == cudaSuccess) { c->kc_ms[sp.kc] += ms; c->kc_n[sp.kc]++; }
        c->event_pool.push_back(sp.e0); c->event_pool.push_back(sp.e1);
    }
    c->spans.clear();
    for (int k = 0; k < KC_COUNT; k++) {
        ms_total[k] = c->kc_ms[k]; launches[k] = c->kc_n[k];
        if (reset) { c->kc_ms[k] = 0; c->kc_n[k] = 0; }
    }
    return DYNAKV_OK;
}

extern "C" int64_t dynakv_launch_count(dynakv_ctx* c) { return c ? c->launches : 0; }

extern "C" int dynakv_checked_build(void) {
#ifdef DYNAKV_CHECKED
    return 1;
#else
    return 0;
#endif
}
