// Host side of the C ABI declared in sirllm.h: argument checks, workspace layout and
// the launch sequences.  No device memory is allocated here.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace sirllm {

static thread_local char g_cuda_msg[256] = "";

int cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_cuda_msg, sizeof g_cuda_msg, "%s: %s", where, cudaGetErrorString(e));
    return SIRLLM_ERR_CUDA;
}

cudaError_t device_props(DeviceProps* out) {
    static DeviceProps cache[kMaxDevices];
    static std::atomic<int> known[kMaxDevices];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices && known[dev].load(std::memory_order_acquire)) {
        *out = cache[dev];
        return cudaSuccess;
    }
    DeviceProps dp;
    dp.device = dev;
    e = cudaDeviceGetAttribute(&dp.n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&dp.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) {  // several threads may fill the slot: they write the same values
        cache[dev] = dp;
        known[dev].store(1, std::memory_order_release);
    }
    *out = dp;
    return cudaSuccess;
}

cudaError_t allow_max_dynamic_smem(const void* kernel, const DeviceProps& dp, unsigned char* done) {
    const bool cached = dp.device >= 0 && dp.device < kMaxDevices;
    if (cached && __atomic_load_n(&done[dp.device], __ATOMIC_ACQUIRE)) return cudaSuccess;
    cudaFuncAttributes fa;
    cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
    if (e != cudaSuccess) return e;
    // static and dynamic shared memory together may reach the opt-in limit
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             dp.smem_optin - (int)fa.sharedSizeBytes);
    if (e == cudaSuccess && cached) __atomic_store_n(&done[dp.device], (unsigned char)1, __ATOMIC_RELEASE);
    return e;
}

int validate_config(const sirllm_config* c) {
    if (c == nullptr) return SIRLLM_ERR_NULL;
    if (c->n_streams < 1 || c->n_layers < 1 || c->n_kv_heads < 1 || c->head_dim < 1)
        return SIRLLM_ERR_BAD_CONFIG;
    if (c->capacity < 1 || c->capacity > SIRLLM_MAX_CAPACITY) return SIRLLM_ERR_BAD_CONFIG;
    if (c->n_sink < 0 || c->n_recent < 0 || c->budget < c->n_sink + c->n_recent)
        return SIRLLM_ERR_BAD_CONFIG;
    if (c->budget < 1 || c->threshold < c->budget || c->capacity < c->threshold)
        return SIRLLM_ERR_BAD_CONFIG;
    if (c->max_new < 0 || c->max_new > c->capacity) return SIRLLM_ERR_BAD_CONFIG;
    if (c->kv_dtype != SIRLLM_BF16 && c->kv_dtype != SIRLLM_F16) return SIRLLM_ERR_BAD_CONFIG;
    if (c->logits_dtype != SIRLLM_F32 && c->logits_dtype != SIRLLM_BF16)
        return SIRLLM_ERR_BAD_CONFIG;
    if (c->vocab < 1 || c->vocab > 0x7FFFFFFF || c->logits_row_stride < c->vocab)
        return SIRLLM_ERR_BAD_CONFIG;
    if ((int64_t)c->head_dim * 2 % 16 != 0 || c->head_dim > SIRLLM_MAX_HEAD_DIM)
        return SIRLLM_ERR_BAD_CONFIG;
    if ((int64_t)c->n_streams * c->n_layers * c->n_kv_heads > 0x3FFFFFFF)
        return SIRLLM_ERR_BAD_CONFIG;
    return SIRLLM_OK;
}

WorkspaceLayout workspace_layout(const sirllm_config& c) {
    WorkspaceLayout L;
    const int64_t epv = 16 / logits_elem_bytes(c.logits_dtype);
    const int64_t nvec = c.vocab / epv;
    const int64_t per_cta = kScoreCtaVecs;
    L.n_part = (int32_t)((nvec + per_cta - 1) / per_cta);
    if (L.n_part < 1) L.n_part = 1;
    size_t off = 256;
    L.plane_progress_off = off;
    {
        const size_t planes = (size_t)2 * c.n_streams * c.n_layers * c.n_kv_heads;
        const size_t chained = planes < (size_t)kChainPlanesMax ? planes : (size_t)kChainPlanesMax;
        off = align_up(off + chained * kMaxSplit * sizeof(unsigned long long), 256);
    }
    L.first_moved_off = off;
    off = align_up(off + (size_t)c.n_streams * 4, 256);
    L.ready_off = off;
    off = align_up(off + (size_t)c.n_streams * 4, 256);
    L.n_keep_off = off;
    off = align_up(off + (size_t)c.n_streams * 4, 256);
    L.keep_off = off;
    off = align_up(off + (size_t)c.n_streams * c.threshold * 4, 256);
    L.tickets_off = off;
    off = align_up(off + (size_t)c.n_streams * c.max_new * 4, 256);
    L.policy_ranks_off = off;
    off = align_up(off + (size_t)c.n_streams * c.capacity * 4, 256);
    L.policy_ones_off = off;
    off = align_up(off + (size_t)c.n_streams * 4, 256);
    L.partials_off = off;
    off = align_up(off + (size_t)c.n_streams * c.max_new * L.n_part * sizeof(float2), 256);
    L.total = off;
    return L;
}

static bool misaligned(const void* p, size_t a) { return ((uintptr_t)p % a) != 0; }

static ScoreParams score_params(const sirllm_config& c, const WorkspaceLayout& L, const void* logits,
                                const int32_t* ids, const int32_t* n_new, void* ws) {
    ScoreParams sp;
    sp.logits = logits;
    sp.token_ids = ids;
    sp.n_new = n_new;
    sp.partials = (float2*)((char*)ws + L.partials_off);
    sp.tickets = (int32_t*)((char*)ws + L.tickets_off);
    sp.status = (int32_t*)ws;
    sp.out_entropy = nullptr;
    sp.scores = nullptr;
    sp.live_len = nullptr;
    sp.pairs_out = nullptr;
    sp.target_out = nullptr;
    sp.pair_stride = 0;
    sp.col0 = 0;
    sp.capacity = c.capacity;
    sp.vocab = c.vocab;
    sp.row_stride = c.logits_row_stride;
    sp.n_streams = c.n_streams;
    sp.max_new = c.max_new;
    sp.n_part = L.n_part;
    sp.logits_dtype = c.logits_dtype;
    return sp;
}

static int check_logits(const sirllm_config& c, const void* logits) {
    if (misaligned(logits, logits_elem_bytes(c.logits_dtype))) return SIRLLM_ERR_ALIGN;
    return SIRLLM_OK;
}

}  // namespace sirllm

using namespace sirllm;

extern "C" {

size_t sirllm_workspace_bytes(const sirllm_config* cfg) {
    if (validate_config(cfg) != SIRLLM_OK) return 0;
    return workspace_layout(*cfg).total;
}

int sirllm_workspace_init(const sirllm_config* cfg, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (ws == nullptr) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    cudaError_t e = cudaMemsetAsync(ws, 0, workspace_layout(*cfg).total, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "cudaMemsetAsync");
}

int sirllm_score(const sirllm_config* cfg, const void* logits, const int32_t* token_ids,
                 const int32_t* n_new, float* out_entropy, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!logits || !token_ids || !out_entropy || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    if ((rc = check_logits(*cfg, logits)) != SIRLLM_OK) return rc;
    const WorkspaceLayout L = workspace_layout(*cfg);
    ScoreParams sp = score_params(*cfg, L, logits, token_ids, n_new, ws);
    sp.out_entropy = out_entropy;
    cudaError_t e = launch_score(sp, (cudaStream_t)cuda_stream, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "score");
}

int sirllm_score_partial(const sirllm_config* cfg, const void* logits_slice, int64_t col0,
                                    int64_t n_cols, int64_t slice_row_stride, const int32_t* token_ids,
                                    const int32_t* n_new, void* pairs_out, int64_t pair_stride,
                                    float* target_out, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if ((!logits_slice && n_cols != 0) || !token_ids || !pairs_out || !target_out || !ws)
        return SIRLLM_ERR_NULL;
    if (col0 < 0 || n_cols < 0 || col0 > cfg->vocab - n_cols || slice_row_stride < n_cols || pair_stride < 1)
        return SIRLLM_ERR_BAD_CONFIG;
    if (misaligned(ws, 256) || misaligned(pairs_out, 8)) return SIRLLM_ERR_ALIGN;
    if ((rc = check_logits(*cfg, logits_slice)) != SIRLLM_OK) return rc;
    const WorkspaceLayout L = workspace_layout(*cfg);
    ScoreParams sp = score_params(*cfg, L, logits_slice, token_ids, n_new, ws);
    sp.pairs_out = (float2*)pairs_out;
    sp.target_out = target_out;
    sp.pair_stride = pair_stride;
    sp.col0 = col0;
    sp.vocab = n_cols;  // columns streamed; a range is never wider than the vocabulary the
    sp.row_stride = slice_row_stride;  // workspace's per-row scratch was sized for
    sirllm_config range = *cfg;
    range.vocab = n_cols > 0 ? n_cols : 1;
    range.logits_row_stride = range.vocab;
    sp.n_part = workspace_layout(range).n_part;
    cudaError_t e = launch_score(sp, (cudaStream_t)cuda_stream, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "score_partial");
}

static SelectParams select_params(const sirllm_config& c, const WorkspaceLayout& L, float* scores,
                                  int64_t* serial, int32_t* live_len, const float* decay,
                                  int32_t* keep_idx, int32_t* n_keep, void* ws) {
    SelectParams p;
    memset(&p, 0, sizeof p);
    p.scores = scores;
    p.serial = serial;
    p.live_len = live_len;
    p.decay = decay;
    p.keep_idx = keep_idx ? keep_idx : (int32_t*)((char*)ws + L.keep_off);
    p.n_keep = n_keep ? n_keep : (int32_t*)((char*)ws + L.n_keep_off);
    p.first_moved = (int32_t*)((char*)ws + L.first_moved_off);
    p.ready = (int32_t*)((char*)ws + L.ready_off);
    p.status = (int32_t*)ws;
    p.epoch = (int32_t*)ws + 1;
    p.ticket = (unsigned long long*)ws + 1;
    p.capacity = c.capacity;
    p.budget = c.budget;
    p.n_sink = c.n_sink;
    p.n_recent = c.n_recent;
    p.threshold = c.threshold;
    return p;
}

int sirllm_decay_select(const sirllm_config* cfg, float* scores, int64_t* serial, int32_t* live_len,
                        const float* decay, int32_t* keep_idx, int32_t* n_keep,
                        int32_t compact_scores, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!scores || !live_len || !decay || !keep_idx || !n_keep || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    const WorkspaceLayout L = workspace_layout(*cfg);
    SelectParams p = select_params(*cfg, L, scores, serial, live_len, decay, keep_idx, n_keep, ws);
    p.compact_scores = compact_scores != 0;
    p.score_new = 0;
    cudaError_t e = launch_select(p, cfg->n_streams, (cudaStream_t)cuda_stream, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "select");
}

static int keep_policy_impl(const sirllm_config* cfg, int32_t policy, const int32_t* live_len,
                            uint64_t seed, int32_t round, int32_t stream_base, int32_t* keep_idx,
                            int32_t* n_keep, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!live_len || !keep_idx || !n_keep || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    if (policy != SIRLLM_POLICY_STREAM && policy != SIRLLM_POLICY_RANDOM &&
        policy != SIRLLM_POLICY_INTERVAL)
        return SIRLLM_ERR_BAD_CONFIG;
    const WorkspaceLayout L = workspace_layout(*cfg);
    PolicyParams pp;
    pp.live_len = live_len;
    pp.ranks = (float*)((char*)ws + L.policy_ranks_off);
    pp.ones = (float*)((char*)ws + L.policy_ones_off);
    pp.seed = seed;
    pp.policy = policy;
    pp.round = round;
    pp.stream_base = stream_base;
    pp.capacity = cfg->capacity;
    pp.budget = cfg->budget;
    pp.n_sink = cfg->n_sink;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = launch_policy_ranks(pp, cfg->n_streams, st);
    if (e != cudaSuccess) return cuda_fail(e, "policy_ranks");
    SelectParams sp = select_params(*cfg, L, pp.ranks, nullptr, const_cast<int32_t*>(live_len),
                                    pp.ones, keep_idx, n_keep, ws);
    sp.compact_scores = 0;  // live_len is only read
    sp.score_new = 0;
    e = launch_select(sp, cfg->n_streams, st, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "select");
}

static int compact_params(const sirllm_config& c, const WorkspaceLayout& L, const void* k_src,
                          const void* v_src, void* k_dst, void* v_dst, const int32_t* keep_idx,
                          const int32_t* n_keep, void* ws, CompactParams* out) {
    if ((k_src == nullptr) != (k_dst == nullptr) || (v_src == nullptr) != (v_dst == nullptr))
        return SIRLLM_ERR_NULL;
    const void* ptrs[4] = {k_src, v_src, k_dst, v_dst};
    for (const void* q : ptrs)
        if (q && misaligned(q, 16)) return SIRLLM_ERR_ALIGN;
    CompactParams p;
    memset(&p, 0, sizeof p);
    p.src[0] = (const char*)k_src;
    p.src[1] = (const char*)v_src;
    p.dst[0] = (char*)k_dst;
    p.dst[1] = (char*)v_dst;
    p.keep_idx = keep_idx;
    p.n_keep = n_keep;
    p.first_moved = (int32_t*)((char*)ws + L.first_moved_off);
    p.ready = (int32_t*)((char*)ws + L.ready_off);
    p.status = (int32_t*)ws;
    p.epoch = (int32_t*)ws + 1;
    p.ticket = (unsigned long long*)ws + 1;
    p.plane_progress = (unsigned long long*)((char*)ws + L.plane_progress_off);
    p.planes_per_stream = c.n_layers * c.n_kv_heads;
    p.planes_per_tensor = (int64_t)c.n_streams * p.planes_per_stream;
    p.capacity = c.capacity;
    p.keep_stride = c.threshold;
    p.row_bytes = c.head_dim * 2;
    const bool k_in = k_src && k_src == k_dst, v_in = v_src && v_src == v_dst;
    const bool k_out = k_src && k_src != k_dst, v_out = v_src && v_src != v_dst;
    if ((k_in || v_in) && (k_out || v_out)) return SIRLLM_ERR_BAD_CONFIG;  // do not mix modes
    p.in_place = (k_in || v_in) ? 1 : 0;
    *out = p;
    return SIRLLM_OK;
}

int sirllm_compact_kv(const sirllm_config* cfg, const void* k_src, const void* v_src, void* k_dst,
                      void* v_dst, const int32_t* keep_idx, const int32_t* n_keep, void* ws,
                      void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!keep_idx || !n_keep || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    const WorkspaceLayout L = workspace_layout(*cfg);
    CompactParams p;
    if ((rc = compact_params(*cfg, L, k_src, v_src, k_dst, v_dst, keep_idx, n_keep, ws, &p)) != SIRLLM_OK)
        return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = launch_compact_plan(p, cfg->n_streams, (int32_t*)((char*)ws + L.first_moved_off), st);
    if (e != cudaSuccess) return cuda_fail(e, "compact_plan");
    e = launch_compact(p, st, true);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "compact");
}

// Where the round's scores come from: the logits, or a producer's per-tile pairs.
struct ScoreSource {
    const void* logits = nullptr;
    const float2* pairs = nullptr;
    const float* target_logit = nullptr;
    int32_t n_tiles = 0;
    int64_t pair_row_stride = 0;
};

static int check_pairs(const ScoreSource& src) {
    if (!src.pairs || !src.target_logit) return SIRLLM_ERR_NULL;
    if (src.n_tiles < 1 || src.pair_row_stride < src.n_tiles) return SIRLLM_ERR_BAD_CONFIG;
    if (misaligned(src.pairs, 8) || misaligned(src.target_logit, 4)) return SIRLLM_ERR_ALIGN;
    return SIRLLM_OK;
}

static PairScoreParams pair_params(const sirllm_config& c, const ScoreSource& src,
                                   const int32_t* ids, const int32_t* n_new, void* ws) {
    PairScoreParams pp;
    memset(&pp, 0, sizeof pp);
    pp.pairs = src.pairs;
    pp.target_logit = src.target_logit;
    pp.token_ids = ids;
    pp.n_new = n_new;
    pp.status = (int32_t*)ws;
    pp.vocab = c.vocab;
    pp.pair_row_stride = src.pair_row_stride;
    pp.n_streams = c.n_streams;
    pp.max_new = c.max_new;
    pp.n_tiles = src.n_tiles;
    pp.capacity = c.capacity;
    return pp;
}

// Everything one round launches, checked and laid out before anything is enqueued.
struct StepPlan {
    bool from_pairs;
    ScoreParams sc;
    PairScoreParams pp;
    SelectParams sp;
    CompactParams cp;
    int n_streams;
    bool small_gather;  // the round's gather is the small two-phase kernel
};

// Host-side validation of a whole round; touches no device and enqueues nothing.
static int step_prepare(const sirllm_config* cfg, const ScoreSource& src, const int32_t* token_ids,
                        const int32_t* n_new, float* scores, int64_t* serial, int32_t* live_len,
                        const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                        float* new_entropy, void* ws, StepPlan* plan) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!token_ids || !scores || !live_len || !decay || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    if (src.pairs == nullptr) {
        if (!src.logits) return SIRLLM_ERR_NULL;
        if ((rc = check_logits(*cfg, src.logits)) != SIRLLM_OK) return rc;
    } else if ((rc = check_pairs(src)) != SIRLLM_OK) {
        return rc;
    }
    const WorkspaceLayout L = workspace_layout(*cfg);
    plan->from_pairs = src.pairs != nullptr;
    plan->n_streams = cfg->n_streams;
    plan->sp = select_params(*cfg, L, scores, serial, live_len, decay, keep_idx, n_keep, ws);
    plan->sc = score_params(*cfg, L, src.logits, token_ids, n_new, ws);
    plan->sc.out_entropy = new_entropy;
    plan->sc.scores = scores;
    plan->sc.live_len = live_len;
    plan->pp = pair_params(*cfg, src, token_ids, n_new, ws);
    plan->pp.out_entropy = new_entropy;
    plan->pp.scores = scores;
    plan->pp.live_len = live_len;
    plan->sp.n_new = n_new;
    plan->sp.max_new = cfg->max_new;
    plan->sp.compact_scores = 1;
    plan->sp.score_new = 1;
    rc = compact_params(*cfg, L, k, v, k, v, plan->sp.keep_idx, plan->sp.n_keep, ws, &plan->cp);
    const int64_t planes = ((k != nullptr) + (v != nullptr)) * plan->cp.planes_per_tensor;
    plan->small_gather = planes > 0 && compact_is_small_job(planes, plan->cp.keep_stride, plan->cp.row_bytes);
    return rc;
}

// The round's three launches (with `ev`: four event records around them, and no overlap
// between the kernels so that the events separate the phases).
static int step_enqueue(const StepPlan& plan, cudaStream_t st, void** ev) {
    cudaError_t e;
#define SIRLLM_MARK(i)                                                        \
    if (ev && (e = cudaEventRecord((cudaEvent_t)ev[i], st)) != cudaSuccess) \
        return cuda_fail(e, "cudaEventRecord");
    SIRLLM_MARK(0)
    // the scorer may overlap the end of a preceding small gather (see launch_score)
    const bool early = ev == nullptr && plan.small_gather;
    e = plan.from_pairs ? launch_score_pairs(plan.pp, st, early) : launch_score(plan.sc, st, early);
    if (e != cudaSuccess) return cuda_fail(e, "score");
    SIRLLM_MARK(1)
    // the selection kernel reads the caller's buffers before it waits for its predecessor: it may
    // only overlap the scorer, which itself started after all earlier work on the stream
    const bool scored = (int64_t)plan.n_streams * plan.sp.max_new > 0;
    e = launch_select(plan.sp, plan.n_streams, st, ev == nullptr && scored);
    if (e != cudaSuccess) return cuda_fail(e, "select");
    SIRLLM_MARK(2)
    e = launch_compact(plan.cp, st, ev == nullptr);
    if (e != cudaSuccess) return cuda_fail(e, "compact");
    SIRLLM_MARK(3)
#undef SIRLLM_MARK
    return SIRLLM_OK;
}

static int step_impl(const sirllm_config* cfg, const ScoreSource& src, const int32_t* token_ids,
                     const int32_t* n_new, float* scores, int64_t* serial, int32_t* live_len,
                     const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                     float* new_entropy, void* ws, void* cuda_stream, void** ev) {
    StepPlan plan;
    const int rc = step_prepare(cfg, src, token_ids, n_new, scores, serial, live_len, decay, k, v,
                                keep_idx, n_keep, new_entropy, ws, &plan);
    if (rc != SIRLLM_OK) return rc;
    return step_enqueue(plan, (cudaStream_t)cuda_stream, ev);
}

int sirllm_step(const sirllm_config* cfg, const void* logits, const int32_t* token_ids,
                const int32_t* n_new, float* scores, int64_t* serial, int32_t* live_len,
                const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                float* new_entropy, void* ws, void* cuda_stream) {
    ScoreSource src;
    src.logits = logits;
    return step_impl(cfg, src, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx,
                     n_keep, new_entropy, ws, cuda_stream, nullptr);
}

int sirllm_score_pairs(const sirllm_config* cfg, const void* pairs, int32_t n_tiles,
                       int64_t pair_row_stride, const float* target_logit,
                       const int32_t* token_ids, const int32_t* n_new, float* out_entropy,
                       void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!token_ids || !out_entropy || !ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    ScoreSource src;
    src.pairs = (const float2*)pairs;
    src.target_logit = target_logit;
    src.n_tiles = n_tiles;
    src.pair_row_stride = pair_row_stride;
    if ((rc = check_pairs(src)) != SIRLLM_OK) return rc;
    PairScoreParams pp = pair_params(*cfg, src, token_ids, n_new, ws);
    pp.out_entropy = out_entropy;
    cudaError_t e = launch_score_pairs(pp, (cudaStream_t)cuda_stream, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "score_pairs");
}

int sirllm_step_pairs(const sirllm_config* cfg, const void* pairs, int32_t n_tiles,
                      int64_t pair_row_stride, const float* target_logit, const int32_t* token_ids,
                      const int32_t* n_new, float* scores, int64_t* serial, int32_t* live_len,
                      const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                      float* new_entropy, void* ws, void* cuda_stream) {
    ScoreSource src;
    src.pairs = (const float2*)pairs;
    src.target_logit = target_logit;
    src.n_tiles = n_tiles;
    src.pair_row_stride = pair_row_stride;
    if (!pairs) return SIRLLM_ERR_NULL;
    return step_impl(cfg, src, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx,
                     n_keep, new_entropy, ws, cuda_stream, nullptr);
}

int sirllm_step_phases(const sirllm_config* cfg, const void* logits, const int32_t* token_ids,
                       const int32_t* n_new, float* scores, int64_t* serial, int32_t* live_len,
                       const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                       float* new_entropy, void* ws, void* cuda_stream, void** phase_events) {
    if (!phase_events) return SIRLLM_ERR_NULL;
    for (int i = 0; i < 4; ++i)
        if (!phase_events[i]) return SIRLLM_ERR_NULL;
    ScoreSource src;
    src.logits = logits;
    return step_impl(cfg, src, token_ids, n_new, scores, serial, live_len, decay, k, v, keep_idx,
                     n_keep, new_entropy, ws, cuda_stream, phase_events);
}

int sirllm_step_host(const sirllm_config* cfg, const void* h_logits, const int32_t* h_token_ids,
                     const int32_t* h_n_new, const void* h_new_k, const void* h_new_v,
                     const int32_t* h_live_len, void* d_logits, int32_t* d_token_ids,
                     int32_t* d_n_new, float* scores, int64_t* serial, int32_t* live_len,
                     const float* decay, void* k, void* v, int32_t* keep_idx, int32_t* n_keep,
                     float* new_entropy, int32_t* h_keep_idx, int32_t* h_n_keep,
                     float* h_new_entropy, void* ws, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!h_logits || !h_token_ids || !h_n_new || !h_live_len || !d_logits || !d_token_ids ||
        !d_n_new || !keep_idx || !n_keep || !new_entropy || !h_keep_idx || !h_n_keep ||
        !h_new_entropy)
        return SIRLLM_ERR_NULL;
    if ((h_new_k != nullptr && k == nullptr) || (h_new_v != nullptr && v == nullptr))
        return SIRLLM_ERR_NULL;
    // every check comes before the first copy: a refused call leaves the device untouched
    for (int s = 0; s < cfg->n_streams; ++s) {
        if (h_n_new[s] < 0 || h_n_new[s] > cfg->max_new || h_live_len[s] < 0)
            return SIRLLM_ERR_BAD_CONFIG;
    }
    ScoreSource src;
    src.logits = d_logits;
    StepPlan plan;
    rc = step_prepare(cfg, src, d_token_ids, d_n_new, scores, serial, live_len, decay, k, v,
                      keep_idx, n_keep, new_entropy, ws, &plan);
    if (rc != SIRLLM_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t es = (size_t)logits_elem_bytes(cfg->logits_dtype);
    const size_t row_bytes = (size_t)cfg->head_dim * 2;
    const size_t planes = (size_t)cfg->n_layers * cfg->n_kv_heads;
    cudaError_t e;
    for (int s = 0; s < cfg->n_streams; ++s) {
        const int T = h_n_new[s], l = h_live_len[s];
        if (T == 0 || l > cfg->capacity - T) continue;  // the device skips and flags an overflow
        const size_t row0 = (size_t)s * cfg->max_new;
        if (cfg->logits_row_stride == cfg->vocab) {
            e = cudaMemcpyAsync((char*)d_logits + row0 * cfg->vocab * es,
                                (const char*)h_logits + row0 * cfg->vocab * es,
                                (size_t)T * cfg->vocab * es, cudaMemcpyHostToDevice, st);
        } else {
            e = cudaMemcpy2DAsync((char*)d_logits + row0 * cfg->logits_row_stride * es,
                                  cfg->logits_row_stride * es,
                                  (const char*)h_logits + row0 * cfg->logits_row_stride * es,
                                  cfg->logits_row_stride * es, cfg->vocab * es, T,
                                  cudaMemcpyHostToDevice, st);
        }
        if (e != cudaSuccess) return cuda_fail(e, "logits H2D");
        const void* hsrc[2] = {h_new_k, h_new_v};
        void* ddst[2] = {k, v};
        for (int c = 0; c < 2; ++c) {
            if (!hsrc[c]) continue;
            e = cudaMemcpy2DAsync((char*)ddst[c] + ((size_t)s * planes * cfg->capacity + l) * row_bytes,
                                  (size_t)cfg->capacity * row_bytes,
                                  (const char*)hsrc[c] + (size_t)s * planes * cfg->max_new * row_bytes,
                                  (size_t)cfg->max_new * row_bytes, (size_t)T * row_bytes, planes,
                                  cudaMemcpyHostToDevice, st);
            if (e != cudaSuccess) return cuda_fail(e, "K/V H2D");
        }
    }
    const size_t n_rows = (size_t)cfg->n_streams * cfg->max_new;
    e = cudaMemcpyAsync(d_token_ids, h_token_ids, n_rows * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "ids H2D");
    e = cudaMemcpyAsync(d_n_new, h_n_new, (size_t)cfg->n_streams * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(e, "n_new H2D");
    if ((rc = step_enqueue(plan, st, nullptr)) != SIRLLM_OK) return rc;
    e = cudaMemcpyAsync(h_keep_idx, keep_idx, (size_t)cfg->n_streams * cfg->threshold * 4,
                        cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "keep D2H");
    e = cudaMemcpyAsync(h_n_keep, n_keep, (size_t)cfg->n_streams * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "n_keep D2H");
    e = cudaMemcpyAsync(h_new_entropy, new_entropy, n_rows * 4, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "entropy D2H");
    return SIRLLM_OK;
}

int sirllm_keep_policy(const sirllm_config* cfg, int32_t policy, const int32_t* live_len,
                       uint64_t seed, int32_t round, int32_t stream_base, int32_t* keep_idx,
                       int32_t* n_keep, void* ws, void* cuda_stream) {
    return keep_policy_impl(cfg, policy, live_len, seed, round, stream_base, keep_idx, n_keep,
                                   ws, cuda_stream);
}

int sirllm_rerotate_keys(const sirllm_config* cfg, void* k, const int32_t* keep_idx,
                         const int32_t* n_keep, double rope_base, int32_t layout, void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!k || !keep_idx || !n_keep) return SIRLLM_ERR_NULL;
    if (misaligned(k, 16)) return SIRLLM_ERR_ALIGN;
    if (cfg->head_dim % 16 != 0 || !(rope_base > 0.0) || !std::isfinite(rope_base) ||
        (layout != SIRLLM_ROPE_HALF && layout != SIRLLM_ROPE_INTERLEAVED))
        return SIRLLM_ERR_BAD_CONFIG;
    RopeParams p;
    p.k = (char*)k;
    p.keep_idx = keep_idx;
    p.n_keep = n_keep;
    for (int i = 0; i < cfg->head_dim / 2; ++i)
        p.theta[i] = std::pow(rope_base, -2.0 * (double)i / (double)cfg->head_dim);
    p.capacity = cfg->capacity;
    p.keep_stride = cfg->threshold;
    p.planes_per_stream = cfg->n_layers * cfg->n_kv_heads;
    p.head_dim = cfg->head_dim;
    p.layout = layout;
    p.planes_per_group = p.planes_per_stream;
    cudaError_t e = launch_rerotate(p, cfg->n_streams, cfg->kv_dtype == SIRLLM_BF16,
                                    (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "rerotate");
}

int sirllm_selftest_bounded_wait(const sirllm_config* cfg, void* ws, uint32_t polls,
                                 void* cuda_stream) {
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!ws) return SIRLLM_ERR_NULL;
    if (misaligned(ws, 256)) return SIRLLM_ERR_ALIGN;
    if (polls > (1u << 20)) return SIRLLM_ERR_BAD_CONFIG;  // keep the self-test short
    const WorkspaceLayout L = workspace_layout(*cfg);
    cudaError_t e = launch_bounded_wait_selftest(
        (unsigned long long*)((char*)ws + L.plane_progress_off), (const int32_t*)((char*)ws + L.keep_off),
        polls, (int32_t*)ws, (cudaStream_t)cuda_stream);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "bounded_wait_selftest");
}

int sirllm_status(void* ws, void* cuda_stream, int32_t* status_out, int32_t clear) {
    if (!ws || !status_out) return SIRLLM_ERR_NULL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(status_out, ws, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync");
    if (clear) {
        e = cudaMemsetAsync(ws, 0, sizeof(int32_t), st);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    }
    e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "cudaStreamSynchronize");
}

const char* sirllm_strerror(int code) {
    switch (code) {
        case SIRLLM_OK: return "ok";
        case SIRLLM_ERR_NULL: return "a required pointer is NULL";
        case SIRLLM_ERR_BAD_CONFIG: return "inconsistent or unsupported configuration";
        case SIRLLM_ERR_ALIGN: return "pointer or stride not aligned as required";
        case SIRLLM_ERR_CUDA: return "CUDA runtime error (see sirllm_last_cuda_error)";
        case SIRLLM_ERR_TOO_LARGE: return "problem larger than the fixed limit of this entry point";
        default: return "unknown error code";
    }
}

const char* sirllm_last_cuda_error(void) { return g_cuda_msg; }

}  // extern "C"
