// Internal declarations shared by the kernels of the retention pass (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include "sirllm.h"

namespace sirllm {

// ---- workspace layout (device memory owned by the caller) -------------------------------
//   [0, 256)                              header: int32 status word, int32 compaction epoch,
//                                         uint64 ticket counter of the KV gather's work units
//   plane_progress[planes][kMaxSplit]     uint64 progress word per plane and segment, for the
//                                         planes (at most kChainPlanesMax) that are cut into segments
//   first_moved[n_streams]                first slot whose row changes place when compacting
//   ready[n_streams]                      1 once a stream's keep list is complete (polled by the gather)
//   n_keep_fallback[n_streams]            used when the caller passes no n_keep
//   keep_fallback[n_streams][threshold]   used when the caller passes no keep_idx
//   policy_ranks[n_streams][capacity]     synthetic scores of the comparison policies, ones[n_streams]
//   tickets[n_streams*max_new]            arrivals per logits row (the last CTA finishes the row)
//   partials[n_streams*max_new][n_part]   (scaled max, sum) pair per CTA of a multi-CTA row
struct WorkspaceLayout {
    size_t plane_progress_off;
    size_t first_moved_off;
    size_t ready_off;
    size_t n_keep_off;
    size_t keep_off;
    size_t tickets_off;
    size_t policy_ranks_off;
    size_t policy_ones_off;
    size_t partials_off;
    size_t total;
    int32_t n_part;  // CTAs (kScoreCtaVecs vectors each) per logits row
};

constexpr int kMaxSplit = 32;           // segments a plane's moved rows may be cut into (one per lane)
constexpr int kChainPlanesMax = 8192;   // with more K and V planes than this, planes are not cut
constexpr int kScoreCtaVecs = 4096;  // 16-byte vectors of one logits row per CTA: 64 KB, shared
                                     // by 4 warps (16 KB each) or, in small grids, 8 or 16

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int logits_elem_bytes(int dtype) { return dtype == SIRLLM_F32 ? 4 : 2; }

// A named NVTX range around the host side of a launch (tracing tools show it on the stream's
// timeline; a handful of nanoseconds when no tool is attached).
struct TraceRange {
    explicit TraceRange(const char* name) { nvtxRangePushA(name); }
    ~TraceRange() { nvtxRangePop(); }
    TraceRange(const TraceRange&) = delete;
    TraceRange& operator=(const TraceRange&) = delete;
};

int validate_config(const sirllm_config* cfg);

// Properties of the current device that the launch code needs at every call, looked up once per
// device and process (they never change): SM count and the opt-in shared-memory limit.
struct DeviceProps {
    int device;
    int n_sm;
    int smem_optin;
};
cudaError_t device_props(DeviceProps* out);
// Raises a kernel's dynamic shared-memory limit to the device's opt-in maximum, once per device.
// `done` is the kernel's own flag array (kMaxDevices entries, zero-initialised).
constexpr int kMaxDevices = 64;
cudaError_t allow_max_dynamic_smem(const void* kernel, const DeviceProps& dp, unsigned char* done);
// Records the message sirllm_last_cuda_error() returns and yields SIRLLM_ERR_CUDA.
int cuda_fail(cudaError_t e, const char* where);
WorkspaceLayout workspace_layout(const sirllm_config& cfg);

struct ScoreParams {
    const void* logits;
    const int32_t* token_ids;
    const int32_t* n_new;  // nullable: max_new for every stream
    float2* partials;
    int32_t* tickets;
    int32_t* status;
    float* out_entropy;        // [n_streams*max_new] raw scores, nullable
    float* scores;             // nullable: also append at scores[s][live_len[s] + t] (fused round)
    const int32_t* live_len;   // with `scores`
    // vocabulary-parallel mode (pairs_out != nullptr): `logits` holds columns [col0, col0 + vocab)
    // of every row; instead of a score the row's (max, sum exp) pair and target logit go out
    float2* pairs_out;         // [rows][pair_stride]
    float* target_out;         // [rows]
    int64_t pair_stride;
    int64_t col0;
    int64_t vocab;             // columns streamed per row
    int64_t row_stride;
    int32_t n_streams, max_new, n_part, logits_dtype, capacity;
};

struct PairScoreParams {
    const float2* pairs;        // [rows][pair_row_stride] (tile max, tile sum of exp(z - max))
    const float* target_logit;  // [rows]
    const int32_t* token_ids;
    const int32_t* n_new;       // nullable
    int32_t* status;
    float* out_entropy;         // nullable
    float* scores;              // nullable: append at scores[s][live_len[s] + t]
    const int32_t* live_len;
    int64_t vocab, pair_row_stride;
    int32_t n_streams, max_new, n_tiles, capacity;
};

struct SelectParams {
    const int32_t* n_new;  // with score_new: tokens appended this round (nullable: max_new)
    int32_t max_new;
    float* scores;
    int64_t* serial;       // nullable
    int32_t* live_len;
    const float* decay;
    int32_t* keep_idx;
    int32_t* n_keep;
    int32_t* first_moved;
    int32_t* ready;   // [n_streams] 1 once the stream's keep list, n_keep and first_moved are out
    int32_t* status;
    int32_t* epoch;
    unsigned long long* ticket;  // hand-out counter of the gather that follows: reset with the epoch
    int32_t capacity, budget, n_sink, n_recent, threshold;
    int32_t compact_scores;  // also gather scores / serial and commit live_len
    int32_t score_new;       // the round's new scores were appended behind live_len by the scorer
};

struct PolicyParams {
    const int32_t* live_len;
    float* ranks;  // [n_streams][capacity] synthetic scores
    float* ones;   // [n_streams] decay ratio 1 for the selection kernel
    uint64_t seed;
    int32_t policy, round, stream_base, capacity, budget, n_sink;
};

struct RopeParams {
    char* k;
    const int32_t* keep_idx;
    const int32_t* n_keep;
    // theta_i = base^(-2i/d) for the d/2 pairs of a row, computed once per call on the host (pow)
    double theta[SIRLLM_MAX_HEAD_DIM / 2];
    int32_t capacity, keep_stride, planes_per_stream, head_dim, layout, planes_per_group;
};

struct CompactParams {
    const char* src[2];  // K, V (nullable)
    char* dst[2];
    const int32_t* keep_idx;
    const int32_t* n_keep;
    const int32_t* first_moved;
    int32_t* ready;        // [n_streams] raised by the preceding kernel once a stream's list is out
    int32_t* status;
    int32_t* epoch;        // bumped once per compaction by the kernel that precedes it
    unsigned long long* ticket;  // next work unit to hand out; zeroed by the same kernel
    unsigned long long* plane_progress;  // [min(planes, kChainPlanesMax)][kMaxSplit]
    int64_t planes_per_tensor;  // n_streams * n_layers * n_kv_heads
    int32_t planes_per_stream;
    int32_t capacity, keep_stride, row_bytes;
    int32_t in_place;
};

// `overlap`: launch with programmatic stream serialization (the kernels wait for their
// predecessor themselves), so that the grid may become resident while a predecessor that
// releases its dependents early is ending.
cudaError_t launch_score(const ScoreParams& p, cudaStream_t st, bool overlap);
cudaError_t launch_score_pairs(const PairScoreParams& p, cudaStream_t st, bool overlap);
// true if a gather over `planes` K and V planes goes to the small two-phase kernel
bool compact_is_small_job(int64_t planes, int keep_stride, int row_bytes);
// `overlap`: launch with programmatic stream serialization, so the grid may become resident
// while the previous kernel on the stream drains; the kernel itself waits for that kernel's
// results (grid_dependency_wait) before it reads them.
cudaError_t launch_select(const SelectParams& p, int n_streams, cudaStream_t st, bool overlap);
cudaError_t launch_policy_ranks(const PolicyParams& p, int n_streams, cudaStream_t st);
cudaError_t launch_rerotate(const RopeParams& p, int n_streams, bool bf16, cudaStream_t st);
cudaError_t launch_compact_plan(const CompactParams& p, int n_streams, int32_t* first_moved,
                                cudaStream_t st);
cudaError_t launch_compact(const CompactParams& p, cudaStream_t st, bool overlap);
cudaError_t launch_bounded_wait_selftest(unsigned long long* prog, const int32_t* keep, uint32_t limit,
                                         int32_t* status, cudaStream_t st);

// ---- small device helpers ----------------------------------------------------------------
#ifdef __CUDACC__
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453;
constexpr float kNegHuge = -3.0e38f;  // "no element seen yet" for a running maximum

// Programmatic dependent launch: wait until the preceding kernel on the stream has
// completed and its writes are visible (no-op for a normally launched kernel); allow the
// following kernel to start becoming resident.
__device__ __forceinline__ void grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- mbarrier / TMA bulk-copy wrappers (non-tensor cp.async.bulk: 16-byte aligned
// addresses, sizes that are multiples of 16 bytes) ------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// The one arrival of a stage's phase plus the bytes its bulk loads will deliver.  Relaxed: the
// arrival publishes nothing (the stage record written before it is read back by the same warp
// after a __syncwarp), so it need not wait for earlier shared-memory stores.
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.relaxed.cta.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint32_t limit) {
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++spins > limit) return false;
    }
    return true;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(smem_u32(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
// polls before a device-side wait gives up (a healthy wait ends within microseconds for an
// mbarrier and within one kernel duration for a progress word; these limits are seconds)
constexpr uint32_t kSpinLimit = 1u << 22;      // global-memory progress words (>= 200 ns a poll)
constexpr uint32_t kMbarSpinLimit = 1u << 20;  // mbarrier phases (each poll may itself suspend)

// Progress words in global memory, GPU scope.
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
// A progress word carries no data besides itself (what it announces - bulk loads that have
// landed - completed before the announcing thread saw their mbarrier flip), so it is written
// relaxed: a release store would first wait for every load the thread still has in flight.
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_relaxed_u32(int32_t* p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const int32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Order-preserving map from fp32 bit patterns to unsigned integers: a larger key is a
// larger score; negatives sort below non-negatives and -0 below +0.
__device__ __forceinline__ uint32_t order_key(uint32_t bits) {
    return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}

__device__ __forceinline__ float load_logit(const void* logits, int dtype, int64_t idx) {
    if (dtype == SIRLLM_F32) return ((const float*)logits)[idx];
    return __uint_as_float((uint32_t)((const uint16_t*)logits)[idx] << 16);
}
#endif

}  // namespace sirllm
