// Token Entropy (Section 3.2): e = -log softmax(z)[id] as a vocabulary-streaming
// log-sum-exp.  Every logits row is cut into 64 KB parts, one CTA each, and every part into
// one segment per warp;
// one warp reduces one segment with an online (running-max) softmax sum, and the
// the warps of a CTA (4, or 8 / 16 when the grid would otherwise leave the GPU
// underfilled) combine their
// (scaled max, sum) pairs through shared memory.  A row that needs several CTAs
// (vocabularies above 32768 bf16 / 16384 fp32 elements) publishes one pair per CTA in
// scratch; the CTA that arrives last on the row's ticket combines them.  Combination is
// in fp64 and in a fixed order, so the score does not depend on which CTA comes last.
// The finishing warp writes the score and, in the fused round, appends it to E.
//
// The kernel is bound by HBM reads (2 or 4 bytes per element, each read once); the
// arithmetic per element is one conversion, one max, one FMA, one ex2 and one add.
#include <cuda_bf16.h>

#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kUnroll = 4;  // 16-byte loads in flight per lane and loop trip

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Running state of one lane: sum_v 2^(z_v*log2e - mL), with mL = (max so far)*log2e
// rounded once; the same rounded value is subtracted inside the FMA, so the pair
// (mL, sum) represents sum_v exp(z_v) = sum * 2^mL without a systematic error.
struct Online {
    float mL = kNegHuge;
    float s0 = 0.f, s1 = 0.f;
    __device__ __forceinline__ void raise(float group_max) {
        float cL = group_max * kLog2e;
        if (cL > mL) {
            float r = ex2_approx(mL - cL);
            s0 *= r;
            s1 *= r;
            mL = cL;
        }
    }
    __device__ __forceinline__ void add0(float z) { s0 += ex2_approx(fmaf(z, kLog2e, -mL)); }
    __device__ __forceinline__ void add1(float z) { s1 += ex2_approx(fmaf(z, kLog2e, -mL)); }
};

__device__ __forceinline__ uint32_t bf162_max(uint32_t a, uint32_t b) {
    __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
    __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
    __nv_bfloat162 m = __hmax2(x, y);
    return *reinterpret_cast<uint32_t*>(&m);
}

// One trip of a warp (kUnroll 16-byte vectors per lane) folded into the lane's running state.
template <bool kBf16>
__device__ __forceinline__ void reduce_trip(const uint4 (&x)[kUnroll], Online& st) {
    if (kBf16) {
        uint32_t m2 = x[0].x;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            m2 = bf162_max(m2, x[u].x);
            m2 = bf162_max(m2, x[u].y);
            m2 = bf162_max(m2, x[u].z);
            m2 = bf162_max(m2, x[u].w);
        }
        st.raise(fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u)));
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const uint32_t w[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                st.add0(__uint_as_float(w[q] << 16));
                st.add1(__uint_as_float(w[q] & 0xFFFF0000u));
            }
        }
    } else {
        float gm = __uint_as_float(x[0].x);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            gm = fmaxf(gm, fmaxf(fmaxf(__uint_as_float(x[u].x), __uint_as_float(x[u].y)),
                                 fmaxf(__uint_as_float(x[u].z), __uint_as_float(x[u].w))));
        }
        st.raise(gm);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            st.add0(__uint_as_float(x[u].x));
            st.add1(__uint_as_float(x[u].y));
            st.add0(__uint_as_float(x[u].z));
            st.add1(__uint_as_float(x[u].w));
        }
    }
}

template <bool kBf16, int kWarps>
__global__ void __launch_bounds__(kWarps * 32)
score_kernel(const ScoreParams p) {
    constexpr int kVecPerSeg = kScoreCtaVecs / kWarps;
    constexpr int ES = kBf16 ? 2 : 4;
    constexpr int EPV = 16 / ES;
    __shared__ float2 warp_pair[kWarps];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    // Possibly launched with programmatic serialization: behind a kernel that lets its
    // dependents go early (the small gather does, at its end) this grid becomes resident while
    // that kernel ends, which hides the launch latency; nothing is read before that kernel has
    // completed.  Only then may the kernel that follows (the selection) start to become
    // resident: what it reads ahead of its own wait is then settled as well.
    grid_dependency_wait();
    grid_launch_dependents();
    // one CTA = kWarps consecutive segments of one logits row
    const int64_t row = blockIdx.x / p.n_part;
    const int part_idx = (int)(blockIdx.x - row * p.n_part);
    const int seg = part_idx * kWarps + wid;
    const int s = (int)(row / p.max_new);
    const int t = (int)(row - (int64_t)s * p.max_new);
    int T = p.max_new;
    if (p.n_new != nullptr) T = min(p.n_new[s], p.max_new);
    if (t >= T) return;
    const int64_t V = p.vocab;
    const char* rowp = (const char*)p.logits + row * p.row_stride * ES;
    // warp 0 finishes the row: fetch what it will need now - the token id, the live length and
    // the target logit itself - so that nothing is waited for after the reduction
    int32_t id = -1;
    int l0 = -1;
    bool has_target = false;
    float z_target = 0.f;
    if (wid == 0) {
        id = p.token_ids[row];
        if (p.scores != nullptr) l0 = p.live_len[s];
        const int64_t col = (int64_t)id - (p.pairs_out != nullptr ? p.col0 : 0);
        has_target = id >= 0 && col >= 0 && col < V;
        if (has_target) z_target = load_logit(rowp, kBf16 ? SIRLLM_BF16 : SIRLLM_F32, col);
    }

    // elements in front of the first 16-byte boundary, whole vectors, elements after them
    int64_t head = (int64_t)(((16u - (uint32_t)((uintptr_t)rowp & 15u)) & 15u) / ES);
    if (head > V) head = V;
    const int64_t nvec = (V - head) / EPV;
    const int64_t tail = V - head - nvec * EPV;
    const uint4* vec = (const uint4*)(rowp + head * ES);
    const int64_t v0 = (int64_t)seg * kVecPerSeg;
    const int64_t v1 = min(v0 + (int64_t)kVecPerSeg, nvec);
    const uint32_t neg_inf = kBf16 ? 0xFF80FF80u : 0xFF800000u;

    // software pipeline: the loads of trip i+1 are in flight while trip i is reduced
    auto fetch = [&](int64_t base, uint4 (&x)[kUnroll]) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t idx = base + u * 32 + lane;
            if (idx < v1)
                x[u] = ld_stream_v4(vec + idx);
            else
                x[u] = make_uint4(neg_inf, neg_inf, neg_inf, neg_inf);
        }
    };
    Online st;
    uint4 x[kUnroll], xn[kUnroll];
    if (v0 < v1) fetch(v0, x);
    for (int64_t base = v0; base < v1; base += 32 * kUnroll) {
        fetch(base + 32 * kUnroll, xn);  // past the end: filled with -inf, never reduced
        reduce_trip<kBf16>(x, st);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) x[u] = xn[u];
    }
    // ragged ends of the row (fewer than one vector each) go to segment 0
    if (seg == 0 && lane < head + tail) {
        const int64_t e = lane < head ? lane : head + nvec * EPV + (lane - head);
        const float z = load_logit(rowp, kBf16 ? SIRLLM_BF16 : SIRLLM_F32, e);
        st.raise(z);
        st.add0(z);
    }
    // warp combine -> one (scaled max, sum) pair per warp
    float M = st.mL;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, o));
    float S = (st.s0 + st.s1) * ex2_approx(st.mL - M);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(0xFFFFFFFFu, S, o);
    if (lane == 0) warp_pair[wid] = make_float2(M, S);
    __syncthreads();
    if (wid != 0) return;

    // CTA combine in fp64 (fixed order): sum_v exp(z_v) over the CTA's segments = acc * 2^Mx
    float2 q = lane < kWarps ? warp_pair[lane] : make_float2(kNegHuge, 0.f);
    float Mx = q.x;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Mx = fmaxf(Mx, __shfl_xor_sync(0xFFFFFFFFu, Mx, o));
    double acc = (double)q.y * exp2((double)q.x - (double)Mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);

    if (p.n_part > 1) {
        // publish; the CTA that arrives last on the row's ticket combines the row
        float2* part = p.partials + row * p.n_part;
        int arrived = 0;
        if (lane == 0) {
            part[part_idx] = make_float2(Mx, (float)acc);
            __threadfence();
            arrived = atomicAdd(&p.tickets[row], 1);
        }
        arrived = __shfl_sync(0xFFFFFFFFu, arrived, 0);
        if (arrived != p.n_part - 1) return;
        __threadfence();
        if (lane == 0) p.tickets[row] = 0;  // ready for the next call
        Mx = kNegHuge;
        for (int i = lane; i < p.n_part; i += 32) Mx = fmaxf(Mx, __ldcg(&part[i]).x);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) Mx = fmaxf(Mx, __shfl_xor_sync(0xFFFFFFFFu, Mx, o));
        acc = 0.0;
        for (int i = lane; i < p.n_part; i += 32) {
            const float2 g = __ldcg(&part[i]);
            acc += (double)g.y * exp2((double)g.x - (double)Mx);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    }
    if (lane == 0 && p.pairs_out != nullptr) {
        // vocabulary-parallel: hand over this column range's share of the row's softmax sum as
        // (m, s) with sum_v exp z_v = s * exp(m), m within rounding of the range's maximum
        // (natural units), and the target logit if the token's column lies in the range
        float2 pr = make_float2(0.f, 0.f);  // an empty or fully masked range contributes nothing
        if (acc > 0.0) {
            pr.x = (float)((double)Mx * kLn2);
            pr.y = (float)(acc * exp2((double)Mx - (double)pr.x * 1.4426950408889634));
        }
        p.pairs_out[row * p.pair_stride] = pr;
        p.target_out[row] = has_target ? z_target : 0.f;
    } else if (lane == 0) {
        // e = ln(sum_v exp z_v) - z_id >= 0; id -1 = no prediction, other bad ids are flagged
        float e = 0.f;
        if (has_target) {
            e = fmaxf((float)(((double)Mx * kLn2 + log(acc)) - (double)z_target), 0.0f);
        } else if (id != -1) {
            atomicOr(p.status, SIRLLM_STATUS_TOKEN_RANGE);
        }
        if (p.out_entropy) p.out_entropy[row] = e;
        // the fused round appends the score behind the live slots (nowhere if it does not fit)
        if (p.scores != nullptr && l0 >= 0 && l0 <= p.capacity - T)
            p.scores[(size_t)s * p.capacity + l0 + t] = e;
    }
}

// Token Entropy from split-vocabulary partial results: a producer (an LM-head GEMM whose
// epilogue reduces every output tile) hands over, per row, n_tiles pairs
// (m_i = tile max, s_i = sum exp(z - m_i)) and the target logit, so the logits row itself is
// never read.  One warp per row; fp64 combine in a fixed order.
__global__ void __launch_bounds__(128) score_pairs_kernel(const PairScoreParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    grid_dependency_wait();
    grid_launch_dependents();
    if (row >= (int64_t)p.n_streams * p.max_new) return;
    const int s = (int)(row / p.max_new);
    const int t = (int)(row - (int64_t)s * p.max_new);
    int T = p.max_new;
    if (p.n_new != nullptr) T = min(p.n_new[s], p.max_new);
    if (t >= T) return;
    const float2* pr = p.pairs + row * p.pair_row_stride;
    float M = kNegHuge;
    for (int i = lane; i < p.n_tiles; i += 32) {
        const float2 q = pr[i];
        if (q.y > 0.f) M = fmaxf(M, q.x);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, o));
    double acc = 0.0;
    for (int i = lane; i < p.n_tiles; i += 32) {
        const float2 q = pr[i];
        if (q.y > 0.f) acc += (double)q.y * exp((double)q.x - (double)M);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) {
        const int32_t id = p.token_ids[row];
        float e = 0.f;
        if (id >= 0 && (int64_t)id < p.vocab) {
            e = fmaxf((float)(((double)M - (double)p.target_logit[row]) + log(acc)), 0.0f);
        } else if (id != -1) {
            atomicOr(p.status, SIRLLM_STATUS_TOKEN_RANGE);
        }
        if (p.out_entropy) p.out_entropy[row] = e;
        if (p.scores != nullptr) {
            const int l0 = p.live_len[s];
            if (l0 >= 0 && l0 <= p.capacity - T) p.scores[(size_t)s * p.capacity + l0 + t] = e;
        }
    }
}

}  // namespace

// A launch that may become resident before the preceding kernel on the stream has finished
// (programmatic stream serialization); the kernels wait for that kernel themselves.
template <typename Kernel, typename Params>
static cudaError_t launch_overlapped(Kernel kernel, unsigned grid, unsigned block, cudaStream_t st,
                                     const Params& p, bool overlap) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

cudaError_t launch_score_pairs(const PairScoreParams& p, cudaStream_t st, bool overlap) {
    TraceRange trace("sirllm:score_pairs");
    const int64_t rows = (int64_t)p.n_streams * p.max_new;
    if (rows == 0) return cudaSuccess;
    return launch_overlapped(score_pairs_kernel, (unsigned)((rows + 3) / 4), 128, st, p, overlap);
}

// With `overlap` the launch is programmatic (see the kernel).  The fused round asks for it only
// where the round's gather is the small two-phase kernel, which releases its dependents at its
// end: tiny rounds gain 1.5 us of launch latency.  Behind the persistent gather it was measured
// and rejected: released early, the parked scorer CTAs slowed the gather by 2-3 %; released at
// the gather's end, the scorer ran slower on SMs still set up for the gather's shared memory.
cudaError_t launch_score(const ScoreParams& p, cudaStream_t st, bool overlap) {
    TraceRange trace("sirllm:score");
    const int64_t ctas = (int64_t)p.n_streams * p.max_new * p.n_part;
    if (ctas == 0) return cudaSuccess;
    if (ctas > 0x7FFFFFFF) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)ctas;
    // 4 warps per CTA stream 16 KB each; a grid too small to give every SM even 8 warps takes
    // 8 or 16 warps per CTA instead (same bytes per CTA, shorter serial loop per warp).  With
    // more warps already resident, wider CTAs measured slower.
    DeviceProps dp;
    cudaError_t e = device_props(&dp);
    if (e != cudaSuccess) return e;
    const bool bf16 = p.logits_dtype == SIRLLM_BF16;
    const int64_t want_warps = (int64_t)dp.n_sm * 8;
    int warps = ctas * 4 >= want_warps ? 4 : (ctas * 8 >= want_warps ? 8 : 16);
    // 10 four-warp CTAs fit an SM (registers).  A grid between one and two such waves would
    // run a second wave that is mostly empty; with 8 warps per CTA the same rows make almost
    // three waves of CTAs half as long (measured -2 us on 2048 rows of 32000 bf16 logits).
    const int64_t one_wave = (int64_t)dp.n_sm * 10;
    if (warps == 4 && ctas > one_wave && ctas <= 2 * one_wave) warps = 8;
    if (warps == 4)
        return bf16 ? launch_overlapped(score_kernel<true, 4>, grid, 128, st, p, overlap)
                    : launch_overlapped(score_kernel<false, 4>, grid, 128, st, p, overlap);
    if (warps == 8)
        return bf16 ? launch_overlapped(score_kernel<true, 8>, grid, 256, st, p, overlap)
                    : launch_overlapped(score_kernel<false, 8>, grid, 256, st, p, overlap);
    return bf16 ? launch_overlapped(score_kernel<true, 16>, grid, 512, st, p, overlap)
                : launch_overlapped(score_kernel<false, 16>, grid, 512, st, p, overlap);
}

}  // namespace sirllm

// ---------------------------------------------------------------------------------------------
// sirllm_score_static: scoring for callers that cannot allocate device memory.
//
// sirllm_score needs a caller-allocated workspace for its tickets and per-CTA partial pairs.
// Some callers cannot provide one: code that runs inside a host framework which owns every
// allocation and hands out no scratch (a plugin or custom-op slot with fixed inputs and
// outputs), or code that must not touch the allocator at that point of the program (an
// allocation may synchronise the device or fail under memory pressure).  For them the same
// kernel runs on a scratch area that is part of the library image: a file-scope device
// array.  Every GPU that loads the library holds these kSsBytes bytes until the process
// exits, every call on a device shares them (so two calls that overlap on the GPU race),
// and the array keeps whatever the last call left in it, so each call first clears the part
// that has to start at zero.
namespace {

constexpr int64_t kSsMaxRows = 16384;    // logits rows (n_streams * max_new) per call
constexpr int64_t kSsMaxPairs = 65536;   // rows * CTAs per row
constexpr size_t kSsStatusOff = 0;                              // int32 status word
constexpr size_t kSsTicketsOff = 256;                           // int32 [kSsMaxRows]
constexpr size_t kSsPairsOff = kSsTicketsOff + kSsMaxRows * 4;  // float2 [kSsMaxPairs]
constexpr size_t kSsBytes = kSsPairsOff + kSsMaxPairs * 8;      // 590080 bytes

static __device__ __align__(256) unsigned char g_score_scratch[kSsBytes];

// In host code `g_score_scratch` is only a handle of the symbol, not a device address: the
// address each device gave the array is looked up once per device and remembered here.
constexpr int kSsMaxDevices = 64;
void* g_scratch_addr[kSsMaxDevices] = {};

cudaError_t scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kSsMaxDevices) return cudaErrorInvalidDevice;
    void* addr = __atomic_load_n(&g_scratch_addr[dev], __ATOMIC_ACQUIRE);
    if (addr == nullptr) {
        e = cudaGetSymbolAddress(&addr, g_score_scratch);  // of the CURRENT device
        if (e != cudaSuccess) return e;
        __atomic_store_n(&g_scratch_addr[dev], addr, __ATOMIC_RELEASE);
    }
    *out = addr;
    return cudaSuccess;
}

}  // namespace

extern "C" int sirllm_score_static(const sirllm_config* cfg, const void* logits,
                                   const int32_t* token_ids, const int32_t* n_new,
                                   float* out_entropy, int32_t* status, void* cuda_stream) {
    using namespace sirllm;
    int rc = validate_config(cfg);
    if (rc != SIRLLM_OK) return rc;
    if (!logits || !token_ids || !out_entropy) return SIRLLM_ERR_NULL;
    if (((uintptr_t)logits % (size_t)logits_elem_bytes(cfg->logits_dtype)) != 0) return SIRLLM_ERR_ALIGN;
    const WorkspaceLayout L = workspace_layout(*cfg);
    const int64_t rows = (int64_t)cfg->n_streams * cfg->max_new;
    if (rows > kSsMaxRows || rows * L.n_part > kSsMaxPairs) return SIRLLM_ERR_TOO_LARGE;
    if (rows == 0) return SIRLLM_OK;
    void* base = nullptr;
    cudaError_t e = scratch_address(&base);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // status word and tickets must start at zero; the pairs are written before they are read
    e = cudaMemsetAsync(base, 0, kSsTicketsOff + (size_t)rows * 4, st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    ScoreParams sp;
    sp.logits = logits;
    sp.token_ids = token_ids;
    sp.n_new = n_new;
    sp.partials = (float2*)((char*)base + kSsPairsOff);
    sp.tickets = (int32_t*)((char*)base + kSsTicketsOff);
    sp.status = status ? status : (int32_t*)((char*)base + kSsStatusOff);
    sp.out_entropy = out_entropy;
    sp.scores = nullptr;
    sp.live_len = nullptr;
    sp.pairs_out = nullptr;
    sp.target_out = nullptr;
    sp.pair_stride = 0;
    sp.col0 = 0;
    sp.vocab = cfg->vocab;
    sp.row_stride = cfg->logits_row_stride;
    sp.n_streams = cfg->n_streams;
    sp.max_new = cfg->max_new;
    sp.n_part = L.n_part;
    sp.logits_dtype = cfg->logits_dtype;
    sp.capacity = cfg->capacity;
    e = launch_score(sp, st, false);
    return e == cudaSuccess ? SIRLLM_OK : cuda_fail(e, "score");
}
