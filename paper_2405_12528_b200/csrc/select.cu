// Append + memory decay + selection + score compaction for one stream per CTA
// (Section 3.3: E = E x eta_decay, Top_k(E); Section 3.1: sink and recent sets;
// Algorithm 1: the test "cache size > L").
//
// All scores of the stream live in shared memory as fp32 bit patterns.  The k-th
// largest middle score is found by a most-significant-digit radix select on the
// order-preserving key (11-bit digits, skipping the bits all keys share), ties at the
// threshold are resolved towards the lower slot, and the keep list is emitted in
// ascending order with warp ballots and a block prefix sum.  Touches at most a few
// hundred KB: this is the latency-bound serial link between scoring and KV compaction.
#include "common.cuh"

namespace sirllm {

namespace {

struct BlockScratch {
    int warp_sum[32];
    int warp_sure[32];
    int warp_eq[32];
    uint32_t red_and[32];
    uint32_t red_or[32];
    int bin;
    int above;
    int first_evicted;
};

// inclusive prefix sum over the 1024 threads of the block
__device__ __forceinline__ int block_inclusive_scan(int v, int* warp_sum) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += n;
    }
    if (lane == 31) warp_sum[wid] = v;
    __syncthreads();
    if (wid == 0) {
        int w = warp_sum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xFFFFFFFFu, w, o);
            if (lane >= o) w += n;
        }
        warp_sum[lane] = w;
    }
    __syncthreads();
    if (wid > 0) v += warp_sum[wid - 1];
    return v;
}

__global__ void __launch_bounds__(kSelectThreads, 1) select_kernel(const SelectParams p) {
    extern __shared__ uint32_t smem[];
    uint32_t* vals = smem;                        // [capacity] fp32 bit patterns
    int* hist = (int*)(smem + p.capacity);        // [kRadixBins]
    __shared__ BlockScratch sh;

    const int s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int cap = p.capacity;
    float* scores = p.scores + (size_t)s * cap;
    int32_t* keep = p.keep_idx + (size_t)s * p.threshold;
    grid_launch_dependents();
    grid_dependency_wait();  // the scorer's appended scores
    if (blockIdx.x == 0 && tid == 0) *p.epoch += 1;  // a new compaction follows

    const int l0 = p.live_len[s];
    const float eta = p.decay[s];  // fetched together with the lengths: one round trip
    int T = 0;
    if (p.score_new) {  // the scorer has appended T raw scores behind slot l0
        T = p.n_new ? p.n_new[s] : p.max_new;
        T = max(0, min(T, p.max_new));
    }
    if (l0 < 0 || l0 > cap - T) {  // the round does not fit: leave the stream alone
        if (tid == 0) {
            atomicOr(p.status, SIRLLM_STATUS_OVERFLOW);
            const int n = max(0, min(l0, min(cap, p.threshold)));
            p.n_keep[s] = n;
            p.first_moved[s] = n;
        }
        return;
    }
    const int l = l0 + T;

    // ---- S3: one fp32 multiply per held score -----------------------------------------
    const bool evict = l > p.threshold;
    const bool write_now = !(evict && p.compact_scores);
    // loads are issued in batches before any of them is used, so the block pays one memory
    // round trip per batch instead of one per element
    constexpr int kLoadBatch = 16;
    for (int base = 0; base < l; base += kLoadBatch * kSelectThreads) {
        float x[kLoadBatch];
#pragma unroll
        for (int q = 0; q < kLoadBatch; ++q) {
            const int i = base + q * kSelectThreads + tid;
            x[q] = i < l ? scores[i] : 0.f;
        }
#pragma unroll
        for (int q = 0; q < kLoadBatch; ++q) {
            const int i = base + q * kSelectThreads + tid;
            if (i < l) {
                const float v = __fmul_rn(x[q], eta);
                vals[i] = __float_as_uint(v);
                if (write_now) scores[i] = v;
            }
        }
    }
    if (!evict) {  // ---- nothing to evict: identity keep list --------------------------
        for (int i = tid; i < l; i += kSelectThreads) keep[i] = i;
        if (tid == 0) {
            p.n_keep[s] = l;
            p.first_moved[s] = l;
            if (p.compact_scores) p.live_len[s] = l;
        }
        return;
    }
    __syncthreads();

    // ---- S4: threshold key of the top-k among the middle slots ---------------------------
    const int lo = p.n_sink, hi = l - p.n_recent;
    const int k = p.budget - p.n_sink - p.n_recent;
    uint32_t tau = 0xFFFFFFFFu;  // with k == 0 nothing in the middle is kept
    int r = 0;                   // how many slots with key == tau are kept (lowest slots first)
    if (k > 0) {
        uint32_t a = 0xFFFFFFFFu, o = 0u;
        for (int i = lo + tid; i < hi; i += kSelectThreads) {
            const uint32_t key = order_key(vals[i]);
            a &= key;
            o |= key;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            a &= __shfl_xor_sync(0xFFFFFFFFu, a, d);
            o |= __shfl_xor_sync(0xFFFFFFFFu, o, d);
        }
        if (lane == 0) {
            sh.red_and[wid] = a;
            sh.red_or[wid] = o;
        }
        __syncthreads();
        a = sh.red_and[lane];
        o = sh.red_or[lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            a &= __shfl_xor_sync(0xFFFFFFFFu, a, d);
            o |= __shfl_xor_sync(0xFFFFFFFFu, o, d);
        }
        const uint32_t diff = a ^ o;
        int undecided = diff ? 32 - __clz(diff) : 0;  // low bits not yet fixed
        uint32_t prefix = undecided < 32 ? (a >> undecided) : 0u;  // the shared high bits
        int need = k;
        while (undecided > 0) {
            const int w = min(kRadixBits, undecided);
            const int sh_amt = undecided - w;
            for (int b = tid; b < kRadixBins; b += kSelectThreads) hist[b] = 0;
            __syncthreads();
            for (int i = lo + tid; i < hi; i += kSelectThreads) {
                const uint32_t key = order_key(vals[i]);
                if ((uint32_t)((uint64_t)key >> undecided) == prefix)
                    atomicAdd(&hist[(key >> sh_amt) & ((1u << w) - 1u)], 1);
            }
            __syncthreads();
            // walk the bins from the largest digit down; thread t owns two of them
            const int c0 = hist[kRadixBins - 1 - 2 * tid];
            const int c1 = hist[kRadixBins - 2 - 2 * tid];
            const int incl = block_inclusive_scan(c0 + c1, sh.warp_sum);
            const int excl = incl - (c0 + c1);
            if (excl < need && need <= excl + c0) {
                sh.bin = kRadixBins - 1 - 2 * tid;
                sh.above = excl;
            } else if (excl + c0 < need && need <= incl) {
                sh.bin = kRadixBins - 2 - 2 * tid;
                sh.above = excl + c0;
            }
            __syncthreads();
            prefix = (prefix << w) | (uint32_t)sh.bin;
            need -= sh.above;
            undecided = sh_amt;
            __syncthreads();
        }
        tau = prefix;
        r = need;
    }

    // ---- S4 (emit) + S5: ascending keep list, compacted scores ------------------------------
    // warp w owns a contiguous span of slots; sure = sink / recent / above the threshold key
    const int span = ((l + 31) / 32 + 31) & ~31;
    const int w_begin = wid * span, w_end = min(l, w_begin + span);
    int n_sure = 0, n_eq = 0;
    for (int base = w_begin; base < w_end; base += 32) {
        const int i = base + lane;
        bool sure = false, eq = false;
        if (i < w_end) {
            if (i < lo || i >= hi) {
                sure = true;
            } else {
                const uint32_t key = order_key(vals[i]);
                sure = key > tau;
                eq = key == tau;
            }
        }
        n_sure += __popc(__ballot_sync(0xFFFFFFFFu, sure));
        n_eq += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (tid == 0) sh.first_evicted = l;
    if (lane == 0) {
        sh.warp_sure[wid] = n_sure;
        sh.warp_eq[wid] = n_eq;
    }
    __syncthreads();
    int sure_before = 0, eq_before = 0;
    for (int q = 0; q < wid; ++q) {
        sure_before += sh.warp_sure[q];
        eq_before += sh.warp_eq[q];
    }
    int kept_before = sure_before + min(eq_before, r);
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int base = w_begin; base < w_end; base += 32) {
        const int i = base + lane;
        bool sure = false, eq = false;
        uint32_t bits = 0;
        if (i < w_end) {
            bits = vals[i];
            if (i < lo || i >= hi) {
                sure = true;
            } else {
                const uint32_t key = order_key(bits);
                sure = key > tau;
                eq = key == tau;
            }
        }
        const uint32_t eq_ballot = __ballot_sync(0xFFFFFFFFu, eq);
        const bool kept = sure || (eq && eq_before + __popc(eq_ballot & lt_mask) < r);
        const uint32_t kept_ballot = __ballot_sync(0xFFFFFFFFu, kept);
        if (kept) {
            const int pos = kept_before + __popc(kept_ballot & lt_mask);
            keep[pos] = i;
            if (p.compact_scores) scores[pos] = __uint_as_float(bits);
        } else if (i < w_end) {
            atomicMin(&sh.first_evicted, i);
        }
        kept_before += __popc(kept_ballot);
        eq_before += __popc(eq_ballot);
    }
    __syncthreads();
    const int first = sh.first_evicted;

    // ---- S5: the 8-byte tags follow, in place, front to back.  A batch of kTagBatch tags
    // per thread is read into registers before any of them is written; a later batch only
    // reads slots at or behind its own first destination, which earlier batches never wrote.
    if (p.serial != nullptr && p.compact_scores) {
        constexpr int kTagBatch = 8;
        int64_t* serial = p.serial + (size_t)s * cap;
        for (int base = first; base < p.budget; base += kTagBatch * kSelectThreads) {
            int64_t v[kTagBatch];
#pragma unroll
            for (int q = 0; q < kTagBatch; ++q) {
                const int j = base + q * kSelectThreads + tid;
                v[q] = j < p.budget ? serial[keep[j]] : 0;
            }
            __syncthreads();
#pragma unroll
            for (int q = 0; q < kTagBatch; ++q) {
                const int j = base + q * kSelectThreads + tid;
                if (j < p.budget) serial[j] = v[q];
            }
            __syncthreads();
        }
    }
    if (tid == 0) {  // ---- S7
        p.n_keep[s] = p.budget;
        p.first_moved[s] = first;
        if (p.compact_scores) p.live_len[s] = p.budget;
    }
}

}  // namespace

cudaError_t launch_select(const SelectParams& p, int n_streams, cudaStream_t st, bool overlap) {
    const size_t smem = (size_t)p.capacity * 4 + (size_t)kRadixBins * 4;
    cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_streams);
    cfg.blockDim = dim3(kSelectThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, select_kernel, p);
}

}  // namespace sirllm
