// Append + memory decay + selection + score compaction for one stream per CTA
// (Section 3.3: E = E x eta_decay, Top_k(E); Section 3.1: sink and recent sets;
// Algorithm 1: the test "cache size > L").
//
// All scores of the stream live in shared memory as fp32 bit patterns.  The k-th largest
// middle score is found on the order-preserving integer key of the bit pattern:
//   1. min and max key of the middle slots (block reduction);
//   2. a most-significant-digit radix pass over d = key - min (11-bit digits of the range the
//      keys really span, 2048-bin shared histogram, block scan from the top bin);
//   3. as soon as the bin that holds the k-th key has at most kListMax members they are listed
//      and ranked directly; otherwise the next digit is taken (ties in bulk, tiny ranges).
// Ties at the threshold are resolved towards the lower slot.  The ascending keep list and the
// compacted scores are then written by threads that each own a contiguous run of slots (count,
// block prefix sum, write), and the 8-byte tags follow in register batches.
// The kernel runs on one SM and touches at most a few hundred KB: it is the instruction- and
// latency-bound serial link between scoring and KV compaction.
#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kSelectThreads = 1024;
constexpr int kRadixBits = 11;
constexpr int kRadixBins = 1 << kRadixBits;
constexpr int kListMax = 256;  // keys ranked directly once a radix bin holds no more

struct BlockScratch {
    uint32_t warp_sum[32];
    uint32_t red_min[32];
    uint32_t red_max[32];
    int bin;
    int above;
    int bin_count;
    int list_n;
    uint32_t tau;
    int r;
    int first_evicted;
};

// inclusive prefix sum over the 1024 threads of the block (unsigned: wraps, never overflows)
__device__ __forceinline__ uint32_t block_inclusive_scan_u32(uint32_t v, uint32_t* warp_sum) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += n;
    }
    if (lane == 31) warp_sum[wid] = v;
    __syncthreads();
    if (wid == 0) {
        uint32_t w = warp_sum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t n = __shfl_up_sync(0xFFFFFFFFu, w, o);
            if (lane >= o) w += n;
        }
        warp_sum[lane] = w;
    }
    __syncthreads();
    if (wid > 0) v += warp_sum[wid - 1];
    return v;
}
__device__ __forceinline__ int block_inclusive_scan(int v, uint32_t* warp_sum) {
    return (int)block_inclusive_scan_u32((uint32_t)v, warp_sum);
}

// The keep list of stream s is complete: make it (and the counts) visible to the whole GPU and
// raise the stream's ready word, which the KV gather that follows polls instead of waiting for
// this whole grid to finish - compaction of K and V then overlaps the rest of this kernel
// (score and tag compaction).  Called by every thread of the block, on every path.
__device__ __forceinline__ void publish_keep_list(const SelectParams& p, int s, int n_keep, int first_moved) {
    __syncthreads();  // every thread's part of the keep list precedes ...
    if (threadIdx.x == 0) {
        p.n_keep[s] = n_keep;
        p.first_moved[s] = first_moved;
        __threadfence();  // ... this fence (cumulative), and so the word raised after it
        st_relaxed_u32(&p.ready[s], 1u);
    }
}

// kStage: the keep list is assembled in shared memory and written out coalesced (the host
// chooses this whenever capacity + threshold words fit); otherwise it goes straight to global
// memory from the owning threads.
template <bool kStage>
__global__ void __launch_bounds__(kSelectThreads, 1) select_kernel(const SelectParams p) {
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* vals = smem;                                      // [capacity] fp32 bit patterns
    int* hist = (int*)(smem + ((p.capacity + 3) & ~3) + 4);     // [kRadixBins]
    int* skeep = hist + kRadixBins;                             // [threshold] when kStage
    __shared__ BlockScratch sh;

    const int s = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int cap = p.capacity;
    float* scores = p.scores + (size_t)s * cap;
    int32_t* keep = p.keep_idx + (size_t)s * p.threshold;
    // the gather polls ready[s]: take it down before any dependent grid can start; with it the
    // gather's epoch and ticket counter are set for the compaction that follows (everything
    // earlier on the stream, the previous gather included, is complete when this grid starts)
    if (tid == 0) {
        st_relaxed_u32(&p.ready[s], 0u);
        if (blockIdx.x == 0) {
            *p.epoch += 1;
            *p.ticket = 0ull;
        }
        __threadfence();
    }
    __syncthreads();
    grid_launch_dependents();
    // In the fused round this grid may become resident while the scorer is still draining
    // (programmatic dependent launch).  Everything up to grid_dependency_wait() uses only
    // what the scorer does not produce - the lengths, the decay ratio and the l0 scores held
    // from earlier rounds - so it overlaps the scorer's tail; only the round's T new scores
    // are folded in after the wait.
    const int l0 = p.live_len[s];
    const float eta = p.decay[s];  // fetched together with the lengths: one round trip
    int T = 0;
    if (p.score_new) {  // the scorer appends T raw scores behind slot l0
        T = p.n_new ? p.n_new[s] : p.max_new;
        T = max(0, min(T, p.max_new));
    }
    if (l0 < 0 || l0 > cap - T) {  // the round does not fit: leave the stream alone
        grid_dependency_wait();
        if (tid == 0) atomicOr(p.status, SIRLLM_STATUS_OVERFLOW);
        const int n = max(0, min(l0, min(cap, p.threshold)));
        publish_keep_list(p, s, n, n);  // nothing moves
        return;
    }
    const int l = l0 + T;

    // ---- S3: one fp32 multiply per held score -----------------------------------------
    const bool evict = l > p.threshold;
    const bool write_now = !(evict && p.compact_scores);
    // loads are issued in batches before any of them is used, so the block pays one memory
    // round trip per batch instead of one per element
    constexpr int kLoadBatch = 16;
    const int lo = p.n_sink, hi = l - p.n_recent;
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;  // over the middle slots' keys (for S4)
    auto decay_range = [&](int begin, int end) {
        for (int base = begin; base < end; base += kLoadBatch * kSelectThreads) {
            float x[kLoadBatch];
#pragma unroll
            for (int q = 0; q < kLoadBatch; ++q) {
                const int i = base + q * kSelectThreads + tid;
                x[q] = i < end ? scores[i] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < kLoadBatch; ++q) {
                const int i = base + q * kSelectThreads + tid;
                if (i < end) {
                    const float v = __fmul_rn(x[q], eta);
                    vals[i] = __float_as_uint(v);
                    if (write_now) scores[i] = v;
                    if (i >= lo && i < hi) {
                        const uint32_t key = order_key(__float_as_uint(v));
                        kmin = min(kmin, key);
                        kmax = max(kmax, key);
                    }
                }
            }
        }
    };
    decay_range(0, l0);      // the scores of earlier rounds
    for (int b = tid; b < kRadixBins; b += kSelectThreads) hist[b] = 0;  // for the first digit pass
    grid_dependency_wait();  // the scorer's appended scores are complete and visible
    decay_range(l0, l);      // this round's scores
    if (!evict) {  // ---- nothing to evict: identity keep list --------------------------
        for (int i = tid; i < l; i += kSelectThreads) keep[i] = i;
        publish_keep_list(p, s, l, l);
        if (tid == 0 && p.compact_scores) p.live_len[s] = l;
        return;
    }

    // ---- S4: threshold key of the top-k among the middle slots ---------------------------
    const int k = p.budget - p.n_sink - p.n_recent;
    uint32_t tau = 0xFFFFFFFFu;  // with k == 0 nothing in the middle is kept
    int r = 0;                   // how many slots with key == tau are kept (lowest slots first)
    if (k > 0) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, d));
            kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, d));
        }
        if (lane == 0) {
            sh.red_min[wid] = kmin;
            sh.red_max[wid] = kmax;
        }
        __syncthreads();  // also orders the writes of vals before the reads below
        kmin = sh.red_min[lane];
        kmax = sh.red_max[lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, d));
            kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, d));
        }
        // from here on keys are taken relative to the smallest one: d = key - kmin < 2^undecided
        const uint32_t range = kmax - kmin;
        int undecided = range ? 32 - __clz(range) : 0;  // low bits of d not yet fixed
        uint32_t prefix = 0u;                           // the fixed high bits of d
        int need = k;
        bool first_pass = true;  // its histogram was zeroed ahead of the wait
        while (undecided > 0) {
            const int w = min(kRadixBits, undecided);
            const int sh_amt = undecided - w;
            if (!first_pass) {
                for (int b = tid; b < kRadixBins; b += kSelectThreads) hist[b] = 0;
                __syncthreads();
            }
            first_pass = false;
            for (int i = lo + tid; i < hi; i += kSelectThreads) {
                const uint32_t d = order_key(vals[i]) - kmin;
                if ((uint32_t)((uint64_t)d >> undecided) == prefix)
                    atomicAdd(&hist[(d >> sh_amt) & ((1u << w) - 1u)], 1);
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
                sh.bin_count = c0;
                sh.list_n = 0;
            } else if (excl + c0 < need && need <= incl) {
                sh.bin = kRadixBins - 2 - 2 * tid;
                sh.above = excl + c0;
                sh.bin_count = c1;
                sh.list_n = 0;
            }
            __syncthreads();
            prefix = (prefix << w) | (uint32_t)sh.bin;
            need -= sh.above;
            undecided = sh_amt;
            const int n_left = sh.bin_count;
            __syncthreads();
            if (undecided > 0 && n_left <= kListMax) {
                // few keys are left in the bin: list them and rank them directly instead of
                // running the remaining digit passes
                uint32_t* list = reinterpret_cast<uint32_t*>(hist);
                for (int i = lo + tid; i < hi; i += kSelectThreads) {
                    const uint32_t d = order_key(vals[i]) - kmin;
                    if ((d >> undecided) == prefix) list[atomicAdd(&sh.list_n, 1)] = d;
                }
                __syncthreads();
                {
                    // a team of four threads ranks one listed key, each against a quarter of the list
                    static_assert(kListMax * 4 == kSelectThreads, "one team of four per listed key");
                    const int e = tid >> 2, part = tid & 3;
                    const uint32_t mine = e < n_left ? list[e] : 0u;
                    int greater = 0, equal = 0;
                    if (e < n_left) {
                        for (int j = part; j < n_left; j += 4) {
                            const uint32_t other = list[j];
                            greater += other > mine;
                            equal += other == mine;
                        }
                    }
                    greater += __shfl_xor_sync(0xFFFFFFFFu, greater, 1);
                    equal += __shfl_xor_sync(0xFFFFFFFFu, equal, 1);
                    greater += __shfl_xor_sync(0xFFFFFFFFu, greater, 2);
                    equal += __shfl_xor_sync(0xFFFFFFFFu, equal, 2);
                    if (e < n_left && part == 0 && greater < need && need <= greater + equal) {
                        sh.tau = mine;  // the need-th largest
                        sh.r = need - greater;
                    }
                }
                __syncthreads();
                prefix = sh.tau;
                need = sh.r;
                undecided = 0;
            }
        }
        tau = kmin + prefix;
        r = need;
    } else {
        __syncthreads();  // vals complete
    }

    // ---- S4 (emit) + S5: ascending keep list, compacted scores ------------------------------
    // every thread owns a contiguous run of slots (a multiple of 4, read as 128-bit vectors);
    // sure = sink / recent / above the threshold key, eq = at the threshold key
    const int run = ((l + kSelectThreads - 1) / kSelectThreads + 3) & ~3;
    const int i0 = min(l, tid * run), i1 = min(l, i0 + run);
    int n_sure = 0, n_eq = 0;
    for (int i = i0; i < i1; i += 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(vals + i);  // beyond l: stale, masked
        const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = i + c;
            if (j < i1) {
                if (j < lo || j >= hi) {
                    ++n_sure;
                } else {
                    const uint32_t key = order_key(w4[c]);
                    n_sure += key > tau;
                    n_eq += key == tau;
                }
            }
        }
    }
    if (tid == 0) sh.first_evicted = l;
    // both counts are at most 49152 < 2^16: one scan of the two packed into an unsigned word
    // (the scan adds ints; the sums are taken modulo 2^32, which is exact for unsigned fields)
    const uint32_t packed = (uint32_t)n_sure | ((uint32_t)n_eq << 16);
    const uint32_t before = block_inclusive_scan_u32(packed, sh.warp_sum) - packed;
    int eq_before = (int)(before >> 16);
    int pos = (int)(before & 0xFFFFu) + min(eq_before, r);
    int my_first_evicted = l;
    for (int i = i0; i < i1; i += 4) {
        const uint4 q = *reinterpret_cast<const uint4*>(vals + i);
        const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int j = i + c;
            if (j < i1) {
                bool kept = true;
                if (j >= lo && j < hi) {
                    const uint32_t key = order_key(w4[c]);
                    kept = key > tau;
                    if (key == tau) {
                        kept = eq_before < r;
                        ++eq_before;
                    }
                }
                if (kept) {
                    if (kStage) {
                        skeep[pos] = j;
                    } else {
                        keep[pos] = j;
                        if (p.compact_scores) scores[pos] = __uint_as_float(w4[c]);
                    }
                    ++pos;
                } else {
                    my_first_evicted = min(my_first_evicted, j);
                }
            }
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1)
        my_first_evicted = min(my_first_evicted, __shfl_xor_sync(0xFFFFFFFFu, my_first_evicted, d));
    if (lane == 0 && my_first_evicted < l) atomicMin(&sh.first_evicted, my_first_evicted);
    __syncthreads();
    const int first = sh.first_evicted;
    if (kStage) {  // coalesced copy-out of the list ...
        for (int j = tid; j < p.budget; j += kSelectThreads) keep[j] = skeep[j];
    }
    publish_keep_list(p, s, p.budget, first);  // the KV gather may start
    if (kStage && p.compact_scores) {  // ... and of the scores it selects
        for (int j = tid; j < p.budget; j += kSelectThreads) scores[j] = __uint_as_float(vals[skeep[j]]);
    }

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
                v[q] = j < p.budget ? serial[kStage ? skeep[j] : keep[j]] : 0;
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
    if (tid == 0 && p.compact_scores) p.live_len[s] = p.budget;  // ---- S7
}

}  // namespace

cudaError_t launch_select(const SelectParams& p, int n_streams, cudaStream_t st, bool overlap) {
    TraceRange trace("sirllm:decay_select");
    // scores (rounded up to whole 128-bit vectors, plus one vector of slack) + histogram
    // (+ the staged keep list when it fits)
    size_t smem = ((size_t)((p.capacity + 3) & ~3) + 4) * 4 + (size_t)kRadixBins * 4;
    DeviceProps dp;
    cudaError_t e = device_props(&dp);
    if (e != cudaSuccess) return e;
    const bool stage = smem + (size_t)p.threshold * 4 + 1024 <= (size_t)dp.smem_optin;
    if (stage) smem += (size_t)p.threshold * 4;
    static unsigned char allowed[2][kMaxDevices];
    auto kernel = stage ? select_kernel<true> : select_kernel<false>;
    e = allow_max_dynamic_smem((const void*)kernel, dp, allowed[stage ? 1 : 0]);
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
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

}  // namespace sirllm
