// Keep-list generators for the paper's comparison policies (Section 4.1.1): StreamLLM,
// RandomLLM, IntervalLLM.  Each policy is turned into a synthetic per-slot rank that the
// selection kernel (sinks + top-k of the middle + recent window, ascending, ties to the lower
// slot) then resolves, so the three policies share the entropy policy's trigger, output
// format and K/V gather:
//   StreamLLM    rank = slot index            -> the most recent middle slots win
//   IntervalLLM  rank = 2*capacity - slot for slots that are a multiple of
//                interval = floor(live length / cache size) behind the sinks, else 0
//                -> the first k multiples win
//   RandomLLM    rank = 24-bit Philox4x32-10 draw keyed by (seed; slot, round, stream)
//                -> a uniformly random k-subset wins
// All ranks are integers below 2^24, exact in fp32.
#include "common.cuh"

namespace sirllm {

namespace {

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): word 0 of the output block.
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t c2,
                                                        uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0;
        c1 = lo1;
        c2 = n2;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}

__global__ void policy_rank_kernel(const PolicyParams p) {
    const int s = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) p.ones[s] = 1.0f;
    const int l = min(max(p.live_len[s], 0), p.capacity);
    if (i >= l) return;
    float rank = 0.f;
    if (p.policy == SIRLLM_POLICY_STREAM) {
        rank = (float)i;
    } else if (p.policy == SIRLLM_POLICY_INTERVAL) {
        const int interval = max(l / p.budget, 1);
        if (i >= p.n_sink && (i - p.n_sink) % interval == 0) rank = (float)(2 * p.capacity - i);
    } else {
        const uint32_t u = philox4x32_10_word0((uint32_t)i, (uint32_t)p.round,
                                               (uint32_t)(p.stream_base + s), 0u,
                                               (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
        rank = (float)(u >> 8);
    }
    p.ranks[(size_t)s * p.capacity + i] = rank;
}

}  // namespace

cudaError_t launch_policy_ranks(const PolicyParams& p, int n_streams, cudaStream_t st) {
    TraceRange trace("sirllm:keep_policy");
    dim3 grid((unsigned)((p.capacity + 255) / 256), (unsigned)n_streams);
    policy_rank_kernel<<<grid, 256, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace sirllm
