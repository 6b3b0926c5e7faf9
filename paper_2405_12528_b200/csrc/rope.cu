// Positions inside the cache for keys stored AFTER rotary embedding (Section 3.3, the
// paragraph on positions): once compaction has moved the key of slot keep[j] to slot j, the
// key is turned by the angle of (j - keep[j]) positions so that it is again the key of a token
// at position j.  Rotary embedding (Su et al., RoFormer): pair i < d/2 of a row is a complex
// number turned by  position * theta_i,  theta_i = base^(-2i/d).
//
// The traffic is the moved rows of the K planes, read once and written once.  The angles depend
// on (stream, slot, pair) only, so a thread computes its eight (cos, sin) once - in fp64, the
// shift can be thousands of positions - and reuses them for every K plane of its group; per
// plane it moves two 16-byte vectors.  The rotation itself is also carried out in fp64 and
// every element is rounded ONCE, from fp64, to bf16/fp16: the result is the exactly rotated
// value rounded to nearest even (an fp32 rotation loses the low bits of the products where
// x cos - y sin cancels).  The single rounding is obtained by truncating to fp32 with a sticky
// last bit and letting the packed fp32 -> 16-bit conversion round; the vectors of the next two
// planes are in flight while one plane is turned.  What limits the kernel is not DRAM but the
// four conversions between fp32 and fp64 per pair: they run on the quarter-rate conversion
// pipe, which the counters show as the busiest unit (about 0.8 of the copy bandwidth is reached).
#include <atomic>

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kRopeThreads = 128;
// six CTAs per SM (80 registers): measured best; eight spill the angles, five leave warps idle,
// and four pairs per thread (half the angle registers) doubled the sincos work for no gain
// (bf16; the fp16 conversions need more registers, so that variant is held to four CTAs)
constexpr int kRopeMinBlocks = 6;
constexpr int kRopeWaves = 3;  // grid size in resident waves

// 16-bit element -> fp64, exactly (two conversions; bf16 -> fp32 is a shift).
template <bool kBf16>
__device__ __forceinline__ double load16(uint32_t word, int hi) {
    if (kBf16) return (double)__uint_as_float(hi ? word & 0xFFFF0000u : word << 16);
    return (double)__half2float(__ushort_as_half((unsigned short)(hi ? word >> 16 : word & 0xFFFFu)));
}

// fp64 -> an fp32 value whose round-to-nearest-even conversion to bf16 / fp16 equals the
// direct, single rounding of the fp64 value: "round to odd".  The fp64 value is truncated to
// fp32 and, if any of the 29 mantissa bits that fp32 cannot hold was set, the last bit of the
// fp32 mantissa is forced to one; fp32 keeps at least two bits more than either 16-bit type, so
// the sticky last bit decides ties and near-ties exactly as the discarded bits would.
// This holds while the truncated value is a NORMAL fp32 number.  Below 2^-126 (possible for
// bf16 when a rotation cancels almost completely) the truncation loses more than 29 bits; the
// caller sees that on the result (|f| < 2^-126, zero included) and redoes the plane with
// to_odd_tiny().  fp16 needs no such care: everything below 2^-25 rounds to zero anyway.
__device__ __forceinline__ float to_odd(double v) {
    float f = __double2float_rz(v);
    if (((uint32_t)__double2loint(v) & 0x1FFFFFFFu) != 0u) f = __uint_as_float(__float_as_uint(f) | 1u);
    return f;
}
// The same for a value that may lie below the smallest normal fp32: such a value is rounded to
// bf16's precision by the fp64 adder (add and subtract 2^(-126 + 53 - 8), which leaves a
// multiple of bf16's smallest subnormal, exact in fp32), its sign kept when it rounds to zero.
__device__ __forceinline__ float to_odd_tiny(double v) {
    const uint32_t hi = (uint32_t)__double2hiint(v), lo = (uint32_t)__double2loint(v);
    const uint32_t mag = hi & 0x7FFFFFFFu;
    if (mag < 0x38100000u && (mag | lo) != 0u) {  // 0 < |v| < 2^-126
        const double big = __hiloint2double((int)((hi & 0x80000000u) | ((uint32_t)(-126 + 1023 + 53 - 8) << 20)), 0);
        return copysignf(__double2float_rn(__dsub_rn(__dadd_rn(v, big), big)), __uint_as_float(hi));
    }
    return to_odd(v);
}
// two fp32 values -> one word of two 16-bit elements (first argument in the low half)
template <bool kBf16>
__device__ __forceinline__ uint32_t pack16(float f0, float f1) {
    uint32_t out;
    if (kBf16)
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(out) : "f"(f1), "f"(f0));
    else
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(out) : "f"(f1), "f"(f0));
    return out;
}
// One pair turned by the angle whose cosine and sine are c and s, in fp64: one product rounded,
// the other fused into the sum (the result is within one rounding of the exact rotation; against
// four products and two sums rounded one by one it can differ in the last bit of the fp64 value,
// which reaches the 16-bit result only when that value sits within 2^-53 of a rounding boundary).
// Returned as round-to-odd fp32 values; `low` tracks the smallest magnitude handed out.
template <bool kTiny>
__device__ __forceinline__ void turn(double x, double y, double c, double s, float& xo, float& yo, float& low) {
    const double xr = __fma_rn(x, c, -__dmul_rn(y, s));
    const double yr = __fma_rn(x, s, __dmul_rn(y, c));
    if (kTiny) {
        xo = to_odd_tiny(xr);
        yo = to_odd_tiny(yr);
    } else {
        xo = to_odd(xr);
        yo = to_odd(yr);
        low = fminf(low, fminf(fabsf(xo), fabsf(yo)));
    }
}

// The two 16-byte vectors of one plane (8 pairs) turned and packed.  Returns the smallest
// magnitude among the 16 results (kTiny = false only).
template <bool kBf16, bool kTiny>
__device__ __forceinline__ float turn_vectors(const uint4 a, const uint4 b, const double (&cs)[8],
                                              const double (&sn)[8], int layout, uint4& out_a, uint4& out_b) {
    const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wb[4] = {b.x, b.y, b.z, b.w};
    uint32_t oa[4], ob[4];
    float low = 1.0f;
    if (layout == SIRLLM_ROPE_HALF) {  // a holds x of pairs 8u..8u+7, b holds their y
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float x[2], y[2];
#pragma unroll
            for (int h = 0; h < 2; ++h)
                turn<kTiny>(load16<kBf16>(wa[q], h), load16<kBf16>(wb[q], h), cs[2 * q + h], sn[2 * q + h],
                            x[h], y[h], low);
            oa[q] = pack16<kBf16>(x[0], x[1]);
            ob[q] = pack16<kBf16>(y[0], y[1]);
        }
    } else {  // every 32-bit word is one pair (x, y): a = pairs 8u..8u+3, b = 8u+4..8u+7
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float xo, yo;
            turn<kTiny>(load16<kBf16>(wa[q], 0), load16<kBf16>(wa[q], 1), cs[q], sn[q], xo, yo, low);
            oa[q] = pack16<kBf16>(xo, yo);
            turn<kTiny>(load16<kBf16>(wb[q], 0), load16<kBf16>(wb[q], 1), cs[4 + q], sn[4 + q], xo, yo, low);
            ob[q] = pack16<kBf16>(xo, yo);
        }
    }
    out_a = make_uint4(oa[0], oa[1], oa[2], oa[3]);
    out_b = make_uint4(ob[0], ob[1], ob[2], ob[3]);
    return low;
}

template <bool kBf16>
__global__ void __launch_bounds__(kRopeThreads, kBf16 ? kRopeMinBlocks : 4) rerotate_kernel(const RopeParams p) {
    const int units = p.head_dim / 16;  // threads per row: 8 pairs (two 16-byte vectors) each
    const int rows_per_block = kRopeThreads / units;
    const int r = threadIdx.x / units, u = threadIdx.x - r * units;
    if (r >= rows_per_block) return;
    const int s = blockIdx.y;
    const int j = blockIdx.x * rows_per_block + r;
    if (j >= min(p.n_keep[s], p.keep_stride)) return;
    const int delta = j - p.keep_idx[(size_t)s * p.keep_stride + j];
    if (delta == 0) return;  // the row did not move

    double cs[8], sn[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int i = 8 * u + q;
        double sv, cv;
        sincos((double)delta * p.theta[i], &sv, &cv);
        cs[q] = cv;
        sn[q] = sv;
    }
    const size_t row_bytes = (size_t)p.head_dim * 2;
    const int pl0 = blockIdx.z * p.planes_per_group;
    const int pl1 = min(p.planes_per_stream, pl0 + p.planes_per_group);
    const size_t plane_stride = (size_t)p.capacity * row_bytes;
    char* row0 = p.k + (((size_t)s * p.planes_per_stream + pl0) * p.capacity + j) * row_bytes;
    const size_t off_a = p.layout == SIRLLM_ROPE_HALF ? 16 * u : 32 * u;
    const size_t off_b = p.layout == SIRLLM_ROPE_HALF ? (size_t)p.head_dim + 16 * u : 32 * u + 16;
    constexpr int kAhead = 2;  // planes whose vectors are in flight while one is turned
    uint4 qa[kAhead], qb[kAhead];
#pragma unroll
    for (int d = 0; d < kAhead; ++d) {
        if (pl0 + d < pl1) {
            qa[d] = *reinterpret_cast<const uint4*>(row0 + d * plane_stride + off_a);
            qb[d] = *reinterpret_cast<const uint4*>(row0 + d * plane_stride + off_b);
        }
    }
    for (int base = pl0; base < pl1; base += kAhead) {
#pragma unroll
        for (int d = 0; d < kAhead; ++d) {
            const int pl = base + d;
            if (pl >= pl1) break;
            char* row = row0 + (size_t)(pl - pl0) * plane_stride;
            const uint4 a = qa[d], b = qb[d];
            if (pl + kAhead < pl1) {  // the plane that takes this buffer next
                qa[d] = *reinterpret_cast<const uint4*>(row + kAhead * plane_stride + off_a);
                qb[d] = *reinterpret_cast<const uint4*>(row + kAhead * plane_stride + off_b);
            }
            uint4 out_a, out_b;
            const float low = turn_vectors<kBf16, false>(a, b, cs, sn, p.layout, out_a, out_b);
            // bf16 only: a result below the smallest normal fp32 (an exact zero counts) sends the
            // plane's two vectors through the variant that rounds such values by the fp64 adder
            // (rare; it reads the vectors again rather than keep them in registers until here)
            if (kBf16 && low < 1.17549435e-38f)
                turn_vectors<kBf16, true>(__ldcg(reinterpret_cast<const uint4*>(row + off_a)),
                                          __ldcg(reinterpret_cast<const uint4*>(row + off_b)), cs, sn, p.layout,
                                          out_a, out_b);
            *reinterpret_cast<uint4*>(row + off_a) = out_a;
            *reinterpret_cast<uint4*>(row + off_b) = out_b;
        }
    }
}

}  // namespace

cudaError_t launch_rerotate(const RopeParams& p, int n_streams, bool bf16, cudaStream_t st) {
    TraceRange trace("sirllm:rerotate_keys");
    const int units = p.head_dim / 16;
    const int rows_per_block = kRopeThreads / units;
    const unsigned gx = (unsigned)((p.keep_stride + rows_per_block - 1) / rows_per_block);
    DeviceProps dp;
    cudaError_t e = device_props(&dp);
    if (e != cudaSuccess) return e;
    // blocks the device keeps resident at once, asked once per device and kernel variant
    static std::atomic<int> occ_cache[2][kMaxDevices];
    const bool slot = dp.device >= 0 && dp.device < kMaxDevices;
    int per_sm = slot ? occ_cache[bf16 ? 1 : 0][dp.device].load(std::memory_order_acquire) : 0;
    if (per_sm == 0) {
        e = bf16 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rerotate_kernel<true>, kRopeThreads, 0)
                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, rerotate_kernel<false>, kRopeThreads, 0);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorLaunchOutOfResources;
        if (slot) occ_cache[bf16 ? 1 : 0][dp.device].store(per_sm, std::memory_order_release);
    }
    // As many blocks as fit in kRopeWaves resident waves, not more: each block reuses its angles
    // over a group of planes, later waves even out SMs of different speed, and a grid that ends
    // just under a whole number of waves leaves no thin last wave (measured: grids of 2.0x and
    // 3.5x the resident blocks are 4-8 % slower than 2.7-2.9x; one exactly resident wave with
    // equal static shares 10 % slower).
    const int64_t resident = (int64_t)dp.n_sm * per_sm;
    int64_t groups = kRopeWaves * resident / ((int64_t)gx * n_streams);
    if (groups < 1) groups = 1;
    if (groups > p.planes_per_stream) groups = p.planes_per_stream;
    RopeParams q = p;
    q.planes_per_group = (int32_t)((p.planes_per_stream + groups - 1) / groups);
    const unsigned gz = (unsigned)((p.planes_per_stream + q.planes_per_group - 1) / q.planes_per_group);
    dim3 grid(gx, (unsigned)n_streams, gz);
    if (bf16)
        rerotate_kernel<true><<<grid, kRopeThreads, 0, st>>>(q);
    else
        rerotate_kernel<false><<<grid, kRopeThreads, 0, st>>>(q);
    return cudaGetLastError();
}

}  // namespace sirllm
