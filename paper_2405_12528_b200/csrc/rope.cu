// Positions inside the cache for keys stored AFTER rotary embedding (Section 3.3, the
// paragraph on positions): once compaction has moved the key of slot keep[j] to slot j, the
// key is turned by the angle of (j - keep[j]) positions so that it is again the key of a token
// at position j.  Rotary embedding (Su et al., RoFormer): pair i < d/2 of a row is a complex
// number turned by  position * theta_i,  theta_i = base^(-2i/d).
//
// Bound by HBM traffic on the moved rows of the K planes (read once, written once).  The
// angles depend on (stream, slot, pair) only, so a thread computes its eight (cos, sin) once -
// in fp64, the shift can be thousands of positions - and reuses them for every K plane of its
// group; per plane it moves two 16-byte vectors.  The rotation itself is also carried out in
// fp64 and every element is rounded ONCE, from fp64, to bf16/fp16: the result is the exactly
// rotated value rounded to nearest even (an fp32 rotation loses the low bits of the products
// where x cos - y sin cancels).  Widening to fp64 and the rounding back are done with integer
// operations on the bit patterns, so the arithmetic stays under the memory time.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "common.cuh"

namespace sirllm {

namespace {

constexpr int kRopeThreads = 128;

// Layout constants of the two storage types inside an fp64 bit pattern: a normal 16-bit value
// is its magnitude bits shifted up by kShift inside the double's high word with the exponent
// re-biased by kBias (1023 - 127 for bf16, 1023 - 15 for fp16).
template <bool kBf16>
struct Fmt {
    static constexpr int kShift = kBf16 ? 13 : 10;             // high-word bits below the 16-bit mantissa
    static constexpr uint32_t kBias = kBf16 ? 896u : 1008u;
    static constexpr uint32_t kExpMask = kBf16 ? 0x7F80u : 0x7C00u;
    static constexpr uint32_t kExpMax = kBf16 ? 255u : 31u;    // exponent field of inf / nan
    static constexpr int kExpPos = kBf16 ? 7 : 10;             // position of the exponent field
};

// 16-bit element -> fp64, exactly.  Normal values and zeros are widened with integer operations
// (conversions to and from fp64 are a quarter-rate pipe and would bound the kernel); subnormals,
// infinities and nans take the conversion instructions.
template <bool kBf16>
__device__ __forceinline__ double load16(uint32_t word, int hi) {
    using F = Fmt<kBf16>;
    const uint32_t h = hi ? word >> 16 : word & 0xFFFFu;
    const uint32_t mag = h & 0x7FFFu, ex = mag & F::kExpMask, sign = (h & 0x8000u) << 16;
    if (ex != 0 && ex != F::kExpMask)
        return __hiloint2double((int)(sign | ((mag << F::kShift) + (F::kBias << 20))), 0);
    if (mag == 0) return __hiloint2double((int)sign, 0);
    if (kBf16) return (double)__uint_as_float(h << 16);
    return (double)__half2float(__ushort_as_half((unsigned short)h));
}

// fp64 -> bit pattern of the nearest bf16 / fp16 value (ties to even), in one rounding.
// Results in the type's normal range are rounded on the bit pattern: the bits below the 16-bit
// mantissa are the low kShift bits of the high word and the whole low word, which only counts as
// "something below" (folded into bit 0); adding half-minus-one plus the kept mantissa's last bit
// carries into the kept part exactly when round-to-nearest-even rounds up, exponent included.
// Everything else (subnormal results, overflow, nan) goes through the fp64 adder: with E the
// exponent of v clamped at the smallest normal exponent, adding and subtracting 2^(E + 53 - p)
// leaves v rounded to p significant bits, exact in fp32 and in the 16-bit type.
template <bool kBf16>
__device__ __forceinline__ uint32_t round16(double v) {
    using F = Fmt<kBf16>;
    const uint32_t hi = (uint32_t)__double2hiint(v), lo = (uint32_t)__double2loint(v);
    const uint32_t mag = hi & 0x7FFFFFFFu, sign16 = (hi >> 16) & 0x8000u;
    const uint32_t t = (mag | (lo != 0u ? 1u : 0u)) + ((1u << (F::kShift - 1)) - 1u) + ((mag >> F::kShift) & 1u);
    const uint32_t ex = t >> 20;  // exponent after rounding (a carry may have raised it)
    if (ex > F::kBias && ex < F::kBias + F::kExpMax)
        return ((t >> F::kShift) - (F::kBias << F::kExpPos)) | sign16;
    if ((mag | lo) == 0u) return sign16;  // keeps the sign of a zero
    constexpr int p = kBf16 ? 8 : 11, emin = kBf16 ? -126 : -14;
    const int e = max((int)(hi & 0x7FF00000u), (emin + 1023) << 20);
    double r = v;
    if (e < 0x7FF00000) {  // finite
        const double big = __hiloint2double((int)(hi & 0x80000000u) | (e + ((53 - p) << 20)), 0);
        r = __dsub_rn(__dadd_rn(v, big), big);
    }
    const float f = __double2float_rn(r);  // exact (or inf / nan)
    uint32_t bits;
    if (kBf16)
        bits = __float_as_uint(f) >> 16;
    else
        bits = (uint32_t)__half_as_ushort(__float2half_rn(f));
    return (bits & 0x7FFFu) | sign16;
}
template <bool kBf16>
__device__ __forceinline__ uint32_t pack16(double lo, double hi) {
    return round16<kBf16>(lo) | (round16<kBf16>(hi) << 16);
}
// one pair turned by the angle whose cosine and sine are c and s: each product and each sum is
// a separately rounded fp64 operation
__device__ __forceinline__ void turn(double x, double y, double c, double s, double& xo, double& yo) {
    xo = __dsub_rn(__dmul_rn(x, c), __dmul_rn(y, s));
    yo = __dadd_rn(__dmul_rn(x, s), __dmul_rn(y, c));
}

template <bool kBf16>
__global__ void __launch_bounds__(kRopeThreads) rerotate_kernel(const RopeParams p) {
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
        const double theta = exp2(-(double)(2 * i) / (double)p.head_dim * p.log2_base);
        double sv, cv;
        sincos((double)delta * theta, &sv, &cv);
        cs[q] = cv;
        sn[q] = sv;
    }
    const size_t row_bytes = (size_t)p.head_dim * 2;
    const int pl0 = blockIdx.z * p.planes_per_group;
    const int pl1 = min(p.planes_per_stream, pl0 + p.planes_per_group);
    for (int pl = pl0; pl < pl1; ++pl) {
        char* row = p.k + (((size_t)s * p.planes_per_stream + pl) * p.capacity + j) * row_bytes;
        uint4* pa = reinterpret_cast<uint4*>(row + (p.layout == SIRLLM_ROPE_HALF ? 16 * u : 32 * u));
        uint4* pb = reinterpret_cast<uint4*>(
            row + (p.layout == SIRLLM_ROPE_HALF ? (size_t)p.head_dim + 16 * u : 32 * u + 16));
        const uint4 a = *pa, b = *pb;
        const uint32_t wa[4] = {a.x, a.y, a.z, a.w}, wb[4] = {b.x, b.y, b.z, b.w};
        uint32_t oa[4], ob[4];
        if (p.layout == SIRLLM_ROPE_HALF) {  // a holds x of pairs 8u..8u+7, b holds their y
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                double x[2], y[2];
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    turn(load16<kBf16>(wa[q], h), load16<kBf16>(wb[q], h), cs[2 * q + h],
                         sn[2 * q + h], x[h], y[h]);
                oa[q] = pack16<kBf16>(x[0], x[1]);
                ob[q] = pack16<kBf16>(y[0], y[1]);
            }
        } else {  // every 32-bit word is one pair (x, y): a = pairs 8u..8u+3, b = 8u+4..8u+7
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                double xo, yo;
                turn(load16<kBf16>(wa[q], 0), load16<kBf16>(wa[q], 1), cs[q], sn[q], xo, yo);
                oa[q] = pack16<kBf16>(xo, yo);
                turn(load16<kBf16>(wb[q], 0), load16<kBf16>(wb[q], 1), cs[4 + q], sn[4 + q], xo, yo);
                ob[q] = pack16<kBf16>(xo, yo);
            }
        }
        *pa = make_uint4(oa[0], oa[1], oa[2], oa[3]);
        *pb = make_uint4(ob[0], ob[1], ob[2], ob[3]);
    }
}

}  // namespace

cudaError_t launch_rerotate(const RopeParams& p, int n_streams, bool bf16, cudaStream_t st) {
    const int units = p.head_dim / 16;
    const int rows_per_block = kRopeThreads / units;
    const unsigned gx = (unsigned)((p.keep_stride + rows_per_block - 1) / rows_per_block);
    DeviceProps dp;
    cudaError_t e = device_props(&dp);
    if (e != cudaSuccess) return e;
    const int n_sm = dp.n_sm;
    // enough blocks to fill the GPU a few times over; each block reuses its angles over a group
    // of planes
    int64_t groups = ((int64_t)8 * n_sm + (int64_t)gx * n_streams - 1) / ((int64_t)gx * n_streams);
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
