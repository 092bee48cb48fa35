// Exact INT8 quantisation arithmetic shared by the activation-quantisation kernels and the INT8
// epilogue of the GEMM kernel.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace gpusq {

// clamp(round-half-even(x / s), -qmax, qmax) as an INT8 code (qmax = 127; 7 for the 4-bit model),
// without the division and without the conversion unit.
//   Rounding: adding 1.5 * 2^23 in binary32 rounds to an integer with ties to even and leaves that
//   integer, as a two's-complement byte, in the low byte of the sum's bit pattern; as the addend of
//   a fused multiply-add it rounds the exact product x * c once.
//   Exactness: with c_lo < 1/s < c_hi (1/s perturbed by -+2^-21, far more than its own rounding
//   error and than the rounding error of the binary32 quotient), x/s and its binary32 rounding both
//   lie between x * c_lo and x * c_hi; rounding is monotonic, so if both products round to the same
//   integer, that integer is the code of the true quotient.  Otherwise (the quotient is within
//   ~1e-4 of k + 0.5), and when 1/s is not finite, the true division decides.
//   Clamping (kClamp, for a scale that was supplied): x is clamped to +-127 s beforehand, which
//   gives the same code because rounding is monotonic and the bounds are integers.  A scale
//   derived from the tensor's own maximum needs none (|x/s| <= 127 by construction).
constexpr float kRoundMagic = 12582912.0f;     // 1.5 * 2^23

struct QuantScale {
    float s;            // the scale
    float2 c_lo, c_hi;  // the bracketing reciprocals, duplicated for packed math
    float x_max;        // qmax s (kClamp)
    float qmax;         // largest code: 127, or 7 for the 4-bit model
    bool always_divide; // 1/s is not finite
};

__device__ __forceinline__ QuantScale make_quant_scale(float s, float qmax = 127.0f)
{
    QuantScale a;
    a.s = s;
    a.qmax = qmax;
    const float inv_s = __frcp_rn(s);
    const float lo = __fmul_rn(inv_s, 1.0f - 4.76837158203125e-7f), hi = __fmul_rn(inv_s, 1.0f + 4.76837158203125e-7f);
    a.c_lo = make_float2(lo, lo);
    a.c_hi = make_float2(hi, hi);
    a.x_max = __fmul_rn(s, qmax);
    a.always_divide = !(fabsf(inv_s) < 3.0e38f) || !(a.x_max < 3.0e38f);
    return a;
}

template <bool kClamp>
__device__ __forceinline__ float quant_exact_sum(float x, float s, float qmax)
{
    float r = __fdiv_rn(x, s);
    if (kClamp) r = fminf(fmaxf(r, -qmax), qmax);
    return r + kRoundMagic;
}

// two values -> the two sums whose low bytes are the codes; `differ` collects the bits in which the
// bracketing products disagree
template <bool kClamp>
__device__ __forceinline__ float2 quant2_sums(float2 f, const QuantScale &a, uint32_t &differ)
{
    if (kClamp) f = make_float2(fminf(fmaxf(f.x, -a.x_max), a.x_max), fminf(fmaxf(f.y, -a.x_max), a.x_max));
    const float2 magic = make_float2(kRoundMagic, kRoundMagic);
    const float2 lo = __ffma2_rn(f, a.c_lo, magic), hi = __ffma2_rn(f, a.c_hi, magic);
    differ |= (__float_as_uint(lo.x) ^ __float_as_uint(hi.x)) | (__float_as_uint(lo.y) ^ __float_as_uint(hi.y));
    return lo;
}

// the same two sums by the true division (the rare case the bracketing test cannot decide)
template <bool kClamp>
__device__ __forceinline__ float2 quant2_exact(float2 f, const QuantScale &a)
{
    return make_float2(quant_exact_sum<kClamp>(f.x, a.s, a.qmax), quant_exact_sum<kClamp>(f.y, a.s, a.qmax));
}

// four sums -> four codes in one word (lowest byte first)
__device__ __forceinline__ uint32_t pack4_low_bytes(float2 m01, float2 m23)
{
    const uint32_t p01 = __byte_perm(__float_as_uint(m01.x), __float_as_uint(m01.y), 0x0040);
    const uint32_t p23 = __byte_perm(__float_as_uint(m23.x), __float_as_uint(m23.y), 0x0040);
    return __byte_perm(p01, p23, 0x5410);
}

}  // namespace gpusq
