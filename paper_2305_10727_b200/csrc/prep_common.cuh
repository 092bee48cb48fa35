// Device and host helpers shared by the operand-preparation kernels (elementwise.cu, int4.cu).
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"
#include "quant_math.cuh"

namespace gpusq {

constexpr int kThreads = 256;

// ---- keep-two rule (Sec. 1 / Sec. 3.1; criterion: two largest magnitudes, lower index wins ties) ----
// Element i beats j when mag_i > mag_j, or when they are equal and i < j.  The
// two elements that win at least two of their three comparisons are kept.
// Returns the 4-bit keep mask (bit i = element i kept); exactly two bits set.
template <typename T>
__device__ __forceinline__ uint32_t keep_two_mask(T m0, T m1, T m2, T m3)
{
    const int b01 = m0 >= m1, b02 = m0 >= m2, b03 = m0 >= m3;
    const int b12 = m1 >= m2, b13 = m1 >= m3, b23 = m2 >= m3;
    const int w0 = b01 + b02 + b03;
    const int w1 = (1 - b01) + b12 + b13;
    const int w2 = (1 - b02) + (1 - b12) + b23;
    const int w3 = (1 - b03) + (1 - b13) + (1 - b23);
    return (uint32_t)(w0 >= 2) | ((uint32_t)(w1 >= 2) << 1) | ((uint32_t)(w2 >= 2) << 2) |
           ((uint32_t)(w3 >= 2) << 3);
}

// ------------------------------------------------------------ quantisation
// code = clamp(round-half-even(x / scale), -127, 127), IEEE division.
__device__ __forceinline__ int quant_code(float x, float scale, int qmax = 127)
{
    int q = __float2int_rn(__fdiv_rn(x, scale));
    return max(-qmax, min(qmax, q));
}

__device__ __forceinline__ float scale_from_amax(float amax, float qmax = 127.0f)
{
    return amax == 0.0f ? 1.0f : __fdiv_rn(amax, qmax);
}

__device__ __forceinline__ float block_max(float v, float *red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();  // red may still be read from a previous use
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) r = fmaxf(r, red[w]);
    return r;
}

constexpr int kMaxDevices = 64;
constexpr int kMaxPartials = 2048;   // workspace: one 32-bit partial maximum per block ...
constexpr int kWorkspaceExtra = 64;  // ... and, behind them, the control words of the one-launch kernel

__device__ __forceinline__ uint32_t absmax_bits8(uint4 v)
{
    // |binary16| as unsigned 15-bit patterns order like the magnitudes (no NaN expected)
    uint32_t a = __vmaxu2(v.x & 0x7FFF7FFFu, v.y & 0x7FFF7FFFu);
    uint32_t b = __vmaxu2(v.z & 0x7FFF7FFFu, v.w & 0x7FFF7FFFu);
    a = __vmaxu2(a, b);
    return max(a & 0xFFFFu, a >> 16);
}

static __global__ void __launch_bounds__(kThreads)
act_absmax_kernel(const uint4 *__restrict__ X, uint32_t *__restrict__ partial, int64_t vec8)
{
    __shared__ float red[kThreads / 32];
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t m = 0;
    for (; i + 3 * stride < vec8; i += 4 * stride) {
        uint4 v0 = __ldg(X + i), v1 = __ldg(X + i + stride), v2 = __ldg(X + i + 2 * stride),
              v3 = __ldg(X + i + 3 * stride);
        m = max(max(m, absmax_bits8(v0)), max(absmax_bits8(v1), max(absmax_bits8(v2), absmax_bits8(v3))));
    }
    for (; i < vec8; i += stride) m = max(m, absmax_bits8(__ldg(X + i)));
    // binary16 bit patterns below 0x8000 are exact small integers in binary32: reuse the float reduction
    const float r = block_max((float)m, red);
    if (threadIdx.x == 0) partial[blockIdx.x] = (uint32_t)r;
}

// eight binary16 values (16 bytes) -> eight INT8 codes (8 bytes); one exactness test for all eight
__device__ __forceinline__ float2 h2f(uint32_t h2) { return __half22float2(*reinterpret_cast<const __half2 *>(&h2)); }

template <bool kClamp>
__device__ __forceinline__ uint2 quant8_f16(uint4 v, const QuantScale &a)
{
    uint32_t differ = 0;
    const float2 f0 = h2f(v.x), f1 = h2f(v.y), f2 = h2f(v.z), f3 = h2f(v.w);
    float2 m0 = quant2_sums<kClamp>(f0, a, differ), m1 = quant2_sums<kClamp>(f1, a, differ);
    float2 m2 = quant2_sums<kClamp>(f2, a, differ), m3 = quant2_sums<kClamp>(f3, a, differ);
    if (differ != 0u || a.always_divide) {
        m0 = quant2_exact<kClamp>(f0, a);
        m1 = quant2_exact<kClamp>(f1, a);
        m2 = quant2_exact<kClamp>(f2, a);
        m3 = quant2_exact<kClamp>(f3, a);
    }
    return make_uint2(pack4_low_bytes(m0, m1), pack4_low_bytes(m2, m3));
}

inline int grid_for(int64_t items, int per_sm)
{
    int64_t blocks = ceil_div(items, kThreads);
    int64_t cap = (int64_t)num_sms() * per_sm;
    return (int)(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}


}  // namespace gpusq
