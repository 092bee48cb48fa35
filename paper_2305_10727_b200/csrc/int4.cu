// The INT4 model of the paper (Sec. 3.1: pair-wise structured sparsity at a granularity of 4:8; Sec. 3.4
// and Table 1: the INT4 compressed models) on a GPU whose tensor cores have no 4-bit integer kind.
//
// Storage is the paper's: four kept 4-bit codes per chunk of eight weights plus two 2-bit sub-chunk
// indices, 0.3125 bytes per weight.  Arithmetic runs on the INT8 2:4 path and is exact: codes in
// [-7, 7] are INT8 codes, and taking, inside every chunk of eight columns, the first elements of the
// four sub-chunks and then the second ones (column e -> (e % 2) * 4 + e / 2) turns "two of four
// sub-chunks kept" into "two of every four columns kept".  A GEMM does not change when weight and
// activation columns are permuted alike, so gpusq_expand48 writes the weight in that column order as
// an ordinary 2:4 INT8 operand, gpusq_quant_act4 (elementwise.cu) writes the 4-bit activation codes in the same
// order, and gpusq_pack24 + gpusq_spgemm_i8 do the rest.  The 2x math rate 4-bit tensor cores gave
// the paper's GPUs is not available; the storage saving and the results are.
#include "prep_common.cuh"

namespace gpusq {

// ------------------------------------------------------------------ prune48
// One chunk of eight weights per thread.  A sub-chunk weighs |a| + |b|, summed in binary64 so that the
// choice is taken on exact sums; the two heaviest stay (lower index on ties).
__global__ void __launch_bounds__(kThreads)
prune48_kernel(const float4 *__restrict__ W, float4 *Wp, uint8_t *mask, int64_t chunks)
{
    // W and Wp may be the same buffer: every thread reads its chunk before it writes it.
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < chunks; i += stride) {
        float4 a = __ldcs(W + 2 * i), b = __ldcs(W + 2 * i + 1);
        const uint32_t mk = keep_two_mask(fabs((double)a.x) + fabs((double)a.y), fabs((double)a.z) + fabs((double)a.w),
                                          fabs((double)b.x) + fabs((double)b.y), fabs((double)b.z) + fabs((double)b.w));
        if (!(mk & 1u)) a.x = a.y = 0.0f;
        if (!(mk & 2u)) a.z = a.w = 0.0f;
        if (!(mk & 4u)) b.x = b.y = 0.0f;
        if (!(mk & 8u)) b.z = b.w = 0.0f;
        __stcs(Wp + 2 * i, a);
        __stcs(Wp + 2 * i + 1, b);
        if (mask) mask[i] = (uint8_t)mk;
    }
}

// ------------------------------------------------------------ quant_weight4
// One block per output channel: max |w|, scale = max / 7, codes in [-7, 7] (INT8 containers).
__global__ void __launch_bounds__(kThreads)
quant_weight4_kernel(const float4 *__restrict__ Wp, uint32_t *__restrict__ Wq, float *__restrict__ w_scale, int N,
                     int K4)
{
    __shared__ float red[kThreads / 32];
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        const float4 *row = Wp + (int64_t)n * K4;
        float m = 0.0f;
        for (int k = threadIdx.x; k < K4; k += blockDim.x) {
            const float4 v = __ldg(row + k);
            m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
        const float s = scale_from_amax(block_max(m, red), 7.0f);
        if (threadIdx.x == 0) w_scale[n] = s;
        uint32_t *out = Wq + (int64_t)n * K4;
        for (int k = threadIdx.x; k < K4; k += blockDim.x) {
            const float4 v = __ldg(row + k);
            out[k] = (uint32_t)(quant_code(v.x, s, 7) & 0xFF) | ((uint32_t)(quant_code(v.y, s, 7) & 0xFF) << 8) |
                     ((uint32_t)(quant_code(v.z, s, 7) & 0xFF) << 16) | ((uint32_t)(quant_code(v.w, s, 7) & 0xFF) << 24);
        }
    }
}

// ---------------------------------------------------------------- compress48
// Two chunks (sixteen codes) per thread: 16 bytes in, four bytes of nibbles and one byte of indices out.
__device__ __forceinline__ void compress_chunk(uint32_t lo, uint32_t hi, uint32_t &nibbles, uint32_t &idx)
{
    // codes e0..e3 in lo, e4..e7 in hi; sub-chunk p = (e_2p, e_2p+1)
    auto mag = [](uint32_t w, int sh) { return abs((int)(int8_t)(w >> sh)) + abs((int)(int8_t)(w >> (sh + 8))); };
    const uint32_t mk = keep_two_mask(mag(lo, 0), mag(lo, 16), mag(hi, 0), mag(hi, 16));
    const uint32_t p0 = __ffs(mk) - 1, p1 = 31 - __clz(mk);
    const uint64_t all = ((uint64_t)hi << 32) | lo;
    const uint32_t a = (uint32_t)(all >> (16 * p0)) & 0xFFFFu, b = (uint32_t)(all >> (16 * p1)) & 0xFFFFu;
    // four codes -> four nibbles, the first in the lowest one
    nibbles = (a & 0xFu) | ((a >> 4) & 0xF0u) | ((b & 0xFu) << 8) | (((b >> 8) & 0xFu) << 12);
    idx = p0 | (p1 << 2);
}

__global__ void __launch_bounds__(kThreads)
compress48_kernel(const uint4 *__restrict__ Wq, uint32_t *__restrict__ vals, uint8_t *__restrict__ meta, int64_t pairs)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        const uint4 w = __ldg(Wq + i);
        uint32_t n0, n1, i0, i1;
        compress_chunk(w.x, w.y, n0, i0);
        compress_chunk(w.z, w.w, n1, i1);
        vals[i] = n0 | (n1 << 16);
        meta[i] = (uint8_t)(i0 | (i1 << 4));
    }
}

// ----------------------------------------------------------------- expand48
// The 4-bit operand as an ordinary 2:4 INT8 operand in the regrouped column order.  Per chunk the kept
// codes (a0, a1) of sub-chunk p0 and (b0, b1) of sub-chunk p1 become group 0 = first elements (a0 at
// position p0, b0 at p1) and group 1 = second elements (a1 at p0, b1 at p1): values a0 b0 a1 b1, and
// both groups carry the chunk's own index nibble.
__global__ void __launch_bounds__(kThreads)
expand48_kernel(const uint32_t *__restrict__ vals4, const uint8_t *__restrict__ meta4, uint2 *__restrict__ vals,
                uint16_t *__restrict__ meta, int64_t pairs)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        const uint32_t v = __ldg(vals4 + i), m = __ldg(meta4 + i);
        auto code = [](uint32_t nib) { return (uint32_t)((int32_t)(nib << 28) >> 28) & 0xFFu; };     // sign-extend 4 -> 8 bits
        auto chunk = [&](uint32_t n) {
            const uint32_t a0 = code(n & 0xF), a1 = code((n >> 4) & 0xF), b0 = code((n >> 8) & 0xF), b1 = code((n >> 12) & 0xF);
            return a0 | (b0 << 8) | (a1 << 16) | (b1 << 24);
        };
        vals[i] = make_uint2(chunk(v & 0xFFFFu), chunk(v >> 16));
        const uint32_t n0 = m & 0xF, n1 = m >> 4;
        meta[i] = (uint16_t)(n0 | (n0 << 4) | (n1 << 8) | (n1 << 12));
    }
}

}  // namespace gpusq

using namespace gpusq;

extern "C" {

int gpusq_prune48(const float *W, float *Wp, uint8_t *mask, int N, int K, void *stream)
{
    if (!W || !Wp) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(W, 16) || !aligned(Wp, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t chunks = (int64_t)N * (K / 8);
    prune48_kernel<<<grid_for(chunks, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const float4 *>(W), reinterpret_cast<float4 *>(Wp), mask, chunks);
    return launch_status();
}

int gpusq_quant_weight4(const float *Wp, int8_t *Wq, float *w_scale, int N, int K, void *stream)
{
    if (!Wp || !Wq || !w_scale) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 4) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wp, 16) || !aligned(Wq, 4)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int grid = N < num_sms() * 8 ? N : num_sms() * 8;
    quant_weight4_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const float4 *>(Wp), reinterpret_cast<uint32_t *>(Wq), w_scale, N, K / 4);
    return launch_status();
}

int gpusq_compress48(const int8_t *Wq, uint8_t *vals4, uint8_t *meta4, int N, int K, void *stream)
{
    if (!Wq || !vals4 || !meta4) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 16) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wq, 16) || !aligned(vals4, 4)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t pairs = (int64_t)N * (K / 16);
    compress48_kernel<<<grid_for(pairs, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint4 *>(Wq), reinterpret_cast<uint32_t *>(vals4), meta4, pairs);
    return launch_status();
}

int gpusq_expand48(const uint8_t *vals4, const uint8_t *meta4, int8_t *vals, uint8_t *meta, int N, int K, void *stream)
{
    if (!vals4 || !meta4 || !vals || !meta) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 16) return GPUSQ_ERR_SHAPE;
    if (!aligned(vals4, 4) || !aligned(vals, 8) || !aligned(meta, 2)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t pairs = (int64_t)N * (K / 16);
    expand48_kernel<<<grid_for(pairs, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint32_t *>(vals4), meta4, reinterpret_cast<uint2 *>(vals),
        reinterpret_cast<uint16_t *>(meta), pairs);
    return launch_status();
}

}  // extern "C"
