// HBM-bound operand-preparation kernels of libgpusq: 2:4 pruning, weight and
// activation quantisation, compression to values + metadata, decompression and
// packing for the tensor-core kernel.  One pass of coalesced 16-byte accesses
// per tensor; no shared-memory staging is needed (no reuse across threads).
#include <cuda_fp16.h>

#include <atomic>
#include <mutex>

#include "prep_common.cuh"

namespace gpusq {

// ------------------------------------------------------------------ prune24
__device__ __forceinline__ float4 prune_group(float4 v, uint32_t &mask)
{
    mask = keep_two_mask(fabsf(v.x), fabsf(v.y), fabsf(v.z), fabsf(v.w));
    v.x = (mask & 1u) ? v.x : 0.0f;
    v.y = (mask & 2u) ? v.y : 0.0f;
    v.z = (mask & 4u) ? v.z : 0.0f;
    v.w = (mask & 8u) ? v.w : 0.0f;
    return v;
}

template <int UNROLL>
__global__ void __launch_bounds__(kThreads)
prune24_kernel(const float4 *__restrict__ W, float4 *Wp, uint8_t *mask, int64_t groups)
{
    // W and Wp may be the same buffer: every thread reads a group before it writes it.
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + (UNROLL - 1) * stride < groups; i += UNROLL * stride) {
        float4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = __ldcs(W + i + u * stride);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            uint32_t mk;
            float4 o = prune_group(v[u], mk);
            __stcs(Wp + i + u * stride, o);
            if (mask) mask[i + u * stride] = (uint8_t)mk;
        }
    }
    for (; i < groups; i += stride) {
        uint32_t mk;
        float4 o = prune_group(__ldcs(W + i), mk);
        __stcs(Wp + i, o);
        if (mask) mask[i] = (uint8_t)mk;
    }
}

// One block per output channel (row): pass 1 finds max|w|, pass 2 re-reads the
// row (L1/L2 resident: a row is at most 20 KB) and writes four codes per store.
__global__ void __launch_bounds__(kThreads)
quant_weight_kernel(const float4 *__restrict__ Wp, uint32_t *__restrict__ Wq,
                    float *__restrict__ w_scale, int N, int K4)
{
    __shared__ float red[kThreads / 32];
    for (int n = blockIdx.x; n < N; n += gridDim.x) {
        const float4 *row = Wp + (int64_t)n * K4;
        float m = 0.0f;
        for (int k = threadIdx.x; k < K4; k += blockDim.x) {
            float4 v = __ldg(row + k);
            m = fmaxf(m, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
        const float s = scale_from_amax(block_max(m, red));
        if (threadIdx.x == 0) w_scale[n] = s;
        uint32_t *out = Wq + (int64_t)n * K4;
        for (int k = threadIdx.x; k < K4; k += blockDim.x) {
            float4 v = __ldg(row + k);
            uint32_t c = (uint32_t)(quant_code(v.x, s) & 0xFF) | ((uint32_t)(quant_code(v.y, s) & 0xFF) << 8) |
                         ((uint32_t)(quant_code(v.z, s) & 0xFF) << 16) |
                         ((uint32_t)(quant_code(v.w, s) & 0xFF) << 24);
            out[k] = c;
        }
    }
}

// ---------------------------------------------------------------- compress
// One group = four INT8 codes in a 32-bit word.  Returns the two kept codes
// (low 16 bits, lower position first) and the metadata nibble i0 | i1 << 2.
__device__ __forceinline__ void compress_group(uint32_t w, uint32_t &pair, uint32_t &nib)
{
    const int c0 = (int8_t)(w & 0xFF), c1 = (int8_t)((w >> 8) & 0xFF);
    const int c2 = (int8_t)((w >> 16) & 0xFF), c3 = (int8_t)(w >> 24);
    const uint32_t mk = keep_two_mask(abs(c0), abs(c1), abs(c2), abs(c3));
    const uint32_t i0 = __ffs(mk) - 1;          // lowest kept position
    const uint32_t i1 = 31 - __clz(mk);         // highest kept position
    pair = ((w >> (8 * i0)) & 0xFF) | (((w >> (8 * i1)) & 0xFF) << 8);
    nib = i0 | (i1 << 2);
}

// Four groups (16 codes) per thread: 16-byte load, 8-byte + 2-byte stores.  K % 16 == 0.
__global__ void __launch_bounds__(kThreads)
compress24_x4_kernel(const uint4 *__restrict__ Wq, uint2 *__restrict__ vals,
                     uint16_t *__restrict__ meta, int64_t quads)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < quads; i += stride) {
        const uint4 w = __ldg(Wq + i);
        uint32_t p0, p1, p2, p3, n0, n1, n2, n3;
        compress_group(w.x, p0, n0);
        compress_group(w.y, p1, n1);
        compress_group(w.z, p2, n2);
        compress_group(w.w, p3, n3);
        vals[i] = make_uint2(p0 | (p1 << 16), p2 | (p3 << 16));
        meta[i] = (uint16_t)(n0 | (n1 << 4) | (n2 << 8) | (n3 << 12));
    }
}

// Two groups per thread for rows whose length is a multiple of 8 only.
__global__ void __launch_bounds__(kThreads)
compress24_x2_kernel(const uint2 *__restrict__ Wq, uint32_t *__restrict__ vals,
                     uint8_t *__restrict__ meta, int64_t pairs)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        const uint2 w = __ldg(Wq + i);
        uint32_t p0, p1, n0, n1;
        compress_group(w.x, p0, n0);
        compress_group(w.y, p1, n1);
        vals[i] = p0 | (p1 << 16);
        meta[i] = (uint8_t)(n0 | (n1 << 4));
    }
}

__device__ __forceinline__ uint32_t decompress_group(uint32_t pair, uint32_t nib)
{
    const uint32_t i0 = nib & 3, i1 = (nib >> 2) & 3;
    uint32_t w = (pair & 0xFF) << (8 * i0);
    w = (w & ~(0xFFu << (8 * i1))) | (((pair >> 8) & 0xFF) << (8 * i1));
    return w;
}

__global__ void __launch_bounds__(kThreads)
decompress24_kernel(const uint32_t *__restrict__ vals, const uint8_t *__restrict__ meta,
                    uint2 *__restrict__ Wq, int64_t pairs)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        const uint32_t v = __ldg(vals + i);
        const uint32_t m = __ldg(meta + i);
        Wq[i] = make_uint2(decompress_group(v & 0xFFFF, m & 0xF), decompress_group(v >> 16, m >> 4));
    }
}

// -------------------------------------------------------------------- pack
// Np = N rounded up to 256 (a CTA pair's features), Kp = K rounded up to 128.
// Values: [Np, Kp/2] zero padded.  Metadata: [Np/128][Kp/128][128 rows][16 bytes],
// i.e. for each 128-row x 128-column block of W the 16 metadata bytes of a row
// are contiguous and rows follow each other: the 2 KB block is what one
// tcgen05.cp 128x128b instruction moves into tensor memory.  Padding groups
// get the well-formed nibble 0x4 (positions 0 and 1); their values are zero.
__global__ void __launch_bounds__(kThreads)
pack24_kernel(const int8_t *__restrict__ vals, const uint8_t *__restrict__ meta,
              uint8_t *__restrict__ packed, int N, int K, int Np, int Kp)
{
    const int row_chunks = Kp / 32;                       // 16-byte chunks per padded value row
    const int64_t val_chunks = (int64_t)Np * row_chunks;
    const int kt = Kp / 128;
    const int64_t meta_chunks = (int64_t)Np * kt;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    uint8_t *meta_out = packed + (int64_t)Np * (Kp / 2);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < val_chunks + meta_chunks;
         i += stride) {
        uint32_t w[4];
        if (i < val_chunks) {
            const int n = (int)(i / row_chunks), c = (int)(i % row_chunks);
            const uint32_t *src = reinterpret_cast<const uint32_t *>(vals + (int64_t)n * (K / 2));
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int byte = 16 * c + 4 * j;          // K/2 is a multiple of 4
                w[j] = (n < N && byte < K / 2) ? __ldg(src + byte / 4) : 0u;
            }
            *reinterpret_cast<uint4 *>(packed + i * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            const int64_t j = i - val_chunks;             // (tile_n, tile_k, r)
            const int r = (int)(j % 128);
            const int tk = (int)((j / 128) % kt);
            const int tn = (int)(j / (128 * (int64_t)kt));
            const int n = tn * 128 + r;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t word = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int byte = 16 * tk + 4 * q + b;
                    const uint32_t v = (n < N && byte < K / 8) ? meta[(int64_t)n * (K / 8) + byte] : 0x44u;
                    word |= v << (8 * b);
                }
                w[q] = word;
            }
            *reinterpret_cast<uint4 *>(meta_out + j * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// ------------------------------------------------- FP16 2:4 sparse model (Sec. 3.1, Sec. 3.4)
// Pruned FP32 weight -> binary16 (round to nearest even) -> the two kept values of every group of
// four plus the metadata nibble, positions re-derived from the binary16 magnitudes with the keep-two
// rule.  Two groups (eight weights) per thread: 32 bytes in, 8 + 1 bytes out.
__global__ void __launch_bounds__(kThreads)
compress24_f16_kernel(const float4 *__restrict__ Wp, uint2 *__restrict__ vals, uint8_t *__restrict__ meta,
                      int64_t pairs)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        uint32_t kept[2], nib[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const float4 w = __ldg(Wp + 2 * i + h);
            const __half q[4] = {__float2half_rn(w.x), __float2half_rn(w.y), __float2half_rn(w.z),
                                 __float2half_rn(w.w)};
            uint32_t bits[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) bits[j] = __half_as_ushort(q[j]);
            // |binary16| patterns order like the magnitudes
            const uint32_t mask = keep_two_mask(bits[0] & 0x7FFFu, bits[1] & 0x7FFFu, bits[2] & 0x7FFFu,
                                                bits[3] & 0x7FFFu);
            const uint32_t i0 = __ffs(mask) - 1, i1 = 31 - __clz(mask);
            kept[h] = bits[i0] | (bits[i1] << 16);
            nib[h] = i0 | (i1 << 2);
        }
        vals[i] = make_uint2(kept[0], kept[1]);
        meta[i] = (uint8_t)(nib[0] | (nib[1] << 4));
    }
}

// Np = N rounded up to 256, Kp = K rounded up to 128.  Values: [Np, Kp/2] binary16, zero padded.
// Metadata: [Np/128][Kp/128] blocks of 2 KB, one per 128 rows x 128 columns of W, in the arrangement
// the tensor core expects for 16-bit operands after a tcgen05.cp 128x128b: the byte that holds columns
// 8 kb .. 8 kb + 7 of local row m sits at
//   256 (m / 16) + 128 ((kb / 2) % 2) + 16 (m % 8) + 4 (kb / 4) + 2 ((m / 8) % 2) + kb % 2.
// Padding groups get the well-formed nibble 0x4 (positions 0 and 1); their values are zero.
__global__ void __launch_bounds__(kThreads)
pack24_f16_kernel(const uint16_t *__restrict__ vals, const uint8_t *__restrict__ meta,
                  uint8_t *__restrict__ packed, int N, int K, int Np, int Kp)
{
    const int row_chunks = Kp / 16;                       // 16-byte chunks (8 values) per padded value row
    const int64_t val_chunks = (int64_t)Np * row_chunks;
    const int kt = Kp / 128;
    const int64_t meta_bytes = (int64_t)Np * (Kp / 8);
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    uint8_t *meta_out = packed + (int64_t)Np * Kp;        // Kp / 2 values of two bytes per row
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < val_chunks + meta_bytes; i += stride) {
        if (i < val_chunks) {
            const int n = (int)(i / row_chunks), c = (int)(i % row_chunks);
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int v = 8 * c + 2 * j;              // K / 2 is a multiple of 4: pairs do not straddle the end
                w[j] = (n < N && v < K / 2)
                           ? __ldg(reinterpret_cast<const uint32_t *>(vals + (int64_t)n * (K / 2)) + v / 2) : 0u;
            }
            *reinterpret_cast<uint4 *>(packed + i * 16) = make_uint4(w[0], w[1], w[2], w[3]);
        } else {
            const int64_t j = i - val_chunks;             // one destination byte: (tile_n, tile_k, offset)
            const int off = (int)(j % 2048);
            const int tk = (int)((j / 2048) % kt);
            const int tn = (int)(j / (2048 * (int64_t)kt));
            const int m = 16 * (off >> 8) + 8 * ((off >> 1) & 1) + ((off >> 4) & 7);
            const int kb = 4 * ((off >> 2) & 3) + 2 * ((off >> 7) & 1) + (off & 1);
            const int n = tn * 128 + m, byte = 16 * tk + kb;
            meta_out[j] = (n < N && byte < K / 8) ? __ldg(meta + (int64_t)n * (K / 8) + byte) : (uint8_t)0x44;
        }
    }
}

// --------------------------------------------------------------- quant_act
// The 4-bit model (int4.cu) wants the codes of every eight columns in the order e0 e2 e4 e6 | e1 e3 e5 e7.
__device__ __forceinline__ uint2 regrouped(uint2 q, int regroup)
{
    return regroup ? make_uint2(__byte_perm(q.x, q.y, 0x6420), __byte_perm(q.x, q.y, 0x7531)) : q;
}

// n_partials > 0: the scale is derived from the partial maxima and written to
// *x_scale by block 0; absmax != NULL: it is derived from *absmax (the tensor's maximum magnitude,
// left there by the kernel that produced X) and written; otherwise *x_scale is read.
__global__ void __launch_bounds__(kThreads)
act_quant_kernel(const uint4 *__restrict__ X, uint2 *__restrict__ Xq, float *x_scale,
                 const uint32_t *__restrict__ partial, int n_partials, int64_t vec8,
                 const float *__restrict__ absmax = nullptr, float qmax = 127.0f, int regroup = 0)
{
    __shared__ float red[kThreads / 32];
    float s;
    if (absmax) {
        s = scale_from_amax(__ldg(absmax), qmax);
        if (blockIdx.x == 0 && threadIdx.x == 0) *x_scale = s;
    } else if (n_partials > 0) {
        uint32_t m = 0;
        for (int i = threadIdx.x; i < n_partials; i += blockDim.x) m = max(m, __ldg(partial + i));
        const uint32_t bits = (uint32_t)block_max((float)m, red);
        const float amax = __half2float(__ushort_as_half((unsigned short)bits));
        s = scale_from_amax(amax, qmax);
        if (blockIdx.x == 0 && threadIdx.x == 0) *x_scale = s;
    } else {
        s = *x_scale;
    }
    const QuantScale a = make_quant_scale(s, qmax);
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + stride < vec8; i += 2 * stride) {
        const uint4 v0 = __ldg(X + i), v1 = __ldg(X + i + stride);
        Xq[i] = regrouped(quant8_f16<true>(v0, a), regroup);
        Xq[i + stride] = regrouped(quant8_f16<true>(v1, a), regroup);
    }
    for (; i < vec8; i += stride) Xq[i] = regrouped(quant8_f16<true>(__ldg(X + i), a), regroup);
}

// ---- patch embedding (Sec. 3.3): quantise an image batch and lay it out as the GEMM's rows ----
// The convolution with kernel = stride = P is the GEMM of patch rows with the flattened weight.
// Xq[t, k] = code(img[b, c, ty P + py, tx P + px]) with t = (b, ty, tx) and k = (c P + py) P + px;
// columns K .. Kp-1 are written as zeros.  A thread makes kVec neighbouring codes of one row: kVec
// divides P and W, so they are kVec neighbouring pixels of one patch row, loaded with one aligned
// vector load.  Consecutive threads write consecutive bytes of Xq; the reads are 2 kVec-byte pieces
// whose 32-byte sectors are shared by the threads of neighbouring patches.
// floor(n / d) for n < 2^31 as one multiply-high and a shift.  With 2^(s-1) < d <= 2^s and
// m = ceil(2^(31+s) / d) < 2^32, m d exceeds 2^(31+s) by less than d <= 2^s, so n m / 2^(31+s) exceeds
// n / d by less than n / 2^31 / d < 1 / d: not enough to reach the next integer.
struct FastDiv {
    uint32_t d, m, sh;
};

static FastDiv make_fast_div(uint32_t d)
{
    FastDiv f = {d, 0u, 0u};
    if (d > 1) {
        uint32_t s = 0;
        while (((uint64_t)1 << s) < d) ++s;
        f.m = (uint32_t)((((uint64_t)1 << (31 + s)) + d - 1) / d);
        f.sh = s - 1;
    }
    return f;
}

__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv &f)
{
    return f.d == 1 ? n : __umulhi(n, f.m) >> f.sh;
}

struct PatchGeom {
    int C, H, W, P;
    int Tx, T;      // patches per image row, per image
    int K, Kp;      // C P P, and the padded row length of Xq
    FastDiv by_row, by_pp, by_p, by_t, by_tx;   // divisors Kp / kVec, P P, P, T, Tx
};

template <int kVec>
__global__ void __launch_bounds__(kThreads)
patch_quant_kernel(const __half *__restrict__ img, int8_t *__restrict__ Xq, float *x_scale,
                   const uint32_t *__restrict__ partial, int n_partials, const PatchGeom g, uint32_t items)
{
    __shared__ float red[kThreads / 32];
    float s;
    if (n_partials > 0) {
        uint32_t m = 0;
        for (int i = threadIdx.x; i < n_partials; i += blockDim.x) m = max(m, __ldg(partial + i));
        const uint32_t bits = (uint32_t)block_max((float)m, red);
        s = scale_from_amax(__half2float(__ushort_as_half((unsigned short)bits)));
        if (blockIdx.x == 0 && threadIdx.x == 0) *x_scale = s;
    } else {
        s = *x_scale;
    }
    const QuantScale a = make_quant_scale(s);
    // item i -> where its codes go, and where its pixels are (nullptr in the padding columns);
    // every dividend is below `items` < 2^31
    auto locate = [&](uint32_t i, int8_t *&dst) -> const __half * {
        const uint32_t t = fast_div(i, g.by_row);
        const uint32_t k0 = (i - t * g.by_row.d) * kVec;
        dst = Xq + (int64_t)t * g.Kp + k0;
        if (k0 >= (uint32_t)g.K) return nullptr;
        const uint32_t c = fast_div(k0, g.by_pp), rem = k0 - c * g.by_pp.d;
        const uint32_t py = fast_div(rem, g.by_p), px = rem - py * g.by_p.d;
        const uint32_t b = fast_div(t, g.by_t), r = t - b * g.by_t.d;
        const uint32_t ty = fast_div(r, g.by_tx), tx = r - ty * g.by_tx.d;
        return img + (((int64_t)b * g.C + c) * g.H + (ty * g.P + py)) * g.W + (tx * g.P + px);
    };
    auto fetch = [&](const __half *src) -> uint4 {         // kVec binary16 values, zero where there are none
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (src) {
            if (kVec == 8) {
                v = __ldg(reinterpret_cast<const uint4 *>(src));
            } else if (kVec == 4) {
                const uint2 h = __ldg(reinterpret_cast<const uint2 *>(src));
                v.x = h.x;
                v.y = h.y;
            } else {
                v.x = __ldg(reinterpret_cast<const uint32_t *>(src));
            }
        }
        return v;
    };
    auto emit = [&](uint4 v, int8_t *dst) {                // code(0) = 0: the padding needs no special case
        if (kVec == 8) {
            *reinterpret_cast<uint2 *>(dst) = quant8_f16<true>(v, a);
        } else {
            uint32_t differ = 0;
            const float2 f0 = h2f(v.x), f1 = h2f(v.y);
            float2 m0 = quant2_sums<true>(f0, a, differ), m1 = quant2_sums<true>(f1, a, differ);
            if (differ != 0u || a.always_divide) {
                m0 = quant2_exact<true>(f0, a);
                m1 = quant2_exact<true>(f1, a);
            }
            const uint32_t codes = pack4_low_bytes(m0, m1);
            if (kVec == 4) *reinterpret_cast<uint32_t *>(dst) = codes;
            else *reinterpret_cast<uint16_t *>(dst) = (uint16_t)codes;
        }
    };
    const uint32_t stride = gridDim.x * blockDim.x;
    uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    for (; i < items && stride < items - i; i += 2 * stride) {       // two items in flight per thread
        int8_t *d0, *d1;
        const __half *s0 = locate(i, d0), *s1 = locate(i + stride, d1);
        const uint4 v0 = fetch(s0), v1 = fetch(s1);
        emit(v0, d0);
        emit(v1, d1);
    }
    if (i < items) {
        int8_t *d0;
        const __half *s0 = locate(i, d0);
        emit(fetch(s0), d0);
    }
}

// ---- one-launch activation quantisation (scale computed from the tensor) ----
// A cooperative grid of one 1024-thread CTA per SM.  Each CTA owns a contiguous slice of X:
//   1. bulk-asynchronous copies bring as much of the slice as fits into shared memory (sixteen-KB
//      pieces, each completing on its own mbarrier, all in flight at once); what does not fit is
//      read with plain loads, last, so that it is still in L2 in step 3.  The threads take the
//      maximum |x| of every piece as it lands;
//   2. grid-wide maximum: the CTA merges its maximum into a word of the workspace, counts itself in
//      and polls, with a bounded wait, until every CTA has been counted;
//   3. quantises the slice, from shared memory where it was kept, and writes the codes.
// So X crosses HBM once when a slice fits (up to 192 KB per SM, 28 MB per tensor) and there is one
// launch instead of two.
// All or nothing: block 0 sets *x_scale to NaN on entry; the CTA that is last to finish step 2 (a
// counter, off the critical path) writes the real scale and puts the control words back to zero.  A
// CTA whose wait expires records GPUSQ_ERR_TIMEOUT in the status word and returns without
// quantising; the scale then stays NaN and the workspace has to be zero-filled again.
constexpr int kFusedThreads = 1024;
constexpr int kPieceVecs = 1024;                                 // 16-byte vectors per bulk copy (16 KB): one per thread
constexpr int kMaxPieces = 12;
constexpr int kFusedCacheVecs = kPieceVecs * kMaxPieces;         // vectors kept per CTA (192 KB)
constexpr int kFusedSmemBytes = kFusedCacheVecs * 16;
constexpr int kWsDone = kMaxPartials;                            // workspace words: CTAs past the barrier ...
constexpr int kWsStatus = kMaxPartials + 1;                      // ... status (0 or GPUSQ_ERR_TIMEOUT) ...
constexpr int kWsBarrier = kMaxPartials + 2;                     // ... and the 8-byte word {arrivals, maximum}
static std::atomic<unsigned long long> g_grid_wait_ns{2000000000ull};    // bound of the waits below (2 s)
static std::atomic<int> g_withhold_slot{0};                      // test hook: the last CTA does not publish

__device__ __forceinline__ uint64_t globaltimer_now()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool mbar_try_wait_parity0(uint32_t bar)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred P;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], 0, 1000;\n"
        "selp.u32 %0, 1, 0, P;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar)
        : "memory");
    return ok != 0;
}

__global__ void __launch_bounds__(kFusedThreads, 1)
act_quant_fused_kernel(const uint4 *__restrict__ X, uint2 *__restrict__ Xq, float *x_scale,
                       uint32_t *ws, int64_t vec8, unsigned long long wait_ns, int withhold, float qmax, int regroup)
{
    extern __shared__ __align__(128) uint4 cache[];
    __shared__ float red[kFusedThreads / 32];
    __shared__ __align__(8) uint64_t piece_bar[kMaxPieces];
    __shared__ uint32_t gave_up;
    const int64_t per = (vec8 + gridDim.x - 1) / gridDim.x;
    const int64_t lo = (int64_t)blockIdx.x * per;
    const int64_t hi = lo + per < vec8 ? lo + per : vec8;
    const int tid = threadIdx.x;

    // The slice in 32-bit terms: n vectors from Xs; the first n_kept of them stay in shared memory.
    const int n = hi > lo ? (int)(hi - lo) : 0;             // host side: per < 2^31
    const int n_kept = n < kFusedCacheVecs ? n : kFusedCacheVecs;
    const int pieces = (n_kept + kPieceVecs - 1) / kPieceVecs;
    const uint4 *Xs = X + lo;
    uint2 *Xqs = Xq + lo;

    if (tid == 0) {
        for (int c = 0; c < pieces; ++c)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"((uint32_t)__cvta_generic_to_shared(&piece_bar[c])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        gave_up = 0;
    }
    __syncthreads();
    // the previous kernel of the stream (a producer of X, or a user of the workspace) is complete from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the next kernel of the stream may be scheduled as soon as CTAs of this grid make room
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0 && tid == 0) *x_scale = __int_as_float(0x7FC00000);

    // 1. the slice into shared memory, all pieces in flight at once
    if (tid == 0) {
        for (int c = 0; c < pieces; ++c) {
            const int v0 = c * kPieceVecs;
            const uint32_t bytes = (uint32_t)((n_kept - v0 < kPieceVecs ? n_kept - v0 : kPieceVecs) * 16);
            const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&piece_bar[c]);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             (uint32_t)__cvta_generic_to_shared(cache + v0)),
                         "l"(Xs + v0), "r"(bytes), "r"(bar)
                         : "memory");
        }
    }
    // what does not fit: maximum only, plain loads that leave the lines in L2 for step 3
    uint32_t m = 0;
    int i = n_kept + tid;
    for (; i + 3 * kFusedThreads < n; i += 4 * kFusedThreads) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldg(Xs + i + u * kFusedThreads);
#pragma unroll
        for (int u = 0; u < 4; ++u) m = max(m, absmax_bits8(v[u]));
    }
    for (; i < n; i += kFusedThreads) m = max(m, absmax_bits8(__ldg(Xs + i)));
    // the pieces as they land: thread t looks at vector t of each
    const uint64_t t0 = globaltimer_now();
    bool ok = true;
    for (int c = 0; c < pieces && ok; ++c) {
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&piece_bar[c]);
        while (!mbar_try_wait_parity0(bar)) {
            if (globaltimer_now() - t0 > wait_ns) {
                ok = false;
                break;
            }
        }
        const int v = c * kPieceVecs + tid;
        if (ok && v < n_kept) m = max(m, absmax_bits8(cache[v]));
    }
    if (!ok) gave_up = 1;                                    // benign race: every writer writes 1
    const uint32_t mine = (uint32_t)block_max((float)m, red);            // has the block-wide barriers

    // 2. grid-wide maximum.  One 8-byte word holds {arrivals, maximum}: a CTA first merges its maximum,
    // then counts itself in, so a single 8-byte read that sees every arrival also sees the final
    // maximum; each CTA has one poll in flight at a time, all on one line.
    uint32_t *bar_word = ws + kWsBarrier;
    uint32_t seen = 0;
    if (tid == 0 && !gave_up) {
        if (!(withhold && blockIdx.x == gridDim.x - 1)) {
            atomicMax(bar_word + 1, mine);
            __threadfence();
            atomicAdd(bar_word, 1u);
        }
        for (uint32_t it = 1;; ++it) {
            const uint2 word = __ldcv(reinterpret_cast<const uint2 *>(bar_word));
            if (word.x >= gridDim.x) {
                seen = word.y;
                break;
            }
            if ((it & 63u) == 0u && globaltimer_now() - t0 > wait_ns) {
                gave_up = 1;
                break;
            }
        }
    }
    const uint32_t all = (uint32_t)block_max((float)seen, red);
    if (gave_up) {
        if (tid == 0) atomicExch(ws + kWsStatus, (uint32_t)GPUSQ_ERR_TIMEOUT);
        // bulk copies that may still be in flight write into this CTA's shared memory: wait for them (bounded)
        if (tid == 0) {
            const uint64_t t1 = globaltimer_now();
            for (int c = 0; c < pieces; ++c) {
                const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&piece_bar[c]);
                while (!mbar_try_wait_parity0(bar) && globaltimer_now() - t1 < wait_ns) {
                }
            }
        }
        __syncthreads();
        return;
    }
    if (tid == 0) {
        // the last CTA past the barrier: nobody polls any more, so the workspace goes back to zero and
        // the scale, which tells the caller that every CTA came through, is written
        __threadfence();
        if (atomicAdd(ws + kWsDone, 1u) == gridDim.x - 1) {
            __stcg(reinterpret_cast<uint2 *>(bar_word), make_uint2(0u, 0u));
            __stcg(ws + kWsDone, 0u);
            *x_scale = scale_from_amax(__half2float(__ushort_as_half((unsigned short)all)), qmax);
        }
    }
    const float s = scale_from_amax(__half2float(__ushort_as_half((unsigned short)all)), qmax);
    const QuantScale a = make_quant_scale(s, qmax);

    // 3. quantise the slice: what was kept, from shared memory; the rest, from L2 / HBM
    for (i = tid; i < n_kept; i += kFusedThreads) __stcs(Xqs + i, regrouped(quant8_f16<false>(cache[i], a), regroup));
    for (; i + 3 * kFusedThreads < n; i += 4 * kFusedThreads) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = __ldg(Xs + i + u * kFusedThreads);
#pragma unroll
        for (int u = 0; u < 4; ++u) __stcs(Xqs + i + u * kFusedThreads, regrouped(quant8_f16<false>(v[u], a), regroup));
    }
    for (; i < n; i += kFusedThreads) __stcs(Xqs + i, regrouped(quant8_f16<false>(__ldg(Xs + i), a), regroup));
}

// ---- library-owned scratch for gpusq_quant_act_static ----
// One fixed array per GPU that loads the library (8 KB, held until the process exits).  In host code
// the symbol below is only a handle: the address the kernels need comes from cudaGetSymbolAddress,
// looked up once per device with that device current.
constexpr int64_t kStaticMaxElems = (int64_t)1 << 32;     // largest M*K the static entry point accepts
static __device__ __align__(256) uint32_t g_act_scratch[kMaxPartials];
static std::mutex g_scratch_mutex;
static uint32_t *g_scratch_addr[kMaxDevices] = {};

static int static_scratch(uint32_t **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GPUSQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_act_scratch) != cudaSuccess || !p) return GPUSQ_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<uint32_t *>(p);
    }
    *out = g_scratch_addr[dev];
    return GPUSQ_OK;
}

}  // namespace gpusq

using namespace gpusq;

extern "C" {

int gpusq_prune24(const float *W, float *Wp, uint8_t *mask, int N, int K, void *stream)
{
    if (!W || !Wp) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 4) return GPUSQ_ERR_SHAPE;
    if (!aligned(W, 16) || !aligned(Wp, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t groups = (int64_t)N * (K / 4);
    prune24_kernel<4><<<grid_for(ceil_div(groups, 4), 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const float4 *>(W), reinterpret_cast<float4 *>(Wp), mask, groups);
    return launch_status();
}

int gpusq_quant_weight(const float *Wp, int8_t *Wq, float *w_scale, int N, int K, void *stream)
{
    if (!Wp || !Wq || !w_scale) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 4) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wp, 16) || !aligned(Wq, 4)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int grid = N < num_sms() * 8 ? N : num_sms() * 8;
    quant_weight_kernel<<<grid, kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const float4 *>(Wp), reinterpret_cast<uint32_t *>(Wq), w_scale, N, K / 4);
    return launch_status();
}

int gpusq_compress24(const int8_t *Wq, int8_t *vals, uint8_t *meta, int N, int K, void *stream)
{
    if (!Wq || !vals || !meta) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wq, 8) || !aligned(vals, 4)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t groups = (int64_t)N * (K / 4);
    if (K % 16 == 0 && aligned(Wq, 16) && aligned(vals, 8) && aligned(meta, 2)) {
        compress24_x4_kernel<<<grid_for(groups / 4, 8), kThreads, 0, (cudaStream_t)stream>>>(
            reinterpret_cast<const uint4 *>(Wq), reinterpret_cast<uint2 *>(vals),
            reinterpret_cast<uint16_t *>(meta), groups / 4);
    } else {
        compress24_x2_kernel<<<grid_for(groups / 2, 8), kThreads, 0, (cudaStream_t)stream>>>(
            reinterpret_cast<const uint2 *>(Wq), reinterpret_cast<uint32_t *>(vals), meta, groups / 2);
    }
    return launch_status();
}

int gpusq_decompress24(const int8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K, void *stream)
{
    if (!Wq || !vals || !meta) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wq, 8) || !aligned(vals, 4)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t pairs = (int64_t)N * (K / 8);
    decompress24_kernel<<<grid_for(pairs, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint32_t *>(vals), meta, reinterpret_cast<uint2 *>(Wq), pairs);
    return launch_status();
}

size_t gpusq_packed_bytes(int N, int K)
{
    if (N <= 0 || K <= 0) return 0;
    const size_t Np = (size_t)round_up(N, 256), Kp = (size_t)round_up(K, 128);
    return Np * Kp / 2 + Np * Kp / 8;
}

int gpusq_pack24(const int8_t *vals, const uint8_t *meta, void *Wpacked, int N, int K, void *stream)
{
    if (!vals || !meta || !Wpacked) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(vals, 4) || !aligned(Wpacked, 256)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int Np = round_up(N, 256), Kp = round_up(K, 128);
    const int64_t chunks = (int64_t)Np * (Kp / 32) + (int64_t)Np * (Kp / 128);
    pack24_kernel<<<grid_for(chunks, 8), kThreads, 0, (cudaStream_t)stream>>>(
        vals, meta, reinterpret_cast<uint8_t *>(Wpacked), N, K, Np, Kp);
    return launch_status();
}

int gpusq_compress24_f16(const float *Wp, void *vals, uint8_t *meta, int N, int K, void *stream)
{
    if (!Wp || !vals || !meta) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(Wp, 16) || !aligned(vals, 8)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t pairs = (int64_t)N * (K / 8);
    compress24_f16_kernel<<<grid_for(pairs, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const float4 *>(Wp), reinterpret_cast<uint2 *>(vals), meta, pairs);
    return launch_status();
}

size_t gpusq_packed_bytes_f16(int N, int K)
{
    if (N <= 0 || K <= 0) return 0;
    const size_t Np = (size_t)round_up(N, 256), Kp = (size_t)round_up(K, 128);
    return Np * Kp + Np * Kp / 8;
}

int gpusq_pack24_f16(const void *vals, const uint8_t *meta, void *Wpacked, int N, int K, void *stream)
{
    if (!vals || !meta || !Wpacked) return GPUSQ_ERR_NULL;
    if (N <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (!aligned(vals, 4) || !aligned(Wpacked, 256)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int Np = round_up(N, 256), Kp = round_up(K, 128);
    const int64_t items = (int64_t)Np * (Kp / 16) + (int64_t)Np * (Kp / 8);
    pack24_f16_kernel<<<grid_for(items, 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint16_t *>(vals), meta, reinterpret_cast<uint8_t *>(Wpacked), N, K, Np, Kp);
    return launch_status();
}

size_t gpusq_quant_act_workspace(int64_t M, int K)
{
    (void)M;
    (void)K;
    return (size_t)(kMaxPartials + kWorkspaceExtra) * sizeof(uint32_t);
}

// gpusq_quant_act (qmax 127) and gpusq_quant_act4 (qmax 7, codes of every eight columns regrouped)
static int quant_act_common(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                            void *workspace, size_t ws_bytes, void *stream, float qmax, int regroup)
{
    static_assert(GPUSQ_QUANT_ACT_STATUS_OFFSET == kWsStatus * sizeof(uint32_t), "status word as documented");
    if (!X || !Xq || !x_scale) return GPUSQ_ERR_NULL;
    if (M <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (scale_mode != GPUSQ_SCALE_COMPUTE && scale_mode != GPUSQ_SCALE_GIVEN) return GPUSQ_ERR_ARG;
    if (!aligned(X, 16) || !aligned(Xq, 16)) return GPUSQ_ERR_ALIGN;
    if (scale_mode == GPUSQ_SCALE_COMPUTE) {
        if (!workspace || ws_bytes < gpusq_quant_act_workspace(M, K)) return GPUSQ_ERR_WORKSPACE;
        if (!aligned(workspace, 16)) return GPUSQ_ERR_ALIGN;
    }
    if (int st = check_arch()) return st;
    const int64_t vec8 = M * (int64_t)K / 8;
    cudaStream_t s = (cudaStream_t)stream;
    if (scale_mode == GPUSQ_SCALE_COMPUTE) {
        // one cooperative launch: every CTA must be resident for the grid-wide barrier.  The opt-in to
        // large dynamic shared memory is per device.
        static std::mutex mu;
        static uint8_t attr_state[kMaxDevices] = {};          // 1 = set, 2 = failed
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GPUSQ_ERR_CUDA;
        {
            std::lock_guard<std::mutex> lock(mu);
            if (attr_state[dev] == 0) {
                const bool ok = cudaFuncSetAttribute(act_quant_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     kFusedSmemBytes) == cudaSuccess;
                if (!ok) (void)cudaGetLastError();
                attr_state[dev] = ok ? 1 : 2;
            }
            if (attr_state[dev] != 1) return GPUSQ_ERR_CUDA;
        }
        int grid = num_sms();
        if (grid > kMaxPartials) grid = kMaxPartials;
        // small tensors: no more CTAs than give every thread two vectors (fewer arrivals at the barrier)
        const int64_t want = ceil_div(vec8, 2 * kFusedThreads);
        if ((int64_t)grid > want) grid = (int)(want < 1 ? 1 : want);
        if (ceil_div(vec8, grid) > 0x7FFFFFFF) return GPUSQ_ERR_SHAPE;      // a CTA's slice is indexed with 32 bits
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid, 1, 1);
        cfg.blockDim = dim3(kFusedThreads, 1, 1);
        cfg.dynamicSmemBytes = kFusedSmemBytes;
        cfg.stream = s;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // set up while the previous kernel drains
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        const unsigned long long wait_ns = g_grid_wait_ns.load(std::memory_order_relaxed);
        const int withhold = g_withhold_slot.load(std::memory_order_relaxed);
        if (cudaLaunchKernelEx(&cfg, act_quant_fused_kernel, reinterpret_cast<const uint4 *>(X),
                               reinterpret_cast<uint2 *>(Xq), x_scale, reinterpret_cast<uint32_t *>(workspace), vec8,
                               wait_ns, withhold, qmax, regroup) != cudaSuccess) {
            (void)cudaGetLastError();
            return GPUSQ_ERR_CUDA;
        }
        return GPUSQ_OK;
    }
    act_quant_kernel<<<grid_for(ceil_div(vec8, 2), 8), kThreads, 0, s>>>(
        reinterpret_cast<const uint4 *>(X), reinterpret_cast<uint2 *>(Xq), x_scale, nullptr, 0, vec8, nullptr, qmax,
        regroup);
    return launch_status();
}

int gpusq_quant_act(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                    void *workspace, size_t ws_bytes, void *stream)
{
    return quant_act_common(X, Xq, x_scale, scale_mode, M, K, workspace, ws_bytes, stream, 127.0f, 0);
}

int gpusq_quant_act4(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                     void *workspace, size_t ws_bytes, void *stream)
{
    return quant_act_common(X, Xq, x_scale, scale_mode, M, K, workspace, ws_bytes, stream, 7.0f, 1);
}

int gpusq_quant_act_absmax(const void *X, int8_t *Xq, float *x_scale, const float *absmax, int64_t M, int K,
                           void *stream)
{
    if (!X || !Xq || !x_scale || !absmax) return GPUSQ_ERR_NULL;
    if (M <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (x_scale == absmax) return GPUSQ_ERR_ARG;
    if (!aligned(X, 16) || !aligned(Xq, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    const int64_t vec8 = M * (int64_t)K / 8;
    act_quant_kernel<<<grid_for(ceil_div(vec8, 2), 8), kThreads, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<const uint4 *>(X), reinterpret_cast<uint2 *>(Xq), x_scale, nullptr, 0, vec8, absmax);
    return launch_status();
}

int gpusq_set_quant_act_wait(unsigned long long limit_ns, int withhold_last_cta)
{
    if (limit_ns == 0) return GPUSQ_ERR_ARG;
    g_grid_wait_ns.store(limit_ns, std::memory_order_relaxed);
    g_withhold_slot.store(withhold_last_cta ? 1 : 0, std::memory_order_relaxed);
    return GPUSQ_OK;
}

int gpusq_quant_act_static(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                           void *stream)
{
    if (!X || !Xq || !x_scale) return GPUSQ_ERR_NULL;
    if (M <= 0 || K <= 0 || K % 8) return GPUSQ_ERR_SHAPE;
    if (scale_mode != GPUSQ_SCALE_COMPUTE && scale_mode != GPUSQ_SCALE_GIVEN) return GPUSQ_ERR_ARG;
    if (M > kStaticMaxElems / K) return GPUSQ_ERR_TOO_LARGE;
    if (!aligned(X, 16) || !aligned(Xq, 16)) return GPUSQ_ERR_ALIGN;
    if (int st = check_arch()) return st;
    uint32_t *scratch = nullptr;
    if (int st = static_scratch(&scratch)) return st;     // first call on a device resolves the address
    const int64_t vec8 = M * (int64_t)K / 8;
    cudaStream_t s = (cudaStream_t)stream;
    int n_partials = 0;
    if (scale_mode == GPUSQ_SCALE_COMPUTE) {
        // every slot that is read below is written here first, so stale contents do not matter
        n_partials = grid_for(ceil_div(vec8, 4), 8);
        if (n_partials > kMaxPartials) n_partials = kMaxPartials;
        act_absmax_kernel<<<n_partials, kThreads, 0, s>>>(reinterpret_cast<const uint4 *>(X), scratch, vec8);
        if (int st = launch_status()) return st;
    }
    act_quant_kernel<<<grid_for(ceil_div(vec8, 2), 8), kThreads, 0, s>>>(
        reinterpret_cast<const uint4 *>(X), reinterpret_cast<uint2 *>(Xq), x_scale, scratch, n_partials, vec8);
    return launch_status();
}

int gpusq_patch_quant(const void *img, int8_t *Xq, float *x_scale, int scale_mode, int B, int C, int H, int W,
                      int P, int Kp, void *workspace, size_t ws_bytes, void *stream)
{
    if (!img || !Xq || !x_scale) return GPUSQ_ERR_NULL;
    if (B <= 0 || C <= 0 || H <= 0 || W <= 0 || P <= 0 || Kp <= 0) return GPUSQ_ERR_SHAPE;
    if (H % P || W % P || P % 2 || Kp % 16) return GPUSQ_ERR_SHAPE;
    const int64_t K = (int64_t)C * P * P;
    const int64_t elems = (int64_t)B * C * H * W;
    if (K > Kp || elems % 8) return GPUSQ_ERR_SHAPE;
    if (scale_mode != GPUSQ_SCALE_COMPUTE && scale_mode != GPUSQ_SCALE_GIVEN) return GPUSQ_ERR_ARG;
    const int vec = (P % 8 == 0) ? 8 : (P % 4 == 0) ? 4 : 2;          // W % P == 0, so vec divides W too
    const int64_t tokens = (int64_t)B * (H / P) * (W / P);
    const int64_t items = tokens * (Kp / vec);
    if (items > 0x7FFFFFFF) return GPUSQ_ERR_TOO_LARGE;               // the kernel indexes its items with 32 bits
    if (!aligned(img, 16) || !aligned(Xq, 16)) return GPUSQ_ERR_ALIGN;
    if (scale_mode == GPUSQ_SCALE_COMPUTE) {
        if (!workspace || ws_bytes < gpusq_quant_act_workspace(tokens, Kp)) return GPUSQ_ERR_WORKSPACE;
        if (!aligned(workspace, 16)) return GPUSQ_ERR_ALIGN;
    }
    if (int st = check_arch()) return st;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t *partial = reinterpret_cast<uint32_t *>(workspace);
    int n_partials = 0;
    if (scale_mode == GPUSQ_SCALE_COMPUTE) {
        // the partial maxima use the first words of the workspace, every one written before it is
        // read; the words behind them (gpusq_quant_act's barrier) are not touched
        const int64_t vec8 = elems / 8;
        n_partials = grid_for(ceil_div(vec8, 4), 8);
        if (n_partials > kMaxPartials) n_partials = kMaxPartials;
        act_absmax_kernel<<<n_partials, kThreads, 0, s>>>(reinterpret_cast<const uint4 *>(img), partial, vec8);
        if (int st = launch_status()) return st;
    }
    PatchGeom g;
    g.C = C; g.H = H; g.W = W; g.P = P;
    g.Tx = W / P; g.T = (H / P) * (W / P);
    g.K = (int)K; g.Kp = Kp;
    g.by_row = make_fast_div((uint32_t)(Kp / vec));
    g.by_pp = make_fast_div((uint32_t)(P * P));
    g.by_p = make_fast_div((uint32_t)P);
    g.by_t = make_fast_div((uint32_t)g.T);
    g.by_tx = make_fast_div((uint32_t)g.Tx);
    const int grid = grid_for(items, 8);
    const __half *src = reinterpret_cast<const __half *>(img);
    if (vec == 8)
        patch_quant_kernel<8><<<grid, kThreads, 0, s>>>(src, Xq, x_scale, partial, n_partials, g, (uint32_t)items);
    else if (vec == 4)
        patch_quant_kernel<4><<<grid, kThreads, 0, s>>>(src, Xq, x_scale, partial, n_partials, g, (uint32_t)items);
    else
        patch_quant_kernel<2><<<grid, kThreads, 0, s>>>(src, Xq, x_scale, partial, n_partials, g, (uint32_t)items);
    return launch_status();
}

const char *gpusq_status_string(int status)
{
    switch (status) {
    case GPUSQ_OK: return "GPUSQ_OK";
    case GPUSQ_ERR_NULL: return "GPUSQ_ERR_NULL: a required pointer is NULL";
    case GPUSQ_ERR_SHAPE: return "GPUSQ_ERR_SHAPE: a dimension is not positive or breaks a divisibility rule";
    case GPUSQ_ERR_ALIGN: return "GPUSQ_ERR_ALIGN: a pointer is not aligned as required";
    case GPUSQ_ERR_WORKSPACE: return "GPUSQ_ERR_WORKSPACE: workspace missing or too small";
    case GPUSQ_ERR_UNSUPPORTED_ARCH: return "GPUSQ_ERR_UNSUPPORTED_ARCH: device is not compute capability 10.x";
    case GPUSQ_ERR_CUDA: return "GPUSQ_ERR_CUDA: a CUDA call failed";
    case GPUSQ_ERR_TIMEOUT: return "GPUSQ_ERR_TIMEOUT: a bounded device-side wait expired";
    case GPUSQ_ERR_ARG: return "GPUSQ_ERR_ARG: an enum argument is out of range";
    case GPUSQ_ERR_TOO_LARGE: return "GPUSQ_ERR_TOO_LARGE: the tensor exceeds the fixed capacity of this entry point";
    default: return "unknown gpusq status";
    }
}

}  // extern "C"
