/*
 * gpusq -- 2:4 fine-grained structured-sparse INT8 linear layers for NVIDIA
 * B200 (sm_100a), the patch-embedding layer on the same GEMM, and the FP16 2:4
 * sparse model the INT8 one is quantised from.  C ABI of libgpusq.so.
 *
 * The layer is Y = X * W^T with
 *   W [N, K]  weight: the 2:4-sparse operand (matrix A of the paper's Fig. 1)
 *   X [M, K]  activations: the dense operand (the paper's B, transposed)
 *   Y [M, N]  output (the paper's C, transposed)
 * all row-major, densely packed (leading dimension = number of columns).
 *
 * Conventions for every call below
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library
 *     allocates nothing, frees nothing and keeps no pointer after the call
 *     returns (the kernels it enqueued read/write them until the stream
 *     reaches that point, as with any stream-ordered call).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work and return without synchronising.
 *   - The return value is a gpusq_status.  Argument errors are detected on
 *     the host before anything is enqueued; no exception, no exit, and no CPU
 *     fallback: on a device that is not sm_100 the compute calls return
 *     GPUSQ_ERR_UNSUPPORTED_ARCH.
 *   - Buffers must not overlap unless a call says it may work in place.
 *   - Calls are thread-safe when they use distinct streams and distinct
 *     buffers.
 */
#ifndef GPUSQ_H
#define GPUSQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gpusq_status {
    GPUSQ_OK = 0,
    GPUSQ_ERR_NULL = 1,             /* a required pointer is NULL */
    GPUSQ_ERR_SHAPE = 2,            /* a dimension is <= 0 or violates a divisibility rule */
    GPUSQ_ERR_ALIGN = 3,            /* a pointer is not aligned as required (16 bytes) */
    GPUSQ_ERR_WORKSPACE = 4,        /* workspace missing or too small */
    GPUSQ_ERR_UNSUPPORTED_ARCH = 5, /* current device is not compute capability 10.x */
    GPUSQ_ERR_CUDA = 6,             /* a CUDA runtime / driver call failed */
    GPUSQ_ERR_TIMEOUT = 7,          /* a bounded device-side wait expired (see status_buf) */
    GPUSQ_ERR_ARG = 8,              /* an enum argument is out of range */
    GPUSQ_ERR_TOO_LARGE = 9         /* the tensor exceeds the fixed capacity of the entry point */
} gpusq_status;

enum { GPUSQ_ACT_NONE = 0, GPUSQ_ACT_GELU = 1 };
enum { GPUSQ_OUT_F16 = 0, GPUSQ_OUT_I8 = 1, GPUSQ_OUT_I32 = 2, GPUSQ_OUT_F32 = 2 /* raw sums of the FP16 model */ };
enum { GPUSQ_SCALE_COMPUTE = 0, GPUSQ_SCALE_GIVEN = 1 };

/* Human-readable name of a status code (static string, never NULL). */
const char *gpusq_status_string(int status);

/* ---------------------------------------------------------------------------
 * gpusq_prune24 -- 2:4 structured pruning along K.
 * Paper: Sec. 1 and Sec. 3.1 (two of every four contiguous elements on a row
 * of the sparse matrix are zero); Sec. 3.4 (the dense model is pruned into
 * the 2:4 sparse one).  Criterion (the paper names none): keep the two
 * largest magnitudes of each aligned group of four; on equal magnitudes the
 * lower index is kept; exactly two positions are kept even if they hold
 * zeros.  NaN inputs give unspecified masks.
 *   W    [N, K] f32 in.
 *   Wp   [N, K] f32 out; may be the same pointer as W (in place).
 *   mask [N, K/4] u8 out, nullable: bit i of the low nibble is set when
 *        element i of the group is kept.
 * Requires N > 0, K > 0, K % 4 == 0, W and Wp 16-byte aligned.
 */
int gpusq_prune24(const float *W, float *Wp, uint8_t *mask, int N, int K, void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_quant_weight -- symmetric per-output-channel INT8 weight quantisation.
 * Paper: Sec. 3.4 (the sparse floating-point model is quantised to INT8 with a
 * scale factor).  w_scale[n] = max_k |Wp[n,k]| / 127 (1.0 for a zero row);
 * Wq = clamp(round-half-even(Wp / w_scale[n]), -127, 127); binary32, true
 * division.
 *   Wp [N, K] f32 in;  Wq [N, K] i8 out;  w_scale [N] f32 out.
 * Requires N > 0, K > 0, K % 4 == 0, Wp 16-byte and Wq 4-byte aligned.
 */
int gpusq_quant_weight(const float *Wp, int8_t *Wq, float *w_scale, int N, int K, void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_compress24 -- kept values + 2-bit position metadata.
 * Paper: Fig. 1, Fig. 2, Sec. 3.1 (M x K/2 values; 2 bits of metadata per kept
 * value).  Per group of four the kept positions i0 < i1 are derived from the
 * INT8 codes with the same keep-two rule as gpusq_prune24, so
 * decompress(compress(Wq)) == Wq for every 2:4 matrix.
 *   Wq   [N, K]   i8 in.
 *   vals [N, K/2] i8 out: vals[n, 2g] = Wq[n, 4g+i0], vals[n, 2g+1] = Wq[n, 4g+i1].
 *   meta [N, K/8] u8 out: nibble = i0 | (i1 << 2); group g of a row is in byte
 *        g/2, even g in the low nibble.
 * Requires N > 0, K > 0, K % 8 == 0, Wq 8-byte, vals 4-byte aligned.
 */
int gpusq_compress24(const int8_t *Wq, int8_t *vals, uint8_t *meta, int N, int K, void *stream);

/* Inverse of gpusq_compress24 (test and debugging aid). Wq [N, K] i8 out. */
int gpusq_decompress24(const int8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K,
                       void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_pack24 -- arrange vals + meta the way the sparse tensor-core kernel
 * reads them (Sec. 3.1: the storage format of the compressed operand; the
 * layout itself is a hardware detail the paper does not give).
 * Wpacked holds gpusq_packed_bytes(N, K) bytes, 256-byte aligned:
 *   [0, Np*Kp/2)            values, row-major [Np, Kp/2], zero padded
 *   [Np*Kp/2, Np*Kp*5/8)    metadata tiles [Np/128][Kp/128][128 rows][16 bytes]
 * with Np = N rounded up to 256 and Kp = K rounded up to 128.
 * Requires N > 0, K > 0, K % 8 == 0.
 */
size_t gpusq_packed_bytes(int N, int K);
int gpusq_pack24(const int8_t *vals, const uint8_t *meta, void *Wpacked, int N, int K,
                 void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_quant_act -- symmetric per-tensor INT8 activation quantisation.
 * Paper: Sec. 2.2 and Sec. 3.4 (a quantise node with one scale factor in front
 * of each GEMM; the paper learns the factor in training).
 *   X [M, K] f16 in;  Xq [M, K] i8 out;  x_scale: device float[1].
 *   scale_mode GPUSQ_SCALE_COMPUTE: *x_scale = max|X| / 127 (1.0 if X is all
 *     zero) is computed and written; GPUSQ_SCALE_GIVEN: *x_scale is read.
 *   Xq = clamp(round-half-even(float(X) / *x_scale), -127, 127).
 *   workspace: device scratch of at least gpusq_quant_act_workspace(M, K)
 *     bytes, 16-byte aligned, needed for GPUSQ_SCALE_COMPUTE only (may be NULL
 *     otherwise).  It must be ZERO-FILLED before its first use (once, e.g.
 *     right after allocation); every call leaves it usable by the next call,
 *     of any size, so one buffer serves a whole stream of calls.  Calls that
 *     can overlap on the GPU need separate workspaces.
 *   GPUSQ_SCALE_COMPUTE runs as one cooperative launch whose CTAs meet at a
 *   grid-wide barrier.  Its waits are bounded (2 s), and the outcome is all or
 *   nothing as far as the scale goes: *x_scale is set to NaN when the kernel
 *   starts and receives the real scale only after EVERY CTA has passed the
 *   barrier.  If a wait ever expires, the int32 at byte offset
 *   GPUSQ_QUANT_ACT_STATUS_OFFSET of the workspace becomes GPUSQ_ERR_TIMEOUT
 *   (it is 0 otherwise), *x_scale stays NaN, Xq is undefined (CTAs that had
 *   passed the barrier may have written their part), and the workspace must be
 *   zero-filled again before it is reused.  The host call never waits for the
 *   device; a caller that wants to know reads the status word (or tests the
 *   scale) after synchronising.
 * Requires M > 0, K > 0, K % 8 == 0, X and Xq 16-byte aligned.  The first
 * GPUSQ_SCALE_COMPUTE call on each device (with that device current) opts the
 * kernel in to large shared memory; it is safe from several threads.
 */
#define GPUSQ_QUANT_ACT_STATUS_OFFSET 8196
size_t gpusq_quant_act_workspace(int64_t M, int K);
int gpusq_quant_act(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                    void *workspace, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_quant_act_static -- gpusq_quant_act for callers that cannot hand over
 * scratch memory.  (An addition of this library; the paper has no counterpart.)
 *
 * Some hosts of this code may not allocate device memory at the point where
 * they quantise activations: an inference-server plugin whose enqueue hook
 * runs after the server has planned and frozen all device memory, a real-time
 * loop that forbids allocator calls for their unbounded latency, or a process
 * that was handed a fixed memory budget it does not own.  gpusq_quant_act
 * needs a small workspace from the caller; this variant needs none.  It uses a
 * fixed 8 KB array that lives inside the library image on every GPU that loads
 * the library (held until the process exits) and performs no cudaMalloc,
 * cudaFree or other allocating call.
 *
 * Same arguments and results as gpusq_quant_act, minus workspace / ws_bytes.
 *   - Capacity: M * K <= 2^32 elements; larger tensors are rejected with
 *     GPUSQ_ERR_TOO_LARGE and nothing is enqueued.
 *   - The first call on each device (with that device current) looks up the
 *     array's device address; make that first call outside any stream capture.
 *   - All calls on one GPU share the one array: two calls whose kernels can
 *     overlap on the GPU (different streams, no ordering between them) race
 *     and may both produce a wrong scale.  Calls ordered on one stream are
 *     safe; what an earlier call left in the array is never read.
 */
int gpusq_quant_act_static(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M,
                           int K, void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_patch_quant -- activation side of the patch-embedding layer.
 * Paper: Sec. 3.3 (the patch embedding is a convolution with kernel size =
 * stride = P, executed as a GEMM whose reduction axis C*P*P carries the 2:4
 * pattern) with the quantise node of Sec. 2.2 in front of it.  One scale for
 * the whole image tensor, as gpusq_quant_act; the codes are written as the
 * rows of that GEMM, so gpusq_spgemm_i8 on (Xq, the packed flattened conv
 * weight [D, Kp]) is the convolution:
 *   Xq[t, k] = code(img[b, c, ty*P + py, tx*P + px]),
 *   t = (b*(H/P) + ty)*(W/P) + tx,   k = (c*P + py)*P + px,
 *   Xq[t, k] = 0 for C*P*P <= k < Kp.
 *   img [B, C, H, W] f16 in;  Xq [B*(H/P)*(W/P), Kp] i8 out;
 *   x_scale device float[1], written (GPUSQ_SCALE_COMPUTE) or read (_GIVEN).
 *   Kp: row length of Xq, >= C*P*P, a multiple of 16 (the GEMM's K); the conv
 *     weight is flattened to [D, C*P*P] row-major and padded with zero
 *     columns to Kp before gpusq_prune24.
 *   workspace: GPUSQ_SCALE_COMPUTE only, >= gpusq_quant_act_workspace(tokens,
 *     Kp) bytes, 16-byte aligned; contents on entry are ignored and the words
 *     gpusq_quant_act keeps zero are not touched, so one array serves both.
 * Two launches (maximum, then quantise and rearrange) with the scale
 * computed, one with the scale supplied.
 * Requires H % P == 0, W % P == 0, P even, B*C*H*W % 8 == 0, img / Xq
 * 16-byte aligned, and tokens * Kp / v < 2^31 with v = 8, 4 or 2, the largest
 * of them that divides P (GPUSQ_ERR_TOO_LARGE otherwise).
 */
int gpusq_patch_quant(const void *img, int8_t *Xq, float *x_scale, int scale_mode, int B, int C,
                      int H, int W, int P, int Kp, void *workspace, size_t workspace_bytes,
                      void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_spgemm_i8 -- the fused layer: 2:4-sparse INT8 GEMM + epilogue.
 * Paper: Fig. 1 and Sec. 3.1 (sparse x dense = dense on the sparse tensor
 * cores, same result matrix as the dense GEMM); Sec. 2.2 (de-quantise node).
 *   acc[m,n] = sum_k Wq[n,k] * Xq[m,k]             (INT32, exact)
 *   y        = fma(float(acc), w_scale[n] * *x_scale, bias ? bias[n] : 0)
 *   act GPUSQ_ACT_GELU: y = 0.5 * y * erfc(-y / sqrt(2))
 *   out_type GPUSQ_OUT_F16: Y f16 = round-half-even(y)
 *            GPUSQ_OUT_I8 : Y i8  = clamp(round-half-even(y / *out_scale), -127, 127)
 *            GPUSQ_OUT_I32: Y i32 = acc (scales, bias, act ignored)
 *   Xq [M, K] i8 in;  Wpacked from gpusq_pack24 (N, K);  w_scale [N] f32;
 *   x_scale device float[1];  bias [N] f32 nullable;  out_scale device
 *   float[1], GPUSQ_OUT_I8 only;  Y [M, N] out.
 *   status_buf: device int32[4], nullable.  If given it must be zero on entry;
 *     a kernel whose bounded wait expires writes {GPUSQ_ERR_TIMEOUT, tile,
 *     role, stage} there and stops issuing work (the output is then
 *     undefined).  The host call itself never waits for the device.
 * Requires M > 0, K % 16 == 0, Xq / Wpacked / Y 16-byte aligned, and a row of
 * Y that is a multiple of 16 bytes: N % 8 == 0 for GPUSQ_OUT_F16, N % 16 == 0
 * for GPUSQ_OUT_I8 (any N for GPUSQ_OUT_I32).  N need not be a multiple of
 * the 128-feature tile (DeiT-Tiny's 192 and 576, Swin-Tiny's 96 and 288).
 */
int gpusq_spgemm_i8(const int8_t *Xq, const void *Wpacked, const float *w_scale,
                    const float *x_scale, const float *bias, int act, int out_type,
                    const float *out_scale, void *Y, int64_t M, int N, int K, int32_t *status_buf,
                    void *stream);

/* ---------------------------------------------------------------------------
 * Chaining layers (Sec. 2.2: a quantise node in front of every GEMM and a
 * de-quantise node behind it, through the whole deployed model; Sec. 4.1:
 * deployment as INT8 layers).  Two ways to spare the next layer's quantise
 * node its pass over the tensor for the maximum:
 *   - gpusq_spgemm_i8 with GPUSQ_OUT_I8 writes the next layer's INT8 codes
 *     directly (supplied *out_scale, e.g. calibrated); the next
 *     gpusq_spgemm_i8 reads them with x_scale = that out_scale;
 *   - gpusq_spgemm_i8_absmax writes FP16 and, beside it, the largest
 *     magnitude of what it wrote; gpusq_quant_act_absmax then derives the
 *     per-tensor scale from that number and quantises in ONE pass, with the
 *     same result as gpusq_quant_act(GPUSQ_SCALE_COMPUTE) on that tensor.
 *
 * gpusq_spgemm_i8_absmax: gpusq_spgemm_i8 with GPUSQ_OUT_F16 (same arguments,
 *   same Y, bit for bit) plus
 *   y_absmax device float[1]: max over all m < M, n < N of |Y[m,n]| (the
 *     rounded binary16 values) is MERGED into it (an atomic maximum on the
 *     bit pattern), so it must hold 0.0f -- or the running maximum of the
 *     tensors it is to cover -- on entry.  Finite outputs assumed.
 * gpusq_quant_act_absmax: X [M, K] f16 in, Xq [M, K] i8 out,
 *   absmax device float[1] in (max |X|), x_scale device float[1] out:
 *   *x_scale = *absmax / 127 (1.0 when it is 0), codes as gpusq_quant_act.
 *   absmax and x_scale must be different addresses.  One launch, no workspace.
 *   Requires M > 0, K % 8 == 0, X / Xq 16-byte aligned.
 */
int gpusq_spgemm_i8_absmax(const int8_t *Xq, const void *Wpacked, const float *w_scale,
                           const float *x_scale, const float *bias, int act, void *Y,
                           float *y_absmax, int64_t M, int N, int K, int32_t *status_buf,
                           void *stream);
int gpusq_quant_act_absmax(const void *X, int8_t *Xq, float *x_scale, const float *absmax,
                           int64_t M, int K, void *stream);

/* ---------------------------------------------------------------------------
 * The FP16 2:4 sparse model.  Paper: Sec. 3.1 (the compressed FP16 operand:
 * half of the values plus 2 bits of position per kept value, 43.75 % smaller)
 * and Sec. 3.4 (the dense model is first pruned to the sparse floating-point
 * model, which is then quantised); this is that intermediate model's layer.
 *
 * gpusq_compress24_f16: Wp [N, K] f32 in, already 2:4 (gpusq_prune24).  Each
 *   weight is rounded to binary16 (nearest even); per group of four the two
 *   values of largest binary16 magnitude (lower index on ties) are kept:
 *   vals [N, K/2] f16 out, meta [N, K/8] u8 out, nibbles as gpusq_compress24.
 *   Requires K % 8 == 0, Wp 16-byte and vals 8-byte aligned.
 * gpusq_packed_bytes_f16 / gpusq_pack24_f16: size and contents of the opaque
 *   operand gpusq_spgemm_f16 reads (values padded to N % 256, K % 128, then the
 *   metadata in the tensor core's arrangement for 16-bit operands).  Wpacked
 *   256-byte aligned.
 * gpusq_spgemm_f16:
 *   acc[m,n] = sum_k f16(W[n,k]) * X[m,k]     (exact products, FP32 accumulation
 *                                              in the tensor core: order unspecified)
 *   y        = acc + (bias ? bias[n] : 0);  act GPUSQ_ACT_GELU as gpusq_spgemm_i8
 *   out_type GPUSQ_OUT_F16: Y f16 = round-half-even(y);
 *            GPUSQ_OUT_F32: Y f32 = acc (bias, act ignored).
 *   X [M, K] f16 in (no quantise node);  bias [N] f32 nullable;  Y [M, N] out;
 *   status_buf as gpusq_spgemm_i8.
 *   Requires M > 0, K % 8 == 0, N % 8 == 0 for GPUSQ_OUT_F16, X / Y 16-byte and
 *   Wpacked 256-byte aligned.
 */
int gpusq_compress24_f16(const float *Wp, void *vals, uint8_t *meta, int N, int K, void *stream);
size_t gpusq_packed_bytes_f16(int N, int K);
int gpusq_pack24_f16(const void *vals, const uint8_t *meta, void *Wpacked, int N, int K, void *stream);
int gpusq_spgemm_f16(const void *X, const void *Wpacked, const float *bias, int act, int out_type,
                     void *Y, int64_t M, int N, int K, int32_t *status_buf, void *stream);

/* ---------------------------------------------------------------------------
 * The INT4 model.  Paper: Sec. 3.1 (for 4-bit operands the sparse format is
 * pair-wise structured at a granularity of 4:8: of the four two-wide sub-chunks
 * of every eight adjacent weights of a row two are kept, two are all zero; the
 * four kept values are stored with two 2-bit sub-chunk indices; 37.5 % smaller
 * than dense INT4) and Sec. 3.4 / Table 1 (the INT4 models, 12.7x smaller than
 * FP32).  sm_100 tensor cores have no 4-bit integer kind, so the storage is the
 * paper's and the arithmetic is the INT8 2:4 path's, exactly: regrouping the
 * columns of every chunk of eight as (first elements of the four sub-chunks,
 * then the second ones; column e -> (e % 2) * 4 + e / 2) turns the pair-wise
 * 4:8 pattern into 2:4, and a GEMM is unchanged when weight and activation
 * columns are permuted alike.
 *
 * gpusq_prune48: W [N, K] f32 -> Wp (may alias W); a sub-chunk weighs
 *   |a| + |b| (compared as exact sums), the two heaviest of each chunk stay,
 *   lower index on ties; mask [N, K/8] u8 nullable, bit p = sub-chunk p kept.
 *   K % 8 == 0, W / Wp 16-byte aligned.
 * gpusq_quant_weight4: as gpusq_quant_weight with 7 in place of 127
 *   (w_scale[n] = max|row| / 7; codes in [-7, 7] in INT8 containers).
 * gpusq_compress48: Wq [N, K] i8 (codes in [-7, 7]) -> vals4 [N, K/4] u8, two
 *   codes per byte in element order, the first in the low nibble (two's
 *   complement), and meta4 [N, K/16] u8, per chunk the nibble p0 | p1 << 2
 *   (p0 < p1 the kept sub-chunks, re-derived from the codes), even chunk in the
 *   low nibble.  0.3125 bytes per weight.  K % 16 == 0, Wq 16-byte aligned.
 * gpusq_expand48: (vals4, meta4) -> vals [N, K/2] i8 and meta [N, K/8] u8 of
 *   the SAME matrix with regrouped columns, in gpusq_compress24's format: feed
 *   them to gpusq_pack24.  vals 8-byte aligned.
 * gpusq_quant_act4: as gpusq_quant_act with 7 in place of 127, and the codes of
 *   every eight columns written in the regrouped order, so that
 *   gpusq_spgemm_i8 on (Xq, packed expanded weight) returns the 4-bit model's
 *   sums.  Workspace, launches and status word exactly as gpusq_quant_act.
 */
int gpusq_prune48(const float *W, float *Wp, uint8_t *mask, int N, int K, void *stream);
int gpusq_quant_weight4(const float *Wp, int8_t *Wq, float *w_scale, int N, int K, void *stream);
int gpusq_compress48(const int8_t *Wq, uint8_t *vals4, uint8_t *meta4, int N, int K, void *stream);
int gpusq_expand48(const uint8_t *vals4, const uint8_t *meta4, int8_t *vals, uint8_t *meta, int N,
                   int K, void *stream);
int gpusq_quant_act4(const void *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K,
                     void *workspace, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * gpusq_gemm_i8_dense -- the same kernel and epilogue on the uncompressed
 * INT8 weight (dense tensor-core instruction): the yardstick for the paper's
 * "2x math throughput" of the sparse GEMM (Sec. 1, Sec. 3.1).
 *   Wq [N, K] i8 in (any values; not required to be 2:4).
 * Other arguments and requirements as gpusq_spgemm_i8.
 */
int gpusq_gemm_i8_dense(const int8_t *Xq, const int8_t *Wq, const float *w_scale,
                        const float *x_scale, const float *bias, int act, int out_type,
                        const float *out_scale, void *Y, int64_t M, int N, int K,
                        int32_t *status_buf, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* GPUSQ_H */
