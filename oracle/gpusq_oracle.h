/*
 * gpusq oracle -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-threaded CPU statement of what the 2:4-sparse INT8
 * linear-layer path computes.  It shares no code with the CUDA library and is
 * never called by it; only the tests, the smoke check and the CPU-baseline
 * leg of the benchmark may use it.
 *
 * Orientation (the layer is Y = X * W^T):
 *   W [N, K]  weight, the 2:4-sparse operand (the paper's matrix A, Fig. 1)
 *   X [M, K]  activations (the paper's B, transposed)
 *   Y [M, N]  output       (the paper's C, transposed)
 * All matrices are row-major and dense in memory.
 *
 * Each function names the passage of the paper it follows.  Where the paper
 * is silent the chosen reading is stated next to the function.
 *
 * Pins (tests/test_oracle_*.py): every function below is pinned by tests that
 * do not restate its own formula; the one quantity with no pin is the
 * end-to-end accuracy of the quantised layer against an unquantised FP32
 * layer -- "parity unpinned": the paper gives task accuracy after training
 * only, so the SQNR that `o_sqnr_db` reports is information, not a check.
 */
#ifndef GPUSQ_ORACLE_H
#define GPUSQ_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Sec. 1 / Sec. 3.1 (2:4 fine-grained structured sparsity): in every group of
 * four contiguous elements along a row of the sparse matrix, two are zero.
 * Reading (paper silent on the criterion): keep the two of largest magnitude;
 * on equal magnitudes the lower index is kept; exactly two positions are kept
 * even when their values are zero.  mask (nullable) [N, K/4]: bit i of the low
 * nibble set when element i of the group is kept.  K % 4 == 0. */
void o_prune24(const float *W, float *Wp, uint8_t *mask, int N, int K);

/* Sec. 3.4 (quantise the sparse floating-point model to INT8 with a scale
 * factor).  Reading: symmetric, one scale per output channel (row),
 * scale = max|row| / 127 (1.0 for an all-zero row), code =
 * clamp(round-half-even(w / scale), -127, 127), all in IEEE binary32 with a
 * true division. */
void o_quant_weight(const float *Wp, int8_t *Wq, float *w_scale, int N, int K);

/* Fig. 1 / Fig. 2 / Sec. 3.1: the compressed operand holds K/2 values per row
 * plus 2 bits of position per kept value.  Reading of the (missing) figure:
 * per group of four the two kept positions i0 < i1 are re-derived from the
 * INT8 codes with the same keep-two rule; nibble = i0 | (i1 << 2); group g of a
 * row sits in byte g/2, low nibble first.  vals [N, K/2], meta [N, K/8].
 * K % 8 == 0. */
void o_compress24(const int8_t *Wq, int8_t *vals, uint8_t *meta, int N, int K);

/* Inverse of o_compress24: scatter the kept values back, zeros elsewhere. */
void o_decompress24(const int8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K);

/* Sec. 2.2 / Sec. 3.4 (a quantise node in front of each GEMM, one scale
 * factor).  Reading: symmetric per-tensor; X is IEEE binary16 (bit patterns
 * in uint16_t), widened exactly to binary32; scale_mode 0: *x_scale =
 * max|X| / 127 (1.0 if the tensor is all zero) is written; scale_mode 1:
 * *x_scale is read.  Codes as in o_quant_weight. */
void o_quant_act(const uint16_t *X, int8_t *Xq, float *x_scale, int scale_mode,
                 int64_t M, int K);

/* Fig. 1 / Sec. 3.1: the sparse GEMM returns the same result matrix as the
 * dense GEMM of the pruned matrix.  Written as the definition: decompress,
 * then acc[m, n] = sum_k Wq[n, k] * Xq[m, k] in 64-bit integers; returns the
 * number of sums that do not fit INT32 (0 for every supported shape). */
int64_t o_spgemm_acc(const int8_t *Xq, const int8_t *vals, const uint8_t *meta,
                     int32_t *acc, int64_t M, int N, int K);

/* Same sums for a list of token rows only: acc_rows [n_rows, N] holds the sums
 * of rows rows[0..n_rows) of X.  Used to check full-size runs by sampling. */
int64_t o_spgemm_acc_rows(const int8_t *Xq, const int8_t *vals, const uint8_t *meta,
                          const int64_t *rows, int64_t n_rows, int32_t *acc_rows,
                          int N, int K);

/* Sec. 3.3 (patch embedding): an image batch [B, C, H, W] is cut into
 * non-overlapping P x P patches and the embedding is a convolution with C
 * input channels, D output channels, kernel size = stride = P, executed as a
 * GEMM whose reduction axis C*P*P is the axis the 2:4 pattern runs along.
 * Readings (paper silent): the image is quantised like any activation tensor
 * (o_quant_act on its B*C*H*W elements, one scale); a token is one patch,
 * tokens ordered (b, ty, tx) row-major as in the usual flatten of the
 * convolution output; reduction index k = (c*P + py)*P + px, the row-major
 * flattening of a convolution weight [D, C, P, P].  H % P == 0, W % P == 0.
 *
 * o_patch_rows: the GEMM's activation matrix, X[t, k] = imgq[b, c, ty*P+py,
 * tx*P+px], columns C*P*P .. Kp-1 zero (Kp >= C*P*P pads the reduction axis
 * to what the GEMM accepts; the weight is padded with zero columns alike). */
void o_patch_rows(const int8_t *imgq, int8_t *X, int B, int C, int H, int W, int P, int Kp);

/* The convolution written as its definition on the INT8 codes:
 * acc[(b, ty, tx), d] = sum_{c, py, px} Wq[d, c, py, px] * imgq[b, c, ty*P+py, tx*P+px]
 * (64-bit sums, stored as INT32).  Returns the number of multiply-adds done:
 * B*C*H*W*D, half the FLOP count Sec. 3.3 states. */
int64_t o_patch_conv_acc(const int8_t *imgq, const int8_t *Wq, int32_t *acc, int B, int C,
                         int H, int W, int P, int D);

/* Sec. 2.2 (de-quantise node; GELU is the activation the paper names).
 * Reading, in binary32 in this order: t = (float)acc (round-to-nearest-even);
 * s = w_scale[n] * x_scale; y = fma(t, s, bias ? bias[n] : 0);
 * act 1: y = 0.5 * y * erfc(-y / sqrt(2)) evaluated in binary64 from the
 * binary32 y and rounded once to binary32 (the exact-erf GELU);
 * out_type 0: binary16, round-to-nearest-even, overflow to infinity (Y16);
 * out_type 1: INT8 clamp(rne(y / out_scale), -127, 127) (Y8);
 * out_type 2: the raw INT32 sums (Y32).  count = number of (m, n) pairs;
 * element e belongs to channel n = e % N. */
void o_epilogue(const int32_t *acc, const float *w_scale, float x_scale,
                const float *bias, int act, int out_type, float out_scale,
                void *Y, int64_t count, int N);

/* ---- FP16 2:4 sparse model: Sec. 3.1 (the compressed FP16 format, 43.75 % smaller) and Sec. 3.4
 * (the dense model is first pruned to the 2:4 sparse floating-point model M_SF).  Readings: the pruned
 * FP32 weight is rounded to binary16 (RNE); the two kept positions of a group are re-derived from the
 * binary16 magnitudes with the keep-two rule; metadata nibbles as in o_compress24; the layer takes
 * binary16 activations as they are (no quantise node) and accumulates wider than binary16. ---- */
void o_to_f16(const float *W, uint16_t *Wh, int64_t count);
void o_compress24_f16(const uint16_t *Wh, uint16_t *vals, uint8_t *meta, int N, int K);
void o_decompress24_f16(const uint16_t *vals, const uint8_t *meta, uint16_t *Wh, int N, int K);

/* Fig. 1 / Sec. 3.1 for FP16 operands, as the definition: acc[r, n] = sum_k W[n, k] * X[rows[r], k]
 * with every product exact and the sum in binary64 (the exact sum to ~1e-16 of mag);
 * mag[r, n] = sum_k |W[n, k] * X[rows[r], k]| (nullable) scales the accumulation error a
 * narrower accumulator may make. */
void o_spgemm_f16_rows(const uint16_t *X, const uint16_t *vals, const uint8_t *meta,
                       const int64_t *rows, int64_t n_rows, double *acc_rows, double *mag_rows,
                       int N, int K);

/* Epilogue of the FP16 layer: t = (float)acc; y = t + bias[n] (binary32); act 1: exact-erf GELU as in
 * o_epilogue; Y = binary16(y), RNE. */
void o_epilogue_f16(const double *acc, const float *bias, int act, uint16_t *Y, int64_t count, int N);

/* ---- INT4 model: Sec. 3.1 (the 4-bit format is pair-wise structured sparse at a granularity of
 * 4:8: every chunk of eight adjacent elements of a row keeps two of its four two-wide sub-chunks,
 * all of the other two is zero; the four kept values are stored, plus two 2-bit indices of the kept
 * sub-chunks; 37.5 % smaller than dense INT4) and Sec. 3.4 / Table 1 (the INT4 model).
 * Readings (paper silent): a sub-chunk's weight in the choice is |a| + |b|; the two heaviest are
 * kept, the lower index on ties, exactly two even if zero (the keep-two rule on sub-chunks); the
 * quantiser is the INT8 one with 7 in place of 127 (symmetric, per output channel, scale =
 * max|row| / 7, round half to even, clamp +-7; activations per tensor alike); kept sub-chunks
 * are re-derived from the codes when compressing.
 * Layout: vals [N, K/4] bytes, two codes per byte in element order, the first in the low nibble
 * (two's complement); meta [N, K/16] bytes, one nibble p0 | p1 << 2 (p0 < p1, sub-chunk indices 0..3)
 * per chunk, the chunk with the even index in the low nibble.  K % 16 == 0.
 * mask (nullable) [N, K/8]: bit p of the low nibble set when sub-chunk p is kept. ---- */
void o_prune48(const float *W, float *Wp, uint8_t *mask, int N, int K);
void o_quant_weight4(const float *Wp, int8_t *Wq, float *w_scale, int N, int K);
void o_compress48(const int8_t *Wq, uint8_t *vals, uint8_t *meta, int N, int K);
void o_decompress48(const uint8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K);
/* Activations of the INT4 model: as o_quant_act with +-7 (scale = max|X| / 7). */
void o_quant_act4(const uint16_t *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K);
/* The sparse GEMM of the 4-bit model as its definition: decompress, then 64-bit integer sums. */
int64_t o_spgemm48_acc(const int8_t *Xq, const uint8_t *vals, const uint8_t *meta, int32_t *acc,
                       int64_t M, int N, int K);

/* binary16 <-> binary32 conversions used above (RNE narrowing). */
uint16_t o_f32_to_f16(float f);
float o_f16_to_f32(uint16_t h);

/* 10 log10(sum ref^2 / sum (ref - test)^2): information only (parity unpinned). */
double o_sqnr_db(const float *ref, const float *test, int64_t count);

#ifdef __cplusplus
}
#endif
#endif
