/*
 * gpusq oracle -- TEST INFRASTRUCTURE (see gpusq_oracle.h).  Plain C, scalar
 * loops, no blocking, no threads.  Build: gcc -O2 -ffp-contract=off -fPIC
 * -shared (no fast-math: the rounding steps below must stay IEEE).
 */
#include "gpusq_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ---- keep-two rule shared by pruning (on |w|) and compression (on |code|) ----
 * Order the four indices by (magnitude descending, index ascending); the first
 * two are kept; they are returned in ascending order. */
static void keep_two(const double mag[4], int *i0, int *i1)
{
    int order[4] = {0, 1, 2, 3};
    /* insertion sort, stable: equal magnitudes keep ascending index order */
    for (int a = 1; a < 4; ++a) {
        int idx = order[a];
        int b = a - 1;
        while (b >= 0 && mag[order[b]] < mag[idx]) {
            order[b + 1] = order[b];
            --b;
        }
        order[b + 1] = idx;
    }
    int p = order[0], q = order[1];
    *i0 = p < q ? p : q;
    *i1 = p < q ? q : p;
}

void o_prune24(const float *W, float *Wp, uint8_t *mask, int N, int K)
{
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < K / 4; ++g) {
            const float *w = W + (int64_t)n * K + 4 * g;
            double mag[4];
            for (int i = 0; i < 4; ++i) mag[i] = fabs((double)w[i]);
            int i0, i1;
            keep_two(mag, &i0, &i1);
            float out[4];
            for (int i = 0; i < 4; ++i) out[i] = (i == i0 || i == i1) ? w[i] : 0.0f;
            memcpy(Wp + (int64_t)n * K + 4 * g, out, sizeof out);
            if (mask) mask[(int64_t)n * (K / 4) + g] = (uint8_t)((1u << i0) | (1u << i1));
        }
    }
}

static int8_t quant_code(float x, float scale)
{
    float q = nearbyintf(x / scale); /* default rounding mode: ties to even */
    if (q > 127.0f) q = 127.0f;
    if (q < -127.0f) q = -127.0f;
    return (int8_t)q;
}

void o_quant_weight(const float *Wp, int8_t *Wq, float *w_scale, int N, int K)
{
    for (int n = 0; n < N; ++n) {
        const float *row = Wp + (int64_t)n * K;
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf(row[k]);
            if (a > amax) amax = a;
        }
        float s = (amax == 0.0f) ? 1.0f : amax / 127.0f;
        w_scale[n] = s;
        for (int k = 0; k < K; ++k) Wq[(int64_t)n * K + k] = quant_code(row[k], s);
    }
}

void o_compress24(const int8_t *Wq, int8_t *vals, uint8_t *meta, int N, int K)
{
    memset(meta, 0, (size_t)N * (size_t)(K / 8));
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < K / 4; ++g) {
            const int8_t *w = Wq + (int64_t)n * K + 4 * g;
            double mag[4];
            for (int i = 0; i < 4; ++i) mag[i] = fabs((double)w[i]);
            int i0, i1;
            keep_two(mag, &i0, &i1);
            vals[(int64_t)n * (K / 2) + 2 * g] = w[i0];
            vals[(int64_t)n * (K / 2) + 2 * g + 1] = w[i1];
            uint8_t nib = (uint8_t)(i0 | (i1 << 2));
            meta[(int64_t)n * (K / 8) + g / 2] |= (uint8_t)(nib << (4 * (g & 1)));
        }
    }
}

void o_decompress24(const int8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K)
{
    memset(Wq, 0, (size_t)N * (size_t)K);
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < K / 4; ++g) {
            uint8_t byte = meta[(int64_t)n * (K / 8) + g / 2];
            uint8_t nib = (uint8_t)((byte >> (4 * (g & 1))) & 0xF);
            int i0 = nib & 3, i1 = (nib >> 2) & 3;
            /* i1 written last: with a well-formed nibble i0 != i1 */
            Wq[(int64_t)n * K + 4 * g + i0] = vals[(int64_t)n * (K / 2) + 2 * g];
            Wq[(int64_t)n * K + 4 * g + i1] = vals[(int64_t)n * (K / 2) + 2 * g + 1];
        }
    }
}

/* ---- binary16 ---- */
float o_f16_to_f32(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24); /* zero and subnormals: f * 2^-24 */
    else if (e == 31)
        v = f ? (double)NAN : (double)INFINITY;
    else
        v = ldexp((double)(f + 1024), e - 25); /* (1 + f/1024) * 2^(e-15) */
    return (float)(sign ? -v : v); /* exact: every binary16 is a binary32 */
}

uint16_t o_f32_to_f16(float x)
{
    uint16_t sign = signbit(x) ? 0x8000u : 0u;
    if (isnan(x)) return (uint16_t)(sign | 0x7E00u);
    double a = fabs((double)x);
    if (isinf(x)) return (uint16_t)(sign | 0x7C00u);
    /* spacing of binary16 at |x|: 2^-24 below 2^-14, else 2^(floor(log2 a) - 10) */
    int ex;
    (void)frexp(a, &ex); /* a = m * 2^ex, m in [0.5, 1)  =>  floor(log2 a) = ex - 1 */
    int e2 = (a == 0.0) ? -15 : ex - 1;
    if (e2 < -14) e2 = -14;
    double step = ldexp(1.0, e2 - 10);
    double q = nearbyint(a / step); /* exact scaling by a power of two; ties to even */
    double r = q * step;
    if (r >= 65520.0) return (uint16_t)(sign | 0x7C00u); /* past the largest finite + half a step */
    if (r == 0.0) return sign;
    /* encode r = q * step */
    int er;
    (void)frexp(r, &er);
    int e3 = er - 1;
    if (e3 < -14) { /* subnormal: r = f * 2^-24 */
        return (uint16_t)(sign | (uint16_t)ldexp(r, 24));
    }
    uint16_t frac = (uint16_t)(ldexp(r, 10 - e3) - 1024.0);
    return (uint16_t)(sign | (uint16_t)((e3 + 15) << 10) | frac);
}

void o_quant_act(const uint16_t *X, int8_t *Xq, float *x_scale, int scale_mode,
                 int64_t M, int K)
{
    int64_t count = M * (int64_t)K;
    float s;
    if (scale_mode == 0) {
        float amax = 0.0f;
        for (int64_t i = 0; i < count; ++i) {
            float a = fabsf(o_f16_to_f32(X[i]));
            if (a > amax) amax = a;
        }
        s = (amax == 0.0f) ? 1.0f : amax / 127.0f;
        *x_scale = s;
    } else {
        s = *x_scale;
    }
    for (int64_t i = 0; i < count; ++i) Xq[i] = quant_code(o_f16_to_f32(X[i]), s);
}

static int64_t dot_rows(const int8_t *xrow, const int8_t *Wd, int32_t *out, int N, int K)
{
    int64_t overflow = 0;
    for (int n = 0; n < N; ++n) {
        int64_t sum = 0;
        const int8_t *wrow = Wd + (int64_t)n * K;
        for (int k = 0; k < K; ++k) sum += (int64_t)wrow[k] * (int64_t)xrow[k];
        if (sum > INT32_MAX || sum < INT32_MIN) ++overflow;
        out[n] = (int32_t)sum;
    }
    return overflow;
}

int64_t o_spgemm_acc(const int8_t *Xq, const int8_t *vals, const uint8_t *meta,
                     int32_t *acc, int64_t M, int N, int K)
{
    int8_t *Wd = (int8_t *)malloc((size_t)N * (size_t)K);
    if (!Wd) return -1;
    o_decompress24(vals, meta, Wd, N, K);
    int64_t overflow = 0;
    for (int64_t m = 0; m < M; ++m)
        overflow += dot_rows(Xq + m * K, Wd, acc + m * N, N, K);
    free(Wd);
    return overflow;
}

int64_t o_spgemm_acc_rows(const int8_t *Xq, const int8_t *vals, const uint8_t *meta,
                          const int64_t *rows, int64_t n_rows, int32_t *acc_rows,
                          int N, int K)
{
    int8_t *Wd = (int8_t *)malloc((size_t)N * (size_t)K);
    if (!Wd) return -1;
    o_decompress24(vals, meta, Wd, N, K);
    int64_t overflow = 0;
    for (int64_t r = 0; r < n_rows; ++r)
        overflow += dot_rows(Xq + rows[r] * K, Wd, acc_rows + r * N, N, K);
    free(Wd);
    return overflow;
}

void o_patch_rows(const int8_t *imgq, int8_t *X, int B, int C, int H, int W, int P, int Kp)
{
    const int Ty = H / P, Tx = W / P;
    for (int b = 0; b < B; ++b)
        for (int ty = 0; ty < Ty; ++ty)
            for (int tx = 0; tx < Tx; ++tx) {
                int8_t *row = X + (((int64_t)b * Ty + ty) * Tx + tx) * Kp;
                for (int k = 0; k < Kp; ++k) row[k] = 0;
                for (int c = 0; c < C; ++c)
                    for (int py = 0; py < P; ++py)
                        for (int px = 0; px < P; ++px)
                            row[(c * P + py) * P + px] =
                                imgq[(((int64_t)b * C + c) * H + ty * P + py) * W + tx * P + px];
            }
}

int64_t o_patch_conv_acc(const int8_t *imgq, const int8_t *Wq, int32_t *acc, int B, int C,
                         int H, int W, int P, int D)
{
    const int Ty = H / P, Tx = W / P;
    int64_t macs = 0;
    for (int b = 0; b < B; ++b)
        for (int d = 0; d < D; ++d)
            for (int ty = 0; ty < Ty; ++ty)
                for (int tx = 0; tx < Tx; ++tx) {
                    int64_t sum = 0;
                    for (int c = 0; c < C; ++c)
                        for (int py = 0; py < P; ++py)
                            for (int px = 0; px < P; ++px) {
                                const int64_t w = Wq[(((int64_t)d * C + c) * P + py) * P + px];
                                const int64_t x =
                                    imgq[(((int64_t)b * C + c) * H + ty * P + py) * W + tx * P + px];
                                sum += w * x;
                                ++macs;
                            }
                    acc[(((int64_t)b * Ty + ty) * Tx + tx) * D + d] = (int32_t)sum;
                }
    return macs;
}

void o_epilogue(const int32_t *acc, const float *w_scale, float x_scale,
                const float *bias, int act, int out_type, float out_scale,
                void *Y, int64_t count, int N)
{
    for (int64_t e = 0; e < count; ++e) {
        int n = (int)(e % N);
        if (out_type == 2) {
            ((int32_t *)Y)[e] = acc[e];
            continue;
        }
        float t = (float)acc[e];          /* int32 -> binary32, ties to even */
        float s = w_scale[n] * x_scale;   /* one binary32 product */
        float y = fmaf(t, s, bias ? bias[n] : 0.0f);
        if (act == 1) {
            double yd = (double)y;
            y = (float)(0.5 * yd * erfc(-yd / sqrt(2.0)));
        }
        if (out_type == 0)
            ((uint16_t *)Y)[e] = o_f32_to_f16(y);
        else
            ((int8_t *)Y)[e] = quant_code(y, out_scale);
    }
}

/* ---- FP16 2:4 sparse model (the paper's M_SF) ---- */
void o_to_f16(const float *W, uint16_t *Wh, int64_t count)
{
    for (int64_t i = 0; i < count; ++i) Wh[i] = o_f32_to_f16(W[i]);
}

void o_compress24_f16(const uint16_t *Wh, uint16_t *vals, uint8_t *meta, int N, int K)
{
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < K / 4; ++g) {
            const uint16_t *q = Wh + (int64_t)n * K + 4 * g;
            double mag[4];
            int i0, i1;
            for (int i = 0; i < 4; ++i) mag[i] = fabs((double)o_f16_to_f32(q[i]));
            keep_two(mag, &i0, &i1);
            vals[(int64_t)n * (K / 2) + 2 * g] = q[i0];
            vals[(int64_t)n * (K / 2) + 2 * g + 1] = q[i1];
            uint8_t nib = (uint8_t)(i0 | (i1 << 2));
            uint8_t *m = meta + (int64_t)n * (K / 8) + g / 2;
            if (g & 1) *m = (uint8_t)((*m & 0x0F) | (nib << 4));
            else *m = (uint8_t)((*m & 0xF0) | nib);
        }
    }
}

void o_decompress24_f16(const uint16_t *vals, const uint8_t *meta, uint16_t *Wh, int N, int K)
{
    for (int64_t i = 0; i < (int64_t)N * K; ++i) Wh[i] = 0;
    for (int n = 0; n < N; ++n) {
        for (int g = 0; g < K / 4; ++g) {
            uint8_t byte = meta[(int64_t)n * (K / 8) + g / 2];
            uint8_t nib = (g & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 0x0F);
            int i0 = nib & 3, i1 = (nib >> 2) & 3;
            Wh[(int64_t)n * K + 4 * g + i0] = vals[(int64_t)n * (K / 2) + 2 * g];
            Wh[(int64_t)n * K + 4 * g + i1] = vals[(int64_t)n * (K / 2) + 2 * g + 1];
        }
    }
}

void o_spgemm_f16_rows(const uint16_t *X, const uint16_t *vals, const uint8_t *meta,
                       const int64_t *rows, int64_t n_rows, double *acc_rows, double *mag_rows,
                       int N, int K)
{
    uint16_t *Wh = (uint16_t *)malloc((size_t)N * (size_t)K * sizeof(uint16_t));
    double *Wd = (double *)malloc((size_t)N * (size_t)K * sizeof(double));
    if (!Wh || !Wd) {
        free(Wh);
        free(Wd);
        return;
    }
    o_decompress24_f16(vals, meta, Wh, N, K);
    for (int64_t i = 0; i < (int64_t)N * K; ++i) Wd[i] = (double)o_f16_to_f32(Wh[i]);
    for (int64_t r = 0; r < n_rows; ++r) {
        const uint16_t *xrow = X + rows[r] * K;
        for (int n = 0; n < N; ++n) {
            double sum = 0.0, mag = 0.0;
            for (int k = 0; k < K; ++k) {
                /* a product of two binary16 values has 22 significant bits: exact in binary64 */
                double p = Wd[(int64_t)n * K + k] * (double)o_f16_to_f32(xrow[k]);
                sum += p;
                mag += fabs(p);
            }
            acc_rows[r * N + n] = sum;
            if (mag_rows) mag_rows[r * N + n] = mag;
        }
    }
    free(Wh);
    free(Wd);
}

void o_epilogue_f16(const double *acc, const float *bias, int act, uint16_t *Y, int64_t count, int N)
{
    for (int64_t e = 0; e < count; ++e) {
        int n = (int)(e % N);
        float t = (float)acc[e];
        float y = t + (bias ? bias[n] : 0.0f);
        if (act == 1) {
            double yd = (double)y;
            y = (float)(0.5 * yd * erfc(-yd / sqrt(2.0)));
        }
        Y[e] = o_f32_to_f16(y);
    }
}

/* ---- INT4 4:8 pair-wise model ---- */
static int8_t quant_code_q(float x, float scale, float qmax)
{
    float q = nearbyintf(x / scale); /* ties to even */
    if (q > qmax) q = qmax;
    if (q < -qmax) q = -qmax;
    return (int8_t)q;
}

void o_prune48(const float *W, float *Wp, uint8_t *mask, int N, int K)
{
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < K / 8; ++c) {
            const float *w = W + (int64_t)n * K + 8 * c;
            double mag[4];
            for (int p = 0; p < 4; ++p) mag[p] = fabs((double)w[2 * p]) + fabs((double)w[2 * p + 1]);
            int p0, p1;
            keep_two(mag, &p0, &p1);
            for (int p = 0; p < 4; ++p) {
                int keep = (p == p0 || p == p1);
                Wp[(int64_t)n * K + 8 * c + 2 * p] = keep ? w[2 * p] : 0.0f;
                Wp[(int64_t)n * K + 8 * c + 2 * p + 1] = keep ? w[2 * p + 1] : 0.0f;
            }
            if (mask) mask[(int64_t)n * (K / 8) + c] = (uint8_t)((1u << p0) | (1u << p1));
        }
    }
}

void o_quant_weight4(const float *Wp, int8_t *Wq, float *w_scale, int N, int K)
{
    for (int n = 0; n < N; ++n) {
        const float *row = Wp + (int64_t)n * K;
        float amax = 0.0f;
        for (int k = 0; k < K; ++k) {
            float a = fabsf(row[k]);
            if (a > amax) amax = a;
        }
        float s = (amax == 0.0f) ? 1.0f : amax / 7.0f;
        w_scale[n] = s;
        for (int k = 0; k < K; ++k) Wq[(int64_t)n * K + k] = quant_code_q(row[k], s, 7.0f);
    }
}

void o_compress48(const int8_t *Wq, uint8_t *vals, uint8_t *meta, int N, int K)
{
    memset(meta, 0, (size_t)N * (size_t)(K / 16));
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < K / 8; ++c) {
            const int8_t *w = Wq + (int64_t)n * K + 8 * c;
            double mag[4];
            for (int p = 0; p < 4; ++p) mag[p] = fabs((double)w[2 * p]) + fabs((double)w[2 * p + 1]);
            int p0, p1;
            keep_two(mag, &p0, &p1);
            const int8_t kept[4] = {w[2 * p0], w[2 * p0 + 1], w[2 * p1], w[2 * p1 + 1]};
            uint8_t *v = vals + (int64_t)n * (K / 4) + 2 * c;
            v[0] = (uint8_t)((kept[0] & 0xF) | ((kept[1] & 0xF) << 4));
            v[1] = (uint8_t)((kept[2] & 0xF) | ((kept[3] & 0xF) << 4));
            uint8_t nib = (uint8_t)(p0 | (p1 << 2));
            meta[(int64_t)n * (K / 16) + c / 2] |= (uint8_t)(nib << (4 * (c & 1)));
        }
    }
}

static int8_t nibble_to_code(uint8_t nib)
{
    return (int8_t)((nib & 0x8) ? (int)nib - 16 : (int)nib); /* 4-bit two's complement */
}

void o_decompress48(const uint8_t *vals, const uint8_t *meta, int8_t *Wq, int N, int K)
{
    memset(Wq, 0, (size_t)N * (size_t)K);
    for (int n = 0; n < N; ++n) {
        for (int c = 0; c < K / 8; ++c) {
            uint8_t byte = meta[(int64_t)n * (K / 16) + c / 2];
            uint8_t nib = (uint8_t)((byte >> (4 * (c & 1))) & 0xF);
            int p0 = nib & 3, p1 = (nib >> 2) & 3;
            const uint8_t *v = vals + (int64_t)n * (K / 4) + 2 * c;
            int8_t *w = Wq + (int64_t)n * K + 8 * c;
            w[2 * p0] = nibble_to_code(v[0] & 0xF);
            w[2 * p0 + 1] = nibble_to_code(v[0] >> 4);
            w[2 * p1] = nibble_to_code(v[1] & 0xF);
            w[2 * p1 + 1] = nibble_to_code(v[1] >> 4);
        }
    }
}

void o_quant_act4(const uint16_t *X, int8_t *Xq, float *x_scale, int scale_mode, int64_t M, int K)
{
    int64_t count = M * (int64_t)K;
    float s;
    if (scale_mode == 0) {
        float amax = 0.0f;
        for (int64_t i = 0; i < count; ++i) {
            float a = fabsf(o_f16_to_f32(X[i]));
            if (a > amax) amax = a;
        }
        s = (amax == 0.0f) ? 1.0f : amax / 7.0f;
        *x_scale = s;
    } else {
        s = *x_scale;
    }
    for (int64_t i = 0; i < count; ++i) Xq[i] = quant_code_q(o_f16_to_f32(X[i]), s, 7.0f);
}

int64_t o_spgemm48_acc(const int8_t *Xq, const uint8_t *vals, const uint8_t *meta, int32_t *acc,
                       int64_t M, int N, int K)
{
    int8_t *Wd = (int8_t *)malloc((size_t)N * (size_t)K);
    if (!Wd) return -1;
    o_decompress48(vals, meta, Wd, N, K);
    int64_t overflow = 0;
    for (int64_t m = 0; m < M; ++m) overflow += dot_rows(Xq + m * K, Wd, acc + m * N, N, K);
    free(Wd);
    return overflow;
}

double o_sqnr_db(const float *ref, const float *test, int64_t count)
{
    double sig = 0.0, noise = 0.0;
    for (int64_t i = 0; i < count; ++i) {
        double r = ref[i], d = (double)ref[i] - (double)test[i];
        sig += r * r;
        noise += d * d;
    }
    return 10.0 * log10(sig / noise);
}
