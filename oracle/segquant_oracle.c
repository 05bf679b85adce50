/*
 * SegQuant CPU oracle  --  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, step-by-step implementation of the quantized linear layer that
 * combines SegLinear (Sec. 4.2.2: output- and input-segmented quantization) with
 * DualScale (Sec. 4.3.2: polarity-split activation quantization).  It exists so
 * that the CUDA library can be checked element by element; nothing in the CUDA
 * library includes, links or calls this file, and this file uses nothing of it.
 *
 * Conventions (paper notation, with nn.Linear weight order):
 *   X  [M,K] row-major activations, W [N,K] row-major weights (the paper's
 *   W in R^{k x n} transposed), Y = X W^T + b.
 *   K-partition kb[0..P] (kb[0]=0, kb[P]=K): input-segmented mode, Sec. 4.2.2 item 2.
 *   N-partition nb[0..Q] (nb[0]=0, nb[Q]=N): output-segmented mode, Sec. 4.2.2 item 1.
 *   One scalar scale per segment ("per-tensor scheme" inside a segment, App. B
 *   "Extra Hyperparameter Settings"): activations s[p] (x polarity when dual),
 *   weights s_w[p*Q+q].
 *
 * Steps, in the paper's order:
 *   1. calibration   s_+ = max(x)/q_max, s_- = |min(x)|/|q_min|   (Sec. 4.3.2, scale formula)
 *   2. weight codes  W^ = clip(round(W/s_w))                      (Sec. 3 quantizer; App. A symmetric case)
 *   3. act. codes    Q_dual(x), X_+ = max(X,0), X_- = min(X,0)    (Sec. 4.3.2)
 *   4. accumulate    X^_+ W^ and X^_- W^ per K-segment            (Sec. 4.3.2 last display; Sec. 4.2.2)
 *   5. dequantize    s_+ s_w (X^_+ W^) + s_- s_w (X^_- W^) (+ b)  (Sec. 4.3.2 last display)
 *
 * Precision: the decision "which integer code" is taken in IEEE fp32 (one fp32
 * division, then round-half-to-even), because that decision must be taken in the
 * same precision on both sides of a parity test.  Everything after the codes is
 * exact integer arithmetic (int8 codes) or fp64 (e4m3 codes, dequantization).
 *
 * Also here, for the rows next to the main path: the zero-point (asymmetric) scheme of App. A that DualScale is
 * compared with, and the activation / per-channel multiplier of the act-to-linear segment in front of the
 * quantizer (Sec. 4.3.2, Sec. 4.2.2 last paragraph).
 *
 * Pins (see tests/test_oracle_pins.py): library quantizers of torch on CPU,
 * on-grid exact reconstruction, brute-force dot products, reduction of one
 * segment to per-tensor, reduction of equal dual scales to symmetric, the
 * half-step error bound, the worked range example of Sec. 4.3.1.
 * The e4m3 encoder is pinned to torch's float8_e4m3fn cast; the paper gives no
 * FP8 format detail, so beyond that cast the FP8 reading itself is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ helpers */

static int seg_of(int64_t i, int nseg, const int32_t *bounds)
{
    int s = 0;
    while (s + 1 < nseg && i >= bounds[s + 1]) s++;
    return s;
}

/* round-half-to-even of an fp32 value (default rounding mode). */
static float rne(float v) { return nearbyintf(v); }

/* ------------------------------------------------------------ e4m3 (finite) */
/* 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities; S.1111.111 is
 * NaN; largest finite value 448; subnormals m * 2^-9.                        */

double sqo_e4m3_decode(uint8_t c)
{
    int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);
    else        v = ldexp(1.0 + m / 8.0, e - 7);
    return sign ? -v : v;
}

/* round-to-nearest-even, saturating to +-448; -0 is written as +0. */
uint8_t sqo_e4m3_encode(float v)
{
    if (v != v) return 0x7F;
    uint8_t sign = (v < 0.0f) ? 0x80 : 0x00;
    double a = fabs((double)v);
    uint8_t mag;
    if (a >= 448.0) {
        mag = 0x7E;
    } else if (a < ldexp(1.0, -6)) {
        mag = (uint8_t)nearbyint(ldexp(a, 9));          /* 0..8; 8 is the first normal */
    } else {
        int e;
        double f = frexp(a, &e);                        /* a = f*2^e, f in [0.5,1) */
        double frac = f * 2.0 - 1.0;                    /* a = (1+frac)*2^(e-1) */
        int q = (int)nearbyint(frac * 8.0);
        int ex = e - 1;
        if (q == 8) { q = 0; ex += 1; }
        int code = ((ex + 7) << 3) | q;
        if (code > 0x7E) code = 0x7E;
        mag = (uint8_t)code;
    }
    if (mag == 0) return 0x00;
    return sign | mag;
}

/* ------------------------------------------------------- step 1: calibration */

/* Activation scales per K-segment from calibration rows (Sec. 4.3.2 scale formula,
 * strict min/max, App. B "Dual Scale Sensitivity Analysis").
 * dual:   s_pos[p] = max(mx,0)/q_max, s_neg[p] = max(-mn,0)/q_min_abs
 * single: s_pos[p] = max(|mx|,|mn|)/q_max   (s_neg untouched)
 * An extremum of 0 gives scale 1 (that polarity then only produces code 0). */
void sqo_calib_act(const float *X, int64_t rows, int64_t K, int64_t ld,
                   int P, const int32_t *kb, int dual,
                   float q_max, float q_min_abs, float *s_pos, float *s_neg)
{
    (void)K;
    for (int p = 0; p < P; p++) {
        float mx = -INFINITY, mn = INFINITY;
        for (int64_t r = 0; r < rows; r++)
            for (int64_t k = kb[p]; k < kb[p + 1]; k++) {
                float x = X[r * ld + k];
                if (x > mx) mx = x;
                if (x < mn) mn = x;
            }
        if (dual) {
            float hi = mx > 0.0f ? mx : 0.0f;
            float lo = mn < 0.0f ? -mn : 0.0f;
            s_pos[p] = hi > 0.0f ? hi / q_max : 1.0f;
            s_neg[p] = lo > 0.0f ? lo / q_min_abs : 1.0f;
        } else {
            float a = fabsf(mx) > fabsf(mn) ? fabsf(mx) : fabsf(mn);
            s_pos[p] = a > 0.0f ? a / q_max : 1.0f;
        }
    }
}

/* Weight scales per (K-segment p, N-segment q) block: s_w[p*Q+q] = max|W|/w_max. */
void sqo_calib_weight(const float *W, int64_t N, int64_t K, int64_t ld,
                      int P, const int32_t *kb, int Q, const int32_t *nb,
                      float w_max, float *s_w)
{
    (void)N; (void)K;
    for (int p = 0; p < P; p++)
        for (int q = 0; q < Q; q++) {
            float a = 0.0f;
            for (int64_t n = nb[q]; n < nb[q + 1]; n++)
                for (int64_t k = kb[p]; k < kb[p + 1]; k++) {
                    float w = fabsf(W[n * ld + k]);
                    if (w > a) a = w;
                }
            s_w[p * Q + q] = a > 0.0f ? a / w_max : 1.0f;
        }
}

/* ---------------------------------------------- steps 2 and 3: quantization */

static float clampf(float v, float lo, float hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* Q_dual (Sec. 4.3.2) with the clip of the Sec. 3 quantizer; int8 codes.
 * s_neg == NULL selects the single-scale symmetric quantizer: c_pos receives
 * clip(round(x/s), -q_max, q_max) and c_neg is not written.
 * Dual: x >= 0 -> c_pos = clip(round(x/s_pos), 0, q_max), c_neg = 0
 *       x <  0 -> c_neg = clip(round(x/s_neg), -q_min_abs, 0), c_pos = 0      */
void sqo_quantize_act_i8(const float *X, int64_t M, int64_t K, int64_t ld,
                         int P, const int32_t *kb,
                         const float *s_pos, const float *s_neg,
                         float q_max, float q_min_abs,
                         int8_t *c_pos, int8_t *c_neg, int64_t ldc)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t k = 0; k < K; k++) {
            int p = seg_of(k, P, kb);
            float x = X[m * ld + k];
            if (!s_neg) {
                float v = x / s_pos[p];
                c_pos[m * ldc + k] = (int8_t)clampf(rne(v), -q_max, q_max);
            } else if (x >= 0.0f) {
                float v = x / s_pos[p];
                c_pos[m * ldc + k] = (int8_t)clampf(rne(v), 0.0f, q_max);
                c_neg[m * ldc + k] = 0;
            } else {
                float v = x / s_neg[p];
                c_neg[m * ldc + k] = (int8_t)clampf(rne(v), -q_min_abs, 0.0f);
                c_pos[m * ldc + k] = 0;
            }
        }
}

/* Same quantizer with e4m3 codes: the "round" of the formula is the
 * round-to-nearest-even cast to e4m3 and the clip is to +-448 (per polarity:
 * [0,448] and [-448,0]).                                                      */
void sqo_quantize_act_e4m3(const float *X, int64_t M, int64_t K, int64_t ld,
                           int P, const int32_t *kb,
                           const float *s_pos, const float *s_neg,
                           uint8_t *c_pos, uint8_t *c_neg, int64_t ldc)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t k = 0; k < K; k++) {
            int p = seg_of(k, P, kb);
            float x = X[m * ld + k];
            if (!s_neg) {
                c_pos[m * ldc + k] = sqo_e4m3_encode(clampf(x / s_pos[p], -448.0f, 448.0f));
            } else if (x >= 0.0f) {
                c_pos[m * ldc + k] = sqo_e4m3_encode(clampf(x / s_pos[p], 0.0f, 448.0f));
                c_neg[m * ldc + k] = 0;
            } else {
                c_neg[m * ldc + k] = sqo_e4m3_encode(clampf(x / s_neg[p], -448.0f, 0.0f));
                c_pos[m * ldc + k] = 0;
            }
        }
}

/* Weight codes, one scale per (p,q) block (Sec. 4.2.2: each W_i quantized separately). */
void sqo_quantize_weight_i8(const float *W, int64_t N, int64_t K, int64_t ld,
                            int P, const int32_t *kb, int Q, const int32_t *nb,
                            const float *s_w, float w_max, int8_t *Wq, int64_t ldq)
{
    for (int64_t n = 0; n < N; n++) {
        int q = seg_of(n, Q, nb);
        for (int64_t k = 0; k < K; k++) {
            int p = seg_of(k, P, kb);
            float v = W[n * ld + k] / s_w[p * Q + q];
            Wq[n * ldq + k] = (int8_t)clampf(rne(v), -w_max, w_max);
        }
    }
}

void sqo_quantize_weight_e4m3(const float *W, int64_t N, int64_t K, int64_t ld,
                              int P, const int32_t *kb, int Q, const int32_t *nb,
                              const float *s_w, uint8_t *Wq, int64_t ldq)
{
    for (int64_t n = 0; n < N; n++) {
        int q = seg_of(n, Q, nb);
        for (int64_t k = 0; k < K; k++) {
            int p = seg_of(k, P, kb);
            float v = W[n * ld + k] / s_w[p * Q + q];
            Wq[n * ldq + k] = sqo_e4m3_encode(clampf(v, -448.0f, 448.0f));
        }
    }
}

/* ------------------------------------------------------- step 4: accumulate */

/* acc[p][m][n] = sum_{k in segment p} Xq[m][k] * Wq[n][k]   (exact integers).
 * Returns the number of sums that did not fit int32 (must be 0).             */
int64_t sqo_accumulate_i8(const int8_t *Xq, int64_t ldx, const int8_t *Wq, int64_t ldw,
                          int64_t M, int64_t N, int64_t K,
                          int P, const int32_t *kb, int32_t *acc)
{
    int64_t overflow = 0;
    (void)K;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t m = 0; m < M; m++)
        for (int p = 0; p < P; p++)
            for (int64_t n = 0; n < N; n++) {
                int64_t s = 0;
                for (int64_t k = kb[p]; k < kb[p + 1]; k++)
                    s += (int64_t)Xq[m * ldx + k] * (int64_t)Wq[n * ldw + k];
                if (s > INT32_MAX || s < INT32_MIN) overflow++;
                acc[((int64_t)p * M + m) * N + n] = (int32_t)s;
            }
    return overflow;
}

/* Same contraction on e4m3 codes, summed in fp64 (every product and, for
 * K <= 2^17, every partial sum is exactly representable).                    */
void sqo_accumulate_e4m3(const uint8_t *Xq, int64_t ldx, const uint8_t *Wq, int64_t ldw,
                         int64_t M, int64_t N, int64_t K,
                         int P, const int32_t *kb, double *acc)
{
    double lut[256];
    for (int c = 0; c < 256; c++) lut[c] = sqo_e4m3_decode((uint8_t)c);
    (void)K;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; m++)
        for (int p = 0; p < P; p++)
            for (int64_t n = 0; n < N; n++) {
                double s = 0.0;
                for (int64_t k = kb[p]; k < kb[p + 1]; k++)
                    s += lut[Xq[m * ldx + k]] * lut[Wq[n * ldw + k]];
                acc[((int64_t)p * M + m) * N + n] = s;
            }
}

/* ------------------------------------------------------- step 5: dequantize */

/* y[m][n] = sum_p ( s_pos[p] s_w[p][q(n)] acc_pos[p][m][n]
 *                 + s_neg[p] s_w[p][q(n)] acc_neg[p][m][n] ) + bias[n]   in fp64.
 * acc_neg / s_neg NULL: single-scale layer (App. A symmetric recovery).
 * ysum_abs (optional) receives sum of |terms| + |bias|, the scale against which
 * an fp32 evaluation of the same expression is judged.                        */
void sqo_dequant(const double *acc_pos, const double *acc_neg,
                 int64_t M, int64_t N, int P, int Q, const int32_t *nb,
                 const float *s_pos, const float *s_neg, const float *s_w,
                 const float *bias, double *y, double *ysum_abs)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            int q = seg_of(n, Q, nb);
            double v = 0.0, av = 0.0;
            for (int p = 0; p < P; p++) {
                int64_t i = ((int64_t)p * M + m) * N + n;
                double sw = (double)s_w[p * Q + q];
                double t = (double)s_pos[p] * sw * acc_pos[i];
                v += t; av += fabs(t);
                if (acc_neg) {
                    double u = (double)s_neg[p] * sw * acc_neg[i];
                    v += u; av += fabs(u);
                }
            }
            if (bias) { v += (double)bias[n]; av += fabs((double)bias[n]); }
            y[m * N + n] = v;
            if (ysum_abs) ysum_abs[m * N + n] = av;
        }
}

uint16_t sqo_bf16_from_f64(double v);

/* ------------------------------------------- comparison scheme: zero-point (asymmetric) quantization */

/* App. A writes the asymmetric quantizer as X^ = round(X / s_X) + z_X with an integer zero-point, recovered by
 * X ~ s_X (X^ - z_X); this is the form taken here (the Sec. 3 display puts z inside the quotient instead, and
 * its inverse does not match it).  One (s, z) pair per K-segment, from strict min/max over the calibration
 * rows with the range widened to contain 0:
 *   lo = min(min x, 0), hi = max(max x, 0), s = (hi - lo) / (q_max - q_min), z = q_min - round(lo / s)
 * so that lo maps to q_min.  A zero range gives s = 1, z = 0.                                              */
void sqo_calib_act_asym(const float *X, int64_t rows, int64_t K, int64_t ld,
                        int P, const int32_t *kb, float q_min, float q_max,
                        float *s, int32_t *z)
{
    (void)K;
    for (int p = 0; p < P; p++) {
        float hi = 0.0f, lo = 0.0f;
        for (int64_t r = 0; r < rows; r++)
            for (int64_t k = kb[p]; k < kb[p + 1]; k++) {
                float x = X[r * ld + k];
                if (x > hi) hi = x;
                if (x < lo) lo = x;
            }
        float range = hi - lo;
        if (range > 0.0f) {
            s[p] = range / (q_max - q_min);
            float zf = q_min - rne(lo / s[p]);
            z[p] = (int32_t)clampf(zf, q_min, q_max);
        } else {
            s[p] = 1.0f;
            z[p] = 0;
        }
    }
}

/* X^ = clip(round(x / s[p]) + z[p], q_min, q_max)   (App. A asymmetric quantizer, Sec. 3 clip), int8 codes. */
void sqo_quantize_act_asym_i8(const float *X, int64_t M, int64_t K, int64_t ld,
                              int P, const int32_t *kb, const float *s, const int32_t *z,
                              float q_min, float q_max, int8_t *c, int64_t ldc)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t k = 0; k < K; k++) {
            int p = seg_of(k, P, kb);
            float v = rne(X[m * ld + k] / s[p]);
            v = clampf(v, -1.0e6f, 1.0e6f);                     /* keeps the integer sum below in range */
            c[m * ldc + k] = (int8_t)clampf(v + (float)z[p], q_min, q_max);
        }
}

/* xsum[p][m] = sum over K-segment p of X^[m][k];  wsum[p][n] = sum over K-segment p of W^[n][k]
 * (the rowsum terms of the App. A recovery; "rowsum(W^)" there sums W in R^{k x n} over k).               */
void sqo_segment_sums_i8(const int8_t *A, int64_t lda, int64_t rows, int P, const int32_t *kb, int64_t *out)
{
    for (int p = 0; p < P; p++)
        for (int64_t r = 0; r < rows; r++) {
            int64_t t = 0;
            for (int64_t k = kb[p]; k < kb[p + 1]; k++) t += A[r * lda + k];
            out[(int64_t)p * rows + r] = t;
        }
}

/* App. A asymmetric recovery, per (K-segment, N-segment) block and summed over K-segments, in fp64:
 *   y[m][n] = sum_p s_x[p] s_w[p][q] ( acc[p][m][n] - z_x[p] wsum[p][n] - z_w[p][q] xsum[p][m]
 *                                      + k_p z_x[p] z_w[p][q] ) + bias[n],      k_p = kb[p+1] - kb[p].
 * z_w may be NULL (symmetric weights).  ysum_abs as in sqo_dequant, every term counted separately.        */
void sqo_dequant_asym(const double *acc, const int64_t *xsum, const int64_t *wsum,
                      int64_t M, int64_t N, int P, const int32_t *kb, int Q, const int32_t *nb,
                      const float *s_x, const int32_t *z_x, const float *s_w, const int32_t *z_w,
                      const float *bias, double *y, double *ysum_abs)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            int q = seg_of(n, Q, nb);
            double v = 0.0, av = 0.0;
            for (int p = 0; p < P; p++) {
                double c = (double)s_x[p] * (double)s_w[p * Q + q];
                double zx = (double)z_x[p], zw = z_w ? (double)z_w[p * Q + q] : 0.0;
                double kp = (double)(kb[p + 1] - kb[p]);
                double t0 = c * acc[((int64_t)p * M + m) * N + n];
                double t1 = c * zx * (double)wsum[(int64_t)p * N + n];
                double t2 = c * zw * (double)xsum[(int64_t)p * M + m];
                double t3 = c * kp * zx * zw;
                v += t0 - t1 - t2 + t3;
                av += fabs(t0) + fabs(t1) + fabs(t2) + fabs(t3);
            }
            if (bias) { v += (double)bias[n]; av += fabs((double)bias[n]); }
            y[m * N + n] = v;
            if (ysum_abs) ysum_abs[m * N + n] = av;
        }
}

/* With symmetric weights the zero-point term does not depend on the row and folds into the bias offline:
 *   bias'[n] = bias[n] - sum_p s_x[p] s_w[p][q(n)] z_x[p] wsum[p][n]      (fp64)                          */
void sqo_fold_zero_point(const int64_t *wsum, int64_t N, int P, int Q, const int32_t *nb,
                         const float *s_x, const int32_t *z_x, const float *s_w, const float *bias,
                         double *bias_folded)
{
    for (int64_t n = 0; n < N; n++) {
        int q = seg_of(n, Q, nb);
        double v = bias ? (double)bias[n] : 0.0;
        for (int p = 0; p < P; p++)
            v -= (double)s_x[p] * (double)s_w[p * Q + q] * (double)z_x[p] * (double)wsum[(int64_t)p * N + n];
        bias_folded[n] = v;
    }
}

/* --------------------------------------------- act-to-linear segment in front of the quantizer (Sec. 4.3.2) */

/* The activation functions DualScale is applied behind (App. B: SiLU, GELU), in fp64 from their definitions:
 *   SiLU(h) = h / (1 + exp(-h)),   GELU(h) = h Phi(h) = (h / 2) erfc(-h / sqrt 2).                          */
double sqo_silu(double h) { return h / (1.0 + exp(-h)); }
double sqo_gelu(double h) { return 0.5 * h * erfc(-h / sqrt(2.0)); }

/* act: 1 = SiLU, 2 = GELU.  The value is rounded ONCE from fp64 to the dtype the unfused graph would have
 * stored it in (bf16 if stored_bf16, else fp32) and returned as fp32; `exact` (optional) receives the fp64 value. */
void sqo_activation(const float *H, int64_t n, int act, int stored_bf16, float *out, double *exact)
{
    for (int64_t i = 0; i < n; i++) {
        double a = act == 1 ? sqo_silu((double)H[i]) : sqo_gelu((double)H[i]);
        if (exact) exact[i] = a;
        if (stored_bf16) {
            uint32_t bits = (uint32_t)sqo_bf16_from_f64(a) << 16;
            float f;
            memcpy(&f, &bits, 4);
            out[i] = f;
        } else {
            out[i] = (float)a;
        }
    }
}

/* Gated GELU (App. B names GEGLU among the polarity-sensitive activations that feed DualScale layers, without a
 * form; the form taken is that of the gated feed-forward: the 2K columns of the pre-activation row are two
 * halves, value half first, gate half second, and a[k] = H[k] * GELU(H[K + k])).  The product is exact in fp64
 * up to one rounding and, as above, the value is rounded ONCE to the stored dtype.                             */
double sqo_geglu(double value, double gate) { return value * sqo_gelu(gate); }

void sqo_activation_gated(const float *H, int64_t M, int64_t K, int64_t ld, int stored_bf16, float *out, int64_t ldo,
                          double *exact)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t k = 0; k < K; k++) {
            double a = sqo_geglu((double)H[m * ld + k], (double)H[m * ld + K + k]);
            if (exact) exact[m * ldo + k] = a;
            if (stored_bf16) {
                uint32_t bits = (uint32_t)sqo_bf16_from_f64(a) << 16;
                float f;
                memcpy(&f, &bits, 4);
                out[m * ldo + k] = f;
            } else {
                out[m * ldo + k] = (float)a;
            }
        }
}

/* Per-channel multiplier in front of the quantizer (Sec. 4.2.2 last paragraph: SmoothQuant's migration, one
 * strength per segment; the multiplier m[k] = 1 / smoothing factor is made offline): out = fl32(x * m[k]).   */
void sqo_smooth(const float *X, int64_t M, int64_t K, int64_t ld, const float *mult, float *out, int64_t ldo)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t k = 0; k < K; k++)
            out[m * ldo + k] = X[m * ld + k] * mult[k];
}

/* ---------------------------------- 4-bit weights with per-channel scales, per-token activation scales (W4A8) */

/* App. B "Extra Hyperparameter Settings": in the 4-bit settings weights are quantized per channel and
 * activations dynamically per token.  Combined with input segmentation (Sec. 4.2.2 item 2) every row r of a
 * matrix gets one scale per K-segment p from its own extrema:
 *   dual:   s_pos[r*P+p] = max(max x, 0) / q_max,  s_neg[r*P+p] = max(-min x, 0) / q_min_abs   (Sec. 4.3.2)
 *   single: s_pos[r*P+p] = max|x| / q_max
 * (an extremum of 0 gives scale 1) and is quantized with it by the same quantizer as everywhere else.
 * Activations: rows are tokens, q_max = 127.  Weights: rows are output channels, q_max = 7 (symmetric 4-bit
 * codes in [-7, 7]), single scale.                                                                          */
void sqo_quantize_per_row_i8(const float *X, int64_t M, int64_t K, int64_t ld,
                             int P, const int32_t *kb, int dual, float q_max, float q_min_abs,
                             float *s_pos, float *s_neg, int8_t *c_pos, int8_t *c_neg, int64_t ldc)
{
    for (int64_t m = 0; m < M; m++) {
        sqo_calib_act(X + m * ld, 1, K, ld, P, kb, dual, q_max, q_min_abs, s_pos + m * P, dual ? s_neg + m * P : NULL);
        sqo_quantize_act_i8(X + m * ld, 1, K, ld, P, kb, s_pos + m * P, dual ? s_neg + m * P : NULL, q_max, q_min_abs,
                            c_pos + m * ldc, dual ? c_neg + m * ldc : NULL, ldc);
    }
}

/* Two 4-bit codes per byte: code 2j in the low nibble, code 2j+1 in the high nibble, two's complement. */
void sqo_pack_w4(const int8_t *Wq, int64_t N, int64_t K, int64_t ld, uint8_t *out, int64_t ldo)
{
    for (int64_t n = 0; n < N; n++)
        for (int64_t j = 0; j < K / 2; j++)
            out[n * ldo + j] = (uint8_t)((Wq[n * ld + 2 * j] & 0xF) | ((Wq[n * ld + 2 * j + 1] & 0xF) << 4));
}
void sqo_unpack_w4(const uint8_t *in, int64_t N, int64_t K, int64_t ldi, int8_t *Wq, int64_t ld)
{
    for (int64_t n = 0; n < N; n++)
        for (int64_t j = 0; j < K / 2; j++) {
            uint8_t b = in[n * ldi + j];
            Wq[n * ld + 2 * j] = (int8_t)(((b & 0xF) ^ 8) - 8);
            Wq[n * ld + 2 * j + 1] = (int8_t)(((b >> 4) ^ 8) - 8);
        }
}

/* y[m][n] = sum_p ( s_pos[m*P+p] s_w[n*P+p] acc_pos[p][m][n] + s_neg[m*P+p] s_w[n*P+p] acc_neg[p][m][n] ) + bias[n]
 * in fp64 (Sec. 4.3.2 recombination with per-token and per-channel scales).                                  */
void sqo_dequant_per_token(const double *acc_pos, const double *acc_neg, int64_t M, int64_t N, int P,
                           const float *s_pos, const float *s_neg, const float *s_w, const float *bias,
                           double *y, double *ysum_abs)
{
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            double v = 0.0, av = 0.0;
            for (int p = 0; p < P; p++) {
                int64_t i = ((int64_t)p * M + m) * N + n;
                double sw = (double)s_w[n * P + p];
                double t = (double)s_pos[m * P + p] * sw * acc_pos[i];
                v += t; av += fabs(t);
                if (acc_neg) {
                    double u = (double)s_neg[m * P + p] * sw * acc_neg[i];
                    v += u; av += fabs(u);
                }
            }
            if (bias) { v += (double)bias[n]; av += fabs((double)bias[n]); }
            y[m * N + n] = v;
            if (ysum_abs) ysum_abs[m * N + n] = av;
        }
}

/* fp64 -> bf16 bit pattern, round-to-nearest-even directly from the fp64 value
 * (no intermediate fp32 rounding).  Finite inputs within bf16 range only.    */
uint16_t sqo_bf16_from_f64(double v)
{
    if (v != v) return 0x7FC0;
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (a == 0.0) return sign;
    int e;
    double f = frexp(a, &e);                 /* a = f*2^e, f in [0.5,1) */
    int ex = e - 1;                          /* a = (2f)*2^ex, 2f in [1,2) */
    if (ex < -126) {                         /* bf16 subnormal: multiples of 2^-133 */
        double q = nearbyint(ldexp(a, 133));
        return sign | (uint16_t)q;           /* q == 128 carries into the first normal */
    }
    double q = nearbyint((f * 2.0 - 1.0) * 128.0);
    if (q == 128.0) { q = 0.0; ex += 1; }
    if (ex > 127) return sign | 0x7F80;
    return sign | (uint16_t)(((ex + 127) << 7) | (int)q);
}

void sqo_bf16_from_f64_array(const double *v, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; i++) out[i] = sqo_bf16_from_f64(v[i]);
}

int sqo_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
