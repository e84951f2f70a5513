/*
 * CPU oracle for the {-1,+1} encoded quantized layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  Nothing in the product path may call it;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg do.
 * It shares no code, header, table or helper with the CUDA sources.
 *
 * What the method computes (all of it an exact integer function of the codes):
 *
 *   - Quantizer (Eq. 15 with the rounding <.> read as round-half-up, and the
 *     Table 2 mapping between quantized numbers and encoded states): a real
 *     x in [-1,1] goes to the level index
 *         u = floor((2^b-1)(x+1)/2 + 1/2) = floor((2^b-1) x / 2) + 2^(b-1)
 *     and to the odd integer q = 2u - (2^b-1), |q| <= 2^b-1 (Eq. 20).
 *     The bits of u are the {-1,+1} code of Eq. 10 (bit 1 <-> +1, bit 0 <-> -1,
 *     bit p has weight 2^p, "x = x1 + 2 x2").  A max-abs scale s generalises
 *     the paper's fixed [-1,1] range: x/s is clamped to [-1,1] (HTanh, Table 1).
 *     The decision is taken in fp32 with two separately rounded multiplies so
 *     that a GPU can reproduce every code bit for bit.
 *   - Layer product (Eq. 1-2, which Eq. 7-10 decompose and re-assemble exactly):
 *     acc[r][c] = sum_t qa[r][t] * qb[c][t].  No bit-planes, no popcount here.
 *   - Convolution: the same dot product over a sliding window; taps that fall
 *     outside the image contribute 0 (true zero padding).
 *   - Decoder scale (Eq. 18, the "1/9" of Fig. 1 at 2x2 bits):
 *     out = acc * (s_a / (2^a-1)) * (s_w[c] / (2^w-1)).
 *
 * Every function below is pinned by tests that do not use this file's own
 * formulas: Table 2's printed values, Eq. 15 evaluated in exact rationals, the
 * trigonometric encoders of Eq. 11, brute force of the branch decomposition
 * over all codes, the 1-bit sign-dot, closed forms and conv-vs-im2col.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <stddef.h>

/* ---- a0: scale = max |x| (NaNs ignored), per tensor or per row ----
 * With hrelu != 0 the range is that of max(x, 0), the HReLU side of Table 1. */
void mpq_oracle_absmax(const float* x, int64_t rows, int64_t k, int64_t ldx,
                       int per_row, int hrelu, float* scale_out)
{
    float tensor_max = 0.0f;
    for (int64_t r = 0; r < rows; ++r) {
        float row_max = 0.0f;
        for (int64_t t = 0; t < k; ++t) {
            /* HReLU (Table 1) zeroes the negative side before the range is taken */
            float v = hrelu ? x[r * ldx + t] : fabsf(x[r * ldx + t]);
            if (v == v && v > row_max) row_max = v;
        }
        if (per_row) scale_out[r] = row_max;
        if (row_max > tensor_max) tensor_max = row_max;
    }
    if (!per_row) scale_out[0] = tensor_max;
}

/* ---- a1: one float -> level index u in [0, 2^b-1]  (Eq. 15, Table 2) ---- */
static int level_index(float x, float inv_s, int bits, int hrelu)
{
    const int H = 1 << (bits - 1);
    const float half_L = 0.5f * (float)((1 << bits) - 1);
    float t = x * inv_s;          /* first rounded multiply: x / s          */
    float y = t * half_L;         /* second rounded multiply: (2^b-1) x / 2 */
    if (y != y) y = 0.0f;         /* NaN -> the level just above zero       */
    if (hrelu && y < 0.0f) y = 0.0f;                 /* HReLU: [0,1] (Table 1) */
    if (y < (float)(-H)) y = (float)(-H);            /* HTanh clamp, low   */
    if (y > (float)H - 0.5f) y = (float)H - 0.5f;    /* HTanh clamp, high  */
    return (int)floorf(y) + H;
}

static float inverse_scale(float s)
{
    return (s > 0.0f && isfinite(s)) ? 1.0f / s : 0.0f;
}

/* Quantize a [rows x k] matrix (row stride ldx) to odd integers q (int16, dense
 * [rows x k]).  scale has 1 entry (per tensor) or rows entries (per row). */
void mpq_oracle_quantize(const float* x, int64_t rows, int64_t k, int64_t ldx,
                         const float* scale, int per_row, int bits, int hrelu, int16_t* q)
{
    const int L = (1 << bits) - 1;
    for (int64_t r = 0; r < rows; ++r) {
        const float inv = inverse_scale(per_row ? scale[r] : scale[0]);
        for (int64_t t = 0; t < k; ++t) {
            int u = level_index(x[r * ldx + t], inv, bits, hrelu);
            q[r * k + t] = (int16_t)(2 * u - L);
        }
    }
}

/* ---- The encoder in its trigonometric form (Section 3.2, Eq. 11; other widths follow the same
 * family: the highest bit has half a period on [-1,1] scaled by (2^b-1)/2^b, every lower bit
 * doubles the frequency and flips the sign).  For y = clamp(x/s) in [-1,1]:
 *     bit b-1 (highest)   = sign( sin((2^b-1)/2^b * pi * y))
 *     bit m-1, 1 <= m < b = sign(-sin((2^b-1)/2^m * pi * y))
 * with +1 stored as 1 and -1 as 0; the level index is the number those bits spell.
 * At a zero of a sine (a level boundary, where Eq. 15 has a tie) the sign is that of the sine just
 * ABOVE the zero, i.e. the sign of its slope there: the tie goes to the upper level, as the
 * round-half-up reading of Eq. 15 does.  (x = 0 is a zero of every one of the sines; taking
 * sign(0) = +1 for all of them would spell the top level.)
 * The argument t = (2^b-1)/2^m * y is formed in fp32 (one rounded multiply: the multiplier is
 * exact), the sine itself in double; a t that is a whole number is a zero of the sine.  This
 * route and the level-index route (level_index above) agree except within a rounding of a zero
 * of a sine, where each takes its own decision. */
static int trig_level_index(float x, float inv_s, int bits, int hrelu)
{
    float y = x * inv_s;
    if (y != y) y = 0.0f;                       /* NaN -> 0, the tie that goes to the level above zero */
    if (hrelu && y < 0.0f) y = 0.0f;
    if (y < -1.0f) y = -1.0f;
    if (y > 1.0f) y = 1.0f;
    const int L = (1 << bits) - 1;
    int u = 0;
    for (int m = 1; m <= bits; ++m) {
        const float t = y * ((float)L / (float)(1 << m));
        const double pi_t = 3.14159265358979323846 * (double)t;
        double sine = (t == floorf(t)) ? cos(pi_t) : sin(pi_t);   /* at a zero: the slope's sign */
        if (m < bits) sine = -sine;
        if (sine > 0.0) u |= 1 << (m - 1);
    }
    return u;
}

void mpq_oracle_quantize_trig(const float* x, int64_t rows, int64_t k, int64_t ldx,
                              const float* scale, int per_row, int bits, int hrelu, int16_t* q)
{
    const int L = (1 << bits) - 1;
    for (int64_t r = 0; r < rows; ++r) {
        const float inv = inverse_scale(per_row ? scale[r] : scale[0]);
        for (int64_t t = 0; t < k; ++t)
            q[r * k + t] = (int16_t)(2 * trig_level_index(x[r * ldx + t], inv, bits, hrelu) - L);
    }
}

/* ---- a3+a4: acc[r][c] = sum_t qa[r][t] qb[c][t]   (Eq. 1-2) ----
 * Returns the number of outputs that do not fit int32 (0 when all fit). */
int64_t mpq_oracle_gemm(const int16_t* qa, const int16_t* qb,
                        int64_t m, int64_t n, int64_t k, int32_t* acc)
{
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t r = 0; r < m; ++r) {
        for (int64_t c = 0; c < n; ++c) {
            int64_t s = 0;
            for (int64_t t = 0; t < k; ++t)
                s += (int64_t)qa[r * k + t] * (int64_t)qb[c * k + t];
            if (s > INT32_MAX || s < INT32_MIN) ++overflow;
            acc[r * n + c] = (int32_t)s;
        }
    }
    return overflow;
}

/* ---- a6: direct convolution on the decoded integers ----
 * qx [N][C][H][W], qw [O][C][KH][KW], acc [N][O][Ho][Wo],
 * Ho = (H + 2 pad - KH)/stride + 1.  Out-of-image taps add 0. */
int64_t mpq_oracle_conv(const int16_t* qx, int64_t N, int64_t C, int64_t H, int64_t W,
                        const int16_t* qw, int64_t O, int64_t KH, int64_t KW,
                        int64_t stride, int64_t pad, int32_t* acc)
{
    const int64_t Ho = (H + 2 * pad - KH) / stride + 1;
    const int64_t Wo = (W + 2 * pad - KW) / stride + 1;
    int64_t overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(+ : overflow)
    for (int64_t b = 0; b < N; ++b) {
        for (int64_t o = 0; o < O; ++o) {
            for (int64_t oh = 0; oh < Ho; ++oh) {
                for (int64_t ow = 0; ow < Wo; ++ow) {
                    int64_t s = 0;
                    for (int64_t c = 0; c < C; ++c) {
                        for (int64_t kh = 0; kh < KH; ++kh) {
                            const int64_t ih = oh * stride + kh - pad;
                            if (ih < 0 || ih >= H) continue;
                            for (int64_t kw = 0; kw < KW; ++kw) {
                                const int64_t iw = ow * stride + kw - pad;
                                if (iw < 0 || iw >= W) continue;
                                s += (int64_t)qx[((b * C + c) * H + ih) * W + iw] *
                                     (int64_t)qw[((o * C + c) * KH + kh) * KW + kw];
                            }
                        }
                    }
                    if (s > INT32_MAX || s < INT32_MIN) ++overflow;
                    acc[((b * O + o) * Ho + oh) * Wo + ow] = (int32_t)s;
                }
            }
        }
    }
    return overflow;
}

/* ---- deconvolution (transposed convolution) on the decoded integers (Section 3.1 names the
 * deconvolution layer among those the decomposition applies to) ----
 * qx [N][C][H][W], qw [O][C][KH][KW] (output channel first), acc [N][O][Ho][Wo],
 * Ho = (H - 1) stride - 2 pad + KH.  Written as the definition: every input pixel spreads its
 * value, times the filter, over the output window that starts at (ih stride - pad, iw stride - pad);
 * what falls outside the output is dropped.  Output positions that no input reaches stay 0. */
int64_t mpq_oracle_deconv(const int16_t* qx, int64_t N, int64_t C, int64_t H, int64_t W,
                          const int16_t* qw, int64_t O, int64_t KH, int64_t KW,
                          int64_t stride, int64_t pad, int32_t* acc)
{
    const int64_t Ho = (H - 1) * stride - 2 * pad + KH;
    const int64_t Wo = (W - 1) * stride - 2 * pad + KW;
    int64_t overflow = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(+ : overflow)
    for (int64_t b = 0; b < N; ++b) {
        for (int64_t o = 0; o < O; ++o) {
            int64_t* sum = (int64_t*)calloc((size_t)(Ho * Wo), sizeof(int64_t));
            for (int64_t c = 0; c < C; ++c) {
                for (int64_t ih = 0; ih < H; ++ih) {
                    for (int64_t iw = 0; iw < W; ++iw) {
                        const int64_t v = qx[((b * C + c) * H + ih) * W + iw];
                        for (int64_t kh = 0; kh < KH; ++kh) {
                            const int64_t oh = ih * stride - pad + kh;
                            if (oh < 0 || oh >= Ho) continue;
                            for (int64_t kw = 0; kw < KW; ++kw) {
                                const int64_t ow = iw * stride - pad + kw;
                                if (ow < 0 || ow >= Wo) continue;
                                sum[oh * Wo + ow] += v * (int64_t)qw[((o * C + c) * KH + kh) * KW + kw];
                            }
                        }
                    }
                }
            }
            for (int64_t i = 0; i < Ho * Wo; ++i) {
                if (sum[i] > INT32_MAX || sum[i] < INT32_MIN) ++overflow;
                acc[(b * O + o) * Ho * Wo + i] = (int32_t)sum[i];
            }
            free(sum);
        }
    }
    return overflow;
}

/* One output element of the convolution (sampling a large layer). */
int64_t mpq_oracle_conv_at(const int16_t* qx, int64_t C, int64_t H, int64_t W,
                           const int16_t* qw, int64_t KH, int64_t KW,
                           int64_t stride, int64_t pad,
                           int64_t b, int64_t o, int64_t oh, int64_t ow)
{
    int64_t s = 0;
    for (int64_t c = 0; c < C; ++c)
        for (int64_t kh = 0; kh < KH; ++kh)
            for (int64_t kw = 0; kw < KW; ++kw) {
                const int64_t ih = oh * stride + kh - pad, iw = ow * stride + kw - pad;
                if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                s += (int64_t)qx[((b * C + c) * H + ih) * W + iw] *
                     (int64_t)qw[((o * C + c) * KH + kh) * KW + kw];
            }
    return s;
}

/* ---- a5: decoder scale (Eq. 18) ----
 * acc and out are [outer][channels][inner]; GEMM: outer=m, channels=n, inner=1;
 * conv (NCHW): outer=N, channels=O, inner=Ho*Wo.  s_w has 1 or `channels` entries.
 * fp32 on purpose: one int->float conversion and one multiply by
 * alpha[c] = (s_a / L_a) * (s_w[c] / L_w), so a chained layer sees the same bits. */
void mpq_oracle_scale(const int32_t* acc, int64_t outer, int64_t channels, int64_t inner,
                      float s_a, const float* s_w, int per_channel,
                      int a_bits, int w_bits, float* out)
{
    const float La = (float)((1 << a_bits) - 1), Lw = (float)((1 << w_bits) - 1);
    const float fa = s_a / La;
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t c = 0; c < channels; ++c) {
            const float fw = (per_channel ? s_w[c] : s_w[0]) / Lw;
            const float alpha = fa * fw;
            for (int64_t i = 0; i < inner; ++i) {
                const int64_t idx = (o * channels + c) * inner + i;
                out[idx] = (float)acc[idx] * alpha;
            }
        }
}

/* The same scale in double, straight from Eq. 18 (used to derive the fp32 tolerance). */
void mpq_oracle_scale_f64(const int32_t* acc, int64_t outer, int64_t channels, int64_t inner,
                          float s_a, const float* s_w, int per_channel,
                          int a_bits, int w_bits, double* out)
{
    const double La = (double)((1 << a_bits) - 1), Lw = (double)((1 << w_bits) - 1);
    for (int64_t o = 0; o < outer; ++o)
        for (int64_t c = 0; c < channels; ++c) {
            const double sw = (double)(per_channel ? s_w[c] : s_w[0]);
            for (int64_t i = 0; i < inner; ++i) {
                const int64_t idx = (o * channels + c) * inner + i;
                out[idx] = (double)acc[idx] * (double)s_a * sw / (La * Lw);
            }
        }
}

/* ---- Full-precision glue of the ResNet-shaped test network (not part of the paper's method;
 * its first layer stays fp32).  Written out as the definition: a 7x7 stride-2 zero-padded
 * convolution whose every output is one chain of fused multiply-adds over (c, kh, kw) in that
 * order (fmaf is exactly rounded, so any implementation that keeps this order gives the same
 * bits), then max(.,0); and a 3x3 stride-2 max-pool with padding 1. */
void mpq_oracle_stem(const float* x, const float* w, int64_t N, int64_t H, int64_t W, int relu, float* y)
{
    const int64_t Ho = (H - 1) / 2 + 1, Wo = (W - 1) / 2 + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t o = 0; o < 64; ++o)
            for (int64_t oh = 0; oh < Ho; ++oh)
                for (int64_t ow = 0; ow < Wo; ++ow) {
                    float acc = 0.0f;
                    for (int64_t c = 0; c < 3; ++c)
                        for (int64_t kh = 0; kh < 7; ++kh)
                            for (int64_t kw = 0; kw < 7; ++kw) {
                                const int64_t ih = 2 * oh + kh - 3, iw = 2 * ow + kw - 3;
                                const float xv = (ih >= 0 && ih < H && iw >= 0 && iw < W)
                                                     ? x[((n * 3 + c) * H + ih) * W + iw] : 0.0f;
                                acc = fmaf(xv, w[((o * 3 + c) * 7 + kh) * 7 + kw], acc);
                            }
                    if (relu && !(acc > 0.0f)) acc = 0.0f;
                    y[((n * 64 + o) * Ho + oh) * Wo + ow] = acc;
                }
}

void mpq_oracle_maxpool3x3s2(const float* x, int64_t planes, int64_t H, int64_t W, float* y)
{
    const int64_t Ho = (H - 1) / 2 + 1, Wo = (W - 1) / 2 + 1;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < planes; ++p)
        for (int64_t oh = 0; oh < Ho; ++oh)
            for (int64_t ow = 0; ow < Wo; ++ow) {
                float m = -INFINITY;
                for (int64_t kh = 0; kh < 3; ++kh)
                    for (int64_t kw = 0; kw < 3; ++kw) {
                        const int64_t ih = 2 * oh + kh - 1, iw = 2 * ow + kw - 1;
                        if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                        const float v = x[(p * H + ih) * W + iw];
                        if (v > m) m = v;
                    }
                y[(p * Ho + oh) * Wo + ow] = m;
            }
}
