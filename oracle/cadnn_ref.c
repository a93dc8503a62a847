/*
 * CPU oracle for pruned / quantized CNN layer inference (CADNN, arXiv 1905.00571).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or helper with
 * the CUDA library and must never be linked into, or called from, the product.
 *
 * What it computes.  The paper's compressed execution (Section 4, "Model
 * computation fusion and transformation") is a result-preserving rewrite of an
 * ordinary CNN layer whose pruned weights are zero (Section 5, "Performance":
 * the same models run dense and compressed).  The oracle is therefore the plain
 * definition: a direct convolution over the DENSE tensor W_eff = mask ? W : 0,
 * visiting every (ky, kx, ci) in that fixed order and skipping nothing,
 * followed by the fused Conv + BatchNorm + Activation epilogue the same section
 * names, with BatchNorm folded into a per-channel (scale, bias).
 *
 * Readings where the paper is silent (each is restated in the project design
 * notes): cross-correlation (no kernel flip); symmetric zero padding;
 * H_out = floor((H + 2p - k) / s) + 1; activations NHWC; weights OHWI
 * [c_out][kh][kw][c_in/groups]; fp32 layers accumulate in double and round
 * once to float; epilogue z = acc*scale + bias, then + residual, then the
 * activation, each a separately rounded float operation; int8 layers
 * accumulate exactly in int32 and requantize with ONE fused multiply-add
 * t = fmaf((float)acc, M, B), ReLU, round-half-even, clamp.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (no -ffast-math).
 * OpenMP is used only over output rows, so the order of additions inside one
 * output element never changes.
 *
 * Pins (see tests/test_oracle_pins.py): hand-worked literals, shift and
 * identity filters, 1x1 == matrix product, FC == mat-vec, linearity, mask
 * additivity, channel-permutation equivariance, a float64 library convolution
 * (square and rectangular kernels, grouped int8 included), library pooling
 * routines with and without padding, and an exact rational check of the
 * requantization scalars (with and without the int8 residual).
 * Parity unpinned: ImageNet accuracy of the paper's Table 2 (needs its data
 * and trained weights).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <float.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { REF_ACT_NONE = 0, REF_ACT_RELU = 1, REF_ACT_RELU6 = 2 };
enum { REF_OUT_S8 = 0, REF_OUT_S32 = 1, REF_OUT_F32 = 2 };

int ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ref_set_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

static int out_extent(int in, int k, int s, int p)
{
    int v = in + 2 * p - k;
    if (v < 0) return 0;
    return v / s + 1;
}

static float activate_f32(float z, int act)
{
    if (act == REF_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == REF_ACT_RELU6) {
        float r = z > 0.0f ? z : 0.0f;
        return r < 6.0f ? r : 6.0f;
    }
    return z;
}

/*
 * Fused epilogue of a float layer (Section 4: Conv + BatchNorm + Activation in
 * one kernel; the residual add of a bottleneck block rides in the same place).
 */
static float epilogue_f32(double acc, const float *scale, const float *bias,
                          const float *residual, size_t ridx, int co, int act)
{
    float z = (float)acc;
    float sc = scale ? scale[co] : 1.0f;
    float bi = bias ? bias[co] : 0.0f;
    z = z * sc;
    z = z + bi;
    if (residual) z = z + residual[ridx];
    return activate_f32(z, act);
}

/*
 * Float convolution layer.  x [n][h][w][c_in], wt [c_out][kh][kw][c_in/groups],
 * mask same shape as wt or NULL (= all kept), y [n][h_out][w_out][c_out].
 * Returns 0, or -1 on an invalid shape.
 */
int ref_conv2d_f32_hw(const float *x, int n, int h, int w, int c_in,
                      const float *wt, const uint8_t *mask,
                      int c_out, int kh, int kw, int stride, int pad_h, int pad_w, int groups,
                      const float *scale, const float *bias, const float *residual,
                      int act, float *y)
{
    if (groups < 1 || c_in % groups || c_out % groups || stride < 1 || pad_h < 0 || pad_w < 0) return -1;
    const int cg = c_in / groups;      /* input channels seen by one filter */
    const int og = c_out / groups;     /* filters per group */
    const int ho = out_extent(h, kh, stride, pad_h);
    const int wo = out_extent(w, kw, stride, pad_w);
    const long rows = (long)n * ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (long row = 0; row < rows; ++row) {
        const int b = (int)(row / ho), oy = (int)(row % ho);
        for (int ox = 0; ox < wo; ++ox) {
            for (int co = 0; co < c_out; ++co) {
                const int g = co / og;
                double acc = 0.0;
                for (int ky = 0; ky < kh; ++ky) {
                    const int iy = oy * stride + ky - pad_h;
                    for (int kx = 0; kx < kw; ++kx) {
                        const int ix = ox * stride + kx - pad_w;
                        const int inside = (iy >= 0 && iy < h && ix >= 0 && ix < w);
                        for (int ci = 0; ci < cg; ++ci) {
                            const size_t wi = (((size_t)co * kh + ky) * kw + kx) * cg + ci;
                            const float wv = (mask == NULL || mask[wi]) ? wt[wi] : 0.0f;
                            float xv = 0.0f;
                            if (inside)
                                xv = x[(((size_t)b * h + iy) * w + ix) * c_in + (size_t)g * cg + ci];
                            acc += (double)wv * (double)xv;
                        }
                    }
                }
                const size_t oi = (((size_t)b * ho + oy) * wo + ox) * c_out + co;
                y[oi] = epilogue_f32(acc, scale, bias, residual, oi, co, act);
            }
        }
    }
    return 0;
}

/* The same layer with one padding for both axes (square-kernel networks). */
int ref_conv2d_f32(const float *x, int n, int h, int w, int c_in,
                   const float *wt, const uint8_t *mask,
                   int c_out, int kh, int kw, int stride, int pad, int groups,
                   const float *scale, const float *bias, const float *residual,
                   int act, float *y)
{
    return ref_conv2d_f32_hw(x, n, h, w, c_in, wt, mask, c_out, kh, kw, stride, pad, pad, groups,
                             scale, bias, residual, act, y);
}

/*
 * Float fully connected layer: y[b][co] = sum_k W_eff[co][k] * x[b][k],
 * same epilogue.  Written separately from the convolution on purpose.
 */
int ref_fc_f32(const float *x, int n, int k, const float *wt, const uint8_t *mask,
               int c_out, const float *scale, const float *bias, const float *residual,
               int act, float *y)
{
#pragma omp parallel for schedule(static)
    for (int co = 0; co < c_out; ++co) {
        for (int b = 0; b < n; ++b) {
            double acc = 0.0;
            for (int j = 0; j < k; ++j) {
                const size_t wi = (size_t)co * k + j;
                const float wv = (mask == NULL || mask[wi]) ? wt[wi] : 0.0f;
                acc += (double)wv * (double)x[(size_t)b * k + j];
            }
            const size_t oi = (size_t)b * c_out + co;
            y[oi] = epilogue_f32(acc, scale, bias, residual, oi, co, act);
        }
    }
    return 0;
}

/*
 * Symmetric per-output-channel int8 weight quantization:
 * q = clamp(round_half_even(w / s_w[co]), -127, 127), IEEE float divide.
 */
int ref_quantize_weights(const float *wt, const float *s_w, int c_out, long per_row, int8_t *q)
{
    for (int co = 0; co < c_out; ++co) {
        for (long j = 0; j < per_row; ++j) {
            float r = wt[(size_t)co * per_row + j] / s_w[co];
            long v = lrintf(r);
            if (v > 127) v = 127;
            if (v < -127) v = -127;
            q[(size_t)co * per_row + j] = (int8_t)v;
        }
    }
    return 0;
}

/*
 * Requantization scalar of the int8 path: exactly one fused multiply-add on
 * the int32 accumulator converted to float (round to nearest even), optional
 * ReLU, round half to even, clamp to [-127, 127].
 */
float ref_requant_f32(int32_t acc, float m, float b, int act)
{
    float t = fmaf((float)acc, m, b);
    if (act == REF_ACT_RELU) t = t > 0.0f ? t : 0.0f;
    return t;
}

int8_t ref_requant_s8(int32_t acc, float m, float b, int act)
{
    float t = ref_requant_f32(acc, m, b, act);
    /* clamp in float first so that lrintf never sees an out-of-range value */
    if (t > 127.0f) t = 127.0f;
    if (t < -127.0f) t = -127.0f;
    return (int8_t)lrintf(t);
}

/*
 * Requantization with an int8 residual (the shortcut of a quantized residual
 * block): two fused multiply-adds in this order,
 *   t = fmaf((float)acc, M, B);  t = fmaf((float)r, residual_scale, t);
 * then ReLU, clamp, round half to even as above.  residual_scale = s_r / s_y is
 * precomputed by the caller.
 */
float ref_requant_res_f32(int32_t acc, float m, float b, int8_t r, float residual_scale, int act)
{
    float t = fmaf((float)acc, m, b);
    t = fmaf((float)r, residual_scale, t);
    if (act == REF_ACT_RELU) t = t > 0.0f ? t : 0.0f;
    return t;
}

int8_t ref_requant_res_s8(int32_t acc, float m, float b, int8_t r, float residual_scale, int act)
{
    float t = ref_requant_res_f32(acc, m, b, r, residual_scale, act);
    if (t > 127.0f) t = 127.0f;
    if (t < -127.0f) t = -127.0f;
    return (int8_t)lrintf(t);
}

static void store_q(void *y, size_t oi, int32_t acc, const float *m, const float *b,
                    const int8_t *residual, float residual_scale, int co, int act, int out_kind)
{
    const float mm = m ? m[co] : 1.0f;
    const float bb = b ? b[co] : 0.0f;
    if (out_kind == REF_OUT_S32) ((int32_t *)y)[oi] = acc;
    else if (residual) {
        if (out_kind == REF_OUT_F32)
            ((float *)y)[oi] = ref_requant_res_f32(acc, mm, bb, residual[oi], residual_scale, act);
        else
            ((int8_t *)y)[oi] = ref_requant_res_s8(acc, mm, bb, residual[oi], residual_scale, act);
    }
    else if (out_kind == REF_OUT_F32) ((float *)y)[oi] = ref_requant_f32(acc, mm, bb, act);
    else ((int8_t *)y)[oi] = ref_requant_s8(acc, mm, bb, act);
}

/*
 * Int8 convolution layer: int8 activations and weights, exact int32
 * accumulation over the dense masked weights, then store_q.  ReLU6 is not
 * defined for this path (returns -1).
 */
int ref_conv2d_s8_res(const int8_t *x, int n, int h, int w, int c_in,
                      const int8_t *wq, const uint8_t *mask,
                      int c_out, int kh, int kw, int stride, int pad, int groups,
                      const float *m, const float *b, const int8_t *residual, float residual_scale,
                      int act, int out_kind, void *y)
{
    if (groups < 1 || c_in % groups || c_out % groups || stride < 1 || pad < 0) return -1;
    if (act == REF_ACT_RELU6) return -1;
    const int cg = c_in / groups;
    const int og = c_out / groups;
    const int ho = out_extent(h, kh, stride, pad);
    const int wo = out_extent(w, kw, stride, pad);
    const long rows = (long)n * ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (long row = 0; row < rows; ++row) {
        const int bi = (int)(row / ho), oy = (int)(row % ho);
        for (int ox = 0; ox < wo; ++ox) {
            for (int co = 0; co < c_out; ++co) {
                const int g = co / og;
                int32_t acc = 0;
                for (int ky = 0; ky < kh; ++ky) {
                    const int iy = oy * stride + ky - pad;
                    for (int kx = 0; kx < kw; ++kx) {
                        const int ix = ox * stride + kx - pad;
                        const int inside = (iy >= 0 && iy < h && ix >= 0 && ix < w);
                        for (int ci = 0; ci < cg; ++ci) {
                            const size_t wi = (((size_t)co * kh + ky) * kw + kx) * cg + ci;
                            const int32_t wv = (mask == NULL || mask[wi]) ? (int32_t)wq[wi] : 0;
                            int32_t xv = 0;
                            if (inside)
                                xv = (int32_t)x[(((size_t)bi * h + iy) * w + ix) * c_in + (size_t)g * cg + ci];
                            acc += wv * xv;
                        }
                    }
                }
                const size_t oi = (((size_t)bi * ho + oy) * wo + ox) * c_out + co;
                store_q(y, oi, acc, m, b, residual, residual_scale, co, act, out_kind);
            }
        }
    }
    return 0;
}

int ref_conv2d_s8(const int8_t *x, int n, int h, int w, int c_in,
                  const int8_t *wq, const uint8_t *mask,
                  int c_out, int kh, int kw, int stride, int pad, int groups,
                  const float *m, const float *b, int act, int out_kind, void *y)
{
    return ref_conv2d_s8_res(x, n, h, w, c_in, wq, mask, c_out, kh, kw, stride, pad, groups,
                             m, b, NULL, 0.0f, act, out_kind, y);
}

int ref_fc_s8(const int8_t *x, int n, int k, const int8_t *wq, const uint8_t *mask,
              int c_out, const float *m, const float *b, int act, int out_kind, void *y)
{
    if (act == REF_ACT_RELU6) return -1;
#pragma omp parallel for schedule(static)
    for (int co = 0; co < c_out; ++co) {
        for (int bi = 0; bi < n; ++bi) {
            int32_t acc = 0;
            for (int j = 0; j < k; ++j) {
                const size_t wi = (size_t)co * k + j;
                const int32_t wv = (mask == NULL || mask[wi]) ? (int32_t)wq[wi] : 0;
                acc += wv * (int32_t)x[(size_t)bi * k + j];
            }
            store_q(y, (size_t)bi * c_out + co, acc, m, b, NULL, 0.0f, co, act, out_kind);
        }
    }
    return 0;
}

/*
 * Max pooling.  Taps that fall in the padding are ignored (they never count
 * as zero); a window with no valid tap cannot occur for pad < k.
 */
int ref_maxpool_f32(const float *x, int n, int h, int w, int c, int k, int stride, int pad, float *y)
{
    if (pad >= k) return -1;
    const int ho = out_extent(h, k, stride, pad), wo = out_extent(w, k, stride, pad);
    for (int b = 0; b < n; ++b)
        for (int oy = 0; oy < ho; ++oy)
            for (int ox = 0; ox < wo; ++ox)
                for (int ch = 0; ch < c; ++ch) {
                    float best = -FLT_MAX;
                    for (int ky = 0; ky < k; ++ky)
                        for (int kx = 0; kx < k; ++kx) {
                            const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
                            if (iy < 0 || iy >= h || ix < 0 || ix >= w) continue;
                            const float v = x[(((size_t)b * h + iy) * w + ix) * c + ch];
                            if (v > best) best = v;
                        }
                    y[(((size_t)b * ho + oy) * wo + ox) * c + ch] = best;
                }
    return 0;
}

int ref_maxpool_s8(const int8_t *x, int n, int h, int w, int c, int k, int stride, int pad, int8_t *y)
{
    if (pad >= k) return -1;
    const int ho = out_extent(h, k, stride, pad), wo = out_extent(w, k, stride, pad);
    for (int b = 0; b < n; ++b)
        for (int oy = 0; oy < ho; ++oy)
            for (int ox = 0; ox < wo; ++ox)
                for (int ch = 0; ch < c; ++ch) {
                    int best = -128;
                    for (int ky = 0; ky < k; ++ky)
                        for (int kx = 0; kx < k; ++kx) {
                            const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
                            if (iy < 0 || iy >= h || ix < 0 || ix >= w) continue;
                            const int v = x[(((size_t)b * h + iy) * w + ix) * c + ch];
                            if (v > best) best = v;
                        }
                    y[(((size_t)b * ho + oy) * wo + ox) * c + ch] = (int8_t)best;
                }
    return 0;
}

/*
 * Average pooling with a k x k window.  Taps that fall in the padding count as
 * zeros and the divisor is always k * k (the convention of the Inception-V3
 * definition the synthetic workload follows).  Double sum, one division, rounded
 * once to float.
 */
int ref_avgpool_f32(const float *x, int n, int h, int w, int c, int k, int stride, int pad, float *y)
{
    if (pad >= k || k < 1 || stride < 1) return -1;
    const int ho = out_extent(h, k, stride, pad), wo = out_extent(w, k, stride, pad);
    for (int b = 0; b < n; ++b)
        for (int oy = 0; oy < ho; ++oy)
            for (int ox = 0; ox < wo; ++ox)
                for (int ch = 0; ch < c; ++ch) {
                    double s = 0.0;
                    for (int ky = 0; ky < k; ++ky)
                        for (int kx = 0; kx < k; ++kx) {
                            const int iy = oy * stride + ky - pad, ix = ox * stride + kx - pad;
                            if (iy < 0 || iy >= h || ix < 0 || ix >= w) continue;
                            s += (double)x[(((size_t)b * h + iy) * w + ix) * c + ch];
                        }
                    y[(((size_t)b * ho + oy) * wo + ox) * c + ch] = (float)(s / (double)(k * k));
                }
    return 0;
}

/* Global average pool: double sum over the H*W positions, divided, rounded once. */
int ref_gavgpool_f32(const float *x, int n, int h, int w, int c, float *y)
{
    for (int b = 0; b < n; ++b)
        for (int ch = 0; ch < c; ++ch) {
            double s = 0.0;
            for (int i = 0; i < h * w; ++i) s += (double)x[((size_t)b * h * w + i) * c + ch];
            y[(size_t)b * c + ch] = (float)(s / (double)(h * w));
        }
    return 0;
}
