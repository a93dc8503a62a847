// Glue layers of the evaluated networks: max pooling (float and int8) and global
// average pooling.  The paper (arXiv 1905.00571) does not discuss them; they are
// bound by one read and one write of the feature map, so lanes map to channels.
#include <algorithm>
#include <cfloat>
#include "cadnn_internal.h"

namespace {

template <typename XT>
__global__ void __launch_bounds__(256) maxpool_kernel(const XT *x, XT *y, int n, int h, int w, int c, int h_out,
                                                      int w_out, int k, int stride, int pad)
{
    const long long total = (long long)n * h_out * w_out * c;
    grid_dep_wait();
    grid_dep_trigger();
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int ch = (int)(idx % c);
        long long pix = idx / c;
        const int ox = (int)(pix % w_out);
        long long r = pix / w_out;
        const int oy = (int)(r % h_out);
        const int b = (int)(r / h_out);
        bool any = false;
        XT best = 0;
        for (int ky = 0; ky < k; ++ky) {
            const int iy = oy * stride + ky - pad;
            if (iy < 0 || iy >= h) continue;
            for (int kx = 0; kx < k; ++kx) {
                const int ix = ox * stride + kx - pad;
                if (ix < 0 || ix >= w) continue;
                const XT v = x[(((size_t)b * h + iy) * w + ix) * c + ch];
                if (!any || v > best) best = v;
                any = true;
            }
        }
        y[idx] = best;
    }
}

// Max (AVG = false) or average pool into a channel window of a wider output tensor: the branches of an
// Inception module end in one concatenated tensor, and a pooling branch writes its channels of it
// directly.  Average: taps in the padding count as zeros, the divisor is always k * k; fp32 sum.
template <typename XT, bool AVG>
__global__ void __launch_bounds__(256) pool_window_kernel(const XT *x, XT *y, int n, int h, int w, int c, int h_out,
                                                          int w_out, int k, int stride, int pad, int ldc, int c_off, float inv)
{
    const long long total = (long long)n * h_out * w_out * c;
    grid_dep_wait();
    grid_dep_trigger();
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int ch = (int)(idx % c);
        long long pix = idx / c;
        const int ox = (int)(pix % w_out);
        long long r = pix / w_out;
        const int oy = (int)(r % h_out);
        const int b = (int)(r / h_out);
        bool any = false;
        XT best = 0;
        float sum = 0.0f;
        for (int ky = 0; ky < k; ++ky) {
            const int iy = oy * stride + ky - pad;
            if (iy < 0 || iy >= h) continue;
            for (int kx = 0; kx < k; ++kx) {
                const int ix = ox * stride + kx - pad;
                if (ix < 0 || ix >= w) continue;
                const XT v = ld_act(x + (((size_t)b * h + iy) * w + ix) * c + ch);
                if (AVG) sum += (float)v;
                else if (!any || v > best) best = v;
                any = true;
            }
        }
        y[(size_t)pix * ldc + c_off + ch] = AVG ? (XT)(sum * inv) : best;
    }
}

// 16 bytes per thread: four floats, or sixteen int8 channels (per-byte signed max).
template <bool S8>
__global__ void __launch_bounds__(256) maxpool_vec_kernel(const uint4 *x, uint4 *y, int n, int h, int w, int cv,
                                                          int h_out, int w_out, int k, int stride, int pad,
                                                          FastDiv d_cv, FastDiv d_wout, FastDiv d_hout)
{
    const unsigned total = (unsigned)n * h_out * w_out * cv;   // < 2^31, checked by the host
    grid_dep_wait();
    grid_dep_trigger();
    for (unsigned idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const unsigned pix = fdiv(idx, d_cv);
        const int ch = (int)(idx - pix * cv);
        const unsigned r = fdiv(pix, d_wout);
        const int ox = (int)(pix - r * w_out);
        const unsigned b = fdiv(r, d_hout);
        const int oy = (int)(r - b * h_out);
        bool any = false;
        uint4 best = make_uint4(0, 0, 0, 0);
        for (int ky = 0; ky < k; ++ky) {
            const int iy = oy * stride + ky - pad;
            if (iy < 0 || iy >= h) continue;
            for (int kx = 0; kx < k; ++kx) {
                const int ix = ox * stride + kx - pad;
                if (ix < 0 || ix >= w) continue;
                const uint4 v = x[(((size_t)b * h + iy) * w + ix) * cv + ch];
                if (!any) {
                    best = v;
                    any = true;
                } else if (S8) {
                    best.x = __vmaxs4(best.x, v.x); best.y = __vmaxs4(best.y, v.y);
                    best.z = __vmaxs4(best.z, v.z); best.w = __vmaxs4(best.w, v.w);
                } else {
                    best.x = __float_as_uint(fmaxf(__uint_as_float(best.x), __uint_as_float(v.x)));
                    best.y = __float_as_uint(fmaxf(__uint_as_float(best.y), __uint_as_float(v.y)));
                    best.z = __float_as_uint(fmaxf(__uint_as_float(best.z), __uint_as_float(v.z)));
                    best.w = __float_as_uint(fmaxf(__uint_as_float(best.w), __uint_as_float(v.w)));
                }
            }
        }
        y[idx] = best;
    }
}

__global__ void __launch_bounds__(256) gavgpool_kernel(const float *x, float *y, int n, int hw, int c, float inv)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    grid_dep_wait();
    grid_dep_trigger();
    if (idx >= n * c) return;
    const int b = idx / c, ch = idx - b * c;
    const float *src = x + (size_t)b * hw * c + ch;
    float s = 0.0f;
    for (int i = 0; i < hw; ++i) s += src[(size_t)i * c];
    y[idx] = s * inv;
}

}  // namespace

cadnn_status launch_maxpool(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype,
                            void *y, bool pdl, cudaStream_t st)
{
    const int h_out = (h + 2 * pad - k) / stride + 1, w_out = (wd + 2 * pad - k) / stride + 1;
    long long total = (long long)n * h_out * w_out * c;
    if (total <= 0) return CADNN_OK;
    const int per = dtype == CADNN_S8 ? 16 : 4;   // channels per 16-byte vector
    if (c % per == 0 && ((uintptr_t)x & 15) == 0 && ((uintptr_t)y & 15) == 0 && total / per < (1LL << 31)) {
        const FastDiv d_cv = make_fastdiv(c / per), d_wout = make_fastdiv(w_out), d_hout = make_fastdiv(h_out);
        long long tv = total / per;
        long long bv = std::min((tv + 255) / 256, 148LL * 32);
        if (dtype == CADNN_S8)
            return launch_kernel(maxpool_vec_kernel<true>, (int)bv, 256, 0, pdl, st, (const uint4 *)x, (uint4 *)y, n, h, wd,
                                 c / per, h_out, w_out, k, stride, pad, d_cv, d_wout, d_hout);
        return launch_kernel(maxpool_vec_kernel<false>, (int)bv, 256, 0, pdl, st, (const uint4 *)x, (uint4 *)y, n, h, wd,
                             c / per, h_out, w_out, k, stride, pad, d_cv, d_wout, d_hout);
    }
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    if (dtype == CADNN_S8)
        return launch_kernel(maxpool_kernel<int8_t>, (int)blocks, 256, 0, pdl, st, (const int8_t *)x, (int8_t *)y, n, h,
                             wd, c, h_out, w_out, k, stride, pad);
    return launch_kernel(maxpool_kernel<float>, (int)blocks, 256, 0, pdl, st, (const float *)x, (float *)y, n, h, wd, c,
                         h_out, w_out, k, stride, pad);
}

cadnn_status launch_pool_window(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype, int kind,
                                void *y, int ldc, int c_off, bool pdl, cudaStream_t st)
{
    if (kind == 0 && (ldc <= 0 || (ldc == c && c_off == 0))) return launch_maxpool(x, n, h, wd, c, k, stride, pad, dtype, y, pdl, st);
    if (ldc <= 0) { ldc = c; c_off = 0; }
    const int h_out = (h + 2 * pad - k) / stride + 1, w_out = (wd + 2 * pad - k) / stride + 1;
    long long total = (long long)n * h_out * w_out * c;
    if (total <= 0) return CADNN_OK;
    long long blocks = std::min((total + 255) / 256, 148LL * 64);
    const float inv = 1.0f / (float)(k * k);
    if (kind == 1) {
        if (dtype != CADNN_F32) return CADNN_E_DTYPE;
        return launch_kernel(pool_window_kernel<float, true>, (int)blocks, 256, 0, pdl, st, (const float *)x, (float *)y, n, h, wd,
                             c, h_out, w_out, k, stride, pad, ldc, c_off, inv);
    }
    if (dtype == CADNN_S8)
        return launch_kernel(pool_window_kernel<signed char, false>, (int)blocks, 256, 0, pdl, st, (const signed char *)x,
                             (signed char *)y, n, h, wd, c, h_out, w_out, k, stride, pad, ldc, c_off, inv);
    return launch_kernel(pool_window_kernel<float, false>, (int)blocks, 256, 0, pdl, st, (const float *)x, (float *)y, n, h, wd, c,
                         h_out, w_out, k, stride, pad, ldc, c_off, inv);
}

cadnn_status launch_gavgpool(const float *x, int n, int h, int wd, int c, float *y, bool pdl, cudaStream_t st)
{
    if (n * c <= 0) return CADNN_OK;
    return launch_kernel(gavgpool_kernel, (n * c + 255) / 256, 256, 0, pdl, st, x, y, n, h * wd, c,
                         1.0f / (float)(h * wd));
}
