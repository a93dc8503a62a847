// Dense layers the pruned networks keep: depthwise k x k convolution (MobileNet),
// fused with BatchNorm fold, residual and activation.
//
// CADNN (arXiv 1905.00571), Section 4, names Depthwise Convolution + BatchNorm +
// Activation as one fused kernel.  A depthwise layer does kh*kw multiply-adds per
// output and is bound by reading the input and writing the output once, so the
// kernel maps lanes to channels (contiguous in NHWC) and keeps the filter taps in
// the tap-major layout the packer wrote.
#include "cadnn_internal.h"

namespace {

struct DwParams {
    const float *x;
    float *y;
    const float *wt;  // [kh*kw][c]
    const float *scale;
    const float *bias;
    const float *residual;
    int n, h, w, c, h_out, w_out, kh, kw, stride, pad, act;
};

__device__ __forceinline__ float dw_act(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

template <int VEC>
__global__ void __launch_bounds__(256) dw_kernel(const DwParams p)
{
    const int cv = p.c / VEC;
    const long long total = (long long)p.n * p.h_out * p.w_out * cv;
    grid_dep_wait();
    grid_dep_trigger();
    for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int c0 = (int)(idx % cv) * VEC;
        long long pix = idx / cv;
        const int ox = (int)(pix % p.w_out);
        long long r = pix / p.w_out;
        const int oy = (int)(r % p.h_out);
        const int b = (int)(r / p.h_out);
        float acc[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = 0.0f;
        for (int ky = 0; ky < p.kh; ++ky) {
            const int iy = oy * p.stride + ky - p.pad;
            if (iy < 0 || iy >= p.h) continue;
            for (int kx = 0; kx < p.kw; ++kx) {
                const int ix = ox * p.stride + kx - p.pad;
                if (ix < 0 || ix >= p.w) continue;
                const float *xs = p.x + (((size_t)b * p.h + iy) * p.w + ix) * p.c + c0;
                const float *ws = p.wt + (size_t)(ky * p.kw + kx) * p.c + c0;
                if (VEC == 4) {
                    const float4 xv = *reinterpret_cast<const float4 *>(xs);
                    const float4 wv = __ldg(reinterpret_cast<const float4 *>(ws));
                    acc[0] = fmaf(xv.x, wv.x, acc[0]);
                    acc[1 % VEC] = fmaf(xv.y, wv.y, acc[1 % VEC]);
                    acc[2 % VEC] = fmaf(xv.z, wv.z, acc[2 % VEC]);
                    acc[3 % VEC] = fmaf(xv.w, wv.w, acc[3 % VEC]);
                } else {
                    acc[0] = fmaf(xs[0], __ldg(ws), acc[0]);
                }
            }
        }
        const size_t oi = (size_t)pix * p.c + c0;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            const int co = c0 + v;
            float z = fmaf(acc[v], p.scale ? p.scale[co] : 1.0f, p.bias ? p.bias[co] : 0.0f);
            if (p.residual) z += p.residual[oi + v];
            acc[v] = dw_act(z, p.act);
        }
        if (VEC == 4) *reinterpret_cast<float4 *>(p.y + oi) = make_float4(acc[0], acc[1 % VEC], acc[2 % VEC], acc[3 % VEC]);
        else p.y[oi] = acc[0];
    }
}

}  // namespace

cadnn_status launch_dw(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                       cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    DwParams p;
    p.x = (const float *)x; p.y = (float *)y; p.wt = w->d_dense;
    p.scale = ep.scale; p.bias = ep.bias; p.residual = (const float *)ep.residual;
    p.n = n; p.h = d.in_h; p.w = d.in_w; p.c = d.c_out; p.h_out = w->h_out; p.w_out = w->w_out;
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.act = ep.act;
    const bool v4 = d.c_out % 4 == 0;
    long long total = (long long)n * w->h_out * w->w_out * (v4 ? d.c_out / 4 : d.c_out);
    if (total <= 0) return CADNN_OK;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    if (v4) return launch_kernel(dw_kernel<4>, (int)blocks, 256, 0, ep.pdl, st, p);
    return launch_kernel(dw_kernel<1>, (int)blocks, 256, 0, ep.pdl, st, p);
}
