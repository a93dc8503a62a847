// Sparse fully connected layer at small batch: one warp per filter.
//
// CADNN (arXiv 1905.00571) evaluates networks whose classifier layers are pruned
// like the convolutions (Section 3 pruning rates; Section 5, Table 2 models).  At
// batch <= 8 the layer is a sparse matrix-vector product bound by streaming the
// stored weights once: lanes stride over a filter's nonzeros with contiguous loads
// of values and 16-bit column indices, gather the activations, and reduce with
// warp shuffles.  Rows are visited in the packer's length-sorted order.
#include "cadnn_internal.h"

namespace {

struct FcParams {
    const void *x;
    void *y;
    const void *vals;
    const uint16_t *idx;
    const int32_t *ptr;
    const int32_t *perm;
    const float *scale;
    const float *bias;
    const void *residual;
    int n, k, c_out, c_pad, act, out_dtype;
};

__device__ __forceinline__ float fc_act(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

template <typename XT, int NB>
__global__ void __launch_bounds__(256) fc_spmv_kernel(const FcParams p)
{
    typedef typename std::conditional<sizeof(XT) == 1, int, float>::type AT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row = blockIdx.x * kWarpsPerBlock + warp;
    grid_dep_wait();
    grid_dep_trigger();
    if (row >= p.c_pad) return;
    const int co = p.perm[row];
    if (co < 0) return;
    const int beg = p.ptr[row], end = p.ptr[row + 1];
    const XT *x = reinterpret_cast<const XT *>(p.x);
    // rows are padded to whole quads of entries: a lane fetches four values and their four column indices per step
    const int qbeg = beg >> 2, qend = end >> 2;
    for (int b0 = 0; b0 < p.n; b0 += NB) {
        AT acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc[b] = 0;
        for (int q = qbeg + lane; q < qend; q += 32) {
            AT wv[4];
            if (sizeof(XT) == 1) {
                const int w4 = __ldg(reinterpret_cast<const int *>(p.vals) + q);
                wv[0] = (AT)(signed char)(w4 & 0xff);
                wv[1] = (AT)(signed char)((w4 >> 8) & 0xff);
                wv[2] = (AT)(signed char)((w4 >> 16) & 0xff);
                wv[3] = (AT)(signed char)((w4 >> 24) & 0xff);
            } else {
                const float4 w4 = __ldg(reinterpret_cast<const float4 *>(p.vals) + q);
                wv[0] = (AT)w4.x; wv[1] = (AT)w4.y; wv[2] = (AT)w4.z; wv[3] = (AT)w4.w;
            }
            const uint2 i4 = __ldg(reinterpret_cast<const uint2 *>(p.idx) + q);
            const int k[4] = {(int)(i4.x & 0xffffu), (int)(i4.x >> 16), (int)(i4.y & 0xffffu), (int)(i4.y >> 16)};
#pragma unroll
            for (int b = 0; b < NB; ++b)
                if (b0 + b < p.n) {
                    const XT *xb = x + (size_t)(b0 + b) * p.k;
                    XT xv[4];
#pragma unroll
                    for (int v = 0; v < 4; ++v) xv[v] = ld_act(xb + k[v]);
#pragma unroll
                    for (int v = 0; v < 4; ++v) acc[b] += wv[v] * (AT)xv[v];
                }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], o);
        if (lane == 0) {
            const float sc = p.scale ? p.scale[co] : 1.0f;
            const float bi = p.bias ? p.bias[co] : 0.0f;
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                if (b0 + b >= p.n) break;
                const size_t oi = (size_t)(b0 + b) * p.c_out + co;
                if (sizeof(XT) == 4) {
                    float z = fmaf((float)acc[b], sc, bi);
                    if (p.residual) z += reinterpret_cast<const float *>(p.residual)[oi];
                    reinterpret_cast<float *>(p.y)[oi] = fc_act(z, p.act);
                } else {
                    const int a = (int)acc[b];
                    if (p.out_dtype == CADNN_S32) {
                        reinterpret_cast<int *>(p.y)[oi] = a;
                    } else {
                        float t = __fmaf_rn(__int2float_rn(a), sc, bi);
                        if (p.act == CADNN_ACT_RELU) t = t > 0.0f ? t : 0.0f;
                        if (p.out_dtype == CADNN_F32) {
                            reinterpret_cast<float *>(p.y)[oi] = t;
                        } else {
                            t = fminf(fmaxf(t, -127.0f), 127.0f);
                            reinterpret_cast<int8_t *>(p.y)[oi] = (int8_t)__float2int_rn(t);
                        }
                    }
                }
            }
        }
    }
}

template <typename XT>
cadnn_status launch_nb(const FcParams &p, int blocks, bool pdl, cudaStream_t st)
{
    if (p.n <= 1) return launch_kernel(fc_spmv_kernel<XT, 1>, blocks, 256, 0, pdl, st, p);
    if (p.n <= 2) return launch_kernel(fc_spmv_kernel<XT, 2>, blocks, 256, 0, pdl, st, p);
    if (p.n <= 4) return launch_kernel(fc_spmv_kernel<XT, 4>, blocks, 256, 0, pdl, st, p);
    return launch_kernel(fc_spmv_kernel<XT, 8>, blocks, 256, 0, pdl, st, p);
}

}  // namespace

cadnn_status launch_fc_spmv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                            cudaStream_t st)
{
    FcParams p;
    p.x = x; p.y = y;
    p.vals = w->d_vals; p.idx = w->d_offs; p.ptr = w->d_ptr; p.perm = w->d_perm;
    p.scale = ep.scale; p.bias = ep.bias; p.residual = ep.residual;
    p.n = n; p.k = w->desc.c_in; p.c_out = w->desc.c_out; p.c_pad = w->c_pad;
    p.act = ep.act; p.out_dtype = ep.out_dtype;
    if (n <= 0) return CADNN_OK;
    int blocks = w->c_pad / kWarpsPerBlock;
    if (w->desc.dtype == CADNN_S8) return launch_nb<int8_t>(p, blocks, ep.pdl, st);
    return launch_nb<float>(p, blocks, ep.pdl, st);
}
