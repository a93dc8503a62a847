// C-ABI entry points for single layers: argument checks and dispatch to the
// kernel the packer scheduled.  No arithmetic lives here.
#include <cstdio>
#include <cstring>
#include <mutex>
#include "cadnn_internal.h"

namespace {
thread_local char g_cuda_err[256] = "";
}

cadnn_status cadnn_note_cuda(cudaError_t e)
{
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    cudaGetLastError();  // clear a non-sticky error so that later calls are not blamed for it
    return CADNN_E_CUDA;
}

cadnn_status raise_smem_limit(const void *kern, int smem, SmemLimit *lim)
{
    static std::mutex mu;
    int dev = 0;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CADNN_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    const int have = lim->allowed[dev] > 0 ? lim->allowed[dev] : 48 * 1024;
    if (smem <= have) return CADNN_OK;
    CADNN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    lim->allowed[dev] = smem;
    return CADNN_OK;
}

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

cadnn_status check_epilogue(const cadnn_weights *w, const cadnn_epilogue *ep, LaunchEpilogue &le)
{
    const int dt = w->desc.dtype;
    le = LaunchEpilogue();
    le.out_dtype = dt;
    if (!ep) return CADNN_OK;
    le.scale = ep->scale;
    le.bias = ep->bias;
    le.residual = ep->residual;
    le.act = ep->act;
    le.out_dtype = ep->out_dtype;
    le.out_c_total = ep->out_c_total;
    le.out_c_off = ep->out_c_off;
    le.res_scale = ep->residual_scale;
    if (le.out_c_total < 0 || le.out_c_off < 0) return CADNN_E_ARG;
    if (le.out_c_total > 0) {   // a channel window of a wider output: sparse conv kernels only, no residual
        if (le.out_c_off + w->desc.c_out > le.out_c_total) return CADNN_E_SHAPE;
        if (le.residual) return CADNN_E_UNSUPPORTED;
        if (w->s.kind != KK_SCONV_SPATIAL && w->s.kind != KK_SCONV_LINEAR) return CADNN_E_UNSUPPORTED;
    } else if (le.out_c_off != 0) return CADNN_E_ARG;
    if (le.act < CADNN_ACT_NONE || le.act > CADNN_ACT_RELU6) return CADNN_E_ARG;
    if (dt == CADNN_F32) {
        if (le.out_dtype != CADNN_F32) return CADNN_E_DTYPE;
    } else {
        if (le.out_dtype != CADNN_S8 && le.out_dtype != CADNN_S32 && le.out_dtype != CADNN_F32) return CADNN_E_DTYPE;
        // an int8 residual joins the requantization in the sparse conv kernels only, and never a raw accumulator
        if (le.residual && (le.out_dtype == CADNN_S32 || (w->s.kind != KK_SCONV_SPATIAL && w->s.kind != KK_SCONV_LINEAR)))
            return CADNN_E_UNSUPPORTED;
        if (le.act == CADNN_ACT_RELU6) return CADNN_E_UNSUPPORTED;
    }
    if (le.residual && !aligned16(le.residual)) return CADNN_E_ARG;
    return CADNN_OK;
}

}  // namespace

cadnn_status check_layer_call(const cadnn_weights *w, bool has_residual, int act, int out_dtype, int out_c_total, int out_c_off)
{
    if (!w || !w->on_device) return CADNN_E_ARG;
    int dev = -1;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    if (w->device != dev) return CADNN_E_ARG;   // packed on another GPU
    cadnn_epilogue ep;
    alignas(16) static const char some_residual[16] = {0};   // only its presence matters here
    ep.scale = nullptr; ep.bias = nullptr; ep.residual = has_residual ? some_residual : nullptr;
    ep.act = act; ep.out_dtype = out_dtype; ep.out_c_total = out_c_total; ep.out_c_off = out_c_off; ep.residual_scale = 0.0f;
    LaunchEpilogue le;
    return check_epilogue(w, &ep, le);
}

cadnn_status conv2d_impl(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y, const cadnn_epilogue *ep,
                         bool pdl, cudaStream_t s, void *workspace, int64_t workspace_bytes)
{
    if (!w || !x || !y || n < 0) return CADNN_E_ARG;
    if (!w->on_device) return CADNN_E_ARG;
    if (h != w->desc.in_h || wd != w->desc.in_w) return CADNN_E_SHAPE;
    if (!aligned16(x) || !aligned16(y) || x == y) return CADNN_E_ARG;
    LaunchEpilogue le;
    cadnn_status st = check_epilogue(w, ep, le);
    if (st != CADNN_OK) return st;
    le.pdl = pdl;
    if (w->has_tc && w->nnz == w->tc_nnz) {
        // every stored weight sits in a dense block: the tensor-core kernel finishes the layer
        return launch_block_tc(w, x, n, nullptr, y, &le, s);
    }
    if (w->has_tc) {
        // dense blocks on the tensor cores first; the sparse kernel then starts from their int32 sums
        const int64_t need = (int64_t)n * w->h_out * w->w_out * w->desc.c_out * 4;
        if (!workspace || !aligned16(workspace) || workspace_bytes < need) return CADNN_E_ARG;
        st = launch_block_tc(w, x, n, (int *)workspace, nullptr, nullptr, s);
        if (st != CADNN_OK) return st;
        le.acc_in = (const int *)workspace;
        le.pdl = false;
    }
    switch (w->s.kind) {
        case KK_SCONV_SPATIAL:
        case KK_SCONV_LINEAR: return launch_sconv(w, x, n, y, le, s);
        case KK_FC_SPMV: return launch_fc_spmv(w, x, n, y, le, s);
        case KK_DW: return launch_dw(w, x, n, y, le, s);
        case KK_DENSE_SMALLC: return launch_dense_smallc(w, x, n, y, le, s);
    }
    return CADNN_E_UNSUPPORTED;
}

extern "C" {

cadnn_status cadnn_conv2d(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y,
                          const cadnn_epilogue *ep, void *stream)
{
    return conv2d_impl(w, x, n, h, wd, y, ep, false, (cudaStream_t)stream);
}

cadnn_status cadnn_weights_workspace_bytes(const cadnn_weights *w, int n, int64_t *bytes)
{
    if (!w || !bytes || n < 0) return CADNN_E_ARG;
    *bytes = (w->has_tc && w->nnz != w->tc_nnz) ? (int64_t)n * w->h_out * w->w_out * w->desc.c_out * 4 : 0;
    return CADNN_OK;
}

cadnn_status cadnn_conv2d_workspace(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y,
                                    const cadnn_epilogue *ep, void *workspace, int64_t workspace_bytes, void *stream)
{
    return conv2d_impl(w, x, n, h, wd, y, ep, false, (cudaStream_t)stream, workspace, workspace_bytes);
}

cadnn_status cadnn_weights_block_info(const cadnn_weights *w, int *n_blocks, int64_t *block_nnz)
{
    if (!w) return CADNN_E_ARG;
    if (n_blocks) *n_blocks = w->has_tc ? (int)(w->tc_blk.size() / 4) : 0;
    if (block_nnz) *block_nnz = w->has_tc ? w->tc_nnz : 0;
    return CADNN_OK;
}

cadnn_status cadnn_conv2d_planar(const cadnn_weights *w, const void *x, int n, void *y, const cadnn_epilogue *ep,
                                 void *stream)
{
    if (!w || !x || !y || n < 0) return CADNN_E_ARG;
    if (!w->on_device || !w->has_planar) return CADNN_E_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(y) || x == y) return CADNN_E_ARG;
    LaunchEpilogue le;
    cadnn_status st = check_epilogue(w, ep, le);
    if (st != CADNN_OK) return st;
    if (w->has_ps && w->use_ps) return launch_sconv_planar_staged(w, x, n, y, le, (cudaStream_t)stream);
    return launch_sconv_planar(w, x, n, y, le, (cudaStream_t)stream);
}

cadnn_status cadnn_fc(const cadnn_weights *w, const void *x, int n, void *y, const cadnn_epilogue *ep, void *stream)
{
    if (!w) return CADNN_E_ARG;
    const cadnn_layer_desc &d = w->desc;
    if (d.kh != 1 || d.kw != 1 || d.in_h != 1 || d.in_w != 1 || d.groups != 1) return CADNN_E_SHAPE;
    return cadnn_conv2d(w, x, n, 1, 1, y, ep, stream);
}

cadnn_status cadnn_maxpool2d(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype,
                             void *y, void *stream)
{
    if (!x || !y || n < 0 || h < 1 || wd < 1 || c < 1 || k < 1 || stride < 1 || pad < 0) return CADNN_E_ARG;
    if (pad >= k || h + 2 * pad < k || wd + 2 * pad < k) return CADNN_E_SHAPE;
    if (dtype != CADNN_F32 && dtype != CADNN_S8) return CADNN_E_DTYPE;
    return launch_maxpool(x, n, h, wd, c, k, stride, pad, dtype, y, false, (cudaStream_t)stream);
}

cadnn_status cadnn_pool2d(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype, int kind,
                          void *y, int out_c_total, int out_c_off, void *stream)
{
    if (!x || !y || n < 0 || h < 1 || wd < 1 || c < 1 || k < 1 || stride < 1 || pad < 0 || out_c_total < 0 || out_c_off < 0)
        return CADNN_E_ARG;
    if (kind != 0 && kind != 1) return CADNN_E_ARG;
    if (pad >= k || h + 2 * pad < k || wd + 2 * pad < k) return CADNN_E_SHAPE;
    if (out_c_total > 0 ? out_c_off + c > out_c_total : out_c_off != 0) return CADNN_E_SHAPE;
    if (dtype != CADNN_F32 && dtype != CADNN_S8) return CADNN_E_DTYPE;
    if (kind == 1 && dtype != CADNN_F32) return CADNN_E_DTYPE;
    return launch_pool_window(x, n, h, wd, c, k, stride, pad, dtype, kind, y, out_c_total, out_c_off, false, (cudaStream_t)stream);
}

cadnn_status cadnn_global_avgpool(const float *x, int n, int h, int wd, int c, float *y, void *stream)
{
    if (!x || !y || n < 0 || h < 1 || wd < 1 || c < 1) return CADNN_E_ARG;
    return launch_gavgpool(x, n, h, wd, c, y, false, (cudaStream_t)stream);
}

cadnn_status cadnn_device_status(int *copy_timeouts)
{
    if (!copy_timeouts) return CADNN_E_ARG;
    CADNN_CUDA_TRY(cudaDeviceSynchronize());
    int copies = 0, barriers = 0, tc = 0;
    cadnn_status s = read_copy_timeouts(&copies);
    if (s != CADNN_OK) return s;
    s = read_barrier_timeouts(&barriers);
    if (s != CADNN_OK) return s;
    s = read_tc_timeouts(&tc);
    if (s != CADNN_OK) return s;
    *copy_timeouts = copies + barriers + tc;
    return CADNN_OK;
}

cadnn_status cadnn_debug_set_device_status(int copy_timeouts, int barrier_timeouts)
{
    cadnn_status s = write_copy_timeouts(copy_timeouts);
    if (s != CADNN_OK) return s;
    return write_barrier_timeouts(barrier_timeouts);
}

void cadnn_free_weights(cadnn_weights *w) { cadnn_weights_free(w); }

const char *cadnn_status_str(cadnn_status s)
{
    switch (s) {
        case CADNN_OK: return "ok";
        case CADNN_E_ARG: return "invalid argument";
        case CADNN_E_SHAPE: return "shape mismatch";
        case CADNN_E_DTYPE: return "dtype combination not defined";
        case CADNN_E_UNSUPPORTED: return "not supported";
        case CADNN_E_ALLOC: return "allocation failed";
        case CADNN_E_CUDA: return "CUDA runtime error";
        case CADNN_E_DEVICE_STATUS: return "device status word set";
    }
    return "unknown status";
}

const char *cadnn_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
