// cadnn_forward_static: run an op list without allocating anything.
//
// cadnn_net_create gives every intermediate tensor its own cudaMalloc'ed buffer.  Some
// callers must not allocate when they run a network: a serving thread on a latency path
// (cudaMalloc and cudaFree synchronize the whole device and stall every other stream), a
// process whose device memory is already handed out in full to a framework's caching
// allocator, or code that has to run a batch size it did not plan a cadnn_net for.  For
// them this entry point places the intermediate tensors in one fixed device array that is
// part of the library image, planned on the host with first-fit reuse of regions whose
// last reader has been issued.  Layers still run in the same kernels as cadnn_forward.
//
// The paper (arXiv 1905.00571) has no counterpart of this call.
#include <algorithm>
#include <mutex>
#include "cadnn_internal.h"

namespace {

// Intermediate activations of one forward live here.  Every GPU that loads the library
// holds these bytes until the process exits.
const size_t kArenaBytes = (size_t)CADNN_STATIC_WORKSPACE_BYTES;
static __device__ __align__(256) unsigned char g_arena[CADNN_STATIC_WORKSPACE_BYTES];

// In host code `g_arena` is only a handle for the runtime's symbol calls; its device
// address has to be asked for, once per device, with that device current.
std::mutex g_mu;
unsigned char *g_arena_dev[kMaxDevices] = {nullptr};

cadnn_status arena_base(unsigned char **out)
{
    int dev = -1;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CADNN_E_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_arena_dev[dev]) {
        void *p = nullptr;
        CADNN_CUDA_TRY(cudaGetSymbolAddress(&p, g_arena));
        g_arena_dev[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_arena_dev[dev];
    return CADNN_OK;
}

struct Tensor {
    int n = 0, h = 0, w = 0, c = 0, dtype = 0;
    bool defined = false;
    size_t off = 0, bytes = 0;   // region inside the arena (intermediate slots only)
    int last_use = -1;           // index of the last op that reads it
};

// The plan lives in fixed-size host arrays on the stack: no heap either.
const int kMaxOps = 512;

struct FreeBlock {
    size_t off, bytes;
};

struct FreeList {
    FreeBlock b[kMaxOps + 2];
    int n = 0;
    void erase(int i)
    {
        for (int j = i; j + 1 < n; ++j) b[j] = b[j + 1];
        --n;
    }
    void insert(int i, FreeBlock v)
    {
        for (int j = n; j > i; --j) b[j] = b[j - 1];
        b[i] = v;
        ++n;
    }
};

// first fit over the free list; regions are multiples of 256 bytes
bool arena_take(FreeList &fl, size_t bytes, size_t *off)
{
    for (int i = 0; i < fl.n; ++i) {
        if (fl.b[i].bytes >= bytes) {
            *off = fl.b[i].off;
            fl.b[i].off += bytes;
            fl.b[i].bytes -= bytes;
            if (fl.b[i].bytes == 0) fl.erase(i);
            return true;
        }
    }
    return false;
}

void arena_give(FreeList &fl, size_t off, size_t bytes)
{
    int i = 0;
    while (i < fl.n && fl.b[i].off < off) ++i;
    fl.insert(i, FreeBlock{off, bytes});
    // merge with neighbours
    if (i + 1 < fl.n && fl.b[i].off + fl.b[i].bytes == fl.b[i + 1].off) {
        fl.b[i].bytes += fl.b[i + 1].bytes;
        fl.erase(i + 1);
    }
    if (i > 0 && fl.b[i - 1].off + fl.b[i - 1].bytes == fl.b[i].off) {
        fl.b[i - 1].bytes += fl.b[i].bytes;
        fl.erase(i);
    }
}

}  // namespace

extern "C" {

cadnn_status cadnn_forward_static(const cadnn_op *ops, int n_ops, int n, int h, int wd, int c, int in_dtype,
                                  const void *x, void *y, void *stream)
{
    if (!ops || n_ops < 1 || n < 1 || h < 1 || wd < 1 || c < 1 || !x || !y) return CADNN_E_ARG;
    if (n_ops > kMaxOps) return CADNN_E_UNSUPPORTED;
    if (in_dtype != CADNN_F32 && in_dtype != CADNN_S8) return CADNN_E_DTYPE;
    cudaStream_t st = (cudaStream_t)stream;

    // ---- shapes, last readers ----
    int max_slot = 0;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i].src < 0 || ops[i].dst < 1 || ops[i].res < -1) return CADNN_E_ARG;
        max_slot = std::max(max_slot, std::max(ops[i].src, std::max(ops[i].dst, ops[i].res)));
    }
    if (max_slot > kMaxOps) return CADNN_E_UNSUPPORTED;
    Tensor t[kMaxOps + 1];
    t[0].n = n; t[0].h = h; t[0].w = wd; t[0].c = c; t[0].dtype = in_dtype; t[0].defined = true;
    const int out_slot = ops[n_ops - 1].dst;
    for (int i = 0; i < n_ops; ++i) {
        const cadnn_op &op = ops[i];
        const Tensor si = t[op.src];
        Tensor &so = t[op.dst];
        const bool window = op.dst_c_total > 0;
        if (op.dst_c_total < 0 || op.dst_c_off < 0 || (!window && op.dst_c_off != 0)) return CADNN_E_ARG;
        if (!si.defined || (so.defined && !window)) return CADNN_E_ARG;
        Tensor sn;   // what this op produces
        sn.n = si.n;
        if (op.kind == CADNN_OP_CONV || op.kind == CADNN_OP_FC) {
            if (!op.w || !op.w->on_device) return CADNN_E_ARG;
            if (op.w->has_tc) return CADNN_E_UNSUPPORTED;   // block-structured layers need a workspace of their own
            const cadnn_layer_desc &d = op.w->desc;
            if (d.dtype != si.dtype) return CADNN_E_DTYPE;
            if (op.kind == CADNN_OP_FC) {
                if ((long long)si.h * si.w * si.c != d.c_in) return CADNN_E_SHAPE;
            } else if (si.h != d.in_h || si.w != d.in_w || si.c != d.c_in) {
                return CADNN_E_SHAPE;
            }
            sn.h = op.w->h_out; sn.w = op.w->w_out; sn.c = d.c_out; sn.dtype = op.out_dtype;
            if (op.res >= 0) {
                const Tensor &sr = t[op.res];
                const int want_dt = d.dtype == CADNN_S8 ? CADNN_S8 : sn.dtype;   // int8 layers take an int8 residual
                if (!sr.defined || sr.h != sn.h || sr.w != sn.w || sr.c != sn.c || sr.dtype != want_dt)
                    return CADNN_E_SHAPE;
            }
            // everything the layer call itself would refuse is refused here, before the first launch:
            // the epilogue combination, weights packed on another GPU, an input beyond the staging limit
            cadnn_status cs = check_layer_call(op.w, op.res >= 0, op.act, op.out_dtype, op.dst_c_total, op.dst_c_off);
            if (cs != CADNN_OK) return cs;
            if ((long long)si.n * si.h * si.w * si.c * dtype_size(si.dtype) >= (1LL << 34)) return CADNN_E_UNSUPPORTED;
        } else if (op.kind == CADNN_OP_MAXPOOL || op.kind == CADNN_OP_AVGPOOL) {
            if (op.pool_k < 1 || op.pool_stride < 1 || op.pool_pad < 0 || op.pool_pad >= op.pool_k ||
                si.h + 2 * op.pool_pad < op.pool_k || si.w + 2 * op.pool_pad < op.pool_k)
                return CADNN_E_SHAPE;
            if (op.kind == CADNN_OP_AVGPOOL && si.dtype != CADNN_F32) return CADNN_E_DTYPE;
            sn.h = (si.h + 2 * op.pool_pad - op.pool_k) / op.pool_stride + 1;
            sn.w = (si.w + 2 * op.pool_pad - op.pool_k) / op.pool_stride + 1;
            sn.c = si.c; sn.dtype = si.dtype;
        } else if (op.kind == CADNN_OP_GAVGPOOL) {
            if (window) return CADNN_E_UNSUPPORTED;
            if (si.dtype != CADNN_F32) return CADNN_E_DTYPE;
            sn.h = 1; sn.w = 1; sn.c = si.c; sn.dtype = CADNN_F32;
        } else {
            return CADNN_E_ARG;
        }
        t[op.src].last_use = i;
        if (op.res >= 0) t[op.res].last_use = i;
        if (window) {
            if (op.dst_c_off + sn.c > op.dst_c_total) return CADNN_E_SHAPE;
            sn.c = op.dst_c_total;
            if (so.defined) {   // a later writer of the same concatenation
                if (so.h != sn.h || so.w != sn.w || so.c != sn.c || so.dtype != sn.dtype || so.n != sn.n) return CADNN_E_SHAPE;
                continue;
            }
        }
        so.n = sn.n; so.h = sn.h; so.w = sn.w; so.c = sn.c; so.dtype = sn.dtype;
        so.defined = true;
        so.bytes = ((size_t)so.n * so.h * so.w * so.c * dtype_size(so.dtype) + 255) / 256 * 256;
    }

    // ---- place the intermediate tensors: first fit, a region returns to the free list once
    //      the last op reading it has been issued (all ops run in order on one stream) ----
    FreeList fl;
    fl.insert(0, FreeBlock{0, kArenaBytes});
    int placed_at[kMaxOps + 1];
    for (int i = 0; i <= max_slot; ++i) placed_at[i] = -1;
    for (int i = 0; i < n_ops; ++i) {
        const cadnn_op &op = ops[i];
        if (op.dst != out_slot && placed_at[op.dst] < 0) {   // (a concatenation is placed by its first writer)
            // does not fit the fixed workspace: refuse rather than allocate
            if (!arena_take(fl, t[op.dst].bytes, &t[op.dst].off)) return CADNN_E_UNSUPPORTED;
            placed_at[op.dst] = i;
        }
        // inputs whose last reader is this op are free for the NEXT op's output (never for this op's own)
        for (int s : {op.src, op.res}) {
            if (s > 0 && s != out_slot && placed_at[s] >= 0 && t[s].last_use == i) {
                arena_give(fl, t[s].off, t[s].bytes);
                placed_at[s] = -1;
            }
        }
    }

    // ---- run ----
    unsigned char *base = nullptr;
    cadnn_status rc = arena_base(&base);
    if (rc != CADNN_OK) return rc;
    auto ptr_of = [&](int slot) -> void * {
        if (slot == 0) return const_cast<void *>(x);
        if (slot == out_slot) return y;
        return base + t[slot].off;
    };
    for (int i = 0; i < n_ops; ++i) {
        const cadnn_op &op = ops[i];
        const Tensor &si = t[op.src];
        const void *src = ptr_of(op.src);
        void *dst = ptr_of(op.dst);
        if (op.kind == CADNN_OP_CONV || op.kind == CADNN_OP_FC) {
            cadnn_epilogue ep;
            ep.scale = op.scale;
            ep.bias = op.bias;
            ep.residual = op.res >= 0 ? ptr_of(op.res) : nullptr;
            ep.act = op.act;
            ep.out_dtype = op.out_dtype;
            ep.out_c_total = op.dst_c_total;
            ep.out_c_off = op.dst_c_off;
            ep.residual_scale = op.res_scale;
            if (op.kind == CADNN_OP_FC) rc = conv2d_impl(op.w, src, si.n, 1, 1, dst, &ep, false, st);
            else rc = conv2d_impl(op.w, src, si.n, si.h, si.w, dst, &ep, false, st);
        } else if (op.kind == CADNN_OP_MAXPOOL || op.kind == CADNN_OP_AVGPOOL) {
            rc = launch_pool_window(src, si.n, si.h, si.w, si.c, op.pool_k, op.pool_stride, op.pool_pad, si.dtype,
                                    op.kind == CADNN_OP_AVGPOOL ? 1 : 0, dst, op.dst_c_total, op.dst_c_off, false, st);
        } else {
            rc = launch_gavgpool((const float *)src, si.n, si.h, si.w, si.c, (float *)dst, false, st);
        }
        if (rc != CADNN_OK) return rc;
    }
    return CADNN_OK;
}

}  // extern "C"
