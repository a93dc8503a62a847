// Internal declarations of the sparse-CNN inference library (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <vector>
#include "cadnn.h"

enum KernelKind {
    KK_SCONV_SPATIAL = 1,  // sparse k x k convolution, spatial tiles with halo
    KK_SCONV_LINEAR = 2,   // sparse 1x1 convolution / fc at large batch: flat pixel ranges
    KK_FC_SPMV = 3,        // sparse fc at small batch: one warp per filter
    KK_DW = 4,             // dense depthwise
    KK_DENSE_SMALLC = 5    // dense conv with <= 4 input channels
};

static const int kWarpsPerBlock = 8;

// Per-layer schedule chosen by the packer (Section 4, "Optimization parameters selection").
struct Schedule {
    int kind = 0;
    int T = 1;        // output pixels per lane
    int RPW = 1;      // filters per warp
    int G = 8;        // filters per thread block = kWarpsPerBlock * RPW
    int CIc = 0;      // input channels staged per chunk
    int PP = 1;       // shared-memory words per staged input pixel (odd: CIc | 1)
    int TH = 1, TW = 1;      // output tile (spatial mode)
    int pitch = 0;           // staged input row pitch in pixels (== TW mod 32)
    int IH_t = 0, IW_t = 0;  // staged input tile extent
    int n_chunks = 1;
    int n_groups = 1;
    int max_entries = 0;     // most nonzeros any (block, chunk) holds
    int tile_words = 0;
    int smem_bytes = 0;
};

struct cadnn_weights {
    cadnn_layer_desc desc;
    int fmt = 0;
    int h_out = 1, w_out = 1;
    int64_t nnz = 0;
    int64_t packed_bytes = 0;
    Schedule s;
    bool on_device = false;
    int device = -1;

    // host image
    std::vector<float> vals_f;       // f32 layers: stored values (packed order)
    std::vector<int8_t> vals_q;      // s8 layers
    std::vector<uint16_t> offs;      // sconv: staged-tile word offset; fc: column index
    std::vector<int32_t> ptr;        // sconv: [n_chunks][c_pad + 1]; fc: [c_pad + 1]
    std::vector<int32_t> perm;       // packed row -> original output channel, -1 = padding row
    std::vector<float> dense_f;      // dense kinds: tap-major weights
    int c_pad = 0;

    // device image (one allocation)
    void *d_blob = nullptr;
    const void *d_vals = nullptr;
    const uint16_t *d_offs = nullptr;
    const int32_t *d_ptr = nullptr;
    const int32_t *d_perm = nullptr;
    const float *d_dense = nullptr;
};

struct LaunchEpilogue {
    const float *scale = nullptr;
    const float *bias = nullptr;
    const void *residual = nullptr;
    int act = 0;
    int out_dtype = 0;
};

// status helpers
cadnn_status cadnn_note_cuda(cudaError_t e);
#define CADNN_CUDA_TRY(expr)                                  \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) return cadnn_note_cuda(e__);  \
    } while (0)

// kernel launchers (each validates nothing; callers did)
cadnn_status launch_sconv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                          cudaStream_t st);
cadnn_status launch_fc_spmv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                            cudaStream_t st);
cadnn_status launch_dw(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                       cudaStream_t st);
cadnn_status launch_dense_smallc(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                 cudaStream_t st);
cadnn_status launch_maxpool(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype,
                            void *y, cudaStream_t st);
cadnn_status launch_gavgpool(const float *x, int n, int h, int wd, int c, float *y, cudaStream_t st);

static inline int dtype_size(int dt) { return dt == CADNN_S8 ? 1 : 4; }
