// Internal declarations of the sparse-CNN inference library (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <memory>
#include <vector>
#include "cadnn.h"

enum KernelKind {
    KK_SCONV_SPATIAL = 1,  // sparse k x k convolution, spatial tiles with halo
    KK_SCONV_LINEAR = 2,   // sparse 1x1 convolution / fc at large batch: flat pixel ranges
    KK_FC_SPMV = 3,        // sparse fc at small batch: one warp per filter
    KK_DW = 4,             // dense depthwise
    KK_DENSE_SMALLC = 5    // dense conv with <= 4 input channels
};

static const int kPlanarHalo = 1;     // zero border of the channel-planar activation layout
// floats from one channel plane of a planar tensor to the next: the padded plane rounded up to a
// multiple of 4, so that 16-byte copies that start at a multiple of 4 inside a plane are aligned
#ifdef __CUDACC__
__host__ __device__
#endif
static inline int planar_pitch(int h, int w) { return ((h + 2 * kPlanarHalo) * (w + 2 * kPlanarHalo) + 3) & ~3; }
static const int kWarpsPerBlock = 8;  // fc kernel; the conv kernels take it from the schedule

// Per-layer schedule chosen by the packer (Section 4, "Optimization parameters selection").
struct Schedule {
    int kind = 0;
    int T = 1;        // pixel bands per lane (one band = up to 32 output pixels, one per lane)
    int RPW = 1;      // filters per warp
    int NW = 8;       // warps per thread block
    int G = 8;        // filters per thread block = NW * RPW
    int CIc = 0;      // input channels staged per chunk
    int PPb = 4;      // bytes per staged input pixel (an odd number of 32-bit words)
    int BW = 32, RB = 1;     // band = RB rows x BW columns of output pixels (RB * BW <= 32)
    int TBX = 1, TBY = 1;    // bands across / down in a tile (T = TBX * TBY)
    int TH = 1, TW = 32;     // output tile = (TBY * RB) x (TBX * BW)
    int pitch = 0;           // staged input row pitch in pixels (padded so a band hits 32 distinct banks)
    int half = 0;            // stride 2: columns per parity plane of a staged row (0 = not de-interleaved)
    int IH_t = 0, IW_t = 0;  // staged input tile extent
    int n_chunks = 1;
    int n_groups = 1;
    int stages = 1;          // shared-memory pipeline depth
    int ksplit = 1;          // thread blocks per cluster splitting the channel chunks (partial sums meet in DSMEM)
    int max_entries = 0;     // (padded) entries of the fullest (chunk, filter block) record
    int tile_bytes = 0, stage_bytes = 0, smem_bytes = 0;
};

// Schedule of the shared-memory-staged planar kernel (planar_staged.cu).
struct PsSchedule {
    int T = 1;        // position bands per lane (a band = 32 consecutive positions of the padded plane)
    int RPW = 1;      // filters per warp slot
    int NW = 8;       // warps per block = filter slots x KS
    int KS = 1;       // warps sharing a filter (each takes a share of its nonzeros in every chunk)
    int G = 8;        // filters per block = (NW / KS) * RPW
    int CIc = 0;      // input channels staged per chunk
    int stages = 1;
    int tma = 0;      // 1: staged by TMA copies on mbarriers (stages may then cover all chunks), 0: cp.async by all threads
    int RB = 0, nb = 0;          // TMA: channel rows per box (<= 256), boxes per chunk
    int KC = 1;                  // TMA: blocks per cluster splitting the channel chunks (partial sums meet in DSMEM)
    int part_off = 0;            // byte offset of the cluster partial sums in shared memory
    int n_chunks = 1, n_groups = 1;
    int A = 0, L = 32;           // staged margin / floats per channel
    int q_start = 0, tiles = 1;  // first computed position, tiles per image
    int R = 0;                   // row-tile mode (stride 2 layers): output rows per tile; 0 = linear mode
    int max_entries = 0;
    int hdr_bytes = 0, block_bytes = 0, tile_bytes = 0, stage_bytes = 0, smem_bytes = 0;
};

// measured schedule choices of one layer, as kept in the schedule cache (pack.cu)
struct TuneRecord {
    Schedule s;
    PsSchedule ps;
    int pl_T, pl_NW, pl_RPW, pl_KSW, pl_D, use_ps;
    float pl_us, ps_us, nhwc_us;
};

struct cadnn_weights {
    cadnn_layer_desc desc;
    uint64_t tune_key = 0;                 // key of this layer in the schedule cache (0 = not a tuned pack)
    std::shared_ptr<TuneRecord> tuned;     // choices taken from the cache instead of timing
    int fmt = 0;
    int h_out = 1, w_out = 1;
    int64_t nnz = 0;
    int64_t packed_bytes = 0;
    Schedule s;
    bool on_device = false;
    int device = -1;

    // host image
    std::vector<uint32_t> ent;       // conv: fixed-size records, one per (chunk, filter block): a header of
                                     // G + 1 row starts, then entries.  f32 entry: {value bits, byte offset};
                                     // s8 entry: (byte offset << 8) | (value & 0xff).  Rows padded to even counts.
    std::vector<int32_t> cnt;        // conv: real entries per [chunk][packed row] (the rest is padding)
    std::vector<float> vals_f;       // fc f32: stored values (packed order)
    std::vector<int8_t> vals_q;      // fc s8
    std::vector<uint16_t> offs;      // fc: column index
    std::vector<int32_t> ptr;        // fc: [c_pad + 1]
    std::vector<int32_t> perm;       // packed row -> original output channel, -1 = padding row
    std::vector<float> dense_f;      // dense kinds: tap-major weights
    std::vector<uint8_t> dense_kept; // dense kinds: which positions the mask kept (host only, for unpack)
    int c_pad = 0;

    // channel-planar variant of a float conv layer (see planar.cu): CSR by output channel,
    // entries {value bits, element offset into the padded planar input}, rows padded to even counts
    bool has_planar = false;
    std::vector<uint32_t> pl_ent;
    std::vector<int32_t> pl_ptr;     // [c_out + 1], in entries
    std::vector<int32_t> pl_order;   // warp slot -> output channel (filters dealt to warps by load)
    std::vector<int64_t> row_nnz;    // stored nonzeros per output channel
    int pl_T = 2, pl_NW = 8, pl_RPW = 1, pl_KSW = 1;   // bands per lane, warps per block, filters per warp slot, warps per filter
    int pl_D = 1;                                      // batch depth of the direct planar kernel (1, 2 or 4)
    const uint32_t *d_pl_ent = nullptr;
    const int32_t *d_pl_ptr = nullptr;
    const int32_t *d_pl_order = nullptr;

    // shared-memory-staged planar variant (stride-1 "same" float conv): records per (chunk, filter block)
    bool has_ps = false;
    bool use_ps = false;             // the network runner prefers it over the direct planar kernel
    PsSchedule ps;
    float ps_us = -1.0f, pl_us = -1.0f;   // measured time of the staged / direct planar kernel (autotune), microseconds
    float nhwc_us = -1.0f;                // ... and of the NHWC kernel
    std::vector<uint32_t> ps_ent;
    std::vector<int32_t> ps_perm;    // packed row -> output channel, -1 = padding row
    const uint32_t *d_ps_ent = nullptr;
    const int32_t *d_ps_perm = nullptr;

    // tensor-core blocks of a block-structured int8 layer (blocktc.cu): the dense 64 x 64 blocks, the rest of the
    // layer stays in the sparse image above
    bool has_tc = false;
    std::vector<int8_t> tc_wblk;        // [n_blocks][64 rows][64 bytes], rows = output channels, 16-byte chunks swizzled
    std::vector<int32_t> tc_blk;        // [n_blocks][4]: column shift, row shift of the tap, first input channel, 0
    std::vector<int32_t> tc_tile_ptr;   // [c_out / 64 + 1] blocks of every tile of 64 output channels
    std::vector<int32_t> tc_grp;        // [n_groups][4]: blocks of one (input chunk, kernel column): column shift, first input
                                        // channel, mask of the kernel rows present, first block
    std::vector<int32_t> tc_grp_ptr;    // [c_out / 64 + 1] groups of every tile of 64 output channels
    std::vector<uint8_t> tc_kept;       // [n_blocks][64][64] which positions of a block the mask kept (host only, for unpack)
    int64_t tc_nnz = 0;                 // kept positions inside the dense blocks
    // float stride-2 layers (3x3 pad 1, 1x1): the same layer packed as a stride-1 layer over the parity planes of its
    // input (owned; null = none)
    cadnn_weights *half = nullptr;
    void *d_tc_blob = nullptr;
    const int8_t *d_tc_wblk = nullptr;
    const int32_t *d_tc_grp = nullptr;
    const int32_t *d_tc_grp_ptr = nullptr;

    // device image (one allocation)
    void *d_blob = nullptr;
    const uint32_t *d_ent = nullptr;
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
    bool pdl = false;   // launch as a programmatic dependent of the previous kernel (inside cadnn_forward)
    bool early_trigger = false;   // trigger dependents at kernel start instead of before the epilogue
    bool planar_out = false;   // dense stem: write the channel-planar layout instead of NHWC
    float res_scale = 0.0f;   // int8 layers: multiplier of the int8 residual
    const int *acc_in = nullptr;   // int8 sparse conv: int32 sums [pixels][c_out] added to the accumulators before the epilogue
    int out_c_total = 0, out_c_off = 0;   // NHWC sparse conv: channel window of a wider output tensor (concatenation)
    // planar sparse convs: a second copy of the output split by row and column parity, for a stride-2 reader
    // (parity_planes_bytes below gives its size); parity_mask = planes wanted, bit (row parity * 2 + column parity)
    float *parity_y = nullptr;
    int parity_mask = 0;
};

// Parity planes of an h x w map of c channels: plane (py * 2 + px) holds the pixels (2 i + py, 2 j + px) at (i, j) of a
// padded plane of ceil(h / 2) x ceil(w / 2) (absent pixels of odd sizes stay zero).  Layout [image][plane][channel][pitch];
// with mask 1 only the (even, even) plane exists.  A stride-2 3x3 (pad 1) layer over the map is a stride-1 layer over
// the 4 c quarter planes, a stride-2 1x1 layer a stride-1 layer over plane 0.
struct ParityPlanes {
    float *y;        // null = none
    int mask, planes, wp, pitch, c;
};
static inline ParityPlanes parity_planes(float *y, int mask, int h, int w, int c)
{
    ParityPlanes pp;
    pp.y = y; pp.mask = mask; pp.planes = mask == 1 ? 1 : 4;
    pp.wp = (w + 1) / 2 + 2 * kPlanarHalo;
    pp.pitch = planar_pitch((h + 1) / 2, (w + 1) / 2);
    pp.c = c;
    return pp;
}
static inline int64_t parity_planes_bytes(int mask, int n, int h, int w, int c)
{
    return (int64_t)n * (mask == 1 ? 1 : 4) * c * planar_pitch((h + 1) / 2, (w + 1) / 2) * 4;
}

// status helpers
cadnn_status cadnn_note_cuda(cudaError_t e);
#define CADNN_CUDA_TRY(expr)                                  \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) return cadnn_note_cuda(e__);  \
    } while (0)

// Dynamic shared memory above 48 KB has to be allowed per kernel AND per device.  One
// SmemLimit per kernel instantiation remembers, for each device, what has been allowed;
// raise_smem_limit raises it when a launch needs more (serialized by one mutex).
const int kMaxDevices = 64;
struct SmemLimit {
    int allowed[kMaxDevices];   // zero = the default 48 KB
};
cadnn_status raise_smem_limit(const void *kern, int smem, SmemLimit *lim);

// epilogue / device checks of one layer call (no launch): what conv2d_impl would refuse
cadnn_status check_layer_call(const cadnn_weights *w, bool has_residual, int act, int out_dtype, int out_c_total = 0,
                              int out_c_off = 0);

// kernel launchers (each validates nothing; callers did)
cadnn_status launch_sconv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                          cudaStream_t st);
cadnn_status launch_fc_spmv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                            cudaStream_t st);
cadnn_status launch_dw(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                       cudaStream_t st);
cadnn_status launch_dense_smallc(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                 cudaStream_t st);
cadnn_status launch_sconv_planar(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                 cudaStream_t st);
cadnn_status launch_sconv_planar_staged(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                        cudaStream_t st);
bool dw_planar_ok(const cadnn_weights *w);   // a depthwise layer the planar layout can run (float, <= 9 taps, pad within the halo)
cadnn_status launch_dw_planar(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                              cudaStream_t st);
// block-structured int8 layers (blocktc.cu)
bool block_tc_extract(cadnn_weights *h, const int8_t *q, const uint8_t *mask, double threshold, std::vector<uint8_t> &rem_mask);
cadnn_status block_tc_upload(cadnn_weights *h);
// acc != null: int32 sums for the sparse kernel; acc == null: the layer has no sparse remainder and the kernel
// applies the epilogue *le and writes y itself
cadnn_status launch_block_tc(const cadnn_weights *w, const void *x, int n, int *acc, void *y, const LaunchEpilogue *le, cudaStream_t st);
cadnn_status read_tc_timeouts(int *count);
cadnn_status read_copy_timeouts(int *count);
cadnn_status read_barrier_timeouts(int *count);
// the same counters copied to (pinned) host memory in stream order, and overwritten (tests)
cadnn_status read_copy_timeouts_async(int *host_dst, cudaStream_t st);
cadnn_status read_barrier_timeouts_async(int *host_dst, cudaStream_t st);
cadnn_status write_copy_timeouts(int value);
cadnn_status write_barrier_timeouts(int value);

// Tensor map (a CUtensorMap, 128 bytes, 64-byte aligned, written to *map) over a float matrix of
// `rows` channel planes by `cols` floats, copied in boxes of box_rows x box_cols; elements outside
// the matrix read as zero.  False when the driver entry point is missing or refuses the shape.
bool encode_plane_rows_map(void *map, const void *base, unsigned long long cols, unsigned long long rows,
                           unsigned box_cols, unsigned box_rows);

// Tensor map over an int8 NHWC tensor [n][h][w][c] copied in boxes of box_h x box_w pixels x box_c (= 64) channels,
// written to shared memory as box_h * box_w rows of 64 bytes with the 64-byte swizzle the tensor cores read;
// pixels outside an image read as zero.
bool encode_nhwc_s8_tiles_map(void *map, const void *base, int c, int w, int h, int n, int box_c, int box_w, int box_h);

// Persistent kernel over a run of planar sparse convs (persist.cu).  One entry per conv, in
// network order; join_phase: the op reads nothing that the ops of the current phase write, so
// it may run in the same phase as its predecessor (no grid barrier between them).
struct PersistPlan;
struct PersistOpDesc {
    const cadnn_weights *w = nullptr;
    const void *x = nullptr;
    void *y = nullptr;
    const void *residual = nullptr;
    const float *scale = nullptr;
    const float *bias = nullptr;
    int act = 0;
    int n = 1;
    bool join_phase = false;
    bool dst_external = false;   // y is read by something outside the run (or is the run's result)
};
cadnn_status persist_create(const std::vector<PersistOpDesc> &descs, PersistPlan **out);
cadnn_status persist_launch(const PersistPlan *plan, cudaStream_t st);
int persist_phases(const PersistPlan *plan);
// plan of op `op` of the run: bands per tile, bands per unit, filters per group, tiles, groups, staged floats per
// channel, channels per chunk, chunks per pass, passes, strided, modelled clocks, phase; 0 if there is no such op
int persist_describe(const PersistPlan *plan, int op, int out[12]);
cadnn_status persist_profile(const PersistPlan *plan, int cap, float *wall_clk, float *busy_max_clk, float *busy_mean_clk,
                             float *issued_clk, float *landed_clk, int *n_out);
void persist_free(PersistPlan *plan);
cadnn_status launch_maxpool_planar(const float *x, int n, int h, int wd, int c, int k, int stride, int pad, float *y,
                                   bool pdl, cudaStream_t st);
cadnn_status launch_gavgpool_planar(const float *x, int n, int h, int wd, int c, float *y, bool pdl, cudaStream_t st);
cadnn_status launch_maxpool(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype,
                            void *y, bool pdl, cudaStream_t st);
// max (kind 0) or average (kind 1, float) pool into channels [c_off, c_off + c) of a y with ldc channels per pixel
cadnn_status launch_pool_window(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype, int kind,
                                void *y, int ldc, int c_off, bool pdl, cudaStream_t st);
cadnn_status launch_gavgpool(const float *x, int n, int h, int wd, int c, float *y, bool pdl, cudaStream_t st);

// layer entry shared by the public calls and the network runner
cadnn_status conv2d_impl(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y, const cadnn_epilogue *ep,
                         bool pdl, cudaStream_t st, void *workspace = nullptr, int64_t workspace_bytes = 0);

#ifdef __CUDACC__
// Division by a runtime constant as multiply-high and shift (the divisor is fixed per
// launch; a hardware integer division costs a few dozen dependent instructions).
// q = umulhi(n, mul) >> shr is exact for 0 <= n < 2^31 when mul = ceil(2^(32 + shr) / d)
// and 2^shr >= d (shr chosen so that mul fits 32 bits); d == 1 is passed through.
struct FastDiv {
    unsigned mul, shr, d;
};
static inline FastDiv make_fastdiv(int d)
{
    FastDiv f;
    f.d = (unsigned)d;
    f.mul = 0;
    f.shr = 0;
    if (d <= 1) return f;
    unsigned l = 0;
    while ((1u << l) < (unsigned)d) ++l;              // ceil(log2 d)
    unsigned long long p2 = 1ull << (31 + l);
    f.mul = (unsigned)((p2 + d - 1) / (unsigned long long)d);
    f.shr = l - 1;
    return f;
}
__device__ __forceinline__ unsigned fdiv(unsigned n, const FastDiv &f)
{
    return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

// Programmatic dependent launch: a kernel launched with the attribute may start before its
// predecessor in the stream has finished; it must not touch data the predecessor writes
// until grid_dep_wait() returns.  Without the attribute both calls do nothing.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Activations and residuals may have been written by the kernel this one depends on
// programmatically, i.e. while this kernel was already running: they are read with ordinary
// loads.  The read-only path (ld.global.nc / __ldg) promises data that is constant for the whole
// lifetime of the kernel and is kept for weights, scales and biases.
__device__ __forceinline__ float ld_act(const float *p)
{
    float v;
    asm volatile("ld.global.f32 %0, [%1];\n" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ signed char ld_act(const signed char *p)
{
    int v;
    asm volatile("ld.global.s8 %0, [%1];\n" : "=r"(v) : "l"(p));
    return (signed char)v;
}

// value v of output pixel (row, col) (interior coordinates), channel co, image img -> its parity plane
__device__ __forceinline__ void parity_store(const ParityPlanes &pp, unsigned img, int co, int row, int col, float v)
{
    const int par = (row & 1) * 2 + (col & 1);
    if (!((pp.mask >> par) & 1)) return;
    const int pl = pp.planes == 4 ? par : 0;
    pp.y[(((size_t)img * pp.planes + pl) * pp.c + co) * pp.pitch + ((row >> 1) + kPlanarHalo) * pp.wp + (col >> 1) + kPlanarHalo] = v;
}

// ---- epilogue arithmetic shared by the conv kernels ----
__device__ __forceinline__ float act_f32(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

// int8 layer: one fused multiply-add on the converted accumulator, a second one for the int8 residual
// of a quantized residual block (r * residual_scale joins before the activation), ReLU
__device__ __forceinline__ float requant_f32(int acc, float m, float b, int act, bool has_res = false, int r = 0, float rs = 0.0f)
{
    float t = __fmaf_rn(__int2float_rn(acc), m, b);
    if (has_res) t = __fmaf_rn(__int2float_rn(r), rs, t);
    if (act == CADNN_ACT_RELU) t = t > 0.0f ? t : 0.0f;
    return t;
}
__device__ __forceinline__ int requant_s8(int acc, float m, float b, int act, bool has_res = false, int r = 0, float rs = 0.0f)
{
    float t = requant_f32(acc, m, b, act, has_res, r, rs);
    t = fminf(fmaxf(t, -127.0f), 127.0f);
    return __float2int_rn(t);
}

template <typename... KArgs, typename... Args>
cadnn_status launch_kernel(void (*kern)(KArgs...), int blocks, int threads, size_t smem, bool pdl, cudaStream_t st,
                           Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    CADNN_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...));
    return CADNN_OK;
}
#endif

static inline int dtype_size(int dt) { return dt == CADNN_S8 ? 1 : 4; }
