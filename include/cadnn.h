/*
 * cadnn.h - C ABI of the sparse-CNN inference library (CUDA, sm_100a).
 *
 * The library runs forward inference of weight-pruned, optionally int8
 * weight-quantized convolutional networks: every conv / FC layer multiplies a
 * fixed, compressed sparse weight tensor by dense activations.  It restates, for
 * one datacenter GPU, the execution stage of CADNN (arXiv 1905.00571, Section 4
 * "Architecture-aware Optimization"): compressed weight storage with an offline
 * layout transformation, fused Conv + BatchNorm + Activation kernels, 1x1
 * convolutions run as a sparse-matrix product, and a per-layer choice of tiling
 * parameters made once per model.
 *
 * Conventions
 *  - Activations are NHWC, contiguous.  Dense weights handed to the packer are
 *    OHWI: [c_out][kh][kw][c_in/groups].
 *  - Every call returns a cadnn_status; nothing aborts or throws across the ABI.
 *    Output pointers are written only when CADNN_OK is returned.
 *  - "host" / "device" on each pointer says where the memory must live.  The
 *    caller owns every buffer it passes; a cadnn_weights / cadnn_net handle owns
 *    the device memory it allocated and releases it in its *_free call.
 *  - Kernels are launched asynchronously on the stream given (a cudaStream_t
 *    passed as void*, NULL = the default stream).  No call synchronizes the
 *    device unless its comment says so.
 *  - Inputs must be finite; NaN / Inf behaviour is unspecified (a pruned weight
 *    contributes exactly 0 only for finite activations).
 *  - There is no CPU fallback: without a CUDA device every compute call fails
 *    with CADNN_E_CUDA.
 */
#ifndef CADNN_H
#define CADNN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CADNN_OK = 0,
    CADNN_E_ARG = 1,          /* NULL or inconsistent argument */
    CADNN_E_SHAPE = 2,        /* shape differs from what the handle was packed for, or is invalid */
    CADNN_E_DTYPE = 3,        /* dtype combination not defined */
    CADNN_E_UNSUPPORTED = 4,  /* valid request the library does not implement */
    CADNN_E_ALLOC = 5,        /* host or device allocation failed */
    CADNN_E_CUDA = 6,         /* a CUDA runtime call failed (cadnn_last_cuda_error) */
    CADNN_E_DEVICE_STATUS = 7 /* a kernel recorded an error in the device status word */
} cadnn_status;

typedef enum { CADNN_F32 = 0, CADNN_S8 = 1, CADNN_S32 = 2 } cadnn_dtype;
typedef enum { CADNN_ACT_NONE = 0, CADNN_ACT_RELU = 1, CADNN_ACT_RELU6 = 2 } cadnn_act;

/* Storage format of a packed layer (reported by cadnn_weights_info). */
typedef enum {
    CADNN_FMT_AUTO = 0,        /* let the packer choose (the only value cadnn_pack needs) */
    CADNN_FMT_TILED_CSR = 1,   /* conv: per channel-chunk CSR by output channel, filters regrouped */
    CADNN_FMT_ROW_CSR = 2,     /* fc at small batch: CSR by output channel, rows sorted by length */
    CADNN_FMT_DENSE_DW = 3,    /* dense depthwise filters, tap-major */
    CADNN_FMT_DENSE_SMALLC = 4, /* dense conv with very few input channels (network stem) */
    CADNN_FMT_GROUPED = 5      /* int8 stride-1 conv with block structure (ask for it in cadnn_layer_desc.fmt): the
                                  64 output channels x 64 input channels x one tap blocks of which the mask keeps at
                                  least CADNN_BLOCK_DENSITY (environment, default 0.5) are stored dense and multiplied
                                  on the tensor cores, the rest stays TILED_CSR; needs c_in and c_out multiples of 64 and
                                  a caller-provided workspace (cadnn_conv2d_workspace) */
} cadnn_fmt;

#define CADNN_PACK_HOST_ONLY 1 /* build the packed image on the host only (no device needed, no compute) */
#define CADNN_PACK_AUTOTUNE 2  /* conv layers: time the candidate schedules on the current device (batch_hint
                                  images of zeros, scratch buffers allocated and freed inside the call) and
                                  keep the fastest, instead of trusting the packer's time model.  With
                                  CADNN_TUNE_CACHE=<file> in the environment the choices are appended to that
                                  text file and a later pack of the same layer (geometry, batch hint, nonzeros
                                  per filter) reads them back instead of timing: tune once per machine, and a
                                  profiled run executes the schedules of the plain run */

/*
 * One layer.  The packer is the offline stage of Section 4 ("Memory layout
 * transformation", "Optimization parameters selection"): tile sizes and the
 * filter regrouping depend on the layer's spatial size, so the input size the
 * layer will run at is part of its description.
 *   conv: c_in, c_out, kh, kw, stride, pad, groups (1, or c_in == c_out for depthwise),
 *         in_h, in_w.  pad pads rows and columns alike unless pad_w >= 0, which then pads the
 *         columns (the 1x7 / 7x1 kernels of an Inception module pad one axis only).
 *   fc:   kh = kw = 1, stride = 1, pad = 0, groups = 1, in_h = in_w = 1, c_in = K.
 *   batch_hint: batch size the schedule is tuned for (>= 1); any batch still runs.
 */
typedef struct {
    int c_in, c_out, kh, kw, stride, pad, groups;
    int in_h, in_w;
    int batch_hint;
    int dtype; /* cadnn_dtype of weights and activations: CADNN_F32 or CADNN_S8 */
    int fmt;   /* CADNN_FMT_AUTO, or CADNN_FMT_GROUPED to ask for the block-structured int8 format */
    int flags; /* CADNN_PACK_HOST_ONLY, CADNN_PACK_AUTOTUNE or 0 */
    int pad_w; /* padding of the columns; -1 = same as pad */
} cadnn_layer_desc;

typedef struct cadnn_weights cadnn_weights;
typedef struct cadnn_net cadnn_net;

/*
 * cadnn_pack - compress one layer (Section 4, "Memory layout transformation and
 * load optimization"; load balance is the obstacle Section 1 names).
 *   w_ohwi  host, float [c_out][kh][kw][c_in/groups].
 *   mask    host, uint8 same shape, nonzero = kept; NULL = every weight kept.
 *           The stored set is exactly the kept positions, even where the value is 0.
 *   w_scale host, float [c_out], required for CADNN_S8 (q = clamp(rne(w / w_scale[co]),
 *           -127, 127)); must be NULL for CADNN_F32.
 *   out     receives a handle owning its buffers (device buffers on the current
 *           device unless CADNN_PACK_HOST_ONLY).  Immutable afterwards; may be used
 *           from several streams.
 * Filters are regrouped so that the warps of a thread block get equal nonzero
 * counts; the permutation is undone when results are stored.
 * Errors: E_ARG (NULL, bad desc), E_DTYPE, E_UNSUPPORTED (grouped conv other than
 * depthwise; int8 depthwise; reduction length whose int32 sum could overflow),
 * E_ALLOC, E_CUDA.  Synchronizes the device copy before returning.
 */
cadnn_status cadnn_pack(const cadnn_layer_desc *desc, const float *w_ohwi, const uint8_t *mask,
                        const float *w_scale, cadnn_weights **out);

/* Same for weights that are already int8 codes (desc->dtype must be CADNN_S8). */
cadnn_status cadnn_pack_q8(const cadnn_layer_desc *desc, const int8_t *q_ohwi, const uint8_t *mask,
                           cadnn_weights **out);

/* nnz = kept positions; packed_bytes = bytes of the device image; fmt = cadnn_fmt used.
 * Any output pointer may be NULL. */
cadnn_status cadnn_weights_info(const cadnn_weights *w, int64_t *nnz, int64_t *packed_bytes, int *fmt);

/*
 * Schedule the packer chose (Section 4, "Optimization parameters selection"):
 * sched[0..15] = kernel kind, pixel bands per lane, filters per warp, filters per block,
 * channel chunk, tile rows, tile columns, shared-memory row pitch, warps per block,
 * pipeline stages, blocks per cluster (reduction split), channel chunks, shared-memory
 * bytes per block, bands across, bands down, entries per weight record.  Host ints.
 * The environment variable CADNN_SCHEDULE ("nw=8,rpw=2,tbx=1,tby=4,cic=64,ks=2", any
 * subset) overrides the packer's pick for conv layers; it exists for tuning.
 */
cadnn_status cadnn_weights_schedule(const cadnn_weights *w, int sched[16]);

/*
 * Schedule of the layer's channel-planar variant (the one cadnn_forward and
 * cadnn_conv2d_planar run): sched[0..13] = variant (0 none, 1 direct loads, 2 tile staged in
 * shared memory), position bands per lane, filters per warp, warps per block, warps sharing
 * a filter, filters per block, channel chunk, pipeline stages (direct variant: batch depth,
 * 16 x depth activation loads in flight per lane), channel chunks, tiles per
 * image, shared-memory bytes per block, entries per weight record, and the times measured
 * by CADNN_PACK_AUTOTUNE for the staged and the direct variant in hundredths of a
 * microsecond (negative = not measured), 1 if the tile is staged by TMA copies (0: cp.async),
 * blocks per cluster splitting the input channels.  Host ints.
 */
cadnn_status cadnn_weights_planar_schedule(const cadnn_weights *w, int sched[16]);

/*
 * Per-warp load of the packed image: for every (filter block, warp) the number of
 * stored nonzeros that warp walks.  n_out receives the count; loads (host, may be
 * NULL) receives up to cap entries.
 */
cadnn_status cadnn_weights_warp_loads(const cadnn_weights *w, int64_t *loads, int cap, int *n_out);

/* Expand the packed image back to dense OHWI (masked-out = 0) and the mask.  Host
 * pointers; dense_f32 receives floats (int8 layers: the integer codes as floats);
 * either may be NULL. */
cadnn_status cadnn_weights_unpack(const cadnn_weights *w, float *dense_f32, uint8_t *mask);

void cadnn_weights_free(cadnn_weights *w);
void cadnn_free_weights(cadnn_weights *w); /* the same call under the name the problem statement uses */

/*
 * Fused epilogue (Section 4, "Model computation fusion": Conv/DWConv + BatchNorm +
 * Activation in one kernel; the residual add of a bottleneck block joins it).
 * Float layers:  z = acc * scale[co] + bias[co];  z += residual;  z = act(z).
 * Int8 layers:   t = fmaf((float)acc, scale[co], bias[co])  (one fused multiply-add,
 *                scale = s_x * s_w[co] / s_y, bias = b[co] / s_y, both precomputed by
 *                the caller); ReLU; out_dtype S8: clamp to [-127,127], round half even;
 *                F32: t as is; S32: the raw accumulator (scale / bias / act ignored).
 *                An int8 residual (a quantized residual block; y's shape, dtype S8) joins with a
 *                second fused multiply-add before the ReLU: t = fmaf((float)r, residual_scale, t),
 *                residual_scale = s_r / s_y precomputed by the caller (sparse conv layers, S8 or
 *                F32 output).  ReLU6 is not defined.
 * scale, bias: device float [c_out], NULL = 1 / 0.  residual: device, same shape as y and of
 * the layer's dtype, or NULL.
 * Channel concatenation (the branches of an Inception module, Section 5 / Table 2): with
 * out_c_total > 0, y has out_c_total channels per pixel and the layer writes channels
 * [out_c_off, out_c_off + c_out) of it, leaving the others alone; 0 = y has exactly c_out
 * channels.  Sparse conv layers only (E_UNSUPPORTED for fc, depthwise and stem kernels), and
 * without a residual.
 */
typedef struct {
    const float *scale;
    const float *bias;
    const void *residual;
    int act;         /* cadnn_act */
    int out_dtype;   /* cadnn_dtype of y */
    int out_c_total; /* channels per pixel of y, 0 = c_out */
    int out_c_off;   /* first channel of y this layer writes */
    float residual_scale; /* int8 layers with a residual */
} cadnn_epilogue;

/*
 * cadnn_conv2d - one sparse convolution layer (Section 4: compressed-model layer
 * execution; 1x1 filters run as a sparse-matrix product).
 *   x device NHWC [n][h][w][c_in], h and w must equal the packed in_h, in_w.
 *   y device NHWC [n][h_out][w_out][c_out], h_out = (h + 2 pad - kh) / stride + 1.
 *   y must not alias x.  Pointers must be 16-byte aligned.  ep may be NULL
 *   (no scale, bias, residual or activation; output dtype = layer dtype).
 * Errors: E_ARG, E_SHAPE, E_DTYPE, E_CUDA (launch failure).
 */
cadnn_status cadnn_conv2d(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y,
                          const cadnn_epilogue *ep, void *stream);

/*
 * cadnn_conv2d_workspace / cadnn_weights_workspace_bytes - a layer packed as CADNN_FMT_GROUPED runs in two
 * kernels (Section 1, "computation pattern transformation": structure left by pruning is executed in the form
 * the processor runs fastest): its dense blocks on the tensor cores into int32 sums, then the sparse kernel
 * over the remaining nonzeros, which adds those sums to its own before the requantization (integer sums are
 * exact in any order, so the result is the one the plain sparse layer gives, bit for bit).  The int32 sums
 * live in a workspace the caller provides: device memory of at least cadnn_weights_workspace_bytes(w, n)
 * bytes, 16-byte aligned, used only during the call's kernels (stream order).  Other formats need none
 * (*bytes = 0) and cadnn_conv2d_workspace then equals cadnn_conv2d.  cadnn_conv2d on a GROUPED handle
 * returns E_ARG.
 */
cadnn_status cadnn_weights_workspace_bytes(const cadnn_weights *w, int n, int64_t *bytes);
cadnn_status cadnn_conv2d_workspace(const cadnn_weights *w, const void *x, int n, int h, int wd, void *y,
                                    const cadnn_epilogue *ep, void *workspace, int64_t workspace_bytes, void *stream);
/* How many dense blocks the packer found and how many kept weights they hold (0, 0 for other formats). */
cadnn_status cadnn_weights_block_info(const cadnn_weights *w, int *n_blocks, int64_t *block_nnz);

/*
 * cadnn_conv2d_planar - the same layer on channel-planar activations (Section 4, "Memory
 * layout transformation": data laid out to fit the processor).  This is the layout
 * cadnn_forward uses between the layers of a float network; the call exists so that it can
 * be checked on its own.
 *   x device float [n][c_in][pitch(in_h, in_w)], y device float [n][c_out][pitch(h_out, w_out)]:
 *   a plane is (h + 2) x (w + 2) values, row-major, and consecutive planes are
 *   pitch(h, w) = (h + 2) * (w + 2) rounded up to a multiple of 4 floats apart.  The one-pixel
 *   border and the padding behind a plane MUST be zero in x; the call never writes them in y
 *   (so a y buffer zeroed once stays a valid input for the next layer).
 *   residual (optional) has y's layout.  Float layers with pad <= 1 and k - 1 - pad <= 1 only:
 *   E_UNSUPPORTED otherwise.  Same epilogue, same errors as cadnn_conv2d.
 */
cadnn_status cadnn_conv2d_planar(const cadnn_weights *w, const void *x, int n, void *y, const cadnn_epilogue *ep,
                                 void *stream);

/*
 * cadnn_fc - one sparse fully connected layer: y[b][co] = sum_k W[co][k] x[b][k],
 * same epilogue.  x device [n][k], y device [n][c_out].
 */
cadnn_status cadnn_fc(const cadnn_weights *w, const void *x, int n, void *y,
                      const cadnn_epilogue *ep, void *stream);

/* Glue layers the evaluated networks need (not discussed by the paper).
 * Max pool ignores padded taps; dtype CADNN_F32 or CADNN_S8. */
cadnn_status cadnn_maxpool2d(const void *x, int n, int h, int wd, int c, int k, int stride, int pad,
                             int dtype, void *y, void *stream);
/* Max or average pool (kind 0 / 1) that writes channels [out_c_off, out_c_off + c) of a y with out_c_total
 * channels per pixel (0 = c).  The average pool is float only; taps that fall in the padding count
 * as zeros and the divisor is always k * k. */
cadnn_status cadnn_pool2d(const void *x, int n, int h, int wd, int c, int k, int stride, int pad, int dtype, int kind,
                          void *y, int out_c_total, int out_c_off, void *stream);
/* Global average pool, float: y[b][c] = mean over h*w. */
cadnn_status cadnn_global_avgpool(const float *x, int n, int h, int wd, int c, float *y, void *stream);

/* Whole network (Section 5: single-image inference of a complete model). */
typedef enum { CADNN_OP_CONV = 0, CADNN_OP_FC = 1, CADNN_OP_MAXPOOL = 2, CADNN_OP_GAVGPOOL = 3, CADNN_OP_AVGPOOL = 4 } cadnn_op_kind;

typedef struct {
    int kind;                 /* cadnn_op_kind */
    const cadnn_weights *w;   /* conv / fc; borrowed, must outlive the net */
    int src, dst, res;        /* tensor slots; slot 0 is the network input; res = -1 for none */
    const float *scale;       /* device [c_out] or NULL; borrowed */
    const float *bias;        /* device [c_out] or NULL; borrowed */
    int act;                  /* cadnn_act */
    int out_dtype;            /* cadnn_dtype of the dst slot */
    int pool_k, pool_stride, pool_pad; /* max / average pool only */
    float res_scale;            /* int8 conv with a residual: multiplier of the residual (s_r / s_y) */
    int dst_c_off, dst_c_total; /* conv and pools: the op writes channels [dst_c_off, dst_c_off + c) of a dst slot
                                   that has dst_c_total channels (channel concatenation); 0, 0 = the whole slot */
} cadnn_op;

/*
 * cadnn_net_create - shape-check an op list for input [n][h][w][c] of dtype in_dtype
 * and allocate one device buffer per intermediate slot (owned by the net).  The dst
 * slot of the last op is the network output and is written straight to the pointer
 * given to cadnn_forward.  Every slot is written by exactly one op, after which it is
 * only read - or, for a concatenation, by several ops that each write their own channel
 * window of it (dst_c_total > 0, same in all of them) before any op reads it.
 */
cadnn_status cadnn_net_create(const cadnn_op *ops, int n_ops, int n, int h, int wd, int c, int in_dtype,
                              cadnn_net **out);

/*
 * cadnn_forward - run the network: x device input, y device output of the last op.
 * use_graph != 0 replays a CUDA graph captured on the first call with this (x, y)
 * pair (re-captured when either pointer changes); 0 launches the layers one by one.
 * Float networks made of a dense stem, sparse convs, dense depthwise convs of up to 9 taps,
 * max pools, a global average pool and fc layers keep their intermediate feature maps
 * channel-planar with a zero halo (see cadnn_conv2d_planar); others (int8) keep NHWC
 * (CADNN_NO_PLANAR_DW: networks with depthwise layers too).  CADNN_NO_PLANAR in the
 * environment at cadnn_net_create forces NHWC.
 * Layers after the first are launched as programmatic dependents of their predecessor
 * (their weight fetch overlaps its stores); set CADNN_NO_PDL in the environment before
 * cadnn_net_create to use plain stream order instead (CADNN_NO_PDL_GRAPH: only inside
 * graphs; NHWC networks use them inside graphs only with CADNN_PDL_GRAPH set, they measured
 * slower there).  In a captured graph an op whose result the next op does not read (a residual
 * block's downsample conv) becomes a parallel branch; CADNN_NO_FORK keeps one chain.
 * CADNN_PERSIST=1 in the environment at cadnn_net_create makes a planar network execute its longest
 * run of consecutive sparse convs as ONE persistent cooperative kernel (one thread block per SM, host-
 * planned work items, device-wide barriers between layers, every wait bounded).  Measured it does not beat
 * one tuned kernel per layer (see cadnn_net_persistent_profile), so it is off by default.  The folded
 * scale / bias vectors of those layers are read once, when the net is created, and a map whose only
 * reader is a stride-2 layer inside that kernel is kept as parity planes only (cadnn_net_slot then
 * shows an unwritten buffer).
 * Asynchronous on stream.
 */
cadnn_status cadnn_forward(cadnn_net *net, const void *x, void *y, int use_graph, void *stream);

/*
 * cadnn_forward_host - the same network run from HOST buffers: copies x_host
 * ([n][h][w][c], pinned memory recommended) to a device staging buffer the net owns
 * (allocated on the first call), runs the network, copies the output to y_host and
 * synchronizes stream before returning.  Every wait inside a kernel is bounded; the words in
 * which kernels count waits that ran out are read in stream order behind the output, and
 * CADNN_E_DEVICE_STATUS is returned (y_host is then not to be trusted) when one of them moved
 * since this net last looked.
 */
cadnn_status cadnn_forward_host(cadnn_net *net, const void *x_host, void *y_host, int use_graph, void *stream);

/*
 * cadnn_forward_static - run an op list WITHOUT allocating anything.  (The paper has no
 * counterpart of this call; it exists for deployment.)
 *
 * cadnn_net_create gives every intermediate tensor a cudaMalloc'ed buffer, and doing
 * that again for each new batch size allocates again.  Some callers must not allocate
 * while they run a network: a serving thread on its latency path (cudaMalloc and
 * cudaFree synchronize the whole device and stall every other stream), a process whose
 * device memory has already been handed in full to a framework's caching allocator, or
 * code that meets a batch size it built no cadnn_net for.  This call takes the same op
 * list as cadnn_net_create (weights packed earlier, scale / bias vectors on the device)
 * plus the input shape, and places the intermediate tensors in a fixed device array of
 * CADNN_STATIC_WORKSPACE_BYTES that is part of the library image: every GPU that loads
 * the library holds that much memory until the process exits.  Regions are reused as
 * soon as the last op reading them has been issued.  It calls no cudaMalloc, cudaFree or
 * other allocating routine, on the device or on the host heap; at most 512 ops.
 *
 *   x  device input [n][h][w][c] of in_dtype; y device output of the last op; both the
 *      caller's.  Asynchronous on stream; the layers run in stream order, one by one.
 * Errors: E_ARG / E_SHAPE / E_DTYPE as cadnn_net_create; E_UNSUPPORTED when the
 * intermediate tensors of this input shape do not fit the fixed workspace (or the list
 * has more than 512 ops) - nothing has been launched in that case.
 *
 * The first call on a device looks up the array's device address (with that device
 * current); make that first call before any stream capture.  All calls on a device
 * share the one array, which keeps whatever the previous call left there: nothing in it
 * needs clearing, because every tensor is written in full before it is read, but two
 * calls that overlap on the GPU (different streams, or the same stream from two threads
 * without ordering) race on it, as does a call that overlaps a kernel still reading the
 * previous call's intermediates.  The output y is safe to read once stream has reached
 * the end of the call's work.
 */
#define CADNN_STATIC_WORKSPACE_BYTES (32 << 20)
cadnn_status cadnn_forward_static(const cadnn_op *ops, int n_ops, int n, int h, int wd, int c, int in_dtype,
                                  const void *x, void *y, void *stream);

/* Number of kernel launches one forward issues; bytes of slot memory the net owns. */
cadnn_status cadnn_net_info(const cadnn_net *net, int *n_launches, int64_t *workspace_bytes);

/*
 * How cadnn_forward runs this net: *planar = 1 if the intermediate feature maps are
 * channel-planar (the planar kernels and schedules apply), 0 for NHWC; *persistent_ops =
 * number of consecutive sparse convs executed by the one persistent kernel (0 = none).
 * Either pointer may be NULL.  Host ints.
 */
cadnn_status cadnn_net_layout(const cadnn_net *net, int *planar, int *persistent_ops);

/*
 * Stride-2 layers in a channel-planar net (Section 4: a layer's data layout is chosen for the layer that reads
 * it).  A float conv of stride 2 (3x3 with padding 1, or 1x1) is packed in a second form as well: a stride-1
 * layer over its input split by row and column parity (four planes of ceil(h/2) x ceil(w/2) per channel, each
 * with its zero border; the 1x1 layer reads the (even, even) plane alone).  cadnn_net_create uses that form
 * where the layer writing the input is a sparse conv - whose epilogue then stores the parity planes beside the
 * tensor itself - and where it measured faster at pack time (both forms timed under CADNN_PACK_AUTOTUNE;
 * CADNN_FORCE_PARITY_PLANES=1 in the environment takes it wherever it exists, CADNN_NO_PARITY_PLANES=1 never).
 * The results are those of the plain form up to summation order.  *count = number of ops run this way; their
 * indices go to ops[0 .. min(*count, cap) - 1] (ops may be NULL with cap 0).  cadnn_weights_parity_form: the
 * second form of a layer (*form = NULL if it has none), owned by w and valid as long as w; it answers
 * cadnn_weights_planar_schedule and cadnn_weights_info like any handle and is not to be freed.
 */
cadnn_status cadnn_net_parity_layers(const cadnn_net *net, int *count, int *ops, int cap);
cadnn_status cadnn_weights_parity_form(const cadnn_weights *w, const cadnn_weights **form);

/*
 * Measurement aids for the persistent kernel (E_UNSUPPORTED when the net has none).
 * cadnn_net_persistent_plan: what the host planner chose for op `op` (Section 4, "Optimization
 * parameters selection"): plan[0..11] = bands of 32 positions per tile, bands per unit, filters per
 * group, tiles, groups, staged floats per channel, channels per chunk, chunks per pass, passes,
 * strided addressing, modelled clocks per item, phase.  Host ints.
 * cadnn_net_persistent_profile: with CADNN_PERSIST_PROFILE set in the environment at
 * cadnn_net_create, every launch records SM clock samples; after the last launch this returns,
 * per phase (up to cap; *n_phases receives how many there are), the clocks from the phase's start to
 * the next one's (mean over blocks), the longest / mean clocks a block spent on its own items, and
 * the mean clocks until a block had issued its tile copies / until they had landed.  Any output
 * pointer but n_phases may be NULL.  Synchronizes the device.
 */
cadnn_status cadnn_net_persistent_plan(const cadnn_net *net, int op, int plan[12]);
cadnn_status cadnn_net_persistent_profile(const cadnn_net *net, int cap, float *wall_clk, float *busy_max_clk,
                                          float *busy_mean_clk, float *issued_clk, float *landed_clk, int *n_phases);

/*
 * Measurement aid: time every op on its own.  Each op is captured into a CUDA graph of
 * `reps` back-to-back launches (so the host launch cost stays out) and replayed between
 * a CUDA event pair on stream; ms[n_ops] (host) receives milliseconds per launch.
 * flush_l2 != 0 overwrites a buffer larger than L2 before the timed replay (meaningful
 * with reps = 1); otherwise the graph is replayed once untimed first.  Synchronizes.
 */
cadnn_status cadnn_net_layer_times(cadnn_net *net, const void *x, void *y, int flush_l2, int reps, float *ms,
                                   void *stream);
/* The same for the single op `op`: ms (host) receives one value.  Both return
 * CADNN_E_DEVICE_STATUS like cadnn_forward_host when a kernel's bounded wait ran out. */
cadnn_status cadnn_net_layer_time(cadnn_net *net, int op, const void *x, void *y, int flush_l2, int reps, float *ms,
                                  void *stream);

/*
 * cadnn_device_status - health flags the kernels leave on the current device (the paper has no
 * counterpart: it exists because every wait inside a kernel is bounded).  *copy_timeouts
 * receives how many thread-block waits on an asynchronous copy barrier ran out since the
 * library was loaded; anything but 0 means results of that launch are invalid.  Synchronizes
 * the device.  Errors: E_ARG, E_CUDA.
 */
cadnn_status cadnn_device_status(int *copy_timeouts);

/*
 * cadnn_debug_set_device_status - overwrite the two device words in which kernels count waits
 * that ran out (copy barriers; the persistent kernel's grid barrier).  For tests of the error
 * path only: it lets a test see CADNN_E_DEVICE_STATUS without making any kernel wait.  The
 * paper has no counterpart.  Synchronous.
 */
cadnn_status cadnn_debug_set_device_status(int copy_timeouts, int barrier_timeouts);

/*
 * cadnn_measure_alu_peak - measurement aid: the multiply-add rate the plain ALUs of the current
 * device sustain, in operations per second (a multiply-add counts 2), from a kernel that does
 * nothing but independent chains of fused multiply-adds.  dtype CADNN_F32: the FP32 lanes (FFMA);
 * CADNN_S8: the 32-bit integer multiply-add the int8 kernels issue.  This is the compute-side
 * denominator of the sparse roofline (the paper has no counterpart; its Section 5 reports
 * latencies only).  Allocates and frees a small scratch buffer; runs a few milliseconds;
 * synchronizes stream.
 */
cadnn_status cadnn_measure_alu_peak(int dtype, double *ops_per_second, void *stream);

/* Device pointer and byte size of slot `slot` (for per-layer inspection). */
cadnn_status cadnn_net_slot(const cadnn_net *net, int slot, void **ptr, int64_t *bytes);

void cadnn_net_free(cadnn_net *net);

const char *cadnn_status_str(cadnn_status s);
/* Text of the last CUDA error this thread saw inside the library ("" if none). */
const char *cadnn_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CADNN_H */
