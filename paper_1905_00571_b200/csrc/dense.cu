// Dense layers the pruned networks keep: depthwise k x k convolution (MobileNet),
// fused with BatchNorm fold, residual and activation.
//
// CADNN (arXiv 1905.00571), Section 4, names Depthwise Convolution + BatchNorm +
// Activation as one fused kernel.  A depthwise layer does kh*kw multiply-adds per
// output and is bound by reading the input and writing the output once, so the
// kernel maps lanes to channels (contiguous in NHWC) and keeps the filter taps in
// the tap-major layout the packer wrote.
#include <cstdlib>
#include "cadnn_internal.h"

namespace {

struct DwParams {
    const float *x;
    float *y;
    const float *wt;  // [kh*kw][c]
    const float *scale;
    const float *bias;
    const float *residual;
    int n, h, w, c, h_out, w_out, kh, kw, stride, pad, pad_w, act;
    FastDiv d_cv, d_wout, d_hout;
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
    // the host refuses tensors with 2^31 or more vectors, so 32-bit index arithmetic is exact
    for (unsigned idx = blockIdx.x * blockDim.x + threadIdx.x; idx < (unsigned)total; idx += gridDim.x * blockDim.x) {
        const unsigned pix = fdiv(idx, p.d_cv);
        const int c0 = (int)(idx - pix * cv) * VEC;
        const unsigned r = fdiv(pix, p.d_wout);
        const int ox = (int)(pix - r * p.w_out);
        const unsigned b = fdiv(r, p.d_hout);
        const int oy = (int)(r - b * p.h_out);
        float acc[VEC];
#pragma unroll
        for (int v = 0; v < VEC; ++v) acc[v] = 0.0f;
        for (int ky = 0; ky < p.kh; ++ky) {
            const int iy = oy * p.stride + ky - p.pad;
            if (iy < 0 || iy >= p.h) continue;
            for (int kx = 0; kx < p.kw; ++kx) {
                const int ix = ox * p.stride + kx - p.pad_w;
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


// Dense convolution with very few input channels (the network stem: 7x7 or 3x3, stride 2,
// 3 -> 32/64 channels).  Genuinely dense, so it is register-tiled like a small GEMM: a warp
// owns 32 output columns x 2 output rows and 16 output channels; per tap it reads 2
// activations per lane and 16 weights as four broadcast 16-byte loads, and issues 32 FMAs.
struct StemParams {
    const float *x;
    float *y;
    const float *wt;   // [taps][c_out], taps = (ky*kw + kx)*c_in + ci
    const float *scale;
    const float *bias;
    const float *residual;
    int n, h, w, c_in, c_out, h_out, w_out, kh, kw, stride, pad, pad_w, act;
    int tiles_x, tiles_y, in_rows, in_cols, taps, co_blocks;
    int planar_out, halo;   // write [n][c][h_out + 2 halo][w_out + 2 halo] instead of NHWC
};

const int kStemCo = 16;      // output channels per warp
const int kStemRows = 4;     // output rows per block (2 warps down x 2 rows per lane)
const int kStemCoBlock = 64; // output channels per block (4 warps across channels)

__global__ void __launch_bounds__(256) stem_kernel(const StemParams p)
{
    extern __shared__ __align__(16) float sm[];
    float *sW = sm;                                   // [taps][64]
    float *sIn = sm + (size_t)p.taps * kStemCoBlock;  // [in_rows][in_cols][c_in]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int b = blockIdx.x;
    const int cb = b % p.co_blocks; b /= p.co_blocks;
    const int tx = b % p.tiles_x; b /= p.tiles_x;
    const int ty = b % p.tiles_y;
    const int img = b / p.tiles_y;
    const int ox0 = tx * 32, oy0 = ty * kStemRows, co0 = cb * kStemCoBlock;

    // weights of this block's 64 channels (static data: before the grid-dependency wait)
    for (int i = tid; i < p.taps * kStemCoBlock; i += blockDim.x) {
        const int t = i / kStemCoBlock, c = i - t * kStemCoBlock;
        sW[i] = (co0 + c < p.c_out) ? p.wt[(size_t)t * p.c_out + co0 + c] : 0.0f;
    }
    grid_dep_wait();
    grid_dep_trigger();
    const int iy0 = oy0 * p.stride - p.pad, ix0 = ox0 * p.stride - p.pad_w;
    const int row_words = p.in_cols * p.c_in;
    for (int i = tid; i < p.in_rows * row_words; i += blockDim.x) {
        const int r = i / row_words, rem = i - r * row_words;
        const int col = rem / p.c_in, ci = rem - col * p.c_in;
        const int iy = iy0 + r, ix = ix0 + col;
        float v = 0.0f;
        if (iy >= 0 && iy < p.h && ix >= 0 && ix < p.w) v = p.x[(((size_t)img * p.h + iy) * p.w + ix) * p.c_in + ci];
        sIn[i] = v;
    }
    __syncthreads();

    const int wc = warp & 3, wr = warp >> 2;          // channel group, row pair
    const int ly = wr * 2;                            // first of this lane's two output rows
    float acc0[kStemCo], acc1[kStemCo];
#pragma unroll
    for (int c = 0; c < kStemCo; ++c) acc0[c] = acc1[c] = 0.0f;
    const float *w_base = sW + wc * kStemCo;
    const float *in0 = sIn + ((ly * p.stride) * p.in_cols + lane * p.stride) * p.c_in;
    const float *in1 = in0 + p.stride * row_words;
    int t = 0;
    for (int ky = 0; ky < p.kh; ++ky) {
        const float *r0 = in0 + ky * row_words, *r1 = in1 + ky * row_words;
        for (int k = 0; k < p.kw * p.c_in; ++k, ++t) {
            const float a0 = r0[k], a1 = r1[k];
            const float4 *wq = reinterpret_cast<const float4 *>(w_base + t * kStemCoBlock);
#pragma unroll
            for (int q = 0; q < kStemCo / 4; ++q) {
                const float4 wv = wq[q];
                acc0[4 * q + 0] = fmaf(a0, wv.x, acc0[4 * q + 0]);
                acc0[4 * q + 1] = fmaf(a0, wv.y, acc0[4 * q + 1]);
                acc0[4 * q + 2] = fmaf(a0, wv.z, acc0[4 * q + 2]);
                acc0[4 * q + 3] = fmaf(a0, wv.w, acc0[4 * q + 3]);
                acc1[4 * q + 0] = fmaf(a1, wv.x, acc1[4 * q + 0]);
                acc1[4 * q + 1] = fmaf(a1, wv.y, acc1[4 * q + 1]);
                acc1[4 * q + 2] = fmaf(a1, wv.z, acc1[4 * q + 2]);
                acc1[4 * q + 3] = fmaf(a1, wv.w, acc1[4 * q + 3]);
            }
        }
    }

    const int ox = ox0 + lane;
    const int cbase = co0 + wc * kStemCo;
    if (ox < p.w_out) {
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            const int oy = oy0 + ly + rr;
            if (oy >= p.h_out) continue;
            const float *acc = rr ? acc1 : acc0;
            const size_t o = (((size_t)img * p.h_out + oy) * p.w_out + ox) * p.c_out + cbase;
            const int wp = p.w_out + 2 * p.halo;
            const size_t plane = (size_t)planar_pitch(p.h_out, p.w_out);
            const size_t opl = (size_t)img * p.c_out * plane + (size_t)(oy + p.halo) * wp + ox + p.halo;
#pragma unroll
            for (int c = 0; c < kStemCo; ++c) {
                const int co = cbase + c;
                if (co >= p.c_out) break;
                float z = fmaf(acc[c], p.scale ? p.scale[co] : 1.0f, p.bias ? p.bias[co] : 0.0f);
                if (p.planar_out) {
                    p.y[opl + (size_t)co * plane] = dw_act(z, p.act);   // lanes are consecutive columns: contiguous
                } else {
                    if (p.residual) z += p.residual[o + c];
                    p.y[o + c] = dw_act(z, p.act);
                }
            }
        }
    }
}

// asynchronous global -> shared copies (4 bytes with zero fill when !ok, 16 bytes)
__device__ __forceinline__ void stem_cp4(unsigned dst, const float *src, bool ok)
{
    const int sz = ok ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void stem_cp16(unsigned dst, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}

// The same register tile specialised at compile time for the stems that occur (7x7x3 and 3x3x3 at
// stride 2): a block is 4 warps of 16 channels (or 8 of 8) on ONE pair of output rows, so a 112 x 112 map
// gives 224 blocks (the generic kernel's 112 leave a quarter of the SMs idle); the staged input
// is split by channel and by column parity, so that lanes on consecutive output columns read
// consecutive words whatever the tap (at stride 2 the interleaved layout is a 2-way bank
// conflict); weights and input rows are copied without any division; the taps of one kernel
// row are fully unrolled with constant offsets.
template <int KH, int KW, int CIN, int CPW>
__global__ void __launch_bounds__(32 * (kStemCoBlock / CPW)) stem2_kernel(const StemParams p)
{
    constexpr int NW = kStemCoBlock / CPW, NT = 32 * NW;   // warps (CPW channels each) and threads per block
    constexpr int STRIDE = 2;
    constexpr int IN_ROWS = STRIDE + KH;            // two output rows
    constexpr int IN_COLS = 31 * STRIDE + KW;
    constexpr int HALF = (IN_COLS + 1) / 2 + 1;     // words per (row, channel, parity); odd or even does not matter: lanes differ in the last index only
    constexpr int ROW_WORDS = CIN * 2 * HALF;
    constexpr int TAPS = KH * KW * CIN;
    extern __shared__ __align__(16) float sm[];
    float *sW = sm;                                  // [TAPS][64]
    float *sIn = sm + TAPS * kStemCoBlock;           // [IN_ROWS][CIN][2][HALF]
    const int tid = threadIdx.x, lane = tid & 31, wc = tid >> 5;
    int b = blockIdx.x;
    const int cb = b % p.co_blocks; b /= p.co_blocks;
    const int tx = b % p.tiles_x; b /= p.tiles_x;
    const int ty = b % p.tiles_y;
    const int img = b / p.tiles_y;
    const int ox0 = tx * 32, oy0 = ty * 2, co0 = cb * kStemCoBlock;

    // Staging is all asynchronous copies: every request is in flight before the first one is
    // waited for (a loop of load-then-store would pay one L2 round trip per iteration).
    // Weights of this block's 64 channels first (static data: before the grid-dependency wait).
    const unsigned sW32 = (unsigned)__cvta_generic_to_shared(sW), sIn32 = (unsigned)__cvta_generic_to_shared(sIn);
    if ((p.c_out & 3) == 0 && co0 + kStemCoBlock <= p.c_out) {
        for (int i = tid; i < TAPS * (kStemCoBlock / 4); i += NT) {
            const int t = i >> 4, c4 = i & 15;
            stem_cp16(sW32 + i * 16, p.wt + (size_t)t * p.c_out + co0 + c4 * 4);
        }
    } else {
        for (int i = tid; i < TAPS * kStemCoBlock; i += NT) {
            const int t = i >> 6, c = i & 63;
            const bool ok = co0 + c < p.c_out;
            stem_cp4(sW32 + i * 4, ok ? p.wt + (size_t)t * p.c_out + co0 + c : p.wt, ok);
        }
    }
    grid_dep_wait();
    grid_dep_trigger();
    const int iy0 = oy0 * STRIDE - p.pad, ix0 = ox0 * STRIDE - p.pad_w;
    // input rows: IN_COLS * CIN consecutive floats of the NHWC image each; warp r mod NW takes row r
    for (int r = wc; r < IN_ROWS; r += NW) {
        const int iy = iy0 + r;
        const bool row_ok = iy >= 0 && iy < p.h;
        const float *src = p.x + (((size_t)img * p.h + (row_ok ? iy : 0)) * p.w) * CIN;
        const unsigned dst = sIn32 + r * ROW_WORDS * 4;
        int col = 0, ci = lane;      // element e = col * CIN + ci, starting at e = lane
        while (ci >= CIN) { ci -= CIN; ++col; }
#pragma unroll
        for (int e0 = 0; e0 < IN_COLS * CIN; e0 += 32) {
            if (e0 + lane < IN_COLS * CIN) {
                const int ix = ix0 + col;
                const bool ok = row_ok && ix >= 0 && ix < p.w;
                stem_cp4(dst + ((ci * 2 + (col & 1)) * HALF + (col >> 1)) * 4, ok ? src + (size_t)ix * CIN + ci : p.x, ok);
            }
            ci += 32 % CIN;
            col += 32 / CIN;
            if (ci >= CIN) { ci -= CIN; ++col; }
        }
    }
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();

    float acc0[CPW], acc1[CPW];
#pragma unroll
    for (int c = 0; c < CPW; ++c) acc0[c] = acc1[c] = 0.0f;
    const float *w_base = sW + wc * CPW;
    const float *in0 = sIn + lane;
#pragma unroll 1
    for (int ky = 0; ky < KH; ++ky) {
        const float *r0 = in0 + ky * ROW_WORDS;
        const float *r1 = r0 + STRIDE * ROW_WORDS;
        const float *wk = w_base + ky * (KW * CIN) * kStemCoBlock;
#pragma unroll
        for (int kx = 0; kx < KW; ++kx)
#pragma unroll
            for (int ci = 0; ci < CIN; ++ci) {
                const int off = (ci * 2 + (kx & 1)) * HALF + (kx >> 1);
                const float a0 = r0[off], a1 = r1[off];
                const float4 *wq = reinterpret_cast<const float4 *>(wk + (kx * CIN + ci) * kStemCoBlock);
#pragma unroll
                for (int q = 0; q < CPW / 4; ++q) {
                    const float4 wv = wq[q];
                    acc0[4 * q + 0] = fmaf(a0, wv.x, acc0[4 * q + 0]);
                    acc0[4 * q + 1] = fmaf(a0, wv.y, acc0[4 * q + 1]);
                    acc0[4 * q + 2] = fmaf(a0, wv.z, acc0[4 * q + 2]);
                    acc0[4 * q + 3] = fmaf(a0, wv.w, acc0[4 * q + 3]);
                    acc1[4 * q + 0] = fmaf(a1, wv.x, acc1[4 * q + 0]);
                    acc1[4 * q + 1] = fmaf(a1, wv.y, acc1[4 * q + 1]);
                    acc1[4 * q + 2] = fmaf(a1, wv.z, acc1[4 * q + 2]);
                    acc1[4 * q + 3] = fmaf(a1, wv.w, acc1[4 * q + 3]);
                }
            }
    }

    const int ox = ox0 + lane;
    const int cbase = co0 + wc * CPW;
    if (ox < p.w_out) {
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            const int oy = oy0 + rr;
            if (oy >= p.h_out) continue;
            const float *acc = rr ? acc1 : acc0;
            const size_t o = (((size_t)img * p.h_out + oy) * p.w_out + ox) * p.c_out + cbase;
            const int wp = p.w_out + 2 * p.halo;
            const size_t plane = (size_t)planar_pitch(p.h_out, p.w_out);
            const size_t opl = (size_t)img * p.c_out * plane + (size_t)(oy + p.halo) * wp + ox + p.halo;
#pragma unroll
            for (int c = 0; c < CPW; ++c) {
                const int co = cbase + c;
                if (co >= p.c_out) break;
                float z = fmaf(acc[c], p.scale ? __ldg(p.scale + co) : 1.0f, p.bias ? __ldg(p.bias + co) : 0.0f);
                if (p.planar_out) {
                    p.y[opl + (size_t)co * plane] = dw_act(z, p.act);   // lanes are consecutive columns: contiguous
                } else {
                    if (p.residual) z += p.residual[o + c];
                    p.y[o + c] = dw_act(z, p.act);
                }
            }
        }
    }
}

template <int KH, int KW, int CIN>
cadnn_status launch_stem2(StemParams &p, int n, bool pdl, cudaStream_t st)
{
    constexpr int IN_ROWS = 2 + KH, IN_COLS = 31 * 2 + KW, HALF = (IN_COLS + 1) / 2 + 1;
    p.tiles_y = (p.h_out + 1) / 2;
    long long blocks = (long long)n * p.tiles_y * p.tiles_x * p.co_blocks;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    const size_t smem = ((size_t)KH * KW * CIN * kStemCoBlock + (size_t)IN_ROWS * CIN * 2 * HALF) * 4;
    // few blocks (one image): 8 warps of 8 channels keep more warps per scheduler than 4 of 16; many blocks: the
    // larger register tile issues fewer shared-memory loads per multiply-add
    static SmemLimit lim8, lim16;
    if (blocks <= 4 * 148) {   // up to four blocks per multiprocessor
        if (smem > 48 * 1024) {
            cadnn_status rs = raise_smem_limit((const void *)stem2_kernel<KH, KW, CIN, 8>, (int)smem, &lim8);
            if (rs != CADNN_OK) return rs;
        }
        return launch_kernel(stem2_kernel<KH, KW, CIN, 8>, (int)blocks, 256, smem, pdl, st, p);
    }
    if (smem > 48 * 1024) {
        cadnn_status rs = raise_smem_limit((const void *)stem2_kernel<KH, KW, CIN, 16>, (int)smem, &lim16);
        if (rs != CADNN_OK) return rs;
    }
    return launch_kernel(stem2_kernel<KH, KW, CIN, 16>, (int)blocks, 128, smem, pdl, st, p);
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
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.pad_w = d.pad_w; p.act = ep.act;
    const bool v4 = d.c_out % 4 == 0;
    long long total = (long long)n * w->h_out * w->w_out * (v4 ? d.c_out / 4 : d.c_out);
    if (total <= 0) return CADNN_OK;
    if (total >= (1LL << 31)) return CADNN_E_UNSUPPORTED;
    p.d_cv = make_fastdiv(v4 ? d.c_out / 4 : d.c_out);
    p.d_wout = make_fastdiv(w->w_out);
    p.d_hout = make_fastdiv(w->h_out);
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 64) blocks = 148LL * 64;
    if (v4) return launch_kernel(dw_kernel<4>, (int)blocks, 256, 0, ep.pdl, st, p);
    return launch_kernel(dw_kernel<1>, (int)blocks, 256, 0, ep.pdl, st, p);
}

cadnn_status launch_dense_smallc(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                 cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    StemParams p;
    p.x = (const float *)x; p.y = (float *)y; p.wt = w->d_dense;
    p.scale = ep.scale; p.bias = ep.bias; p.residual = (const float *)ep.residual;
    p.n = n; p.h = d.in_h; p.w = d.in_w; p.c_in = d.c_in; p.c_out = d.c_out;
    p.h_out = w->h_out; p.w_out = w->w_out; p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad; p.pad_w = d.pad_w;
    p.act = ep.act;
    p.planar_out = ep.planar_out ? 1 : 0;
    p.halo = kPlanarHalo;
    if (ep.planar_out && ep.residual) return CADNN_E_UNSUPPORTED;
    p.tiles_x = (w->w_out + 31) / 32;
    p.tiles_y = (w->h_out + kStemRows - 1) / kStemRows;
    p.in_rows = (kStemRows - 1) * d.stride + d.kh;
    p.in_cols = 31 * d.stride + d.kw;
    p.taps = d.kh * d.kw * d.c_in;
    p.co_blocks = (d.c_out + kStemCoBlock - 1) / kStemCoBlock;
    if (d.stride == 2 && d.c_in == 3 && getenv("CADNN_GENERIC_STEM") == nullptr) {
        if (d.kh == 7 && d.kw == 7) return launch_stem2<7, 7, 3>(p, n, ep.pdl, st);
        if (d.kh == 3 && d.kw == 3) return launch_stem2<3, 3, 3>(p, n, ep.pdl, st);
    }
    long long blocks = (long long)n * p.tiles_y * p.tiles_x * p.co_blocks;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    size_t smem = ((size_t)p.taps * kStemCoBlock + (size_t)p.in_rows * p.in_cols * d.c_in) * 4;
    static SmemLimit lim;
    if (smem > 48 * 1024) {
        if (smem > 200 * 1024) return CADNN_E_UNSUPPORTED;
        cadnn_status rs = raise_smem_limit((const void *)stem_kernel, (int)smem, &lim);
        if (rs != CADNN_OK) return rs;
    }
    return launch_kernel(stem_kernel, (int)blocks, 256, smem, ep.pdl, st, p);
}
