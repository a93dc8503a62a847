// Sparse convolution kernels (k x k with halo tiles, and 1x1 as a sparse-matrix
// product over flat pixel ranges), float and int8, with the fused epilogue.
//
// CADNN (arXiv 1905.00571), Section 4: the compressed layer is executed as one
// fused kernel (Conv + BatchNorm + Activation), 1x1 filters are run as a matrix
// product, and filter elements are not reloaded redundantly.  Here:
//   * a thread block owns a tile of output pixels and a block of G filters;
//   * the input tile is staged in shared memory chunk by chunk of input channels,
//     pixel-major with an odd word pitch per pixel, so that the lanes of a warp
//     (consecutive output pixels) read 32 distinct banks for any nonzero;
//   * each stored nonzero is (value, offset into the staged tile); a warp walks
//     the nonzeros of its filters, broadcasts one nonzero to all lanes and issues
//     T multiply-adds per lane, the accumulators living in registers for the
//     whole layer (each weight is read once per block and chunk);
//   * results go through shared memory so that stores to NHWC are contiguous
//     over the block's G output channels, with the epilogue applied on the way.
#include "cadnn_internal.h"

namespace {

struct SconvParams {
    const void *x;
    void *y;
    const void *vals;
    const uint16_t *offs;
    const int32_t *ptr;
    const int32_t *perm;
    const float *scale;
    const float *bias;
    const void *residual;
    int n, h, w, c_in, h_out, w_out, c_out;
    int kh, kw, stride, pad;
    int TH, TW, pitch, IH_t, IW_t, CIc, PP, n_chunks, G, c_pad, n_groups;
    int tiles_y, tiles_x;
    long long P;  // total output pixels (linear mode)
    int tile_words, max_entries;
    int act, out_dtype, linear;
};

template <typename XT> struct AccOf { typedef float type; };
template <> struct AccOf<int8_t> { typedef int type; };

__device__ __forceinline__ float act_f32(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

// float layer: BatchNorm fold, residual, activation
__device__ __forceinline__ float finish_f32(float acc, float sc, float bi, bool has_res, float res, int act)
{
    float z = fmaf(acc, sc, bi);
    if (has_res) z += res;
    return act_f32(z, act);
}

// int8 layer: one fused multiply-add on the converted accumulator, ReLU
__device__ __forceinline__ float requant_f32(int acc, float m, float b, int act)
{
    float t = __fmaf_rn(__int2float_rn(acc), m, b);
    if (act == CADNN_ACT_RELU) t = t > 0.0f ? t : 0.0f;
    return t;
}
__device__ __forceinline__ int requant_s8(int acc, float m, float b, int act)
{
    float t = requant_f32(acc, m, b, act);
    t = fminf(fmaxf(t, -127.0f), 127.0f);
    return __float2int_rn(t);
}

template <typename XT, int T, int RPW>
__global__ void __launch_bounds__(256) sconv_kernel(const SconvParams p)
{
    typedef typename AccOf<XT>::type AT;
    extern __shared__ __align__(16) unsigned char smem[];
    AT *sX = reinterpret_cast<AT *>(smem);
    uint2 *sW = reinterpret_cast<uint2 *>(smem + (size_t)p.tile_words * 4);
    int *sPtr = reinterpret_cast<int *>(sW + p.max_entries);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grp = blockIdx.x % p.n_groups;
    int tile = blockIdx.x / p.n_groups;
    const int G = p.G;

    // tile origin
    int img = 0, oy0 = 0, ox0 = 0;
    long long p0 = 0;
    if (p.linear) {
        p0 = (long long)tile * (32 * T);
    } else {
        int tx = tile % p.tiles_x;
        tile /= p.tiles_x;
        int ty = tile % p.tiles_y;
        img = tile / p.tiles_y;
        oy0 = ty * p.TH;
        ox0 = tx * p.TW;
    }

    // byte offset, inside the staged tile, of the top-left tap of each of this lane's pixels
    int pixoff[T];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        int q = lane + 32 * t;
        if (p.linear) {
            pixoff[t] = q * p.PP * 4;
        } else {
            int ly = q / p.TW, lx = q - ly * p.TW;
            bool ok = (ly < p.TH) && (oy0 + ly < p.h_out) && (ox0 + lx < p.w_out);
            pixoff[t] = ok ? ((ly * p.stride) * p.pitch + lx * p.stride) * p.PP * 4 : 0;
        }
    }

    AT acc[RPW][T];
#pragma unroll
    for (int j = 0; j < RPW; ++j)
#pragma unroll
        for (int t = 0; t < T; ++t) acc[j][t] = 0;

    const XT *xg = reinterpret_cast<const XT *>(p.x);
    const bool vec4 = (p.c_in % 4 == 0) && (p.CIc % 4 == 0);

    for (int c = 0; c < p.n_chunks; ++c) {
        __syncthreads();  // the previous chunk's tile and weights are no longer read
        const int c0 = c * p.CIc;

        // ---- stage this block's nonzeros of the chunk: (value, byte offset) ----
        {
            const int32_t *pp = p.ptr + (size_t)c * (p.c_pad + 1) + grp * G;
            const int gbeg = pp[0];
            const int cnt = pp[G] - gbeg;
            if (tid <= G) sPtr[tid] = pp[tid] - gbeg;
            for (int e = tid; e < cnt; e += blockDim.x) {
                uint2 ent;
                if (sizeof(XT) == 1) ent.x = (unsigned)(int)reinterpret_cast<const int8_t *>(p.vals)[gbeg + e];
                else ent.x = reinterpret_cast<const unsigned *>(p.vals)[gbeg + e];
                ent.y = (unsigned)p.offs[gbeg + e] * 4u;
                sW[e] = ent;
            }
        }

        // ---- stage the activation tile: pixel-major, PP words per pixel ----
        if (p.linear) {
            const int npx = 32 * T;
            if (vec4) {
                const int cv = p.CIc >> 2;
                for (int idx = tid; idx < npx * cv; idx += blockDim.x) {
                    int q = idx / cv, v = idx - q * cv;
                    long long op = p0 + q;
                    int ci = c0 + v * 4;
                    AT a0 = 0, a1 = 0, a2 = 0, a3 = 0;
                    if (op < p.P && ci < p.c_in) {
                        long long ip = op;
                        if (p.stride != 1) {
                            int ox = (int)(op % p.w_out);
                            long long r = op / p.w_out;
                            int oy = (int)(r % p.h_out);
                            long long b = r / p.h_out;
                            ip = (b * p.h + (long long)oy * p.stride) * p.w + (long long)ox * p.stride;
                        }
                        const XT *src = xg + ip * p.c_in + ci;
                        if (sizeof(XT) == 4) {
                            float4 f = *reinterpret_cast<const float4 *>(src);
                            a0 = f.x; a1 = f.y; a2 = f.z; a3 = f.w;
                        } else {
                            char4 q4 = *reinterpret_cast<const char4 *>(src);
                            a0 = q4.x; a1 = q4.y; a2 = q4.z; a3 = q4.w;
                        }
                    }
                    AT *dst = sX + q * p.PP + v * 4;
                    dst[0] = a0; dst[1] = a1; dst[2] = a2; dst[3] = a3;
                }
            } else {
                for (int idx = tid; idx < npx * p.CIc; idx += blockDim.x) {
                    int q = idx / p.CIc, cl = idx - q * p.CIc;
                    long long op = p0 + q;
                    int ci = c0 + cl;
                    AT a = 0;
                    if (op < p.P && ci < p.c_in) {
                        long long ip = op;
                        if (p.stride != 1) {
                            int ox = (int)(op % p.w_out);
                            long long r = op / p.w_out;
                            int oy = (int)(r % p.h_out);
                            long long b = r / p.h_out;
                            ip = (b * p.h + (long long)oy * p.stride) * p.w + (long long)ox * p.stride;
                        }
                        a = (AT)xg[ip * p.c_in + ci];
                    }
                    sX[q * p.PP + cl] = a;
                }
            }
        } else {
            const int iy0 = oy0 * p.stride - p.pad, ix0 = ox0 * p.stride - p.pad;
            const XT *ximg = xg + (size_t)img * p.h * p.w * p.c_in;
            if (vec4) {
                const int cv = p.CIc >> 2;
                const int total = p.IH_t * p.IW_t * cv;
                for (int idx = tid; idx < total; idx += blockDim.x) {
                    int pix = idx / cv, v = idx - pix * cv;
                    int r = pix / p.IW_t, col = pix - r * p.IW_t;
                    int iy = iy0 + r, ix = ix0 + col, ci = c0 + v * 4;
                    AT a0 = 0, a1 = 0, a2 = 0, a3 = 0;
                    if (iy >= 0 && iy < p.h && ix >= 0 && ix < p.w && ci < p.c_in) {
                        const XT *src = ximg + ((size_t)iy * p.w + ix) * p.c_in + ci;
                        if (sizeof(XT) == 4) {
                            float4 f = *reinterpret_cast<const float4 *>(src);
                            a0 = f.x; a1 = f.y; a2 = f.z; a3 = f.w;
                        } else {
                            char4 q4 = *reinterpret_cast<const char4 *>(src);
                            a0 = q4.x; a1 = q4.y; a2 = q4.z; a3 = q4.w;
                        }
                    }
                    AT *dst = sX + (r * p.pitch + col) * p.PP + v * 4;
                    dst[0] = a0; dst[1] = a1; dst[2] = a2; dst[3] = a3;
                }
            } else {
                const int total = p.IH_t * p.IW_t * p.CIc;
                for (int idx = tid; idx < total; idx += blockDim.x) {
                    int pix = idx / p.CIc, cl = idx - pix * p.CIc;
                    int r = pix / p.IW_t, col = pix - r * p.IW_t;
                    int iy = iy0 + r, ix = ix0 + col, ci = c0 + cl;
                    AT a = 0;
                    if (iy >= 0 && iy < p.h && ix >= 0 && ix < p.w && ci < p.c_in)
                        a = (AT)ximg[((size_t)iy * p.w + ix) * p.c_in + ci];
                    sX[(r * p.pitch + col) * p.PP + cl] = a;
                }
            }
        }
        __syncthreads();

        // ---- walk the nonzeros of this warp's filters ----
        const unsigned char *sXb = reinterpret_cast<const unsigned char *>(sX);
#pragma unroll
        for (int j = 0; j < RPW; ++j) {
            const int row = warp * RPW + j;
            const int beg = sPtr[row], end = sPtr[row + 1];
#pragma unroll 4
            for (int e = beg; e < end; ++e) {
                const uint2 ent = sW[e];
                AT wv;
                if (sizeof(XT) == 4) wv = (AT)__uint_as_float(ent.x);
                else wv = (AT)(int)ent.x;
                const unsigned char *base = sXb + ent.y;
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    AT xv = *reinterpret_cast<const AT *>(base + pixoff[t]);
                    acc[j][t] += wv * xv;
                }
            }
        }
    }

    // ---- results to shared memory, [pixel][G + 1], at the original channel position ----
    __syncthreads();
    AT *sOut = reinterpret_cast<AT *>(smem);
    const int op = G + 1;
#pragma unroll
    for (int j = 0; j < RPW; ++j) {
        int co = p.perm[grp * G + warp * RPW + j];
        if (co >= 0) {
            int lc = co - grp * G;
#pragma unroll
            for (int t = 0; t < T; ++t) sOut[(lane + 32 * t) * op + lc] = acc[j][t];
        }
    }
    __syncthreads();

    // ---- epilogue and contiguous NHWC stores ----
    const int co_base = grp * G;
    const int gw = min(G, p.c_out - co_base);  // real channels in this block
    const int npx = 32 * T;
    const bool has_res = p.residual != nullptr;
    for (int idx = tid; idx < npx * gw; idx += blockDim.x) {
        int q = idx / gw, lc = idx - q * gw;
        long long opix;
        if (p.linear) {
            opix = p0 + q;
            if (opix >= p.P) continue;
        } else {
            int ly = q / p.TW, lx = q - ly * p.TW;
            int oy = oy0 + ly, ox = ox0 + lx;
            if (ly >= p.TH || oy >= p.h_out || ox >= p.w_out) continue;
            opix = ((long long)img * p.h_out + oy) * p.w_out + ox;
        }
        const int co = co_base + lc;
        const size_t oi = (size_t)opix * p.c_out + co;
        const AT a = sOut[q * op + lc];
        const float sc = p.scale ? p.scale[co] : 1.0f;
        const float bi = p.bias ? p.bias[co] : 0.0f;
        if (sizeof(XT) == 4) {
            float r = has_res ? reinterpret_cast<const float *>(p.residual)[oi] : 0.0f;
            reinterpret_cast<float *>(p.y)[oi] = finish_f32((float)a, sc, bi, has_res, r, p.act);
        } else {
            if (p.out_dtype == CADNN_S32) reinterpret_cast<int *>(p.y)[oi] = (int)a;
            else if (p.out_dtype == CADNN_F32) reinterpret_cast<float *>(p.y)[oi] = requant_f32((int)a, sc, bi, p.act);
            else reinterpret_cast<int8_t *>(p.y)[oi] = (int8_t)requant_s8((int)a, sc, bi, p.act);
        }
    }
}

template <typename XT, int T, int RPW>
cadnn_status launch_one(const SconvParams &p, int blocks, int smem, cudaStream_t st)
{
    auto kern = sconv_kernel<XT, T, RPW>;
    static int smem_allowed = 48 * 1024;  // raised once per instantiation, as layers need it
    if (smem > smem_allowed) {
        CADNN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        smem_allowed = smem;
    }
    kern<<<blocks, 256, smem, st>>>(p);
    CADNN_CUDA_TRY(cudaGetLastError());
    return CADNN_OK;
}

template <typename XT, int T>
cadnn_status launch_rpw(const SconvParams &p, int rpw, int blocks, int smem, cudaStream_t st)
{
    switch (rpw) {
        case 1: return launch_one<XT, T, 1>(p, blocks, smem, st);
        case 2: return launch_one<XT, T, 2>(p, blocks, smem, st);
        case 4: return launch_one<XT, T, 4>(p, blocks, smem, st);
    }
    return CADNN_E_UNSUPPORTED;
}

template <typename XT>
cadnn_status launch_T(const SconvParams &p, int T, int rpw, int blocks, int smem, cudaStream_t st)
{
    switch (T) {
        case 1: return launch_rpw<XT, 1>(p, rpw, blocks, smem, st);
        case 2: return launch_rpw<XT, 2>(p, rpw, blocks, smem, st);
        case 4: return launch_rpw<XT, 4>(p, rpw, blocks, smem, st);
        case 7: return launch_rpw<XT, 7>(p, rpw, blocks, smem, st);
        case 8: return launch_rpw<XT, 8>(p, rpw, blocks, smem, st);
    }
    return CADNN_E_UNSUPPORTED;
}

}  // namespace

cadnn_status launch_sconv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                          cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    const Schedule &s = w->s;
    SconvParams p;
    p.x = x;
    p.y = y;
    p.vals = w->d_vals;
    p.offs = w->d_offs;
    p.ptr = w->d_ptr;
    p.perm = w->d_perm;
    p.scale = ep.scale;
    p.bias = ep.bias;
    p.residual = ep.residual;
    p.n = n; p.h = d.in_h; p.w = d.in_w; p.c_in = d.c_in;
    p.h_out = w->h_out; p.w_out = w->w_out; p.c_out = d.c_out;
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.pad = d.pad;
    p.TH = s.TH; p.TW = s.TW; p.pitch = s.pitch; p.IH_t = s.IH_t; p.IW_t = s.IW_t;
    p.CIc = s.CIc; p.PP = s.PP; p.n_chunks = s.n_chunks; p.G = s.G; p.c_pad = w->c_pad; p.n_groups = s.n_groups;
    p.linear = s.kind == KK_SCONV_LINEAR;
    p.P = (long long)n * w->h_out * w->w_out;
    p.tile_words = s.tile_words;
    p.max_entries = s.max_entries;
    p.act = ep.act;
    p.out_dtype = ep.out_dtype;
    long long tiles;
    if (p.linear) {
        p.tiles_x = p.tiles_y = 1;
        tiles = (p.P + 32 * s.T - 1) / (32 * s.T);
    } else {
        p.tiles_y = (w->h_out + s.TH - 1) / s.TH;
        p.tiles_x = (w->w_out + s.TW - 1) / s.TW;
        tiles = (long long)n * p.tiles_y * p.tiles_x;
    }
    long long blocks = tiles * s.n_groups;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    if (d.dtype == CADNN_S8) return launch_T<int8_t>(p, s.T, s.RPW, (int)blocks, s.smem_bytes, st);
    return launch_T<float>(p, s.T, s.RPW, (int)blocks, s.smem_bytes, st);
}
