// Sparse convolution kernels (k x k with halo tiles, and 1x1 as a sparse-matrix
// product over flat pixel ranges), float and int8, with the fused epilogue.
//
// CADNN (arXiv 1905.00571), Section 4: the compressed layer is executed as one
// fused kernel (Conv + BatchNorm + Activation), 1x1 filters are run as a matrix
// product, and filter elements are not reloaded redundantly.  Here:
//   * a thread block owns a tile of output pixels and a block of G filters; the
//     reduction over input channels can additionally be split over the blocks of a
//     thread-block cluster, whose partial sums meet in distributed shared memory;
//   * the input tile is staged in shared memory chunk by chunk of input channels
//     with cp.async, pixel-major with an odd word pitch per pixel, so that the lanes
//     of a warp (one band of up to 32 output pixels) read 32 distinct banks for any
//     nonzero; stride-2 layers stage even and odd columns in separate planes for the
//     same reason;
//   * each stored nonzero is (value, byte offset into the staged tile); a warp
//     walks the nonzeros of its filters two at a time, broadcasts them to all
//     lanes and issues T multiply-adds per lane and nonzero, the accumulators
//     living in registers for the whole layer;
//   * results go through shared memory so that stores to NHWC are contiguous
//     over the block's G output channels, with the epilogue applied on the way;
//   * weights, tables and epilogue vectors are fetched before the grid-dependency
//     wait, so that inside a network they overlap the previous layer's tail.
#include <algorithm>
#include <cooperative_groups.h>
#include "cadnn_internal.h"

namespace cg = cooperative_groups;

namespace {

struct SconvParams {
    const void *x;
    void *y;
    const uint32_t *ent;
    const int32_t *perm;
    const float *scale;
    const float *bias;
    const void *residual;
    int n, h, w, c_in, h_out, w_out, c_out;
    int stride, pad, pad_w;
    float res_scale;  // int8 layers: multiplier of the int8 residual
    const int *acc_in; // int8 layers: int32 sums [pixels][c_out] added to the accumulators (tensor-core blocks), or null
    int ldc, c_off;   // channels per output pixel of y and first channel written (a window of a wider tensor for concatenations)
    int BW, RB, TBX, TBY, TH, TW, pitch, half, IH_t, IW_t;
    int CIc, PPb, n_chunks, G, n_groups, stages, esz;
    int ksplit;   // thread blocks per cluster; each takes a contiguous range of the channel chunks
    int tiles_y, tiles_x;
    long long P;  // total output pixels (linear mode)
    int tile_bytes, stage_bytes;
    int tab_off;                  // byte offset of the pixel table / epilogue vectors in shared memory
    int hdr_bytes, block_bytes;   // per (chunk, filter block) record: row-start header + entries, fixed size
    int act, out_dtype, linear;
    int ks_shift;                 // log2(ksplit)
    int unit_ok;                  // activations are staged in 4-byte units (always for f32; int8 needs c_in % 4 == 0)
    FastDiv d_groups, d_tiles_x, d_tiles_y, d_tbx, d_bw, d_cols_full;
};

// dst: 32-bit shared-window address
__device__ __forceinline__ void cp_async4(unsigned dst, const void *src, bool pred)
{
    int sz = pred ? 4 : 0;   // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async16(unsigned dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <typename XT> struct Traits;
template <> struct Traits<float> {
    typedef float acc_t;
    static const int kEntryBytes = 8;
    static const int kUnitElems = 1;   // elements per 4-byte staging unit
};
template <> struct Traits<int8_t> {
    typedef int acc_t;
    static const int kEntryBytes = 4;
    static const int kUnitElems = 4;
};

// Per-block staging table, built once: for every staged input pixel the offset of its first
// channel in x, in 4-byte units (the pixel index when activations are staged byte by byte;
// -1 = zero padding / outside), and its byte offset inside a stage.
__device__ __forceinline__ void build_pixel_table(const SconvParams &p, int2 *pix, int npx, int img, int oy0, int ox0,
                                                  long long p0)
{
    const int tid = threadIdx.x, NT = blockDim.x;
    if (p.linear) {
        for (int q = tid; q < npx; q += NT) {
            long long op = p0 + q;
            long long ip = -1;
            if (op < p.P) {
                ip = op;
                if (p.stride != 1) {
                    int ox = (int)(op % p.w_out);
                    long long r = op / p.w_out;
                    int oy = (int)(r % p.h_out);
                    long long b = r / p.h_out;
                    ip = (b * p.h + (long long)oy * p.stride) * p.w + (long long)ox * p.stride;
                }
            }
            const int src = ip < 0 ? -1 : (p.unit_ok ? (int)(unsigned)((ip * p.c_in * (long long)p.esz) >> 2) : (int)ip);
            pix[q] = make_int2(src, q * p.PPb);
        }
    } else {
        const int iy0 = oy0 * p.stride - p.pad, ix0 = ox0 * p.stride - p.pad_w;
        for (int i = tid; i < npx; i += NT) {
            int r = i / p.IW_t, col = i - r * p.IW_t;
            int iy = iy0 + r, ix = ix0 + col;
            int src = -1;
            if (iy >= 0 && iy < p.h && ix >= 0 && ix < p.w) {
                const long long ip = ((long long)img * p.h + iy) * p.w + ix;
                src = p.unit_ok ? (int)(unsigned)((ip * p.c_in * p.esz) >> 2) : (int)ip;
            }
            const int pos = p.half ? ((col & 1) * p.half + (col >> 1)) : col;
            pix[i] = make_int2(src, (r * p.pitch + pos) * p.PPb);
        }
    }
}

// Asynchronous copy of this block's nonzeros of chunk c (header + entries, one fixed-size
// record) behind the activation tile of a stage.  The weights never change, so this may be
// issued before the producer of x has finished.
__device__ __forceinline__ void stage_weights(const SconvParams &p, unsigned st32, int c, int grp)
{
    const uint4 *src = reinterpret_cast<const uint4 *>(
        reinterpret_cast<const unsigned char *>(p.ent) + ((size_t)c * p.n_groups + grp) * p.block_bytes);
    const unsigned dst = st32 + p.tile_bytes;
    for (int e = threadIdx.x; e < (p.block_bytes >> 4); e += blockDim.x) cp_async16(dst + e * 16, src + e);
}

// Asynchronous copies that stage the activation tile of chunk c: pixel-major, PPb bytes per
// pixel, 4 bytes per copy.
template <typename XT>
__device__ __forceinline__ void stage_acts(const SconvParams &p, const int2 *pixtab, int npx, long long p0,
                                           unsigned char *smem, unsigned smem32, unsigned stage_off, int c)
{
    typedef Traits<XT> TR;
    const int tid = threadIdx.x, NT = blockDim.x;
    const int c0 = c * p.CIc;
    const XT *xg = reinterpret_cast<const XT *>(p.x);
    const unsigned st32 = smem32 + stage_off;
    if (p.unit_ok) {
        const int upp = p.CIc / TR::kUnitElems;   // 4-byte units per staged pixel
        const unsigned char *xb = reinterpret_cast<const unsigned char *>(p.x);
        if ((upp & (upp - 1)) == 0 && upp <= NT && pixtab == nullptr) {
            // flat pixel range at stride 1: source and destination follow from the pixel number
            const int sh = 31 - __clz(upp);
            const int u = tid & (upp - 1);
            const int ci = c0 + u * TR::kUnitElems;
            const bool ch_ok = ci < p.c_in;
            const size_t pix_bytes = (size_t)p.c_in * sizeof(XT);
            const unsigned char *xcol = xb + (size_t)p0 * pix_bytes + (size_t)ci * sizeof(XT);
            const unsigned dcol = st32 + u * 4;
            const int pstep = NT >> sh;
            const long long left = p.P - p0;   // pixels that exist from p0 on
#pragma unroll 4
            for (int pix = tid >> sh; pix < npx; pix += pstep) {
                const bool ok = ch_ok && pix < left;
                const unsigned char *src = ok ? xcol + (size_t)pix * pix_bytes : xb;
                cp_async4(dcol + pix * p.PPb, src, ok);
            }
        } else if ((upp & (upp - 1)) == 0 && upp <= NT) {
            // each thread keeps one unit column and walks the pixels
            const int sh = 31 - __clz(upp);
            const int u = tid & (upp - 1);
            const int ci = c0 + u * TR::kUnitElems;
            const bool ch_ok = ci < p.c_in;
            const unsigned char *xcol = xb + (size_t)ci * sizeof(XT);
            const unsigned dcol = st32 + u * 4;
            const int pstep = NT >> sh;
#pragma unroll 4
            for (int pix = tid >> sh; pix < npx; pix += pstep) {
                const int2 te = pixtab[pix];
                const bool ok = ch_ok && te.x != -1;
                const unsigned char *src = ok ? xcol + ((size_t)(unsigned)te.x << 2) : xb;
                cp_async4(dcol + te.y, src, ok);
            }
        } else {
            const int total = npx * upp;
            for (int idx = tid; idx < total; idx += NT) {
                const int pix = idx / upp, u = idx - pix * upp;
                const int2 te = pixtab[pix];
                const int ci = c0 + u * TR::kUnitElems;
                const bool ok = te.x != -1 && ci < p.c_in;
                const unsigned char *src = ok ? xb + ((size_t)(unsigned)te.x << 2) + (size_t)ci * sizeof(XT) : xb;
                cp_async4(st32 + te.y + u * 4, src, ok);
            }
        }
    } else {
        // int8 with a channel count that is not a multiple of 4: plain byte copies
        const int cw = p.CIc;
        XT *stage = reinterpret_cast<XT *>(smem + stage_off);
        for (int idx = tid; idx < npx * cw; idx += NT) {
            const int pix = idx / cw, cl = idx - pix * cw;
            const int2 te = pixtab[pix];
            const int ci = c0 + cl;
            XT v = 0;
            if (te.x != -1 && ci < p.c_in) v = xg[(size_t)te.x * p.c_in + ci];
            stage[te.y + cl] = v;
        }
    }
}

template <typename XT, int T, int RPW>
__global__ void __launch_bounds__(512) sconv_kernel(const SconvParams p)
{
    typedef Traits<XT> TR;
    typedef typename TR::acc_t AT;
    extern __shared__ __align__(16) unsigned char smem[];
    const unsigned smem32 = (unsigned)__cvta_generic_to_shared(smem);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int KS = p.ksplit;
    const int rank = blockIdx.x & (KS - 1);
    const unsigned rest = blockIdx.x >> p.ks_shift;
    unsigned tile = fdiv(rest, p.d_groups);
    const int grp = (int)(rest - tile * p.n_groups);
    const int G = p.G;

    // tile origin
    int img = 0, oy0 = 0, ox0 = 0;
    long long p0 = 0;
    if (p.linear) {
        p0 = (long long)tile * (32 * T);
    } else {
        const unsigned t1 = fdiv(tile, p.d_tiles_x);
        const int tx = (int)(tile - t1 * p.tiles_x);
        const unsigned t2 = fdiv(t1, p.d_tiles_y);
        const int ty = (int)(t1 - t2 * p.tiles_y);
        img = (int)t2;
        oy0 = ty * p.TH;
        ox0 = tx * p.TW;
    }

    // this block's range of channel chunks
    const int per = (p.n_chunks + KS - 1) / KS;
    const int c_lo = min(p.n_chunks, rank * per), c_hi = min(p.n_chunks, c_lo + per);

    // Byte offset of a lane's pixel inside the staged tile = lane part + band part; the band
    // part is the same for every lane, so the T loads of one nonzero share one address add.
    const int xs = p.half ? 1 : p.stride;
    unsigned lanebase, band[T];
    if (p.linear) {
        lanebase = lane * p.PPb;
#pragma unroll
        for (int t = 0; t < T; ++t) band[t] = t * 32 * p.PPb;
    } else {
        const int lr = (int)fdiv(lane, p.d_bw), lc = lane - lr * p.BW;
        lanebase = (lr < p.RB) ? ((lr * p.stride) * p.pitch + lc * xs) * p.PPb : 0;
#pragma unroll
        for (int t = 0; t < T; ++t) {
            const int ty = (int)fdiv(t, p.d_tbx), tx = t - ty * p.TBX;
            band[t] = ((ty * p.RB * p.stride) * p.pitch + tx * p.BW * xs) * p.PPb;
        }
    }

    AT acc[RPW][T];
#pragma unroll
    for (int j = 0; j < RPW; ++j)
#pragma unroll
        for (int t = 0; t < T; ++t) acc[j][t] = 0;

    // ---- staging table and epilogue vectors (behind the pipeline stages in shared memory) ----
    const int S = p.stages;
    const int npx_in = p.linear ? 32 * T : p.IH_t * p.IW_t;
    int2 *pixtab = reinterpret_cast<int2 *>(smem + p.tab_off);
    float *sScale = reinterpret_cast<float *>(pixtab + npx_in);
    float *sBias = sScale + G;
    const int upp_chk = p.CIc / TR::kUnitElems;
    const bool direct = p.linear && p.stride == 1 && p.unit_ok && (upp_chk & (upp_chk - 1)) == 0 &&
                        upp_chk <= (int)blockDim.x;
    if (direct) pixtab = nullptr;   // no table needed
    else build_pixel_table(p, pixtab, npx_in, img, oy0, ox0, p0);
    if (tid < G) {   // epilogue vectors ride in the first copy group
        const int co = grp * G + tid;
        const unsigned ds = smem32 + p.tab_off + npx_in * 8 + tid * 4;
        if (p.scale && co < p.c_out) cp_async4(ds, p.scale + co, true); else sScale[tid] = 1.0f;
        if (p.bias && co < p.c_out) cp_async4(ds + G * 4, p.bias + co, true); else sBias[tid] = 0.0f;
    }
    int co_of[RPW];
#pragma unroll
    for (int j = 0; j < RPW; ++j) co_of[j] = p.perm[grp * G + warp * RPW + j];

    // ---- pipeline prologue: weights first (they do not depend on the previous layer) ----
    const int npre = (S == 1) ? 1 : S - 1;
    for (int s = 0; s < npre; ++s)
        if (c_lo + s < c_hi) stage_weights(p, smem32 + (unsigned)(s * p.stage_bytes), c_lo + s, grp);
    __syncthreads();          // the pixel table is complete
    grid_dep_wait();          // x (and the residual) are final from here on
    for (int s = 0; s < npre; ++s) {
        if (c_lo + s < c_hi) stage_acts<XT>(p, pixtab, npx_in, p0, smem, smem32, (unsigned)(s * p.stage_bytes), c_lo + s);
        cp_async_commit();
    }

    int buf = 0;   // stage holding chunk c
    for (int c = c_lo; c < c_hi; ++c) {
        if (S == 1) {
            if (c > c_lo) {
                __syncthreads();   // everyone is done with chunk c - 1
                stage_weights(p, smem32, c, grp);
                stage_acts<XT>(p, pixtab, npx_in, p0, smem, smem32, 0u, c);
                cp_async_commit();
            }
            cp_async_wait<0>();
            __syncthreads();
        } else {
            if (S == 3) cp_async_wait<1>(); else cp_async_wait<0>();
            __syncthreads();   // chunk c has landed for everyone; everyone is done with chunk c - 1
            const int nxt = c + S - 1;
            int nbuf = buf + S - 1;
            if (nbuf >= S) nbuf -= S;
            if (nxt < c_hi) {
                stage_weights(p, smem32 + (unsigned)(nbuf * p.stage_bytes), nxt, grp);
                stage_acts<XT>(p, pixtab, npx_in, p0, smem, smem32, (unsigned)(nbuf * p.stage_bytes), nxt);
            }
            cp_async_commit();
        }
        const unsigned stage_off = (unsigned)(buf * p.stage_bytes);
        const int *sP = reinterpret_cast<const int *>(smem + stage_off + p.tile_bytes);
        const unsigned sW = stage_off + p.tile_bytes + p.hdr_bytes;
        const unsigned lanep = stage_off + lanebase;
#pragma unroll
        for (int j = 0; j < RPW; ++j) {
            const int row = warp * RPW + j;
            const int beg = sP[row], end = sP[row + 1];
            // software pipeline: the next pair of nonzeros is fetched while this pair is used
            // (reading one pair past the row stays inside the record: the packer leaves slack)
            if (TR::kEntryBytes == 8) {
                uint4 nx = *reinterpret_cast<const uint4 *>(smem + sW + beg * 8);
#pragma unroll 2
                for (int e = beg; e < end; e += 2) {
                    const uint4 v = nx;
                    nx = *reinterpret_cast<const uint4 *>(smem + sW + (e + 2) * 8);
                    const AT w0 = (AT)__uint_as_float(v.x), w1 = (AT)__uint_as_float(v.z);
                    const unsigned a0 = lanep + v.y;
                    const unsigned a1 = lanep + v.w;
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += w0 * (AT)(*reinterpret_cast<const XT *>(smem + a0 + band[t]));
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += w1 * (AT)(*reinterpret_cast<const XT *>(smem + a1 + band[t]));
                }
            } else {
                uint2 nx = *reinterpret_cast<const uint2 *>(smem + sW + beg * 4);
#pragma unroll 2
                for (int e = beg; e < end; e += 2) {
                    const uint2 v = nx;
                    nx = *reinterpret_cast<const uint2 *>(smem + sW + (e + 2) * 4);
                    const AT w0 = (AT)(int)(int8_t)(v.x & 0xffu), w1 = (AT)(int)(int8_t)(v.y & 0xffu);
                    const unsigned a0 = lanep + (v.x >> 8);
                    const unsigned a1 = lanep + (v.y >> 8);
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += w0 * (AT)(*reinterpret_cast<const XT *>(smem + a0 + band[t]));
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += w1 * (AT)(*reinterpret_cast<const XT *>(smem + a1 + band[t]));
                }
            }
        }
        if (++buf == S) buf = 0;
    }
    cp_async_wait<0>();

    // ---- results to shared memory, [pixel][G + 1], at the original channel position ----
    __syncthreads();
    AT *sOut = reinterpret_cast<AT *>(smem);
    const int op = G + 1;
#pragma unroll
    for (int j = 0; j < RPW; ++j) {
        const int co = co_of[j];
        if (co >= 0) {
            int lc = co - grp * G;
#pragma unroll
            for (int t = 0; t < T; ++t) sOut[(lane + 32 * t) * op + lc] = acc[j][t];
        }
    }

    // ---- channel-split blocks of a cluster: sum the partial results over distributed shared memory ----
    const int npx = 32 * T;
    int q_lo = 0, q_hi = npx;
    if (KS > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();   // every block's partial sums are in its shared memory
        const int span = (npx + KS - 1) / KS;
        q_lo = min(npx, rank * span);
        q_hi = min(npx, q_lo + span);
        for (int idx = tid + q_lo * op; idx < q_hi * op; idx += blockDim.x) {
            AT v = sOut[idx];
            for (int k = 1; k < KS; ++k) {
                int other = rank + k;
                if (other >= KS) other -= KS;
                v += *cluster.map_shared_rank(sOut + idx, other);
            }
            sOut[idx] = v;
        }
    }
    __syncthreads();
    // The next layer may start its prologue now: it overlaps this block's stores and the
    // tail of the grid without competing with the multiply-add loop.
    grid_dep_trigger();

    // ---- epilogue and contiguous NHWC stores ----
    const int co_base = grp * G;
    const int gw = min(G, p.c_out - co_base);  // real channels in this block
    const bool has_res = p.residual != nullptr;
    const bool quad = ((gw & 3) == 0) && ((p.c_out & 3) == 0) && ((p.ldc & 3) == 0) && ((p.c_off & 3) == 0);
    const int cols = quad ? (gw >> 2) : gw;
    const bool full = quad && gw == G;   // the usual case: a precomputed divisor
    for (int idx = tid + q_lo * cols; idx < q_hi * cols; idx += blockDim.x) {
        const int q = full ? (int)fdiv(idx, p.d_cols_full) : idx / cols;
        const int cq = idx - q * cols;
        long long opix;
        if (p.linear) {
            opix = p0 + q;
            if (opix >= p.P) continue;
        } else {
            const int t = q >> 5, l = q & 31;
            const int ty = (int)fdiv(t, p.d_tbx), tx = t - ty * p.TBX;
            const int lr = (int)fdiv(l, p.d_bw), lcx = l - lr * p.BW;
            const int oy = oy0 + ty * p.RB + lr, ox = ox0 + tx * p.BW + lcx;
            if (lr >= p.RB || oy >= p.h_out || ox >= p.w_out) continue;
            opix = ((long long)img * p.h_out + oy) * p.w_out + ox;
        }
        const int lc = quad ? cq * 4 : cq;
        const int co = co_base + lc;
        const size_t ri = (size_t)opix * p.c_out + co;              // residual: a tensor of exactly c_out channels
        const size_t oi = (size_t)opix * p.ldc + p.c_off + co;      // output: possibly a channel window of a wider tensor
        const AT *a0 = sOut + q * op + lc;
        AT a[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) a[v] = (quad || v == 0) ? a0[v] : (AT)0;
        if (sizeof(XT) == 1 && p.acc_in) {   // sums of the layer's dense blocks, computed on the tensor cores
#pragma unroll
            for (int v = 0; v < 4; ++v)
                if (quad || v == 0) a[v] = (AT)((int)a[v] + p.acc_in[ri + v]);
        }
        if (quad) {
            float sc[4], bi[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                sc[v] = sScale[lc + v];
                bi[v] = sBias[lc + v];
            }
            if (sizeof(XT) == 4) {
                float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
                if (has_res) r = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(p.residual) + ri);
                float4 o;
                o.x = act_f32(fmaf((float)a[0], sc[0], bi[0]) + r.x, p.act);
                o.y = act_f32(fmaf((float)a[1], sc[1], bi[1]) + r.y, p.act);
                o.z = act_f32(fmaf((float)a[2], sc[2], bi[2]) + r.z, p.act);
                o.w = act_f32(fmaf((float)a[3], sc[3], bi[3]) + r.w, p.act);
                *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.y) + oi) = o;
            } else if (p.out_dtype == CADNN_S32) {
                *reinterpret_cast<int4 *>(reinterpret_cast<int *>(p.y) + oi) = make_int4((int)a[0], (int)a[1], (int)a[2], (int)a[3]);
            } else if (p.out_dtype == CADNN_F32) {
                char4 r = make_char4(0, 0, 0, 0);
                if (has_res) r = *reinterpret_cast<const char4 *>(reinterpret_cast<const int8_t *>(p.residual) + ri);
                float4 o;
                o.x = requant_f32((int)a[0], sc[0], bi[0], p.act, has_res, r.x, p.res_scale);
                o.y = requant_f32((int)a[1], sc[1], bi[1], p.act, has_res, r.y, p.res_scale);
                o.z = requant_f32((int)a[2], sc[2], bi[2], p.act, has_res, r.z, p.res_scale);
                o.w = requant_f32((int)a[3], sc[3], bi[3], p.act, has_res, r.w, p.res_scale);
                *reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.y) + oi) = o;
            } else {
                char4 r = make_char4(0, 0, 0, 0);
                if (has_res) r = *reinterpret_cast<const char4 *>(reinterpret_cast<const int8_t *>(p.residual) + ri);
                char4 o;
                o.x = (signed char)requant_s8((int)a[0], sc[0], bi[0], p.act, has_res, r.x, p.res_scale);
                o.y = (signed char)requant_s8((int)a[1], sc[1], bi[1], p.act, has_res, r.y, p.res_scale);
                o.z = (signed char)requant_s8((int)a[2], sc[2], bi[2], p.act, has_res, r.z, p.res_scale);
                o.w = (signed char)requant_s8((int)a[3], sc[3], bi[3], p.act, has_res, r.w, p.res_scale);
                *reinterpret_cast<char4 *>(reinterpret_cast<int8_t *>(p.y) + oi) = o;
            }
        } else {
            const float sc = sScale[lc];
            const float bi = sBias[lc];
            if (sizeof(XT) == 4) {
                float z = fmaf((float)a[0], sc, bi);
                if (has_res) z += reinterpret_cast<const float *>(p.residual)[ri];
                reinterpret_cast<float *>(p.y)[oi] = act_f32(z, p.act);
            } else if (p.out_dtype == CADNN_S32) {
                reinterpret_cast<int *>(p.y)[oi] = (int)a[0];
            } else {
                const int r = has_res ? (int)reinterpret_cast<const int8_t *>(p.residual)[ri] : 0;
                if (p.out_dtype == CADNN_F32)
                    reinterpret_cast<float *>(p.y)[oi] = requant_f32((int)a[0], sc, bi, p.act, has_res, r, p.res_scale);
                else
                    reinterpret_cast<int8_t *>(p.y)[oi] = (int8_t)requant_s8((int)a[0], sc, bi, p.act, has_res, r, p.res_scale);
            }
        }
    }
    // peers may still be reading this block's partial sums
    if (KS > 1) cg::this_cluster().sync();
}

template <typename XT, int T, int RPW>
cadnn_status launch_one(const SconvParams &p, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    auto kern = sconv_kernel<XT, T, RPW>;
    static SmemLimit lim;   // per instantiation, per device
    if (smem > 48 * 1024) {
        cadnn_status rs = raise_smem_limit((const void *)kern, smem, &lim);
        if (rs != CADNN_OK) return rs;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks, 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (p.ksplit > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)p.ksplit;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)na;
    CADNN_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p));
    return CADNN_OK;
}

template <typename XT, int T>
cadnn_status launch_rpw(const SconvParams &p, int rpw, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    switch (rpw) {
        case 1: return launch_one<XT, T, 1>(p, blocks, threads, smem, pdl, st);
        case 2: return launch_one<XT, T, 2>(p, blocks, threads, smem, pdl, st);
        case 4: return launch_one<XT, T, 4>(p, blocks, threads, smem, pdl, st);
        // many filters per warp only with few pixel bands per lane (accumulators = RPW * T registers)
        case 8: if (T <= 4) return launch_one<XT, (T <= 4 ? T : 1), 8>(p, blocks, threads, smem, pdl, st); break;
        case 16: if (T <= 2) return launch_one<XT, (T <= 2 ? T : 1), 16>(p, blocks, threads, smem, pdl, st); break;
    }
    return CADNN_E_UNSUPPORTED;
}

template <typename XT>
cadnn_status launch_T(const SconvParams &p, int T, int rpw, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    switch (T) {
        case 1: return launch_rpw<XT, 1>(p, rpw, blocks, threads, smem, pdl, st);
        case 2: return launch_rpw<XT, 2>(p, rpw, blocks, threads, smem, pdl, st);
        case 3: return launch_rpw<XT, 3>(p, rpw, blocks, threads, smem, pdl, st);
        case 4: return launch_rpw<XT, 4>(p, rpw, blocks, threads, smem, pdl, st);
        case 5: return launch_rpw<XT, 5>(p, rpw, blocks, threads, smem, pdl, st);
        case 6: return launch_rpw<XT, 6>(p, rpw, blocks, threads, smem, pdl, st);
        case 7: return launch_rpw<XT, 7>(p, rpw, blocks, threads, smem, pdl, st);
        case 8: return launch_rpw<XT, 8>(p, rpw, blocks, threads, smem, pdl, st);
    }
    return CADNN_E_UNSUPPORTED;
}

}  // namespace

cadnn_status launch_sconv(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                          cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    const Schedule &s = w->s;
    const bool s8 = d.dtype == CADNN_S8;
    SconvParams p;
    p.x = x;
    p.y = y;
    p.ent = w->d_ent;
    p.perm = w->d_perm;
    p.scale = ep.scale;
    p.bias = ep.bias;
    p.residual = ep.residual;
    p.n = n; p.h = d.in_h; p.w = d.in_w; p.c_in = d.c_in;
    p.h_out = w->h_out; p.w_out = w->w_out; p.c_out = d.c_out;
    p.stride = d.stride; p.pad = d.pad; p.pad_w = d.pad_w;
    p.res_scale = ep.res_scale;
    p.acc_in = ep.acc_in;
    p.ldc = ep.out_c_total > 0 ? ep.out_c_total : d.c_out; p.c_off = ep.out_c_total > 0 ? ep.out_c_off : 0;
    p.BW = s.BW; p.RB = s.RB; p.TBX = s.TBX; p.TBY = s.TBY; p.TH = s.TH; p.TW = s.TW;
    p.pitch = s.pitch; p.half = s.half; p.IH_t = s.IH_t; p.IW_t = s.IW_t;
    p.CIc = s.CIc; p.PPb = s.PPb; p.n_chunks = s.n_chunks; p.G = s.G; p.n_groups = s.n_groups;
    p.stages = s.stages;
    p.ksplit = s.ksplit;
    p.linear = s.kind == KK_SCONV_LINEAR;
    p.P = (long long)n * w->h_out * w->w_out;
    p.tile_bytes = s.tile_bytes;
    p.stage_bytes = s.stage_bytes;
    p.tab_off = (std::max(s.stages * s.stage_bytes, 32 * s.T * (s.G + 1) * 4) + 15) / 16 * 16;
    p.hdr_bytes = (s.G + 1 + 3) / 4 * 16;
    p.block_bytes = p.hdr_bytes + s.max_entries * (s8 ? 4 : 8);
    p.act = ep.act;
    p.out_dtype = ep.out_dtype;
    p.esz = s8 ? 1 : 4;
    p.unit_ok = (!s8 || (d.c_in & 3) == 0) ? 1 : 0;
    p.ks_shift = s.ksplit == 8 ? 3 : s.ksplit == 4 ? 2 : s.ksplit == 2 ? 1 : 0;
    long long tiles;
    if (p.linear) {
        p.tiles_x = p.tiles_y = 1;
        tiles = (p.P + 32 * s.T - 1) / (32 * s.T);
    } else {
        p.tiles_y = (w->h_out + s.TH - 1) / s.TH;
        p.tiles_x = (w->w_out + s.TW - 1) / s.TW;
        tiles = (long long)n * p.tiles_y * p.tiles_x;
    }
    p.d_groups = make_fastdiv(s.n_groups);
    p.d_tiles_x = make_fastdiv(p.tiles_x);
    p.d_tiles_y = make_fastdiv(p.tiles_y);
    p.d_tbx = make_fastdiv(s.TBX);
    p.d_bw = make_fastdiv(s.BW);
    p.d_cols_full = make_fastdiv(std::max(1, s.G / 4));
    long long blocks = tiles * s.n_groups * s.ksplit;
    if (blocks <= 0) return CADNN_OK;
    // the staging table addresses x in 4-byte units through 32 bits
    if ((long long)n * d.in_h * d.in_w * d.c_in * p.esz >= (1LL << 34)) return CADNN_E_UNSUPPORTED;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    if (s8) return launch_T<int8_t>(p, s.T, s.RPW, (int)blocks, s.NW * 32, s.smem_bytes, ep.pdl, st);
    return launch_T<float>(p, s.T, s.RPW, (int)blocks, s.NW * 32, s.smem_bytes, ep.pdl, st);
}
