// Sparse convolution over channel-planar activations with a zero halo, and the glue
// kernels of that layout.
//
// CADNN (arXiv 1905.00571), Section 4, "Memory layout transformation": the layout of the
// data is changed to fit the processor.  Inside cadnn_forward the float activations of a
// network are kept as [n][c][h + 2][w + 2] planes whose one-pixel border stays zero:
//   * the lanes of a warp are 32 consecutive positions of a (padded) plane, so for ANY stored
//     nonzero (ci, ky, kx) their activation loads are one contiguous 128-byte segment
//     straight from L1/L2 - no shared-memory staging, no bank layout, no transposition;
//   * zero padding of the convolution is the halo itself: no bounds test in the loop;
//   * a warp walks a whole filter (all input channels) by itself, so no reduction across
//     blocks is ever needed, however many channels the layer has;
//   * results are stored by the same lanes, contiguously, with the epilogue applied
//     (BatchNorm fold, residual read from a planar tensor, ReLU / ReLU6); halo positions are
//     never written, so they stay zero for the next layer.
// The layer-level C entry points keep NHWC; this layout is internal to the network runner
// (and reachable for tests through cadnn_conv2d_planar).
#include <algorithm>
#include "cadnn_internal.h"

namespace {

struct PlanarParams {
    const float *x;
    float *y;
    const uint4 *ent;     // pairs of {value bits, element offset}
    const int32_t *ptr;   // [c_out + 1] in entries (even), by original output channel
    const int4 *order;    // [n_groups * G] per warp slot {filter (-1 = none), first pair, end pair, 0}: one load tells a
                          // warp everything it needs to start fetching nonzeros
    const float *scale;
    const float *bias;
    const float *residual;
    int n, c_in, c_out;
    int wp_in, plane_in, wp_out, plane_out, h_out, w_out;
    int stride, halo, qtot;
    int G, RPW, n_groups, tiles, act;
    int ksw_shift;   // log2 of the warps that share one filter (each walks a slice of its nonzeros)
    FastDiv d_wp_out, d_groups, d_tiles;
    ParityPlanes par;   // second copy of the output for a stride-2 reader (par.y null = none)
};

__device__ __forceinline__ float pl_act(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

// D: depth of a batch of nonzeros (16 * D activation loads in flight per lane).  At batch 1 no
// layer fills the device, registers are free, and what a warp pays is one L1 / L2 round trip per
// batch: deeper batches mean fewer of them.
template <int T, int D>
__global__ void __launch_bounds__(512) sconv_planar_kernel(const PlanarParams p)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // block -> (image, pixel tile, filter group); groups vary fastest so that blocks running
    // together read the same activations
    const unsigned r1 = fdiv(blockIdx.x, p.d_groups);
    const int grp = (int)(blockIdx.x - r1 * p.n_groups);
    const unsigned img = fdiv(r1, p.d_tiles);
    const int tile = (int)(r1 - img * p.tiles);
    const int q0 = tile * (32 * T);

    // positions of this lane: q runs over the interior rows of the padded output plane,
    // halo columns included (they are computed but not stored)
    int inb[T];
    unsigned okmask = 0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = q0 + 32 * t + lane;
        const int oy = (int)fdiv((unsigned)min(q, p.qtot - 1), p.d_wp_out);
        const int oxp = min(q, p.qtot - 1) - oy * p.wp_out;
        const bool ok = q < p.qtot && oxp >= p.halo && oxp < p.halo + p.w_out;
        if (ok) okmask |= 1u << t;
        // lanes that store nothing still load: give them a position that is inside the plane
        const int oxs = ok ? oxp : p.halo;
        inb[t] = (oy * p.stride) * p.wp_in + (oxs - p.halo) * p.stride;
    }
    grid_dep_wait();
    grid_dep_trigger();
    const float *ximg = p.x + (size_t)img * p.c_in * p.plane_in;

    // KSW warps share a filter: each walks a slice of its nonzeros, slice 0 adds the partial sums
    // (through shared memory) and stores.  Few-pixel layers get their parallelism this way.
    __shared__ float sRed[(T <= 4 ? 16 : 8)][T][32];   // as many warps as a block of this T may have
    const int KSW = 1 << p.ksw_shift;
    const int rslot = warp >> p.ksw_shift, slice = warp & (KSW - 1);
    for (int j = 0; j < p.RPW; ++j) {
        const int4 slot = __ldg(p.order + grp * p.G + rslot * p.RPW + j);
        const int co = slot.x;
        float acc[T];
#pragma unroll
        for (int t = 0; t < T; ++t) acc[t] = 0.0f;
        // epilogue operands are requested now, so that their round trip to L2 overlaps the loop
        float sc = 1.0f, bi = 0.0f, res[T];
#pragma unroll
        for (int t = 0; t < T; ++t) res[t] = 0.0f;
        const size_t obase = ((size_t)img * p.c_out + max(co, 0)) * p.plane_out + (size_t)p.halo * p.wp_out + q0 + lane;
        if (co >= 0 && slice == 0) {
            if (p.scale) sc = __ldg(p.scale + co);
            if (p.bias) bi = __ldg(p.bias + co);
            if (p.residual) {
#pragma unroll
                for (int t = 0; t < T; ++t)
                    if (okmask & (1u << t)) res[t] = ld_act(p.residual + obase + 32 * t);
            }
        }
        if (co >= 0) {
            const int rbeg = slot.y, rend = slot.z;   // in pairs
            const int per = (rend - rbeg + KSW - 1) >> p.ksw_shift;
            const int beg = min(rend, rbeg + slice * per), end = min(rend, beg + per);
            // Every lane reads the same pairs of nonzeros (broadcast transactions), one batch ahead.
            // A batch issues all its activation loads before the first multiply-add: the loads are
            // independent L1/L2 round trips and only their number in flight hides that latency.
            // Slots past the end of the slice hold {0, offset 0}: they add nothing.
            constexpr int P = (8 * D / T) > 8 ? 8 : (8 * D / T);   // pairs per batch
            const uint4 zero4 = make_uint4(0, 0, 0, 0);
            uint4 nx[P];
#pragma unroll
            for (int i = 0; i < P; ++i) nx[i] = (beg + i < end) ? __ldg(p.ent + beg + i) : zero4;
            for (int e = beg; e < end; e += P) {
                uint4 v[P];
#pragma unroll
                for (int i = 0; i < P; ++i) v[i] = nx[i];
#pragma unroll
                for (int i = 0; i < P; ++i) nx[i] = (e + P + i < end) ? __ldg(p.ent + e + P + i) : zero4;
                float a[P][2][T];
#pragma unroll
                for (int i = 0; i < P; ++i)
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        a[i][0][t] = ld_act(ximg + v[i].y + inb[t]);
                        a[i][1][t] = ld_act(ximg + v[i].w + inb[t]);
                    }
#pragma unroll
                for (int i = 0; i < P; ++i) {
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[t] = fmaf(__uint_as_float(v[i].x), a[i][0][t], acc[t]);
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[t] = fmaf(__uint_as_float(v[i].z), a[i][1][t], acc[t]);
                }
            }
        }
        if (KSW > 1) {
#pragma unroll
            for (int t = 0; t < T; ++t) sRed[warp][t][lane] = acc[t];
            __syncthreads();
            if (slice == 0) {
                for (int s2 = 1; s2 < KSW; ++s2)
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[t] += sRed[warp + s2][t][lane];
            }
            __syncthreads();   // sRed is reused by the next filter
        }
        if (co >= 0 && slice == 0) {
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (okmask & (1u << t)) {
                    const float z = pl_act(fmaf(acc[t], sc, bi) + res[t], p.act);
                    p.y[obase + 32 * t] = z;
                    if (p.par.y) {
                        const int q = q0 + 32 * t + lane;   // interior rows, padded columns
                        const int oy = (int)fdiv((unsigned)q, p.d_wp_out);
                        parity_store(p.par, img, co, oy, q - oy * p.wp_out - p.halo, z);
                    }
                }
            }
        }
    }
}

// max pool over planar tensors: padded taps are ignored (explicit bounds, the halo is not used)
__global__ void __launch_bounds__(256) maxpool_planar_kernel(const float *x, float *y, int nc, int h, int w, int wp_in,
                                                             int plane_in, int h_out, int w_out, int wp_out,
                                                             int plane_out, int halo, int k, int stride, int pad,
                                                             FastDiv d_wout, FastDiv d_hout)
{
    const unsigned total = (unsigned)nc * h_out * w_out;
    grid_dep_wait();
    grid_dep_trigger();
    for (unsigned idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const unsigned r = fdiv(idx, d_wout);
        const int ox = (int)(idx - r * w_out);
        const unsigned pl = fdiv(r, d_hout);
        const int oy = (int)(r - pl * h_out);
        const float *src = x + (size_t)pl * plane_in;
        bool any = false;
        float best = 0.0f;
        for (int ky = 0; ky < k; ++ky) {
            const int iy = oy * stride + ky - pad;
            if (iy < 0 || iy >= h) continue;
            for (int kx = 0; kx < k; ++kx) {
                const int ix = ox * stride + kx - pad;
                if (ix < 0 || ix >= w) continue;
                const float v = src[(iy + halo) * wp_in + ix + halo];
                if (!any || v > best) best = v;
                any = true;
            }
        }
        y[(size_t)pl * plane_out + (oy + halo) * wp_out + ox + halo] = best;
    }
}

// global average pool: one warp per plane, y[n][c] dense
__global__ void __launch_bounds__(256) gavgpool_planar_kernel(const float *x, float *y, int nc, int h, int w, int wp,
                                                              int plane, int halo, float inv)
{
    const int lane = threadIdx.x & 31;
    const int pl = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    grid_dep_wait();
    grid_dep_trigger();
    if (pl >= nc) return;
    const float *src = x + (size_t)pl * plane;
    float s = 0.0f;
    for (int i = lane; i < h * w; i += 32) {
        const int r = i / w, c = i - r * w;
        s += src[(r + halo) * wp + c + halo];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) y[pl] = s * inv;
}

// Dense depthwise convolution over planar tensors: a warp takes 32 * T consecutive positions of ONE
// channel plane; a tap is one contiguous 128-byte load per band, the zero halo is the padding,
// the kh * kw taps of the channel are broadcast loads from the tap-major weights.
struct DwPlanarParams {
    const float *x;
    float *y;
    const float *wt;   // [kh * kw][c]
    const float *scale;
    const float *bias;
    int nc, c, wp_in, plane_in, wp_out, plane_out, h_out, w_out, kh, kw, stride, off0, halo, qtot, tiles, act;
    FastDiv d_wp_out, d_tiles, d_c;
};

template <int T>
__global__ void __launch_bounds__(256) dw_planar_kernel(const DwPlanarParams p)
{
    const int lane = threadIdx.x & 31;
    const unsigned task = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const unsigned pl = fdiv(task, p.d_tiles);
    const int tile = (int)(task - pl * p.tiles);
    const bool live = pl < (unsigned)p.nc;
    const int ch = live ? (int)(pl - fdiv(pl, p.d_c) * p.c) : 0;
    const int q0 = tile * (32 * T);
    int inb[T];
    unsigned okmask = 0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = q0 + 32 * t + lane;
        const int qc = min(q, p.qtot - 1);
        const int oy = (int)fdiv((unsigned)qc, p.d_wp_out);
        const int oxp = qc - oy * p.wp_out;
        const bool ok = live && q < p.qtot && oxp >= p.halo && oxp < p.halo + p.w_out;
        if (ok) okmask |= 1u << t;
        const int oxs = ok ? oxp : p.halo;
        inb[t] = (oy * p.stride + p.off0) * p.wp_in + (oxs - p.halo) * p.stride + p.off0;
    }
    // static data first: the taps and the epilogue pair of this channel
    float wv[9];
    const int taps = p.kh * p.kw;   // <= 9 (the host checks)
#pragma unroll
    for (int k = 0; k < 9; ++k) wv[k] = k < taps ? __ldg(p.wt + (size_t)k * p.c + ch) : 0.0f;
    const float sc = p.scale ? __ldg(p.scale + ch) : 1.0f;
    const float bi = p.bias ? __ldg(p.bias + ch) : 0.0f;
    grid_dep_wait();
    grid_dep_trigger();
    if (!live) return;
    const float *xp = p.x + (size_t)pl * p.plane_in;
    float acc[T];
#pragma unroll
    for (int t = 0; t < T; ++t) acc[t] = 0.0f;
#pragma unroll
    for (int k = 0; k < 9; ++k) {
        if (k < taps) {
            const int ky = k / p.kw, kx = k - ky * p.kw;
            const int off = ky * p.wp_in + kx;
#pragma unroll
            for (int t = 0; t < T; ++t) acc[t] = fmaf(wv[k], ld_act(xp + inb[t] + off), acc[t]);
        }
    }
    float *yp = p.y + (size_t)pl * p.plane_out + (size_t)p.halo * p.wp_out + q0 + lane;
#pragma unroll
    for (int t = 0; t < T; ++t)
        if (okmask & (1u << t)) yp[32 * t] = pl_act(fmaf(acc[t], sc, bi), p.act);
}

}  // namespace

cadnn_status launch_sconv_planar(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                 cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    const int halo = kPlanarHalo;
    PlanarParams p;
    p.x = (const float *)x; p.y = (float *)y;
    p.ent = (const uint4 *)w->d_pl_ent; p.ptr = w->d_pl_ptr; p.order = (const int4 *)w->d_pl_order;
    p.scale = ep.scale; p.bias = ep.bias; p.residual = (const float *)ep.residual;
    p.n = n; p.c_in = d.c_in; p.c_out = d.c_out;
    p.wp_in = d.in_w + 2 * halo; p.plane_in = planar_pitch(d.in_h, d.in_w);
    p.h_out = w->h_out; p.w_out = w->w_out;
    p.wp_out = w->w_out + 2 * halo; p.plane_out = planar_pitch(w->h_out, w->w_out);
    p.stride = d.stride; p.halo = halo; p.qtot = w->h_out * p.wp_out;
    const int T = w->pl_T;
    if (w->pl_NW > (T <= 4 ? 16 : 8)) return CADNN_E_UNSUPPORTED;
    const int ksw = std::max(1, std::min(w->pl_KSW, w->pl_NW));
    p.ksw_shift = ksw >= 8 ? 3 : ksw >= 4 ? 2 : ksw >= 2 ? 1 : 0;
    p.G = (w->pl_NW >> p.ksw_shift) * w->pl_RPW; p.RPW = w->pl_RPW;
    p.n_groups = (d.c_out + p.G - 1) / p.G;
    p.tiles = (p.qtot + 32 * T - 1) / (32 * T);
    p.act = ep.act;
    p.par = parity_planes(ep.parity_y, ep.parity_mask, w->h_out, w->w_out, d.c_out);
    p.d_wp_out = make_fastdiv(p.wp_out);
    p.d_groups = make_fastdiv(p.n_groups);
    p.d_tiles = make_fastdiv(p.tiles);
    long long blocks = (long long)n * p.tiles * p.n_groups;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    const int threads = w->pl_NW * 32;
    switch (T * 10 + (w->pl_D >= 4 ? 4 : w->pl_D >= 2 ? 2 : 1)) {
        case 11: case 12: case 14: return launch_kernel(sconv_planar_kernel<1, 1>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 21: return launch_kernel(sconv_planar_kernel<2, 1>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 22: case 24: return launch_kernel(sconv_planar_kernel<2, 2>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 41: return launch_kernel(sconv_planar_kernel<4, 1>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 42: return launch_kernel(sconv_planar_kernel<4, 2>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 44: return launch_kernel(sconv_planar_kernel<4, 4>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 81: return launch_kernel(sconv_planar_kernel<8, 1>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 82: return launch_kernel(sconv_planar_kernel<8, 2>, (int)blocks, threads, 0, ep.pdl, st, p);
        case 84: return launch_kernel(sconv_planar_kernel<8, 4>, (int)blocks, threads, 0, ep.pdl, st, p);
    }
    return CADNN_E_UNSUPPORTED;
}

cadnn_status launch_maxpool_planar(const float *x, int n, int h, int wd, int c, int k, int stride, int pad, float *y,
                                   bool pdl, cudaStream_t st)
{
    const int halo = kPlanarHalo;
    const int h_out = (h + 2 * pad - k) / stride + 1, w_out = (wd + 2 * pad - k) / stride + 1;
    long long total = (long long)n * c * h_out * w_out;
    if (total <= 0) return CADNN_OK;
    if (total >= (1LL << 31)) return CADNN_E_UNSUPPORTED;
    long long blocks = std::min((total + 255) / 256, 148LL * 32);
    return launch_kernel(maxpool_planar_kernel, (int)blocks, 256, 0, pdl, st, x, y, n * c, h, wd, wd + 2 * halo,
                         planar_pitch(h, wd), h_out, w_out, w_out + 2 * halo, planar_pitch(h_out, w_out), halo, k, stride, pad, make_fastdiv(w_out),
                         make_fastdiv(h_out));
}

cadnn_status launch_gavgpool_planar(const float *x, int n, int h, int wd, int c, float *y, bool pdl, cudaStream_t st)
{
    const int halo = kPlanarHalo;
    if (n * c <= 0) return CADNN_OK;
    return launch_kernel(gavgpool_planar_kernel, (n * c + 7) / 8, 256, 0, pdl, st, x, y, n * c, h, wd, wd + 2 * halo,
                         planar_pitch(h, wd), halo, 1.0f / (float)(h * wd));
}

bool dw_planar_ok(const cadnn_weights *w)
{
    const cadnn_layer_desc &d = w->desc;
    return w->s.kind == KK_DW && d.dtype == CADNN_F32 && d.kh * d.kw <= 9 && d.pad <= kPlanarHalo &&
           d.kh - 1 - d.pad <= kPlanarHalo && d.kw - 1 - d.pad <= kPlanarHalo && w->d_dense != nullptr;
}

cadnn_status launch_dw_planar(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                              cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    if (!dw_planar_ok(w) || ep.residual) return CADNN_E_UNSUPPORTED;
    const int halo = kPlanarHalo;
    DwPlanarParams p;
    p.x = (const float *)x; p.y = (float *)y; p.wt = w->d_dense;
    p.scale = ep.scale; p.bias = ep.bias;
    p.nc = n * d.c_out; p.c = d.c_out;
    p.wp_in = d.in_w + 2 * halo; p.plane_in = planar_pitch(d.in_h, d.in_w);
    p.h_out = w->h_out; p.w_out = w->w_out;
    p.wp_out = w->w_out + 2 * halo; p.plane_out = planar_pitch(w->h_out, w->w_out);
    p.kh = d.kh; p.kw = d.kw; p.stride = d.stride; p.off0 = halo - d.pad; p.halo = halo;
    p.qtot = w->h_out * p.wp_out;
    p.act = ep.act;
    const int T = p.qtot >= 1024 ? 4 : p.qtot >= 256 ? 2 : 1;
    p.tiles = (p.qtot + 32 * T - 1) / (32 * T);
    p.d_wp_out = make_fastdiv(p.wp_out);
    p.d_tiles = make_fastdiv(p.tiles);
    p.d_c = make_fastdiv(p.c);
    const long long tasks = (long long)p.nc * p.tiles;
    if (tasks <= 0) return CADNN_OK;
    const long long blocks = (tasks + 7) / 8;
    if (blocks > 2147483647LL || tasks >= (1LL << 31)) return CADNN_E_UNSUPPORTED;
    switch (T) {
        case 1: return launch_kernel(dw_planar_kernel<1>, (int)blocks, 256, 0, ep.pdl, st, p);
        case 2: return launch_kernel(dw_planar_kernel<2>, (int)blocks, 256, 0, ep.pdl, st, p);
        default: return launch_kernel(dw_planar_kernel<4>, (int)blocks, 256, 0, ep.pdl, st, p);
    }
}
