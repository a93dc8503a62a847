// Sparse stride-1 convolution over channel-planar activations, with the input tile staged
// in shared memory.
//
// CADNN (arXiv 1905.00571), Section 4: one fused kernel per compressed layer (Conv +
// BatchNorm + Activation), a memory layout made to fit the processor, no redundant loads.
// In the padded planar layout ([n][c][plane], plane = (h + 2) x (w + 2) with a zero border) a
// "same" convolution at stride 1 is a one-dimensional stencil over the linear position q of a
// plane: tap (ky, kx) reads q + (ky - pad) * (w + 2) + (kx - pad).  So
//   * a thread block owns 32 * T consecutive positions and G filters; per chunk of input
//     channels it stages, for every channel, ONE contiguous run of the plane (the positions
//     plus a margin for the taps) with 16-byte asynchronous copies - no pixel table, no
//     transposition, and consecutive lanes read consecutive words of shared memory (never a
//     bank conflict), whatever the tap;
//   * the nonzeros of the block's filters in that chunk arrive in the same copy group as
//     {value, byte offset into the staged tile}; a warp walks them two at a time,
//     broadcasts them and issues T multiply-adds per lane and nonzero; accumulators stay
//     in registers across chunks;
//   * KS warps share a filter (each takes an equal share of its nonzeros in every chunk) and
//     add their partial sums through shared memory: few-pixel layers get their parallelism
//     inside the block, without a cluster;
//   * lanes store their own positions (contiguous in the output plane) with the epilogue
//     applied; border positions are computed but never stored, so the border stays zero.
#include <algorithm>
#include "cadnn_internal.h"

namespace {

struct PsParams {
    const float *x;
    float *y;
    const uint32_t *ent;   // records [n_chunks][n_groups], block_bytes each: header of G * KS + 1 starts, entries
    const int32_t *perm;   // [n_groups * G] packed row -> output channel, -1 = none
    const float *scale;
    const float *bias;
    const float *residual;
    int c_in, c_out;
    int h, w, wp, pitch;   // interior size, padded row length, floats between planes
    int q_start, tiles;    // first computed position (a multiple of 4), tiles of 32 * T positions per image
    int A, L;              // staged margin on either side and staged floats per channel (multiples of 4)
    int CIc, n_chunks, G, n_groups, stages;
    int ks_shift;
    int tile_bytes, stage_bytes, hdr_bytes, block_bytes;
    int act;
    FastDiv d_groups, d_tiles, d_wp, d_l4;
};

__device__ __forceinline__ void cp16(unsigned dst, const void *src, bool pred)
{
    const int sz = pred ? 16 : 0;   // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ float ps_act(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

// weights of chunk c for this block's filters: one fixed-size record behind the tile of a stage
__device__ __forceinline__ void ps_stage_weights(const PsParams &p, unsigned st32, int c, int grp)
{
    const uint4 *src = reinterpret_cast<const uint4 *>(
        reinterpret_cast<const unsigned char *>(p.ent) + ((size_t)c * p.n_groups + grp) * p.block_bytes);
    const unsigned dst = st32 + p.tile_bytes;
    for (int e = threadIdx.x; e < (p.block_bytes >> 4); e += blockDim.x) cp16(dst + e * 16, src + e, true);
}

// activations of chunk c: per channel the run [q0 - A, q0 + 32 T + A) of its plane; 16-byte pieces
// that fall outside the plane (or past the last channel) are zero-filled
__device__ __forceinline__ void ps_stage_acts(const PsParams &p, const float *ximg, unsigned st32, int c, int q0)
{
    const int l4 = p.L >> 2;
    const int total = p.CIc * l4;
    const int c0 = c * p.CIc;
    const int qa0 = q0 - p.A;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
        const int r = (int)fdiv((unsigned)idx, p.d_l4);
        const int k = idx - r * l4;
        const int ci = c0 + r;
        const int qa = qa0 + 4 * k;
        const bool ok = ci < p.c_in && qa >= 0 && qa + 4 <= p.pitch;
        const float *src = ok ? ximg + (size_t)ci * p.pitch + qa : ximg;
        cp16(st32 + (unsigned)idx * 16u, src, ok);
    }
}

template <int T, int RPW>
__global__ void __launch_bounds__(512) sconv_planar_staged_kernel(const PsParams p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const unsigned smem32 = (unsigned)__cvta_generic_to_shared(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // block -> (image, tile, filter group); groups vary fastest: blocks that run together share activations in L2
    const unsigned r1 = fdiv(blockIdx.x, p.d_groups);
    const int grp = (int)(blockIdx.x - r1 * p.n_groups);
    const unsigned img = fdiv(r1, p.d_tiles);
    const int tile = (int)(r1 - img * p.tiles);
    const int q0 = p.q_start + tile * (32 * T);
    const float *ximg = p.x + (size_t)img * p.c_in * p.pitch;

    const int KS = 1 << p.ks_shift;
    const int rslot = warp >> p.ks_shift, slice = warp & (KS - 1);

    // which of this lane's positions are interior (stored)
    unsigned okmask = 0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = q0 + 32 * t + lane;
        const int row = (int)fdiv((unsigned)q, p.d_wp);
        const int col = q - row * p.wp;
        if (row >= kPlanarHalo && row < kPlanarHalo + p.h && col >= kPlanarHalo && col < kPlanarHalo + p.w) okmask |= 1u << t;
    }
    // filters of this warp and their epilogue constants (independent of the previous layer)
    int co_of[RPW];
#pragma unroll
    for (int j = 0; j < RPW; ++j) co_of[j] = p.perm[grp * p.G + rslot * RPW + j];

    float acc[RPW][T];
#pragma unroll
    for (int j = 0; j < RPW; ++j)
#pragma unroll
        for (int t = 0; t < T; ++t) acc[j][t] = 0.0f;

    // ---- pipeline prologue: weights first, activations after the grid-dependency wait ----
    const int S = p.stages;
    const int npre = (S == 1) ? 1 : S - 1;
    for (int s = 0; s < npre; ++s)
        if (s < p.n_chunks) ps_stage_weights(p, smem32 + (unsigned)(s * p.stage_bytes), s, grp);
    grid_dep_wait();
    for (int s = 0; s < npre; ++s) {
        if (s < p.n_chunks) ps_stage_acts(p, ximg, smem32 + (unsigned)(s * p.stage_bytes), s, q0);
        cp_commit();
    }

    // epilogue constants: their loads are in flight while the first chunk arrives
    float sc[RPW], bi[RPW];
#pragma unroll
    for (int j = 0; j < RPW; ++j) {
        sc[j] = (p.scale && co_of[j] >= 0) ? p.scale[co_of[j]] : 1.0f;
        bi[j] = (p.bias && co_of[j] >= 0) ? p.bias[co_of[j]] : 0.0f;
    }

    int buf = 0;
    for (int c = 0; c < p.n_chunks; ++c) {
        if (S == 1) {
            if (c > 0) {
                __syncthreads();   // everyone is done with chunk c - 1
                ps_stage_weights(p, smem32, c, grp);
                ps_stage_acts(p, ximg, smem32, c, q0);
                cp_commit();
            }
            cp_wait<0>();
            __syncthreads();
        } else {
            if (S == 3) cp_wait<1>(); else cp_wait<0>();
            __syncthreads();   // chunk c has landed for everyone; everyone is done with chunk c - 1
            const int nxt = c + S - 1;
            int nbuf = buf + S - 1;
            if (nbuf >= S) nbuf -= S;
            if (nxt < p.n_chunks) {
                ps_stage_weights(p, smem32 + (unsigned)(nbuf * p.stage_bytes), nxt, grp);
                ps_stage_acts(p, ximg, smem32 + (unsigned)(nbuf * p.stage_bytes), nxt, q0);
            }
            cp_commit();
        }
        const unsigned stage_off = (unsigned)(buf * p.stage_bytes);
        const int *sP = reinterpret_cast<const int *>(smem + stage_off + p.tile_bytes);
        const unsigned sW = stage_off + p.tile_bytes + p.hdr_bytes;
        const unsigned lanep = stage_off + lane * 4;
#pragma unroll
        for (int j = 0; j < RPW; ++j) {
            const int seg = ((rslot * RPW + j) << p.ks_shift) + slice;
            const int beg = sP[seg], end = sP[seg + 1];
            // A batch of P pairs of nonzeros is read with broadcast loads one batch ahead; the batch's
            // activation loads are all issued before its first multiply-add, so that a warp keeps
            // 2 * P * T shared-memory loads in flight (with few warps per SM nothing else hides
            // their latency).  Slots past the end of the segment get weight 0 (their offsets
            // point inside the tile; the packer leaves two batches of slack behind a record).
            constexpr int P = T == 1 ? 4 : T <= 4 ? 2 : 1;
            uint4 nx[P];
#pragma unroll
            for (int i = 0; i < P; ++i) nx[i] = *reinterpret_cast<const uint4 *>(smem + sW + (beg + 2 * i) * 8);
            for (int e = beg; e < end; e += 2 * P) {
                uint4 v[P];
#pragma unroll
                for (int i = 0; i < P; ++i) {
                    v[i] = nx[i];
                    if (P > 1 && e + 2 * i >= end) v[i].x = v[i].z = 0u;
                }
#pragma unroll
                for (int i = 0; i < P; ++i) nx[i] = *reinterpret_cast<const uint4 *>(smem + sW + (e + 2 * P + 2 * i) * 8);
                float a[P][2][T];
#pragma unroll
                for (int i = 0; i < P; ++i)
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        a[i][0][t] = *reinterpret_cast<const float *>(smem + lanep + v[i].y + t * 128);
                        a[i][1][t] = *reinterpret_cast<const float *>(smem + lanep + v[i].w + t * 128);
                    }
#pragma unroll
                for (int i = 0; i < P; ++i) {
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] = fmaf(__uint_as_float(v[i].x), a[i][0][t], acc[j][t]);
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] = fmaf(__uint_as_float(v[i].z), a[i][1][t], acc[j][t]);
                }
            }
        }
        if (++buf == S) buf = 0;
    }
    cp_wait<0>();

    // ---- warps that share a filter: partial sums meet in shared memory (the stages are free now) ----
    if (KS > 1) {
        __syncthreads();
        float *sRed = reinterpret_cast<float *>(smem);
        if (slice > 0) {
            float *dst = sRed + (size_t)((rslot * (KS - 1) + slice - 1) * RPW) * T * 32 + lane;
#pragma unroll
            for (int j = 0; j < RPW; ++j)
#pragma unroll
                for (int t = 0; t < T; ++t) dst[(j * T + t) * 32] = acc[j][t];
        }
        __syncthreads();
        if (slice == 0) {
            for (int s2 = 1; s2 < KS; ++s2) {
                const float *srcp = sRed + (size_t)((rslot * (KS - 1) + s2 - 1) * RPW) * T * 32 + lane;
#pragma unroll
                for (int j = 0; j < RPW; ++j)
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += srcp[(j * T + t) * 32];
            }
        }
    }
    grid_dep_trigger();

    // ---- epilogue: every lane stores its own positions, contiguous in the output plane ----
    if (slice == 0) {
#pragma unroll
        for (int j = 0; j < RPW; ++j) {
            const int co = co_of[j];
            if (co < 0) continue;
            const size_t obase = ((size_t)img * p.c_out + co) * p.pitch + q0 + lane;
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (okmask & (1u << t)) {
                    const size_t oi = obase + 32 * t;
                    float z = fmaf(acc[j][t], sc[j], bi[j]);
                    if (p.residual) z += p.residual[oi];
                    p.y[oi] = ps_act(z, p.act);
                }
            }
        }
    }
}

template <int T, int RPW>
cadnn_status ps_launch_one(const PsParams &p, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    auto kern = sconv_planar_staged_kernel<T, RPW>;
    static int smem_allowed = 48 * 1024;   // raised once per instantiation, as layers need it
    if (smem > smem_allowed) {
        CADNN_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        smem_allowed = smem;
    }
    return launch_kernel(kern, blocks, threads, (size_t)smem, pdl, st, p);
}

template <int T>
cadnn_status ps_launch_rpw(const PsParams &p, int rpw, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    switch (rpw) {
        case 1: return ps_launch_one<T, 1>(p, blocks, threads, smem, pdl, st);
        case 2: return ps_launch_one<T, 2>(p, blocks, threads, smem, pdl, st);
        case 4: return ps_launch_one<T, 4>(p, blocks, threads, smem, pdl, st);
        case 8: if (T <= 4) return ps_launch_one<(T <= 4 ? T : 1), 8>(p, blocks, threads, smem, pdl, st); break;
    }
    return CADNN_E_UNSUPPORTED;
}

}  // namespace

cadnn_status launch_sconv_planar_staged(const cadnn_weights *w, const void *x, int n, void *y, const LaunchEpilogue &ep,
                                        cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    const PsSchedule &s = w->ps;
    PsParams p;
    p.x = (const float *)x; p.y = (float *)y;
    p.ent = w->d_ps_ent; p.perm = w->d_ps_perm;
    p.scale = ep.scale; p.bias = ep.bias; p.residual = (const float *)ep.residual;
    p.c_in = d.c_in; p.c_out = d.c_out;
    p.h = d.in_h; p.w = d.in_w; p.wp = d.in_w + 2 * kPlanarHalo; p.pitch = planar_pitch(d.in_h, d.in_w);
    p.q_start = s.q_start; p.tiles = s.tiles;
    p.A = s.A; p.L = s.L;
    p.CIc = s.CIc; p.n_chunks = s.n_chunks; p.G = s.G; p.n_groups = s.n_groups; p.stages = s.stages;
    p.ks_shift = s.KS >= 8 ? 3 : s.KS >= 4 ? 2 : s.KS >= 2 ? 1 : 0;
    p.tile_bytes = s.tile_bytes; p.stage_bytes = s.stage_bytes; p.hdr_bytes = s.hdr_bytes; p.block_bytes = s.block_bytes;
    p.act = ep.act;
    p.d_groups = make_fastdiv(s.n_groups);
    p.d_tiles = make_fastdiv(s.tiles);
    p.d_wp = make_fastdiv(p.wp);
    p.d_l4 = make_fastdiv(s.L >> 2);
    const long long blocks = (long long)n * s.tiles * s.n_groups;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    const int threads = s.NW * 32;
    switch (s.T) {
        case 1: return ps_launch_rpw<1>(p, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 2: return ps_launch_rpw<2>(p, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 4: return ps_launch_rpw<4>(p, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 8: return ps_launch_rpw<8>(p, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
    }
    return CADNN_E_UNSUPPORTED;
}
