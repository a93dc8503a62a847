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
//
// Two ways of staging: 16-byte cp.async copies issued by all threads, or (schedule flag tma) one
// thread issuing TMA copies - a 2-D tensor copy per box of up to 256 channels x L floats of the
// [n * c_in][pitch] view of x (out-of-range columns and rows are zero-filled by the unit) and a
// bulk copy of the weight record - that complete on one mbarrier per stage, so the other
// warps spend no issue slots on staging and several chunks are in flight from the first cycles.
#include <algorithm>
#include <cuda.h>
#include "cadnn_internal.h"

// set when a wait on a copy barrier ran out (never expected; the kernel then finishes with
// whatever it has, and cadnn_device_status reports it)
__device__ int g_copy_timeout;

cadnn_status read_copy_timeouts(int *count)
{
    int v = 0;
    CADNN_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_copy_timeout, sizeof(int)));
    *count = v;
    return CADNN_OK;
}

cadnn_status read_copy_timeouts_async(int *host_dst, cudaStream_t st)
{
    CADNN_CUDA_TRY(cudaMemcpyFromSymbolAsync(host_dst, g_copy_timeout, sizeof(int), 0, cudaMemcpyDeviceToHost, st));
    return CADNN_OK;
}

cadnn_status write_copy_timeouts(int value)
{
    CADNN_CUDA_TRY(cudaMemcpyToSymbol(g_copy_timeout, &value, sizeof(int)));
    return CADNN_OK;
}

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
    int h, w, wp, pitch;   // input: interior size, padded row length, floats between planes
    int h_out, w_out, wp_out, pitch_out;   // output (the same numbers at stride 1)
    int stride, R, lead_rows;   // row-tile mode (R > 0): output rows per tile; first staged input row = stride * oy0 + lead_rows
    int q_start, tiles;    // first computed position (a multiple of 4), tiles of 32 * T positions per image
    int A, L;              // staged margin on either side and staged floats per channel (multiples of 4)
    int CIc, n_chunks, G, n_groups, stages;
    int ks_shift;
    int tile_bytes, stage_bytes, hdr_bytes, block_bytes;
    int act;
    int kc_shift, chunks_per_rank;   // TMA kernel: log2 of the blocks per cluster that split the channel chunks; chunks each takes
    int part_off;          // byte offset of the cluster partial sums in shared memory
    int early_trigger;     // as a programmatic primary: let the next layer's prologue start at once
    int RB, nb, bar_off;   // TMA staging: rows per box, boxes per chunk, byte offset of the stage barriers
    FastDiv d_groups, d_tiles, d_wp, d_wp_out, d_l4;
    ParityPlanes par;      // second copy of the output for a stride-2 reader (par.y null = none)
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

// thread-block cluster helpers (all threads of all blocks of the cluster call cluster_sync)
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ unsigned map_shared_rank(unsigned addr, unsigned rank)
{
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_shared_cluster(unsigned addr)
{
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];\n" : "=f"(v) : "r"(addr) : "memory");
    return v;
}

// multiply-adds of one staged chunk for the filters of this warp
// (ROWS: the lane's positions are not 32 t apart in the tile, their byte offsets come in lb[])
template <int T, int RPW, bool ROWS = false>
__device__ __forceinline__ void ps_compute_chunk(const PsParams &p, const unsigned char *smem, unsigned stage_off, int lane,
                                                 int rslot, int slice, float (&acc)[RPW][T], const unsigned *lb = nullptr)
{
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
                    if (ROWS) {
                        a[i][0][t] = *reinterpret_cast<const float *>(smem + stage_off + lb[t] + v[i].y);
                        a[i][1][t] = *reinterpret_cast<const float *>(smem + stage_off + lb[t] + v[i].w);
                    } else {
                        a[i][0][t] = *reinterpret_cast<const float *>(smem + lanep + v[i].y + t * 128);
                        a[i][1][t] = *reinterpret_cast<const float *>(smem + lanep + v[i].w + t * 128);
                    }
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
}

// partial sums of the warps that share a filter, epilogue, stores
template <int T, int RPW>
__device__ __forceinline__ void ps_block_tail(const PsParams &p, unsigned char *smem, int lane, int rslot, int slice, int KS,
                                              unsigned img, int q0, unsigned okmask, const int (&co_of)[RPW],
                                              const float (&sc)[RPW], const float (&bi)[RPW], float (&acc)[RPW][T],
                                              int KC = 1, int rank = 0, const float (*res)[T] = nullptr)
{
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
    if (!p.early_trigger) grid_dep_trigger();

    // ---- blocks of a cluster that split the input channels: every block leaves its partial sums in
    // its shared memory; filter slot r is then finished by the block whose rank is r mod KC, which
    // adds the other blocks' partial sums read over distributed shared memory ----
    if (KC > 1) {
        float *sPart = reinterpret_cast<float *>(smem + p.part_off);
        __syncthreads();   // the stages are free: every warp has finished its multiply-adds
        if (slice == 0) {
#pragma unroll
            for (int j = 0; j < RPW; ++j)
#pragma unroll
                for (int t = 0; t < T; ++t) sPart[((rslot * RPW + j) * T + t) * 32 + lane] = acc[j][t];
        }
        cluster_sync();   // every block's partial sums are in place
        if (slice == 0) {
            const unsigned mine = (unsigned)__cvta_generic_to_shared(sPart);
#pragma unroll
            for (int j = 0; j < RPW; ++j) {
                const int slot = rslot * RPW + j;
                if ((slot & (KC - 1)) != rank) continue;
                for (int k = 1; k < KC; ++k) {
                    const unsigned peer = map_shared_rank(mine + (unsigned)((slot * T) * 32 + lane) * 4u, (unsigned)((rank + k) & (KC - 1)));
#pragma unroll
                    for (int t = 0; t < T; ++t) acc[j][t] += ld_shared_cluster(peer + t * 128);
                }
            }
        }
    }

    // ---- epilogue: every lane stores its own positions, contiguous in the output plane ----
    if (slice == 0) {
#pragma unroll
        for (int j = 0; j < RPW; ++j) {
            const int co = co_of[j];
            if (co < 0 || (KC > 1 && ((rslot * RPW + j) & (KC - 1)) != rank)) continue;
            const size_t obase = ((size_t)img * p.c_out + co) * p.pitch_out + q0 + lane;
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (okmask & (1u << t)) {
                    const size_t oi = obase + 32 * t;
                    float z = fmaf(acc[j][t], sc[j], bi[j]);
                    if (res) z += res[j][t];               // fetched before the multiply-add loop
                    else if (p.residual) z += p.residual[oi];
                    z = ps_act(z, p.act);
                    p.y[oi] = z;
                    if (p.par.y) {
                        const int q = q0 + lane + 32 * t;
                        const int row = (int)fdiv((unsigned)q, p.d_wp_out);
                        parity_store(p.par, img, co, row - kPlanarHalo, q - row * p.wp_out - kPlanarHalo, z);
                    }
                }
            }
        }
    }
    if (KC > 1) cluster_sync();   // peers may still be reading this block's partial sums
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
        ps_compute_chunk<T, RPW>(p, smem, (unsigned)(buf * p.stage_bytes), lane, rslot, slice, acc);
        if (++buf == S) buf = 0;
    }
    cp_wait<0>();

    ps_block_tail<T, RPW>(p, smem, lane, rslot, slice, KS, img, q0, okmask, co_of, sc, bi, acc);
}


// ---- TMA staging ----

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\nselp.u32 %0, 1, 0, q;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Wait for a stage's copies.  The wait is bounded: if the barrier has not completed after
// about a second the block records it and goes on (its results are then wrong, and the host
// learns of it through the flag), after a second bounded wait that lets copies in flight land.
__device__ __forceinline__ void mbar_wait(unsigned bar, unsigned parity)
{
    for (int it = 0; it < (1 << 22); ++it)
        if (mbar_try_wait(bar, parity)) return;
    atomicAdd(&g_copy_timeout, 1);
    for (int it = 0; it < (1 << 22); ++it)
        if (mbar_try_wait(bar, parity)) return;
}
__device__ __forceinline__ void bulk_copy(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tensor_copy_2d(unsigned dst, const CUtensorMap *map, int x, int y, unsigned bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// one thread: start the copies of chunk c into stage `buf`; the weight record first (it never
// depends on the previous layer), the activation boxes after `before_acts` has run
template <class F>
__device__ __forceinline__ void ps_tma_issue(const PsParams &p, const CUtensorMap *map, unsigned smem32, int buf, int c, int grp,
                                             int row0, int xq, bool weights, bool acts, F before_acts)
{
    const unsigned bar = smem32 + p.bar_off + buf * 8;
    const unsigned st32 = smem32 + (unsigned)(buf * p.stage_bytes);
    if (weights) {
        mbar_expect_tx(bar, (unsigned)(p.tile_bytes + p.block_bytes));
        const unsigned char *rec = reinterpret_cast<const unsigned char *>(p.ent) + ((size_t)c * p.n_groups + grp) * p.block_bytes;
        bulk_copy(st32 + p.tile_bytes, rec, (unsigned)p.block_bytes, bar);
    }
    before_acts();
    if (acts) {
        const unsigned box_bytes = (unsigned)(p.RB * p.L * 4);
        for (int b = 0; b < p.nb; ++b) tensor_copy_2d(st32 + b * box_bytes, map, xq, row0 + c * p.CIc + b * p.RB, bar);
    }
}

template <int T, int RPW, bool ROWS>
__global__ void __launch_bounds__(512) sconv_planar_tma_kernel(const PsParams p, const __grid_constant__ CUtensorMap tmap)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const unsigned smem32 = (unsigned)__cvta_generic_to_shared(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // consecutive blocks form a cluster: same tile and filters, consecutive ranges of the channel chunks
    const int KC = 1 << p.kc_shift;
    const int rank = (int)(blockIdx.x & (unsigned)(KC - 1));
    const unsigned rest = blockIdx.x >> p.kc_shift;
    const unsigned r1 = fdiv(rest, p.d_groups);
    const int grp = (int)(rest - r1 * p.n_groups);
    const unsigned img = fdiv(r1, p.d_tiles);
    const int tile = (int)(r1 - img * p.tiles);
    // linear mode: 32 T consecutive positions of the (common) plane, staged with a margin of A on
    // either side.  Row-tile mode (any stride): R output rows; the staged run starts at the input
    // row of their first tap, rounded down to 16 bytes (`lead` floats of slack in front).
    const int q0 = ROWS ? (kPlanarHalo + tile * p.R) * p.wp_out : p.q_start + tile * (32 * T);
    int xq = q0 - p.A, lead = 0;
    if (ROWS) {
        const int run = (p.stride * tile * p.R + p.lead_rows) * p.wp;
        xq = run & ~3;
        lead = run - xq;
    }
    const int S = p.stages;
    const int my_chunks = p.chunks_per_rank, c_first = rank * my_chunks;
    const int npre = min(S, my_chunks);

    // Everything up to the grid-dependency wait touches only constants of the layer, so as a
    // programmatic dependent it overlaps the tail of the previous layer: barriers, the weight
    // records of the first stages, the filter permutation and the epilogue vectors.
    if (p.early_trigger) grid_dep_trigger();
    if (tid == 0) {
        for (int s = 0; s < S; ++s) mbar_init(smem32 + p.bar_off + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&tmap) : "memory");
    }
    if (warp == 0) {
        // lane s starts the copies of stage s: issuing a copy takes a few hundred clocks, and the lanes' issues overlap
        __syncwarp();
        if (lane < npre) ps_tma_issue(p, &tmap, smem32, lane, c_first + lane, grp, 0, 0, true, false, [] {});
    }
    const int KS = 1 << p.ks_shift;
    const int rslot = warp >> p.ks_shift, slice = warp & (KS - 1);
    int co_of[RPW];
#pragma unroll
    for (int j = 0; j < RPW; ++j) co_of[j] = p.perm[grp * p.G + rslot * RPW + j];
    unsigned okmask = 0;
    unsigned lb[T];
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = q0 + 32 * t + lane;
        const int row = (int)fdiv((unsigned)q, p.d_wp_out);
        const int col = q - row * p.wp_out;
        bool ok = row >= kPlanarHalo && row < kPlanarHalo + p.h_out && col >= kPlanarHalo && col < kPlanarHalo + p.w_out;
        lb[t] = 0;
        if (ROWS) {
            const int ro = row - kPlanarHalo - tile * p.R;   // output row inside the tile
            ok = ok && ro < p.R;
            // lanes that store nothing still load: from the tile's first position
            lb[t] = ok ? (unsigned)((p.stride * ro * p.wp + p.stride * (col - kPlanarHalo) + lead) * 4) : (unsigned)(lead * 4);
        }
        if (ok) okmask |= 1u << t;
    }
    float acc[RPW][T];
#pragma unroll
    for (int j = 0; j < RPW; ++j)
#pragma unroll
        for (int t = 0; t < T; ++t) acc[j][t] = 0.0f;

    grid_dep_wait();   // x (and the residual) are final from here on
    if (warp == 0 && lane < npre) ps_tma_issue(p, &tmap, smem32, lane, c_first + lane, grp, (int)img * p.c_in, xq, false, true, [] {});
    float sc[RPW], bi[RPW];
#pragma unroll
    for (int j = 0; j < RPW; ++j) {
        sc[j] = (p.scale && co_of[j] >= 0) ? p.scale[co_of[j]] : 1.0f;
        bi[j] = (p.bias && co_of[j] >= 0) ? p.bias[co_of[j]] : 0.0f;
    }
    // the residual is requested now, so that its round trip to L2 overlaps the multiply-add loop
    float res[RPW][T];
#pragma unroll
    for (int j = 0; j < RPW; ++j)
#pragma unroll
        for (int t = 0; t < T; ++t) {
            res[j][t] = 0.0f;
            if (p.residual && slice == 0 && co_of[j] >= 0 && (okmask & (1u << t)))
                res[j][t] = ld_act(p.residual + ((size_t)img * p.c_out + co_of[j]) * p.pitch_out + q0 + lane + 32 * t);
        }
    __syncthreads();   // the barriers are initialised for everyone

    int buf = 0;
    unsigned parity = 0;
    for (int c = 0; c < my_chunks; ++c) {
        mbar_wait(smem32 + p.bar_off + buf * 8, parity);
        ps_compute_chunk<T, RPW, ROWS>(p, smem, (unsigned)(buf * p.stage_bytes), lane, rslot, slice, acc, lb);
        if (c + S < my_chunks) {
            __syncthreads();   // everyone is done with this stage
            if (tid == 0) {
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // reads above before the unit's writes
                ps_tma_issue(p, &tmap, smem32, buf, c_first + c + S, grp, (int)img * p.c_in, xq, true, true, [] {});
            }
        }
        if (++buf == S) {
            buf = 0;
            parity ^= 1u;
        }
    }
    ps_block_tail<T, RPW>(p, smem, lane, rslot, slice, KS, img, q0, okmask, co_of, sc, bi, acc, KC, rank,
                          p.residual ? res : nullptr);
}

template <int T, int RPW>
cadnn_status ps_launch_one(const PsParams &p, const CUtensorMap *map, int blocks, int threads, int smem, bool pdl, cudaStream_t st)
{
    if (map) {
        auto kern = p.R > 0 ? sconv_planar_tma_kernel<T, RPW, true> : sconv_planar_tma_kernel<T, RPW, false>;
        static SmemLimit lim[2];   // per instantiation (row-tile / linear), per device
        if (smem > 48 * 1024) {
            cadnn_status rs = raise_smem_limit((const void *)kern, smem, &lim[p.R > 0 ? 1 : 0]);
            if (rs != CADNN_OK) return rs;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks, 1, 1);
        cfg.blockDim = dim3((unsigned)threads, 1, 1);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        int na = 0;
        if (p.kc_shift > 0) {
            attr[na].id = cudaLaunchAttributeClusterDimension;
            attr[na].val.clusterDim.x = 1u << p.kc_shift;
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
        CADNN_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, p, *map));
        return CADNN_OK;
    }
    auto kern = sconv_planar_staged_kernel<T, RPW>;
    static SmemLimit lim;
    if (smem > 48 * 1024) {
        cadnn_status rs = raise_smem_limit((const void *)kern, smem, &lim);
        if (rs != CADNN_OK) return rs;
    }
    return launch_kernel(kern, blocks, threads, (size_t)smem, pdl, st, p);
}

template <int T>
cadnn_status ps_launch_rpw(const PsParams &p, const CUtensorMap *map, int rpw, int blocks, int threads, int smem, bool pdl,
                           cudaStream_t st)
{
    switch (rpw) {
        case 1: return ps_launch_one<T, 1>(p, map, blocks, threads, smem, pdl, st);
        case 2: return ps_launch_one<T, 2>(p, map, blocks, threads, smem, pdl, st);
        case 4: return ps_launch_one<T, 4>(p, map, blocks, threads, smem, pdl, st);
        case 8: if (T <= 4) return ps_launch_one<(T <= 4 ? T : 1), 8>(p, map, blocks, threads, smem, pdl, st); break;
    }
    return CADNN_E_UNSUPPORTED;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against the driver library)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
        else
            cudaGetLastError();
    }
    return fn;
}

}  // namespace

bool encode_plane_rows_map(void *map, const void *base, unsigned long long cols, unsigned long long rows,
                           unsigned box_cols, unsigned box_rows)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(reinterpret_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), dims, strides,
               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_nhwc_s8_tiles_map(void *map, const void *base, int c, int w, int h, int n, int box_c, int box_w, int box_h)
{
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[4] = {(cuuint64_t)c, (cuuint64_t)w, (cuuint64_t)h, (cuuint64_t)n};
    const cuuint64_t strides[3] = {(cuuint64_t)c, (cuuint64_t)c * w, (cuuint64_t)c * w * h};
    const cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(reinterpret_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void *>(base), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

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
    p.h_out = w->h_out; p.w_out = w->w_out; p.wp_out = w->w_out + 2 * kPlanarHalo; p.pitch_out = planar_pitch(w->h_out, w->w_out);
    p.stride = d.stride; p.R = s.R; p.lead_rows = kPlanarHalo - d.pad;
    if (s.R > 0 && !s.tma) return CADNN_E_UNSUPPORTED;
    p.q_start = s.q_start; p.tiles = s.tiles;
    p.A = s.A; p.L = s.L;
    p.CIc = s.CIc; p.n_chunks = s.n_chunks; p.G = s.G; p.n_groups = s.n_groups; p.stages = s.stages;
    p.ks_shift = s.KS >= 8 ? 3 : s.KS >= 4 ? 2 : s.KS >= 2 ? 1 : 0;
    p.tile_bytes = s.tile_bytes; p.stage_bytes = s.stage_bytes; p.hdr_bytes = s.hdr_bytes; p.block_bytes = s.block_bytes;
    p.act = ep.act;
    p.par = parity_planes(ep.parity_y, ep.parity_mask, w->h_out, w->w_out, d.c_out);
    p.early_trigger = ep.early_trigger ? 1 : 0;
    p.d_groups = make_fastdiv(s.n_groups);
    p.d_tiles = make_fastdiv(s.tiles);
    p.d_wp = make_fastdiv(p.wp);
    p.d_wp_out = make_fastdiv(p.wp_out);
    p.d_l4 = make_fastdiv(s.L >> 2);
    const int kc = s.tma ? std::max(1, s.KC) : 1;
    p.kc_shift = kc >= 8 ? 3 : kc >= 4 ? 2 : kc >= 2 ? 1 : 0;
    p.chunks_per_rank = s.n_chunks / kc;
    p.part_off = s.part_off;
    const long long blocks = (long long)n * s.tiles * s.n_groups * kc;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    const int threads = s.NW * 32;
    CUtensorMap map;
    const CUtensorMap *mp = nullptr;
    if (s.tma) {
        // x as a matrix of n * c_in rows (planes) by pitch columns; a box is RB rows by L columns
        EncodeTiledFn enc = encode_tiled_fn();
        if (!enc) return CADNN_E_UNSUPPORTED;
        const cuuint64_t dims[2] = {(cuuint64_t)p.pitch, (cuuint64_t)n * (cuuint64_t)d.c_in};
        const cuuint64_t strides[1] = {(cuuint64_t)p.pitch * 4};
        const cuuint32_t box[2] = {(cuuint32_t)s.L, (cuuint32_t)s.RB};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(x), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CADNN_E_UNSUPPORTED;
        mp = &map;
        p.RB = s.RB; p.nb = s.nb; p.bar_off = s.stages * s.stage_bytes;
    } else {
        p.RB = 0; p.nb = 0; p.bar_off = 0;
    }
    switch (s.T) {
        case 1: return ps_launch_rpw<1>(p, mp, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 2: return ps_launch_rpw<2>(p, mp, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 4: return ps_launch_rpw<4>(p, mp, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
        case 8: return ps_launch_rpw<8>(p, mp, s.RPW, (int)blocks, threads, s.smem_bytes, ep.pdl, st);
    }
    return CADNN_E_UNSUPPORTED;
}
