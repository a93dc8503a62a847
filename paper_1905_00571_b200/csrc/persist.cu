// Persistent whole-network kernel for runs of sparse convolutions over channel-planar
// activations.
//
// CADNN (arXiv 1905.00571), Section 4, "Model computation fusion and transformation": layers
// are fused into larger kernels to cut the cost between them.  At batch 1 a pruned layer's
// work (a fraction of a microsecond at the machine's peak) is far below the cost of a kernel
// boundary (launch ramp and drain), so a whole run of sparse conv layers executes inside ONE
// cooperative kernel of one thread block per SM:
//   * who does what is decided on the host when the net is created ("Optimization parameters
//     selection"): per layer a tile size (bands of 32 consecutive plane positions), a split of
//     the filters into groups, and the dealing of (filter, bands) units to the 15 compute warps
//     of a block by longest processing time.  A block's share of a layer is one ITEM, and the
//     item's weights are stored as one contiguous record {header, units, nonzeros as
//     {value, byte offset into the staged tile}} in the order that block walks them;
//   * a control warp fetches the record of the block's NEXT item with one bulk copy while the
//     current item computes (weights never depend on a previous layer), and, once the layer's
//     inputs are final, stages the item's activation tile - for every input channel one
//     contiguous run of its plane - with 2-D TMA tensor copies, a few channel chunks each on its
//     own mbarrier, so that the multiply-adds of the first chunk overlap the arrival of the rest;
//   * the lanes of a compute warp are 32 consecutive positions (conflict-free shared-memory loads
//     for any tap), a unit's nonzeros are broadcast two at a time and feed T multiply-adds per
//     lane; scale, bias, residual and activation are applied to the registers and stored;
//   * input tiles larger than shared memory are taken in several passes over channel ranges with
//     the partial sums parked in shared memory;
//   * layers that do not read each other's output (a bottleneck's downsample branch and its first
//     1x1 conv) share a phase and split the blocks in proportion to their work; between phases all
//     blocks meet at a barrier in global memory (release / acquire at device scope).
// Every wait - on a copy barrier or on the grid barrier - is bounded: a block that gives up raises
// a device flag (see cadnn_device_status) and carries on to the end.  No multicast copies.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>
#include <cuda.h>
#include "cadnn_internal.h"

// set when a wait of the persistent kernel ran out (never expected)
__device__ int g_barrier_timeout;

cadnn_status read_barrier_timeouts(int *count)
{
    int v = 0;
    CADNN_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_barrier_timeout, sizeof(int)));
    *count = v;
    return CADNN_OK;
}

cadnn_status read_barrier_timeouts_async(int *host_dst, cudaStream_t st)
{
    CADNN_CUDA_TRY(cudaMemcpyFromSymbolAsync(host_dst, g_barrier_timeout, sizeof(int), 0, cudaMemcpyDeviceToHost, st));
    return CADNN_OK;
}

cadnn_status write_barrier_timeouts(int value)
{
    CADNN_CUDA_TRY(cudaMemcpyToSymbol(g_barrier_timeout, &value, sizeof(int)));
    return CADNN_OK;
}

namespace {

const int kPnWarps = 15;                       // compute warps per block (with the control warp: 512 threads, 128 registers each)
const int kPnThreads = (kPnWarps + 1) * 32;    // + one control warp
const int kPnMaxSeg = 8;                       // channel chunks of a layer, all passes together
const int kPnMaxCpp = 4;                       // chunks (copy barriers) per pass
const int kPnMaxT = 4;                         // bands of 32 positions a unit covers at most
const unsigned kSpinLimit = 1u << 22;          // polls before a wait gives up (seconds)
const int kPnSmemMax = 227 * 1024;
const int kPnPhaseEnd = 0x7fffffff;
const int kPnMaxLayers = 96;                   // tensor maps travel as a kernel parameter (128 bytes each)

// The layers' tensor maps, passed by value: a copy engine fetches a map it has not seen from wherever
// it lives, and from the parameter space that is a hit in the constant cache instead of a trip to L2.
struct PnMaps {
    CUtensorMap m[kPnMaxLayers];
};

// One block's share of one layer (global memory; the control warp reads it one item ahead).
struct PnItem {
    int phase;            // kPnPhaseEnd terminates a block's list
    int layer;            // index of the layer's tensor map
    unsigned rec_off;     // byte offset of the record (16-byte aligned)
    int rec_bytes;        // a multiple of 16
    int x0, row0;         // tensor coordinates of the tile's first chunk: element of a plane (a multiple of 4, may be negative), plane
    int L, CIc;           // staged floats per channel (box width), channels per chunk
    int RB, nrb;          // channel rows per box, boxes per chunk
    int cpp, passes;      // chunks per pass, passes
    int T, strided;       // kernel variant: bands per unit, lane addresses not consecutive (stride 2)
    int pad0, pad1;
};
static_assert(sizeof(PnItem) == 64, "PnItem is copied as four 16-byte words");

struct PnUnit {           // (filter, up to T bands of the tile): the work of one warp at a time
    int co;               // output channel
    int band0, nb;        // first band inside the tile, bands
    int e_begin;          // first entry (even index into the record's entries)
    int e_end[kPnMaxSeg]; // end of the unit's entries in channel chunk s (even; the tail of a segment is padding)
    float scale, bias;    // folded BatchNorm of the output channel
};
static_assert(sizeof(PnUnit) == 56, "unit layout");

struct alignas(16) PnHdr { // head of a record
    float *y;             // output planes of the item's image, or null when only the parity planes are read
    const float *res;     // residual planes of the item's image or null
    int q0;               // first output position of the tile
    int n_units;
    int ent_off, unit_off;   // byte offsets inside the record
    int wp_out, h_out, w_out, pitch_out;
    unsigned dmul, dshr;  // division by wp_out
    int stride, wp_in;
    int act, lb_bias;     // lane address = (origin of the lane's position + lb_bias) * 4: lb_bias = first tap offset - x0
    int bs;               // positions per band (32; fewer where a band is whole rows of a strided layer's output)
    int par_mask;         // parity planes written to y2: bit (row parity * 2 + column parity)
    int wp2, pitch2;      // parity planes: padded row length, floats per plane
    float *y2;            // parity planes of the item's image [4 or 1][c_out][pitch2] or null
    int c2_stride;        // planes between two parities (c_out)
    int pad;
    int wbeg[kPnWarps + 1];   // units of warp w: [wbeg[w], wbeg[w + 1])
};
static_assert(sizeof(PnHdr) % 16 == 0, "record head keeps 16-byte alignment");

struct PnLayout {         // byte offsets inside dynamic shared memory
    int wbuf[2];          // the two record buffers
    int tile;             // staged activations
    int part;             // partial sums between passes
    int bars;             // mbarriers: record barriers [2], then chunk barriers [kPnMaxCpp]
    int items;            // PnItem[2]
};

__device__ __forceinline__ float pn_act(float z, int act)
{
    if (act == CADNN_ACT_RELU) return z > 0.0f ? z : 0.0f;
    if (act == CADNN_ACT_RELU6) return fminf(z > 0.0f ? z : 0.0f, 6.0f);
    return z;
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release(unsigned *p, unsigned v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;\n" ::"l"(p), "r"(v) : "memory");
}
// L2-only load: the residual was written by another SM earlier in this same kernel
__device__ __forceinline__ float ld_cg(const float *p)
{
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];\n" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void pn_mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void pn_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool pn_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\nselp.u32 %0, 1, 0, q;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait on a copy barrier: gives up after about a second, records it, and lets copies in
// flight land during a second bounded wait
__device__ __forceinline__ void pn_mbar_wait(unsigned bar, unsigned parity)
{
    for (unsigned it = 0; it < kSpinLimit; ++it)
        if (pn_try_wait(bar, parity)) return;
    atomicAdd(&g_barrier_timeout, 1);
    for (unsigned it = 0; it < kSpinLimit; ++it)
        if (pn_try_wait(bar, parity)) return;
}
__device__ __forceinline__ void pn_bulk_copy(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void pn_tensor_copy(unsigned dst, const CUtensorMap *map, int x, int y, unsigned bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                 ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}

// All blocks of the grid have finished the phase when this returns (or the wait ran out).  Called by
// one thread, after a block-wide barrier that followed the block's last store of the phase.
__device__ __forceinline__ void pn_grid_barrier(unsigned *arrive, unsigned target)
{
    // The release is cumulative: the stores of the block's other threads, ordered before this thread by
    // the block barrier, are visible device-wide before the count moves; the acquire orders everything
    // after it.  (The writers ordered their stores against the copy unit's reads with a proxy fence.)
    red_release(arrive, 1u);
    unsigned spins = 0;
    while (ld_acquire(arrive) < target) {
        if (++spins > kSpinLimit) {
            atomicAdd(&g_barrier_timeout, 1);
            break;
        }
    }
}

// multiply-adds of entries [beg, end) of a unit (pairs; both even) against the staged tile
template <int T, bool STRIDED>
__device__ __forceinline__ void pn_mac(const unsigned char *smem, unsigned ent, int beg, int end, unsigned tile,
                                       const unsigned (&lb)[T], float (&acc)[T])
{
    // A batch of P pairs of nonzeros is read with broadcast loads one batch ahead; the batch's
    // activation loads are all issued before its first multiply-add.  Slots past the end get weight 0;
    // their offsets stay inside the tile (they are the next entries of the record, or its zero tail), and
    // shared memory never holds anything but finite numbers.  (Requesting the NEXT batch's activations
    // before the current multiply-adds measured no faster and costs loads on short rows.)
    constexpr int P = T == 1 ? 4 : 2;
    uint4 nx[P];
#pragma unroll
    for (int i = 0; i < P; ++i) nx[i] = *reinterpret_cast<const uint4 *>(smem + ent + (beg + 2 * i) * 8);
    const unsigned base0 = tile + lb[0];
    for (int e = beg; e < end; e += 2 * P) {
        uint4 v[P];
#pragma unroll
        for (int i = 0; i < P; ++i) {
            v[i] = nx[i];
            if (e + 2 * i >= end) v[i].x = v[i].z = 0u;
        }
#pragma unroll
        for (int i = 0; i < P; ++i) nx[i] = *reinterpret_cast<const uint4 *>(smem + ent + (e + 2 * P + 2 * i) * 8);
        float a[P][2][T];
#pragma unroll
        for (int i = 0; i < P; ++i)
#pragma unroll
            for (int t = 0; t < T; ++t) {
                if (STRIDED) {
                    a[i][0][t] = *reinterpret_cast<const float *>(smem + tile + lb[t] + v[i].y);
                    a[i][1][t] = *reinterpret_cast<const float *>(smem + tile + lb[t] + v[i].w);
                } else {
                    a[i][0][t] = *reinterpret_cast<const float *>(smem + base0 + v[i].y + t * 128);
                    a[i][1][t] = *reinterpret_cast<const float *>(smem + base0 + v[i].w + t * 128);
                }
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

// what a lane needs to know about a unit: where its positions are and whether it stores them
template <int T>
struct PnLaneGeom {
    unsigned lb[T];     // byte offset of the lane's position inside a staged channel row, per band
    unsigned ok;        // bit t: the lane's position of band t is an interior position (stored)
    size_t obase;       // index of the lane's first position in the output (and residual) planes
};

template <int T, bool STRIDED>
__device__ __forceinline__ void pn_geometry(const PnHdr *h, const PnUnit &un, int lane, PnLaneGeom<T> &g)
{
    const int bs = h->bs, wp_out = h->wp_out;
    g.ok = 0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = h->q0 + bs * (un.band0 + (t < un.nb ? t : 0)) + lane;
        const int row = (int)(__umulhi((unsigned)q, h->dmul) >> h->dshr);
        const int col = q - row * wp_out;
        const bool v = t < un.nb && lane < bs && row >= kPlanarHalo && row < kPlanarHalo + h->h_out && col >= kPlanarHalo &&
                       col < kPlanarHalo + h->w_out;
        if (v) g.ok |= 1u << t;
        if (STRIDED)   // lanes that store nothing still load: from the tile's first element
            g.lb[t] = v ? (unsigned)((((row - kPlanarHalo) * h->stride) * h->wp_in + (col - kPlanarHalo) * h->stride + h->lb_bias) * 4) : 0u;
        else
            g.lb[t] = (unsigned)((q - wp_out - 1 + h->lb_bias) * 4);
    }
    g.obase = (size_t)un.co * h->pitch_out + h->q0 + bs * un.band0 + lane;
}

// A compute warp's part of one item: its units, pass by pass.
template <int T, bool STRIDED>
__device__ __forceinline__ void pn_compute(const PnItem &it, unsigned char *smem, const PnLayout &lay, unsigned rec,
                                           unsigned smem32, unsigned &cpar, int warp, int lane)
{
    const PnHdr *h = reinterpret_cast<const PnHdr *>(smem + rec);
    const int ub = h->wbeg[warp], ue = h->wbeg[warp + 1];
    const PnUnit *units = reinterpret_cast<const PnUnit *>(smem + rec + h->unit_off);
    const unsigned ent = rec + (unsigned)h->ent_off;
    const unsigned tile = (unsigned)lay.tile;
    const int bs = h->bs;
    float *part = reinterpret_cast<float *>(smem + lay.part);
    const int cpp = it.cpp, passes = it.passes;
    const unsigned all_landed = (1u << cpp) - 1u;
    for (int p = 0; p < passes; ++p) {
        const bool last = p + 1 == passes;
        const bool with_res = last && h->res != nullptr;
        unsigned landed = 0;
        // The geometry and the residual of a unit are fetched one unit ahead: a residual comes from L2,
        // and the multiply-add loop of a single short unit would not cover that round trip.
        PnLaneGeom<T> g, gn;
        float res[T], resn[T];
#pragma unroll
        for (int t = 0; t < T; ++t) res[t] = resn[t] = 0.0f;
        if (ub < ue) {
            pn_geometry<T, STRIDED>(h, units[ub], lane, g);
            if (with_res) {
#pragma unroll
                for (int t = 0; t < T; ++t)
                    if (g.ok & (1u << t)) res[t] = ld_cg(h->res + g.obase + bs * t);
            }
        }
        for (int u = ub; u < ue; ++u) {
            const PnUnit &un = units[u];
            if (u + 1 < ue) {
                pn_geometry<T, STRIDED>(h, units[u + 1], lane, gn);
                if (with_res) {
#pragma unroll
                    for (int t = 0; t < T; ++t) {
                        resn[t] = 0.0f;
                        if (gn.ok & (1u << t)) resn[t] = ld_cg(h->res + gn.obase + bs * t);
                    }
                }
            }
            float acc[T];
#pragma unroll
            for (int t = 0; t < T; ++t) acc[t] = p > 0 ? part[((size_t)u * T + t) * 32 + lane] : 0.0f;
            int e = p == 0 ? un.e_begin : un.e_end[p * cpp - 1];
            if (landed == all_landed) {
                // the whole pass is in shared memory: one run over all its segments (the padding entries
                // between segments have weight 0 and offset 0)
                const int end = un.e_end[p * cpp + cpp - 1];
                if (e < end) pn_mac<T, STRIDED>(smem, ent, e, end, tile, g.lb, acc);
            } else {
                for (int c = 0; c < cpp; ++c) {
                    const int end = un.e_end[p * cpp + c];
                    if (!(landed & (1u << c))) {
                        pn_mbar_wait(smem32 + lay.bars + 16 + c * 8, (cpar >> c) & 1u);
                        landed |= 1u << c;
                    }
                    if (e < end) pn_mac<T, STRIDED>(smem, ent, e, end, tile, g.lb, acc);
                    e = end;
                }
            }
            if (last) {
#pragma unroll
                for (int t = 0; t < T; ++t)
                    if (g.ok & (1u << t)) {
                        float z = fmaf(acc[t], un.scale, un.bias);
                        if (with_res) z += res[t];
                        z = pn_act(z, h->act);
                        if (h->y) h->y[g.obase + bs * t] = z;
                        if (h->y2) {
                            // A stride-2 layer reads this map: its positions also go, split by row and column
                            // parity, to planes of half the size, over which that layer is a stride-1 stencil.
                            const int q = h->q0 + bs * (un.band0 + t) + lane;
                            const int row = (int)(__umulhi((unsigned)q, h->dmul) >> h->dshr);
                            const int r = row - kPlanarHalo, c = q - row * h->wp_out - kPlanarHalo;
                            const int par = (r & 1) * 2 + (c & 1);
                            if (h->par_mask & (1 << par))
                                h->y2[((size_t)par * h->c2_stride + un.co) * h->pitch2 + ((r >> 1) + kPlanarHalo) * h->wp2 + (c >> 1) + kPlanarHalo] = z;
                        }
                    }
            } else {
#pragma unroll
                for (int t = 0; t < T; ++t) part[((size_t)u * T + t) * 32 + lane] = acc[t];
            }
            g = gn;
#pragma unroll
            for (int t = 0; t < T; ++t) res[t] = resn[t];
        }
        cpar ^= all_landed;   // every chunk barrier of the pass has been armed once
        if (p + 1 < passes) __syncthreads();   // the tile is free: the control warp stages the next pass
    }
    // the maps this warp stored are read by the copy unit in a later phase
    asm volatile("fence.proxy.async.global;\n" ::: "memory");
}

// control warp: lane c starts the copies of chunk c of one pass of an item's tile (issuing a tensor copy
// takes a few hundred clocks; the lanes' issues overlap)
__device__ __forceinline__ void pn_issue_pass(const PnItem &it, const PnMaps &maps, unsigned smem32, const PnLayout &lay, int p, int c)
{
    const CUtensorMap *map = &maps.m[it.layer];
    const unsigned box_bytes = (unsigned)(it.RB * it.L * 4);
    const unsigned chunk_bytes = box_bytes * (unsigned)it.nrb;
    const unsigned bar = smem32 + lay.bars + 16 + c * 8;
    pn_expect_tx(bar, chunk_bytes);
    const int row = it.row0 + (p * it.cpp + c) * it.CIc;
    for (int b = 0; b < it.nrb; ++b)
        pn_tensor_copy(smem32 + lay.tile + c * chunk_bytes + b * box_bytes, map, it.x0, row + b * it.RB, bar);
}

__global__ void __launch_bounds__(kPnThreads, 1)
net_persistent_kernel(const PnItem *items, const int *blk_first, const __grid_constant__ PnMaps maps, const unsigned char *recs,
                      int n_phases, unsigned *sync, const PnLayout lay, long long *prof)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const unsigned smem32 = (unsigned)__cvta_generic_to_shared(smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool ctrl_warp = warp == kPnWarps;
    const bool ctrl = ctrl_warp && lane == 0;
    PnItem *sItem = reinterpret_cast<PnItem *>(smem + lay.items);
    const PnItem *mine = items + blk_first[blockIdx.x];
    int next = 0;   // control thread: index of the next item to prefetch

    // control thread: fetch descriptor `next` into slot s and start the copy of its record
    auto prefetch = [&](int s) {
        const uint4 *src = reinterpret_cast<const uint4 *>(mine + next);
        uint4 *dst = reinterpret_cast<uint4 *>(sItem + s);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = __ldg(src + i);
        ++next;
        const PnItem &ni = sItem[s];
        if (ni.phase != kPnPhaseEnd) {
            asm volatile("prefetch.tensormap [%0];\n" ::"l"(&maps.m[ni.layer]) : "memory");
            const unsigned bar = smem32 + lay.bars + s * 8;
            pn_expect_tx(bar, (unsigned)ni.rec_bytes);
            pn_bulk_copy(smem32 + lay.wbuf[s], recs + ni.rec_off, (unsigned)ni.rec_bytes, bar);
        }
    };

    // Shared memory starts as zeros: look-ahead loads may touch bytes no copy has written yet, and
    // whatever they read is multiplied by a zero weight - it must be a finite number.
    for (int i = tid; i < lay.bars / 16; i += kPnThreads) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    if (ctrl) {
        for (int i = 0; i < 2 + kPnMaxCpp; ++i) pn_mbar_init(smem32 + lay.bars + i * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        prefetch(0);
    }
    __syncthreads();

    int sel = 0;              // record buffer / descriptor slot of the current item
    unsigned wpar = 0;        // parity to wait for on the two record barriers
    unsigned cpar = 0;        // parity to wait for on the chunk barriers
    unsigned target = 0;
    for (int ph = 0; ph < n_phases; ++ph) {
        // optional profile: SM clock at the start of the phase and when this block's items are done
        if (prof && ctrl) prof[((size_t)ph * 4) * gridDim.x + blockIdx.x] = clock64();
        while (sItem[sel].phase == ph) {
            const PnItem it = sItem[sel];
            if (ctrl_warp) {
                // the whole warp walks the same path (block barriers are warp-wide); lane 0 does the work
                for (int p = 0; p < it.passes; ++p) {
                    if (p > 0) __syncthreads();   // the compute warps are done with the previous pass
                    if (p > 0 && lane == 0) asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // reads of the tile before the unit's writes
                    __syncwarp();
                    if (lane < it.cpp) pn_issue_pass(it, maps, smem32, lay, p, lane);
                    __syncwarp();
                    if (lane == 0) {
                        if (prof && p == 0) prof[((size_t)ph * 4 + 1) * gridDim.x + blockIdx.x] = clock64();
                        if (p == 0) prefetch(sel ^ 1);   // those buffers were released by the block barrier that ended the previous item
                        // every copy of the pass has landed before its barriers are armed again
                        for (int c = 0; c < it.cpp; ++c) pn_mbar_wait(smem32 + lay.bars + 16 + c * 8, (cpar >> c) & 1u);
                        if (prof && p + 1 == it.passes) prof[((size_t)ph * 4 + 2) * gridDim.x + blockIdx.x] = clock64();

                    }
                    cpar ^= (1u << it.cpp) - 1u;
                    __syncwarp();
                }
            } else {
                pn_mbar_wait(smem32 + lay.bars + sel * 8, (wpar >> sel) & 1u);   // the record is in place
                const unsigned rec = (unsigned)lay.wbuf[sel];
                switch (it.T * 2 + it.strided) {
                    case 2: pn_compute<1, false>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 3: pn_compute<1, true>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 4: pn_compute<2, false>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 5: pn_compute<2, true>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 6: pn_compute<3, false>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 7: pn_compute<3, true>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    case 8: pn_compute<4, false>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                    default: pn_compute<4, true>(it, smem, lay, rec, smem32, cpar, warp, lane); break;
                }
            }
            wpar ^= 1u << sel;
            __syncthreads();   // the item is done: its tile, record buffer and descriptor slot are free
            sel ^= 1;
            if (ctrl) {
                // off the critical path: order the warps' reads of the tile before the copy unit's next writes,
                // and let the copy unit see the next item's tensor map (a prefetch of its first box into L2;
                // what the box holds does not matter yet)
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                const PnItem &ni = sItem[sel];
                if (ni.phase != kPnPhaseEnd)
                    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];\n"
                                 ::"l"(&maps.m[ni.layer]), "r"(ni.x0), "r"(ni.row0) : "memory");
            }
        }
        if (prof && ctrl) prof[((size_t)ph * 4 + 3) * gridDim.x + blockIdx.x] = clock64();
        if (ph + 1 < n_phases) {
            target += gridDim.x;
            if (ctrl) pn_grid_barrier(sync, target);
            __syncthreads();
        }
    }
    if (prof && ctrl) prof[((size_t)n_phases * 4) * gridDim.x + blockIdx.x] = clock64();
    // the last block to leave zeroes the barrier words for the next launch
    if (ctrl) {
        const unsigned left = atomicAdd(sync + 1, 1u);
        if (left == gridDim.x - 1) {
            sync[0] = 0u;
            sync[1] = 0u;
            __threadfence();
        }
    }
}

size_t round_up_sz(size_t v, size_t a) { return (v + a - 1) / a * a; }
int ceil_div_i(int a, int b) { return (a + b - 1) / b; }
int floor4(int v) { return v >= 0 ? (v & ~3) : -(((-v) + 3) & ~3); }

}  // namespace

// ---- host planner ---------------------------------------------------------------------------

struct PersistLayer {                 // geometry, nonzeros and chosen plan of one conv of the run
    const cadnn_weights *w = nullptr;
    PersistOpDesc d;
    int c_in = 0, c_out = 0, stride = 1;
    int wp_in = 0, pitch_in = 0, wp_out = 0, pitch_out = 0, h_out = 0, w_out = 0;
    int rel_min = 0, rel_max = 0;     // smallest / largest tap offset inside a plane
    int bs = 32;                      // positions per band
    int q_start = 0, q_end = 0, n_bands = 0;
    std::vector<float> scale, bias;
    // stored nonzeros by output channel, sorted by input plane: {value bits, plane, tap offset inside the plane}
    std::vector<int32_t> ptr;
    std::vector<uint32_t> bits;
    std::vector<int32_t> ch, rel;
    const float *x_planes = nullptr;  // the planes the tensor map covers (the layer's input, or its parity planes)
    int img_rows = 0;                 // planes per image in that buffer
    // parity planes this layer writes for a stride-2 reader (see the epilogue)
    float *y2 = nullptr;
    int par_mask = 0, wp2 = 0, pitch2 = 0;
    bool write_main = true;
    double work = 0.0;                // stored nonzeros x output positions
    int TB = 1, T = 1, G = 1, tiles = 1, groups = 1, L = 32, CIc = 4, RB = 4, nrb = 1, cpp = 1, passes = 1, strided = 0;
    double est = 0.0;
    int phase = 0;
};

namespace {

struct HostItem {
    int phase = 0, layer = 0, x0 = 0, row0 = 0;
    int n_units = 0;
    std::vector<unsigned char> rec;
};

// extent of the input a tile of bands [b0, b0 + nb) needs: first staged element (multiple of 4) and floats per channel
void tile_extent(const PersistLayer &l, int b0, int nb, int *x0, int *len)
{
    const int q0 = l.q_start + l.bs * b0;
    int lo = 0, hi = 0;
    if (l.stride == 1) {   // every lane loads, interior or not
        lo = q0 - l.wp_out - 1;
        hi = q0 + 32 * nb - 1 - l.wp_out - 1;
    } else {
        bool any = false;
        for (int q = q0; q < q0 + l.bs * nb; ++q) {
            const int row = q / l.wp_out, col = q - row * l.wp_out;
            if (row < kPlanarHalo || row >= kPlanarHalo + l.h_out || col < kPlanarHalo || col >= kPlanarHalo + l.w_out) continue;
            const int o = ((row - kPlanarHalo) * l.stride) * l.wp_in + (col - kPlanarHalo) * l.stride;
            if (!any) { lo = hi = o; any = true; }
            lo = std::min(lo, o);
            hi = std::max(hi, o);
        }
    }
    *x0 = floor4(lo + l.rel_min);
    *len = hi + l.rel_max - *x0 + 1;
}

// Cost model (clock cycles) of one block's item, fitted to clock samples of the kernel on a B200:
//  * the first bytes of a tile arrive ~2000 clocks into the phase, and with every SM copying at once the
//    copies share ~3800 bytes per clock (26 per SM); a lone SM gets ~60;
//  * a further pass over the channels waits for every warp and then for its own copies;
//  * the multiply-adds are bound by one shared-memory wavefront per clock and SM, and a single warp walks
//    about 100 clocks per batch of nonzeros.
double item_cost(const PersistLayer &l, int TB, int T, int G, int L, int passes, int cpp, double nnz_avg, int active)
{
    const double rate = std::min(60.0, 3800.0 / std::max(1, active));
    const double bytes_pass = (double)l.c_in * L * 4.0 / passes;
    const double t_first = 2000.0 + bytes_pass / cpp / rate;                    // first chunk in place
    const double t_fill = passes * (2000.0 + bytes_pass / rate) + (passes - 1) * 3000.0;
    const int upf = ceil_div_i(TB, T);
    const double wave = (double)G * nnz_avg * (TB + 0.5 * upf) * 1.15;
    const int batch = T == 1 ? 8 : 4;
    const double t_unit = 300.0 + (nnz_avg / batch + 1.0 + passes * cpp * 0.5) * 110.0 + (l.d.residual ? 150.0 : 0.0);
    const double t_path = (double)ceil_div_i(G * upf, kPnWarps) * t_unit * passes;
    const double t_comp = std::max(wave, t_path);
    return std::max(t_fill + 0.35 * t_comp, t_first + t_comp) + 400.0;
}

// choose tile, groups and chunking of a layer that may use `budget` blocks
bool plan_layer(PersistLayer &l, int budget, int n_img, int tile_cap, int rec_cap)
{
    const double nnz_avg = (double)l.bits.size() / std::max(1, l.c_out);
    int force_tb = 0;
    if (const char *e = getenv("CADNN_PERSIST_TB")) force_tb = atoi(e);   // tuning / test switch
    bool found = false;
    double best = 0.0;
    for (int TB : {1, 2, 3, 4, 6, 8}) {
        if (force_tb > 0 ? TB != force_tb : (TB > 1 && TB - 1 >= l.n_bands)) continue;
        const int tiles = ceil_div_i(l.n_bands, TB);
        const int T = TB <= kPnMaxT ? TB : (TB % 4 == 0 ? 4 : 3);
        int L = 0;
        for (int ti = 0; ti < tiles; ++ti) {
            int x0, len;
            // stride 1: the lanes of a unit's unused bands and of short last tiles still address whole bands
            const int nb = l.stride == 1 ? ceil_div_i(TB, T) * T : std::min(TB, l.n_bands - ti * TB);
            tile_extent(l, ti * TB, nb, &x0, &len);
            L = std::max(L, len);
        }
        L = (L + 7) & ~7;
        if (L > 256) continue;
        const long long items_sp = (long long)tiles * n_img;
        // channels per pass are bounded by the tile buffer
        int passes = 0, cpp = 1, CIc = 4, nrb = 1, RB = 4;
        bool fits = false;
        for (passes = 1; passes <= kPnMaxSeg; ++passes) {
            const int c_pass = ceil_div_i(l.c_in, passes);
            cpp = std::min(kPnMaxCpp, std::max(1, kPnMaxSeg / passes));
            while (cpp > 1 && c_pass / cpp < 8) --cpp;
            CIc = (ceil_div_i(c_pass, cpp) + 3) & ~3;
            nrb = ceil_div_i(CIc, 256);
            RB = (ceil_div_i(CIc, nrb) + 3) & ~3;
            fits = (long long)cpp * nrb * RB * L * 4 <= tile_cap;
            if (fits) break;
        }
        if (!fits) continue;
        const int upf = ceil_div_i(TB, T);
        // every split of the filters into equal groups: fewer filters per item make smaller records,
        // more items than blocks make several rounds
        int prev_groups = 0;
        for (int G = l.c_out; G >= 1; --G) {
            const int groups = ceil_div_i(l.c_out, G);
            if (groups == prev_groups) continue;
            prev_groups = groups;
            const double rec_est = sizeof(PnHdr) + (double)G * upf * sizeof(PnUnit) +
                                   (double)G * upf * (nnz_avg * 1.15 + 2.0 * passes * cpp) * 8.0 + 256.0;
            if (rec_est > rec_cap) continue;
            if (passes > 1 && (long long)G * upf * T * 128 > 16 * 1024) continue;   // partial sums between passes
            const long long n_items = items_sp * groups;
            const double rounds = std::ceil((double)n_items / std::max(1, budget));
            if (rounds > 64.0) break;
            // (a further round starts only when a block's previous item is done: it pays the copy start-up again)
            const double cost = rounds * item_cost(l, TB, T, G, L, passes, cpp, nnz_avg, (int)std::min<long long>(n_items, budget)) +
                                (rounds - 1.0) * 1500.0;
            if (!found || cost < best) {
                found = true;
                best = cost;
                l.TB = TB; l.T = T; l.G = G; l.tiles = tiles; l.groups = groups; l.L = L;
                l.CIc = CIc; l.RB = RB; l.nrb = nrb; l.cpp = cpp; l.passes = passes;
                l.strided = l.stride != 1 ? 1 : 0;
                l.est = cost;
            }
        }
    }
    return found;
}

// records of all items of a layer
bool build_items(const PersistLayer &l, int layer_idx, int phase, int n_img, std::vector<HostItem> &out)
{
    auto rn = [&](int co) { return (int)(l.ptr[co + 1] - l.ptr[co]); };
    // filters dealt to groups by decreasing nonzero count, snake order: equal work per group
    std::vector<int> order(l.c_out);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return rn(a) > rn(b); });
    std::vector<std::vector<int>> members(l.groups);
    for (int i = 0; i < l.c_out; ++i) {
        const int round = i / l.groups, pos = i % l.groups;
        members[(round & 1) ? l.groups - 1 - pos : pos].push_back(order[i]);
    }
    const int c_pass = l.cpp * l.CIc;
    const int rows_per_chunk = l.nrb * l.RB;
    const FastDiv fd = make_fastdiv(l.wp_out);
    for (int img = 0; img < n_img; ++img)
        for (int ti = 0; ti < l.tiles; ++ti) {
            const int b0 = ti * l.TB, nbt = std::min(l.TB, l.n_bands - b0);
            int x0, len;
            tile_extent(l, b0, nbt, &x0, &len);
            for (int gi = 0; gi < l.groups; ++gi) {
                const std::vector<int> &fs = members[gi];
                if (fs.empty()) continue;
                struct U { int co, band0, nb; long long load; };
                std::vector<U> us;
                for (int co : fs)
                    for (int bb = 0; bb < nbt; bb += l.T) {
                        const int nb = std::min(l.T, nbt - bb);
                        us.push_back({co, bb, nb, (long long)rn(co) * nb + 24});
                    }
                // longest processing time: heaviest unit to the least loaded warp
                std::vector<int> idx(us.size());
                std::iota(idx.begin(), idx.end(), 0);
                std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return us[a].load > us[b].load; });
                std::vector<std::vector<int>> of_warp(kPnWarps);
                std::vector<long long> wl(kPnWarps, 0);
                for (int id : idx) {
                    int bw = 0;
                    for (int k = 1; k < kPnWarps; ++k)
                        if (wl[k] < wl[bw]) bw = k;
                    of_warp[bw].push_back(id);
                    wl[bw] += us[id].load;
                }
                HostItem item;
                item.phase = phase;
                item.layer = layer_idx;
                item.x0 = x0;
                item.row0 = img * l.img_rows;
                item.n_units = (int)us.size();
                PnHdr hdr;
                memset(&hdr, 0, sizeof(hdr));
                hdr.y = l.write_main ? const_cast<float *>((const float *)l.d.y) + (size_t)img * l.c_out * l.pitch_out : nullptr;
                if (l.y2) {
                    const int n_par = (l.par_mask & ~1) ? 4 : 1;
                    hdr.y2 = l.y2 + (size_t)img * n_par * l.c_out * l.pitch2;
                    hdr.par_mask = l.par_mask; hdr.wp2 = l.wp2; hdr.pitch2 = l.pitch2; hdr.c2_stride = l.c_out;
                }
                hdr.res = l.d.residual ? (const float *)l.d.residual + (size_t)img * l.c_out * l.pitch_out : nullptr;
                hdr.q0 = l.q_start + l.bs * b0;
                hdr.n_units = item.n_units;
                hdr.unit_off = (int)sizeof(PnHdr);
                hdr.ent_off = (int)round_up_sz(sizeof(PnHdr) + sizeof(PnUnit) * us.size(), 16);
                hdr.wp_out = l.wp_out; hdr.h_out = l.h_out; hdr.w_out = l.w_out; hdr.pitch_out = l.pitch_out;
                hdr.dmul = fd.mul; hdr.dshr = fd.shr;
                hdr.stride = l.stride; hdr.wp_in = l.wp_in;
                hdr.act = l.d.act; hdr.lb_bias = l.rel_min - x0;
                hdr.bs = l.bs;
                std::vector<PnUnit> units;
                std::vector<uint32_t> ent;
                int wpos = 0;
                for (int wi = 0; wi < kPnWarps; ++wi) {
                    hdr.wbeg[wi] = wpos;
                    for (int id : of_warp[wi]) {
                        const U &u = us[id];
                        PnUnit pu;
                        memset(&pu, 0, sizeof(pu));
                        pu.co = u.co; pu.band0 = u.band0; pu.nb = u.nb;
                        pu.scale = l.scale[u.co]; pu.bias = l.bias[u.co];
                        pu.e_begin = (int)(ent.size() / 2);
                        // the filter's stored nonzeros are sorted by input plane: cut them at the chunk borders
                        const int n_ent = rn(u.co), e0 = l.ptr[u.co];
                        int k = 0;
                        for (int s = 0; s < kPnMaxSeg; ++s) {
                            if (s < l.passes * l.cpp) {
                                const int p = s / l.cpp, c = s % l.cpp;
                                const int ch_lo = p * c_pass + c * l.CIc, ch_hi = ch_lo + l.CIc;
                                int cnt = 0;
                                while (k < n_ent) {
                                    const int ci = l.ch[e0 + k], rel = l.rel[e0 + k];
                                    if (ci >= ch_hi) break;
                                    if (ci < ch_lo) return false;   // not sorted as expected
                                    if (rel > l.rel_max || rel < l.rel_min) return false;
                                    const int srow = c * rows_per_chunk + (ci - ch_lo);
                                    ent.push_back(l.bits[e0 + k]);
                                    ent.push_back((uint32_t)((srow * l.L + rel - l.rel_min) * 4));
                                    ++cnt;
                                    ++k;
                                }
                                if (cnt & 1) { ent.push_back(0u); ent.push_back(0u); }
                            }
                            pu.e_end[s] = (int)(ent.size() / 2);
                        }
                        if (k < n_ent) return false;
                        units.push_back(pu);
                        ++wpos;
                    }
                }
                hdr.wbeg[kPnWarps] = wpos;
                for (int z = 0; z < 64; ++z) ent.push_back(0u);   // zero tail for the look-ahead loads (up to three batches of 8)
                item.rec.assign(round_up_sz((size_t)hdr.ent_off + ent.size() * 4, 16), 0);
                memcpy(item.rec.data(), &hdr, sizeof(hdr));
                memcpy(item.rec.data() + hdr.unit_off, units.data(), units.size() * sizeof(PnUnit));
                memcpy(item.rec.data() + hdr.ent_off, ent.data(), ent.size() * 4);
                out.push_back(std::move(item));
            }
        }
    return true;
}

}  // namespace

struct PersistPlan {
    int device = -1;
    int n_ops = 0, n_phases = 0;
    int grid = 0, smem = 0;
    PnLayout lay;
    void *d_blob = nullptr;   // items, block starts, tensor maps, records, barrier words: one allocation
    const PnItem *d_items = nullptr;
    const int *d_blk_first = nullptr;
    PnMaps maps;              // host copy, passed by value at every launch
    const unsigned char *d_recs = nullptr;
    unsigned *d_sync = nullptr;
    long long *d_prof = nullptr;        // [4 * n_phases + 1][grid] clock samples (only with CADNN_PERSIST_PROFILE)
    std::vector<void *> aux;            // parity planes of the maps that stride-2 layers read
    std::vector<PersistLayer> layers;   // the plan, for reports
};

int persist_phases(const PersistPlan *plan) { return plan ? plan->n_phases : 0; }

void persist_free(PersistPlan *plan)
{
    if (!plan) return;
    if (plan->d_blob) cudaFree(plan->d_blob);
    if (plan->d_prof) cudaFree(plan->d_prof);
    for (void *q : plan->aux) cudaFree(q);
    delete plan;
}

int persist_describe(const PersistPlan *plan, int op, int out[12])
{
    if (!plan || op < 0 || op >= (int)plan->layers.size()) return 0;
    const PersistLayer &l = plan->layers[op];
    const int v[12] = {l.TB, l.T, l.G, l.tiles, l.groups, l.L, l.CIc, l.cpp, l.passes, l.strided, (int)l.est, l.phase};
    for (int i = 0; i < 12; ++i) out[i] = v[i];
    return 1;
}

cadnn_status persist_create(const std::vector<PersistOpDesc> &descs, PersistPlan **out)
{
    *out = nullptr;
    if (descs.empty()) return CADNN_E_ARG;
    int dev = 0, sms = 0, coop = 0;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    CADNN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CADNN_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    if (!coop) return CADNN_E_UNSUPPORTED;
    int grid = sms;
    if (const char *e = getenv("CADNN_PERSIST_GRID")) {   // tuning / test switch: fewer blocks, several items per block and phase
        const int v = atoi(e);
        if (v >= 1 && v <= sms) grid = v;
    }
    const int n_ops = (int)descs.size();
    const int n_img = std::max(1, descs[0].n);
    if (n_ops > kPnMaxLayers) return CADNN_E_UNSUPPORTED;

    std::vector<PersistLayer> layers(n_ops);
    int n_phases = 0;
    for (int i = 0; i < n_ops; ++i) {
        const PersistOpDesc &d = descs[i];
        const cadnn_weights *w = d.w;
        if (!w || !w->has_planar || w->pl_ptr.empty() || d.n != n_img) return CADNN_E_ARG;
        const cadnn_layer_desc &ld = w->desc;
        if (ld.stride != 1 && ld.stride != 2) return CADNN_E_UNSUPPORTED;
        PersistLayer &l = layers[i];
        l.w = w;
        l.d = d;
        l.x_planes = (const float *)d.x;
        l.c_in = ld.c_in; l.c_out = ld.c_out; l.stride = ld.stride;
        l.img_rows = ld.c_in;
        l.wp_in = ld.in_w + 2 * kPlanarHalo; l.pitch_in = planar_pitch(ld.in_h, ld.in_w);
        l.h_out = w->h_out; l.w_out = w->w_out;
        l.wp_out = w->w_out + 2 * kPlanarHalo; l.pitch_out = planar_pitch(w->h_out, w->w_out);
        l.rel_min = (kPlanarHalo - ld.pad) * (l.wp_in + 1);
        l.rel_max = (ld.kh - 1 + kPlanarHalo - ld.pad) * l.wp_in + (ld.kw - 1 + kPlanarHalo - ld.pad);
        // the layer's stored nonzeros out of the planar image (rows there are padded to even counts with {0, 0})
        l.ptr.assign(l.c_out + 1, 0);
        for (int co = 0; co < l.c_out; ++co) {
            l.ptr[co] = (int32_t)l.bits.size();
            const uint32_t *row = w->pl_ent.data() + (size_t)w->pl_ptr[co] * 2;
            int n_ent = w->pl_ptr[co + 1] - w->pl_ptr[co];
            if (n_ent >= 2 && row[2 * (n_ent - 1)] == 0u && row[2 * (n_ent - 1) + 1] == 0u) --n_ent;
            for (int k = 0; k < n_ent; ++k) {
                const uint32_t off = row[2 * k + 1];
                const int ci = (int)(off / (uint32_t)l.pitch_in);
                l.bits.push_back(row[2 * k]);
                l.ch.push_back(ci);
                l.rel.push_back((int)(off - (uint32_t)ci * (uint32_t)l.pitch_in));
            }
        }
        l.ptr[l.c_out] = (int32_t)l.bits.size();
        l.work = (double)w->nnz * l.h_out * l.w_out;
        l.scale.assign(l.c_out, 1.0f);
        l.bias.assign(l.c_out, 0.0f);
        if (d.scale) CADNN_CUDA_TRY(cudaMemcpy(l.scale.data(), d.scale, (size_t)l.c_out * 4, cudaMemcpyDeviceToHost));
        if (d.bias) CADNN_CUDA_TRY(cudaMemcpy(l.bias.data(), d.bias, (size_t)l.c_out * 4, cudaMemcpyDeviceToHost));
        if (i > 0 && !d.join_phase) ++n_phases;
        l.phase = n_phases;
    }
    ++n_phases;

    // Stride-2 layers (Section 4, "Memory layout transformation"): where the producer of a stride-2
    // layer's input runs inside this kernel, it also writes its map split by row and column parity into
    // planes of half the size; over those a stride-2 k x k layer is a stride-1 stencil with taps
    // in {-1, 0}^2 (a 1x1 layer reads the even/even plane alone), staged and walked like any other.
    // A map with no other reader is written in that form only.
    PersistPlan *plan = new (std::nothrow) PersistPlan();
    if (!plan) return CADNN_E_ALLOC;
    std::vector<void *> &aux_buffers = plan->aux;
    auto fail = [&](cadnn_status st) { persist_free(plan); return st; };
    const bool no_parity = getenv("CADNN_PERSIST_NO_PARITY") != nullptr;   // tuning / test switch
    for (int k = 0; k < n_ops && !no_parity; ++k) {
        PersistLayer &l = layers[k];
        const cadnn_layer_desc &ld = l.w->desc;
        if (l.stride != 2) continue;
        int prod = -1;
        for (int j = 0; j < k; ++j)
            if (descs[j].y == descs[k].x) prod = j;
        if (prod < 0 || layers[prod].phase >= l.phase) continue;
        const int need = (ld.kh == 1 && ld.kw == 1) ? 1 : 15;   // parities this layer reads
        layers[prod].par_mask |= need;
    }
    for (int j = 0; j < n_ops; ++j) {
        PersistLayer &pl = layers[j];
        if (!pl.par_mask) continue;
        const int hq = (pl.h_out + 1) / 2, wq = (pl.w_out + 1) / 2;
        const int n_par = (pl.par_mask & ~1) ? 4 : 1;
        pl.wp2 = wq + 2 * kPlanarHalo;
        pl.pitch2 = planar_pitch(hq, wq);
        const size_t bytes = (size_t)n_img * n_par * pl.c_out * pl.pitch2 * 4;
        void *buf = nullptr;
        if (cudaMalloc(&buf, bytes) != cudaSuccess || cudaMemset(buf, 0, bytes) != cudaSuccess) {
            cudaGetLastError();
            if (buf) cudaFree(buf);
            return fail(CADNN_E_ALLOC);
        }
        aux_buffers.push_back(buf);
        pl.y2 = (float *)buf;
        // does anybody still read the map itself?
        bool main_read = descs[j].dst_external;
        for (int k = 0; k < n_ops; ++k) {
            if (descs[k].residual == descs[j].y) main_read = true;
            if (descs[k].x == descs[j].y && !(layers[k].stride == 2 && layers[k].phase > pl.phase)) main_read = true;
        }
        pl.write_main = main_read;
        // rewrite the readers: input planes [parity][c_in], stride 1
        for (int k = j + 1; k < n_ops; ++k) {
            PersistLayer &l = layers[k];
            if (descs[k].x != descs[j].y || l.stride != 2 || l.phase <= pl.phase) continue;
            const int wp_old = l.wp_in;
            for (size_t e = 0; e < l.bits.size(); ++e) {
                const int ky = l.rel[e] / wp_old - kPlanarHalo, kx = l.rel[e] % wp_old - kPlanarHalo;   // tap relative to 2*oy, 2*ox
                const int pr = ky & 1, pc = kx & 1;
                const int dr = (ky - pr) / 2, dc = (kx - pc) / 2;   // -1 or 0
                l.ch[e] = (pr * 2 + pc) * l.c_in + l.ch[e];
                l.rel[e] = (dr + kPlanarHalo) * pl.wp2 + dc + kPlanarHalo;
            }
            // keep every filter's entries sorted by input plane
            for (int co = 0; co < l.c_out; ++co) {
                const int lo = l.ptr[co], hi = l.ptr[co + 1];
                std::vector<int> idx(hi - lo);
                std::iota(idx.begin(), idx.end(), lo);
                std::stable_sort(idx.begin(), idx.end(), [&](int a, int b) { return l.ch[a] < l.ch[b]; });
                std::vector<uint32_t> nb(hi - lo);
                std::vector<int32_t> nc(hi - lo), nr(hi - lo);
                for (int t = 0; t < hi - lo; ++t) { nb[t] = l.bits[idx[t]]; nc[t] = l.ch[idx[t]]; nr[t] = l.rel[idx[t]]; }
                std::copy(nb.begin(), nb.end(), l.bits.begin() + lo);
                std::copy(nc.begin(), nc.end(), l.ch.begin() + lo);
                std::copy(nr.begin(), nr.end(), l.rel.begin() + lo);
            }
            const bool one_by_one = l.w->desc.kh == 1 && l.w->desc.kw == 1;
            l.img_rows = n_par * l.c_in;
            l.c_in = (one_by_one ? 1 : 4) * l.c_in;   // a 1x1 layer stops at the even/even planes
            l.stride = 1;
            l.wp_in = pl.wp2;
            l.pitch_in = pl.pitch2;
            l.x_planes = pl.y2;
            l.rel_min = one_by_one ? pl.wp2 + 1 : 0;
            l.rel_max = pl.wp2 + 1;
        }
    }
    // geometry of the bands
    for (int i = 0; i < n_ops; ++i) {
        PersistLayer &l = layers[i];
        l.q_end = (l.h_out + kPlanarHalo - 1) * l.wp_out + l.w_out + kPlanarHalo;
        if (l.stride == 1) {
            // bands of 32 consecutive positions, from the first interior position rounded down to 16 bytes
            l.bs = 32;
            l.q_start = (kPlanarHalo * (l.wp_out + 1)) & ~3;
            l.n_bands = ceil_div_i(l.q_end - l.q_start, 32);
        } else {
            // a band is as many whole output rows as fit 32 lanes: its inputs are then a few whole input rows
            const int rows = 32 / l.wp_out;
            if (rows < 1) return fail(CADNN_E_UNSUPPORTED);
            l.bs = rows * l.wp_out;
            l.q_start = kPlanarHalo * l.wp_out;
            l.n_bands = ceil_div_i(l.h_out, rows);
        }
    }

    // Shared memory: two record buffers, the tile, partial sums, barriers, two descriptors.  Larger record
    // buffers allow more filters per item (fewer, fuller blocks) but leave a smaller tile: the split
    // is searched too, by the modelled time of the whole run.
    const int part_cap = 16 * 1024, misc = 256;
    int tile_limit = kPnSmemMax;
    if (const char *e = getenv("CADNN_PERSIST_TILE_KB")) {   // test switch: a small tile buffer forces several passes
        const int v = atoi(e);
        if (v >= 1) tile_limit = v * 1024;
    }
    auto layout_for = [&](int rec_cap, PnLayout &lay, int &tile_cap) {
        lay.wbuf[0] = 0;
        lay.wbuf[1] = rec_cap;
        lay.tile = 2 * rec_cap;
        tile_cap = std::min(tile_limit, (kPnSmemMax - 2 * rec_cap - part_cap - misc) & ~127);
        lay.part = lay.tile + ((kPnSmemMax - 2 * rec_cap - part_cap - misc) & ~127);
        lay.bars = lay.part + part_cap;
        lay.items = lay.bars + 64;
        return lay.items + 2 * (int)sizeof(PnItem);
    };
    // blocks each layer of a phase may use: in proportion to its work
    auto plan_all = [&](std::vector<PersistLayer> &ls, int tile_cap, int rec_plan, double *total_est) {
        *total_est = 0.0;
        for (int ph = 0, i = 0; ph < n_phases; ++ph) {
            int j = i;
            double total = 0.0, worst = 0.0;
            while (j < n_ops && ls[j].phase == ph) total += ls[j++].work + 1.0;
            int left = grid;
            for (int k = i; k < j; ++k) {
                PersistLayer &l = ls[k];
                int budget = k + 1 == j ? left : (int)(grid * (l.work + 1.0) / total + 0.5);
                budget = std::max(1, std::min(budget, left - (j - k - 1)));
                if (!plan_layer(l, budget, n_img, tile_cap, rec_plan)) return k;
                left = std::max(1, left - std::min(budget, l.tiles * l.groups * n_img));
                worst = std::max(worst, l.est);
            }
            *total_est += worst;
            i = j;
        }
        return -1;
    };
    PnLayout lay;
    int smem = 0, rec_cap = 0, tile_cap = 0;
    std::vector<HostItem> items;
    std::vector<int> first_item_of_phase(n_phases + 1, 0);
    bool built = false;
    for (int attempt = 0; attempt < 2 && !built; ++attempt) {
        // the records are planned against a margin below the buffer size; a second attempt widens it
        const double margin = attempt == 0 ? 0.92 : 0.75;
        double best_est = 0.0;
        int best_cap = 0;
        for (int cap_kb : {20, 28, 40, 52, 64}) {
            PnLayout lay_try;
            int tile_try = 0;
            layout_for(cap_kb * 1024, lay_try, tile_try);
            if (tile_try < 16 * 1024 && tile_limit == kPnSmemMax) continue;
            std::vector<PersistLayer> ls = layers;
            double est = 0.0;
            const int bad = plan_all(ls, tile_try, (int)(cap_kb * 1024 * margin), &est);
            if (bad >= 0) continue;
            if (best_cap == 0 || est < best_est) { best_cap = cap_kb; best_est = est; }
        }
        if (best_cap == 0) {
            if (getenv("CADNN_PERSIST_VERBOSE")) fprintf(stderr, "persist: no plan fits shared memory\n");
            return fail(CADNN_E_UNSUPPORTED);
        }
        rec_cap = best_cap * 1024;
        smem = layout_for(rec_cap, lay, tile_cap);
        double est = 0.0;
        plan_all(layers, tile_cap, (int)(rec_cap * margin), &est);
        items.clear();
        built = true;
        for (int k = 0; k < n_ops && built; ++k) {
            PersistLayer &l = layers[k];
            if (k == 0 || layers[k - 1].phase != l.phase) first_item_of_phase[l.phase] = (int)items.size();
            const size_t before = items.size();
            if (!build_items(l, k, l.phase, n_img, items)) {
                if (getenv("CADNN_PERSIST_VERBOSE")) fprintf(stderr, "persist: records of op %d could not be built\n", k);
                return fail(CADNN_E_UNSUPPORTED);
            }
            for (size_t q = before; q < items.size() && built; ++q) {
                const bool too_big = (int)items[q].rec.size() > rec_cap || (l.passes > 1 && items[q].n_units * l.T * 128 > part_cap);
                if (too_big) {
                    if (getenv("CADNN_PERSIST_VERBOSE")) fprintf(stderr, "persist: a record of op %d has %zu bytes, %d units\n", k, items[q].rec.size(), items[q].n_units);
                    built = false;
                }
            }
        }
    }
    if (!built) return fail(CADNN_E_UNSUPPORTED);
    first_item_of_phase[n_phases] = (int)items.size();

    // items of a phase go to blocks round robin; a block's list is phase-major and ends with a sentinel
    std::vector<std::vector<int>> of_block(grid);
    for (int ph = 0; ph < n_phases; ++ph)
        for (int q = first_item_of_phase[ph]; q < first_item_of_phase[ph + 1]; ++q)
            of_block[(q - first_item_of_phase[ph]) % grid].push_back(q);
    std::vector<PnItem> dev_items;
    std::vector<int> blk_first(grid);
    std::vector<size_t> rec_off(items.size());
    size_t rec_total = 0;
    for (size_t q = 0; q < items.size(); ++q) {
        rec_off[q] = rec_total;
        rec_total += round_up_sz(items[q].rec.size(), 128);
    }
    if (rec_total >= (1ull << 32)) return fail(CADNN_E_UNSUPPORTED);
    for (int b = 0; b < grid; ++b) {
        blk_first[b] = (int)dev_items.size();
        for (int q : of_block[b]) {
            const HostItem &hi = items[q];
            const PersistLayer &l = layers[hi.layer];
            PnItem it;
            memset(&it, 0, sizeof(it));
            it.phase = hi.phase; it.layer = hi.layer;
            it.rec_off = (unsigned)rec_off[q]; it.rec_bytes = (int)hi.rec.size();
            it.x0 = hi.x0; it.row0 = hi.row0;
            it.L = l.L; it.CIc = l.CIc; it.RB = l.RB; it.nrb = l.nrb; it.cpp = l.cpp; it.passes = l.passes;
            it.T = l.T; it.strided = l.strided;
            dev_items.push_back(it);
        }
        PnItem end;
        memset(&end, 0, sizeof(end));
        end.phase = kPnPhaseEnd;
        dev_items.push_back(end);
    }

    const size_t items_bytes = round_up_sz(dev_items.size() * sizeof(PnItem), 256);
    const size_t blk_bytes = round_up_sz((size_t)grid * 4, 256);
    const size_t maps_bytes = 0;
    const size_t recs_bytes = round_up_sz(rec_total + 256, 256);
    const size_t total = items_bytes + blk_bytes + maps_bytes + recs_bytes + 256;
    cudaError_t e = cudaMalloc(&plan->d_blob, total);
    if (e != cudaSuccess) {
        plan->d_blob = nullptr;
        persist_free(plan);
        cadnn_note_cuda(e);
        return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
    }
    std::vector<unsigned char> host(total, 0);
    unsigned char *base = (unsigned char *)plan->d_blob;
    memcpy(host.data(), dev_items.data(), dev_items.size() * sizeof(PnItem));
    memcpy(host.data() + items_bytes, blk_first.data(), (size_t)grid * 4);
    memset(&plan->maps, 0, sizeof(plan->maps));
    // one tensor map per layer: its input as [n * c_in planes][pitch], boxes of RB planes x L floats
    for (int i = 0; i < n_ops; ++i) {
        const PersistLayer &l = layers[i];
        const unsigned long long rows = (unsigned long long)n_img * l.img_rows;
        if (!encode_plane_rows_map(&plan->maps.m[i], l.x_planes, (unsigned long long)l.pitch_in, rows, (unsigned)l.L, (unsigned)l.RB)) {
            persist_free(plan);
            return CADNN_E_UNSUPPORTED;
        }
    }
    for (size_t q = 0; q < items.size(); ++q)
        memcpy(host.data() + items_bytes + blk_bytes + maps_bytes + rec_off[q], items[q].rec.data(), items[q].rec.size());
    e = cudaMemcpy(plan->d_blob, host.data(), total, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(net_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    int per_sm = 0;
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, net_persistent_kernel, kPnThreads, (size_t)smem);
    if (e != cudaSuccess || per_sm < 1) {
        persist_free(plan);
        if (e != cudaSuccess) return cadnn_note_cuda(e);
        return CADNN_E_UNSUPPORTED;
    }
    plan->device = dev;
    plan->n_ops = n_ops;
    plan->n_phases = n_phases;
    plan->grid = grid;
    plan->smem = smem;
    plan->lay = lay;
    plan->d_items = (const PnItem *)base;
    plan->d_blk_first = (const int *)(base + items_bytes);
    plan->d_recs = base + items_bytes + blk_bytes + maps_bytes;
    plan->d_sync = (unsigned *)(base + items_bytes + blk_bytes + maps_bytes + recs_bytes);
    plan->layers = std::move(layers);
    if (getenv("CADNN_PERSIST_PROFILE")) {
        const size_t pb = (size_t)(4 * n_phases + 1) * grid * sizeof(long long);
        if (cudaMalloc((void **)&plan->d_prof, pb) == cudaSuccess) cudaMemset(plan->d_prof, 0, pb);
        else { plan->d_prof = nullptr; cudaGetLastError(); }
    }
    if (getenv("CADNN_PERSIST_VERBOSE")) {
        for (int i = 0; i < n_ops; ++i) {
            const PersistLayer &l = plan->layers[i];
            fprintf(stderr, "persist op %2d phase %2d: %4d->%4d %dx%d s%d  TB %d T %d G %3d tiles %3d groups %3d L %3d CIc %4d cpp %d passes %d est %.0f clk\n",
                    i, l.phase, l.c_in, l.c_out, l.h_out, l.w_out, l.stride, l.TB, l.T, l.G, l.tiles, l.groups, l.L, l.CIc,
                    l.cpp, l.passes, l.est);
        }
    }
    *out = plan;
    return CADNN_OK;
}

cadnn_status persist_launch(const PersistPlan *plan, cudaStream_t st)
{
    if (!plan) return CADNN_E_ARG;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)plan->grid, 1, 1);
    cfg.blockDim = dim3(kPnThreads, 1, 1);
    cfg.dynamicSmemBytes = (size_t)plan->smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;   // all blocks resident at once, or the launch fails
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CADNN_CUDA_TRY(cudaLaunchKernelEx(&cfg, net_persistent_kernel, plan->d_items, plan->d_blk_first, plan->maps, plan->d_recs,
                                      plan->n_phases, plan->d_sync, plan->lay, plan->d_prof));
    return CADNN_OK;
}

// Clock samples of the last launch (after the caller synchronized): per phase the SM clocks from the phase's
// start to the next phase's start (mean over blocks), the longest / mean time a block spent on its own items,
// and (mean over blocks that had an item) the clocks until the tile copies were issued and until they had landed.
cadnn_status persist_profile(const PersistPlan *plan, int cap, float *wall_clk, float *busy_max_clk, float *busy_mean_clk,
                             float *issued_clk, float *landed_clk, int *n_out)
{
    if (!plan || !n_out) return CADNN_E_ARG;
    *n_out = plan->n_phases;
    if (!plan->d_prof) return CADNN_E_UNSUPPORTED;
    const int g = plan->grid, np = plan->n_phases;
    std::vector<long long> h((size_t)(4 * np + 1) * g);
    CADNN_CUDA_TRY(cudaMemcpy(h.data(), plan->d_prof, h.size() * sizeof(long long), cudaMemcpyDeviceToHost));
    CADNN_CUDA_TRY(cudaMemset(plan->d_prof, 0, h.size() * sizeof(long long)));
    for (int ph = 0; ph < np && ph < cap; ++ph) {
        double bmax = 0.0, bsum = 0.0, wsum = 0.0, isum = 0.0, lsum = 0.0;
        int with_item = 0;
        for (int b = 0; b < g; ++b) {
            const long long t0 = h[((size_t)ph * 4) * g + b];
            const double busy = (double)(h[((size_t)ph * 4 + 3) * g + b] - t0);
            bmax = std::max(bmax, busy);
            bsum += busy;
            wsum += (double)(h[((size_t)ph * 4 + 4) * g + b] - t0);
            if (h[((size_t)ph * 4 + 2) * g + b] > t0) {
                ++with_item;
                isum += (double)(h[((size_t)ph * 4 + 1) * g + b] - t0);
                lsum += (double)(h[((size_t)ph * 4 + 2) * g + b] - t0);
            }
        }
        if (wall_clk) wall_clk[ph] = (float)(wsum / g);
        if (busy_max_clk) busy_max_clk[ph] = (float)bmax;
        if (busy_mean_clk) busy_mean_clk[ph] = (float)(bsum / g);
        if (issued_clk) issued_clk[ph] = with_item ? (float)(isum / with_item) : 0.0f;
        if (landed_clk) landed_clk[ph] = with_item ? (float)(lsum / with_item) : 0.0f;
    }
    return CADNN_OK;
}
