// Tensor-core path for block-structured int8 layers.
//
// CADNN (arXiv 1905.00571), Section 1 ("computation pattern transformation") and Section 4
// ("Model computation fusion and transformation"): where pruning leaves regular structure, the
// computation is transformed to a form the processor runs at full rate.  Here: after the
// packer has found the 64 output channels x 64 input channels x one tap blocks of an int8
// stride-1 convolution whose kept fraction reaches a threshold, those blocks are stored dense
// (pruned positions as zeros) and multiplied on the 5th-generation tensor cores; whatever else
// the mask kept stays in the sparse image and runs in the sparse kernel, which adds these
// int32 sums to its own before the requantization.  Integer sums are exact in any order, so the
// layer's result does not depend on which route a weight took.
//
// One thread block computes 128 output pixels (a 16 x 8 patch of one image) x 64 output channels.
// The dense blocks of a tile of output channels are grouped by (chunk of 64 input channels, kernel
// column kx): the taps (ky, kx) of a group read the same input columns, shifted by whole rows, so
//   * one lane of warp 0 is the producer: per group ONE 4-D TMA tensor copy of the 16 x (8 + kh - 1)
//     x 64-channel input patch at the column shift of kx (pixels outside the image read as zero: the
//     padding) and one bulk copy per present block of its 64 x 64 weights, all in the
//     64-byte-swizzled K-major layout, into a ring of stages, each on its own "full" mbarrier;
//   * thread 32 issues the multiply-adds: per block two tcgen05.mma of M 128 x N 64 x K 32
//     (s8 x s8 -> s32) on the patch rows ky .. ky + 7 (a shift of ky KB in the stage: the swizzle
//     pattern repeats every 512 bytes), accumulator in 64 columns of tensor memory, then a
//     tcgen05.commit that frees the stage ("empty" mbarrier) once the tensor core has read it;
//   * after the last commit the four warps read their 32 accumulator rows with tcgen05.ld and store
//     them as int32 [pixel][channel].
// Tensor memory is allocated by one warp and released by the same warp on every path; every
// mbarrier wait is bounded, and a wait that runs out raises a device flag (cadnn_device_status)
// and lets the block run to its end.  No multicast copies.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <vector>
#include <cuda.h>
#include "cadnn_internal.h"

// waits of this kernel that ran out (never expected)
__device__ int g_tc_timeout;

cadnn_status read_tc_timeouts(int *count)
{
    int v = 0;
    CADNN_CUDA_TRY(cudaMemcpyFromSymbol(&v, g_tc_timeout, sizeof(int)));
    *count = v;
    return CADNN_OK;
}

namespace {

const int kTcM = 128;          // output pixels per block: 16 columns x 8 rows
const int kTcBW = 16, kTcBH = 8;
const int kTcN = 64;           // output channels per block
const int kTcK = 64;           // input channels per dense block (bytes of a K-major row)
const int kTcMaxStages = 8;
const int kTcRowBytes = kTcBW * kTcK;   // one patch row of 16 pixels: 1024 bytes
const int kTcBBytes = kTcN * kTcK;      // 4096
const int kTcSmemBudget = 200 * 1024;
const unsigned kTcSpin = 1u << 22;

struct TcParams {
    const int8_t *wblk;
    const int4 *grp;          // {column shift, first input channel, mask of the kernel rows present, first block}
    const int *grp_ptr;       // groups of every tile of 64 output channels
    int kh, pad;              // kernel rows, padding above
    int a_bytes, stage_bytes, stages;   // patch bytes, stage bytes (patch + kh blocks), ring depth
    int *acc;                 // [n][h_out][w_out][c_out] int32 sums for the sparse kernel, or null:
    void *y;                  // then the layer's epilogue runs here and writes the output tensor
    const float *scale, *bias;
    const int8_t *residual;   // [n][h_out][w_out][c_out] or null
    float res_scale;
    int act, out_dtype;
    int ldc, c_off;           // channels of the output tensor and first channel of this layer's window in it
    int vec_ok;               // the window allows 16-byte stores
    int h_out, w_out, c_out;
    int tiles_x, tiles_y, n_ntiles;
};

__device__ __forceinline__ void tc_mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool tc_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n.reg .pred q;\nmbarrier.try_wait.parity.shared::cta.b64 q, [%1], %2;\nselp.u32 %0, 1, 0, q;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait; false = gave up (recorded)
__device__ __forceinline__ bool tc_wait(unsigned bar, unsigned parity)
{
    for (unsigned it = 0; it < kTcSpin; ++it)
        if (tc_try_wait(bar, parity)) return true;
    atomicAdd(&g_tc_timeout, 1);
    return false;
}
__device__ __forceinline__ void tc_bulk_copy(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_tensor_copy_4d(unsigned dst, const CUtensorMap *map, int c, int x, int y, int n, unsigned bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];\n"
                 ::"r"(dst), "l"(map), "r"(c), "r"(x), "r"(y), "r"(n), "r"(bar) : "memory");
}

// Shared-memory operand descriptor of a K-major tile whose rows are 64 bytes with the 64-byte swizzle:
// start address / 16, 8-row groups 512 bytes apart, descriptor version 1, layout type 4.
__device__ __forceinline__ unsigned long long tc_smem_desc(unsigned addr)
{
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3fffu);
    d |= (unsigned long long)1u << 16;                      // leading byte offset (unused for swizzled K-major): 16 bytes
    d |= (unsigned long long)((512u >> 4) & 0x3fffu) << 32; // stride byte offset between groups of 8 rows
    d |= (unsigned long long)1u << 46;                      // descriptor version
    d |= (unsigned long long)4u << 61;                      // 64-byte swizzle
    return d;
}

// instruction descriptor: s32 accumulator, signed 8-bit A and B, both K-major, N = 64, M = 128
__device__ __forceinline__ unsigned tc_instr_desc()
{
    return (2u << 4) | (1u << 7) | (1u << 10) | ((unsigned)(kTcN >> 3) << 17) | ((unsigned)(kTcM >> 4) << 24);
}

__device__ __forceinline__ void tc_mma_i8(unsigned tmem_d, unsigned long long adesc, unsigned long long bdesc, unsigned idesc,
                                          unsigned accumulate)
{
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n}\n"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
                 : "memory");
}
__device__ __forceinline__ void tc_commit(unsigned bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}

// 32 accumulator columns of this warp's 32 rows: thread = row, register j = column col0 + j
__device__ __forceinline__ void tc_ld32(unsigned taddr, int (&v)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr)
                 : "memory");
}

__global__ void __launch_bounds__(128) block_tc_kernel(const TcParams p, const __grid_constant__ CUtensorMap xmap)
{
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // stages at a 1024-byte boundary (the swizzle pattern repeats every 512 bytes)
    const int S = p.stages;
    const unsigned base32 = ((unsigned)__cvta_generic_to_shared(smem_raw) + 1023u) & ~1023u;
    const unsigned bars = base32 + S * p.stage_bytes;   // full[S], empty[S], done, then the TMEM address word, row masks
    const unsigned slot32 = bars + (2 * S + 1) * 8;
    unsigned char *smem_gen = smem_raw + (base32 - (unsigned)__cvta_generic_to_shared(smem_raw));
    volatile unsigned *slot = reinterpret_cast<volatile unsigned *>(smem_gen + S * p.stage_bytes + (2 * S + 1) * 8);
    volatile int *smask = reinterpret_cast<volatile int *>(smem_gen + S * p.stage_bytes + (2 * S + 1) * 8 + 16);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // block -> (image, patch row, patch column, output-channel tile); channel tiles vary fastest
    int b = blockIdx.x;
    const int nt = b % p.n_ntiles; b /= p.n_ntiles;
    const int tx = b % p.tiles_x; b /= p.tiles_x;
    const int ty = b % p.tiles_y;
    const int img = b / p.tiles_y;
    const int x0 = tx * kTcBW, y0 = ty * kTcBH;
    const int g_lo = p.grp_ptr[nt], n_grp = p.grp_ptr[nt + 1] - g_lo;

    if (tid == 0) {
        for (int i = 0; i < 2 * S + 1; ++i) tc_mbar_init(bars + i * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("prefetch.tensormap [%0];\n" ::"l"(&xmap) : "memory");
    }
    if (warp == 2) {   // one warp owns the tensor-memory allocation: 64 columns of 128 lanes
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(slot32), "r"(64u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const unsigned tmem = *slot;

    if (warp == 0) {
        // producer: the stages are a ring; a stage is refilled once the tensor core has read it.  The warp reads the
        // group list 32 entries at a time (one ahead), lane 0 waits for the stage and starts its copies.
        const int4 zero = make_int4(0, 0, 0, 0);
        int4 mine = lane < n_grp ? p.grp[g_lo + lane] : zero;
        bool alive = true;
        int s = 0;
        unsigned round = 0;   // times the ring has wrapped
        for (int base = 0; base < n_grp; base += 32) {
            const int4 ahead = base + 32 + lane < n_grp ? p.grp[g_lo + base + 32 + lane] : zero;
            const int cnt = min(32, n_grp - base);
            for (int j = 0; j < cnt; ++j) {
                const int xs = __shfl_sync(0xffffffffu, mine.x, j), ci0 = __shfl_sync(0xffffffffu, mine.y, j);
                const int rows = __shfl_sync(0xffffffffu, mine.z, j), b0 = __shfl_sync(0xffffffffu, mine.w, j);
                if (lane == 0 && alive) {
                    if (round > 0 && !tc_wait(bars + (S + s) * 8, (round - 1) & 1u)) {
                        alive = false;
                    } else {
                        const unsigned full = bars + s * 8, st32 = base32 + s * p.stage_bytes;
                        const int nb = __popc(rows);
                        smask[s] = rows;   // read by the issuing thread after its wait on the full barrier
                        tc_expect_tx(full, (unsigned)(p.a_bytes + nb * kTcBBytes));
                        tc_tensor_copy_4d(st32, &xmap, ci0, x0 + xs, y0 - p.pad, img, full);
                        for (int k = 0; k < nb; ++k)
                            tc_bulk_copy(st32 + p.a_bytes + k * kTcBBytes, p.wblk + (size_t)(b0 + k) * kTcBBytes, (unsigned)kTcBBytes, full);
                    }
                }
                if (++s == S) { s = 0; ++round; }
                __syncwarp();
            }
            mine = ahead;
        }
    } else if (tid == 32) {
        // multiply-add issuer
        const unsigned idesc = tc_instr_desc();
        int s = 0;
        unsigned round = 0, first = 1;
        for (int i = 0; i < n_grp; ++i) {
            if (!tc_wait(bars + s * 8, round & 1u)) break;
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            const unsigned st32 = base32 + s * p.stage_bytes;
            int rows = smask[s];
            unsigned b0 = st32 + p.a_bytes;
            while (rows) {
                const int ky = __ffs(rows) - 1;
                rows &= rows - 1;
                const unsigned a0 = st32 + ky * kTcRowBytes;   // patch rows ky .. ky + 7
#pragma unroll
                for (int k = 0; k < kTcK / 32; ++k) {
                    tc_mma_i8(tmem, tc_smem_desc(a0 + k * 32), tc_smem_desc(b0 + k * 32), idesc, first ? 0u : 1u);
                    first = 0;
                }
                b0 += kTcBBytes;
            }
            tc_commit(bars + (S + s) * 8);   // the stage is free when these multiply-adds have read it
            if (++s == S) { s = 0; ++round; }
        }
        tc_commit(bars + 2 * S * 8);         // everything issued so far has completed
    }

    // ---- epilogue: warp w owns accumulator rows 32 w .. 32 w + 31 (thread = row = pixel) ----
    __syncwarp();
    bool have = n_grp > 0;
    if (have) have = tc_wait(bars + 2 * S * 8, 0u);
    have = __all_sync(0xffffffffu, have) != 0;   // the tensor-memory loads below are warp-wide
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const int m = warp * 32 + lane;
    const int oy = y0 + m / kTcBW, ox = x0 + m % kTcBW;
    const bool inside = oy < p.h_out && ox < p.w_out;
    const size_t pix = ((size_t)img * p.h_out + oy) * p.w_out + ox;
#pragma unroll
    for (int half = 0; half < kTcN / 32; ++half) {
        int v[32];
        __syncwarp();   // the tensor-memory load is warp-wide
        if (have) {
            tc_ld32(tmem + ((unsigned)(warp * 32) << 16) + half * 32, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0;
        }
        if (!inside) continue;
        const int c0 = nt * kTcN + half * 32;
        if (p.acc) {
            int *dst = p.acc + pix * p.c_out + c0;
#pragma unroll
            for (int j = 0; j < 32; j += 4) *reinterpret_cast<int4 *>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            continue;
        }
        // no sparse remainder: requantize here (same arithmetic as the sparse kernel's epilogue)
        const size_t oi = pix * p.ldc + p.c_off + c0;
        if (p.out_dtype == CADNN_S32) {
            int *dst = reinterpret_cast<int *>(p.y) + oi;
            if (p.vec_ok) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) *reinterpret_cast<int4 *>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[j] = v[j];
            }
            continue;
        }
        const bool has_res = p.residual != nullptr;
        union { int4 q[2]; signed char b[32]; } res;
        res.q[0] = res.q[1] = make_int4(0, 0, 0, 0);
        if (has_res) {
            const int4 *rp = reinterpret_cast<const int4 *>(p.residual + pix * p.c_out + c0);
            asm volatile("ld.global.v4.s32 {%0, %1, %2, %3}, [%4];\n" : "=r"(res.q[0].x), "=r"(res.q[0].y), "=r"(res.q[0].z), "=r"(res.q[0].w) : "l"(rp));
            asm volatile("ld.global.v4.s32 {%0, %1, %2, %3}, [%4];\n" : "=r"(res.q[1].x), "=r"(res.q[1].y), "=r"(res.q[1].z), "=r"(res.q[1].w) : "l"(rp + 1));
        }
        if (p.out_dtype == CADNN_F32) {
            float o[32];
#pragma unroll
            for (int j = 0; j < 32; ++j)
                o[j] = requant_f32(v[j], p.scale ? __ldg(p.scale + c0 + j) : 1.0f, p.bias ? __ldg(p.bias + c0 + j) : 0.0f, p.act,
                                   has_res, (int)res.b[j], p.res_scale);
            float *dst = reinterpret_cast<float *>(p.y) + oi;
            if (p.vec_ok) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4 *>(dst + j) = make_float4(o[j], o[j + 1], o[j + 2], o[j + 3]);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[j] = o[j];
            }
        } else {
            union { int4 q[2]; signed char b[32]; } out;
#pragma unroll
            for (int j = 0; j < 32; ++j)
                out.b[j] = (signed char)requant_s8(v[j], p.scale ? __ldg(p.scale + c0 + j) : 1.0f, p.bias ? __ldg(p.bias + c0 + j) : 0.0f,
                                                   p.act, has_res, (int)res.b[j], p.res_scale);
            int8_t *dst = reinterpret_cast<int8_t *>(p.y) + oi;
            if (p.vec_ok) {
                *reinterpret_cast<int4 *>(dst) = out.q[0];
                *reinterpret_cast<int4 *>(dst + 16) = out.q[1];
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) dst[j] = out.b[j];
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(64u) : "memory");
}

}  // namespace

// ---- host: block extraction (called by the packer) and launch --------------------------------

// Finds the dense blocks of an int8 stride-1 conv: for every tile of 64 output channels, tap and chunk of 64
// input channels, the block is taken when the mask keeps at least `threshold` of its 4096 positions.  Fills the
// handle's tensor-core image and clears those positions in rem_mask (what the sparse kernel still has to do).
bool block_tc_extract(cadnn_weights *h, const int8_t *q, const uint8_t *mask, double threshold, std::vector<uint8_t> &rem_mask)
{
    const cadnn_layer_desc &d = h->desc;
    if (d.dtype != CADNN_S8 || d.stride != 1 || d.groups != 1 || d.c_in % kTcK || d.c_out % kTcN || !q) return false;
    if (d.in_h + 2 * d.pad - d.kh + 1 != h->h_out || d.c_in < kTcK) return false;
    const size_t numel = (size_t)d.c_out * d.kh * d.kw * d.c_in;
    rem_mask.assign(numel, 1);
    if (mask) memcpy(rem_mask.data(), mask, numel);
    if (d.kh > 16 || kTcRowBytes * (kTcBH + d.kh - 1) + d.kh * kTcBBytes > kTcSmemBudget / 2) return false;   // two stages must fit
    const int n_nt = d.c_out / kTcN, n_ck = d.c_in / kTcK;
    h->tc_tile_ptr.assign(n_nt + 1, 0);
    h->tc_grp_ptr.assign(n_nt + 1, 0);
    h->tc_blk.clear();
    h->tc_grp.clear();
    h->tc_wblk.clear();
    h->tc_kept.clear();
    h->tc_nnz = 0;
    // blocks in the order (channel tile, input chunk, kernel column, kernel row): the blocks of one kernel column
    // form a group that shares its staged input patch
    for (int nt = 0; nt < n_nt; ++nt) {
        h->tc_tile_ptr[nt] = (int32_t)(h->tc_blk.size() / 4);
        h->tc_grp_ptr[nt] = (int32_t)(h->tc_grp.size() / 4);
        for (int ck = 0; ck < n_ck; ++ck)
            for (int kx = 0; kx < d.kw; ++kx) {
                int rows = 0;
                const int first_block = (int)(h->tc_blk.size() / 4);
                for (int ky = 0; ky < d.kh; ++ky) {
                    int kept = 0;
                    for (int r = 0; r < kTcN; ++r) {
                        const size_t wi = ((((size_t)(nt * kTcN + r)) * d.kh + ky) * d.kw + kx) * d.c_in + (size_t)ck * kTcK;
                        for (int c = 0; c < kTcK; ++c) kept += rem_mask[wi + c] != 0;
                    }
                    if (kept == 0 || (double)kept < threshold * kTcN * kTcK) continue;
                    const size_t at = h->tc_wblk.size();
                    h->tc_wblk.resize(at + kTcBBytes, 0);
                    h->tc_kept.resize(at + kTcBBytes, 0);
                    for (int r = 0; r < kTcN; ++r) {
                        const size_t wi = ((((size_t)(nt * kTcN + r)) * d.kh + ky) * d.kw + kx) * d.c_in + (size_t)ck * kTcK;
                        for (int c = 0; c < kTcK; ++c) {
                            // K-major row of 64 bytes, its 16-byte chunks permuted by the 64-byte swizzle:
                            // chunk ^= (row / 2) % 4
                            const int chunk = (c >> 4) ^ ((r >> 1) & 3);
                            const size_t o = at + (size_t)r * kTcK + (size_t)chunk * 16 + (c & 15);
                            if (rem_mask[wi + c]) {
                                h->tc_wblk[o] = q[wi + c];
                                h->tc_kept[at + (size_t)r * kTcK + c] = 1;
                                rem_mask[wi + c] = 0;
                                ++h->tc_nnz;
                            }
                        }
                    }
                    h->tc_blk.push_back(kx - d.pad_w);
                    h->tc_blk.push_back(ky - d.pad);
                    h->tc_blk.push_back(ck * kTcK);
                    h->tc_blk.push_back(0);
                    rows |= 1 << ky;
                }
                if (rows) {
                    h->tc_grp.push_back(kx - d.pad_w);
                    h->tc_grp.push_back(ck * kTcK);
                    h->tc_grp.push_back(rows);
                    h->tc_grp.push_back(first_block);
                }
            }
    }
    h->tc_tile_ptr[n_nt] = (int32_t)(h->tc_blk.size() / 4);
    h->tc_grp_ptr[n_nt] = (int32_t)(h->tc_grp.size() / 4);
    h->has_tc = true;
    return true;
}

cadnn_status block_tc_upload(cadnn_weights *h)
{
    if (!h->has_tc) return CADNN_OK;
    auto al = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t b_w = h->tc_wblk.size(), b_b = h->tc_grp.size() * 4, b_t = h->tc_grp_ptr.size() * 4;
    h->packed_bytes += (int64_t)(b_w + b_b + b_t);
    if (h->desc.flags & CADNN_PACK_HOST_ONLY) return CADNN_OK;
    const size_t total = al(b_w) + al(b_b) + al(b_t) + 256;
    cudaError_t e = cudaMalloc(&h->d_tc_blob, total);
    if (e != cudaSuccess) {
        cadnn_note_cuda(e);
        return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
    }
    char *base = (char *)h->d_tc_blob;
    if (b_w) CADNN_CUDA_TRY(cudaMemcpy(base, h->tc_wblk.data(), b_w, cudaMemcpyHostToDevice));
    if (b_b) CADNN_CUDA_TRY(cudaMemcpy(base + al(b_w), h->tc_grp.data(), b_b, cudaMemcpyHostToDevice));
    CADNN_CUDA_TRY(cudaMemcpy(base + al(b_w) + al(b_b), h->tc_grp_ptr.data(), b_t, cudaMemcpyHostToDevice));
    CADNN_CUDA_TRY(cudaStreamSynchronize(cudaStreamLegacy));
    h->d_tc_wblk = (const int8_t *)base;
    h->d_tc_grp = (const int32_t *)(base + al(b_w));
    h->d_tc_grp_ptr = (const int32_t *)(base + al(b_w) + al(b_b));
    return CADNN_OK;
}

cadnn_status launch_block_tc(const cadnn_weights *w, const void *x, int n, int *acc, void *y, const LaunchEpilogue *le, cudaStream_t st)
{
    const cadnn_layer_desc &d = w->desc;
    if (!w->has_tc || !w->d_tc_grp_ptr || (!acc && !(y && le))) return CADNN_E_ARG;
    TcParams p = {};
    p.wblk = w->d_tc_wblk;
    p.grp = (const int4 *)w->d_tc_grp;
    p.grp_ptr = w->d_tc_grp_ptr;
    p.kh = d.kh; p.pad = d.pad;
    p.a_bytes = kTcRowBytes * (kTcBH + d.kh - 1);
    p.stage_bytes = p.a_bytes + d.kh * kTcBBytes;
    p.stages = std::min(kTcMaxStages, kTcSmemBudget / p.stage_bytes);
    if (p.stages < 2) return CADNN_E_UNSUPPORTED;
    p.acc = acc;
    if (!acc) {
        p.y = y;
        p.scale = le->scale; p.bias = le->bias;
        p.residual = (const int8_t *)le->residual;
        p.res_scale = le->res_scale;
        p.act = le->act; p.out_dtype = le->out_dtype;
        p.ldc = le->out_c_total > 0 ? le->out_c_total : d.c_out;
        p.c_off = le->out_c_total > 0 ? le->out_c_off : 0;
        const int esz = le->out_dtype == CADNN_S8 ? 1 : 4;
        p.vec_ok = (p.ldc * esz) % 16 == 0 && (p.c_off * esz) % 16 == 0;
    }
    p.h_out = w->h_out; p.w_out = w->w_out; p.c_out = d.c_out;
    p.tiles_x = (w->w_out + kTcBW - 1) / kTcBW;
    p.tiles_y = (w->h_out + kTcBH - 1) / kTcBH;
    p.n_ntiles = d.c_out / kTcN;
    const long long blocks = (long long)n * p.tiles_y * p.tiles_x * p.n_ntiles;
    if (blocks <= 0) return CADNN_OK;
    if (blocks > 2147483647LL) return CADNN_E_UNSUPPORTED;
    // more blocks than multiprocessors: two blocks per multiprocessor with half the ring each
    if (blocks > 148) p.stages = std::max(2, std::min(p.stages, kTcSmemBudget / 2 / p.stage_bytes));
    alignas(64) CUtensorMap map;
    if (!encode_nhwc_s8_tiles_map(&map, x, d.c_in, d.in_w, d.in_h, n, kTcK, kTcBW, kTcBH + d.kh - 1)) return CADNN_E_UNSUPPORTED;
    const int smem = p.stages * p.stage_bytes + (2 * p.stages + 1) * 8 + 16 + p.stages * 4 + 1024;
    static SmemLimit lim;
    cadnn_status rs = raise_smem_limit((const void *)block_tc_kernel, smem, &lim);
    if (rs != CADNN_OK) return rs;
    block_tc_kernel<<<(unsigned)blocks, 128, smem, st>>>(p, map);
    CADNN_CUDA_TRY(cudaGetLastError());
    return CADNN_OK;
}
