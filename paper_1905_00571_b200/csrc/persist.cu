// Persistent whole-network kernel for runs of sparse convolutions over channel-planar
// activations.
//
// CADNN (arXiv 1905.00571), Section 4, "Model computation fusion and transformation": layers
// are fused into larger kernels to cut the cost between them.  At batch 1 a pruned layer's
// work (a fraction of a microsecond at the machine's peak) is far below the cost of a kernel
// boundary, so here a whole run of sparse conv layers executes inside ONE cooperative kernel:
//   * the grid is exactly as many thread blocks as fit on the device at once; each block keeps
//     its 16 warps for the whole run;
//   * a layer is cut into tasks (pixel tile of 32 T consecutive plane positions) x (filter);
//     a slot of KSW warps takes tasks round robin, filter fastest (warps running together read
//     the same activations) and filters in order of decreasing nonzero count (long rows first);
//     the KSW warps of a slot split the filter's nonzeros and add their partial sums through
//     shared memory;
//   * the multiply-add loop is the direct planar one: the lanes of a warp are 32 consecutive
//     positions, a stored nonzero is {value, element offset}, activations come straight from
//     L1 / L2, the zero halo of the layout is the convolution's padding;
//   * layers that do not read each other's output (a bottleneck's downsample branch and its first
//     1x1 conv) share a phase; between phases all blocks meet at a barrier in global memory
//     (release / acquire at device scope).  Every wait on it is bounded: a block that gives up
//     raises a device flag (see cadnn_device_status) and carries on.
// Activations are read with ordinary (coherent) loads, never through the read-only path:
// they are written inside this same kernel.  The stored weights never change and use __ldg.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>
#include "cadnn_internal.h"

// set when a wait on the grid barrier ran out (never expected)
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

const int kPersistWarps = 16;            // warps per block
const unsigned kBarrierSpinLimit = 1u << 22;   // polls of the barrier word before a block gives up (seconds)

struct PersistOp {
    const float *x;
    float *y;
    const uint4 *ent;       // pairs of {value bits, element offset}
    const int32_t *ptr;     // [c_out + 1] in entries (even), by output channel
    const int32_t *order;   // [c_out] output channels by decreasing nonzero count
    const float *scale;
    const float *bias;
    const float *residual;
    int c_in, c_out;
    int wp_in, plane_in, wp_out, plane_out, h_out, w_out;
    int stride, halo, qtot;
    int T, tiles, act;
    int n_tasks;            // images x tiles x filters
    FastDiv d_wp_out, d_cout, d_tiles;
};

struct PersistPhase {
    int first_op, n_ops;
    int ksw_shift;          // log2 of the warps of a slot
    int pad;
};

__device__ __forceinline__ float pp_act(float z, int act)
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

__device__ __forceinline__ void slot_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;\n" ::"r"(id), "r"(threads) : "memory");
}

// All blocks of the grid have finished the phase when this returns (or the wait ran out).
__device__ __forceinline__ void grid_barrier(unsigned *arrive, unsigned target)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();   // this block's stores are visible device-wide before it arrives
        atomicAdd(arrive, 1u);
        unsigned spins = 0;
        while (ld_acquire(arrive) < target) {
            if (++spins > kBarrierSpinLimit) {
                atomicAdd(&g_barrier_timeout, 1);
                break;
            }
        }
        __threadfence();
    }
    __syncthreads();
}

// One task: T bands of 32 positions of one filter; the KSW warps of the slot split its nonzeros.
template <int T>
__device__ __forceinline__ void conv_task(const PersistOp &p, int task, int lane, int warp, int slice, int ksw_shift,
                                          int slot_local, float (*sRed)[8][32])
{
    const unsigned r1 = fdiv((unsigned)task, p.d_cout);
    const int frank = task - (int)r1 * p.c_out;
    const unsigned img = fdiv(r1, p.d_tiles);
    const int tile = (int)(r1 - img * p.tiles);
    const int q0 = tile * (32 * T);
    const int co = __ldg(p.order + frank);

    int inb[T];
    unsigned okmask = 0;
#pragma unroll
    for (int t = 0; t < T; ++t) {
        const int q = q0 + 32 * t + lane;
        const int qc = min(q, p.qtot - 1);
        const int oy = (int)fdiv((unsigned)qc, p.d_wp_out);
        const int oxp = qc - oy * p.wp_out;
        const bool ok = q < p.qtot && oxp >= p.halo && oxp < p.halo + p.w_out;
        if (ok) okmask |= 1u << t;
        const int oxs = ok ? oxp : p.halo;   // lanes that store nothing still load inside the plane
        inb[t] = (oy * p.stride) * p.wp_in + (oxs - p.halo) * p.stride;
    }
    const float *ximg = p.x + (size_t)img * p.c_in * p.plane_in;
    const int KSW = 1 << ksw_shift;

    float acc[T];
#pragma unroll
    for (int t = 0; t < T; ++t) acc[t] = 0.0f;
    {
        const int rbeg = __ldg(p.ptr + co) >> 1, rend = __ldg(p.ptr + co + 1) >> 1;   // in pairs
        const int per = (rend - rbeg + KSW - 1) >> ksw_shift;
        const int beg = min(rend, rbeg + slice * per), end = min(rend, beg + per);
        constexpr int P = T == 1 ? 8 : T == 2 ? 4 : T == 4 ? 2 : 1;   // pairs per batch
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
        slot_barrier(1 + slot_local, KSW * 32);
        if (slice == 0) {
            for (int s2 = 1; s2 < KSW; ++s2)
#pragma unroll
                for (int t = 0; t < T; ++t) acc[t] += sRed[warp + s2][t][lane];
        }
        slot_barrier(1 + slot_local, KSW * 32);   // sRed is reused by the slot's next task
    }
    if (slice == 0) {
        const float sc = p.scale ? __ldg(p.scale + co) : 1.0f;
        const float bi = p.bias ? __ldg(p.bias + co) : 0.0f;
        const size_t obase = ((size_t)img * p.c_out + co) * p.plane_out + (size_t)p.halo * p.wp_out + q0 + lane;
#pragma unroll
        for (int t = 0; t < T; ++t) {
            if (okmask & (1u << t)) {
                const size_t oi = obase + 32 * t;
                float z = fmaf(acc[t], sc, bi);
                if (p.residual) z += ld_act(p.residual + oi);
                p.y[oi] = pp_act(z, p.act);
            }
        }
    }
}

__global__ void __launch_bounds__(kPersistWarps * 32, 2)
net_persistent_kernel(const PersistOp *ops, const PersistPhase *phases, int n_phases, unsigned *sync)
{
    __shared__ float sRed[kPersistWarps][8][32];
    __shared__ PersistOp sOp;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned target = 0;
    for (int ph = 0; ph < n_phases; ++ph) {
        const int first_op = __ldg(&phases[ph].first_op), n_ops = __ldg(&phases[ph].n_ops);
        const int ksw_shift = __ldg(&phases[ph].ksw_shift);
        const int slots_per_block = kPersistWarps >> ksw_shift;
        const int slot_local = warp >> ksw_shift, slice = warp & ((1 << ksw_shift) - 1);
        const int slot = blockIdx.x * slots_per_block + slot_local;
        const int n_slots = gridDim.x * slots_per_block;
        int base = 0;   // tasks of the phase's earlier ops, modulo the slots
        for (int oi = 0; oi < n_ops; ++oi) {
            // the op's descriptor goes through shared memory once per block
            __syncthreads();
            {
                const int words = (int)(sizeof(PersistOp) / 4);
                const unsigned *src = reinterpret_cast<const unsigned *>(ops + first_op + oi);
                unsigned *dst = reinterpret_cast<unsigned *>(&sOp);
                for (int i = threadIdx.x; i < words; i += blockDim.x) dst[i] = __ldg(src + i);
            }
            __syncthreads();
            const PersistOp &op = sOp;
            int first = slot - base;
            if (first < 0) first += n_slots;
            switch (op.T) {
                case 1:
                    for (int task = first; task < op.n_tasks; task += n_slots)
                        conv_task<1>(op, task, lane, warp, slice, ksw_shift, slot_local, sRed);
                    break;
                case 2:
                    for (int task = first; task < op.n_tasks; task += n_slots)
                        conv_task<2>(op, task, lane, warp, slice, ksw_shift, slot_local, sRed);
                    break;
                case 4:
                    for (int task = first; task < op.n_tasks; task += n_slots)
                        conv_task<4>(op, task, lane, warp, slice, ksw_shift, slot_local, sRed);
                    break;
                default:
                    for (int task = first; task < op.n_tasks; task += n_slots)
                        conv_task<8>(op, task, lane, warp, slice, ksw_shift, slot_local, sRed);
                    break;
            }
            base = (base + op.n_tasks) % n_slots;
        }
        if (ph + 1 < n_phases) {
            target += gridDim.x;
            grid_barrier(sync, target);
        }
    }
    // the last block to leave zeroes the barrier words for the next launch
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned left = atomicAdd(sync + 1, 1u);
        if (left == gridDim.x - 1) {
            sync[0] = 0u;
            sync[1] = 0u;
            __threadfence();
        }
    }
}

size_t round_up_sz(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace

struct PersistPlan {
    int device = -1;
    int n_ops = 0, n_phases = 0;
    int grid = 0;
    void *d_blob = nullptr;   // ops, phases, filter orders, barrier words: one allocation
    const PersistOp *d_ops = nullptr;
    const PersistPhase *d_phases = nullptr;
    unsigned *d_sync = nullptr;
};

int persist_phases(const PersistPlan *plan) { return plan ? plan->n_phases : 0; }

void persist_free(PersistPlan *plan)
{
    if (!plan) return;
    if (plan->d_blob) cudaFree(plan->d_blob);
    delete plan;
}

// Bands per lane and warps per slot of one layer inside the persistent kernel: the packer's
// measured launch shape by default; CADNN_PERSIST_T / CADNN_PERSIST_KSW override both for tuning.
static void persist_shape(const cadnn_weights *w, int *T_out, int *ksw_out)
{
    int T = w->pl_T, ksw = std::max(1, w->pl_KSW);
    int v;
    const char *e;
    if ((e = getenv("CADNN_PERSIST_T")) && sscanf(e, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) T = v;
    if ((e = getenv("CADNN_PERSIST_KSW")) && sscanf(e, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) ksw = v;
    *T_out = T;
    *ksw_out = ksw;
}

cadnn_status persist_create(const std::vector<PersistOpDesc> &descs, PersistPlan **out)
{
    *out = nullptr;
    if (descs.empty()) return CADNN_E_ARG;
    int dev = 0, sms = 0, per_sm = 0, coop = 0;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    CADNN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CADNN_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    if (!coop) return CADNN_E_UNSUPPORTED;
    CADNN_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, net_persistent_kernel, kPersistWarps * 32, 0));
    if (per_sm < 1) return CADNN_E_UNSUPPORTED;
    per_sm = std::min(per_sm, 2);
    const int grid = per_sm * sms;

    const int n_ops = (int)descs.size();
    std::vector<PersistOp> ops(n_ops);
    std::vector<PersistPhase> phases;
    std::vector<std::vector<int32_t>> orders(n_ops);
    std::vector<int> ksw_of(n_ops);
    size_t order_words = 0;
    for (int i = 0; i < n_ops; ++i) {
        const PersistOpDesc &d = descs[i];
        const cadnn_weights *w = d.w;
        if (!w || !w->has_planar || !w->d_pl_ent || !w->d_pl_ptr) return CADNN_E_ARG;
        const cadnn_layer_desc &ld = w->desc;
        const int halo = kPlanarHalo;
        PersistOp &p = ops[i];
        p.x = (const float *)d.x; p.y = (float *)d.y;
        p.ent = (const uint4 *)w->d_pl_ent; p.ptr = w->d_pl_ptr; p.order = nullptr;
        p.scale = d.scale; p.bias = d.bias; p.residual = (const float *)d.residual;
        p.c_in = ld.c_in; p.c_out = ld.c_out;
        p.wp_in = ld.in_w + 2 * halo; p.plane_in = planar_pitch(ld.in_h, ld.in_w);
        p.h_out = w->h_out; p.w_out = w->w_out;
        p.wp_out = w->w_out + 2 * halo; p.plane_out = planar_pitch(w->h_out, w->w_out);
        p.stride = ld.stride; p.halo = halo; p.qtot = w->h_out * p.wp_out;
        int T, ksw;
        persist_shape(w, &T, &ksw);
        p.T = T;
        ksw_of[i] = ksw;
        p.tiles = (p.qtot + 32 * T - 1) / (32 * T);
        p.act = d.act;
        const long long tasks = (long long)d.n * p.tiles * ld.c_out;
        if (tasks <= 0 || tasks > 2147483647LL) return CADNN_E_UNSUPPORTED;
        p.n_tasks = (int)tasks;
        p.d_wp_out = make_fastdiv(p.wp_out);
        p.d_cout = make_fastdiv(ld.c_out);
        p.d_tiles = make_fastdiv(p.tiles);
        // filters by decreasing stored nonzeros (ties by channel): the long rows start first
        std::vector<int32_t> &ord = orders[i];
        ord.resize(ld.c_out);
        std::iota(ord.begin(), ord.end(), 0);
        if ((int)w->row_nnz.size() == ld.c_out)
            std::stable_sort(ord.begin(), ord.end(), [&](int a, int b) { return w->row_nnz[a] > w->row_nnz[b]; });
        order_words += (size_t)ld.c_out;
        // phases: an op joins the current phase unless it reads what that phase writes
        bool joins = !phases.empty() && d.join_phase;
        if (joins) {
            PersistPhase &ph = phases.back();
            ph.n_ops += 1;
            ph.ksw_shift = std::max(ph.ksw_shift, ksw >= 8 ? 3 : ksw >= 4 ? 2 : ksw >= 2 ? 1 : 0);
        } else {
            PersistPhase ph;
            ph.first_op = i; ph.n_ops = 1; ph.pad = 0;
            ph.ksw_shift = ksw >= 8 ? 3 : ksw >= 4 ? 2 : ksw >= 2 ? 1 : 0;
            phases.push_back(ph);
        }
    }

    const size_t ops_bytes = round_up_sz(sizeof(PersistOp) * ops.size(), 256);
    const size_t ph_bytes = round_up_sz(sizeof(PersistPhase) * phases.size(), 256);
    const size_t ord_bytes = round_up_sz(order_words * 4, 256);
    const size_t total = ops_bytes + ph_bytes + ord_bytes + 256;
    PersistPlan *plan = new (std::nothrow) PersistPlan();
    if (!plan) return CADNN_E_ALLOC;
    cudaError_t e = cudaMalloc(&plan->d_blob, total);
    if (e != cudaSuccess) {
        delete plan;
        cadnn_note_cuda(e);
        return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
    }
    unsigned char *base = (unsigned char *)plan->d_blob;
    std::vector<unsigned char> host(total, 0);
    {
        int32_t *ord_dev = (int32_t *)(base + ops_bytes + ph_bytes);
        int32_t *ord_host = (int32_t *)(host.data() + ops_bytes + ph_bytes);
        size_t at = 0;
        for (int i = 0; i < n_ops; ++i) {
            ops[i].order = ord_dev + at;
            std::copy(orders[i].begin(), orders[i].end(), ord_host + at);
            at += orders[i].size();
        }
        memcpy(host.data(), ops.data(), sizeof(PersistOp) * ops.size());
        memcpy(host.data() + ops_bytes, phases.data(), sizeof(PersistPhase) * phases.size());
    }
    e = cudaMemcpy(plan->d_blob, host.data(), total, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        persist_free(plan);
        return cadnn_note_cuda(e);
    }
    plan->device = dev;
    plan->n_ops = n_ops;
    plan->n_phases = (int)phases.size();
    plan->grid = grid;
    plan->d_ops = (const PersistOp *)base;
    plan->d_phases = (const PersistPhase *)(base + ops_bytes);
    plan->d_sync = (unsigned *)(base + ops_bytes + ph_bytes + ord_bytes);
    *out = plan;
    return CADNN_OK;
}

cadnn_status persist_launch(const PersistPlan *plan, cudaStream_t st)
{
    if (!plan) return CADNN_E_ARG;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)plan->grid, 1, 1);
    cfg.blockDim = dim3(kPersistWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;   // all blocks resident at once, or the launch fails
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    CADNN_CUDA_TRY(cudaLaunchKernelEx(&cfg, net_persistent_kernel, plan->d_ops, plan->d_phases, plan->n_phases, plan->d_sync));
    return CADNN_OK;
}
