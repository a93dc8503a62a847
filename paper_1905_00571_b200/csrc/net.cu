// Whole-network runner: shape inference over an op list, one device buffer per
// intermediate tensor, layer-by-layer launch or CUDA-graph replay.
//
// CADNN (arXiv 1905.00571), Section 5, reports single-image inference of complete
// networks.  At batch 1 a pruned layer's work is far below a kernel launch, so the
// layer sequence is captured once into a CUDA graph and replayed.
#include <cstdlib>
#include <new>
#include <vector>
#include <cstdio>
#include "cadnn_internal.h"

struct SlotInfo {
    int n = 0, h = 0, w = 0, c = 0, dtype = 0;
    bool defined = false;
    void *ptr = nullptr;  // owned unless slot 0 or the output slot
    int64_t bytes = 0;
    // planar nets: second copy of the tensor split by row and column parity, written by the producing sparse conv for
    // stride-2 readers (owned); par_mask = planes present, bit (row parity * 2 + column parity)
    void *par_ptr = nullptr;
    int par_mask = 0;
};

struct cadnn_net {
    std::vector<cadnn_op> ops;
    std::vector<SlotInfo> slots;
    int out_slot = -1;
    bool use_pdl = true;   // layers after the first launch as programmatic dependents
    bool pdl_graph = true;       // ... also inside captured graphs
    bool early_trigger = false;
    bool fork_branches = true;   // graph capture: ops off the critical path become parallel branches
    bool planar = false;   // intermediate feature maps are channel-planar with a zero halo (planar.cu)
    // run of planar sparse convs [persist_first, persist_last] executed by one persistent kernel (persist.cu)
    PersistPlan *persist = nullptr;
    int persist_first = -1, persist_last = -1;
    int64_t workspace = 0;
    std::vector<char> use_half;   // per op: a stride-2 conv that runs as its stride-1 form over its input's parity planes
    // graph cache: [0] caller's device pointers, [1] the net's own staging buffers
    struct GraphCache {
        cudaGraph_t graph = nullptr;
        cudaGraphExec_t exec = nullptr;
        const void *x = nullptr;
        void *y = nullptr;
    } cache[2];
    // device staging for cadnn_forward_host
    void *stage_x = nullptr, *stage_y = nullptr;
    int64_t in_bytes = 0, out_bytes = 0;
    // int32 sums of block-structured layers (tensor-core blocks), shared by all such ops of the net
    void *tc_ws = nullptr;
    int64_t tc_ws_bytes = 0;
    // L2 flush buffer for layer timing
    void *flush = nullptr;
    size_t flush_bytes = 0;
    // device status words (bounded waits that ran out): pinned host copy written in stream order
    // at the net's synchronization points, and the values seen when the net was created
    int *status_host = nullptr;
    int status_seen[2] = {0, 0};
};

namespace {

void *slot_ptr(cadnn_net *net, int slot, const void *x, void *y)
{
    if (slot == 0) return const_cast<void *>(x);
    if (slot == net->out_slot) return y;
    return net->slots[slot].ptr;
}

cadnn_status run_op(cadnn_net *net, const cadnn_op &op, const void *x, void *y, cudaStream_t st, bool pdl = false)
{
    const SlotInfo &si = net->slots[op.src];
    const void *src = slot_ptr(net, op.src, x, y);
    void *dst = slot_ptr(net, op.dst, x, y);
    if (net->planar && op.kind != CADNN_OP_FC) {
        if (op.kind == CADNN_OP_CONV) {
            LaunchEpilogue le;
            le.scale = op.scale;
            le.bias = op.bias;
            le.residual = op.res >= 0 ? slot_ptr(net, op.res, x, y) : nullptr;
            le.act = op.act;
            le.out_dtype = CADNN_F32;
            le.pdl = pdl;
            le.early_trigger = net->early_trigger;
            const SlotInfo &so = net->slots[op.dst];
            if (so.par_ptr) {
                le.parity_y = (float *)so.par_ptr;
                le.parity_mask = so.par_mask;
            }
            const size_t op_index = (size_t)(&op - net->ops.data());
            if (op_index < net->use_half.size() && net->use_half[op_index]) {
                const cadnn_weights *hw = op.w->half;
                if (hw->has_ps && hw->use_ps) return launch_sconv_planar_staged(hw, si.par_ptr, si.n, dst, le, st);
                return launch_sconv_planar(hw, si.par_ptr, si.n, dst, le, st);
            }
            if (op.w->s.kind == KK_DENSE_SMALLC) {   // the stem reads the NHWC image and writes planes
                le.planar_out = true;
                return launch_dense_smallc(op.w, src, si.n, dst, le, st);
            }
            if (op.w->s.kind == KK_DW) return launch_dw_planar(op.w, src, si.n, dst, le, st);
            if (op.w->has_ps && op.w->use_ps) return launch_sconv_planar_staged(op.w, src, si.n, dst, le, st);
            return launch_sconv_planar(op.w, src, si.n, dst, le, st);
        }
        if (op.kind == CADNN_OP_MAXPOOL)
            return launch_maxpool_planar((const float *)src, si.n, si.h, si.w, si.c, op.pool_k, op.pool_stride,
                                         op.pool_pad, (float *)dst, pdl, st);
        return launch_gavgpool_planar((const float *)src, si.n, si.h, si.w, si.c, (float *)dst, pdl, st);
    }
    if (op.kind == CADNN_OP_CONV || op.kind == CADNN_OP_FC) {
        cadnn_epilogue ep;
        ep.scale = op.scale;
        ep.bias = op.bias;
        ep.residual = op.res >= 0 ? slot_ptr(net, op.res, x, y) : nullptr;
        ep.act = op.act;
        ep.out_dtype = op.out_dtype;
        ep.out_c_total = op.dst_c_total;
        ep.out_c_off = op.dst_c_off;
        ep.residual_scale = op.res_scale;
        if (op.kind == CADNN_OP_FC) return conv2d_impl(op.w, src, si.n, 1, 1, dst, &ep, pdl, st);
        return conv2d_impl(op.w, src, si.n, si.h, si.w, dst, &ep, pdl, st, net->tc_ws, net->tc_ws_bytes);
    }
    if (op.kind == CADNN_OP_MAXPOOL || op.kind == CADNN_OP_AVGPOOL)
        return launch_pool_window(src, si.n, si.h, si.w, si.c, op.pool_k, op.pool_stride, op.pool_pad, si.dtype,
                                  op.kind == CADNN_OP_AVGPOOL ? 1 : 0, dst, op.dst_c_total, op.dst_c_off, pdl, st);
    if (op.kind == CADNN_OP_GAVGPOOL)
        return launch_gavgpool((const float *)src, si.n, si.h, si.w, si.c, (float *)dst, pdl, st);
    return CADNN_E_ARG;
}

// With pdl, every op after the first is launched as a programmatic dependent of its
// predecessor: its prologue (weights, tables) overlaps the predecessor's stores, and it waits
// on the grid dependency before touching activations.  Measured on the pruned ResNet-50 at
// batch 1 (channel-planar kernels) it shortens both stream launches and graph replays
// (450 -> 444 us per replay; 429 us together with the forked branches of run_all_forked).
cadnn_status run_all(cadnn_net *net, const void *x, void *y, cudaStream_t st, bool pdl = false)
{
    bool first = true;
    const int n_ops = (int)net->ops.size();
    for (int i = 0; i < n_ops; ++i) {
        if (net->persist && i == net->persist_first) {
            // the whole run of sparse convs is one cooperative launch; its successor takes a full dependency on it
            cadnn_status s = persist_launch(net->persist, st);
            if (s != CADNN_OK) return s;
            i = net->persist_last;
            first = true;
            continue;
        }
        cadnn_status s = run_op(net, net->ops[i], x, y, st, pdl && !first);
        if (s != CADNN_OK) return s;
        first = false;
    }
    return CADNN_OK;
}

// Capture-time variant of run_all: an op whose result the next op does not read (a bottleneck's
// downsample conv, whose result is only needed as the residual of the block's last conv) is
// issued on a second stream, forked from and joined back to the captured one with events, so
// that in the graph it is a parallel branch.  At batch 1 no single layer fills the device, so
// the branch runs beside the block's first convs instead of in front of them.
cadnn_status run_all_forked(cadnn_net *net, const void *x, void *y, cudaStream_t st, cudaStream_t side, bool pdl)
{
    const int n_ops = (int)net->ops.size();
    std::vector<cudaEvent_t> join(n_ops, nullptr);   // recorded on the side stream after op i
    std::vector<cudaEvent_t> events;
    cadnn_status rs = CADNN_OK;
    auto new_event = [&](cudaEvent_t *e) {
        if (cudaEventCreateWithFlags(e, cudaEventDisableTiming) != cudaSuccess) return false;
        events.push_back(*e);
        return true;
    };
    bool first = true;
    for (int i = 0; i < n_ops && rs == CADNN_OK; ++i) {
        if (net->persist && i == net->persist_first) {
            rs = persist_launch(net->persist, st);
            i = net->persist_last;
            first = true;
            continue;
        }
        const cadnn_op &op = net->ops[i];
        // join the branches this op reads
        for (int j = 0; j < i; ++j) {
            if (!join[j]) continue;
            const int dj = net->ops[j].dst;
            if (dj == op.src || dj == op.res) {
                if (cudaStreamWaitEvent(st, join[j], 0) != cudaSuccess) rs = CADNN_E_CUDA;
                join[j] = nullptr;
                first = true;   // the next launch must not be a programmatic dependent across the join
            }
        }
        if (rs != CADNN_OK) break;
        bool branch = false;
        if (i + 1 < n_ops && i > 0 && op.dst != net->out_slot) {
            const cadnn_op &nx = net->ops[i + 1];
            const bool inside_run = net->persist && i + 1 >= net->persist_first && i + 1 <= net->persist_last;
            branch = nx.src != op.dst && nx.res != op.dst && !inside_run;
        }
        if (branch) {
            cudaEvent_t fork = nullptr;
            if (!new_event(&fork) || !new_event(&join[i]) || cudaEventRecord(fork, st) != cudaSuccess ||
                cudaStreamWaitEvent(side, fork, 0) != cudaSuccess) { rs = CADNN_E_CUDA; break; }
            rs = run_op(net, op, x, y, side, false);
            if (rs == CADNN_OK && cudaEventRecord(join[i], side) != cudaSuccess) rs = CADNN_E_CUDA;
        } else {
            rs = run_op(net, op, x, y, st, pdl && !first);
            first = false;
        }
    }
    // branches nobody read still have to end inside the capture
    for (int j = 0; j < n_ops; ++j)
        if (join[j] && cudaStreamWaitEvent(st, join[j], 0) != cudaSuccess && rs == CADNN_OK) rs = CADNN_E_CUDA;
    for (cudaEvent_t e : events) cudaEventDestroy(e);
    if (rs == CADNN_E_CUDA) cadnn_note_cuda(cudaGetLastError());
    return rs;
}

// Capture-time scheduling of a general op list (no persistent run): every op depends on the ops that wrote the
// tensors it reads (all writers of a concatenated slot) and, for block-structured layers, on the previous user of
// the shared int32 workspace.  Ops are issued on a few streams ("lanes"): an op continues the lane whose last op
// it depends on, otherwise it takes the lane that has been quiet longest and waits for its producers' events -
// so the branches of a residual block or of an Inception module become parallel branches of the graph.
cadnn_status run_all_dag(cadnn_net *net, const void *x, void *y, cudaStream_t st, cudaStream_t *sides, int n_sides, bool pdl)
{
    const int n_ops = (int)net->ops.size();
    const int n_lanes = 1 + n_sides;
    std::vector<cudaStream_t> lane(n_lanes);
    lane[0] = st;
    for (int k = 0; k < n_sides; ++k) lane[1 + k] = sides[k];
    std::vector<int> tail(n_lanes, -1);        // last op issued on the lane
    std::vector<bool> live(n_lanes, false);    // the lane has joined the capture
    live[0] = true;
    std::vector<int> lane_of(n_ops, 0);
    std::vector<cudaEvent_t> done(n_ops, nullptr);
    cadnn_status rs = CADNN_OK;
    int last_ws_user = -1;
    for (int i = 0; i < n_ops && rs == CADNN_OK; ++i) {
        const cadnn_op &op = net->ops[i];
        std::vector<int> deps;
        int src_writer = -1;
        for (int j = 0; j < i; ++j) {
            const int dj = net->ops[j].dst;
            if (dj == op.src) { deps.push_back(j); src_writer = j; }
            else if (dj == op.res) deps.push_back(j);
        }
        const bool uses_ws = (op.kind == CADNN_OP_CONV) && op.w && op.w->has_tc && op.w->nnz != op.w->tc_nnz;
        if (uses_ws && last_ws_user >= 0) deps.push_back(last_ws_user);
        // lane: continue the producer of the input if it is a lane's last op, else any producer that is, else the quietest live
        // lane or a lane not used yet (ops without producers stay on the captured stream itself)
        // An op nobody reads next (a downsample conv, a one-conv branch) whose input has other readers leaves the
        // producer's lane to them: the chain that follows keeps its programmatic launches.
        bool yields = false;
        if (src_writer >= 0 && i + 1 < n_ops && net->ops[i + 1].src != op.dst && net->ops[i + 1].res != op.dst) {
            int readers = 0;
            for (int k = src_writer + 1; k < n_ops; ++k)
                readers += net->ops[k].src == op.src || net->ops[k].res == op.src;
            yields = readers > 1;
        }
        int l = -1;
        if (deps.empty()) l = 0;
        if (l < 0 && !yields && src_writer >= 0 && tail[lane_of[src_writer]] == src_writer) l = lane_of[src_writer];
        for (size_t d = 0; d < deps.size() && l < 0 && !yields; ++d)
            if (tail[lane_of[deps[d]]] == deps[d]) l = lane_of[deps[d]];
        if (l < 0) {
            for (int k = 0; k < n_lanes; ++k) {
                if (yields && src_writer >= 0 && k == lane_of[src_writer] && tail[k] == src_writer) continue;
                if (l < 0 || tail[k] < tail[l]) l = k;
            }
            if (l < 0) l = 0;
        }
        bool waited = false;
        for (int d : deps) {
            if (lane_of[d] == l) continue;   // stream order
            if (cudaStreamWaitEvent(lane[l], done[d], 0) != cudaSuccess) { rs = CADNN_E_CUDA; break; }
            waited = true;
            live[l] = true;
        }
        if (rs != CADNN_OK) break;
        if (!live[l]) { l = 0; }   // cannot happen (a lane goes live with its first wait); stay inside the capture
        // launched behind a kernel of its own lane with no event wait in between: may be its programmatic dependent (what it
        // reads was written on this lane before that kernel, or by it)
        const bool chain = tail[l] >= 0 && !waited;
        rs = run_op(net, op, x, y, lane[l], pdl && chain);
        if (rs != CADNN_OK) break;
        if (cudaEventCreateWithFlags(&done[i], cudaEventDisableTiming) != cudaSuccess || cudaEventRecord(done[i], lane[l]) != cudaSuccess) {
            rs = CADNN_E_CUDA;
            break;
        }
        tail[l] = i;
        lane_of[i] = l;
        if (uses_ws) last_ws_user = i;
    }
    // every lane ends inside the capture
    for (int k = 1; k < n_lanes; ++k)
        if (live[k] && tail[k] >= 0 && done[tail[k]] && cudaStreamWaitEvent(st, done[tail[k]], 0) != cudaSuccess && rs == CADNN_OK)
            rs = CADNN_E_CUDA;
    for (cudaEvent_t e : done)
        if (e) cudaEventDestroy(e);
    if (rs == CADNN_E_CUDA) cadnn_note_cuda(cudaGetLastError());
    return rs;
}

// Plan the persistent kernel over the longest run of consecutive planar sparse convs whose
// tensors all live in slots the net owns.  Leaves net->persist null when there is no such run
// (or the device cannot launch cooperatively); the layer-by-layer path then runs everything.
void plan_persistent(cadnn_net *net)
{
    const int n_ops = (int)net->ops.size();
    auto owned = [&](int slot) { return slot > 0 && slot != net->out_slot && net->slots[slot].ptr != nullptr; };
    auto eligible = [&](const cadnn_op &op) {
        return op.kind == CADNN_OP_CONV && op.w && op.w->has_planar && op.w->s.kind != KK_DENSE_SMALLC &&
               !op.w->pl_ptr.empty() && owned(op.src) && owned(op.dst) && (op.res < 0 || owned(op.res));
    };
    int best_lo = -1, best_len = 0;
    for (int i = 0; i < n_ops;) {
        if (!eligible(net->ops[i])) { ++i; continue; }
        int j = i;
        while (j < n_ops && eligible(net->ops[j])) ++j;
        if (j - i > best_len) { best_len = j - i; best_lo = i; }
        i = j;
    }
    if (best_len < 3) return;
    std::vector<PersistOpDesc> descs;
    std::vector<int> phase_dsts;
    for (int i = best_lo; i < best_lo + best_len; ++i) {
        const cadnn_op &op = net->ops[i];
        PersistOpDesc d;
        d.w = op.w;
        d.x = net->slots[op.src].ptr;
        d.y = net->slots[op.dst].ptr;
        d.residual = op.res >= 0 ? net->slots[op.res].ptr : nullptr;
        d.scale = op.scale;
        d.bias = op.bias;
        d.act = op.act;
        d.n = net->slots[op.src].n;
        d.dst_external = i == best_lo + best_len - 1;
        for (int j = 0; j < n_ops; ++j)
            if ((j < best_lo || j >= best_lo + best_len) && (net->ops[j].src == op.dst || net->ops[j].res == op.dst)) d.dst_external = true;
        bool reads_phase = false;
        for (int s : phase_dsts) reads_phase = reads_phase || s == op.src || s == op.res;
        d.join_phase = !descs.empty() && !reads_phase && getenv("CADNN_PERSIST_NO_MERGE") == nullptr;
        if (!d.join_phase) phase_dsts.clear();
        phase_dsts.push_back(op.dst);
        descs.push_back(d);
    }
    PersistPlan *plan = nullptr;
    if (persist_create(descs, &plan) != CADNN_OK) { cudaGetLastError(); return; }
    net->persist = plan;
    net->persist_first = best_lo;
    net->persist_last = best_lo + best_len - 1;
}

void drop_graph(cadnn_net::GraphCache &gc)
{
    if (gc.exec) cudaGraphExecDestroy(gc.exec);
    if (gc.graph) cudaGraphDestroy(gc.graph);
    gc.exec = nullptr;
    gc.graph = nullptr;
}

cadnn_status forward_impl(cadnn_net *net, const void *x, void *y, int use_graph, cudaStream_t st, int slot)
{
    if (!use_graph) return run_all(net, x, y, st, net->use_pdl);
    cadnn_net::GraphCache &gc = net->cache[slot];
    if (!gc.exec || gc.x != x || gc.y != y) {
        drop_graph(gc);
        // run every kernel once outside capture (first launches raise function attributes)
        cadnn_status s = run_all(net, x, y, st);
        if (s != CADNN_OK) return s;
        cudaStream_t cap = st;
        bool own = false;
        if (cap == nullptr || cap == cudaStreamLegacy) {
            CADNN_CUDA_TRY(cudaStreamSynchronize(st));
            CADNN_CUDA_TRY(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
            own = true;
        }
        cudaError_t e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
        if (e != cudaSuccess) { if (own) cudaStreamDestroy(cap); return cadnn_note_cuda(e); }
        const int kSides = 3;
        cudaStream_t sides[kSides] = {nullptr, nullptr, nullptr};
        int n_sides = 0;
        if (net->fork_branches)
            for (; n_sides < kSides; ++n_sides)
                if (cudaStreamCreateWithFlags(&sides[n_sides], cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); break; }
        if (n_sides == 0) s = run_all(net, x, y, cap, net->pdl_graph);
        else {
            // networks with concatenations have branches of several ops (measured on Inception-V3, batch 1: 0.78 ms
            // against 0.87 ms with one-op branches only); residual networks measured the same or slightly slower
            // with the general scheduler, so they keep the simple fork of ops nobody reads next
            bool concat = false;
            for (const cadnn_op &op : net->ops) concat = concat || op.dst_c_total > 0;
            const char *force = getenv("CADNN_GRAPH_LANES");   // "1": general scheduler always, "0": never
            if (force) concat = atoi(force) != 0;
            if (net->persist || !concat) s = run_all_forked(net, x, y, cap, sides[0], net->pdl_graph);
            else s = run_all_dag(net, x, y, cap, sides, n_sides, net->pdl_graph);
        }
        e = cudaStreamEndCapture(cap, &gc.graph);
        for (int k = 0; k < n_sides; ++k) cudaStreamDestroy(sides[k]);
        if (own) cudaStreamDestroy(cap);
        if (s != CADNN_OK) { drop_graph(gc); return s; }
        if (e != cudaSuccess) { drop_graph(gc); return cadnn_note_cuda(e); }
        e = cudaGraphInstantiate(&gc.exec, gc.graph, 0);
        if (e != cudaSuccess) { drop_graph(gc); return cadnn_note_cuda(e); }
        gc.x = x;
        gc.y = y;
    }
    CADNN_CUDA_TRY(cudaGraphLaunch(gc.exec, st));
    return CADNN_OK;
}

// The kernels' waits are bounded; one that ran out leaves a count in a device word.  The net
// reads the words in stream order right before it synchronizes, so a forward whose kernels gave
// up is reported instead of returning wrong numbers silently.
cadnn_status queue_status_read(cadnn_net *net, cudaStream_t st)
{
    cadnn_status s = read_copy_timeouts_async(&net->status_host[0], st);
    if (s == CADNN_OK && net->persist) s = read_barrier_timeouts_async(&net->status_host[1], st);
    return s;
}

// after the stream has been synchronized: did a counter move since the net last looked?
bool status_moved(cadnn_net *net)
{
    const bool moved = net->status_host[0] != net->status_seen[0] || net->status_host[1] != net->status_seen[1];
    net->status_seen[0] = net->status_host[0];
    net->status_seen[1] = net->status_host[1];
    return moved;
}

__global__ void flush_kernel(float *buf, size_t n)
{
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        buf[i] = 0.0f;
}

}  // namespace

namespace {

// Stride-2 layers of a planar net whose handle carries the stride-1 form over parity planes (cadnn_weights::half) use
// it when the layer that writes their input is a sparse conv (its epilogue then stores the parity planes as well) and
// the form measured faster at pack time (CADNN_FORCE_PARITY_PLANES=1: whenever it exists).  A 1x1 reader takes the
// (even, even) plane, which is a tensor of its own only when no 3x3 reader asks for all four.
cadnn_status plan_parity_planes(cadnn_net *net)
{
    const int n_ops = (int)net->ops.size();
    net->use_half.assign(n_ops, 0);
    const char *pe = getenv("CADNN_PERSIST");
    if (!net->planar || getenv("CADNN_NO_PARITY_PLANES") || (pe && atoi(pe) != 0)) return CADNN_OK;
    const bool force = getenv("CADNN_FORCE_PARITY_PLANES") != nullptr;
    std::vector<int> writer(net->slots.size(), -1);
    for (int i = 0; i < n_ops; ++i) writer[net->ops[i].dst] = i;
    auto time_of = [](const cadnn_weights *w) { return (w->has_ps && w->use_ps) ? w->ps_us : w->pl_us; };
    auto eligible = [&](int i, bool k3) {
        const cadnn_op &op = net->ops[i];
        if (op.kind != CADNN_OP_CONV || !op.w || !op.w->half || op.w->desc.stride != 2 || (op.w->desc.kh == 3) != k3) return false;
        if (op.src == 0 || op.src == net->out_slot || writer[op.src] < 0) return false;
        const cadnn_op &pr = net->ops[writer[op.src]];
        if (pr.kind != CADNN_OP_CONV || !pr.w || !pr.w->has_planar || pr.w->s.kind == KK_DENSE_SMALLC || pr.w->s.kind == KK_DW) return false;
        const float t_half = time_of(op.w->half), t_full = time_of(op.w);
        return force || (t_half > 0.0f && t_full > 0.0f && t_half < t_full);
    };
    for (int i = 0; i < n_ops; ++i)
        if (eligible(i, true)) {
            net->use_half[i] = 1;
            net->slots[net->ops[i].src].par_mask = 0xf;
        }
    for (int i = 0; i < n_ops; ++i)
        if (eligible(i, false) && net->slots[net->ops[i].src].par_mask != 0xf) {
            net->use_half[i] = 1;
            net->slots[net->ops[i].src].par_mask = 0x1;
        }
    for (SlotInfo &sl : net->slots) {
        if (!sl.par_mask) continue;
        const size_t bytes = (size_t)parity_planes_bytes(sl.par_mask, sl.n, sl.h, sl.w, sl.c);
        const size_t alloc = (bytes + 255) / 256 * 256;
        cudaError_t e = cudaMalloc(&sl.par_ptr, alloc);
        if (e == cudaSuccess) e = cudaMemset(sl.par_ptr, 0, alloc);   // borders and absent pixels read as zero
        if (e != cudaSuccess) {
            cadnn_note_cuda(e);
            return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
        }
        net->workspace += (int64_t)alloc;
    }
    return CADNN_OK;
}

}  // namespace

extern "C" {

cadnn_status cadnn_net_create(const cadnn_op *ops, int n_ops, int n, int h, int wd, int c, int in_dtype,
                              cadnn_net **out)
{
    if (!ops || !out || n_ops < 1 || n < 1 || h < 1 || wd < 1 || c < 1) return CADNN_E_ARG;
    if (in_dtype != CADNN_F32 && in_dtype != CADNN_S8) return CADNN_E_DTYPE;
    cadnn_net *net = new (std::nothrow) cadnn_net();
    if (!net) return CADNN_E_ALLOC;
    net->use_pdl = getenv("CADNN_NO_PDL") == nullptr;
    net->pdl_graph = net->use_pdl && getenv("CADNN_NO_PDL_GRAPH") == nullptr;
    net->fork_branches = getenv("CADNN_NO_FORK") == nullptr;
    net->early_trigger = getenv("CADNN_PDL_EARLY") != nullptr;   // tuning switch: plain stream order between layers
    cadnn_status st = CADNN_OK;
    int max_slot = 0;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i].src < 0 || ops[i].dst < 1 || ops[i].res < -1) { st = CADNN_E_ARG; break; }
        max_slot = std::max(max_slot, std::max(ops[i].src, std::max(ops[i].dst, ops[i].res)));
    }
    if (st == CADNN_OK) {
        net->ops.assign(ops, ops + n_ops);
        net->slots.assign(max_slot + 1, SlotInfo());
        SlotInfo &in = net->slots[0];
        in.n = n; in.h = h; in.w = wd; in.c = c; in.dtype = in_dtype; in.defined = true;
        net->out_slot = ops[n_ops - 1].dst;
        net->in_bytes = (int64_t)n * h * wd * c * dtype_size(in_dtype);
        // Channel-planar intermediates are used when every op has a planar kernel: a dense stem on
        // the NHWC input, then sparse float convs, max pools, a global average pool, and fc layers
        // fed by it, and dense depthwise layers of up to 9 taps.  (int8 layers keep NHWC.)
        bool planar = in_dtype == CADNN_F32 && getenv("CADNN_NO_PLANAR") == nullptr && n_ops >= 2 &&
                      ops[n_ops - 1].kind == CADNN_OP_FC;
        std::vector<char> flat(max_slot + 1, 0);   // slot holds a dense [n][c] vector
        for (int i = 0; i < n_ops && planar; ++i) {
            const cadnn_op &op = ops[i];
            if (op.dst_c_total > 0 || op.kind == CADNN_OP_AVGPOOL) { planar = false; break; }   // concatenations stay NHWC
            if (op.kind == CADNN_OP_CONV) {
                if (!op.w) { planar = false; break; }
                const bool stem = op.w->s.kind == KK_DENSE_SMALLC && op.src == 0 && op.res < 0;
                const bool dw = dw_planar_ok(op.w) && op.res < 0 && op.src != 0 && !flat[op.src] && getenv("CADNN_NO_PLANAR_DW") == nullptr;
                if (!stem && !dw && (!op.w->has_planar || op.src == 0 || flat[op.src])) planar = false;
                // a residual must be a padded planar tensor too: not the NHWC input, not an [n][c] vector
                if (op.res == 0 || (op.res > 0 && flat[op.res])) planar = false;
            } else if (op.kind == CADNN_OP_FC) {
                if (!flat[op.src]) planar = false;
                flat[op.dst] = 1;
            } else if (op.kind == CADNN_OP_GAVGPOOL) {
                if (op.src == 0 || flat[op.src]) planar = false;
                flat[op.dst] = 1;
            } else if (op.kind == CADNN_OP_MAXPOOL) {
                if (op.src == 0 || flat[op.src]) planar = false;
            }
        }
        // Where the packer timed both layouts for every sparse conv, the measured sums decide.
        if (planar && getenv("CADNN_FORCE_PLANAR") == nullptr) {
            double t_planar = 0.0, t_nhwc = 0.0;
            bool all = true;
            for (int i = 0; i < n_ops; ++i) {
                const cadnn_weights *w = ops[i].kind == CADNN_OP_CONV ? ops[i].w : nullptr;
                if (!w || !w->has_planar) continue;
                float tp = (w->has_ps && w->use_ps) ? w->ps_us : w->pl_us;
                if (w->half) {   // a stride-2 layer would run in its parity-plane form where that measured faster
                    const float th = (w->half->has_ps && w->half->use_ps) ? w->half->ps_us : w->half->pl_us;
                    if (th > 0.0f && (tp <= 0.0f || th < tp)) tp = th;
                }
                if (tp <= 0.0f || w->nhwc_us <= 0.0f) { all = false; break; }
                t_planar += tp;
                t_nhwc += w->nhwc_us;
            }
            if (getenv("CADNN_VERBOSE"))
                fprintf(stderr, "cadnn_net_create: sparse convs timed at pack time: planar %.1f us, NHWC %.1f us%s\n", t_planar, t_nhwc,
                        all ? "" : " (incomplete)");
            if (all && t_nhwc > 0.0 && t_planar > t_nhwc) planar = false;
        }
        net->planar = planar;
    }
    for (int i = 0; i < n_ops && st == CADNN_OK; ++i) {
        const cadnn_op &op = ops[i];
        const SlotInfo si = net->slots[op.src];
        SlotInfo &so = net->slots[op.dst];
        const bool window = op.dst_c_total > 0;
        if (op.dst_c_total < 0 || op.dst_c_off < 0 || (!window && op.dst_c_off != 0)) { st = CADNN_E_ARG; break; }
        // a slot has one writer, or several that each fill a channel window of it
        if (!si.defined || (so.defined && !window)) { st = CADNN_E_ARG; break; }
        SlotInfo sn;   // what this op produces
        sn.n = si.n;
        if (op.kind == CADNN_OP_CONV || op.kind == CADNN_OP_FC) {
            if (!op.w || !op.w->on_device) { st = CADNN_E_ARG; break; }
            const cadnn_layer_desc &d = op.w->desc;
            if (d.dtype != si.dtype) { st = CADNN_E_DTYPE; break; }
            if (op.kind == CADNN_OP_FC) {
                if ((long long)si.h * si.w * si.c != d.c_in) { st = CADNN_E_SHAPE; break; }
            } else if (si.h != d.in_h || si.w != d.in_w || si.c != d.c_in) { st = CADNN_E_SHAPE; break; }
            sn.h = op.w->h_out; sn.w = op.w->w_out; sn.c = d.c_out; sn.dtype = op.out_dtype;
            if (op.res >= 0) {
                const SlotInfo &sr = net->slots[op.res];
                // a residual has the output's shape; int8 layers take an int8 residual whatever they store
                const int want_dt = d.dtype == CADNN_S8 ? CADNN_S8 : sn.dtype;
                if (!sr.defined || sr.h != sn.h || sr.w != sn.w || sr.c != sn.c || sr.dtype != want_dt) {
                    st = CADNN_E_SHAPE;
                    break;
                }
            }
            // what the layer call would refuse (epilogue combination, weights of another GPU) is refused now
            st = check_layer_call(op.w, op.res >= 0, op.act, op.out_dtype, op.dst_c_total, op.dst_c_off);
            if (st != CADNN_OK) break;
            if (op.w->has_tc && op.w->nnz != op.w->tc_nnz)
                net->tc_ws_bytes = std::max(net->tc_ws_bytes, (int64_t)si.n * op.w->h_out * op.w->w_out * d.c_out * 4);
        } else if (op.kind == CADNN_OP_MAXPOOL || op.kind == CADNN_OP_AVGPOOL) {
            if (op.pool_k < 1 || op.pool_stride < 1 || op.pool_pad < 0 || op.pool_pad >= op.pool_k ||
                si.h + 2 * op.pool_pad < op.pool_k || si.w + 2 * op.pool_pad < op.pool_k) { st = CADNN_E_SHAPE; break; }
            if (op.kind == CADNN_OP_AVGPOOL && si.dtype != CADNN_F32) { st = CADNN_E_DTYPE; break; }
            sn.h = (si.h + 2 * op.pool_pad - op.pool_k) / op.pool_stride + 1;
            sn.w = (si.w + 2 * op.pool_pad - op.pool_k) / op.pool_stride + 1;
            sn.c = si.c; sn.dtype = si.dtype;
        } else if (op.kind == CADNN_OP_GAVGPOOL) {
            if (si.dtype != CADNN_F32 || window) { st = window ? CADNN_E_UNSUPPORTED : CADNN_E_DTYPE; break; }
            sn.h = 1; sn.w = 1; sn.c = si.c; sn.dtype = CADNN_F32;
        } else { st = CADNN_E_ARG; break; }
        if (window) {
            if (op.dst_c_off + sn.c > op.dst_c_total) { st = CADNN_E_SHAPE; break; }
            sn.c = op.dst_c_total;
            if (so.defined) {   // a later writer of the same concatenation: same shape, nothing more to allocate
                if (so.h != sn.h || so.w != sn.w || so.c != sn.c || so.dtype != sn.dtype || so.n != sn.n) st = CADNN_E_SHAPE;
                if (st != CADNN_OK) break;
                continue;
            }
        }
        so.n = sn.n; so.h = sn.h; so.w = sn.w; so.c = sn.c; so.dtype = sn.dtype;
        so.defined = true;
        so.bytes = (int64_t)so.n * so.h * so.w * so.c * dtype_size(so.dtype);
        const bool padded = net->planar && (op.kind == CADNN_OP_CONV || op.kind == CADNN_OP_MAXPOOL);
        if (padded) so.bytes = (int64_t)so.n * so.c * planar_pitch(so.h, so.w) * 4;
        if (op.dst != net->out_slot) {
            size_t alloc = (size_t)((so.bytes + 255) / 256 * 256);
            cudaError_t e = cudaMalloc(&so.ptr, alloc ? alloc : 256);
            // the halo of a planar tensor must read as zero and is never written afterwards
            if (e == cudaSuccess && padded) e = cudaMemset(so.ptr, 0, alloc);
            if (e != cudaSuccess) {
                cadnn_note_cuda(e);
                st = e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
                break;
            }
            net->workspace += (int64_t)alloc;
        }
    }
    if (st != CADNN_OK) {
        cadnn_net_free(net);
        return st;
    }
    net->out_bytes = net->slots[net->out_slot].bytes;
    st = plan_parity_planes(net);
    if (st != CADNN_OK) {
        cadnn_net_free(net);
        return st;
    }
    if (net->tc_ws_bytes > 0) {
        cudaError_t e = cudaMalloc(&net->tc_ws, (size_t)net->tc_ws_bytes);
        if (e != cudaSuccess) {
            cadnn_note_cuda(e);
            cadnn_net_free(net);
            return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
        }
        net->workspace += net->tc_ws_bytes;
    }
    if (cudaHostAlloc((void **)&net->status_host, 2 * sizeof(int), cudaHostAllocDefault) != cudaSuccess) {
        cudaGetLastError();
        cadnn_net_free(net);
        return CADNN_E_ALLOC;
    }
    if (read_copy_timeouts(&net->status_seen[0]) != CADNN_OK || read_barrier_timeouts(&net->status_seen[1]) != CADNN_OK) {
        cadnn_net_free(net);
        return CADNN_E_CUDA;
    }
    net->status_host[0] = net->status_seen[0];
    net->status_host[1] = net->status_seen[1];
    // inside graphs, programmatic launches pay off for the planar kernels only (the NHWC sparse conv
    // measured slower with them: 556 -> 608 us on ResNet-50, 367 -> 410 us on the int8 VGG-16)
    if (!net->planar && getenv("CADNN_PDL_GRAPH") == nullptr) net->pdl_graph = false;
    {
        // The persistent kernel trades the launch ramp and drain of every layer boundary for a device-wide
        // barrier and a copy start-up per layer.  Measured on a B200 (pruned ResNet-50, batch 1) a phase costs
        // about 2400 clocks of barrier and skew, 3400 clocks until its first tile is complete in shared memory,
        // and multiply-adds bound by shared-memory bandwidth: no less than one tuned kernel per layer under
        // programmatic launches.  So it stays opt-in.
        const char *pe = getenv("CADNN_PERSIST");   // "1": on; unset / "0": off
        if (net->planar && pe && atoi(pe) != 0) plan_persistent(net);
    }
    *out = net;
    return CADNN_OK;
}

cadnn_status cadnn_forward(cadnn_net *net, const void *x, void *y, int use_graph, void *stream)
{
    if (!net || !x || !y) return CADNN_E_ARG;
    return forward_impl(net, x, y, use_graph, (cudaStream_t)stream, 0);
}

cadnn_status cadnn_forward_host(cadnn_net *net, const void *x_host, void *y_host, int use_graph, void *stream)
{
    if (!net || !x_host || !y_host) return CADNN_E_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (!net->stage_x) {
        cudaError_t e = cudaMalloc(&net->stage_x, (size_t)((net->in_bytes + 255) / 256 * 256));
        if (e == cudaSuccess) e = cudaMalloc(&net->stage_y, (size_t)((net->out_bytes + 255) / 256 * 256));
        if (e != cudaSuccess) {
            cadnn_note_cuda(e);
            return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
        }
    }
    CADNN_CUDA_TRY(cudaMemcpyAsync(net->stage_x, x_host, (size_t)net->in_bytes, cudaMemcpyHostToDevice, st));
    cadnn_status s = forward_impl(net, net->stage_x, net->stage_y, use_graph, st, 1);
    if (s != CADNN_OK) return s;
    CADNN_CUDA_TRY(cudaMemcpyAsync(y_host, net->stage_y, (size_t)net->out_bytes, cudaMemcpyDeviceToHost, st));
    s = queue_status_read(net, st);
    if (s != CADNN_OK) return s;
    CADNN_CUDA_TRY(cudaStreamSynchronize(st));
    return status_moved(net) ? CADNN_E_DEVICE_STATUS : CADNN_OK;
}

cadnn_status cadnn_net_info(const cadnn_net *net, int *n_launches, int64_t *workspace_bytes)
{
    if (!net) return CADNN_E_ARG;
    if (n_launches) *n_launches = (int)net->ops.size() - (net->persist ? net->persist_last - net->persist_first : 0);
    if (workspace_bytes) *workspace_bytes = net->workspace;
    return CADNN_OK;
}

cadnn_status cadnn_net_parity_layers(const cadnn_net *net, int *count, int *ops, int cap)
{
    if (!net || !count || cap < 0 || (cap > 0 && !ops)) return CADNN_E_ARG;
    *count = 0;
    for (size_t i = 0; i < net->use_half.size(); ++i)
        if (net->use_half[i]) {
            if (*count < cap) ops[*count] = (int)i;
            ++*count;
        }
    return CADNN_OK;
}

cadnn_status cadnn_net_layout(const cadnn_net *net, int *planar, int *persistent_ops)
{
    if (!net) return CADNN_E_ARG;
    if (planar) *planar = net->planar ? 1 : 0;
    if (persistent_ops) *persistent_ops = net->persist ? net->persist_last - net->persist_first + 1 : 0;
    return CADNN_OK;
}

static cadnn_status layer_times_range(cadnn_net *net, const void *x, void *y, int flush_l2, int reps, float *ms,
                                      size_t op_lo, size_t op_hi, cudaStream_t st)
{
    const size_t nops = op_hi;
    if (flush_l2 && !net->flush) {
        net->flush_bytes = 256u << 20;
        CADNN_CUDA_TRY(cudaMalloc(&net->flush, net->flush_bytes));
    }
    // one pass in order so that every slot holds real data
    cadnn_status s = run_all(net, x, y, st);
    if (s != CADNN_OK) return s;
    CADNN_CUDA_TRY(cudaStreamSynchronize(st));
    cudaStream_t cap;
    CADNN_CUDA_TRY(cudaStreamCreateWithFlags(&cap, cudaStreamNonBlocking));
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    for (size_t i = op_lo; i < nops && s == CADNN_OK; ++i) {
        // a graph of `reps` back-to-back launches of this op: the host launch cost stays out of the timing
        cudaGraph_t g = nullptr;
        cudaGraphExec_t ge = nullptr;
        cudaError_t e = cudaStreamBeginCapture(cap, cudaStreamCaptureModeThreadLocal);
        if (e != cudaSuccess) { s = cadnn_note_cuda(e); break; }
        for (int r = 0; r < reps && s == CADNN_OK; ++r) s = run_op(net, net->ops[i], x, y, cap);
        e = cudaStreamEndCapture(cap, &g);
        if (s == CADNN_OK && e != cudaSuccess) s = cadnn_note_cuda(e);
        if (s == CADNN_OK && (e = cudaGraphInstantiate(&ge, g, 0)) != cudaSuccess) s = cadnn_note_cuda(e);
        if (s == CADNN_OK) {
            if (flush_l2) flush_kernel<<<148 * 8, 256, 0, st>>>((float *)net->flush, net->flush_bytes / 4);
            else cudaGraphLaunch(ge, st);   // warm
            cudaEventRecord(e0, st);
            cudaGraphLaunch(ge, st);
            cudaEventRecord(e1, st);
            e = cudaStreamSynchronize(st);
            if (e != cudaSuccess) s = cadnn_note_cuda(e);
            else {
                cudaEventElapsedTime(&ms[i - op_lo], e0, e1);
                ms[i - op_lo] /= (float)reps;
            }
        }
        if (ge) cudaGraphExecDestroy(ge);
        if (g) cudaGraphDestroy(g);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaStreamDestroy(cap);
    if (s == CADNN_OK) {
        s = queue_status_read(net, st);
        if (s == CADNN_OK && cudaStreamSynchronize(st) != cudaSuccess) s = cadnn_note_cuda(cudaGetLastError());
        if (s == CADNN_OK && status_moved(net)) s = CADNN_E_DEVICE_STATUS;
    }
    return s;
}

cadnn_status cadnn_net_layer_times(cadnn_net *net, const void *x, void *y, int flush_l2, int reps, float *ms,
                                   void *stream)
{
    if (!net || !x || !y || !ms || reps < 1) return CADNN_E_ARG;
    return layer_times_range(net, x, y, flush_l2, reps, ms, 0, net->ops.size(), (cudaStream_t)stream);
}

cadnn_status cadnn_net_layer_time(cadnn_net *net, int op, const void *x, void *y, int flush_l2, int reps, float *ms,
                                  void *stream)
{
    if (!net || !x || !y || !ms || reps < 1 || op < 0 || op >= (int)net->ops.size()) return CADNN_E_ARG;
    return layer_times_range(net, x, y, flush_l2, reps, ms, (size_t)op, (size_t)op + 1, (cudaStream_t)stream);
}

cadnn_status cadnn_net_persistent_plan(const cadnn_net *net, int op, int plan[12])
{
    if (!net || !plan) return CADNN_E_ARG;
    if (!net->persist || op < net->persist_first || op > net->persist_last) return CADNN_E_UNSUPPORTED;
    return persist_describe(net->persist, op - net->persist_first, plan) ? CADNN_OK : CADNN_E_ARG;
}

cadnn_status cadnn_net_persistent_profile(const cadnn_net *net, int cap, float *wall_clk, float *busy_max_clk,
                                          float *busy_mean_clk, float *issued_clk, float *landed_clk, int *n_phases)
{
    if (!net || !n_phases) return CADNN_E_ARG;
    if (!net->persist) return CADNN_E_UNSUPPORTED;
    CADNN_CUDA_TRY(cudaDeviceSynchronize());
    return persist_profile(net->persist, cap, wall_clk, busy_max_clk, busy_mean_clk, issued_clk, landed_clk, n_phases);
}

cadnn_status cadnn_net_slot(const cadnn_net *net, int slot, void **ptr, int64_t *bytes)
{
    if (!net || slot < 0 || slot >= (int)net->slots.size() || !net->slots[slot].defined) return CADNN_E_ARG;
    if (ptr) *ptr = net->slots[slot].ptr;
    if (bytes) *bytes = net->slots[slot].bytes;
    return CADNN_OK;
}

void cadnn_net_free(cadnn_net *net)
{
    if (!net) return;
    drop_graph(net->cache[0]);
    drop_graph(net->cache[1]);
    if (net->stage_x) cudaFree(net->stage_x);
    if (net->stage_y) cudaFree(net->stage_y);
    for (SlotInfo &s : net->slots) {
        if (s.ptr) cudaFree(s.ptr);
        if (s.par_ptr) cudaFree(s.par_ptr);
    }
    if (net->flush) cudaFree(net->flush);
    if (net->tc_ws) cudaFree(net->tc_ws);
    if (net->status_host) cudaFreeHost(net->status_host);
    persist_free(net->persist);
    delete net;
}

}  // extern "C"
