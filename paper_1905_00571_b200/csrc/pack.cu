// Offline weight packer and per-layer schedule (host code).
//
// Restates, for one large GPU, the offline stage of CADNN (arXiv 1905.00571,
// Section 4): "Memory layout transformation" - the pruned filters are stored in a
// compressed layout whose element offsets already point into the shared-memory
// activation tile the kernel stages, padded so that a warp's loads never collide
// on a bank - and "Optimization parameters selection" - tile sizes, the channel
// chunk, the filters per warp and the split of the reduction over a thread-block
// cluster are chosen per layer from its shape, by a time model or by timing the
// candidates on the device.  Filters are regrouped so that the warps of a block
// get equal nonzero counts (the load-balance obstacle Section 1 names).
#include <algorithm>
#include <memory>
#include <string>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <numeric>
#include "cadnn_internal.h"

namespace {

const int kSmCount = 148;
const int kSmemPerSm = 200 * 1024;        // shared memory the schedule lets resident blocks use per SM
const int kMaxStageBytes = 100 * 1024;

int round_up(int v, int m) { return (v + m - 1) / m * m; }
int ceil_div(int a, int b) { return (a + b - 1) / b; }

struct Geometry {
    int c_in, c_out, kh, kw, stride, pad, h, w, h_out, w_out;
    bool s8;
    double nnz;   // stored nonzeros of the layer
};

// Bytes per staged pixel: an odd number of 32-bit words, so that lanes reading the
// same channel of consecutive pixels touch distinct banks.
int pixel_pitch_bytes(int cic, bool s8)
{
    int words = s8 ? ceil_div(cic, 4) : cic;
    return 4 * (words | 1);
}

// Smallest staged row pitch (pixels) >= need for which one band - RB rows of BW
// consecutive pixels, rows row_step * pitch apart - touches RB * BW distinct banks.
int pick_pitch(int need, int BW, int RB, int row_step)
{
    for (int p = need; p < need + 64; ++p) {
        bool used[32] = {false};
        bool ok = true;
        for (int r = 0; r < RB && ok; ++r)
            for (int x = 0; x < BW; ++x) {
                int b = (r * row_step * p + x) & 31;
                if (used[b]) { ok = false; break; }
                used[b] = true;
            }
        if (ok) return p;
    }
    return need;
}

// Derived fields of a candidate (everything but the entry counts).
bool finish_candidate(const Geometry &g, Schedule &s, bool linear)
{
    s.G = s.NW * s.RPW;
    s.T = s.TBX * s.TBY;
    if (s.T < 1 || s.T > 8) return false;
    s.n_groups = ceil_div(g.c_out, s.G);
    s.PPb = pixel_pitch_bytes(s.CIc, g.s8);
    s.n_chunks = ceil_div(g.c_in, s.CIc);
    if (s.ksplit < 1 || s.ksplit > 8 || s.ksplit > s.n_chunks) return false;
    if (linear) {
        s.BW = 32; s.RB = 1; s.TBX = s.T; s.TBY = 1;
        s.TH = 1; s.TW = 32 * s.T;
        s.pitch = s.half = s.IH_t = s.IW_t = 0;
        s.tile_bytes = 32 * s.T * s.PPb;
    } else {
        s.TH = s.TBY * s.RB;
        s.TW = s.TBX * s.BW;
        s.IH_t = (s.TH - 1) * g.stride + g.kh;
        s.IW_t = (s.TW - 1) * g.stride + g.kw;
        if (g.stride == 2) {
            s.half = ceil_div(s.IW_t, 2);
            s.pitch = pick_pitch(2 * s.half, s.BW, s.RB, 2);
        } else {
            s.half = 0;
            s.pitch = pick_pitch(s.IW_t, s.BW, s.RB, g.stride);
        }
        s.tile_bytes = s.IH_t * s.pitch * s.PPb;
    }
    s.tile_bytes = round_up(s.tile_bytes, 16);
    return true;
}

int header_words(const Schedule &s) { return round_up(s.G + 1, 4); }

void finish_smem(Schedule &s, bool s8)
{
    int ew = s8 ? 4 : 8;
    s.stage_bytes = s.tile_bytes + header_words(s) * 4 + round_up(s.max_entries * ew, 16);
    int out = 32 * s.T * (s.G + 1) * 4;
    int per_block = ceil_div(s.n_chunks, s.ksplit);   // chunks one block walks
    s.stages = (3 * s.stage_bytes <= 72 * 1024 && per_block >= 3) ? 3 : 2;
    if (per_block == 1) s.stages = 1;
    int npx = s.kind == KK_SCONV_LINEAR ? 32 * s.T : s.IH_t * s.IW_t;
    int tables = npx * 8 + 2 * s.G * 4;
    s.smem_bytes = round_up(std::max(s.stages * s.stage_bytes, out), 16) + round_up(tables, 16);
}

// Rough time model (SM clocks) of one candidate: the kernel is bound by shared-memory
// wavefronts (one per 32 multiply-adds plus the broadcast of each nonzero), by issue
// slots, by the bytes each block pulls through L2, and by per-block fixed latencies.
double estimate_clocks(const Geometry &g, const Schedule &s, int batch, bool linear)
{
    double tiles;
    double in_px;
    if (linear) {
        double P = (double)batch * g.h_out * g.w_out;
        tiles = std::ceil(P / (32.0 * s.T));
        in_px = 32.0 * s.T;
    } else {
        tiles = (double)batch * ceil_div(g.h_out, s.TH) * ceil_div(g.w_out, s.TW);
        in_px = (double)s.IH_t * s.IW_t;
    }
    const double KS = s.ksplit;
    double ctas = tiles * s.n_groups * KS;
    double nnz_cta = g.nnz * s.G / std::max(1, g.c_out) / KS;
    double cin_cta = std::min((double)g.c_in, (double)ceil_div(s.n_chunks, s.ksplit) * s.CIc);
    double esz = g.s8 ? 1.0 : 4.0;
    double units = in_px * cin_cta / (g.s8 ? 4.0 : 1.0);          // 4-byte staging copies
    double wf = nnz_cta * (s.T + 0.5) + units / 32.0 * 4.0 + 32.0 * s.T * s.G / 32.0 * (2.0 + KS);
    double instr = (nnz_cta * (2.2 * s.T + 3.0) + units / 32.0 * 12.0 + 32.0 * s.T * s.G / 32.0 * 30.0) / 4.0;
    double l2 = (in_px * cin_cta * esz + nnz_cta * (g.s8 ? 4.0 : 8.0) + 32.0 * s.T * s.G * 4.0) / 40.0;
    int by_smem = std::max(1, kSmemPerSm / std::max(1, s.smem_bytes));
    int by_thr = std::max(1, 2048 / (s.NW * 32));
    int resident = std::min(std::min(by_smem, by_thr), 8);
    double per_sm = std::ceil(ctas / kSmCount);
    double in_round = std::min((double)resident, per_sm);
    double warps = in_round * s.NW;
    double ipc_eff = std::min(1.0, warps / 24.0);                  // few warps cannot fill the issue slots
    double busy = std::max(std::max(wf, instr / std::max(0.15, ipc_eff)), l2);
    double fixed = 3000.0 + 500.0 * ceil_div(s.n_chunks, s.ksplit) + (KS > 1 ? 1500.0 : 0.0);
    double rounds = std::ceil(per_sm / resident);
    return rounds * std::max(in_round * busy, busy + fixed);
}

// Longest-processing-time assignment of the G filters of one block to the warps,
// RPW filters each; returns, per warp slot, the local filter index (or -1).
void balance_block(const std::vector<int64_t> &load, int G, int RPW, std::vector<int> &slot_to_local)
{
    int nw = G / RPW;
    std::vector<int> order(load.size());
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return load[a] > load[b]; });
    std::vector<int64_t> wl(nw, 0);
    std::vector<int> cnt(nw, 0);
    slot_to_local.assign(G, -1);
    for (int idx : order) {
        int best = -1;
        for (int w = 0; w < nw; ++w) {
            if (cnt[w] >= RPW) continue;
            if (best < 0 || wl[w] < wl[best]) best = w;
        }
        slot_to_local[best * RPW + cnt[best]] = idx;
        wl[best] += load[idx];
        cnt[best]++;
    }
}

cadnn_status upload(cadnn_weights *h)
{
    auto al = [](size_t b) { return (b + 255) / 256 * 256; };
    size_t b_vals = h->desc.dtype == CADNN_S8 ? h->vals_q.size() : h->vals_f.size() * 4;
    size_t b_offs = h->offs.size() * 2, b_ptr = h->ptr.size() * 4, b_perm = h->perm.size() * 4;
    size_t b_dense = h->dense_f.size() * 4, b_ent = h->ent.size() * 4;
    size_t b_ple = h->pl_ent.size() * 4, b_plp = h->pl_ptr.size() * 4, b_plo = h->pl_order.size() * 4;
    size_t o_vals = 0, o_offs = o_vals + al(b_vals), o_ptr = o_offs + al(b_offs), o_perm = o_ptr + al(b_ptr);
    size_t o_dense = o_perm + al(b_perm), o_ent = o_dense + al(b_dense);
    size_t b_pse = h->ps_ent.size() * 4, b_psp = h->ps_perm.size() * 4;
    size_t o_ple = o_ent + al(b_ent), o_plp = o_ple + al(b_ple), o_plo = o_plp + al(b_plp), o_pse = o_plo + al(b_plo);
    size_t o_psp = o_pse + al(b_pse), total = o_psp + al(b_psp);
    h->packed_bytes = (int64_t)(b_vals + b_offs + b_ptr + b_perm + b_dense + b_ent);
    if (h->desc.flags & CADNN_PACK_HOST_ONLY) return CADNN_OK;
    if (total == 0) total = 256;
    CADNN_CUDA_TRY(cudaGetDevice(&h->device));
    cudaError_t e = cudaMalloc(&h->d_blob, total);
    if (e != cudaSuccess) {
        cadnn_note_cuda(e);
        return e == cudaErrorMemoryAllocation ? CADNN_E_ALLOC : CADNN_E_CUDA;
    }
    char *base = (char *)h->d_blob;
    const void *src_vals = h->desc.dtype == CADNN_S8 ? (const void *)h->vals_q.data() : (const void *)h->vals_f.data();
    if (b_vals) CADNN_CUDA_TRY(cudaMemcpy(base + o_vals, src_vals, b_vals, cudaMemcpyHostToDevice));
    if (b_offs) CADNN_CUDA_TRY(cudaMemcpy(base + o_offs, h->offs.data(), b_offs, cudaMemcpyHostToDevice));
    if (b_ptr) CADNN_CUDA_TRY(cudaMemcpy(base + o_ptr, h->ptr.data(), b_ptr, cudaMemcpyHostToDevice));
    if (b_perm) CADNN_CUDA_TRY(cudaMemcpy(base + o_perm, h->perm.data(), b_perm, cudaMemcpyHostToDevice));
    if (b_dense) CADNN_CUDA_TRY(cudaMemcpy(base + o_dense, h->dense_f.data(), b_dense, cudaMemcpyHostToDevice));
    if (b_ent) CADNN_CUDA_TRY(cudaMemcpy(base + o_ent, h->ent.data(), b_ent, cudaMemcpyHostToDevice));
    h->d_ent = (const uint32_t *)(base + o_ent);
    if (b_ple) CADNN_CUDA_TRY(cudaMemcpy(base + o_ple, h->pl_ent.data(), b_ple, cudaMemcpyHostToDevice));
    if (b_plp) CADNN_CUDA_TRY(cudaMemcpy(base + o_plp, h->pl_ptr.data(), b_plp, cudaMemcpyHostToDevice));
    if (b_plo) CADNN_CUDA_TRY(cudaMemcpy(base + o_plo, h->pl_order.data(), b_plo, cudaMemcpyHostToDevice));
    if (b_pse) CADNN_CUDA_TRY(cudaMemcpy(base + o_pse, h->ps_ent.data(), b_pse, cudaMemcpyHostToDevice));
    if (b_psp) CADNN_CUDA_TRY(cudaMemcpy(base + o_psp, h->ps_perm.data(), b_psp, cudaMemcpyHostToDevice));
    h->d_ps_ent = (const uint32_t *)(base + o_pse);
    h->d_ps_perm = (const int32_t *)(base + o_psp);
    h->d_pl_ent = (const uint32_t *)(base + o_ple);
    h->d_pl_ptr = (const int32_t *)(base + o_plp);
    h->d_pl_order = (const int32_t *)(base + o_plo);
    // A copy from pageable host memory may return before its DMA has landed; kernels on
    // non-blocking streams are not ordered behind it, so wait for it here.
    CADNN_CUDA_TRY(cudaStreamSynchronize(cudaStreamLegacy));
    h->d_vals = base + o_vals;
    h->d_offs = (const uint16_t *)(base + o_offs);
    h->d_ptr = (const int32_t *)(base + o_ptr);
    h->d_perm = (const int32_t *)(base + o_perm);
    h->d_dense = (const float *)(base + o_dense);
    h->on_device = true;
    return CADNN_OK;
}

// value accessors over either float or int8 source weights
struct Src {
    const float *f = nullptr;
    const int8_t *q = nullptr;
    const uint8_t *mask = nullptr;
    const float *w_scale = nullptr;
    bool s8 = false;
    bool kept(size_t i) const { return mask == nullptr || mask[i] != 0; }
    float fval(size_t i) const { return f ? f[i] : (float)q[i]; }
    int8_t qval(size_t i, int co) const
    {
        if (q) return q[i];
        float r = f[i] / w_scale[co];
        long v = lrintf(r);
        v = std::max(-127L, std::min(127L, v));
        return (int8_t)v;
    }
};

struct Candidate {
    Schedule s;
    double t;
};

// Candidate schedules for a layer, best first by the time model.
void enumerate_schedules(const Geometry &g, int batch, bool linear, std::vector<Candidate> &out)
{
    out.clear();
    // band shape follows the output width
    int BW, RB, nbx_total;
    if (linear) {
        BW = 32; RB = 1; nbx_total = 1;
    } else if (g.w_out <= 32) {
        BW = g.w_out;
        RB = std::max(1, std::min(32 / BW, g.h_out));
        nbx_total = 1;
    } else {
        nbx_total = ceil_div(g.w_out, 32);
        BW = ceil_div(g.w_out, nbx_total);
        RB = 1;
    }
    // channel-chunk candidates: powers of two up to 512, never far beyond the layer's channels
    std::vector<int> cics;
    if (g.s8) {
        for (int c = 512; c >= 4; c /= 2)
            if (c == 4 || c / 2 < g.c_in) cics.push_back(c);
    } else if (g.c_in < 4) {
        cics.push_back(g.c_in);
    } else {
        for (int c = 512; c >= 4; c /= 2)
            if (c == 4 || c / 2 < g.c_in) cics.push_back(std::min(c, g.c_in));
    }
    const int tbx_full = std::min(8, nbx_total);
    for (int nw : {16, 8, 4})
        for (int rpw : {16, 8, 4, 2, 1})
            for (int cic : cics)
                for (int ks : {1, 2, 4, 8})
                    for (int tbx = 1; tbx <= (linear ? 8 : tbx_full); ++tbx)
                        for (int tby = 1; tby * tbx <= 8; ++tby) {
                            if (linear && tby > 1) break;
                            if (!linear && tbx != tbx_full && tbx != 1 && tbx * 2 != tbx_full) continue;
                            if (!linear && (tby - 1) * RB >= g.h_out) break;
                            if (rpw * tbx * tby > 32) continue;            // accumulator registers per lane
                            if (nw * rpw > std::max(8, round_up(g.c_out, 8))) continue;   // more filter slots than filters
                            Schedule s;
                            s.kind = linear ? KK_SCONV_LINEAR : KK_SCONV_SPATIAL;
                            s.NW = nw; s.RPW = rpw; s.CIc = cic; s.ksplit = ks;
                            s.BW = BW; s.RB = RB; s.TBX = tbx; s.TBY = tby;
                            if (!finish_candidate(g, s, linear)) continue;
                            // expected entries per (chunk, block) record, with headroom; the real count is set when packing
                            double per_chunk = g.nnz / std::max(1, g.c_out) * s.G / s.n_chunks;
                            s.max_entries = (int)(per_chunk * 1.3) + 2 * s.G + 16;
                            finish_smem(s, g.s8);
                            if (s.stage_bytes > kMaxStageBytes || s.smem_bytes > kSmemPerSm) continue;
                            out.push_back({s, estimate_clocks(g, s, batch, linear)});
                        }
    std::stable_sort(out.begin(), out.end(), [](const Candidate &a, const Candidate &b) { return a.t < b.t; });
    if (out.empty()) {   // nothing fit: smallest everything
        Schedule s;
        s.kind = linear ? KK_SCONV_LINEAR : KK_SCONV_SPATIAL;
        s.NW = 4; s.RPW = 1; s.CIc = g.s8 ? 4 : 1; s.BW = BW; s.RB = RB; s.TBX = 1; s.TBY = 1;
        finish_candidate(g, s, linear);
        out.push_back({s, 0.0});
    }
}

// Manual override for tuning: CADNN_SCHEDULE="nw=4,rpw=1,tbx=1,tby=2,cic=32,ks=2" (unset keys keep the model's pick).
void apply_env_override(const Geometry &g, bool linear, Schedule &best)
{
    const char *env = getenv("CADNN_SCHEDULE");
    if (!env) return;
    Schedule s = best;
    int v;
    const char *q;
    if ((q = strstr(env, "nw=")) && sscanf(q + 3, "%d", &v) == 1 && (v == 4 || v == 8 || v == 16)) s.NW = v;
    if ((q = strstr(env, "rpw=")) && sscanf(q + 4, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8 || v == 16)) s.RPW = v;
    if ((q = strstr(env, "tbx=")) && sscanf(q + 4, "%d", &v) == 1 && v >= 1 && v <= 8) s.TBX = v;
    if ((q = strstr(env, "tby=")) && sscanf(q + 4, "%d", &v) == 1 && v >= 1 && v <= 8) s.TBY = v;
    if ((q = strstr(env, "cic=")) && sscanf(q + 4, "%d", &v) == 1 && v >= 1 && v <= 512 && (!g.s8 || v % 4 == 0))
        s.CIc = std::min(v, g.s8 ? round_up(g.c_in, 4) : g.c_in);
    if ((q = strstr(env, "ks=")) && sscanf(q + 3, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) s.ksplit = v;
    if (linear) { s.TBX = std::min(8, s.TBX * s.TBY); s.TBY = 1; }
    s.ksplit = std::min(s.ksplit, ceil_div(g.c_in, s.CIc));
    if (finish_candidate(g, s, linear)) best = s;
}

// Build the packed image of a conv layer for schedule h->s (already through finish_candidate).
cadnn_status build_sconv_image(cadnn_weights *h, const Src &src, const Geometry &g,
                               const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    Schedule &s = h->s;
    const bool linear = s.kind == KK_SCONV_LINEAR;
    const bool s8 = src.s8;
    const int ew = s8 ? 1 : 2;   // 32-bit words per entry
    for (int attempt = 0;; ++attempt) {
        s.n_groups = ceil_div(d.c_out, s.G);
        h->c_pad = s.n_groups * s.G;
        s.n_chunks = ceil_div(d.c_in, s.CIc);
        // balanced regrouping of the filters of each block over its warps
        h->perm.assign(h->c_pad, -1);
        for (int gi = 0; gi < s.n_groups; ++gi) {
            int lo = gi * s.G, hi = std::min(d.c_out, lo + s.G);
            std::vector<int64_t> load(row_nnz.begin() + lo, row_nnz.begin() + hi);
            std::vector<int> slot;
            balance_block(load, s.G, s.RPW, slot);
            for (int sl = 0; sl < s.G; ++sl)
                if (slot[sl] >= 0) h->perm[lo + sl] = lo + slot[sl];
        }
        // One record per (chunk, block of G filters): a header of G + 1 row starts (in entries)
        // followed by the entries, every row padded to an even count.  All records get the
        // same size, so a thread block finds its nonzeros without reading a pointer first.
        const int hdr_words = header_words(s);
        std::vector<std::vector<uint32_t>> blocks((size_t)s.n_chunks * s.n_groups);
        h->cnt.assign((size_t)s.n_chunks * h->c_pad, 0);
        s.max_entries = 0;
        for (int c = 0; c < s.n_chunks; ++c) {
            int c0 = c * s.CIc, c1 = std::min(d.c_in, c0 + s.CIc);
            for (int gi = 0; gi < s.n_groups; ++gi) {
                std::vector<uint32_t> &blk = blocks[(size_t)c * s.n_groups + gi];
                blk.assign(hdr_words, 0u);
                int running = 0;
                for (int sl = 0; sl < s.G; ++sl) {
                    const int r = gi * s.G + sl;
                    blk[sl] = (uint32_t)running;
                    int co = h->perm[r];
                    int real = 0;
                    if (co >= 0) {
                        for (int ky = 0; ky < d.kh; ++ky)
                            for (int kx = 0; kx < d.kw; ++kx)
                                for (int ci = c0; ci < c1; ++ci) {
                                    size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + ci;
                                    if (!src.kept(wi)) continue;
                                    int pos = kx;
                                    if (!linear && s.half) pos = (kx & 1) * s.half + (kx >> 1);
                                    uint32_t off = linear ? 0u : (uint32_t)(ky * s.pitch + pos) * (uint32_t)s.PPb;
                                    off += (uint32_t)(ci - c0) * (s8 ? 1u : 4u);
                                    if (s8) {
                                        blk.push_back((off << 8) | (uint32_t)(uint8_t)src.qval(wi, co));
                                    } else {
                                        float v = src.fval(wi);
                                        uint32_t bits;
                                        memcpy(&bits, &v, 4);
                                        blk.push_back(bits);
                                        blk.push_back(off);
                                    }
                                    ++real;
                                }
                        if (real & 1) {   // padding entry: weight 0 at offset 0
                            blk.push_back(0u);
                            if (!s8) blk.push_back(0u);
                        }
                    }
                    h->cnt[(size_t)c * h->c_pad + r] = real;
                    running += real + (real & 1);
                }
                blk[s.G] = (uint32_t)running;
                s.max_entries = std::max(s.max_entries, running);
            }
        }
        s.max_entries = round_up(std::max(s.max_entries, 2) + 2, 4);   // + one pair of slack for the kernel's look-ahead
        finish_smem(s, s8);
        // A dense or skewed layer can overflow the stage budget: halve the chunk and repack.
        if ((s.stage_bytes > kMaxStageBytes || s.smem_bytes > kSmemPerSm) && s.CIc > (s8 ? 4 : 1) && attempt < 8) {
            s.CIc = std::max(s8 ? 4 : 1, s.CIc / 2);
            finish_candidate(g, s, linear);
            continue;
        }
        const int block_words = hdr_words + s.max_entries * ew;
        h->ent.assign((size_t)block_words * blocks.size(), 0u);
        for (size_t b = 0; b < blocks.size(); ++b)
            std::copy(blocks[b].begin(), blocks[b].end(), h->ent.begin() + b * block_words);
        break;
    }
    if (s.smem_bytes > 220 * 1024) return CADNN_E_UNSUPPORTED;
    if (s8 && (uint64_t)s.tile_bytes >= (1u << 24)) return CADNN_E_UNSUPPORTED;
    h->fmt = CADNN_FMT_TILED_CSR;
    return CADNN_OK;
}

// Time one packed conv layer on the current device: a CUDA graph of `reps` back-to-back
// launches on zero-filled activations, replayed once untimed and once between events.
// Returns microseconds per launch, or a negative value if the schedule cannot run.
float time_schedule(cadnn_weights *h, int batch, const void *x, void *y, cudaStream_t st, int reps)
{
    LaunchEpilogue ep;
    ep.out_dtype = h->desc.dtype;
    ep.act = CADNN_ACT_RELU;
    if (launch_sconv(h, x, batch, y, ep, st) != CADNN_OK) return -1.0f;   // also raises the kernel's smem limit
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return -1.0f; }
    cudaGraph_t g = nullptr;
    cudaGraphExec_t ge = nullptr;
    float us = -1.0f;
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return -1.0f; }
    bool ok = true;
    for (int r = 0; r < reps && ok; ++r) ok = launch_sconv(h, x, batch, y, ep, st) == CADNN_OK;
    if (cudaStreamEndCapture(st, &g) != cudaSuccess) ok = false;
    if (ok && cudaGraphInstantiate(&ge, g, 0) == cudaSuccess) {
        cudaEvent_t e0, e1;
        cudaEventCreate(&e0);
        cudaEventCreate(&e1);
        cudaGraphLaunch(ge, st);
        float best = 1e30f;
        for (int rep = 0; rep < 2; ++rep) {
            cudaEventRecord(e0, st);
            cudaGraphLaunch(ge, st);
            cudaEventRecord(e1, st);
            if (cudaStreamSynchronize(st) == cudaSuccess) {
                float ms = 0.0f;
                cudaEventElapsedTime(&ms, e0, e1);
                best = std::min(best, ms);
            }
        }
        if (best < 1e29f) us = best * 1e3f / (float)reps;
        cudaEventDestroy(e0);
        cudaEventDestroy(e1);
    }
    if (ge) cudaGraphExecDestroy(ge);
    if (g) cudaGraphDestroy(g);
    cudaGetLastError();
    return us;
}

// Measured parameter selection (Section 4, "Optimization parameters selection": the search
// space is pruned with knowledge of the layer and the machine - here the time model keeps
// the best candidate of every structural class - and the survivors are timed).
cadnn_status autotune_sconv(cadnn_weights *h, const Src &src, const Geometry &g, const std::vector<int64_t> &row_nnz,
                            const std::vector<Candidate> &cands)
{
    const cadnn_layer_desc &d = h->desc;
    const int batch = std::max(1, d.batch_hint);
    // best candidate by the model of every (warps, filters per warp, cluster split, bands) class
    std::vector<Candidate> pick;
    std::vector<long> seen;
    for (const Candidate &c : cands) {
        long key = ((c.s.NW * 8L + c.s.RPW) * 16 + c.s.ksplit) * 16 + c.s.T;
        if (std::find(seen.begin(), seen.end(), key) != seen.end()) continue;
        seen.push_back(key);
        pick.push_back(c);
    }
    // large batches: a launch takes milliseconds, so only the model's best dozen classes are timed, with fewer launches
    const size_t kMaxTimed = batch >= 32 ? 12 : 80;
    const int reps = batch >= 32 ? 3 : 8;
    if (pick.size() > kMaxTimed) pick.resize(kMaxTimed);
    const size_t esz = src.s8 ? 1 : 4;
    const size_t xb = (size_t)batch * d.in_h * d.in_w * d.c_in * esz;
    const size_t yb = (size_t)batch * h->h_out * h->w_out * d.c_out * 4;
    void *x = nullptr, *y = nullptr;
    cudaStream_t st = nullptr;
    if (cudaMalloc(&x, std::max<size_t>(xb, 256)) != cudaSuccess || cudaMalloc(&y, std::max<size_t>(yb, 256)) != cudaSuccess ||
        cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) {
        if (x) cudaFree(x);
        if (y) cudaFree(y);
        cudaGetLastError();
        return CADNN_E_ALLOC;
    }
    cudaMemsetAsync(x, 0, std::max<size_t>(xb, 256), st);
    float best_us = -1.0f;
    Schedule best = h->s;
    for (const Candidate &c : pick) {
        cadnn_weights tmp;
        tmp.desc = d;
        tmp.desc.flags &= ~CADNN_PACK_HOST_ONLY;
        tmp.h_out = h->h_out;
        tmp.w_out = h->w_out;
        tmp.s = c.s;
        if (build_sconv_image(&tmp, src, g, row_nnz) != CADNN_OK) continue;
        if (upload(&tmp) != CADNN_OK) { if (tmp.d_blob) cudaFree(tmp.d_blob); continue; }
        float us = time_schedule(&tmp, batch, x, y, st, reps);
        if (us > 0.0f && (best_us < 0.0f || us < best_us)) {
            best_us = us;
            best = c.s;
        }
        cudaFree(tmp.d_blob);
    }
    cudaStreamDestroy(st);
    cudaFree(x);
    cudaFree(y);
    h->s = best;
    h->nhwc_us = best_us;
    Geometry gg = g;
    bool linear = best.kind == KK_SCONV_LINEAR;
    finish_candidate(gg, h->s, linear);
    return CADNN_OK;
}

// Filters dealt to the warp slots of the planar kernel: blocks of G consecutive output
// channels, longest-processing-time inside a block so that a block's warps finish together.
void planar_order(cadnn_weights *h, const std::vector<int64_t> &row_nnz)
{
    const int c_out = h->desc.c_out;
    const int G = std::max(1, h->pl_NW / std::max(1, h->pl_KSW)) * h->pl_RPW;
    const int n_groups = ceil_div(c_out, G);
    // constant capacity whatever the grouping, so that the device copy can be rewritten in place;
    // four words per warp slot: {filter (-1 = none), first pair, end pair of its nonzeros, 0}
    const size_t cap = std::max((size_t)n_groups * G, (size_t)round_up(c_out, 128) + 128);
    h->pl_order.assign(cap * 4, 0);
    for (size_t i = 0; i < cap; ++i) h->pl_order[i * 4] = -1;
    for (int gi = 0; gi < n_groups; ++gi) {
        int lo = gi * G, hi = std::min(c_out, lo + G);
        std::vector<int64_t> load(row_nnz.begin() + lo, row_nnz.begin() + hi);
        std::vector<int> slot;
        balance_block(load, G, h->pl_RPW, slot);
        for (int sl = 0; sl < G; ++sl)
            if (slot[sl] >= 0) {
                const int co = lo + slot[sl];
                int32_t *rec = &h->pl_order[(size_t)(lo + sl) * 4];
                rec[0] = co;
                rec[1] = h->pl_ptr[co] >> 1;
                rec[2] = h->pl_ptr[co + 1] >> 1;
            }
    }
}

// Channel-planar image of a float conv layer: offsets address [c_in][in_h + 2][in_w + 2].
void build_planar_image(cadnn_weights *h, const Src &src, const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    const int halo = kPlanarHalo;
    if (src.s8 || d.groups != 1 || d.pad_w != d.pad || d.pad > halo || d.kh - 1 - d.pad > halo || d.kw - 1 - d.pad > halo) return;
    const long long plane = planar_pitch(d.in_h, d.in_w);
    if (plane * d.c_in >= (1LL << 31)) return;
    const int wp = d.in_w + 2 * halo;
    h->pl_ptr.assign(d.c_out + 1, 0);
    h->pl_ent.clear();
    int32_t running = 0;
    for (int co = 0; co < d.c_out; ++co) {
        h->pl_ptr[co] = running;
        int real = 0;
        for (int ci = 0; ci < d.c_in; ++ci)
            for (int ky = 0; ky < d.kh; ++ky)
                for (int kx = 0; kx < d.kw; ++kx) {
                    size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + ci;
                    if (!src.kept(wi)) continue;
                    float v = src.fval(wi);
                    uint32_t bits;
                    memcpy(&bits, &v, 4);
                    h->pl_ent.push_back(bits);
                    h->pl_ent.push_back((uint32_t)(ci * plane + (long long)(ky + halo - d.pad) * wp + kx + halo - d.pad));
                    ++real;
                }
        if (real & 1) {   // padding entry: weight 0 at offset 0
            h->pl_ent.push_back(0u);
            h->pl_ent.push_back(0u);
        }
        running += real + (real & 1);
    }
    h->pl_ptr[d.c_out] = running;
    // schedule: pixel bands per lane from the plane size, one or two filters per warp
    const long long qtot = (long long)h->h_out * (h->w_out + 2 * halo) * std::max(1, d.batch_hint);
    h->pl_NW = 8;
    h->pl_T = qtot >= 8L * 32 * kSmCount ? 8 : qtot >= 2L * 32 * kSmCount ? 4 : qtot >= 512 ? 2 : 1;
    long long warps = ((qtot + 32 * h->pl_T - 1) / (32 * h->pl_T)) * d.c_out;
    h->pl_RPW = warps >= 64L * kSmCount * 8 ? 4 : warps >= 32L * kSmCount * 4 ? 2 : 1;
    // few warps in the whole layer: let several warps share a filter's nonzeros
    h->pl_KSW = 1;
    const long long mean_pairs = std::max<long long>(1, running / 2 / std::max(1, d.c_out));
    while (h->pl_KSW < 8 && warps * h->pl_KSW < 24L * kSmCount && mean_pairs / (h->pl_KSW * 2) >= 8) h->pl_KSW *= 2;
    planar_order(h, row_nnz);
    h->has_planar = true;
}

template <class F>
float time_launches(F launch, cudaStream_t st, int reps, int replays = 2)
{
    if (launch() != CADNN_OK) return -1.0f;   // also raises the kernel's shared-memory limit outside the capture
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return -1.0f; }
    cudaGraph_t g = nullptr;
    cudaGraphExec_t ge = nullptr;
    float us = -1.0f;
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); return -1.0f; }
    bool ok = true;
    for (int r = 0; r < reps && ok; ++r) ok = launch() == CADNN_OK;
    if (cudaStreamEndCapture(st, &g) != cudaSuccess) ok = false;
    if (ok && cudaGraphInstantiate(&ge, g, 0) == cudaSuccess) {
        cudaEvent_t e0, e1;
        cudaEventCreate(&e0);
        cudaEventCreate(&e1);
        cudaGraphLaunch(ge, st);
        float best = 1e30f;
        for (int rep = 0; rep < replays; ++rep) {
            cudaEventRecord(e0, st);
            cudaGraphLaunch(ge, st);
            cudaEventRecord(e1, st);
            if (cudaStreamSynchronize(st) == cudaSuccess) {
                float ms = 0.0f;
                cudaEventElapsedTime(&ms, e0, e1);
                best = std::min(best, ms);
            }
        }
        if (best < 1e29f) us = best * 1e3f / (float)reps;
        cudaEventDestroy(e0);
        cudaEventDestroy(e1);
    }
    if (ge) cudaGraphExecDestroy(ge);
    if (g) cudaGraphDestroy(g);
    cudaGetLastError();
    return us;
}

// Time the planar kernel's launch shapes on the device and keep the fastest (the stored image does
// not depend on them; only the dealing of filters to warps does).
void autotune_planar(cadnn_weights *h, const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    const int halo = kPlanarHalo, batch = std::max(1, d.batch_hint);
    const size_t xb = (size_t)batch * d.c_in * planar_pitch(d.in_h, d.in_w) * 4;
    const size_t yb = (size_t)batch * d.c_out * planar_pitch(h->h_out, h->w_out) * 4;
    void *x = nullptr, *y = nullptr;
    cudaStream_t st = nullptr;
    if (cudaMalloc(&x, xb) != cudaSuccess || cudaMalloc(&y, yb) != cudaSuccess ||
        cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) {
        if (x) cudaFree(x);
        if (y) cudaFree(y);
        cudaGetLastError();
        return;
    }
    cudaMemsetAsync(x, 0, xb, st);
    cudaMemsetAsync(y, 0, yb, st);
    int32_t *d_order = const_cast<int32_t *>(h->d_pl_order);
    const size_t order_cap = h->pl_order.size();   // device room reserved for the order array
    float best_us = -1.0f;
    int bT = h->pl_T, bNW = h->pl_NW, bRPW = h->pl_RPW, bKSW = h->pl_KSW, bD = h->pl_D;
    LaunchEpilogue ep;
    ep.out_dtype = CADNN_F32;
    ep.act = CADNN_ACT_RELU;
    for (int T : {1, 2, 4, 8})
        for (int nw : {4, 8, 16})
            for (int ksw : {1, 2, 4, 8})
                for (int rpw : {1, 2, 4})
                  for (int dep : {1, 2, 4}) {
                    if (ksw > nw || nw > (T <= 4 ? 16 : 8)) continue;
                    if (dep > 1 && (T == 1 || dep > T)) continue;   // the kernel has no deeper variant there
                    // large batches fill the device with whole filters per warp and wide bands: the rest is not timed
                    if (batch >= 32 && (ksw > 1 || T < 4 || nw < 8 || dep > 2)) continue;
                    h->pl_T = T; h->pl_NW = nw; h->pl_KSW = ksw; h->pl_RPW = rpw; h->pl_D = dep;
                    planar_order(h, row_nnz);
                    if (h->pl_order.size() > order_cap) continue;
                    if (cudaMemcpyAsync(d_order, h->pl_order.data(), h->pl_order.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
                        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); continue; }
                    cudaGraph_t g = nullptr;
                    cudaGraphExec_t ge = nullptr;
                    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) { cudaGetLastError(); continue; }
                    bool ok = true;
                    const int reps = batch >= 32 ? 3 : 8;
                    for (int r = 0; r < reps && ok; ++r) ok = launch_sconv_planar(h, x, batch, y, ep, st) == CADNN_OK;
                    if (cudaStreamEndCapture(st, &g) != cudaSuccess) ok = false;
                    if (ok && cudaGraphInstantiate(&ge, g, 0) == cudaSuccess) {
                        cudaEvent_t e0, e1;
                        cudaEventCreate(&e0);
                        cudaEventCreate(&e1);
                        cudaGraphLaunch(ge, st);
                        cudaEventRecord(e0, st);
                        cudaGraphLaunch(ge, st);
                        cudaEventRecord(e1, st);
                        if (cudaStreamSynchronize(st) == cudaSuccess) {
                            float ms = 0.0f;
                            cudaEventElapsedTime(&ms, e0, e1);
                            float us = ms * 1e3f / (float)reps;
                            if (best_us < 0.0f || us < best_us) { best_us = us; bT = T; bNW = nw; bRPW = rpw; bKSW = ksw; bD = dep; }
                        }
                        cudaEventDestroy(e0);
                        cudaEventDestroy(e1);
                    }
                    if (ge) cudaGraphExecDestroy(ge);
                    if (g) cudaGraphDestroy(g);
                    cudaGetLastError();
                }
    h->pl_T = bT; h->pl_NW = bNW; h->pl_RPW = bRPW; h->pl_KSW = bKSW; h->pl_D = bD;
    // the chosen shape once more, longer: the figure the staged variant's is compared with
    if (best_us > 0.0f) {
        planar_order(h, row_nnz);
        if (cudaMemcpyAsync(d_order, h->pl_order.data(), h->pl_order.size() * 4, cudaMemcpyHostToDevice, st) == cudaSuccess &&
            cudaStreamSynchronize(st) == cudaSuccess) {
            const float us = time_launches([&]() { return launch_sconv_planar(h, x, batch, y, ep, st); }, st, batch >= 16 ? 4 : 16, 4);
            if (us > 0.0f) best_us = us;
        }
        cudaStreamSynchronize(st);
        cudaGetLastError();
    }
    h->pl_us = best_us;
    // the staged variant runs when it measured faster (an unmeasured one is not trusted against a measured one)
    if (h->has_ps && best_us > 0.0f) h->use_ps = (h->ps_us > 0.0f && h->ps_us <= best_us) || getenv("CADNN_FORCE_STAGED") != nullptr;
    planar_order(h, row_nnz);
    cudaMemcpyAsync(d_order, h->pl_order.data(), h->pl_order.size() * 4, cudaMemcpyHostToDevice, st);
    cudaStreamSynchronize(st);
    cudaStreamDestroy(st);
    cudaFree(x);
    cudaFree(y);
    cudaGetLastError();
}

// ---- shared-memory-staged planar kernel (planar_staged.cu): schedule, image, timing ----

// kept weights of every filter as (input channel, tap shift inside the padded plane, value), channel-major
struct PsRows {
    std::vector<int32_t> ptr;   // [c_out + 1]
    std::vector<int32_t> ci, tap;
    std::vector<float> v;
};

bool ps_eligible(const cadnn_layer_desc &d, bool s8)
{
    if (s8 || d.groups != 1 || (d.stride != 1 && d.stride != 2) || d.kh != d.kw || d.pad_w != d.pad || 2 * d.pad != d.kh - 1 || d.pad > kPlanarHalo) return false;
    return (long long)planar_pitch(d.in_h, d.in_w) * d.c_in < (1LL << 31);
}

void ps_collect_rows(const cadnn_layer_desc &d, const Src &src, PsRows &r)
{
    const int wp = d.in_w + 2 * kPlanarHalo;
    r.ptr.assign(d.c_out + 1, 0);
    for (int co = 0; co < d.c_out; ++co) {
        r.ptr[co] = (int32_t)r.ci.size();
        for (int ci = 0; ci < d.c_in; ++ci)
            for (int ky = 0; ky < d.kh; ++ky)
                for (int kx = 0; kx < d.kw; ++kx) {
                    const size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + ci;
                    if (!src.kept(wi)) continue;
                    r.ci.push_back(ci);
                    r.tap.push_back((ky - d.pad) * wp + (kx - d.pad));
                    r.v.push_back(src.fval(wi));
                }
    }
    r.ptr[d.c_out] = (int32_t)r.ci.size();
}

// derived fields of a staged-planar schedule from (T, RPW, NW, KS, CIc, stages); false if it cannot run
bool ps_finish(const cadnn_layer_desc &d, PsSchedule &s)
{
    const int wp = d.in_w + 2 * kPlanarHalo;
    if (s.KS < 1 || s.KS > s.NW || s.NW % s.KS || s.RPW * s.T > 32) return false;
    s.G = (s.NW / s.KS) * s.RPW;
    s.n_groups = ceil_div(d.c_out, s.G);
    s.CIc = std::max(1, std::min(s.CIc, d.c_in));
    s.n_chunks = ceil_div(d.c_in, s.CIc);
    if (!s.tma) s.KC = 1;
    if (s.KC > 1) {   // every block of a cluster takes the same number of chunks
        s.n_chunks = round_up(s.n_chunks, s.KC);
        s.CIc = round_up(ceil_div(d.c_in, s.n_chunks), 4);
        if ((s.n_chunks - 1) * s.CIc >= d.c_in) return false;   // a rank would have nothing to do
    }
    s.stages = std::max(1, std::min(std::min(s.stages, s.tma ? 8 : 3), s.n_chunks / s.KC));
    if (d.stride == 1) {
        s.R = 0;
        s.A = round_up(d.pad * (wp + 1), 4);
        s.L = 32 * s.T + 2 * s.A;
        if (s.tma && s.L > 256) return false;   // a box is at most 256 elements wide
        s.q_start = (kPlanarHalo * (wp + 1)) & ~3;                         // first interior position, rounded down
        const int q_end = (d.in_h + kPlanarHalo - 1) * wp + d.in_w + kPlanarHalo;   // one past the last interior position
        s.tiles = ceil_div(q_end - s.q_start, 32 * s.T);
    } else {
        // row tiles: as many output rows as fit the lanes' 32 T positions and a box of 256 input floats
        if (!s.tma) return false;
        const int h_out = (d.in_h + 2 * d.pad - d.kh) / d.stride + 1, w_out = (d.in_w + 2 * d.pad - d.kw) / d.stride + 1;
        const int wp_out = w_out + 2 * kPlanarHalo;
        int R = std::min(h_out, (32 * s.T) / wp_out);
        while (R >= 1 && (d.stride * (R - 1) + d.kh) * wp + 3 > 256) --R;
        if (R < 1) return false;
        if (s.T > 1 && R * wp_out <= 32 * (s.T / 2)) return false;   // fewer bands would do
        s.R = R;
        s.A = d.pad * wp + kPlanarHalo;   // entry offsets count from the first tap of the tile's first position
        s.L = round_up((d.stride * (R - 1) + d.kh) * wp + 3, 4);
        s.q_start = 0;
        s.tiles = ceil_div(h_out, R);
    }
    s.tile_bytes = s.CIc * s.L * 4;
    if (s.tma) {   // boxes of equal height (a multiple of 4 rows keeps every box 128-byte aligned in shared memory)
        s.nb = ceil_div(s.CIc, 256);
        s.RB = round_up(ceil_div(s.CIc, s.nb), 4);
        s.tile_bytes = s.nb * s.RB * s.L * 4;
    }
    s.hdr_bytes = round_up(s.G * s.KS + 1, 4) * 4;
    return true;
}

void ps_finish_smem(PsSchedule &s)
{
    s.block_bytes = s.hdr_bytes + s.max_entries * 8;
    s.stage_bytes = s.tile_bytes + s.block_bytes;
    if (s.tma) s.stage_bytes = round_up(s.stage_bytes, 128);
    const int red = (s.NW / s.KS) * (s.KS - 1) * s.RPW * s.T * 128;   // partial sums of the warps that share filters
    s.part_off = round_up(red, 128);
    const int part = s.KC > 1 ? s.G * s.T * 128 : 0;                   // partial sums of the blocks of a cluster
    s.smem_bytes = std::max(s.stages * s.stage_bytes + (s.tma ? 8 * s.stages : 0), s.part_off + part);
}

// Image for schedule h->ps (through ps_finish): one fixed-size record per (chunk, filter block): a header
// of G * KS + 1 segment starts, then the entries {value bits, byte offset into the staged tile}; the
// nonzeros a filter has in the chunk are cut into KS equal segments, each padded to an even count.
bool build_ps_image(cadnn_weights *h, const PsRows &rows, const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    PsSchedule &s = h->ps;
    const int c_pad = s.n_groups * s.G;
    h->ps_perm.assign(c_pad, -1);
    for (int gi = 0; gi < s.n_groups; ++gi) {
        int lo = gi * s.G, hi = std::min(d.c_out, lo + s.G);
        std::vector<int64_t> load(row_nnz.begin() + lo, row_nnz.begin() + hi);
        std::vector<int> slot;
        balance_block(load, s.G, s.RPW, slot);
        for (int sl = 0; sl < s.G; ++sl)
            if (slot[sl] >= 0) h->ps_perm[lo + sl] = lo + slot[sl];
    }
    const int hdr_words = s.hdr_bytes / 4;
    std::vector<std::vector<uint32_t>> blocks((size_t)s.n_chunks * s.n_groups);
    std::vector<int32_t> cur(rows.ptr.begin(), rows.ptr.end() - 1);   // next unread nonzero of every filter
    s.max_entries = 0;
    for (int c = 0; c < s.n_chunks; ++c) {
        const int c0 = c * s.CIc, c1 = std::min(d.c_in, c0 + s.CIc);
        for (int gi = 0; gi < s.n_groups; ++gi) {
            std::vector<uint32_t> &blk = blocks[(size_t)c * s.n_groups + gi];
            blk.assign(hdr_words, 0u);
            int running = 0;
            for (int sl = 0; sl < s.G; ++sl) {
                const int co = h->ps_perm[gi * s.G + sl];
                int lo = 0, cnt = 0;
                if (co >= 0) {
                    lo = cur[co];
                    int e = lo;
                    while (e < rows.ptr[co + 1] && rows.ci[e] < c1) ++e;
                    cnt = e - lo;
                    cur[co] = e;
                }
                for (int k = 0; k < s.KS; ++k) {
                    blk[sl * s.KS + k] = (uint32_t)running;
                    const int a = (int)((long long)cnt * k / s.KS), b = (int)((long long)cnt * (k + 1) / s.KS);
                    for (int e = lo + a; e < lo + b; ++e) {
                        uint32_t bits;
                        memcpy(&bits, &rows.v[e], 4);
                        blk.push_back(bits);
                        blk.push_back((uint32_t)(((rows.ci[e] - c0) * s.L + s.A + rows.tap[e]) * 4));
                    }
                    if ((b - a) & 1) {   // padding entry: weight 0 at offset 0
                        blk.push_back(0u);
                        blk.push_back(0u);
                    }
                    running += (b - a) + ((b - a) & 1);
                }
            }
            blk[s.G * s.KS] = (uint32_t)running;
            s.max_entries = std::max(s.max_entries, running);
        }
    }
    s.max_entries = std::max(s.max_entries, 2) + 16;   // + two batches of slack for the kernel's look-ahead (stays even)
    ps_finish_smem(s);
    if (s.smem_bytes > 220 * 1024) return false;
    const size_t block_words = (size_t)s.block_bytes / 4;
    h->ps_ent.assign(block_words * blocks.size(), 0u);
    for (size_t b = 0; b < blocks.size(); ++b) std::copy(blocks[b].begin(), blocks[b].end(), h->ps_ent.begin() + b * block_words);
    return true;
}

// default staged-planar schedule from the layer's shape
void ps_default(const cadnn_layer_desc &d, int64_t nnz, PsSchedule &s)
{
    const int wp = d.in_w + 2 * kPlanarHalo;
    const int range = d.in_h * wp;
    const int batch = std::max(1, d.batch_hint);
    s.T = (long long)range * batch >= 16L * 32 * kSmCount ? 8 : (long long)range * batch >= 2L * 32 * kSmCount ? 4 : range >= 512 ? 2 : 1;
    s.NW = 8;
    s.RPW = 2;
    s.KS = 1;
    const long long tiles = (long long)ceil_div(range, 32 * s.T) * batch;
    while (s.KS < 8 && tiles * ceil_div(d.c_out, (s.NW / s.KS) * s.RPW) < 2L * kSmCount && nnz / std::max(1, d.c_out) / (2 * s.KS) >= 8) s.KS *= 2;
    // the largest chunk whose two stages (tile + about its share of the nonzeros) fit 96 KB
    const int A = round_up(d.pad * (wp + 1), 4), L = 32 * s.T + 2 * A;
    s.CIc = d.c_in;
    s.stages = 1;
    const double per_ci = (double)L * 4 + 8.0 * 1.3 * (double)nnz / std::max(1, d.c_in) / std::max(1, ceil_div(d.c_out, (s.NW / s.KS) * s.RPW));
    if (per_ci * d.c_in > 64.0 * 1024) {
        s.stages = 2;
        s.CIc = std::max(4, (int)(48.0 * 1024 / per_ci) & ~3);
    }
}

// Time staged-planar schedules on the device and keep the fastest in h->ps (image not built here).
void autotune_ps(cadnn_weights *h, const PsRows &rows, const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    const int batch = std::max(1, d.batch_hint);
    // ways of cutting the input channels into chunks {chunks, stages, tma}: cp.async staging with
    // 1-3 stages; TMA staging with every chunk in flight at once, or a ring of fewer stages
    static const int kStaging[][3] = {{4, 4, 1}, {8, 4, 1}, {16, 4, 1}, {4, 2, 0},   // defaults of the first pass, in order of preference
                                      {1, 1, 1}, {2, 2, 1}, {8, 8, 1}, {4, 2, 1}, {1, 1, 0}, {2, 2, 0}, {8, 3, 0}};
    const int kDefaults = 4, kAll = 11;
    const bool no_tma = getenv("CADNN_NO_TMA") != nullptr;
    const bool no_cluster = getenv("CADNN_NO_CLUSTER") != nullptr;
    const int range = d.in_h * (d.in_w + 2 * kPlanarHalo);   // computed positions of a plane, about
    auto make = [&](int T, int nw, int ks, int rpw, int kc, const int *o, PsSchedule &s) {
        s = PsSchedule();
        s.T = T; s.NW = nw; s.KS = ks; s.RPW = rpw; s.KC = kc;
        s.tma = o[2];
        s.CIc = round_up(ceil_div(d.c_in, o[0] * kc), 4);
        s.stages = o[1];
        if ((s.tma && no_tma) || ((kc > 1 || d.stride != 1) && !s.tma)) return false;
        if (o[0] * kc > 1 && ceil_div(d.c_in, s.CIc) < 2) return false;
        if (!ps_finish(d, s)) return false;
        // nonzeros spread evenly is the optimistic guess for the record size
        const double rec = s.hdr_bytes + 8.0 * (double)h->nnz / s.n_chunks / s.n_groups;
        return s.stages * (s.tile_bytes + rec) <= 216.0 * 1024;
    };
    // first pass: the launch shape (bands, warps, warps per filter, filters per warp) with a default staging
    std::vector<PsSchedule> shapes;
    long long max_warps = 0;
    for (int T : {1, 2, 4, 8})
        for (int nw : {4, 8, 16})
            for (int ks : {1, 2, 4, 8})
                for (int rpw : {1, 2, 4, 8})
                    for (int kc : {1, 2, 4, 8}) {
                        if (ks > nw || rpw * T > 16 || (rpw == 8 && T > 1)) continue;
                        if (T > 1 && 32 * (T / 2) >= range) continue;   // bands nobody needs
                        if ((nw / ks) * rpw > d.c_out && rpw > 1) continue;
                        // a cluster split pays when many filters per block share the staged activations
                        if (kc > 1 && (no_cluster || d.c_in / kc < 64 || nw < 8 || ks > 2 || rpw < 2)) continue;
                        PsSchedule s;
                        bool ok = false;
                        if (kc > 1) {
                            static const int kc_staging[][3] = {{1, 1, 1}, {2, 2, 1}, {4, 2, 1}};
                            for (int k = 0; k < 3 && !ok; ++k) ok = make(T, nw, ks, rpw, kc, kc_staging[k], s);
                        } else {
                            for (int k = 0; k < kDefaults && !ok; ++k) ok = make(T, nw, ks, rpw, 1, kStaging[k], s);
                        }
                        if (!ok) continue;
                        shapes.push_back(s);
                        max_warps = std::max(max_warps, (long long)batch * s.tiles * s.n_groups * nw * s.KC);
                    }
    const long long want = std::min<long long>(8L * kSmCount, max_warps) / 2;
    const size_t xb = (size_t)batch * d.c_in * planar_pitch(d.in_h, d.in_w) * 4;
    const size_t yb = (size_t)batch * d.c_out * planar_pitch(h->h_out, h->w_out) * 4;
    void *x = nullptr, *y = nullptr;
    cudaStream_t st = nullptr;
    if (cudaMalloc(&x, xb) != cudaSuccess || cudaMalloc(&y, yb) != cudaSuccess ||
        cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) != cudaSuccess) {
        if (x) cudaFree(x);
        if (y) cudaFree(y);
        cudaGetLastError();
        return;
    }
    cudaMemsetAsync(x, 0, xb, st);
    cudaMemsetAsync(y, 0, yb, st);
    LaunchEpilogue ep;
    ep.out_dtype = CADNN_F32;
    ep.act = CADNN_ACT_RELU;
    auto time_one = [&](const PsSchedule &c, PsSchedule &built) -> float {
        cadnn_weights tmp;
        tmp.desc = d;
        tmp.desc.flags &= ~CADNN_PACK_HOST_ONLY;
        tmp.h_out = h->h_out;
        tmp.w_out = h->w_out;
        tmp.ps = c;
        if (!build_ps_image(&tmp, rows, row_nnz)) return -1.0f;
        if (upload(&tmp) != CADNN_OK) { if (tmp.d_blob) cudaFree(tmp.d_blob); return -1.0f; }
        const float us = time_launches([&]() { return launch_sconv_planar_staged(&tmp, x, batch, y, ep, st); }, st, batch >= 16 ? 3 : 8);
        built = tmp.ps;
        cudaFree(tmp.d_blob);
        return us;
    };
    std::vector<std::pair<float, PsSchedule>> timed;
    for (const PsSchedule &c : shapes) {
        const long long warps = (long long)batch * c.tiles * c.n_groups * c.NW * c.KC;
        if (warps < want) continue;
        PsSchedule built;
        const float us = time_one(c, built);
        if (us > 0.0f) timed.push_back({us, built});
    }
    std::stable_sort(timed.begin(), timed.end(), [](const std::pair<float, PsSchedule> &a, const std::pair<float, PsSchedule> &b) { return a.first < b.first; });
    // second pass: every staging for the best few shapes
    const size_t keep = std::min<size_t>(timed.size(), 4);
    for (size_t i = 0; i < keep; ++i) {
        const PsSchedule base = timed[i].second;
        for (int k = 0; k < kAll; ++k) {
            PsSchedule s, built;
            if (!make(base.T, base.NW, base.KS, base.RPW, base.KC, kStaging[k], s)) continue;
            if (s.tma == base.tma && s.CIc == base.CIc && s.stages == base.stages) continue;
            const float us = time_one(s, built);
            if (us > 0.0f) timed.push_back({us, built});
        }
    }
    // last pass: the few fastest once more, longer, and with a residual tensor in the epilogue (most layers of a
    // residual network have one); candidates within the noise of the short runs get separated here
    std::stable_sort(timed.begin(), timed.end(), [](const std::pair<float, PsSchedule> &a, const std::pair<float, PsSchedule> &b) { return a.first < b.first; });
    void *res = nullptr;
    if (!timed.empty() && cudaMalloc(&res, yb) == cudaSuccess) {
        cudaMemsetAsync(res, 0, yb, st);
        ep.residual = res;
        const size_t finals = std::min<size_t>(timed.size(), 4);
        std::vector<std::pair<float, PsSchedule>> again;
        for (size_t i = 0; i < finals; ++i) {
            cadnn_weights tmp;
            tmp.desc = d;
            tmp.desc.flags &= ~CADNN_PACK_HOST_ONLY;
            tmp.h_out = h->h_out;
            tmp.w_out = h->w_out;
            tmp.ps = timed[i].second;
            if (!build_ps_image(&tmp, rows, row_nnz)) continue;
            if (upload(&tmp) == CADNN_OK) {
                const float us = time_launches([&]() { return launch_sconv_planar_staged(&tmp, x, batch, y, ep, st); }, st,
                                               batch >= 16 ? 4 : 16, 4);
                if (us > 0.0f) again.push_back({us, tmp.ps});
            }
            if (tmp.d_blob) cudaFree(tmp.d_blob);
        }
        ep.residual = nullptr;
        if (!again.empty()) {
            // the winner's time WITHOUT the residual is what gets compared with the other kernels of the layer (direct
            // planar, NHWC), which are timed without one
            size_t bi = 0;
            for (size_t i = 1; i < again.size(); ++i)
                if (again[i].first < again[bi].first) bi = i;
            std::pair<float, PsSchedule> best = again[bi];
            cadnn_weights tmp;
            tmp.desc = d;
            tmp.desc.flags &= ~CADNN_PACK_HOST_ONLY;
            tmp.h_out = h->h_out;
            tmp.w_out = h->w_out;
            tmp.ps = best.second;
            if (build_ps_image(&tmp, rows, row_nnz) && upload(&tmp) == CADNN_OK) {
                const float us = time_launches([&]() { return launch_sconv_planar_staged(&tmp, x, batch, y, ep, st); }, st,
                                               batch >= 16 ? 4 : 16, 4);
                if (us > 0.0f) best.first = us;
            }
            if (tmp.d_blob) cudaFree(tmp.d_blob);
            timed.assign(1, best);
        }
        cudaStreamSynchronize(st);
        cudaFree(res);
    }
    cudaGetLastError();
    cudaStreamDestroy(st);
    cudaFree(x);
    cudaFree(y);
    cudaGetLastError();
    float best_us = -1.0f;
    for (const auto &t : timed)
        if (best_us < 0.0f || t.first < best_us) {
            best_us = t.first;
            h->ps = t.second;
        }
    if (best_us > 0.0f) h->ps_us = best_us;
}

// ---- schedule cache -------------------------------------------------------------------------
// Section 4, "Optimization parameters selection": the parameters of a layer are searched once.
// With CADNN_TUNE_CACHE=<file> in the environment the measured choices of every layer packed
// with CADNN_PACK_AUTOTUNE are appended to that file, and a later pack of the same layer (same
// geometry, batch hint and nonzeros per filter) takes them from it instead of timing again.  So a
// model is tuned once per machine, and a run under a profiler (whose overhead perturbs the
// timings) executes exactly the schedules of the plain run.
uint64_t tune_key(const cadnn_layer_desc &d, const std::vector<int64_t> &row_nnz)
{
    uint64_t hsh = 1469598103934665603ull;
    auto mix = [&](uint64_t v) {
        for (int i = 0; i < 8; ++i) {
            hsh ^= (v >> (8 * i)) & 0xffu;
            hsh *= 1099511628211ull;
        }
    };
    for (int v : {d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad, d.pad_w, d.groups, d.in_h, d.in_w, std::max(1, d.batch_hint), (int)d.dtype})
        mix((uint64_t)(int64_t)v);
    mix(sizeof(Schedule));
    mix(sizeof(PsSchedule));
    for (int64_t v : row_nnz) mix((uint64_t)v);
    return hsh;
}

void to_hex(const void *p, size_t n, std::string &out)
{
    static const char *dig = "0123456789abcdef";
    const unsigned char *b = (const unsigned char *)p;
    for (size_t i = 0; i < n; ++i) {
        out.push_back(dig[b[i] >> 4]);
        out.push_back(dig[b[i] & 15]);
    }
}

bool from_hex(const char *txt, void *p, size_t n)
{
    unsigned char *b = (unsigned char *)p;
    for (size_t i = 0; i < n; ++i) {
        int v = 0;
        for (int k = 0; k < 2; ++k) {
            const char c = txt[2 * i + k];
            int d;
            if (c >= '0' && c <= '9') d = c - '0';
            else if (c >= 'a' && c <= 'f') d = c - 'a' + 10;
            else return false;
            v = v * 16 + d;
        }
        b[i] = (unsigned char)v;
    }
    return true;
}

bool tune_lookup(uint64_t key, TuneRecord &rec)
{
    const char *path = getenv("CADNN_TUNE_CACHE");
    if (!path || !*path) return false;
    FILE *f = fopen(path, "r");
    if (!f) return false;
    const size_t hexlen = 2 * sizeof(TuneRecord);
    std::vector<char> line(hexlen + 64);
    bool found = false;
    while (fgets(line.data(), (int)line.size(), f)) {
        unsigned long long k = 0;
        int pos = 0;
        if (sscanf(line.data(), "%llx %n", &k, &pos) < 1 || k != key) continue;
        if (strlen(line.data() + pos) < hexlen) continue;
        TuneRecord r;
        if (from_hex(line.data() + pos, &r, sizeof(r))) {
            rec = r;
            found = true;   // the last record of a key wins
        }
    }
    fclose(f);
    return found;
}

void tune_store(uint64_t key, const TuneRecord &rec)
{
    const char *path = getenv("CADNN_TUNE_CACHE");
    if (!path || !*path) return;
    std::string out;
    char head[32];
    snprintf(head, sizeof(head), "%016llx ", (unsigned long long)key);
    out = head;
    to_hex(&rec, sizeof(rec), out);
    out.push_back('\n');
    FILE *f = fopen(path, "a");
    if (!f) return;
    fwrite(out.data(), 1, out.size(), f);   // one write per record: concurrent packers do not interleave
    fclose(f);
}

void pack_ps(cadnn_weights *h, const Src &src, const std::vector<int64_t> &row_nnz)
{
    const cadnn_layer_desc &d = h->desc;
    if (!ps_eligible(d, src.s8) || getenv("CADNN_NO_STAGED")) return;
    PsRows rows;
    ps_collect_rows(d, src, rows);
    ps_default(d, h->nnz, h->ps);
    if (d.stride != 1) {   // row tiles are staged by TMA only
        h->ps.tma = 1;
        h->ps.T = std::min(h->ps.T, 2);
        while (h->ps.T < 8 && !ps_finish(d, h->ps)) h->ps.T *= 2;
    }
    if (!ps_finish(d, h->ps)) return;
    const char *env = getenv("CADNN_PLANAR_SCHEDULE");   // tuning / test switch: "t=2,nw=16,ks=2,rpw=1,chunks=4,stages=2,tma=1,kc=2" (any subset)
    if (env) {
        PsSchedule s = h->ps;
        int v, chunks = s.n_chunks;
        const char *q;
        if ((q = strstr(env, "t=")) && sscanf(q + 2, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) s.T = v;
        if ((q = strstr(env, "nw=")) && sscanf(q + 3, "%d", &v) == 1 && (v == 4 || v == 8 || v == 16)) s.NW = v;
        if ((q = strstr(env, "ks=")) && sscanf(q + 3, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) s.KS = v;
        if ((q = strstr(env, "rpw=")) && sscanf(q + 4, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) s.RPW = v;
        if ((q = strstr(env, "kc=")) && sscanf(q + 3, "%d", &v) == 1 && (v == 1 || v == 2 || v == 4 || v == 8)) s.KC = v;
        if ((q = strstr(env, "tma=")) && sscanf(q + 4, "%d", &v) == 1 && (v == 0 || v == 1)) s.tma = v;
        if ((q = strstr(env, "chunks=")) && sscanf(q + 7, "%d", &v) == 1 && v >= 1 && v <= 64) chunks = v;
        if ((q = strstr(env, "stages=")) && sscanf(q + 7, "%d", &v) == 1 && v >= 1 && v <= 8) s.stages = v;
        s.CIc = round_up(ceil_div(d.c_in, chunks), 4);
        if (s.RPW * s.T <= 16 && !(s.RPW == 8 && s.T > 4) && ps_finish(d, s)) h->ps = s;
    } else if (h->tuned && h->tuned->ps.T > 0) {
        h->ps = h->tuned->ps;
        h->ps_us = h->tuned->ps_us;
    } else if ((d.flags & CADNN_PACK_AUTOTUNE) && !(d.flags & CADNN_PACK_HOST_ONLY)) {
        autotune_ps(h, rows, row_nnz);
    }
    ps_finish(d, h->ps);
    for (int attempt = 0; attempt < 8; ++attempt) {
        if (build_ps_image(h, rows, row_nnz)) {
            h->has_ps = true;
            h->use_ps = true;
            return;
        }
        // a dense or skewed layer can overflow shared memory: halve the chunk and repack
        if (h->ps.CIc <= 1) break;
        h->ps.CIc = std::max(1, (h->ps.CIc / 2 + 3) & ~3);
        h->ps.stages = 2;
        if (!ps_finish(d, h->ps)) break;
    }
    h->ps_ent.clear();
    h->ps_perm.clear();
}

cadnn_status pack_sconv(cadnn_weights *h, const Src &src)
{
    const cadnn_layer_desc &d = h->desc;
    const bool linear = (d.kh == 1 && d.kw == 1 && d.pad == 0 && d.pad_w == 0);
    const int K = d.kh * d.kw * d.c_in;
    int bh = std::max(1, d.batch_hint);
    std::vector<int64_t> row_nnz(d.c_out, 0);
    for (int co = 0; co < d.c_out; ++co) {
        int64_t c = 0;
        for (int k = 0; k < K; ++k) c += src.kept((size_t)co * K + k);
        row_nnz[co] = c;
        h->nnz += c;
    }
    Geometry g{d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad, d.in_h, d.in_w, h->h_out, h->w_out, src.s8, (double)h->nnz};
    std::vector<Candidate> cands;
    enumerate_schedules(g, bh, linear, cands);
    h->s = cands[0].s;
    const bool tune = (d.flags & CADNN_PACK_AUTOTUNE) && !(d.flags & CADNN_PACK_HOST_ONLY) && !getenv("CADNN_SCHEDULE") &&
                      !getenv("CADNN_PLANAR_SCHEDULE");
    if (tune) {
        h->tune_key = tune_key(d, row_nnz);
        TuneRecord rec;
        if (tune_lookup(h->tune_key, rec)) h->tuned = std::make_shared<TuneRecord>(rec);
    }
    if (h->tuned) {
        h->s = h->tuned->s;
        h->nhwc_us = h->tuned->nhwc_us;
    } else if ((d.flags & CADNN_PACK_AUTOTUNE) && !(d.flags & CADNN_PACK_HOST_ONLY) && !getenv("CADNN_SCHEDULE")) {
        cadnn_status st = autotune_sconv(h, src, g, row_nnz, cands);
        if (st != CADNN_OK) return st;
    }
    apply_env_override(g, linear, h->s);
    h->row_nnz = row_nnz;
    build_planar_image(h, src, row_nnz);
    if (h->has_planar && h->tuned) {   // the cached launch shape of the direct planar kernel
        h->pl_T = h->tuned->pl_T; h->pl_NW = h->tuned->pl_NW; h->pl_RPW = h->tuned->pl_RPW;
        h->pl_KSW = h->tuned->pl_KSW; h->pl_D = h->tuned->pl_D; h->pl_us = h->tuned->pl_us;
        planar_order(h, row_nnz);
    }
    if (h->has_planar) pack_ps(h, src, row_nnz);
    if (h->tuned && h->has_ps) h->use_ps = h->tuned->use_ps != 0;
    return build_sconv_image(h, src, g, row_nnz);
}

cadnn_status pack_fc_spmv(cadnn_weights *h, const Src &src)
{
    const cadnn_layer_desc &d = h->desc;
    const int K = d.c_in;
    if (K > 65536) return CADNN_E_UNSUPPORTED;
    Schedule &s = h->s;
    s.kind = KK_FC_SPMV;
    s.T = 1;
    s.RPW = 1;
    s.NW = kWarpsPerBlock;
    s.G = kWarpsPerBlock;
    s.n_groups = ceil_div(d.c_out, s.G);
    h->c_pad = s.n_groups * s.G;
    std::vector<int64_t> row_nnz(d.c_out, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int k = 0; k < K; ++k) row_nnz[co] += src.kept((size_t)co * K + k);
    // rows sorted by length: the warps of a block walk rows of similar length and the
    // longest rows are scheduled first
    std::vector<int> order(d.c_out);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return row_nnz[a] > row_nnz[b]; });
    h->perm.assign(h->c_pad, -1);
    for (int i = 0; i < d.c_out; ++i) h->perm[i] = order[i];
    // rows are padded to a multiple of 4 entries (weight 0 at column 0), so that a lane fetches four values and four
    // column indices with one load each; cnt keeps the real lengths
    h->ptr.assign(h->c_pad + 1, 0);
    h->cnt.assign(h->c_pad, 0);
    int32_t running = 0;
    int64_t real = 0;
    for (int r = 0; r < h->c_pad; ++r) {
        h->ptr[r] = running;
        int co = h->perm[r];
        if (co < 0) continue;
        int len = 0;
        for (int k = 0; k < K; ++k) {
            size_t wi = (size_t)co * K + k;
            if (!src.kept(wi)) continue;
            h->offs.push_back((uint16_t)k);
            if (src.s8) h->vals_q.push_back(src.qval(wi, co));
            else h->vals_f.push_back(src.fval(wi));
            ++len;
        }
        h->cnt[r] = len;
        real += len;
        for (; len & 3; ++len) {
            h->offs.push_back(0);
            if (src.s8) h->vals_q.push_back(0);
            else h->vals_f.push_back(0.0f);
        }
        running += len;
    }
    h->ptr[h->c_pad] = running;
    h->nnz = real;
    h->fmt = CADNN_FMT_ROW_CSR;
    return CADNN_OK;
}

cadnn_status pack_dense(cadnn_weights *h, const Src &src, int kind)
{
    const cadnn_layer_desc &d = h->desc;
    if (src.s8) return CADNN_E_UNSUPPORTED;
    const int cg = d.c_in / d.groups;
    const int taps = d.kh * d.kw * cg;
    // tap-major: [kh][kw][cg][c_out], so that lanes over output channels read contiguously
    h->dense_f.assign((size_t)taps * d.c_out, 0.0f);
    h->dense_kept.assign((size_t)taps * d.c_out, 0);
    for (int co = 0; co < d.c_out; ++co)
        for (int t = 0; t < taps; ++t) {
            size_t wi = (size_t)co * taps + t;
            if (src.kept(wi)) {
                h->dense_f[(size_t)t * d.c_out + co] = src.fval(wi);
                h->dense_kept[wi] = 1;
                h->nnz++;
            }
        }
    h->s.kind = kind;
    h->fmt = kind == KK_DW ? CADNN_FMT_DENSE_DW : CADNN_FMT_DENSE_SMALLC;
    return CADNN_OK;
}

cadnn_status pack_common(const cadnn_layer_desc *desc, const Src &src, cadnn_weights **out)
{
    if (!desc || !out || (!src.f && !src.q)) return CADNN_E_ARG;
    cadnn_layer_desc dn = *desc;
    if (dn.pad_w < 0) dn.pad_w = dn.pad;   // from here on pad = rows, pad_w = columns
    const cadnn_layer_desc &d = dn;
    if (d.c_in < 1 || d.c_out < 1 || d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0 || d.groups < 1 ||
        d.in_h < 1 || d.in_w < 1)
        return CADNN_E_ARG;
    if (d.dtype != CADNN_F32 && d.dtype != CADNN_S8) return CADNN_E_DTYPE;
    if (d.dtype == CADNN_S8 && !src.q && !src.w_scale) return CADNN_E_ARG;
    if (d.dtype == CADNN_F32 && (src.q || src.w_scale)) return CADNN_E_DTYPE;
    if (d.in_h + 2 * d.pad < d.kh || d.in_w + 2 * d.pad_w < d.kw) return CADNN_E_SHAPE;
    if (d.pad >= d.kh || d.pad_w >= d.kw) return CADNN_E_UNSUPPORTED;
    const bool depthwise = d.groups > 1 && d.groups == d.c_in && d.c_in == d.c_out;
    if (d.groups != 1 && !depthwise) return CADNN_E_UNSUPPORTED;
    const long K = (long)d.kh * d.kw * d.c_in / d.groups;
    if (d.dtype == CADNN_S8 && (double)K * 127.0 * 127.0 >= 2147483648.0) return CADNN_E_UNSUPPORTED;

    cadnn_weights *h = new (std::nothrow) cadnn_weights();
    if (!h) return CADNN_E_ALLOC;
    h->desc = d;
    h->h_out = (d.in_h + 2 * d.pad - d.kh) / d.stride + 1;
    h->w_out = (d.in_w + 2 * d.pad_w - d.kw) / d.stride + 1;
    cadnn_status st;
    try {
        const bool is_fc = d.kh == 1 && d.kw == 1 && d.in_h == 1 && d.in_w == 1 && d.pad == 0 && d.pad_w == 0;
        // a float layer with <= 4 input channels whose mask keeps (nearly) everything is a dense stem
        bool dense_stem = false;
        if (!depthwise && d.dtype == CADNN_F32 && d.c_in <= 4 && (d.kh > 1 || d.kw > 1) &&
            (size_t)d.kh * d.kw * d.c_in * 64 * 4 <= 160 * 1024) {
            size_t numel = (size_t)d.c_out * d.kh * d.kw * d.c_in, kept = 0;
            for (size_t i = 0; i < numel; ++i) kept += src.kept(i);
            dense_stem = kept * 2 >= numel;
        }
        std::vector<uint8_t> rem_mask;
        std::vector<int8_t> q_codes;
        if (d.fmt == CADNN_FMT_GROUPED) {
            // block-structured int8 layer: the dense blocks go to the tensor-core image, the sparse image keeps the rest
            if (depthwise || d.dtype != CADNN_S8) st = CADNN_E_UNSUPPORTED;
            else {
                const size_t numel = (size_t)d.c_out * d.kh * d.kw * d.c_in;
                const int8_t *qp = src.q;
                if (!qp) {
                    q_codes.resize(numel);
                    const size_t per = numel / d.c_out;
                    for (size_t i = 0; i < numel; ++i) q_codes[i] = src.qval(i, (int)(i / per));
                    qp = q_codes.data();
                }
                double thr = 0.5;
                if (const char *e = getenv("CADNN_BLOCK_DENSITY")) thr = std::min(1.0, std::max(0.0, atof(e)));
                if (!block_tc_extract(h, qp, src.mask, thr, rem_mask)) st = CADNN_E_UNSUPPORTED;
                else {
                    Src rest = src;
                    rest.mask = rem_mask.data();
                    st = pack_sconv(h, rest);
                    h->nnz += h->tc_nnz;
                    h->fmt = CADNN_FMT_GROUPED;
                }
            }
        }
        else if (depthwise) st = pack_dense(h, src, KK_DW);
        else if (dense_stem) st = pack_dense(h, src, KK_DENSE_SMALLC);
        else if (is_fc && std::max(1, d.batch_hint) <= 8 && d.c_in <= 65536) st = pack_fc_spmv(h, src);
        else st = pack_sconv(h, src);
        if (st == CADNN_OK) st = upload(h);
        if (st == CADNN_OK) st = block_tc_upload(h);
        if (st == CADNN_OK && h->has_planar && h->on_device && (d.flags & CADNN_PACK_AUTOTUNE) && !h->tuned)
            autotune_planar(h, h->row_nnz);
        if (st == CADNN_OK && h->tune_key && !h->tuned && h->on_device) {   // remember what was measured
            TuneRecord rec;
            memset(&rec, 0, sizeof(rec));
            rec.s = h->s;
            if (h->has_ps) rec.ps = h->ps; else rec.ps.T = 0;
            rec.pl_T = h->pl_T; rec.pl_NW = h->pl_NW; rec.pl_RPW = h->pl_RPW; rec.pl_KSW = h->pl_KSW; rec.pl_D = h->pl_D;
            rec.use_ps = (h->has_ps && h->use_ps) ? 1 : 0;
            rec.pl_us = h->pl_us; rec.ps_us = h->ps_us; rec.nhwc_us = h->nhwc_us;
            tune_store(h->tune_key, rec);
        }
        // A float stride-2 layer (3x3 with padding 1, or 1x1) also gets the form a network uses when the layer before it
        // writes its map split by row and column parity: input pixel (2 oy + ky - 1, 2 ox + kx - 1) is pixel
        // (oy + dy, ox + dx) of parity plane ((ky - 1) & 1, (kx - 1) & 1) with dy = -1 for ky = 0 and 0 otherwise, so the
        // layer is a stride-1 layer over the 4 c_in quarter planes (taps 0 and 1 of a padded 3x3 frame); a 1x1 layer
        // reads the (even, even) plane alone.
        const bool k3 = d.kh == 3 && d.kw == 3 && d.pad == 1 && d.pad_w == 1, k1 = d.kh == 1 && d.kw == 1 && d.pad == 0 && d.pad_w == 0;
        if (st == CADNN_OK && d.dtype == CADNN_F32 && d.stride == 2 && d.groups == 1 && (k3 || k1) && h->has_planar &&
            (h->on_device || (d.flags & CADNN_PACK_HOST_ONLY)) && src.f && getenv("CADNN_NO_PARITY_PLANES") == nullptr) {
            cadnn_layer_desc dc = d;
            dc.stride = 1;
            dc.in_h = (d.in_h + 1) / 2;
            dc.in_w = (d.in_w + 1) / 2;
            dc.c_in = k3 ? 4 * d.c_in : d.c_in;
            const size_t per = (size_t)d.kh * d.kw * dc.c_in, numel = per * d.c_out;
            std::vector<float> wc(numel, 0.0f);
            std::vector<uint8_t> mc(numel, 0);
            for (int co = 0; co < d.c_out; ++co)
                for (int ky = 0; ky < d.kh; ++ky)
                    for (int kx = 0; kx < d.kw; ++kx)
                        for (int ci = 0; ci < d.c_in; ++ci) {
                            const size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + ci;
                            if (!src.kept(wi)) continue;
                            size_t wo = wi;
                            if (k3) {
                                const int par = (ky == 1 ? 0 : 2) + (kx == 1 ? 0 : 1);
                                const int ty = ky == 0 ? 0 : 1, tx = kx == 0 ? 0 : 1;
                                wo = (((size_t)co * 3 + ty) * 3 + tx) * dc.c_in + (size_t)par * d.c_in + ci;
                            }
                            wc[wo] = src.f[wi];
                            mc[wo] = 1;
                        }
            Src sc;
            sc.f = wc.data();
            sc.mask = mc.data();
            cadnn_weights *child = nullptr;
            if (pack_common(&dc, sc, &child) == CADNN_OK) {
                if (child->has_planar && child->h_out == h->h_out && child->w_out == h->w_out) h->half = child;
                else cadnn_weights_free(child);
            }
        }
    } catch (const std::bad_alloc &) {
        st = CADNN_E_ALLOC;
    }
    if (st != CADNN_OK) {
        cadnn_weights_free(h);
        return st;
    }
    *out = h;
    return CADNN_OK;
}

}  // namespace

extern "C" {

cadnn_status cadnn_pack(const cadnn_layer_desc *desc, const float *w_ohwi, const uint8_t *mask,
                        const float *w_scale, cadnn_weights **out)
{
    Src s;
    s.f = w_ohwi;
    s.mask = mask;
    s.w_scale = w_scale;
    s.s8 = desc && desc->dtype == CADNN_S8;
    return pack_common(desc, s, out);
}

cadnn_status cadnn_pack_q8(const cadnn_layer_desc *desc, const int8_t *q_ohwi, const uint8_t *mask,
                           cadnn_weights **out)
{
    if (desc && desc->dtype != CADNN_S8) return CADNN_E_DTYPE;
    Src s;
    s.q = q_ohwi;
    s.mask = mask;
    s.s8 = true;
    return pack_common(desc, s, out);
}

cadnn_status cadnn_weights_info(const cadnn_weights *w, int64_t *nnz, int64_t *packed_bytes, int *fmt)
{
    if (!w) return CADNN_E_ARG;
    if (nnz) *nnz = w->nnz;
    if (packed_bytes) *packed_bytes = w->packed_bytes;
    if (fmt) *fmt = w->fmt;
    return CADNN_OK;
}

cadnn_status cadnn_weights_schedule(const cadnn_weights *w, int sched[16])
{
    if (!w || !sched) return CADNN_E_ARG;
    const Schedule &s = w->s;
    int v[16] = {s.kind, s.T, s.RPW, s.G, s.CIc, s.TH, s.TW, s.pitch, s.NW, s.stages, s.ksplit, s.n_chunks,
                 s.smem_bytes, s.TBX, s.TBY, s.max_entries};
    memcpy(sched, v, sizeof(v));
    return CADNN_OK;
}

cadnn_status cadnn_weights_planar_schedule(const cadnn_weights *w, int sched[16])
{
    if (!w || !sched) return CADNN_E_ARG;
    int v[16] = {0};
    if (w->has_ps && w->use_ps) {
        const PsSchedule &s = w->ps;
        int t[16] = {2, s.T, s.RPW, s.NW, s.KS, s.G, s.CIc, s.stages, s.n_chunks, s.tiles, s.smem_bytes, s.max_entries,
                     (int)lrintf(w->ps_us * 100.0f), (int)lrintf(w->pl_us * 100.0f), s.tma, s.KC};
        memcpy(v, t, sizeof(v));
    } else if (w->has_planar) {
        const int slots = std::max(1, w->pl_NW / std::max(1, w->pl_KSW));
        int t[16] = {1, w->pl_T, w->pl_RPW, w->pl_NW, w->pl_KSW, slots * w->pl_RPW, w->desc.c_in, w->pl_D, 1, 0, 0, 0,
                     (int)lrintf(w->ps_us * 100.0f), (int)lrintf(w->pl_us * 100.0f), 0, 0};
        memcpy(v, t, sizeof(v));
    }
    memcpy(sched, v, sizeof(v));
    return CADNN_OK;
}

cadnn_status cadnn_weights_parity_form(const cadnn_weights *w, const cadnn_weights **form)
{
    if (!w || !form) return CADNN_E_ARG;
    *form = w->half;
    return CADNN_OK;
}

cadnn_status cadnn_weights_warp_loads(const cadnn_weights *w, int64_t *loads, int cap, int *n_out)
{
    if (!w || !n_out) return CADNN_E_ARG;
    const Schedule &s = w->s;
    if (s.kind != KK_SCONV_SPATIAL && s.kind != KK_SCONV_LINEAR && s.kind != KK_FC_SPMV) {
        *n_out = 0;
        return CADNN_OK;
    }
    int chunks = s.kind == KK_FC_SPMV ? 1 : s.n_chunks;
    int n_warps = w->c_pad / s.RPW;
    *n_out = n_warps;
    if (!loads) return CADNN_OK;
    for (int i = 0; i < n_warps && i < cap; ++i) {
        int64_t tot = 0;
        for (int c = 0; c < chunks; ++c) {
            if (s.kind == KK_FC_SPMV) {
                for (int j = 0; j < s.RPW; ++j) tot += w->cnt[(size_t)i * s.RPW + j];   // real entries, without row padding
            } else {
                for (int j = 0; j < s.RPW; ++j) tot += w->cnt[(size_t)c * w->c_pad + i * s.RPW + j];
            }
        }
        loads[i] = tot;
    }
    return CADNN_OK;
}

cadnn_status cadnn_weights_unpack(const cadnn_weights *w, float *dense, uint8_t *mask)
{
    if (!w) return CADNN_E_ARG;
    const cadnn_layer_desc &d = w->desc;
    const Schedule &s = w->s;
    const int cg = d.c_in / d.groups;
    const size_t K = (size_t)d.kh * d.kw * cg, numel = K * d.c_out;
    if (dense) std::fill(dense, dense + numel, 0.0f);
    if (mask) std::fill(mask, mask + numel, (uint8_t)0);
    auto val = [&](size_t e) { return d.dtype == CADNN_S8 ? (float)w->vals_q[e] : w->vals_f[e]; };
    if (s.kind == KK_DW || s.kind == KK_DENSE_SMALLC) {
        for (int co = 0; co < d.c_out; ++co)
            for (size_t t = 0; t < K; ++t) {
                if (dense) dense[co * K + t] = w->dense_f[t * d.c_out + co];
                if (mask) mask[co * K + t] = w->dense_kept[co * K + t];
            }
        return CADNN_OK;
    }
    if (s.kind == KK_FC_SPMV) {
        for (int r = 0; r < w->c_pad; ++r) {
            int co = w->perm[r];
            if (co < 0) continue;
            for (int e = w->ptr[r]; e < w->ptr[r] + w->cnt[r]; ++e) {   // the rest of the row is padding
                size_t wi = (size_t)co * K + w->offs[e];
                if (dense) dense[wi] = val(e);
                if (mask) mask[wi] = 1;
            }
        }
        return CADNN_OK;
    }
    const bool linear = s.kind == KK_SCONV_LINEAR;
    const bool s8 = d.dtype == CADNN_S8;
    const int ew = s8 ? 1 : 2;
    const int hdr_words = header_words(s);
    const size_t block_words = (size_t)hdr_words + (size_t)s.max_entries * ew;
    for (int c = 0; c < s.n_chunks; ++c) {
        for (int r = 0; r < w->c_pad; ++r) {
            int co = w->perm[r];
            if (co < 0) continue;
            const uint32_t *blk = &w->ent[((size_t)c * s.n_groups + r / s.G) * block_words];
            const uint32_t *ents = blk + hdr_words;
            const int real = w->cnt[(size_t)c * w->c_pad + r];
            const int first = (int)blk[r % s.G];
            for (int e = first; e < first + real; ++e) {
                uint32_t off;
                float v;
                if (s8) {
                    uint32_t word = ents[e];
                    off = word >> 8;
                    v = (float)(int8_t)(word & 0xffu);
                } else {
                    uint32_t bits = ents[(size_t)e * ew];
                    memcpy(&v, &bits, 4);
                    off = ents[(size_t)e * ew + 1];
                }
                int cl = (int)(off % (uint32_t)s.PPb) / (s8 ? 1 : 4);
                int t = (int)(off / (uint32_t)s.PPb);
                int kx = 0, ky = 0;
                if (!linear) {
                    int pos = t % s.pitch;
                    ky = t / s.pitch;
                    kx = s.half ? (pos >= s.half ? 2 * (pos - s.half) + 1 : 2 * pos) : pos;
                }
                size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + (size_t)c * s.CIc + cl;
                if (dense) dense[wi] = v;
                if (mask) mask[wi] = 1;
            }
        }
    }
    if (w->has_tc) {   // the dense blocks of a block-structured layer
        const int n_nt = d.c_out / 64;
        for (int nt = 0; nt < n_nt; ++nt)
            for (int bi = w->tc_tile_ptr[nt]; bi < w->tc_tile_ptr[nt + 1]; ++bi) {
                const int kx = w->tc_blk[bi * 4] + d.pad_w, ky = w->tc_blk[bi * 4 + 1] + d.pad, c0 = w->tc_blk[bi * 4 + 2];
                for (int r = 0; r < 64; ++r)
                    for (int c = 0; c < 64; ++c) {
                        if (!w->tc_kept[(size_t)bi * 4096 + r * 64 + c]) continue;
                        const size_t wi = ((((size_t)(nt * 64 + r)) * d.kh + ky) * d.kw + kx) * d.c_in + c0 + c;
                        const int chunk = (c >> 4) ^ ((r >> 1) & 3);
                        if (dense) dense[wi] = (float)w->tc_wblk[(size_t)bi * 4096 + r * 64 + chunk * 16 + (c & 15)];
                        if (mask) mask[wi] = 1;
                    }
            }
    }
    return CADNN_OK;
}

void cadnn_weights_free(cadnn_weights *w)
{
    if (!w) return;
    if (w->half) cadnn_weights_free(w->half);
    if (w->d_blob) cudaFree(w->d_blob);
    if (w->d_tc_blob) cudaFree(w->d_tc_blob);
    delete w;
}

}  // extern "C"
