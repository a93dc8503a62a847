// Offline weight packer and per-layer schedule (host code).
//
// Restates, for one large GPU, the offline stage of CADNN (arXiv 1905.00571,
// Section 4): "Memory layout transformation" - the pruned filters are stored in a
// compressed layout whose element offsets already point into the shared-memory
// activation tile the kernel stages, padded so that a warp's loads never collide
// on a bank - and "Optimization parameters selection" - tile sizes, the channel
// chunk and the number of filters per warp are chosen per layer from its shape.
// Filters are regrouped so that the warps of a block get equal nonzero counts
// (the load-balance obstacle Section 1 names).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <numeric>
#include "cadnn_internal.h"

namespace {

const int kSmCount = 148;
const int kTileSmemBudget = 72 * 1024;   // activation tile bytes per block (two blocks per SM)
const int kWeightSmemBudget = 40 * 1024; // staged nonzeros per (block, chunk)

int round_up(int v, int m) { return (v + m - 1) / m * m; }
int ceil_div(int a, int b) { return (a + b - 1) / b; }

int pick_T(int npix)
{
    static const int allowed[] = {1, 2, 4, 7, 8};
    int need = ceil_div(npix, 32);
    for (int t : allowed)
        if (t >= need) return t;
    return 8;
}

// Row pitch (in pixels) of the staged input tile: at least `need`, and congruent
// to TW modulo 32 so that lanes walking consecutive output pixels across a row
// boundary still touch 32 distinct banks.
int pick_pitch(int need, int TW)
{
    int p = need;
    while (((p - TW) % 32) != 0) ++p;
    return p;
}

struct Geometry {
    int c_in, c_out, kh, kw, stride, pad, h, w, h_out, w_out;
};

void choose_spatial(const Geometry &g, int batch_hint, Schedule &s)
{
    s.kind = KK_SCONV_SPATIAL;
    s.TW = g.w_out <= 256 ? g.w_out : 128;
    int th_max = std::max(1, 256 / s.TW);
    th_max = std::min(th_max, g.h_out);
    int tiles_y = ceil_div(g.h_out, th_max);
    s.TH = ceil_div(g.h_out, tiles_y);
    s.T = pick_T(s.TH * s.TW);
    s.IH_t = (s.TH - 1) * g.stride + g.kh;
    s.IW_t = (s.TW - 1) * g.stride + g.kw;
    s.pitch = pick_pitch(s.IW_t, s.TW);
    long tiles = (long)batch_hint * tiles_y * ceil_div(g.w_out, s.TW);
    s.RPW = 1;
    for (int rpw : {4, 2}) {
        if (tiles * ceil_div(g.c_out, kWarpsPerBlock * rpw) >= 2L * kSmCount) {
            s.RPW = rpw;
            break;
        }
    }
    s.G = kWarpsPerBlock * s.RPW;
    int cic = 64;
    while (cic > 4 && cic / 2 >= g.c_in) cic /= 2;          // do not stage far more channels than exist
    if (g.c_in < 4) cic = g.c_in;
    for (;;) {
        s.CIc = cic;
        s.PP = cic | 1;
        long words = (long)s.IH_t * s.pitch * s.PP;
        if ((words * 4 <= kTileSmemBudget && words <= 65535) || cic <= 1) break;
        cic = cic > 4 ? cic / 2 : cic - 1;
    }
    s.tile_words = s.IH_t * s.pitch * s.PP;
}

void choose_linear(const Geometry &g, int batch_hint, Schedule &s)
{
    s.kind = KK_SCONV_LINEAR;
    long P = (long)batch_hint * g.h_out * g.w_out;
    s.RPW = 1;
    s.T = 1;
    bool done = false;
    for (int rpw : {4, 2, 1}) {
        for (int t : {8, 4, 2, 1}) {
            long ctas = ((P + 32 * t - 1) / (32 * t)) * ceil_div(g.c_out, kWarpsPerBlock * rpw);
            if (ctas >= 2L * kSmCount || (rpw == 1 && t == 1)) {
                s.RPW = rpw;
                s.T = t;
                done = true;
                break;
            }
        }
        if (done) break;
    }
    // never give a lane more pixels than the layer has
    while (s.T > 1 && 32L * (s.T / 2) >= P) s.T /= 2;
    s.G = kWarpsPerBlock * s.RPW;
    int cic = 64;
    while (cic > 4 && cic / 2 >= g.c_in) cic /= 2;
    if (g.c_in < 4) cic = g.c_in;
    s.CIc = cic;
    s.PP = cic | 1;
    s.TH = 1;
    s.TW = 32 * s.T;
    s.pitch = s.IH_t = s.IW_t = 0;
    s.tile_words = 32 * s.T * s.PP;
}

void finish_smem(Schedule &s)
{
    s.tile_words = round_up(s.tile_words, 4);
    int work = s.tile_words * 4 + s.max_entries * 8 + round_up((s.G + 1) * 4, 16);
    int out = 32 * s.T * (s.G + 1) * 4;
    s.smem_bytes = std::max(work, out);
}

struct Entry {
    uint16_t off;
    float v;
    int8_t q;
};

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
    size_t b_dense = h->dense_f.size() * 4;
    size_t o_vals = 0, o_offs = o_vals + al(b_vals), o_ptr = o_offs + al(b_offs), o_perm = o_ptr + al(b_ptr);
    size_t o_dense = o_perm + al(b_perm), total = o_dense + al(b_dense);
    h->packed_bytes = (int64_t)(b_vals + b_offs + b_ptr + b_perm + b_dense);
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

cadnn_status pack_sconv(cadnn_weights *h, const Src &src)
{
    const cadnn_layer_desc &d = h->desc;
    Geometry g{d.c_in, d.c_out, d.kh, d.kw, d.stride, d.pad, d.in_h, d.in_w, h->h_out, h->w_out};
    Schedule &s = h->s;
    const bool linear = (d.kh == 1 && d.kw == 1 && d.pad == 0);
    const int K = d.kh * d.kw * d.c_in;
    int bh = std::max(1, d.batch_hint);
    if (linear) choose_linear(g, bh, s); else choose_spatial(g, bh, s);

    // per-filter nonzero counts, then the balanced regrouping
    std::vector<int64_t> row_nnz(d.c_out, 0);
    for (int co = 0; co < d.c_out; ++co) {
        int64_t c = 0;
        for (int k = 0; k < K; ++k) c += src.kept((size_t)co * K + k);
        row_nnz[co] = c;
        h->nnz += c;
    }
    for (int attempt = 0;; ++attempt) {
        s.n_groups = ceil_div(d.c_out, s.G);
        h->c_pad = s.n_groups * s.G;
        s.n_chunks = ceil_div(d.c_in, s.CIc);
        h->perm.assign(h->c_pad, -1);
        for (int gi = 0; gi < s.n_groups; ++gi) {
            int lo = gi * s.G, hi = std::min(d.c_out, lo + s.G);
            std::vector<int64_t> load(row_nnz.begin() + lo, row_nnz.begin() + hi);
            std::vector<int> slot;
            balance_block(load, s.G, s.RPW, slot);
            for (int sl = 0; sl < s.G; ++sl)
                if (slot[sl] >= 0) h->perm[lo + sl] = lo + slot[sl];
        }
        // entries, chunk-major then packed-row-major
        h->ptr.assign((size_t)s.n_chunks * (h->c_pad + 1), 0);
        h->vals_f.clear();
        h->vals_q.clear();
        h->offs.clear();
        h->vals_f.reserve(src.s8 ? 0 : (size_t)h->nnz);
        h->vals_q.reserve(src.s8 ? (size_t)h->nnz : 0);
        h->offs.reserve((size_t)h->nnz);
        s.max_entries = 0;
        int32_t running = 0;
        for (int c = 0; c < s.n_chunks; ++c) {
            int c0 = c * s.CIc, c1 = std::min(d.c_in, c0 + s.CIc);
            int32_t *pp = &h->ptr[(size_t)c * (h->c_pad + 1)];
            for (int r = 0; r < h->c_pad; ++r) {
                pp[r] = running;
                int co = h->perm[r];
                if (co >= 0) {
                    for (int ky = 0; ky < d.kh; ++ky)
                        for (int kx = 0; kx < d.kw; ++kx)
                            for (int ci = c0; ci < c1; ++ci) {
                                size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + ci;
                                if (!src.kept(wi)) continue;
                                int off = linear ? (ci - c0) : ((ky * s.pitch + kx) * s.PP + (ci - c0));
                                h->offs.push_back((uint16_t)off);
                                if (src.s8) h->vals_q.push_back(src.qval(wi, co));
                                else h->vals_f.push_back(src.fval(wi));
                                ++running;
                            }
                }
                if ((r + 1) % s.G == 0) {
                    int first = pp[r + 1 - s.G];
                    s.max_entries = std::max(s.max_entries, running - first);
                }
            }
            pp[h->c_pad] = running;
        }
        // Dense or nearly dense layers can overflow the staged-weight budget: halve the chunk.
        if (s.max_entries * 8 > kWeightSmemBudget && s.CIc > 1 && attempt < 8) {
            s.CIc = std::max(1, s.CIc / 2);
            s.PP = s.CIc | 1;
            s.tile_words = linear ? 32 * s.T * s.PP : s.IH_t * s.pitch * s.PP;
            continue;
        }
        break;
    }
    s.max_entries = round_up(std::max(s.max_entries, 1), 2);
    finish_smem(s);
    if (s.smem_bytes > 200 * 1024) return CADNN_E_UNSUPPORTED;
    h->fmt = CADNN_FMT_TILED_CSR;
    return CADNN_OK;
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
    h->ptr.assign(h->c_pad + 1, 0);
    int32_t running = 0;
    for (int r = 0; r < h->c_pad; ++r) {
        h->ptr[r] = running;
        int co = h->perm[r];
        if (co < 0) continue;
        for (int k = 0; k < K; ++k) {
            size_t wi = (size_t)co * K + k;
            if (!src.kept(wi)) continue;
            h->offs.push_back((uint16_t)k);
            if (src.s8) h->vals_q.push_back(src.qval(wi, co));
            else h->vals_f.push_back(src.fval(wi));
            ++running;
        }
    }
    h->ptr[h->c_pad] = running;
    h->nnz = running;
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
    for (int co = 0; co < d.c_out; ++co)
        for (int t = 0; t < taps; ++t) {
            size_t wi = (size_t)co * taps + t;
            if (src.kept(wi)) {
                h->dense_f[(size_t)t * d.c_out + co] = src.fval(wi);
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
    const cadnn_layer_desc &d = *desc;
    if (d.c_in < 1 || d.c_out < 1 || d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0 || d.groups < 1 ||
        d.in_h < 1 || d.in_w < 1)
        return CADNN_E_ARG;
    if (d.dtype != CADNN_F32 && d.dtype != CADNN_S8) return CADNN_E_DTYPE;
    if (d.dtype == CADNN_S8 && !src.q && !src.w_scale) return CADNN_E_ARG;
    if (d.dtype == CADNN_F32 && (src.q || src.w_scale)) return CADNN_E_DTYPE;
    if (d.in_h + 2 * d.pad < d.kh || d.in_w + 2 * d.pad < d.kw) return CADNN_E_SHAPE;
    if (d.pad >= d.kh || d.pad >= d.kw) return CADNN_E_UNSUPPORTED;
    const bool depthwise = d.groups > 1 && d.groups == d.c_in && d.c_in == d.c_out;
    if (d.groups != 1 && !depthwise) return CADNN_E_UNSUPPORTED;
    const long K = (long)d.kh * d.kw * d.c_in / d.groups;
    if (d.dtype == CADNN_S8 && (double)K * 127.0 * 127.0 >= 2147483648.0) return CADNN_E_UNSUPPORTED;

    cadnn_weights *h = new (std::nothrow) cadnn_weights();
    if (!h) return CADNN_E_ALLOC;
    h->desc = d;
    h->h_out = (d.in_h + 2 * d.pad - d.kh) / d.stride + 1;
    h->w_out = (d.in_w + 2 * d.pad - d.kw) / d.stride + 1;
    cadnn_status st;
    try {
        const bool is_fc = d.kh == 1 && d.kw == 1 && d.in_h == 1 && d.in_w == 1 && d.pad == 0;
        if (depthwise) st = pack_dense(h, src, KK_DW);
        else if (is_fc && std::max(1, d.batch_hint) <= 8 && d.c_in <= 65536) st = pack_fc_spmv(h, src);
        else st = pack_sconv(h, src);
        if (st == CADNN_OK) st = upload(h);
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

cadnn_status cadnn_weights_schedule(const cadnn_weights *w, int sched[8])
{
    if (!w || !sched) return CADNN_E_ARG;
    const Schedule &s = w->s;
    int v[8] = {s.kind, s.T, s.RPW, s.G, s.CIc, s.TH, s.TW, s.pitch};
    memcpy(sched, v, sizeof(v));
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
            const int32_t *pp = &w->ptr[(size_t)c * (w->c_pad + 1)];
            tot += pp[(i + 1) * s.RPW] - pp[i * s.RPW];
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
                if (mask) mask[co * K + t] = 1;
            }
        return CADNN_OK;
    }
    if (s.kind == KK_FC_SPMV) {
        for (int r = 0; r < w->c_pad; ++r) {
            int co = w->perm[r];
            if (co < 0) continue;
            for (int e = w->ptr[r]; e < w->ptr[r + 1]; ++e) {
                size_t wi = (size_t)co * K + w->offs[e];
                if (dense) dense[wi] = val(e);
                if (mask) mask[wi] = 1;
            }
        }
        return CADNN_OK;
    }
    const bool linear = s.kind == KK_SCONV_LINEAR;
    for (int c = 0; c < s.n_chunks; ++c) {
        const int32_t *pp = &w->ptr[(size_t)c * (w->c_pad + 1)];
        for (int r = 0; r < w->c_pad; ++r) {
            int co = w->perm[r];
            if (co < 0) continue;
            for (int e = pp[r]; e < pp[r + 1]; ++e) {
                int off = w->offs[e];
                int cl = off % s.PP, t = off / s.PP;
                int kx = linear ? 0 : t % s.pitch, ky = linear ? 0 : t / s.pitch;
                size_t wi = (((size_t)co * d.kh + ky) * d.kw + kx) * d.c_in + (size_t)c * s.CIc + cl;
                if (dense) dense[wi] = val(e);
                if (mask) mask[wi] = 1;
            }
        }
    }
    return CADNN_OK;
}

void cadnn_weights_free(cadnn_weights *w)
{
    if (!w) return;
    if (w->d_blob) cudaFree(w->d_blob);
    delete w;
}

}  // extern "C"
