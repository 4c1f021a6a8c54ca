// Host side of the C ABI: validation, handles, table upload, argument checks, kernel dispatch.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "guide_internal.cuh"

namespace guide {

static thread_local std::string g_err;

int fail(int code, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

int cuda_fail(cudaError_t e, const char *what) {
    return fail(GUIDE_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int num_sms() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// ---- 64-bit overflow proof for the integer FLOP / byte counts --------------------------------

typedef unsigned __int128 u128;
static const u128 LIMIT = (u128)1 << 63;   // one bit of margin below wrap-around

struct Maxima { u128 T, E, A, C, R; };

static bool counts_fit(const guide_model &m, uint32_t t_max, const Maxima &x) {
    const u128 H = m.hidden, I = m.ffn, V = m.vocab, nh = m.n_heads, ab = m.a_bytes, wb = m.w_bytes,
               kvb = m.kv_bytes, Dkv = (u128)m.n_kv_heads * (m.hidden / m.n_heads), g = m.gated;
    const u128 T = x.T, E = x.E, A = x.A, C = x.C, R = x.R;
    const u128 big = H > I ? H : I;
    const u128 terms[] = {
        4 * T * big, 3 * T * H * ab, 2 * T * H * big, R * H * big * wb + T * big * ab + T * H * ab,
        2 * T * H * Dkv, R * H * Dkv * wb + T * Dkv * kvb, (2 + g) * T * I * ab,
        2 * H * A, T * H * ab + C * Dkv * kvb + nh * A * ab, 5 * nh * A, 2 * nh * A * ab,
        2 * E * H * V, R * H * V * wb + E * V * ab, E * H * ab,
        R * 2 * t_max, (u128)2 * t_max * T * H * ab,
    };
    for (u128 v : terms)
        if (v >= LIMIT) return false;
    return true;
}

static u128 weight_bytes(const guide_model &m) {
    const u128 H = m.hidden, I = m.ffn, V = m.vocab, Dkv = (u128)m.n_kv_heads * (m.hidden / m.n_heads);
    return ((u128)m.n_layers * (2 * H * H + 2 * H * Dkv + (2 + (u128)m.gated) * H * I) + 2 * V * H) * m.w_bytes;
}

static int check_closed_form_overflow(const guide_space &s) {
    for (size_t mi = 0; mi < s.models.size(); mi++) {
        const guide_model &m = s.models[mi];
        const u128 b = s.max_batch;
        for (const guide_len_pair &p : s.pairs) {
            const u128 lin = p.lin, n = p.lout - 1;
            Maxima pre{b * lin, b, b * lin * lin, b * lin, 1};
            Maxima dec{b * n, b * n, b * (n * lin + n * (n + 1) / 2), b * (n * lin + n * (n + 1) / 2), n};
            if (!counts_fit(m, s.max_tp, pre) || !counts_fit(m, s.max_tp, dec))
                return fail(GUIDE_ERR_OVERFLOW,
                            "model %zu with batch %u and lengths (%u, %u) overflows a 64-bit FLOP/byte count",
                            mi, s.max_batch, p.lin, p.lout);
            if (b * (1 + n) >= LIMIT) return fail(GUIDE_ERR_OVERFLOW, "request-iteration count overflows");
            if (dec.A * 1000 >= LIMIT) return fail(GUIDE_ERR_OVERFLOW, "decode context x 1000 (kept share of the KV cache) overflows");
        }
    }
    return GUIDE_OK;
}

static int check_trace_overflow(const guide_space &s, const guide_trace &t) {
    const u128 q = std::max<uint64_t>(t.max_tokens, t.n_zero ? (uint64_t)s.max_lin + s.max_lout : 0);
    const u128 b = s.max_batch;
    uint32_t max_block = 1;
    for (const guide_fw &f : s.fw) max_block = std::max(max_block, f.kv_block);
    for (const guide_model &m : s.models)
        if ((q + max_block) * (2ull * m.n_layers * m.n_kv_heads * (m.hidden / m.n_heads) * m.kv_bytes) >= LIMIT)
            return fail(GUIDE_ERR_OVERFLOW, "KV bytes of the longest request overflow");
    for (size_t mi = 0; mi < s.models.size(); mi++) {
        Maxima pre{b * q, b, b * q * q, b * q, 1};
        Maxima dec{b, b, b * q, b * q, 1};
        if (!counts_fit(s.models[mi], s.max_tp, pre) || !counts_fit(s.models[mi], s.max_tp, dec))
            return fail(GUIDE_ERR_OVERFLOW, "model %zu overflows a 64-bit FLOP/byte count on this trace", mi);
    }
    return GUIDE_OK;
}

// ---- device tables ------------------------------------------------------------------------------

// Derived per-model quantities and the reciprocal rates of every hardware x framework pair.
__global__ void k_build_tables(const guide_model *gm, u32 n_m, const guide_hw *gh, u32 n_h, const guide_fw *gf,
                               u32 n_f, const u32 *tp, const u32 *dp, u32 n_t, DModel *dm, DRate *dr, double *cost_hr,
                               double *cost_sec, ulonglong2 *hfmem, double *rate10, StageConst *stage_consts, RateF *ratef) {
    const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_m) {
        const guide_model m = gm[i];
        DModel d;
        d.N = m.n_layers; d.H = m.hidden; d.nh = m.n_heads; d.nkv = m.n_kv_heads; d.I = m.ffn; d.V = m.vocab;
        d.g = m.gated; d.wb = m.w_bytes; d.ab = m.a_bytes; d.kvb = m.kv_bytes;
        d.Dkv = m.n_kv_heads * (m.hidden / m.n_heads);
        d.pad = 0;
        const u64 H = d.H, Dkv = d.Dkv, I = d.I, V = d.V;
        const u64 per_layer = 2 * H * H + 2 * H * Dkv + (2 + (u64)d.g) * H * I;
        d.wbytes = ((u64)d.N * per_layer + 2 * V * H) * d.wb;
        d.kv2 = 2 * (u64)d.N * Dkv * d.kvb;
        dm[i] = d;
        for (u32 k = 0; k <= n_t; k++) stage_consts[(size_t)k * n_m + i] = stage_const(d, k < n_t ? tp[k] : 1u);
    }
    if (i < n_h * n_f) {
        const guide_hw h = gh[i / n_f];
        const guide_fw f = gf[i % n_f];
        DRate r;
        for (int k = 0; k < 3; k++) {
            r.inv_c[k] = 1.0 / (h.peak_flops * f.e_c[k]);
            r.inv_m[k] = 1.0 / (h.mem_bw * f.e_m[k]);
        }
        r.inv_comm = 1.0 / (h.comm_bw * f.e_comm);
        r.clat = h.comm_lat;
        r.tovh = f.t_ovh;
        r.price = h.price_per_hr;
        r.usable = h.mem_bytes - (h.mem_bytes / 1000) * f.reserve_permille;
        r.flash = f.flash;
        r.kv_block = f.kv_block;
        r.split = f.split_size;
        r.seg = f.seg_tokens;
        r.policy = f.policy;
        r.keep = (f.kv_keep_permille == 0 || f.kv_keep_permille >= 1000) ? 1000u : f.kv_keep_permille;
        dr[i] = r;
        hfmem[i] = make_ulonglong2(r.usable, (u64)r.kv_block);
        RateF rf;
        for (int k = 0; k < 3; k++) {
            rf.inv_c[k] = 1.0f / ((float)h.peak_flops * (float)f.e_c[k]);
            rf.inv_m[k] = 1.0f / ((float)h.mem_bw * (float)f.e_m[k]);
        }
        rf.inv_comm = 1.0f / ((float)h.comm_bw * (float)f.e_comm);
        rf.clat = (float)h.comm_lat; rf.tovh = (float)f.t_ovh; rf.price = (float)h.price_per_hr;
        rf.flash = f.flash; rf.pad = 0;
        ratef[i] = rf;
        double *q = rate10 + (size_t)i * 10;
        for (int k = 0; k < 3; k++) { q[k] = r.inv_c[k]; q[3 + k] = r.inv_m[k]; }
        q[6] = r.inv_comm; q[7] = r.clat; q[8] = r.tovh; q[9] = r.flash ? 1.0 : 0.0;
        for (u32 k = 0; k < n_t; k++) {
            const double c = h.price_per_hr * (double)((u64)tp[k] * dp[k]);      // every GPU of every replica
            cost_hr[i * n_t + k] = c;
            cost_sec[i * n_t + k] = c / 3600.0;
        }
    }
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Work orders for the closed-form model kernel.  They decide which thread evaluates what, never a
// value: any permutation gives the same outputs.
//
// The pairs, grouped by KV block size and, inside a group, by falling usable memory (the formula
// of k_build_tables): the pairs a config fits are then a prefix of each group.
static std::vector<HfSorted> sorted_pairs(const guide_space &s) {
    const size_t n_f = s.fw.size(), n = s.hw.size() * n_f;
    std::vector<HfSorted> v(n);
    for (size_t i = 0; i < n; i++) {
        const guide_hw &h = s.hw[i / n_f];
        const guide_fw &f = s.fw[i % n_f];
        v[i].usable = h.mem_bytes - (h.mem_bytes / 1000) * f.reserve_permille;
        v[i].block = f.kv_block;
        v[i].hf = (u32)i;
        v[i].seg_end = 0; v[i].pad = 0;
    }
    std::stable_sort(v.begin(), v.end(), [](const HfSorted &a, const HfSorted &b) {
        return a.block != b.block ? a.block < b.block : a.usable > b.usable;
    });
    for (size_t i = n; i-- > 0;) v[i].seg_end = (i + 1 < n && v[i + 1].block == v[i].block) ? v[i + 1].seg_end : (u32)(i + 1);
    return v;
}

// Per model, the groups of `group` consecutive positions of the (TP, length) plane (foursomes: one
// memory sector of every metric array; lines of sixteen: 128 bytes) by growing memory need of
// their cheapest position (weights per GPU plus the KV cache of a middle batch size); groups whose
// TP degree does not divide the heads last.  Heavy work items then come first and lanes of a warp
// fit about the same number of pairs.  When the plane does not divide into such groups the table
// is not used.
static std::vector<u32> plane_orders(const guide_space &s, size_t group) {
    const size_t n_t = s.tp.size(), n_l = s.pairs.size(), n_tl = n_t * n_l, n_four = n_tl / group;
    std::vector<u32> out(s.models.size() * std::max<size_t>(n_four, 1), 0);
    if (n_l % group != 0) return out;
    const double b_ref = (double)s.batch[s.batch.size() / 2];
    const double blk = (double)std::max<u32>(s.fw[0].kv_block, 1);
    std::vector<double> key(n_four);
    for (size_t mi = 0; mi < s.models.size(); mi++) {
        const guide_model &m = s.models[mi];
        const double H = m.hidden, Dkv = (double)m.n_kv_heads * (m.hidden / m.n_heads), I = m.ffn, V = m.vocab;
        const double wbytes = (m.n_layers * (2 * H * H + 2 * H * Dkv + (2.0 + m.gated) * H * I) + 2 * V * H) * m.w_bytes;
        const double kv2 = 2.0 * m.n_layers * Dkv * m.kv_bytes;
        for (size_t q = 0; q < n_four; q++) {
            const u32 t = s.tp[(group * q) / n_l];
            const double b_rep = std::ceil(b_ref / (double)s.dp[(group * q) / n_l]);   // one replica's share
            const bool bad = (m.n_heads % t) != 0 || (m.n_kv_heads % t) != 0;
            double best = INFINITY;
            for (size_t u = 0; u < group && !bad; u++) {
                const guide_len_pair &pr = s.pairs[(group * q + u) % n_l];
                const double S = std::ceil(((double)pr.lin + pr.lout) / blk) * blk;
                best = std::min(best, wbytes / t + b_rep * S * (kv2 / t));
            }
            key[q] = best;
        }
        u32 *o = out.data() + mi * n_four;
        for (size_t q = 0; q < n_four; q++) o[q] = (u32)q;
        std::stable_sort(o, o + n_four, [&](u32 a, u32 b) { return key[a] < key[b]; });
    }
    return out;
}

// One work-counter slot per stream that has used the handle on this device: calls on one stream are
// ordered, so they can share a slot; calls on different streams never do.  When more streams than
// slots turn up, everything in flight on the device is waited for and the slots are handed out anew.
static int ticket_for(DeviceTables &d, cudaStream_t st, unsigned **ticket) {
    for (size_t i = 0; i < d.ticket_streams.size(); i++)
        if (d.ticket_streams[i] == (void *)st) { *ticket = d.tickets + 32 * i; return GUIDE_OK; }
    if (d.ticket_streams.size() == TICKET_SLOTS) {
        GUIDE_CUDA(cudaDeviceSynchronize());
        d.ticket_streams.clear();
    }
    d.ticket_streams.push_back((void *)st);
    *ticket = d.tickets + 32 * (d.ticket_streams.size() - 1);
    return GUIDE_OK;
}

int space_on_device(guide_space *s, DSpace *out, unsigned **ticket, cudaStream_t st) {
    int dev = 0;
    GUIDE_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(s->mu);
    for (DeviceTables &d : s->dev)
        if (d.device == dev) {
            *out = d.view;
            return ticket ? ticket_for(d, st, ticket) : GUIDE_OK;
        }

    const size_t n_m = s->models.size(), n_h = s->hw.size(), n_f = s->fw.size();
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t o_gm = take(n_m * sizeof(guide_model)), o_gh = take(n_h * sizeof(guide_hw)),
                 o_gf = take(n_f * sizeof(guide_fw)), o_dm = take(n_m * sizeof(DModel)),
                 o_dr = take(n_h * n_f * sizeof(DRate)), o_b = take(s->batch.size() * 4),
                 o_t = take(s->tp.size() * 4), o_d = take(s->tp.size() * 4), o_p = take(s->pairs.size() * 8),
                 o_ch = take(n_h * n_f * s->tp.size() * 8), o_cs = take(n_h * n_f * s->tp.size() * 8),
                 o_hm = take(n_h * n_f * 16), o_hs = take(n_h * n_f * sizeof(HfSorted)),
                 o_po = take(std::max<size_t>(n_m * (s->tp.size() * s->pairs.size() / 4), 1) * 4),
                 o_lo = take(std::max<size_t>(n_m * (s->tp.size() * s->pairs.size() / 16), 1) * 4),
                 o_tk = take(TICKET_SLOTS * 128), o_r10 = take(n_h * n_f * 80),
                 o_sc = take((s->tp.size() + 1) * n_m * sizeof(StageConst)), o_rf = take(n_h * n_f * sizeof(RateF));
    char *blob = nullptr;
    GUIDE_CUDA(cudaMalloc(&blob, off));
    cudaError_t e = cudaSuccess;
    auto put = [&](size_t o, const void *src, size_t bytes) {
        if (e == cudaSuccess) e = cudaMemcpyAsync(blob + o, src, bytes, cudaMemcpyHostToDevice, st);
    };
    put(o_gm, s->models.data(), n_m * sizeof(guide_model));
    put(o_gh, s->hw.data(), n_h * sizeof(guide_hw));
    put(o_gf, s->fw.data(), n_f * sizeof(guide_fw));
    put(o_b, s->batch.data(), s->batch.size() * 4);
    put(o_t, s->tp.data(), s->tp.size() * 4);
    put(o_d, s->dp.data(), s->dp.size() * 4);
    put(o_p, s->pairs.data(), s->pairs.size() * 8);
    const std::vector<HfSorted> hf_sorted = sorted_pairs(*s);
    const std::vector<u32> plane_order = plane_orders(*s, 4), line_order = plane_orders(*s, 16);
    put(o_hs, hf_sorted.data(), hf_sorted.size() * sizeof(HfSorted));
    put(o_po, plane_order.data(), plane_order.size() * 4);
    put(o_lo, line_order.data(), line_order.size() * 4);
    if (e == cudaSuccess) {
        const u32 n = (u32)std::max(n_m, n_h * n_f);
        k_build_tables<<<(n + 127) / 128, 128, 0, st>>>((const guide_model *)(blob + o_gm), (u32)n_m,
                                                 (const guide_hw *)(blob + o_gh), (u32)n_h,
                                                 (const guide_fw *)(blob + o_gf), (u32)n_f,
                                                 (const u32 *)(blob + o_t), (const u32 *)(blob + o_d), (u32)s->tp.size(),
                                                 (DModel *)(blob + o_dm), (DRate *)(blob + o_dr),
                                                 (double *)(blob + o_ch), (double *)(blob + o_cs),
                                                 (ulonglong2 *)(blob + o_hm), (double *)(blob + o_r10),
                                                 (StageConst *)(blob + o_sc), (RateF *)(blob + o_rf));
        e = cudaGetLastError();
        // the host arrays must outlive the copies, and another stream may use the tables next
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    }
    if (e != cudaSuccess) { cudaFree(blob); return cuda_fail(e, "uploading the space tables"); }
    DeviceTables d;
    d.device = dev;
    d.blob = blob;
    d.view.models = (const DModel *)(blob + o_dm);
    d.view.rates = (const DRate *)(blob + o_dr);
    d.view.batch = (const u32 *)(blob + o_b);
    d.view.tp = (const u32 *)(blob + o_t);
    d.view.dp = (const u32 *)(blob + o_d);
    d.view.chunked = s->chunked ? 1u : 0u;
    d.view.clamp_seq = 0;
    d.view.pairs = (const uint2 *)(blob + o_p);
    d.view.cost_hr = (const double *)(blob + o_ch);
    d.view.cost_sec = (const double *)(blob + o_cs);
    d.view.hfmem = (const ulonglong2 *)(blob + o_hm);
    d.view.rate10 = (const double *)(blob + o_r10);
    d.view.stage_consts = (const StageConst *)(blob + o_sc);
    d.view.ratef = (const RateF *)(blob + o_rf);
    d.view.hf_sorted = (const HfSorted *)(blob + o_hs);
    d.view.plane_order = (const u32 *)(blob + o_po);
    d.view.line_order = (const u32 *)(blob + o_lo);
    d.view.n_m = (u32)n_m; d.view.n_h = (u32)n_h; d.view.n_f = (u32)n_f;
    d.view.n_b = (u32)s->batch.size(); d.view.n_t = (u32)s->tp.size(); d.view.n_l = (u32)s->pairs.size();
    d.tickets = (unsigned *)(blob + o_tk);
    s->dev.push_back(d);
    *out = d.view;
    return ticket ? ticket_for(s->dev.back(), st, ticket) : GUIDE_OK;
}

int trace_on_device(guide_trace *t, DTrace *out, cudaStream_t st) {
    int dev = 0;
    GUIDE_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(t->mu);
    for (const DeviceTrace &d : t->dev)
        if (d.device == dev) { *out = d.view; return GUIDE_OK; }
    const size_t n = t->arrival.size();
    const size_t o_a = 0, o_i = align_up(n * 8, 256), o_o = o_i + align_up(n * 4, 256), total = o_o + align_up(n * 4, 256);
    char *blob = nullptr;
    GUIDE_CUDA(cudaMalloc(&blob, total));
    cudaError_t e = cudaMemcpyAsync(blob + o_a, t->arrival.data(), n * 8, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(blob + o_i, t->in_len.data(), n * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(blob + o_o, t->out_len.data(), n * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);      // the copies are done before another stream can use the trace
    if (e != cudaSuccess) { cudaFree(blob); return cuda_fail(e, "uploading the trace"); }
    DeviceTrace d;
    d.device = dev;
    d.blob = blob;
    d.view.arrival = (const double *)(blob + o_a);
    d.view.in_len = (const u32 *)(blob + o_i);
    d.view.out_len = (const u32 *)(blob + o_o);
    d.view.n = (u32)n;
    d.view.max_tokens = t->max_tokens;
    d.view.any_zero = t->n_zero ? 1 : 0;
    d.view.sum_out = t->sum_out;
    d.view.sum_in = t->sum_in;
    d.view.n_zero = t->n_zero;
    t->dev.push_back(d);
    *out = d.view;
    return GUIDE_OK;
}

static bool pow2(uint32_t v) { return v && !(v & (v - 1)); }

static int resolve_range(const guide_space *s, const guide_sim_opts *o, Range *r) {
    r->first = o ? o->first : 0;
    r->count = o ? o->count : 0;
    if (r->first > s->size) return fail(GUIDE_ERR_INVALID, "first (%llu) is past the end of the space", (unsigned long long)r->first);
    if (r->count == 0) r->count = s->size - r->first;
    if (r->count > s->size - r->first) return fail(GUIDE_ERR_INVALID, "range runs past the end of the space");
    if (o && (o->time_model < 0 || o->time_model > 1 || o->tp_model < 0 || o->tp_model > 1))
        return fail(GUIDE_ERR_INVALID, "unknown time_model or tp_model");
    if (o && (o->clamp_seq < 0 || o->clamp_seq > 1)) return fail(GUIDE_ERR_INVALID, "clamp_seq must be 0 or 1");
    if (o && o->precision != GUIDE_PREC_F64 && o->precision != GUIDE_PREC_F32) return fail(GUIDE_ERR_INVALID, "unknown precision");
    return GUIDE_OK;
}

static int check_workspace(const void *ws, size_t have, size_t need) {
    if (need == 0) return GUIDE_OK;
    if (!ws) return fail(GUIDE_ERR_WORKSPACE, "workspace is NULL, %zu bytes needed", need);
    if ((uintptr_t)ws % 256) return fail(GUIDE_ERR_WORKSPACE, "workspace must be 256-byte aligned");
    if (have < need) return fail(GUIDE_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", have, need);
    return GUIDE_OK;
}

static const double *metric_array(const guide_outputs &o, int key) {
    switch (key) {
    case GUIDE_LATENCY: return o.latency;
    case GUIDE_TTFT: return o.ttft;
    case GUIDE_TTFT_P99: return o.ttft_p99;
    case GUIDE_TPOT: return o.tpot;
    case GUIDE_THROUGHPUT: return o.thr_decode;
    case GUIDE_COST_PER_HR: return o.cost_per_hr;
    case GUIDE_COST_PER_TOKEN: return o.cost_per_token;
    }
    return nullptr;
}

static int check_selection_args(const guide_space *space, const guide_trace *trace, const guide_outputs *outputs,
                                const guide_constraints *cons, const int *keys, int n_keys) {
    if (!space || !cons) return fail(GUIDE_ERR_INVALID, "space and constraints are required");
    for (int i = 0; i < n_keys; i++)
        if (keys[i] < GUIDE_LATENCY || keys[i] > GUIDE_COST_PER_TOKEN) return fail(GUIDE_ERR_INVALID, "unknown metric %d", keys[i]);
    if (cons->ttft_stat < GUIDE_STAT_MEAN || cons->ttft_stat > GUIDE_STAT_P99) return fail(GUIDE_ERR_INVALID, "unknown ttft_stat");
    if (std::isnan(cons->max_ttft) || std::isnan(cons->max_latency) || std::isnan(cons->max_cost_per_hr) ||
        std::isnan(cons->min_throughput))
        return fail(GUIDE_ERR_INVALID, "a constraint is NaN");
    if (!outputs) {
        if (trace) return fail(GUIDE_ERR_UNSUPPORTED, "fused selection evaluates the closed form only: run guide_simulate on the trace and pass its outputs");
        return GUIDE_OK;
    }
    if (!outputs->status) return fail(GUIDE_ERR_INVALID, "materialised selection needs outputs->status");
    for (int i = 0; i < n_keys; i++)
        if (!metric_array(*outputs, keys[i])) return fail(GUIDE_ERR_INVALID, "the array of metric %d is NULL", keys[i]);
    const double *ttft = cons->ttft_stat == GUIDE_STAT_MEAN ? outputs->ttft
                         : cons->ttft_stat == GUIDE_STAT_P50 ? outputs->ttft_p50 : outputs->ttft_p99;
    if (cons->max_ttft < INFINITY && !ttft) return fail(GUIDE_ERR_INVALID, "max_ttft is set but its array is NULL");
    if (cons->max_latency < INFINITY && !outputs->latency) return fail(GUIDE_ERR_INVALID, "max_latency is set but latency is NULL");
    if (cons->max_cost_per_hr < INFINITY && !outputs->cost_per_hr) return fail(GUIDE_ERR_INVALID, "max_cost_per_hr is set but cost_per_hr is NULL");
    if (cons->min_throughput > 0.0 && !outputs->thr_decode) return fail(GUIDE_ERR_INVALID, "min_throughput is set but thr_decode is NULL");
    return GUIDE_OK;
}

}  // namespace guide

using namespace guide;

extern "C" {

const char *guide_last_error(void) { return g_err.c_str(); }

int guide_space_create(const guide_space_desc *d, guide_space **out) {
    if (!d || !out) return fail(GUIDE_ERR_INVALID, "desc and out are required");
    *out = nullptr;
    if (!d->models || !d->hw || !d->fw || !d->batch || !d->tp || !d->pairs)
        return fail(GUIDE_ERR_INVALID, "an axis pointer is NULL");
    if (!d->n_models || !d->n_hw || !d->n_fw || !d->n_batch || !d->n_tp || !d->n_pairs)
        return fail(GUIDE_ERR_INVALID, "an axis is empty");
    if (d->n_models > 4096 || (uint64_t)d->n_hw * d->n_fw > 65536)
        return fail(GUIDE_ERR_INVALID, "too many models (max 4096) or hardware x framework pairs (max 65536)");
    guide_space *s = new (std::nothrow) guide_space;
    if (!s) return fail(GUIDE_ERR_INVALID, "out of host memory");
    s->models.assign(d->models, d->models + d->n_models);
    s->hw.assign(d->hw, d->hw + d->n_hw);
    s->fw.assign(d->fw, d->fw + d->n_fw);
    s->batch.assign(d->batch, d->batch + d->n_batch);
    s->tp.assign(d->tp, d->tp + d->n_tp);
    if (d->dp) s->dp.assign(d->dp, d->dp + d->n_tp); else s->dp.assign(d->n_tp, 1u);
    s->pairs.assign(d->pairs, d->pairs + d->n_pairs);
    int rc = GUIDE_OK;
    for (uint32_t v : s->dp) {
        if (!v || v > 65536) { rc = fail(GUIDE_ERR_INVALID, "data-parallel degree %u is outside 1..65536", v); break; }
        s->max_dp = std::max(s->max_dp, v);
    }
    for (uint32_t v : s->tp) {
        if (!pow2(v) || v > 1024) { rc = fail(GUIDE_ERR_UNSUPPORTED, "TP degree %u is not a power of two in 1..1024", v); break; }
        s->max_tp = std::max(s->max_tp, v);
    }
    for (uint32_t v : s->batch) {
        if (rc) break;
        if (!v) rc = fail(GUIDE_ERR_INVALID, "batch size 0");
        s->max_batch = std::max(s->max_batch, v);
    }
    for (const guide_len_pair &p : s->pairs) {
        if (rc) break;
        if (!p.lin || !p.lout) rc = fail(GUIDE_ERR_INVALID, "a length pair has a zero length");
        s->max_lin = std::max(s->max_lin, p.lin);
        s->max_lout = std::max(s->max_lout, p.lout);
    }
    for (size_t i = 0; i < s->models.size() && !rc; i++) {
        const guide_model &m = s->models[i];
        if (!m.n_layers || !m.hidden || !m.n_heads || !m.n_kv_heads || !m.ffn || !m.vocab || !m.w_bytes ||
            !m.a_bytes || !m.kv_bytes || m.gated > 1)
            rc = fail(GUIDE_ERR_INVALID, "model %zu has a zero size or gated > 1", i);
        else if (m.hidden % m.n_heads)
            rc = fail(GUIDE_ERR_INVALID, "model %zu: hidden is not a multiple of n_heads", i);
        else if (2ull * m.n_layers * m.n_kv_heads * (m.hidden / m.n_heads) * m.kv_bytes < s->max_tp)
            rc = fail(GUIDE_ERR_INVALID, "model %zu: KV bytes per token per GPU would round to zero", i);
        else if (weight_bytes(m) >= LIMIT)
            rc = fail(GUIDE_ERR_OVERFLOW, "model %zu: weight bytes overflow", i);
    }
    for (size_t i = 0; i < s->hw.size() && !rc; i++) {
        const guide_hw &h = s->hw[i];
        if (!(h.peak_flops > 0) || !(h.mem_bw > 0) || !(h.comm_bw > 0) || !(h.comm_lat >= 0) ||
            !(h.price_per_hr >= 0) || !std::isfinite(h.peak_flops + h.mem_bw + h.comm_bw + h.comm_lat + h.price_per_hr))
            rc = fail(GUIDE_ERR_INVALID, "hardware profile %zu has a non-positive or non-finite rate", i);
    }
    for (size_t i = 0; i < s->fw.size() && !rc; i++) {
        const guide_fw &f = s->fw[i];
        bool ok = f.kv_block >= 1 && f.reserve_permille <= 1000 && f.flash <= 1 && f.e_comm > 0 && f.t_ovh >= 0 &&
                  std::isfinite(f.e_comm + f.t_ovh);
        for (int k = 0; k < 3; k++) ok = ok && f.e_c[k] > 0 && f.e_m[k] > 0 && std::isfinite(f.e_c[k] + f.e_m[k]);
        if (!ok) rc = fail(GUIDE_ERR_INVALID, "framework profile %zu has a bad efficiency, kv_block or reserve", i);
        else if (f.policy != GUIDE_POLICY_PREFILL_FIRST && f.policy != GUIDE_POLICY_SPLIT_FUSE)
            rc = fail(GUIDE_ERR_UNSUPPORTED, "framework profile %zu: unknown policy", i);
        else if (f.kv_keep_permille > 1000)
            rc = fail(GUIDE_ERR_INVALID, "framework profile %zu: kv_keep_permille above 1000", i);
        s->evicting = s->evicting || (f.kv_keep_permille != 0 && f.kv_keep_permille != 1000);
        s->chunked = s->chunked || f.split_size || f.seg_tokens || (f.kv_keep_permille != 0 && f.kv_keep_permille != 1000);
    }
    if (!rc) {
        u128 n = (u128)d->n_models * d->n_hw * d->n_fw * d->n_batch * d->n_tp * d->n_pairs;
        if (n >= ((u128)1 << 48)) rc = fail(GUIDE_ERR_OVERFLOW, "the space has 2^48 configs or more");
        s->size = (uint64_t)n;
    }
    if (!rc) {
        // capacity arithmetic: (lin+lout rounded up to whole blocks) x KV bytes per token
        uint32_t max_block = 1;
        for (const guide_fw &f : s->fw) max_block = std::max(max_block, f.kv_block);
        u128 worst = (u128)s->max_lin + s->max_lout + max_block;
        for (const guide_model &m : s->models)
            if (worst * (2ull * m.n_layers * m.n_kv_heads * (m.hidden / m.n_heads) * m.kv_bytes) >= LIMIT)
                rc = fail(GUIDE_ERR_OVERFLOW, "KV bytes of one request overflow");
    }
    if (!rc) rc = check_closed_form_overflow(*s);
    if (rc) { delete s; return rc; }
    *out = s;
    return GUIDE_OK;
}

void guide_space_destroy(guide_space *s) {
    if (!s) return;
    int cur = 0;
    const bool have = cudaGetDevice(&cur) == cudaSuccess;
    for (DeviceTables &d : s->dev) {
        if (have && cudaSetDevice(d.device) == cudaSuccess) cudaFree(d.blob);
    }
    if (have && !s->dev.empty()) cudaSetDevice(cur);
    delete s;
}

uint64_t guide_space_size(const guide_space *s) { return s ? s->size : 0; }

int guide_space_decode(const guide_space *s, uint64_t idx, guide_config *o) {
    if (!s || !o) return fail(GUIDE_ERR_INVALID, "space and out are required");
    if (idx >= s->size) return fail(GUIDE_ERR_INVALID, "index %llu is outside the space", (unsigned long long)idx);
    o->pair_pos = (uint32_t)(idx % s->pairs.size()); idx /= s->pairs.size();
    o->tp_pos = (uint32_t)(idx % s->tp.size()); idx /= s->tp.size();
    o->batch_pos = (uint32_t)(idx % s->batch.size()); idx /= s->batch.size();
    o->fw = (uint32_t)(idx % s->fw.size()); idx /= s->fw.size();
    o->hw = (uint32_t)(idx % s->hw.size()); idx /= s->hw.size();
    o->model = (uint32_t)idx;
    o->batch = s->batch[o->batch_pos];
    o->dp = s->dp[o->tp_pos];
    o->tp = s->tp[o->tp_pos];
    o->lin = s->pairs[o->pair_pos].lin;
    o->lout = s->pairs[o->pair_pos].lout;
    return GUIDE_OK;
}

int guide_trace_load(const double *arrival, const uint32_t *in_len, const uint32_t *out_len, uint64_t n,
                     guide_trace **out) {
    if (!out) return fail(GUIDE_ERR_INVALID, "out is required");
    *out = nullptr;
    if (!arrival || !in_len || !out_len) return fail(GUIDE_ERR_INVALID, "a trace array is NULL");
    if (n == 0 || n > 65536) return fail(GUIDE_ERR_INVALID, "n_req must be in 1..65536");
    guide_trace *t = new (std::nothrow) guide_trace;
    if (!t) return fail(GUIDE_ERR_INVALID, "out of host memory");
    t->arrival.assign(arrival, arrival + n);
    t->in_len.assign(in_len, in_len + n);
    t->out_len.assign(out_len, out_len + n);
    int rc = GUIDE_OK;
    for (uint64_t i = 0; i < n && !rc; i++) {
        if (!(arrival[i] >= 0) || !std::isfinite(arrival[i])) rc = fail(GUIDE_ERR_INVALID, "arrival[%llu] is negative or not finite", (unsigned long long)i);
        else if (i && arrival[i] < arrival[i - 1]) rc = fail(GUIDE_ERR_INVALID, "arrivals must be non-decreasing (entry %llu)", (unsigned long long)i);
        else if (in_len[i] && !out_len[i]) rc = fail(GUIDE_ERR_INVALID, "request %llu has an input length but no output length", (unsigned long long)i);
        else if (in_len[i] > (1u << 24) || out_len[i] > (1u << 24)) rc = fail(GUIDE_ERR_INVALID, "request %llu is longer than 2^24 tokens", (unsigned long long)i);
        if (in_len[i]) {
            t->max_in = std::max(t->max_in, in_len[i]);
            t->max_out = std::max(t->max_out, out_len[i]);
            t->max_tokens = std::max(t->max_tokens, in_len[i] + out_len[i]);
            t->sum_out += out_len[i];
            t->sum_in += in_len[i];
        } else t->n_zero++;
    }
    if (rc) { delete t; return rc; }
    *out = t;
    return GUIDE_OK;
}

void guide_trace_destroy(guide_trace *t) {
    if (!t) return;
    int cur = 0;
    const bool have = cudaGetDevice(&cur) == cudaSuccess;
    for (DeviceTrace &d : t->dev)
        if (have && cudaSetDevice(d.device) == cudaSuccess) cudaFree(d.blob);
    if (have && !t->dev.empty()) cudaSetDevice(cur);
    delete t;
}

uint64_t guide_trace_size(const guide_trace *t) { return t ? t->arrival.size() : 0; }

size_t guide_workspace_bytes(const guide_space *space, const guide_trace *trace, const guide_sim_opts *) {
    if (!space || !trace) return 0;
    return trace_workspace_bytes((u32)trace->arrival.size(), lane_hints(*space));
}

int guide_simulate(const guide_space *space_c, const guide_trace *trace_c, const guide_sim_opts *opts,
                   const guide_outputs *out, void *ws, size_t ws_bytes, void *stream) {
    guide_space *space = const_cast<guide_space *>(space_c);
    guide_trace *trace = const_cast<guide_trace *>(trace_c);
    if (!space || !out) return fail(GUIDE_ERR_INVALID, "space and out are required");
    Range r;
    int rc = resolve_range(space, opts, &r);
    if (rc) return rc;
    const int time_model = opts ? opts->time_model : GUIDE_TIME_MAX, tp_model = opts ? opts->tp_model : GUIDE_TP_EXPLICIT;
    if (!trace && (out->req_ttft || out->req_tpot))
        return fail(GUIDE_ERR_INVALID, "per-request outputs need a trace");
    if (trace) {
        if (opts && opts->precision == GUIDE_PREC_F32)
            return fail(GUIDE_ERR_UNSUPPORTED, "the binary32 variant covers the closed form only: a trace simulation sums its clock over "
                                               "too many iterations for admission decisions to survive the rounding");
        if (opts && opts->clamp_seq)
            return fail(GUIDE_ERR_UNSUPPORTED, "clamp_seq cuts the lengths of a closed-form config; a trace fixes the lengths of its requests");
        if (space->evicting)
            return fail(GUIDE_ERR_UNSUPPORTED, "a framework profile evicts part of the KV cache (kv_keep_permille): modelled in the closed form only");
        if (space->max_dp > 1)
            return fail(GUIDE_ERR_UNSUPPORTED, "the trace simulation models one replica: the space has a data-parallel degree of %u",
                        space->max_dp);
        for (size_t i = 0; i < space->fw.size(); i++) {
            const guide_fw &f = space->fw[i];
            if (f.policy == GUIDE_POLICY_PREFILL_FIRST && (f.split_size || f.seg_tokens))
                return fail(GUIDE_ERR_UNSUPPORTED, "framework profile %zu: prompt-first iterations take whole prompts and whole "
                                                   "batches; split_size and seg_tokens apply to the closed form or to the "
                                                   "split-and-fuse policy", i);
            if (f.policy == GUIDE_POLICY_SPLIT_FUSE && (f.seg_tokens == 0 || f.split_size != 0))
                return fail(GUIDE_ERR_INVALID, "framework profile %zu: the split-and-fuse policy needs seg_tokens >= 1 (its token "
                                               "budget per iteration) and split_size 0", i);
        }
        if (space->max_batch > GUIDE_TRACE_MAX_BATCH)
            return fail(GUIDE_ERR_UNSUPPORTED, "the trace kernel keeps at most %u requests resident; the batch axis goes to %u",
                        GUIDE_TRACE_MAX_BATCH, space->max_batch);
        if ((rc = check_trace_overflow(*space, *trace))) return rc;
        if ((rc = check_workspace(ws, ws_bytes, trace_workspace_bytes((u32)trace->arrival.size(), lane_hints(*space))))) return rc;
    }
    if (r.count == 0) return GUIDE_OK;
    DSpace ds;
    unsigned *ticket = nullptr;
    if ((rc = space_on_device(space, &ds, &ticket, (cudaStream_t)stream))) return rc;
    if (!trace) {
        // options and outputs only the one-thread-per-config evaluation knows: keep the whole-space kernels out
        if ((opts && opts->clamp_seq) || out->seq_used) ds.chunked = 1;
        ds.clamp_seq = opts ? (u32)opts->clamp_seq : 0u;
        if (opts && opts->precision == GUIDE_PREC_F32)
            return launch_closed_form_f32(ds, r, time_model, tp_model, *out, (cudaStream_t)stream);
        return launch_closed_form(ds, r, time_model, tp_model, *out, ticket, (cudaStream_t)stream);
    }
    DTrace dt;
    if ((rc = trace_on_device(trace, &dt, (cudaStream_t)stream))) return rc;
    u32 policies = 0;
    for (const guide_fw &f : space->fw) policies |= f.policy == GUIDE_POLICY_SPLIT_FUSE ? 2u : 1u;
    return launch_trace_sim(ds, dt, r, time_model, tp_model, opts ? opts->max_iters : 0, *out, ws, ws_bytes,
                            (cudaStream_t)stream, policies, lane_hints(*space));
}

size_t guide_select_workspace_bytes(const guide_space *, uint32_t k) {
    return (k == 0 || k > GUIDE_TOPK_MAX) ? 0 : topk_workspace_bytes(k);
}
size_t guide_pareto_workspace_bytes(const guide_space *) { return pareto_workspace_bytes(); }

int guide_select_topk(const guide_space *space_c, const guide_trace *trace, const guide_outputs *outputs,
                      const guide_sim_opts *opts, const guide_constraints *cons, int key, uint32_t k,
                      uint64_t *idx_out, double *key_out, uint32_t *count_out, void *ws, size_t ws_bytes,
                      void *stream) {
    guide_space *space = const_cast<guide_space *>(space_c);
    int rc = check_selection_args(space, trace, outputs, cons, &key, 1);
    if (rc) return rc;
    if (k == 0 || k > GUIDE_TOPK_MAX) return fail(GUIDE_ERR_INVALID, "k must be in 1..%u", GUIDE_TOPK_MAX);
    if (!idx_out || !key_out || !count_out) return fail(GUIDE_ERR_INVALID, "an output pointer is NULL");
    Range r;
    if ((rc = resolve_range(space, opts, &r))) return rc;
    if ((rc = check_workspace(ws, ws_bytes, topk_workspace_bytes(k)))) return rc;
    DSpace ds;
    unsigned *ticket = nullptr;                  // the fused path's model walk takes its work items through it
    if ((rc = space_on_device(space, &ds, outputs ? nullptr : &ticket, (cudaStream_t)stream))) return rc;
    if (!outputs && opts && opts->precision == GUIDE_PREC_F32)
        return fail(GUIDE_ERR_UNSUPPORTED, "the fused selection evaluates in binary64: run guide_simulate with the binary32 option and select on its outputs");
    if (!outputs && opts && opts->clamp_seq) { ds.chunked = 1; ds.clamp_seq = 1; }     // fused: evaluated with the option
    return launch_topk(ds, r, outputs, opts ? opts->time_model : 0, opts ? opts->tp_model : 0, *cons, key, k,
                       (u64 *)idx_out, key_out, count_out, ws, ticket, (cudaStream_t)stream);
}

int guide_pareto(const guide_space *space_c, const guide_trace *trace, const guide_outputs *outputs,
                 const guide_sim_opts *opts, const guide_constraints *cons, int xm, int ym, uint64_t *idx_out,
                 uint32_t cap, uint32_t *count_out, void *ws, size_t ws_bytes, void *stream) {
    guide_space *space = const_cast<guide_space *>(space_c);
    const int keys[2] = {xm, ym};
    int rc = check_selection_args(space, trace, outputs, cons, keys, 2);
    if (rc) return rc;
    if (!count_out || (cap && !idx_out)) return fail(GUIDE_ERR_INVALID, "an output pointer is NULL");
    Range r;
    if ((rc = resolve_range(space, opts, &r))) return rc;
    if ((rc = check_workspace(ws, ws_bytes, pareto_workspace_bytes()))) return rc;
    DSpace ds;
    unsigned *ticket = nullptr;
    if ((rc = space_on_device(space, &ds, outputs ? nullptr : &ticket, (cudaStream_t)stream))) return rc;
    if (!outputs && opts && opts->precision == GUIDE_PREC_F32)
        return fail(GUIDE_ERR_UNSUPPORTED, "the fused selection evaluates in binary64: run guide_simulate with the binary32 option and select on its outputs");
    if (!outputs && opts && opts->clamp_seq) { ds.chunked = 1; ds.clamp_seq = 1; }
    return launch_pareto(ds, r, outputs, opts ? opts->time_model : 0, opts ? opts->tp_model : 0, *cons, xm, ym,
                         (u64 *)idx_out, cap, count_out, ws, ticket, (cudaStream_t)stream);
}

int guide_simulate_select(const guide_space *space_c, const guide_sim_opts *opts, const guide_outputs *out,
                          const guide_selection *sel, void *ws_t, size_t ws_t_bytes, void *ws_p, size_t ws_p_bytes,
                          void *stream) {
    guide_space *space = const_cast<guide_space *>(space_c);
    if (!space || !out || !sel) return fail(GUIDE_ERR_INVALID, "space, out and sel are required");
    if (out->req_ttft || out->req_tpot) return fail(GUIDE_ERR_INVALID, "per-request outputs need a trace");
    if (opts && (opts->clamp_seq || opts->precision == GUIDE_PREC_F32))
        return fail(GUIDE_ERR_UNSUPPORTED, "clamp_seq and the binary32 variant go through guide_simulate and the separate selection calls");
    if (out->seq_used) return fail(GUIDE_ERR_UNSUPPORTED, "seq_used is written by guide_simulate with clamp_seq only");
    int key = sel->key;
    int rc = check_selection_args(space, nullptr, out, sel->topk_cons, &key, 1);
    if (rc) return rc;
    const int xy[2] = {sel->x_metric, sel->y_metric};
    if ((rc = check_selection_args(space, nullptr, out, sel->pareto_cons, xy, 2))) return rc;
    if (sel->k == 0 || sel->k > GUIDE_TOPK_MAX) return fail(GUIDE_ERR_INVALID, "k must be in 1..%u", GUIDE_TOPK_MAX);
    if (!sel->topk_idx_dev || !sel->topk_key_dev || !sel->topk_count_dev || !sel->front_count_dev ||
        (sel->front_cap && !sel->front_idx_dev))
        return fail(GUIDE_ERR_INVALID, "an output pointer is NULL");
    Range r;
    if ((rc = resolve_range(space, opts, &r))) return rc;
    if ((rc = check_workspace(ws_t, ws_t_bytes, topk_workspace_bytes(sel->k)))) return rc;
    if ((rc = check_workspace(ws_p, ws_p_bytes, pareto_workspace_bytes()))) return rc;
    DSpace ds;
    unsigned *ticket = nullptr;
    if ((rc = space_on_device(space, &ds, &ticket, (cudaStream_t)stream))) return rc;
    return launch_simulate_select(ds, r, *out, opts ? opts->time_model : GUIDE_TIME_MAX, opts ? opts->tp_model : GUIDE_TP_EXPLICIT,
                                  *sel->topk_cons, key, sel->k, (u64 *)sel->topk_idx_dev, sel->topk_key_dev, sel->topk_count_dev, ws_t,
                                  *sel->pareto_cons, xy[0], xy[1], (u64 *)sel->front_idx_dev, sel->front_cap, sel->front_count_dev,
                                  ws_p, ticket, (cudaStream_t)stream, (cudaEvent_t)sel->sweep_begin_event,
                                  (cudaEvent_t)sel->sweep_end_event);
}

int guide_select_topk_noalloc(const guide_outputs *outputs, uint64_t first, uint64_t count,
                              const guide_constraints *cons, int key, uint32_t k, uint64_t *idx_out,
                              double *key_out, uint32_t *count_out, void *stream) {
    if (!outputs || !cons) return fail(GUIDE_ERR_INVALID, "outputs and constraints are required");
    if (k == 0) return fail(GUIDE_ERR_INVALID, "k must be at least 1");
    if (k > GUIDE_NOALLOC_TOPK_MAX)
        return fail(GUIDE_ERR_UNSUPPORTED, "k = %u is above GUIDE_NOALLOC_TOPK_MAX (%u): the built-in scratch array cannot hold it; "
                    "use guide_select_topk with a workspace", k, GUIDE_NOALLOC_TOPK_MAX);
    if (count == 0 || count > GUIDE_NOALLOC_COUNT_MAX)
        return fail(GUIDE_ERR_UNSUPPORTED, "count must be in 1..%llu for the no-allocation variant", (unsigned long long)GUIDE_NOALLOC_COUNT_MAX);
    if (first > UINT64_MAX - count) return fail(GUIDE_ERR_INVALID, "first + count overflows");
    if (!idx_out || !key_out || !count_out) return fail(GUIDE_ERR_INVALID, "an output pointer is NULL");
    if (key < GUIDE_LATENCY || key > GUIDE_COST_PER_TOKEN) return fail(GUIDE_ERR_INVALID, "unknown metric %d", key);
    if (cons->ttft_stat < GUIDE_STAT_MEAN || cons->ttft_stat > GUIDE_STAT_P99) return fail(GUIDE_ERR_INVALID, "unknown ttft_stat");
    if (std::isnan(cons->max_ttft) || std::isnan(cons->max_latency) || std::isnan(cons->max_cost_per_hr) ||
        std::isnan(cons->min_throughput))
        return fail(GUIDE_ERR_INVALID, "a constraint is NaN");
    if (!outputs->status) return fail(GUIDE_ERR_INVALID, "outputs->status is required");
    if (!metric_array(*outputs, key)) return fail(GUIDE_ERR_INVALID, "the array of metric %d is NULL", key);
    const double *ttft = cons->ttft_stat == GUIDE_STAT_MEAN ? outputs->ttft
                         : cons->ttft_stat == GUIDE_STAT_P50 ? outputs->ttft_p50 : outputs->ttft_p99;
    if (cons->max_ttft < INFINITY && !ttft) return fail(GUIDE_ERR_INVALID, "max_ttft is set but its array is NULL");
    if (cons->max_latency < INFINITY && !outputs->latency) return fail(GUIDE_ERR_INVALID, "max_latency is set but latency is NULL");
    if (cons->max_cost_per_hr < INFINITY && !outputs->cost_per_hr) return fail(GUIDE_ERR_INVALID, "max_cost_per_hr is set but cost_per_hr is NULL");
    if (cons->min_throughput > 0.0 && !outputs->thr_decode) return fail(GUIDE_ERR_INVALID, "min_throughput is set but thr_decode is NULL");
    Range r{first, count};
    return launch_topk_noalloc(r, *outputs, *cons, key, k, (u64 *)idx_out, key_out, count_out, (cudaStream_t)stream);
}

}  // extern "C"
