// Closed-form evaluation kernels: one prefill stage + one aggregated decode stage per config
// (Sec. 3.2 Steps 1-2, roofline of Sec. 3.4.2, time decomposition of Sec. 3.5.1).
#include "guide_internal.cuh"

namespace guide {

__device__ __forceinline__ void store_metrics(const guide_outputs &o, u64 j, const Metrics &m) {
    if (o.latency) __stcs(o.latency + j, m.latency);
    if (o.ttft) __stcs(o.ttft + j, m.ttft);
    if (o.ttft_p50) __stcs(o.ttft_p50 + j, m.ttft);
    if (o.ttft_p99) __stcs(o.ttft_p99 + j, m.ttft);
    if (o.tpot) __stcs(o.tpot + j, m.tpot);
    if (o.thr_decode) __stcs(o.thr_decode + j, m.thr);
    if (o.cost_per_hr) __stcs(o.cost_per_hr + j, m.cost_hr);
    if (o.cost_per_token) __stcs(o.cost_per_token + j, m.cost_tok);
    if (o.status) o.status[j] = (uint8_t)m.status;
    if (o.bmax) __stcs(o.bmax + j, m.bmax);
    if (o.n_iters) __stcs(o.n_iters + j, m.n_iters);
    if (o.n_req_iters) __stcs(o.n_req_iters + j, m.n_req_iters);
}

// One thread per config, nothing shared between configs.
template <int TIME_SUM>
__global__ void __launch_bounds__(256) k_closed_form_flat(DSpace s, Range r, int tp_model, guide_outputs o) {
    const u64 j = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= r.count) return;
    const Cfg c = decode_index(s, r.first + j);
    Metrics m;
    closed_form_eval<TIME_SUM>(s, c, tp_model, m);
    store_metrics(o, j, m);
}

// Tiled evaluation.  The integer task table of a config depends on (model, batch, TP, lengths)
// only, and within one (model, batch) the (TP, length) positions are the fastest-running part of
// the config index.  A thread therefore owns one (model, batch, TP, length) point, builds both
// stage tables once, and walks a chunk of the hardware x framework pairs, which are the only
// things the roofline evaluation needs beyond the table.  A warp's 32 threads hold 32
// consecutive config indices for every pair, so each store instruction writes one 256-byte run.
template <int TIME_SUM>
__global__ void __launch_bounds__(256) k_closed_form_tiled(DSpace s, Range r, int tp_model, u32 hf_chunk,
                                                           u32 tiles_per_mb, guide_outputs o) {
    const u32 n_tl = s.n_t * s.n_l;
    const u32 n_hf = s.n_h * s.n_f;
    // blockIdx.x -> (model, batch, tile of the (TP, length) plane); blockIdx.y -> chunk of pairs
    const u32 tile = blockIdx.x % tiles_per_mb;
    const u32 mb = blockIdx.x / tiles_per_mb;
    const u32 bpos = mb % s.n_b, mpos = mb / s.n_b;
    const u32 tl = tile * blockDim.x + threadIdx.x;
    if (tl >= n_tl) return;
    const u32 tpos = tl / s.n_l, lpos = tl % s.n_l;
    const u32 hf0 = blockIdx.y * hf_chunk;
    const u32 hf1 = min(hf0 + hf_chunk, n_hf);

    const DModel m = s.models[mpos];
    const u32 t = s.tp[tpos], b = s.batch[bpos];
    const uint2 pr = s.pairs[lpos];
    const u32 lin = pr.x, lout = pr.y, n = lout - 1;
    const MemInfo mi = mem_info(m, t);
    const u32 tt = tp_model ? 1u : t;
    const double lf = log2_rule_factor(t, tp_model);
    const double Nd = (double)m.N;

    TaskTab kp, kd;
    const u64 Tp = (u64)b * lin;
    build_fixed_tasks(m, tt, Tp, b, 1, kp);
    build_attn_tasks(m, tt, Tp, Tp * lin, Tp, kp);
    if (n > 0) {
        const u64 Td = (u64)b * n;
        const u64 ctx = (u64)b * ((u64)n * lin + ((u64)n * (n + 1)) / 2);
        build_fixed_tasks(m, tt, Td, Td, n, kd);
        build_attn_tasks(m, tt, Td, ctx, ctx, kd);
    }
    // index of this thread's config for pair (h, f): ((((m n_h + h) n_f + f) n_b + b) n_t n_l) + tl
    const u64 stride_hf = (u64)s.n_b * n_tl;
    const u64 base = ((u64)mpos * n_hf) * stride_hf + (u64)bpos * n_tl + tl;

    for (u32 hf = hf0; hf < hf1; hf++) {
        const u64 idx = base + (u64)hf * stride_hf;
        if (idx < r.first || idx - r.first >= r.count) continue;
        const DRate rt = s.rates[hf];
        Metrics out;
        out.status = closed_form_feasibility(m, rt, mi, t, b, lin, lout, out.bmax);
        if (out.status) set_infeasible(out);
        else {
            const double t_pre = eval_phase<TIME_SUM>(kp, rt, Nd, lf);
            const double t_dec = n > 0 ? eval_phase<TIME_SUM>(kd, rt, Nd, lf) : 0.0;
            closed_form_metrics(t_pre, t_dec, b, n, t, rt.price, out);
        }
        store_metrics(o, idx - r.first, out);
    }
}

int launch_closed_form(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o,
                       cudaStream_t st) {
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f;
    const u64 total = (u64)s.n_m * n_hf * s.n_b * n_tl;
    // The tiled kernel pays off when a (TP, length) plane fills warps and the range is (most of)
    // the space; slivers of the space go through the flat kernel.
    const bool tiled = n_tl >= 32 && r.count * 2 >= total;
    if (!tiled) {
        const u64 blocks = (r.count + 255) / 256;
        if (blocks > 0x7FFFFFFFull) return fail(GUIDE_ERR_UNSUPPORTED, "range too large for one launch");
        if (time_model) k_closed_form_flat<1><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
        else k_closed_form_flat<0><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
    } else {
        const u32 threads = n_tl >= 256 ? 256 : ((n_tl + 31) / 32) * 32;
        const u32 tiles = (n_tl + threads - 1) / threads;
        const u64 gx = (u64)s.n_m * s.n_b * tiles;
        // Split the pair loop so the grid has a few waves of blocks; longer chunks amortise the
        // table building over more configs.
        const u64 want_blocks = (u64)num_sms() * 16;
        u32 splits = (u32)std::min<u64>(n_hf, std::max<u64>(1, (want_blocks + gx - 1) / gx));
        u32 chunk = (n_hf + splits - 1) / splits;
        splits = (n_hf + chunk - 1) / chunk;
        if (gx > 0x7FFFFFFFull || splits > 65535) return fail(GUIDE_ERR_UNSUPPORTED, "space too large for one launch");
        const dim3 grid((u32)gx, splits);
        if (time_model) k_closed_form_tiled<1><<<grid, threads, 0, st>>>(s, r, tp_model, chunk, tiles, o);
        else k_closed_form_tiled<0><<<grid, threads, 0, st>>>(s, r, tp_model, chunk, tiles, o);
    }
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

}  // namespace guide
