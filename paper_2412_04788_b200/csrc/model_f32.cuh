// The closed form with every operation of the performance model in binary32: the reduced-precision
// variant of guide_simulate (opts->precision = GUIDE_PREC_F32).  Integer FLOP / byte counts, the
// memory check and the counters are the same exact integers as in the binary64 path; each count is
// rounded to binary32 once, and the task times, sums and metrics follow in the same written order
// (per task: sharded part / t + replicated part, the two times, their maximum or sum; tasks with
// their multiplicities; the eight non-attention tasks summed left to right, then attention, the
// all-reduce term, layers, head, overhead).  Nothing is cached or shared between configs: one thread
// evaluates one config.  Results are handed back widened to double, which is exact.
#pragma once
#include "model.cuh"

namespace guide {

// reciprocal rates of one (hardware, framework) pair in binary32: product first, then one reciprocal
struct RateF {
    float inv_c[3], inv_m[3], inv_comm, clat, tovh, price;
    u32 flash, pad;
};

__device__ __forceinline__ float cvtf(u64 x) { return __ull2float_rn(x); }

template <int TIME_SUM>
__device__ __forceinline__ float task_time_f(u64 F_sh, u64 F_rp, u64 B_sh, u64 B_rp, float t, float ic, float im) {
    const float F = cvtf(F_sh) / t + cvtf(F_rp);       // sharded part splits over t GPUs
    const float B = cvtf(B_sh) / t + cvtf(B_rp);
    const float tc = F * ic;                           // compute time (Sec. 3.5.1)
    const float tm = B * im;                           // read/write time
    return TIME_SUM ? tc + tm : (tc > tm ? tc : tm);   // literal sum, or the roofline of Sec. 3.4.2
}

// Time of one stage: T new tokens, E sequences emitting a token, A = sum(query x context),
// C = sum(context), R repeats (Sec. 3.2 Step 2, Sec. 3.4.1, Sec. 3.5.1).
template <int TIME_SUM>
__device__ __noinline__ float stage_time_f(const DModel &m, const RateF &r, u32 tp, u64 T, u64 E, u64 A, u64 C, u64 R,
                                           int tp_model) {
    const u32 tt = tp_model ? 1u : tp;                 // log2 rule: single-GPU formulas, scaled below
    const float t = (float)tt;
    const u64 H = m.H, I = m.I, Dkv = m.Dkv, V = m.V, ab = m.ab, wb = m.wb, kvb = m.kvb;
    const u64 TH = T * H, THa = TH * ab, TI = T * I, TIa = TI * ab;
    const u64 X = r.flash ? 0 : (u64)m.nh * A * ab;    // score-matrix traffic, gone with FlashAttention
    const float icL = r.inv_c[CLS_LINEAR], imL = r.inv_m[CLS_LINEAR], icA = r.inv_c[CLS_ATTN], imA = r.inv_m[CLS_ATTN],
                icE = r.inv_c[CLS_ELEM], imE = r.inv_m[CLS_ELEM];
    float s = 2.0f * task_time_f<TIME_SUM>(0, 4 * TH, 0, 2 * THa, t, icE, imE);                                // norm x2
    s = s + task_time_f<TIME_SUM>(2 * TH * H, 0, R * (H * H * wb) + THa, THa, t, icL, imL);                     // q_proj
    s = s + 2.0f * task_time_f<TIME_SUM>(2 * TH * Dkv, 0, R * (H * Dkv * wb) + T * Dkv * kvb, THa, t, icL, imL);   // k, v
    s = s + task_time_f<TIME_SUM>(2 * TH * H, 0, R * (H * H * wb) + THa, THa, t, icL, imL);                     // o_proj
    s = s + 2.0f * task_time_f<TIME_SUM>(0, TH, 0, 3 * THa, t, icE, imE);                                       // residual x2
    s = s + (float)(1 + m.g) * task_time_f<TIME_SUM>(2 * TH * I, 0, R * (H * I * wb) + TIa, THa, t, icL, imL);  // up (+ gate)
    s = s + task_time_f<TIME_SUM>(4 * TI, 0, (2 + (u64)m.g) * TIa, 0, t, icE, imE);                             // activation
    s = s + task_time_f<TIME_SUM>(2 * TI * H, 0, R * (I * H * wb) + TIa, THa, t, icL, imL);                     // down
    const u64 kv_read = C * Dkv * kvb;
    const float t9 = task_time_f<TIME_SUM>(2 * H * A, 0, THa + kv_read + X, 0, t, icA, imA);                    // qk
    const float t10 = task_time_f<TIME_SUM>(5 * (u64)m.nh * A, 0, 2 * X, 0, t, icA, imA);                       // softmax
    const float t11 = task_time_f<TIME_SUM>(2 * H * A, 0, kv_read + THa + X, 0, t, icA, imA);                   // sv
    float s_att = t9 + t10;
    s_att = s_att + t11;
    // no sequence emits a token (a prompt segment that is not the last one): no LM head at all
    const float head = E == 0 ? 0.0f
                              : task_time_f<TIME_SUM>(2 * (E * H) * V, 0, R * (H * V * wb) + E * V * ab, E * H * ab, t, icL, imL);
    // ring all-reduce of the T x H activations, twice per layer; only when really sharded
    float s_comm = 0.0f;
    if (tt > 1) {
        const float t12 = cvtf(R * (u64)(2 * (tt - 1))) * r.clat + (cvtf((u64)(2 * (tt - 1)) * THa) / t) * r.inv_comm;
        s_comm = 2.0f * t12;
    }
    const float layer = (s + s_att) + s_comm;
    float tph = cvtf(R) * r.tovh + ((float)m.N * layer + head);
    if (tp_model) {
        const u32 lg = 31 - __clz(tp);
        tph = tph * ((float)(1 + lg) / (float)tp);     // throughput rule of Sec. 3.2: time x (1 + log2 t) / t
    }
    return tph;
}

template <int TIME_SUM>
__device__ __forceinline__ float segmented_prefill_f(const DModel &m, const RateF &r, u32 t, u32 sb, u32 lin, u32 seg,
                                                     int tp_model) {
    float sum = 0.0f;
    for (u32 done = 0; done < lin; done += seg) {
        const u32 q = min(seg, lin - done);
        const u64 T = (u64)sb * q;
        const u64 E = done + q == lin ? sb : 0;
        sum = sum + stage_time_f<TIME_SUM>(m, r, t, T, E, T * (done + q), (u64)sb * (done + q), 1, tp_model);
    }
    return sum;
}

// One config in closed form, binary32 (same memory check, clamp, eviction share and counters as
// closed_form_eval).
template <int TIME_SUM>
__device__ __forceinline__ void closed_form_eval_f32(const DSpace &s, const RateF *rates, const Cfg &c, int tp_model, Metrics &o) {
    const DModel m = s.models[c.m];
    const DRate &r = s.rates[c.h * s.n_f + c.f];
    const RateF rf = rates[c.h * s.n_f + c.f];
    const u32 t = s.tp[c.t], b_all = s.batch[c.b], dp = s.dp[c.t];
    const u32 b = replica_batch(b_all, dp);
    const uint2 pr = s.pairs[c.l];
    u32 lin = pr.x;
    const u32 lout = pr.y;
    const MemInfo mi = mem_info(m, t);
    if (s.clamp_seq && r.usable > mi.w_gpu) {
        const u64 cap_tok = floor_div(r.usable - mi.w_gpu, mi.kv_tok * b);
        const u64 cap_blk = (cap_tok / r.kv_block) * r.kv_block;
        const u64 s_max = (r.keep >= 1000 || cap_blk >= (1ull << 40)) ? cap_blk : (1000 * cap_blk) / r.keep;
        if ((u64)lin + lout > s_max && s_max > lout) lin = (u32)(s_max - lout);
    }
    o.status = closed_form_feasibility(m, r, mi, t, b, lin, lout, o.bmax);
    o.seq_used = o.status ? 0u : lin + lout;
    if (o.status) { set_infeasible(o); return; }
    const u32 split = (r.split == 0 || r.split > b) ? b : r.split;
    const u32 seg = (r.seg == 0 || r.seg > lin) ? lin : r.seg;
    const u32 n_full = b / split, rest = b % split;
    float t_pre = (float)n_full * segmented_prefill_f<TIME_SUM>(m, rf, t, split, lin, seg, tp_model);
    if (rest) t_pre = t_pre + segmented_prefill_f<TIME_SUM>(m, rf, t, rest, lin, seg, tp_model);
    const u64 n_seg = (lin + seg - 1) / seg;
    const u32 n = lout - 1;
    float t_dec = 0.0f;
    if (n > 0) {
        const u64 Td = (u64)b * n;
        const u64 ctx = kept_tokens((u64)b * ((u64)n * lin + ((u64)n * (n + 1)) / 2), r.keep);
        t_dec = stage_time_f<TIME_SUM>(m, rf, t, Td, Td, ctx, ctx, n, tp_model);
    }
    const float inf = __int_as_float(0x7F800000);
    const float lat = t_pre + t_dec;
    const float cost_hr = rf.price * cvtf((u64)t * dp);          // every GPU of every replica is paid for
    float tpot = 0.0f, thr = 0.0f, cost_tok = inf;
    if (n > 0) {
        tpot = t_dec / (float)n;
        thr = cvtf((u64)b_all * n) / t_dec;
        cost_tok = (cost_hr / 3600.0f) / thr;
    }
    o.ttft = t_pre; o.latency = lat; o.tpot = tpot; o.thr = thr; o.cost_hr = cost_hr; o.cost_tok = cost_tok;
    o.n_iters = (u64)(n_full + (rest != 0)) * n_seg + (u64)n;
    o.n_req_iters = (u64)b_all * (n_seg + (u64)n);
}

}  // namespace guide
