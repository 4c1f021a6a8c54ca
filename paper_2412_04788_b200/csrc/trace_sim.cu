// Trace-driven continuous-batching simulation, one warp per config (dynamic batching of Sec. 3.1;
// prompt-priority scheduling and fixed-granularity paged KV of the vLLM-like framework model,
// Sec. 2.3.2 / 2.4.1 / 2.4.2).
//
// A warp owns one config at a time and pulls the next one from a global counter, smallest
// max-batch first (those schedules have the most iterations), so long schedules start early and
// do not hold back a whole block.  The clock, counters and the iteration time are warp-uniform.
//
// Between events a decode iteration costs O(1): nothing per request is touched.
//   - Resident requests live in per-warp shared-memory slots in ascending request order and store
//     invariants, not running values: with D = decode iterations done so far, a slot keeps
//     base = cache - D and fin = D + tokens still to generate, both constant while it is resident.
//   - The number of requests whose last KV block is full comes from a histogram of
//     (cache - D) mod block; the next completion is a countdown; the summed context grows by the
//     running count each step.
//   - The attention tasks are re-evaluated every iteration from the summed context; everything
//     that depends only on the running count is cached until that count changes.  When every
//     integer FLOP/byte count of the config stays below 2^53 the counts are carried as doubles
//     (products and sums of integers below 2^53 are exact in binary64), which removes the
//     integer-to-double conversions from the loop without changing a bit.
// Events (admission, prompt pass, completion, eviction) scan the slots with all 32 lanes.
// Per-request results that outlive residency (tokens generated so far, first-token time, time per
// output token) sit in a per-warp slice of the workspace.  The request trace is the same for every
// config and is read through the read-only path, so it stays cache resident.
#include <cstdlib>

#include "guide_internal.cuh"
#include "trace_fuse.cuh"
#include "trace_lanes.cuh"

namespace guide {

#ifndef SIM_MIN_BLOCKS
#define SIM_MIN_BLOCKS 2          // resident blocks per SM k_trace_sim is compiled for (128 registers, no spills: it keeps the
                                  // event-heavy large batches now; 3 blocks of 80 registers measured 3 % slower)
#endif
#ifndef FUSE_MIN_BLOCKS
#define FUSE_MIN_BLOCKS 2         // ... and k_trace_fuse (measured 2.5 % faster than 3 blocks of 80 registers)
#endif
#ifndef SIM_BLOCK_WARPS
#define SIM_BLOCK_WARPS 8
#endif
static constexpr u32 SIM_WARPS_PER_BLOCK = SIM_BLOCK_WARPS;
static constexpr u32 SIM_THREADS = SIM_WARPS_PER_BLOCK * 32;
static constexpr u32 SIM_MAX_WARPS = 3072;        // workspace is sized for this many resident warps: the warp-per-config kernels
                                                  // keep two blocks of eight on an SM (148 SMs use 2,368; launches are capped here)
static constexpr u32 LANE_MAX_WARPS = 148 * 16;   // ... and for this many warps of the lane kernel
static constexpr u32 SLOTS = GUIDE_TRACE_MAX_BATCH;
static constexpr u32 HIST = 64;                   // block sizes up to this use the phase histogram
static constexpr u32 M_PHASE = 0x3F, M_FIRST = 0x40, M_NEEDS_PREFILL = 0x80;
static constexpr u32 GEN_DONE = 0x80000000u;
static constexpr u32 NO_COMPLETION = 0xFFFFFFFFu;

static u32 pow2_at_least(u32 v) { u32 p = 1; while (p < v) p <<= 1; return p; }

static size_t per_warp_bytes(u32 n_req) {
    // gen u32[n] | first f64[n] | tpot f64[pow2(n)] (reused as the sort buffer)
    const size_t n = n_req, p = pow2_at_least(n_req);
    return ((n * 4 + 255) / 256 * 256) + ((n * 8 + 255) / 256 * 256) + ((p * 8 + 255) / 256 * 256);
}


// Sum over the warp of values below 2^51 (block and token counts), by the integer reduction unit:
// the low 24 bits and the rest are summed apart so that neither sum leaves 32 bits.
__device__ __forceinline__ u64 warp_sum(u64 v) {
    const u32 lo = __reduce_add_sync(0xFFFFFFFFu, (u32)v & 0xFFFFFFu), hi = __reduce_add_sync(0xFFFFFFFFu, (u32)(v >> 24));
    return ((u64)hi << 24) + lo;
}
__device__ __forceinline__ u32 warp_min(u32 v) { return __reduce_min_sync(0xFFFFFFFFu, v); }
__device__ __forceinline__ u32 ceil_div32(u32 a, u32 b) { return (a + b - 1) / b; }

// Time of one decode iteration from the summed context (as an exact double), when every integer
// count of the config is below 2^53: the same products and sums as the integer form, in doubles.
// B9 = (T H a_b + ctx (Dkv kv_b + score bytes)) / t is a sum of exact terms, so its association
// does not matter; with FlashAttention the score constants are 0 and t10's memory time is 0.
template <int TIME_SUM>
__device__ __forceinline__ double decode_time(double ctxd, double c_f9, double tha, double c_kvx, double c_f10, double c_b10,
                                              double ic, double im, double fix, double comm, double head, double Nd,
                                              double tovh, double lf) {
    const double t9 = task_time<TIME_SUM>(ctxd * c_f9, tha + ctxd * c_kvx, ic, im);
    const double t10 = task_time<TIME_SUM>(ctxd * c_f10, ctxd * c_b10, ic, im);
    const double s_att = (t9 + t10) + t9;
    return combine_phase(fix, s_att, comm, head, 1.0, Nd, tovh, lf);
}

static_assert(sizeof(DModel) <= 128 && sizeof(DRate) <= 128, "a warp copies each of them with one word per lane");
struct SlotArrays {
    double tbuf[32];    // times of the 32 iterations a run computes at once
    double dterm[32][4];   // decode terms (fixed tasks, all-reduce, head, activation bytes) of 32 neighbouring resident counts
    double sc[32];         // the config's task-table factors as doubles (a StageConst), when its counts stay exact in them
    double rate[10];       // its row of rate10
    double cst[8];         // its attention and stage constants (read where they are used: they need not live in registers)
    DModel m;              // the config's model and (hardware, framework) rates
    DRate rt;
    u32 req[SLOTS];     // request index
    u32 base[SLOTS];    // resident: cache - D (mod 2^32); waiting for its prompt pass: prompt + recompute tokens
    u32 fin[SLOTS];     // resident: D at which it completes; waiting for its prompt pass: tokens still to emit
    u32 hist[HIST];     // residents per (cache - D) mod block
    unsigned char meta[SLOTS];   // phase (6 bits) | first-ever prompt pass | waiting for its prompt pass
};

// Results of one simulated config: per-request values, means in request order, nearest-rank
// percentiles (sorted in the tpot slice, which is free by then).  Called by the whole warp.
// tpot[i] holds the time of request i's last token on entry; the time per output token is worked out
// here, 32 requests at a time (Lout: output length of the requests that take the config's lengths).
__device__ __forceinline__ void write_trace_results(const guide_outputs &o, u64 j, u32 n, u32 st, u32 fit, double clock,
                                                    double dec_time, u64 dec_tok, u64 n_iters, u64 n_req_iters, double cost_hr,
                                                    const DTrace &tr, u32 Lout, double *first, double *tpot, u32 lane) {
    const double *arrival = tr.arrival;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    double *rq_ttft = o.req_ttft ? o.req_ttft + j * n : nullptr;
    double *rq_tpot = o.req_tpot ? o.req_tpot + j * n : nullptr;
    __syncwarp();
    if (st) {
        if (lane == 0) {
            if (o.latency) o.latency[j] = inf;
            if (o.ttft) o.ttft[j] = inf;
            if (o.ttft_p50) o.ttft_p50[j] = inf;
            if (o.ttft_p99) o.ttft_p99[j] = inf;
            if (o.tpot) o.tpot[j] = inf;
            if (o.thr_decode) o.thr_decode[j] = 0.0;
            if (o.cost_per_hr) o.cost_per_hr[j] = inf;
            if (o.cost_per_token) o.cost_per_token[j] = inf;
            if (o.status) o.status[j] = (uint8_t)st;
            if (o.bmax) o.bmax[j] = fit;
            if (o.n_iters) o.n_iters[j] = 0;
            if (o.n_req_iters) o.n_req_iters[j] = 0;
            if (o.seq_used) o.seq_used[j] = 0;
        }
        for (u32 i = lane; i < n; i += 32) {
            if (rq_ttft) __stcs(rq_ttft + i, inf);
            if (rq_tpot) __stcs(rq_tpot + i, inf);
        }
        return;
    }
    // means in request order: 32 values at a time, added one after the other
    double s_ttft = 0.0, s_tpot = 0.0;
    for (u32 base = 0; base < n; base += 32) {
        const u32 i = base + lane;
        double vt = 0.0, vp = 0.0;
        if (i < n) {
            const double f = first[i];
            vt = f - __ldg(arrival + i);
            vp = tpot[i];
            const u32 out = __ldg(tr.in_len + i) ? __ldg(tr.out_len + i) : Lout;
            vp = out > 1 ? (vp - f) / (double)(out - 1) : 0.0;
            if (rq_ttft) __stcs(rq_ttft + i, vt);
            if (rq_tpot) __stcs(rq_tpot + i, vp);
        }
        const u32 lim = min(32u, n - base);
        for (u32 l = 0; l < lim; l++) {
            s_ttft = s_ttft + __shfl_sync(0xFFFFFFFFu, vt, l);
            s_tpot = s_tpot + __shfl_sync(0xFFFFFFFFu, vp, l);
        }
        if (i < n) first[i] = vt;             // keep TTFT for the percentile sort
    }
    // nearest-rank percentiles: sort the TTFTs in the (now free) tpot slice
    u32 P = 1;
    while (P < n) P <<= 1;
    __syncwarp();
    for (u32 i = lane; i < P; i += 32) tpot[i] = i < n ? first[i] : inf;
    __syncwarp();
    for (u32 size = 2; size <= P; size <<= 1) {
        for (u32 stride = size >> 1; stride > 0; stride >>= 1) {
            for (u32 i = lane; i < (P >> 1); i += 32) {
                const u32 lo = ((i & ~(stride - 1)) << 1) | (i & (stride - 1));
                const u32 hi = lo + stride;
                const bool up = (lo & size) == 0;
                const double a = tpot[lo], bb = tpot[hi];
                if ((bb < a) == up) { tpot[lo] = bb; tpot[hi] = a; }
            }
            __syncwarp();
        }
    }
    if (lane == 0) {
        const double nd = (double)n;
        const double thr = dec_time > 0.0 ? cvt(dec_tok) / dec_time : 0.0;
                    if (o.latency) o.latency[j] = clock;
        if (o.ttft) o.ttft[j] = s_ttft / nd;
        if (o.ttft_p50) o.ttft_p50[j] = tpot[(50ull * n + 99) / 100 - 1];
        if (o.ttft_p99) o.ttft_p99[j] = tpot[(99ull * n + 99) / 100 - 1];
        if (o.tpot) o.tpot[j] = s_tpot / nd;
        if (o.thr_decode) o.thr_decode[j] = thr;
        if (o.cost_per_hr) o.cost_per_hr[j] = cost_hr;
        if (o.cost_per_token) o.cost_per_token[j] = thr > 0.0 ? (cost_hr / 3600.0) / thr : inf;
        if (o.status) o.status[j] = 0;
        if (o.bmax) o.bmax[j] = fit;
        if (o.n_iters) o.n_iters[j] = n_iters;
        if (o.n_req_iters) o.n_req_iters[j] = n_req_iters;
        if (o.seq_used) o.seq_used[j] = 0;          // closed form only
    }
}

// Results of one config simulated by k_trace_sim or the lane kernel: per-request values, means in request order, nearest-rank
// percentiles.  first[i]: time of request i's first token; finish[i]: time of its last one (the
// slice has room for the next power of two of doubles and serves as the sort buffer afterwards).
// Called by the whole warp; out of line, so that its registers (the sort keeps a batch of pairs in
// flight) do not weigh on the simulation loops of its callers.
__device__ __noinline__ void write_lane_results(const guide_outputs &o, u64 j, u32 n, u32 st, u32 fit, double clock,
                                                 double dec_time, u64 dec_tok, u64 n_iters, u64 n_req_iters, double cost_hr,
                                                 const DTrace &tr, u32 Lout, double *first, double *finish, u32 lane) {
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    double *rq_ttft = o.req_ttft ? o.req_ttft + j * n : nullptr;
    double *rq_tpot = o.req_tpot ? o.req_tpot + j * n : nullptr;
    __syncwarp();
    if (st) {
        if (lane == 0) {
            if (o.latency) o.latency[j] = inf;
            if (o.ttft) o.ttft[j] = inf;
            if (o.ttft_p50) o.ttft_p50[j] = inf;
            if (o.ttft_p99) o.ttft_p99[j] = inf;
            if (o.tpot) o.tpot[j] = inf;
            if (o.thr_decode) o.thr_decode[j] = 0.0;
            if (o.cost_per_hr) o.cost_per_hr[j] = inf;
            if (o.cost_per_token) o.cost_per_token[j] = inf;
            if (o.status) o.status[j] = (uint8_t)st;
            if (o.bmax) o.bmax[j] = fit;
            if (o.n_iters) o.n_iters[j] = 0;
            if (o.n_req_iters) o.n_req_iters[j] = 0;
            if (o.seq_used) o.seq_used[j] = 0;
        }
        for (u32 i = lane; i < n; i += 32) {
            if (rq_ttft) __stcs(rq_ttft + i, inf);
            if (rq_tpot) __stcs(rq_tpot + i, inf);
        }
        return;
    }
    // means in request order: 32 values at a time, added one after the other
    double s_ttft = 0.0, s_tpot = 0.0;
    for (u32 base = 0; base < n; base += 32) {
        const u32 i = base + lane;
        double vt = 0.0, vp = 0.0;
        if (i < n) {
            const double f = first[i];
            const u32 out = __ldg(tr.in_len + i) ? __ldg(tr.out_len + i) : Lout;
            vt = f - __ldg(tr.arrival + i);
            vp = out > 1 ? (finish[i] - f) / (double)(out - 1) : 0.0;     // time per output token after the first
            if (rq_ttft) __stcs(rq_ttft + i, vt);
            if (rq_tpot) __stcs(rq_tpot + i, vp);
        }
        const u32 lim = min(32u, n - base);
        for (u32 l = 0; l < lim; l++) {
            s_ttft = s_ttft + __shfl_sync(0xFFFFFFFFu, vt, l);
            s_tpot = s_tpot + __shfl_sync(0xFFFFFFFFu, vp, l);
        }
        if (i < n) first[i] = vt;             // keep TTFT for the percentile sort
    }
    // nearest-rank percentiles: bitonic sort of the TTFTs in the (now free) finish slice.  The pairs of
    // a stage are disjoint, so a lane loads a batch of them before it stores any: the loads overlap.
    double *buf = finish;
    if (o.ttft_p50 || o.ttft_p99) {
        u32 P = 1;
        while (P < n) P <<= 1;
        __syncwarp();
        for (u32 i = lane; i < P; i += 32) buf[i] = i < n ? first[i] : inf;
        __syncwarp();
        constexpr u32 BATCH = 8;
        for (u32 size = 2; size <= P; size <<= 1) {
            for (u32 stride = size >> 1; stride > 0; stride >>= 1) {
                for (u32 i0 = lane; i0 < (P >> 1); i0 += 32 * BATCH) {
                    double a[BATCH], bb[BATCH];
                    u32 lo[BATCH];
#pragma unroll
                    for (u32 u = 0; u < BATCH; u++) {
                        const u32 i = i0 + 32 * u;
                        lo[u] = ((i & ~(stride - 1)) << 1) | (i & (stride - 1));
                        if (i < (P >> 1)) { a[u] = buf[lo[u]]; bb[u] = buf[lo[u] + stride]; }
                    }
#pragma unroll
                    for (u32 u = 0; u < BATCH; u++) {
                        const u32 i = i0 + 32 * u;
                        const bool up = (lo[u] & size) == 0;
                        if (i < (P >> 1) && (bb[u] < a[u]) == up) { buf[lo[u]] = bb[u]; buf[lo[u] + stride] = a[u]; }
                    }
                }
                __syncwarp();
            }
        }
    }
    if (lane == 0) {
        const double nd = (double)n;
        const double thr = dec_time > 0.0 ? cvt(dec_tok) / dec_time : 0.0;
        if (o.latency) o.latency[j] = clock;
        if (o.ttft) o.ttft[j] = s_ttft / nd;
        if (o.ttft_p50) o.ttft_p50[j] = buf[(50ull * n + 99) / 100 - 1];
        if (o.ttft_p99) o.ttft_p99[j] = buf[(99ull * n + 99) / 100 - 1];
        if (o.tpot) o.tpot[j] = s_tpot / nd;
        if (o.thr_decode) o.thr_decode[j] = thr;
        if (o.cost_per_hr) o.cost_per_hr[j] = cost_hr;
        if (o.cost_per_token) o.cost_per_token[j] = thr > 0.0 ? (cost_hr / 3600.0) / thr : inf;
        if (o.status) o.status[j] = 0;
        if (o.bmax) o.bmax[j] = fit;
        if (o.n_iters) o.n_iters[j] = n_iters;
        if (o.n_req_iters) o.n_req_iters[j] = n_req_iters;
        if (o.seq_used) o.seq_used[j] = 0;          // closed form only
    }
}

template <int TIME_SUM>
__global__ void __launch_bounds__(SIM_THREADS, SIM_MIN_BLOCKS)
k_trace_sim(DSpace s, DTrace tr, Range r, int tp_model, u64 max_iters_opt, guide_outputs o, u32 *counter,
            unsigned char *scratch, size_t per_warp, u32 gen_bytes, u32 first_bytes, int reorder, u32 lane_maxb, u32 lane_hist) {
    __shared__ SlotArrays sh[SIM_WARPS_PER_BLOCK];
    const u32 lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const u32 warp_global = blockIdx.x * SIM_WARPS_PER_BLOCK + wib;
    SlotArrays &sl = sh[wib];
    unsigned char *mine = scratch + (size_t)warp_global * per_warp;
    u32 *gen = (u32 *)mine;
    double *first = (double *)(mine + gen_bytes);
    double *tpot = (double *)(mine + gen_bytes + first_bytes);
    const u32 n = tr.n;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    const u32 lt_mask = (1u << lane) - 1;

    for (;;) {
        u64 w = 0;
        if (lane == 0) w = atomicAdd(counter, 1u);
        w = __shfl_sync(0xFFFFFFFFu, w, 0);
        if (w >= r.count) break;
        const u64 idx = reorder ? work_to_index(s, w, true) : r.first + w;
        const u64 j = idx - r.first;
        const Cfg c = decode_index(s, idx);
        const DRate *rate_g = s.rates + (c.h * s.n_f + c.f);
        if (rate_g->policy != GUIDE_POLICY_PREFILL_FIRST) continue;  // k_trace_fuse simulates those
        // the model and the pair's rates next to the warp: their fields are read where they are used
        __syncwarp();
        if (lane < sizeof(DModel) / 4) reinterpret_cast<u32 *>(&sl.m)[lane] = reinterpret_cast<const u32 *>(s.models + c.m)[lane];
        if (lane < sizeof(DRate) / 4) reinterpret_cast<u32 *>(&sl.rt)[lane] = reinterpret_cast<const u32 *>(rate_g)[lane];
        __syncwarp();
        const DModel &m = sl.m;
        const DRate &rt = sl.rt;
        const u32 t = s.tp[c.t], b = s.batch[c.b];
        const uint2 pr = s.pairs[c.l];
        const u32 Lin = pr.x, Lout = pr.y, blk = rt.kv_block;
        const MemInfo mi = mem_info(m, t);
        const u32 tt = tp_model ? 1u : t;
        const double inv_tt = 1.0 / (double)tt;
        // per-config constants of the iteration time: kept next to the warp in shared memory
        const double &lf = sl.cst[0], &Nd = sl.cst[1], &icA = sl.cst[2], &imA = sl.cst[3];
        const double &c_f9 = sl.cst[4], &c_kvx = sl.cst[5], &c_f10 = sl.cst[6], &c_b10 = sl.cst[7];
        // configs the lane kernel was launched for are simulated there
        const bool sc_ok = lanes_exact(m, tt, b, max(tr.max_tokens, tr.any_zero ? Lin + Lout : 0u));   // stage tables from doubles are exact
        if (lanes_take(lane_maxb, lane_hist, b, blk, sc_ok)) continue;

        // ---- what fits (Sec. 3.2 Step 1) ----
        const u64 blocks_total = rt.usable > mi.w_gpu ? floor_div(rt.usable - mi.w_gpu, (u64)blk * mi.kv_tok) : 0;
        const u32 longest = max(tr.max_tokens, tr.any_zero ? Lin + Lout : 0u);
        const u64 worst = ceil_div32(longest, blk);
        u32 st = 0;
        if (rt.usable <= mi.w_gpu) st |= GUIDE_ST_WEIGHTS;
        if (worst > blocks_total) st |= GUIDE_ST_KV;
        if ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) st |= GUIDE_ST_HEADS;
        const u32 fit = clamp_u32(blocks_total / worst);

        // ---- constants of the per-iteration attention terms ----
        // Largest summed context this config can see: every resident at its full length plus one.
        const u64 ctx_max = (u64)b * ((u64)longest + 1);
        const u64 lim53 = 1ull << 53;
        const u64 xw = rt.flash ? 0ull : (u64)m.nh * m.ab;                 // score-matrix bytes per unit of A
        const bool exact53 = 2 * (u64)m.H * ctx_max < lim53 && 5 * (u64)m.nh * ctx_max < lim53 &&
                             (u64)b * m.H * m.ab + ctx_max * ((u64)m.Dkv * m.kvb + xw) < lim53 && 2 * xw * ctx_max < lim53;
        __syncwarp();                                                      // the previous config's last reads of the constants
        if (lane == 0) {
            sl.cst[0] = log2_rule_factor(t, tp_model); sl.cst[1] = (double)m.N;
            sl.cst[2] = rt.inv_c[CLS_ATTN]; sl.cst[3] = rt.inv_m[CLS_ATTN];
            sl.cst[4] = (double)(2 * (u64)m.H) * inv_tt;                   // F9  = ctx * 2H / t
            sl.cst[5] = (double)((u64)m.Dkv * m.kvb + xw) * inv_tt;        // KV read + score bytes per context token / t
            sl.cst[6] = (double)(5 * (u64)m.nh) * inv_tt;                  // F10 = ctx * 5 n_h / t
            sl.cst[7] = (double)(2 * xw) * inv_tt;                         // B10 = ctx * 2 n_h a_b / t (0 with flash)
        }
        __syncwarp();

        double clock = 0.0, dec_time = 0.0, csum_d = 0.0;   // csum_d mirrors csum when exact53
        u64 dec_tok = 0, n_iters = 0, n_req_iters = 0, free_blocks = blocks_total, csum = 0;
        u32 next = 0, high_water = 0, nrun = 0, n_new = 0;
        u32 D = 0, Dmod = 0, min_rem = NO_COMPLETION;
        const bool use_hist = blk > 1 && blk <= HIST;
        const bool burst_ok = exact53 && (blk == 1 || use_hist);
        const u32 lmod = lane % blk, m32 = 32u % blk;     // lane and warp width modulo the block size
        // block sizes are powers of two as a rule: their divisions are shifts
        const u32 blk_shift = (blk & (blk - 1)) == 0 ? (u32)__ffs(blk) - 1 : 0xFFFFFFFFu;
        auto divb = [&](u32 x) { return blk_shift != 0xFFFFFFFFu ? x >> blk_shift : x / blk; };
        auto modb = [&](u32 x) { return blk_shift != 0xFFFFFFFFu ? x & (blk - 1) : x % blk; };
        auto blocks_of = [&](u32 tokens) { return divb(tokens + blk - 1); };
        const u64 max_iters = max_iters_opt ? max_iters_opt : 64 * (tr.sum_out + (u64)tr.n_zero * Lout) + 4 * (u64)n;
        // cached while the running count stays the same
        u32 dc_n = 0;
        double dc_fix = 0.0, dc_comm = 0.0, dc_head = 0.0, dc_tha = 0.0, dc_nd = 0.0;
        u32 dc_w0 = 0x80000000u;         // first resident count of the window of decode terms in shared memory (none yet)
        u64 pre_T = 0, pre_A = 0;        // prompt tokens (and their squares) admitted since the last prompt pass
        // the head of the waiting queue: its arrival time and the blocks it needs
        double arr_next = 0.0;
        u32 need_next = 0, in_next = 0, g_next = 0;              // ... its prompt length (0: the config's) and the tokens kept from before an eviction
        auto refresh_head = [&]() {
            while (next < high_water && (gen[next] & GEN_DONE)) next++;
            if (next < n) {
                arr_next = __ldg(tr.arrival + next);
                g_next = next < high_water ? gen[next] : 0u;
                in_next = __ldg(tr.in_len + next);
                need_next = blocks_of((in_next ? in_next : Lin) + g_next);
            } else {
                arr_next = inf; need_next = 0;
            }
        };
        if (!st) {
            for (u32 i = lane; i < HIST; i += 32) sl.hist[i] = 0;
            if (sc_ok) {
                // what a prompt pass needs, next to the warp: the (model, TP degree) factors and the pair's rates
                const double *scg = reinterpret_cast<const double *>(s.stage_consts + (size_t)(tp_model ? s.n_t : c.t) * s.n_m + c.m);
                sl.sc[lane] = scg[lane];
                if (lane < 10) sl.rate[lane] = s.rate10[(size_t)(c.h * s.n_f + c.f) * 10 + lane];
            }
            refresh_head();
            __syncwarp();
        }

        while (!st) {
            // ---- 1. admit in arrival order, no overtaking ----
            if (nrun < b && arr_next <= clock && need_next <= free_blocks) {
                do {
                    const u32 g = g_next;
                    u32 in = in_next, out = Lout;
                    if (in == 0) in = Lin;
                    else out = __ldg(tr.out_len + next);
                    free_blocks -= need_next;
                    if (lane == 0) {
                        sl.req[nrun] = next;
                        sl.base[nrun] = in + g;                           // prompt + tokens to recompute
                        sl.fin[nrun] = out - g;
                        sl.meta[nrun] = (unsigned char)(M_NEEDS_PREFILL | (g == 0 ? M_FIRST : 0u));
                    }
                    pre_T += (u64)(in + g); pre_A += (u64)(in + g) * (in + g);
                    nrun++; n_new++; next++;
                    if (next > high_water) high_water = next;
                    refresh_head();
                } while (nrun < b && arr_next <= clock && need_next <= free_blocks);
                __syncwarp();
            }
            // ---- 2. nothing to run: finished, or jump to the next arrival ----
            if (nrun == 0) {
                if (next >= n) break;
                if (arr_next > clock) { clock = arr_next; continue; }
                st |= GUIDE_ST_ITER;                                   // cannot happen when each request fits alone
                break;
            }
            if (n_iters >= max_iters) { st |= GUIDE_ST_ITER; break; }
            // ---- 3./4. build the iteration (prompts first, everything else stalls) and advance the clock ----
            bool any_done;
            if (n_new > 0) {
                const u64 T = pre_T, A = pre_A;          // summed at admission: tokens and tokens squared of the new prompts
                pre_T = 0; pre_A = 0;
                double t_iter;
                if (sc_ok) {
                    // the same operations on doubles (exact for this config), the factors read from shared memory as they are used
                    const StageConst &sc = *reinterpret_cast<const StageConst *>(sl.sc);
                    const double Td = (double)(long long)T, Ad = (double)(long long)A;
                    const StageFixed sf = stage_fixed<TIME_SUM>(sc, sl.rate, Td, (double)n_new);
                    const double xw = rt.flash ? 0.0 : sc.xb;
                    const double t9 = task_time<TIME_SUM>(Ad * c_f9, ((Td * sc.ha + Td * sc.kv) + Ad * xw) * sc.inv_t, icA, imA);
                    const double t10 = task_time<TIME_SUM>(Ad * c_f10, Ad * c_b10, icA, imA);
                    t_iter = combine_phase(sf.fix, (t9 + t10) + t9, sf.comm, sf.head, 1.0, Nd, rt.tovh, lf);
                } else {
                    TaskTab kt;
                    build_fixed_tasks(m, tt, T, n_new, 1, kt);
                    build_attn_tasks(m, tt, T, A, T, kt);
                    t_iter = eval_phase<TIME_SUM>(kt, rt, Nd, lf);
                }
                const double after = clock + t_iter;
                u32 local_min = NO_COMPLETION;
                for (u32 base = nrun - n_new; base < nrun; base += 32) {     // admissions append: the new ones are the last slots
                    const u32 k = base + lane;
                    if (k < nrun) {
                        const u32 mt = sl.meta[k];
                        if (mt & M_NEEDS_PREFILL) {
                            if (mt & M_FIRST) first[sl.req[k]] = after;    // first token of this request
                            const u32 q = sl.base[k], left = sl.fin[k] - 1;
                            u32 ph = 0;
                            if (use_hist) {
                                ph = modb(q) + blk - Dmod;                  // (cache - D) mod block
                                if (ph >= blk) ph -= blk;
                                atomicAdd(&sl.hist[ph], 1u);
                            }
                            sl.base[k] = q - D;
                            sl.fin[k] = D + left;
                            sl.meta[k] = (unsigned char)ph;
                            local_min = min(local_min, left);
                        }
                    }
                }
                __syncwarp();
                min_rem = min(min_rem, warp_min(local_min));
                any_done = min_rem == 0;
                csum += T;
                csum_d = (double)(long long)csum;
                n_req_iters += n_new;
                n_new = 0;
                clock = after;
                n_iters++;
            } else {
                // every sequence whose last block is full needs one more block
                u32 needed;
                if (blk == 1) needed = nrun;
                else if (use_hist) needed = sl.hist[Dmod == 0 ? 0 : blk - Dmod];
                else {
                    needed = 0;
                    for (u32 base = 0; base < nrun; base += 32) {
                        const u32 k = base + lane;
                        needed += __popc(__ballot_sync(0xFFFFFFFFu, k < nrun && modb(sl.base[k] + D) == 0));
                    }
                }
                if (needed > free_blocks) {
                    while (needed > free_blocks) {                     // evict the youngest, recompute later
                        const u32 v = nrun - 1;
                        const u32 cv = sl.base[v] + D, rq = sl.req[v], rem = sl.fin[v] - D, ph = sl.meta[v] & M_PHASE;
                        free_blocks += blocks_of(cv);
                        if (modb(cv) == 0) needed--;
                        csum -= cv;
                        const u32 out = __ldg(tr.in_len + rq) ? __ldg(tr.out_len + rq) : Lout;
                        __syncwarp();
                        if (lane == 0) {
                            gen[rq] = out - rem;
                            if (use_hist) sl.hist[ph] -= 1;
                        }
                        nrun--;
                        next = rq;
                    }
                    __syncwarp();
                    refresh_head();
                    csum_d = (double)(long long)csum;
                }
                free_blocks -= needed;
                if (dc_n != nrun) {
                    if (nrun - dc_w0 >= 32u) {
                        // The terms of a decode iteration that depend on the resident count only, for 32
                        // neighbouring counts at once (one per lane): the count moves by one or two per
                        // event, so most events find theirs in the window.
                        dc_w0 = nrun > 16 ? nrun - 16 : 1;
                        const u32 nl = dc_w0 + lane;
                        TaskTab kt;
                        build_fixed_tasks(m, tt, nl, nl, 1, kt);
                        __syncwarp();
                        sl.dterm[lane][0] = eval_fixed<TIME_SUM>(kt, rt);
                        sl.dterm[lane][1] = eval_comm(kt, rt);
                        sl.dterm[lane][2] = eval_head<TIME_SUM>(kt, rt);
                        sl.dterm[lane][3] = (double)((u64)nl * m.H * m.ab) * inv_tt;
                        __syncwarp();
                    }
                    dc_n = nrun;
                    const double2 d01 = *(const double2 *)&sl.dterm[nrun - dc_w0][0], d23 = *(const double2 *)&sl.dterm[nrun - dc_w0][2];
                    dc_fix = d01.x; dc_comm = d01.y; dc_head = d23.x; dc_tha = d23.y;
                    dc_nd = (double)nrun;
                }
                if (burst_ok) {
                    // A run of decode iterations up to the next event.  Nothing per request is
                    // touched; integer counters are settled once after the run.  The next
                    // iteration's time is computed before the clock-dependent exit test so the two
                    // dependency chains overlap.
                    const u64 cap_left = max_iters - n_iters;
                    const u32 steps_max = (u32)min((u64)min_rem, cap_left);
                    const u32 fb0 = (u32)min(free_blocks, (u64)0xFFFFFFFFu);
                    u32 fb = fb0, it = 0;
                    u32 hidx = Dmod + 1 == blk ? 0 : blk - (Dmod + 1);     // histogram bin of the next iteration's needers
                    const bool room = nrun < b;
                    const double nd = dc_nd, cd0 = csum_d;
                    // The iterations of a run do not depend on one another except through the clock:
                    // the summed context of the i-th is cd0 + i * nd (exact), so the 32 lanes compute
                    // the times of 32 consecutive iterations at once; which of them ends the run on
                    // block counts is a prefix sum over the histogram bins, and the clock is then
                    // advanced one iteration after the other (same order of additions as a scalar
                    // loop), watching for the arrival of the queue head where it could come in.
                    for (;;) {
                        const u32 nb = min(32u, steps_max - it);
                        const double t_k = decode_time<TIME_SUM>(cd0 + nd * ((double)it + (double)(lane + 1)), c_f9, dc_tha, c_kvx, c_f10, c_b10,
                                                                 icA, imA, dc_fix, dc_comm, dc_head, Nd, rt.tovh, lf);
                        // blocks the residents need before the iteration after lane's, and what is free by then
                        u32 need_k = 0;
                        if (lane < nb) need_k = blk == 1 ? nrun : sl.hist[hidx >= lmod ? hidx - lmod : hidx + blk - lmod];
                        // Usually the free blocks cover the whole batch and the queue head's need: then only the
                        // completion count can end the run on integers, and what is free afterwards is one sum.
                        const u32 total = __reduce_add_sync(0xFFFFFFFFu, need_k);
                        const bool plenty = (u64)total + need_next <= fb;
                        u32 fb_k = 0, stops, last, watch;
                        if (plenty) {
                            last = nb - 1;
                            stops = steps_max - it <= 32u ? 1u << last : 0u;
                            watch = room ? 0xFFFFFFFFu >> (31 - last) : 0u;
                        } else {
                            u32 incl = need_k;
                            #pragma unroll
                            for (int d = 1; d < 32; d <<= 1) {
                                const u32 up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                                if (lane >= (u32)d) incl += up;
                            }
                            fb_k = fb - (incl - need_k);                  // wraps only behind a lane that already stops
                            stops = __ballot_sync(0xFFFFFFFFu, lane < nb && (it + lane + 1 == steps_max || need_k > fb_k));
                            last = stops ? (u32)__ffs(stops) - 1 : 31u;   // a completion, the cap or an eviction follows it
                            watch = __ballot_sync(0xFFFFFFFFu, room && need_next <= fb_k) & (0xFFFFFFFFu >> (31 - last));
                        }
                        sl.tbuf[lane] = t_k;
                        __syncwarp();
                        // the clock, one iteration after the other: four per trip, the arrival tests of a trip taken together
                        u32 k = 0;
                        bool arrived = false;
                        const u32 cnt = last + 1;
                        double2 va = *(const double2 *)&sl.tbuf[0], vb = *(const double2 *)&sl.tbuf[2];
                        while (k + 4 <= cnt) {
                            // the next trip's times are loaded ahead of this trip's additions (past the end: wraps, unused)
                            const double2 na = *(const double2 *)&sl.tbuf[(k + 4) & 31], nb2 = *(const double2 *)&sl.tbuf[(k + 6) & 31];
                            const double c1 = clock + va.x, c2 = c1 + va.y, c3 = c2 + vb.x, c4 = c3 + vb.y;
                            const double d1 = dec_time + va.x, d2 = d1 + va.y, d3 = d2 + vb.x, d4 = d3 + vb.y;
                            const u32 wbits = (watch >> k) & 15u;
                            u32 hit = 0;
                            if (wbits)
                                hit = ((u32)(arr_next <= c1) | ((u32)(arr_next <= c2) << 1) | ((u32)(arr_next <= c3) << 2) |
                                       ((u32)(arr_next <= c4) << 3)) & wbits;
                            if (hit) {                                             // the queue head can come in after one of the four
                                const u32 f = (u32)__ffs(hit) - 1;
                                clock = f == 0 ? c1 : f == 1 ? c2 : f == 2 ? c3 : c4;
                                dec_time = f == 0 ? d1 : f == 1 ? d2 : f == 2 ? d3 : d4;
                                k += f;
                                arrived = true;
                                break;
                            }
                            clock = c4; dec_time = d4;
                            va = na; vb = nb2;
                            k += 4;
                        }
                        if (!arrived) {
                            for (; k < cnt; k++) {
                                const double v = sl.tbuf[k];
                                clock = clock + v;
                                dec_time = dec_time + v;
                                if (((watch >> k) & 1u) && arr_next <= clock) { arrived = true; break; }
                            }
                            if (!arrived) k = last;
                        }
                        it += k + 1;
                        __syncwarp();
                        if (stops || arrived) {
                            fb = plenty ? fb - __reduce_add_sync(0xFFFFFFFFu, lane < k ? need_k : 0u) : __shfl_sync(0xFFFFFFFFu, fb_k, k);
                            break;
                        }
                        fb = plenty ? fb - total : __shfl_sync(0xFFFFFFFFu, fb_k - need_k, 31);
                        hidx = hidx >= m32 ? hidx - m32 : hidx + blk - m32;
                    }
                    const double cd = cd0 + nd * (double)it;
                    const u64 tok = (u64)it * nrun;
                    D += it;
                    Dmod += it < blk ? it : modb(it);           // short runs are the rule
                    if (Dmod >= blk) Dmod -= blk;
                    csum += tok; csum_d = cd;
                    dec_tok += tok; n_req_iters += tok; n_iters += it;
                    min_rem -= it;
                    free_blocks -= fb0 - fb;
                    any_done = min_rem == 0;
                } else {
                    const u64 ctx = csum + nrun;                       // cached tokens + the new one, summed
                    const u64 X = xw * ctx;
                    const double F9 = cvt(2 * (u64)m.H * ctx) * inv_tt;
                    const double B9 = cvt((u64)nrun * m.H * m.ab + ctx * m.Dkv * m.kvb + X) * inv_tt;
                    const double F10 = cvt(5 * (u64)m.nh * ctx) * inv_tt;
                    const double B10 = cvt(2 * X) * inv_tt;
                    const double t9 = task_time<TIME_SUM>(F9, B9, icA, imA);
                    const double t10 = task_time<TIME_SUM>(F10, B10, icA, imA);
                    const double s_att = (t9 + t10) + t9;
                    const double t_iter = combine_phase(dc_fix, s_att, dc_comm, dc_head, 1.0, Nd, rt.tovh, lf);
                    D++;
                    Dmod = Dmod + 1 == blk ? 0 : Dmod + 1;
                    csum += nrun;
                    dec_time = dec_time + t_iter;
                    dec_tok += nrun;
                    n_req_iters += nrun;
                    n_iters++;
                    min_rem--;
                    any_done = min_rem == 0;
                    clock = clock + t_iter;
                }
            }
            // ---- 5. retire finished sequences, keep the rest in order ----
            if (any_done) {
                __syncwarp();
                u32 kept = 0, local_min = NO_COMPLETION;
                u64 freed = 0, gone = 0;
                const u32 n_before = nrun;
                for (u32 base = 0; base < n_before; base += 32) {
                    const u32 k = base + lane;
                    const bool valid = k < n_before;
                    u32 rq = 0, bs = 0, fn = 0, mt = 0;
                    if (valid) { rq = sl.req[k]; bs = sl.base[k]; fn = sl.fin[k]; mt = sl.meta[k]; }
                    const u32 rem = fn - D;
                    const bool done = valid && rem == 0;
                    if (done) {
                        const u32 cv = bs + D;
                        gen[rq] = GEN_DONE;
                        tpot[rq] = clock;              // time of its last token; the results turn it into time per output token
                        freed += blocks_of(cv);
                        gone += cv;
                        if (use_hist) atomicSub(&sl.hist[mt & M_PHASE], 1u);
                    }
                    const bool keep = valid && !done;
                    if (keep) local_min = min(local_min, rem);
                    const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);
                    __syncwarp();
                    if (keep) {
                        const u32 d = kept + __popc(ballot & lt_mask);
                        sl.req[d] = rq; sl.base[d] = bs; sl.fin[d] = fn; sl.meta[d] = (unsigned char)mt;
                    }
                    kept += __popc(ballot);
                    __syncwarp();
                }
                free_blocks += warp_sum(freed);
                csum -= warp_sum(gone);
                min_rem = warp_min(local_min);
                nrun = kept;
                csum_d = (double)(long long)csum;
            }
        }

        // ---- results ----
        write_trace_results(o, j, n, st, fit, clock, dec_time, dec_tok, n_iters, n_req_iters, rt.price * (double)t, tr, Lout,
                                  first, tpot, lane);
        __syncwarp();
    }
}

// Configs whose framework schedules by split and fuse (trace_fuse.cuh): the same work loop, memory
// check and results as k_trace_sim around fuse_schedule.  Configs of the other policy are skipped
// here and simulated there.
template <int TIME_SUM>
__global__ void __launch_bounds__(SIM_THREADS, FUSE_MIN_BLOCKS)
k_trace_fuse(DSpace s, DTrace tr, Range r, int tp_model, u64 max_iters_opt, guide_outputs o, u32 *counter,
             unsigned char *scratch, size_t per_warp, u32 gen_bytes, u32 first_bytes, int reorder) {
    __shared__ FuseSlots sh[SIM_WARPS_PER_BLOCK];
    const u32 lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const u32 warp_global = blockIdx.x * SIM_WARPS_PER_BLOCK + wib;
    unsigned char *mine = scratch + (size_t)warp_global * per_warp;
    u32 *gen = (u32 *)mine;
    double *first = (double *)(mine + gen_bytes);
    double *tpot = (double *)(mine + gen_bytes + first_bytes);
    const u32 n = tr.n;
    for (;;) {
        u64 w = 0;
        if (lane == 0) w = atomicAdd(counter, 1u);
        w = __shfl_sync(0xFFFFFFFFu, w, 0);
        if (w >= r.count) break;
        const u64 idx = reorder ? work_to_index(s, w, true) : r.first + w;
        const u64 j = idx - r.first;
        const Cfg c = decode_index(s, idx);
        const DRate *rp = s.rates + (c.h * s.n_f + c.f);
        if (rp->policy != GUIDE_POLICY_SPLIT_FUSE) continue;
        const DModel *mp = s.models + c.m;
        const u32 t = s.tp[c.t], b = s.batch[c.b];
        const uint2 pr = s.pairs[c.l];
        const u32 Lin = pr.x, Lout = pr.y, blk = rp->kv_block;
        const MemInfo mi = mem_info(*mp, t);
        // ---- what fits (Sec. 3.2 Step 1) ----
        const u64 usable = rp->usable;
        const u64 blocks_total = usable > mi.w_gpu ? floor_div(usable - mi.w_gpu, (u64)blk * mi.kv_tok) : 0;
        const u32 longest = max(tr.max_tokens, tr.any_zero ? Lin + Lout : 0u);
        const u64 worst = ceil_div32(longest, blk);
        u32 st = 0;
        if (usable <= mi.w_gpu) st |= GUIDE_ST_WEIGHTS;
        if (worst > blocks_total) st |= GUIDE_ST_KV;
        if ((mp->nh & (t - 1)) != 0 || (mp->nkv & (t - 1)) != 0) st |= GUIDE_ST_HEADS;
        const u32 fit = clamp_u32(blocks_total / worst);
        // prompt chunks take iterations too: the default backstop counts prompt tokens as well
        const u64 sched_tokens = tr.sum_out + tr.sum_in + (u64)tr.n_zero * ((u64)Lin + Lout);
        const u64 max_iters = max_iters_opt ? max_iters_opt : 64 * sched_tokens + 4 * (u64)n;
        FuseResult fr = {0.0, 0.0, 0, 0, 0};
        if (!st) {
            __syncwarp();
            // stage tables from doubles where every count of the config stays exact in binary64
            const double *scg = lanes_exact(*mp, tp_model ? 1u : t, b, longest)
                                    ? reinterpret_cast<const double *>(s.stage_consts + (size_t)(tp_model ? s.n_t : c.t) * s.n_m + c.m)
                                    : nullptr;
            st |= fuse_schedule<TIME_SUM>(mp, rp, tr.arrival, tr.in_len, tr.out_len, n, tp_model ? 1u : t, b, Lin, Lout, blocks_total,
                                          log2_rule_factor(t, tp_model), max_iters, sh[wib], gen, first, tpot, scg);
            fr = sh[wib].res;
        }
        write_trace_results(o, j, n, st, fit, fr.clock, fr.dec_time, fr.dec_tok, fr.n_iters, fr.n_req_iters,
                                   rp->price * (double)t, tr, Lout, first, tpot, lane);
        __syncwarp();
    }
}

// Prompt-first configs, one per lane (trace_lanes.cuh), max batch in [minb, maxb]; everything else is
// skipped here and simulated by another launch of this kernel or by k_trace_sim.
template <int TIME_SUM, int UNROLL>
__global__ void __launch_bounds__(LANE_MAX_THREADS, 4)
k_trace_lanes(DSpace s, DTrace tr, Range r, int tp_model, u64 max_iters_opt, guide_outputs o, unsigned long long *counter,
              unsigned char *scratch, size_t per_lane, u32 gen_bytes, u32 first_bytes, int reorder, u32 minb, u32 maxb,
              u32 hist_n, u32 lanes_used, u32 round_len) {
    extern __shared__ __align__(16) unsigned char lane_smem[];
    const u32 lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    unsigned char *wsm = lane_smem + (size_t)wib * lanes_used * (12 * maxb + 4 * hist_n);
    const u32 n = tr.n;
    lanes_simulate<TIME_SUM, UNROLL>(s, tr, r, tp_model, max_iters_opt, counter, scratch, per_lane, gen_bytes, first_bytes, reorder, minb,
                             maxb, hist_n, lanes_used, round_len, wsm,
                             [&](u64 j, u32 st, u32 fit, double clock, double dec_time, u64 dec_tok, u64 n_iters, u64 n_req_iters,
                                 double cost_hr, u32 Lout, double *first, double *tpot) {
                                 write_lane_results(o, j, n, st, fit, clock, dec_time, dec_tok, n_iters, n_req_iters, cost_hr,
                                                    tr, Lout, first, tpot, lane);
                                 __syncwarp();
                             });
}

// The lane kernel is launched once per class of max batch: the slots of a lane take 12 bytes per
// resident request, so a launch for large batches gives a warp fewer lanes.
// round: decode iterations a lane may run between two event phases (events come more often with larger batches)
// unroll: iterations per trip of the run loop (4: long runs, where a lane's own chain latency is the limit)
// min_configs: the class is launched only when the space has at least this many of its configs.  The
// lane kernel handles events one lane at a time and its run loop is one dependent chain per lane, so it
// needs most lanes of every resident warp busy to beat the warp-per-config kernel, whose run loop
// spreads the iterations of one config over the lanes (measured on workload 3, max batch 6-16: 4,096
// configs 110 ms in lanes against 42 ms in warps; 32,768 configs 215 against 283 ms; max batch 24-64
// on workload 4, 262,144 configs: 117 against about 220 ms).
struct LaneClass { u32 minb, maxb, lanes, round, unroll; u64 min_configs; };
#ifndef LANE_CLASS0_MIN_WAVES
#define LANE_CLASS0_MIN_WAVES 8
#endif
static const LaneClass LANE_CLASSES[LANE_N_CLASSES] = {{1, 16, 32, 128, 4, (u64)LANE_MAX_WARPS * LANE_CLASS0_MIN_WAVES},
                                                       {17, 64, 32, 32, 1, (u64)LANE_MAX_WARPS * 32},
                                                       {65, GUIDE_TRACE_MAX_BATCH, 8, 8, 1, ~0ull}};

typedef void (*LaneKernel)(DSpace, DTrace, Range, int, u64, guide_outputs, unsigned long long *, unsigned char *, size_t, u32, u32,
                           int, u32, u32, u32, u32, u32);
template <int TIME_SUM>
static LaneKernel lane_kernel(u32 unroll) {
    return unroll == 4 ? (LaneKernel)k_trace_lanes<TIME_SUM, 4> : (LaneKernel)k_trace_lanes<TIME_SUM, 1>;
}
static constexpr u32 LANE_BLOCK_WARPS = 4;
static constexpr size_t LANE_SMEM_LIMIT = 112 * 1024;

static size_t lane_block_smem(const LaneClass &c, u32 lanes, u32 hist_n) {
    return (size_t)LANE_BLOCK_WARPS * lanes * (12 * c.maxb + 4 * hist_n);
}

LaneHints lane_hints(const guide_space &s) {
    LaneHints h{};
    h.hist_n = 1;
    u64 n_fw = 0;
    for (const guide_fw &f : s.fw)
        if (f.policy == GUIDE_POLICY_PREFILL_FIRST && f.kv_block <= LANE_HIST_MAX) {
            n_fw++;
            h.hist_n = std::max(h.hist_n, f.kv_block);
        }
    const u64 per_b = (u64)s.models.size() * s.hw.size() * n_fw * s.tp.size() * s.pairs.size();
    u64 all[LANE_N_CLASSES] = {};
    for (uint32_t b : s.batch)
        for (u32 c = 0; c < LANE_N_CLASSES; c++)
            if (b >= LANE_CLASSES[c].minb && b <= LANE_CLASSES[c].maxb) all[c] += per_b;
    // Classes are taken from the first one up, without gaps (the warp-per-config kernel leaves out every
    // max batch up to the last launched class's limit), each only when it is large enough to pay.
    // GUIDE_LANE_MIN_CONFIGS in the environment replaces the thresholds of the first two classes (the
    // tests set it to 1 so that small spaces reach the lane kernel too); read once per process.
    static const char *forced = getenv("GUIDE_LANE_MIN_CONFIGS");
    for (u32 c = 0; c < LANE_N_CLASSES; c++) {
        const u64 need = (forced && c < 2) ? strtoull(forced, nullptr, 10) : LANE_CLASSES[c].min_configs;
        if (all[c] < need || all[c] == 0) break;
        h.class_configs[c] = all[c];
    }
    return h;
}

// The kernels of a call run one after the other and share the region: a slice per resident warp of
// the warp-per-config kernels, a slice per lane that can get a config in a launch of the lane kernel
// (a launch rounds its warps up to whole blocks: one block of slack covers that).
size_t trace_workspace_bytes(u32 n_req, const LaneHints &hints) {
    size_t slices = SIM_MAX_WARPS;
    for (u32 c = 0; c < LANE_N_CLASSES; c++) {
        const u64 lanes = LANE_CLASSES[c].lanes;
        slices = std::max<size_t>(slices, std::min<u64>((u64)LANE_MAX_WARPS * lanes,
                                                        hints.class_configs[c] + LANE_BLOCK_WARPS * lanes));
    }
    return 256 + slices * per_warp_bytes(n_req);
}

struct LanePlan { u32 blocks, lanes_used; size_t smem; };

template <int TIME_SUM>
static int plan_lanes(const DSpace &s, const LaneHints &h, Range r, u32 cls, LanePlan *p) {
    const LaneClass &c = LANE_CLASSES[cls];
    p->blocks = 0; p->lanes_used = c.lanes; p->smem = 0;
    if (h.class_configs[cls] == 0) return GUIDE_OK;
    static std::mutex mu;
    static bool opted[64] = {};
    int dev = 0;
    GUIDE_CUDA(cudaGetDevice(&dev));
    {
        std::lock_guard<std::mutex> lock(mu);
        if (dev < 64 && !opted[dev]) {
            for (u32 u : {1u, 4u})
                GUIDE_CUDA(cudaFuncSetAttribute(lane_kernel<TIME_SUM>(u), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)LANE_SMEM_LIMIT));
            opted[dev] = true;
        }
    }
    // configs of this launch among the range: all of the class for a whole space, else at most the range
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    const u64 mine = r.count == total ? h.class_configs[cls] : std::min<u64>(r.count, h.class_configs[cls]);
    // The kernel is bound by the latency of each lane's own chain, so warps are worth more than lanes:
    // as few lanes per warp as still lets every config be resident at once (fewer lanes also need less
    // shared memory per block, so more blocks fit; two rounds settle that).
    const LaneKernel kern = lane_kernel<TIME_SUM>(c.unroll);
    const u64 fit = LANE_SMEM_LIMIT / lane_block_smem(c, 1, h.hist_n);      // lanes whose slots fit a block's shared memory (>= 8)
    u64 lanes = std::min<u64>(c.lanes, fit), resident_warps = 1;
    for (int round = 0; round < 3; round++) {
        int per_sm = 0;
        GUIDE_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, LANE_BLOCK_WARPS * 32,
                                                                 lane_block_smem(c, (u32)lanes, h.hist_n)));
        if (per_sm < 1) per_sm = 1;
        resident_warps = std::min<u64>((u64)num_sms() * per_sm * LANE_BLOCK_WARPS, LANE_MAX_WARPS);
        lanes = std::max<u64>(1, std::min<u64>(std::min<u64>(c.lanes, fit), (mine + resident_warps - 1) / resident_warps));
    }
    p->lanes_used = (u32)lanes;
    p->smem = lane_block_smem(c, p->lanes_used, h.hist_n);
    const u64 warps = std::min<u64>(resident_warps, (mine + p->lanes_used - 1) / p->lanes_used);
    p->blocks = (u32)((warps + LANE_BLOCK_WARPS - 1) / LANE_BLOCK_WARPS);
    return GUIDE_OK;
}

template <int TIME_SUM>
static int launch_one(const DSpace &s, const DTrace &t, Range r, int tp_model, u64 max_iters, const guide_outputs &o,
                      void *ws, size_t ws_bytes, cudaStream_t st, u32 policies, const LaneHints &hints) {
    const size_t pw = per_warp_bytes(t.n);
    const u32 gen_bytes = (u32)(((size_t)t.n * 4 + 255) / 256 * 256);
    const u32 first_bytes = (u32)(((size_t)t.n * 8 + 255) / 256 * 256);
    // resident warps: as many as the SMs hold, never more than the workspace was sized for
    int per_sm = 0;
    GUIDE_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_trace_sim<TIME_SUM>, SIM_THREADS, 0));
    if (per_sm < 1) per_sm = 1;
    u32 blocks = (u32)num_sms() * (u32)per_sm;
    blocks = std::min<u32>(blocks, SIM_MAX_WARPS / SIM_WARPS_PER_BLOCK);
    blocks = (u32)std::min<u64>(blocks, (r.count + SIM_WARPS_PER_BLOCK - 1) / SIM_WARPS_PER_BLOCK);
    int per_sm_f = 0;
    GUIDE_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_f, k_trace_fuse<TIME_SUM>, SIM_THREADS, 0));
    if (per_sm_f < 1) per_sm_f = 1;
    u32 blocks_f = (u32)num_sms() * (u32)per_sm_f;
    blocks_f = std::min<u32>(blocks_f, SIM_MAX_WARPS / SIM_WARPS_PER_BLOCK);
    blocks_f = (u32)std::min<u64>(blocks_f, (r.count + SIM_WARPS_PER_BLOCK - 1) / SIM_WARPS_PER_BLOCK);
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    const int reorder = r.first == 0 && r.count == total;
    unsigned char *scratch = (unsigned char *)ws + 256;
    // one kernel per scheduling policy present in the space; each skips the other's configs.  The
    // prompt-first configs with a small max batch go to the lane kernel first (the long schedules).
    if ((policies & 3) && 256 + (size_t)std::max(blocks, blocks_f) * SIM_WARPS_PER_BLOCK * pw > ws_bytes)
        return fail(GUIDE_ERR_WORKSPACE, "workspace too small for the resident warps");
    if (policies & 1) {
        u32 lane_maxb = 0;
        for (u32 cls = 0; cls < LANE_N_CLASSES; cls++) {
            const LaneClass &lc = LANE_CLASSES[cls];
            LanePlan lp;
            int rc = plan_lanes<TIME_SUM>(s, hints, r, cls, &lp);
            if (rc) return rc;
            if (lp.blocks == 0) continue;
            // every lane that can get a config has its slice inside the workspace
            if (256 + (size_t)lp.blocks * LANE_BLOCK_WARPS * lp.lanes_used * pw > ws_bytes)
                return fail(GUIDE_ERR_WORKSPACE, "workspace too small for the lane kernel's %u blocks", lp.blocks);
            GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
            lane_kernel<TIME_SUM>(lc.unroll)<<<lp.blocks, LANE_BLOCK_WARPS * 32, lp.smem, st>>>(
                s, t, r, tp_model, max_iters, o, (unsigned long long *)ws, scratch, pw, gen_bytes, first_bytes, reorder,
                lc.minb, lc.maxb, hints.hist_n, lp.lanes_used, lc.round);
            GUIDE_CUDA(cudaGetLastError());
            lane_maxb = std::max(lane_maxb, lc.maxb);
        }
        // always launched: the lane kernel leaves it the configs whose counts do not stay below 2^53
        // or whose block size the phase histogram does not cover
        GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
        k_trace_sim<TIME_SUM><<<blocks, SIM_THREADS, 0, st>>>(s, t, r, tp_model, max_iters, o, (u32 *)ws, scratch, pw,
                                                             gen_bytes, first_bytes, reorder, lane_maxb, hints.hist_n);
        GUIDE_CUDA(cudaGetLastError());
    }
    if (policies & 2) {
        GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
        k_trace_fuse<TIME_SUM><<<blocks_f, SIM_THREADS, 0, st>>>(s, t, r, tp_model, max_iters, o, (u32 *)ws, scratch, pw,
                                                                gen_bytes, first_bytes, reorder);
        GUIDE_CUDA(cudaGetLastError());
    }
    return GUIDE_OK;
}

// policies: bit 0 = some framework schedules prompt-first, bit 1 = some by split and fuse
int launch_trace_sim(const DSpace &s, const DTrace &t, Range r, int time_model, int tp_model, u64 max_iters,
                     const guide_outputs &o, void *ws, size_t ws_bytes, cudaStream_t st, u32 policies, const LaneHints &hints) {
    if (r.count > 0xFFFFFFF0ull) return fail(GUIDE_ERR_UNSUPPORTED, "at most 2^32 - 16 configs per trace launch");
    return time_model ? launch_one<1>(s, t, r, tp_model, max_iters, o, ws, ws_bytes, st, policies, hints)
                      : launch_one<0>(s, t, r, tp_model, max_iters, o, ws, ws_bytes, st, policies, hints);
}

}  // namespace guide
