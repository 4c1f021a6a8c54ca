// Trace-driven simulation with one LANE per config (prompt-first policy), for configs whose max batch
// is small, when a space has enough of them to fill most lanes of every resident warp.  Those are the
// long schedules - with a max batch of 1 every output token of the trace is its own iteration - and
// a scheduler event (admission, prompt pass, completion) handles one or two requests, so a warp that
// steps one config has most of its lanes idle at events.  Here every lane of a warp steps its own config.
//
// A warp alternates between two phases so that its lanes stay on the same instructions:
//   - run: every lane that is between events advances its config by up to round_len decode iterations
//     (one scalar chain per lane; the clock is advanced by the same additions in the same order as in
//     the warp-per-config kernel);
//   - events: every lane whose run ended (a completion, a block shortage, room for the head of the
//     queue) makes scheduler passes - settle the run, retire, admit, a prompt pass, evictions, refresh
//     of the cached stage terms - until it is ready to run again or its trace is finished.
// Lanes whose run ended early wait for the end of the round, which is what keeps the heavy event
// code from being issued for one lane at a time.  A finished config's results are reduced by the
// whole warp (means in request order, percentiles by a bitonic sort) and the lane takes the next
// config from the work counter.
//
// Resident requests of a lane live in shared memory, slot k of lane l at [k][l] (a launch for large
// max batches uses fewer lanes per warp so that the slots still fit), with the same invariants as
// the warp-per-config kernel: base = cache - D, fin = D at completion, a histogram of
// (cache - D) mod block; here they are kept as a min-heap on fin, so the next completion is the root.  What outlives
// residency (tokens generated before an eviction, first-token time, time per output token) sits in
// the lane's slice of the workspace.
//
// Configs this kernel does not take (larger max batch, integer counts beyond 2^53, block sizes
// beyond the histogram, the split-and-fuse policy) are left to the warp-per-config kernels; both
// sides decide with lanes_take().
#pragma once
#include "guide_internal.cuh"

namespace guide {

static constexpr u32 LANE_MAX_THREADS = 128;     // block size limit of the lane kernel
static constexpr u32 LANE_HIST_MAX = 64;         // block sizes up to this use the phase histogram

enum { LM_NEED = 0, LM_SCHED = 1, LM_RUN = 2, LM_FINISHED = 3, LM_OUT = 4 };
static constexpr u32 LS_FIRST = 0x400000u, LS_PHASE_SHIFT = 16, LS_PHASE_MASK = 0x3Fu;

// Constants of the attention terms of a decode iteration and whether every integer count of the
// config stays below 2^53 (then they can be carried as exact doubles).
struct DecodeConst {
    double c_f9, c_kvx, c_f10, c_b10;
    u64 xw;
    bool exact53;
};
__device__ __forceinline__ DecodeConst decode_const(const DModel &m, const DRate &rt, u32 b, u32 longest, double inv_tt) {
    DecodeConst d;
    // Largest summed context this config can see: every resident at its full length plus one.
    const u64 ctx_max = (u64)b * ((u64)longest + 1);
    const u64 lim53 = 1ull << 53;
    d.xw = rt.flash ? 0ull : (u64)m.nh * m.ab;                       // score-matrix bytes per unit of A
    d.exact53 = 2 * (u64)m.H * ctx_max < lim53 && 5 * (u64)m.nh * ctx_max < lim53 &&
                (u64)b * m.H * m.ab + ctx_max * ((u64)m.Dkv * m.kvb + d.xw) < lim53 && 2 * d.xw * ctx_max < lim53;
    d.c_f9 = (double)(2 * (u64)m.H) * inv_tt;                        // F9  = ctx * 2H / t
    d.c_kvx = (double)((u64)m.Dkv * m.kvb + d.xw) * inv_tt;          // KV read + score bytes per context token / t
    d.c_f10 = (double)(5 * (u64)m.nh) * inv_tt;                      // F10 = ctx * 5 n_h / t
    d.c_b10 = (double)(2 * d.xw) * inv_tt;                           // B10 = ctx * 2 n_h a_b / t (0 with flash)
    return d;
}

// Which kernel simulates a prompt-first config: the lane kernel when it is launched (maxb > 0) and
// the config's max batch, block size and counts allow it.
__device__ __forceinline__ bool lanes_take(u32 maxb, u32 hist_n, u32 b, u32 blk, bool exact) {
    return maxb != 0 && b <= maxb && exact && (blk == 1 || blk <= hist_n);
}

// The lane kernel builds every stage table from doubles (StageConst) and divides by the block size
// with a multiply: both are exact while every integer count a stage of this config can produce
// stays below 2^53 and token counts stay below 2^25.  Largest stages: a prompt pass over b requests
// of the longest length, a decode step over b residents at their full length plus one.
__device__ __forceinline__ bool lanes_exact(const DModel &m, u32 tt, u32 b, u32 longest) {
    const double bd = (double)b, q = (double)longest;
    const double Tm = bd * q, Am = fmax(bd * q * q, bd * (q + 1.0)), Cm = bd * (q + 1.0);
    return longest < (1u << 25) && stage_count_bound(m, tt, Tm, bd, Am, Cm) < 4503599627370496.0;   // 2^52
}

// x / d and x % d for 1 <= d <= 64 and x < 2^26 with magic = ceil(2^32 / d) (d >= 2): the product's
// high word is the quotient exactly, since the error x * (magic * d - 2^32) stays below 2^32.
__device__ __forceinline__ u32 div_small(u32 x, u32 d, u32 magic) { return d == 1 ? x : __umulhi(x, magic); }

// The work order visits the batch axis slowest when the whole space is simulated, so configs with
// a small max batch (the long schedules) are started first.
__device__ __forceinline__ u64 work_to_index(const DSpace &s, u64 w, bool reorder) {
    if (!reorder) return w;
    const u64 tl = (u64)s.n_t * s.n_l;
    const u64 per_b = (u64)s.n_m * s.n_h * s.n_f * tl;
    const u64 b = w / per_b, rest = w % per_b;
    const u64 mhf = rest / tl, x = rest % tl;
    return (mhf * s.n_b + b) * tl + x;
}

template <int TIME_SUM>
__device__ __forceinline__ double lane_decode_time(double ctxd, double c_f9, double tha, double c_kvx, double c_f10, double c_b10,
                                                   double ic, double im, double fix, double comm, double head, double Nd,
                                                   double tovh, double lf) {
    const double t9 = task_time<TIME_SUM>(ctxd * c_f9, tha + ctxd * c_kvx, ic, im);
    const double t10 = task_time<TIME_SUM>(ctxd * c_f10, ctxd * c_b10, ic, im);
    const double s_att = (t9 + t10) + t9;
    return combine_phase(fix, s_att, comm, head, 1.0, Nd, tovh, lf);
}

// Everything a lane keeps about its config.  The struct lives in the thread's local memory: the
// scheduler functions below are not inlined and work on it through a pointer, and the run loop
// copies the dozen values it needs into registers, so the compiler never has to choose between the
// loop's variables and the scheduler's when registers run out.
struct LaneState {
    // the config
    u64 j;                                    // output slot
    u64 max_iters;
    const StageConst *scp;                    // task-table factors of the config's (model, TP degree)
    u32 hf, t, b, Lin, Lout, blk, magic;
    u32 st, fit;
    double lf, Nd, icA, imA, tovh;
    double c_f9, c_kvx, c_f10, c_b10;
    // the schedule
    double clock, dec_time, csum_d;
    u64 dec_tok, n_iters, n_req_iters, free_blocks, csum;
    u64 pre_T, pre_A;                         // prompt tokens (and their squares) admitted since the last prompt pass
    u32 next, high_water, nheap, n_new, D, Dmod;
    u32 need_next, dc_n;
    double arr_next;
    double dc_fix, dc_comm, dc_head, dc_tha, dc_nd;   // decode-stage terms that depend on the resident count only
    // a run in progress
    double tcur, ctxd, cd;
    u32 it, fb, fb0, hidx, steps_max, in_run;
    u32 mode;
};

// What the scheduler functions need besides the lane's state (the same for every call of a thread).
struct LaneEnv {
    const DSpace *s;
    const DTrace *tr;
    u32 *s_base, *s_fin, *s_rqm, *s_hist;     // the lane's columns of the warp's shared-memory arrays (stride lanes_used)
    u32 stride;                               // lanes_used
    u32 *gen;                                 // per-request slices of the workspace: tokens generated before an eviction | done flag
    double *first, *finish;                   // first-token time, last-token time
};

#define SL(arr, k) e.arr[(k) * e.stride]

__device__ __forceinline__ void lane_refresh_head(LaneState &L, const LaneEnv &e) {
    const DTrace &tr = *e.tr;
    while (L.next < L.high_water && (e.gen[L.next] & 0x80000000u)) L.next++;
    if (L.next < tr.n) {
        L.arr_next = __ldg(tr.arrival + L.next);
        const u32 g = L.next < L.high_water ? e.gen[L.next] : 0u;       // tokens kept from before an eviction
        const u32 in = __ldg(tr.in_len + L.next);
        L.need_next = div_small((in ? in : L.Lin) + g + L.blk - 1, L.blk, L.magic);
    } else {
        L.arr_next = __longlong_as_double(0x7FF0000000000000LL);
        L.need_next = 0;
    }
}

// Residents form a binary min-heap on fin (the decode count at which they complete, compared as
// iterations still to go): the next completion is the root, a completion costs a sift-down instead
// of a pass over all slots.  Nothing depends on the order of the slots: sums are integer sums and
// the eviction victim is found by its request index.
__device__ __forceinline__ void lane_sift_down(const LaneEnv &e, u32 nheap, u32 D, u32 pos, u32 efin, u32 ebase, u32 erqm) {
    const u32 key = efin - D;
    for (;;) {
        u32 c = 2 * pos + 1;
        if (c >= nheap) break;
        u32 cf = SL(s_fin, c);
        if (c + 1 < nheap) {
            const u32 cf2 = SL(s_fin, c + 1);
            if (cf2 - D < cf - D) { c++; cf = cf2; }
        }
        if (key <= cf - D) break;
        SL(s_fin, pos) = cf; SL(s_base, pos) = SL(s_base, c); SL(s_rqm, pos) = SL(s_rqm, c);
        pos = c;
    }
    SL(s_fin, pos) = efin; SL(s_base, pos) = ebase; SL(s_rqm, pos) = erqm;
}
__device__ __forceinline__ void lane_sift_up(const LaneEnv &e, u32 D, u32 pos, u32 efin, u32 ebase, u32 erqm) {
    const u32 key = efin - D;
    while (pos > 0) {
        const u32 par = (pos - 1) >> 1;
        const u32 pf = SL(s_fin, par);
        if (pf - D <= key) break;
        SL(s_fin, pos) = pf; SL(s_base, pos) = SL(s_base, par); SL(s_rqm, pos) = SL(s_rqm, par);
        pos = par;
    }
    SL(s_fin, pos) = efin; SL(s_base, pos) = ebase; SL(s_rqm, pos) = erqm;
}

// retire every resident that has just emitted its last token
__device__ __forceinline__ void lane_retire(LaneState &L, const LaneEnv &e) {
    while (L.nheap > 0 && SL(s_fin, 0) == L.D) {
        const u32 rqm = SL(s_rqm, 0);
        const u32 rq = rqm & 0xFFFFu, cv = SL(s_base, 0) + L.D;
        e.gen[rq] = 0x80000000u;
        e.finish[rq] = L.clock;                              // its last token; the results turn it into time per output token
        L.free_blocks += div_small(cv + L.blk - 1, L.blk, L.magic);
        L.csum -= cv;
        if (L.blk > 1) {
            const u32 ph = (rqm >> LS_PHASE_SHIFT) & LS_PHASE_MASK;
            SL(s_hist, ph) -= 1;
        }
        L.nheap--;
        if (L.nheap > 0) lane_sift_down(e, L.nheap, L.D, 0, SL(s_fin, L.nheap), SL(s_base, L.nheap), SL(s_rqm, L.nheap));
    }
    L.csum_d = (double)(long long)L.csum;
}

// One pass of the scheduler: settle the run that just ended, retire, admit, a prompt pass for the
// newly admitted, the set-up of the next run.  Leaves the lane in LM_RUN, LM_FINISHED, or LM_SCHED
// (another pass: after an idle jump, or when the prompt pass made room for admissions).
// Slots [0, nheap) hold the residents (heap), slots [nheap, nheap + n_new) the requests admitted
// since the last prompt pass, in admission order.
template <int TIME_SUM>
__device__ __forceinline__ void lane_sched_body(LaneState &L, const LaneEnv &e) {
    const DTrace &tr = *e.tr;
    if (L.in_run) {
        const u64 tok = (u64)L.it * L.nheap;
        L.D += L.it;
        { const u32 x = L.Dmod + L.it; L.Dmod = x - div_small(x, L.blk, L.magic) * L.blk; }
        L.csum += tok; L.csum_d = L.cd;
        L.dec_tok += tok; L.n_req_iters += tok; L.n_iters += L.it;
        L.free_blocks -= L.fb0 - L.fb;
        L.in_run = 0;
        lane_retire(L, e);
    }
    // ---- 1. admit in arrival order, no overtaking ----
    while (L.nheap + L.n_new < L.b && L.arr_next <= L.clock && L.need_next <= L.free_blocks) {
        const u32 next = L.next;
        const u32 g = next < L.high_water ? e.gen[next] : 0u;
        u32 in = __ldg(tr.in_len + next), out = __ldg(tr.out_len + next);
        if (in == 0) { in = L.Lin; out = L.Lout; }
        L.free_blocks -= L.need_next;
        const u32 k = L.nheap + L.n_new;
        SL(s_rqm, k) = next | (g == 0 ? LS_FIRST : 0u);
        SL(s_base, k) = in + g;                              // prompt + tokens to recompute
        SL(s_fin, k) = out - g;                              // tokens still to emit
        L.pre_T += (u64)(in + g); L.pre_A += (u64)(in + g) * (in + g);
        L.n_new++; L.next = next + 1;
        if (L.next > L.high_water) L.high_water = L.next;
        lane_refresh_head(L, e);
    }
    // ---- 2. nothing to run: finished, or jump to the next arrival ----
    if (L.nheap + L.n_new == 0) {
        if (L.next >= tr.n) { L.mode = LM_FINISHED; return; }
        if (L.arr_next > L.clock) { L.clock = L.arr_next; return; }
        L.st |= GUIDE_ST_ITER;                               // cannot happen when each request fits alone
        L.mode = LM_FINISHED;
        return;
    }
    if (L.n_iters >= L.max_iters) { L.st |= GUIDE_ST_ITER; L.mode = LM_FINISHED; return; }
    const double *rate = e.s->rate10 + (size_t)L.hf * 10;    // inv_c[LINEAR, ATTN, ELEM], inv_m[...], inv_comm, clat, tovh, flash
    // ---- 3./4. prompts first, everything else stalls ----
    if (L.n_new > 0) {
        const u64 T = L.pre_T, A = L.pre_A;                  // summed at admission: tokens and tokens squared of the new prompts
        L.pre_T = 0; L.pre_A = 0;
        const AttnRates ar = {L.c_f9, L.c_f10, L.c_b10, L.icA, L.imA, L.Nd, L.tovh, L.lf};
        const double t_iter = stage_prompt_pass<TIME_SUM>(L.scp, rate, (double)(long long)T, (double)L.n_new, (double)(long long)A, &ar);
        const double after = L.clock + t_iter;
        for (u32 i = 0; i < L.n_new; i++) {                  // the new ones become residents: into the heap
            const u32 rqm = SL(s_rqm, L.nheap);
            const u32 rq = rqm & 0xFFFFu;
            if (rqm & LS_FIRST) e.first[rq] = after;         // first token of this request
            const u32 q = SL(s_base, L.nheap), left = SL(s_fin, L.nheap) - 1;
            u32 ph = 0;
            if (L.blk > 1) {
                ph = q - div_small(q, L.blk, L.magic) * L.blk + L.blk - L.Dmod;     // (cache - D) mod block
                if (ph >= L.blk) ph -= L.blk;
                SL(s_hist, ph) += 1;
            }
            lane_sift_up(e, L.D, L.nheap, L.D + left, q - L.D, rq | (ph << LS_PHASE_SHIFT));
            L.nheap++;
        }
        L.csum += T;
        L.n_req_iters += L.n_new;
        L.n_new = 0;
        L.clock = after;
        L.n_iters++;
        lane_retire(L, e);                                   // requests with a single output token are done already
        // the clock has moved: if the head of the queue can come in now, or nobody is left, take another pass
        if (L.nheap == 0 || (L.nheap < L.b && L.arr_next <= L.clock && L.need_next <= L.free_blocks)) return;
        if (L.n_iters >= L.max_iters) { L.st |= GUIDE_ST_ITER; L.mode = LM_FINISHED; return; }
    }
    // ---- decode: every sequence whose last block is full needs one more block ----
    u32 needed = L.blk == 1 ? L.nheap : SL(s_hist, L.Dmod == 0 ? 0 : L.blk - L.Dmod);
    if (needed > L.free_blocks) {
        while (needed > L.free_blocks) {                     // evict the youngest, recompute later
            u32 v = 0, vrq = SL(s_rqm, 0) & 0xFFFFu;
            for (u32 k = 1; k < L.nheap; k++) {
                const u32 rq = SL(s_rqm, k) & 0xFFFFu;
                if (rq > vrq) { vrq = rq; v = k; }
            }
            const u32 rqm = SL(s_rqm, v);
            const u32 cv = SL(s_base, v) + L.D, rem = SL(s_fin, v) - L.D;
            const u32 held = div_small(cv + L.blk - 1, L.blk, L.magic);
            L.free_blocks += held;
            if (held * L.blk == cv) needed--;
            L.csum -= cv;
            const u32 out = __ldg(tr.in_len + vrq) ? __ldg(tr.out_len + vrq) : L.Lout;
            e.gen[vrq] = out - rem;
            if (L.blk > 1) {
                const u32 ph = (rqm >> LS_PHASE_SHIFT) & LS_PHASE_MASK;
                SL(s_hist, ph) -= 1;
            }
            L.nheap--;
            if (v < L.nheap) {                               // the last entry takes the hole, then finds its level
                const u32 efin = SL(s_fin, L.nheap), ebase = SL(s_base, L.nheap), erqm = SL(s_rqm, L.nheap);
                if (v > 0 && efin - L.D < SL(s_fin, (v - 1) >> 1) - L.D) lane_sift_up(e, L.D, v, efin, ebase, erqm);
                else lane_sift_down(e, L.nheap, L.D, v, efin, ebase, erqm);
            }
            L.next = vrq;
        }
        lane_refresh_head(L, e);
        L.csum_d = (double)(long long)L.csum;
    }
    L.free_blocks -= needed;
    if (L.dc_n != L.nheap) {
        const StageFixed sf = stage_decode_terms<TIME_SUM>(L.scp, rate, (double)L.nheap);
        L.dc_n = L.nheap;
        L.dc_fix = sf.fix; L.dc_comm = sf.comm; L.dc_head = sf.head; L.dc_tha = sf.tha;
        L.dc_nd = (double)L.nheap;
    }
    // set up the run: the first iteration's time is ready when the run phase starts
    const u64 cap_left = L.max_iters - L.n_iters;
    L.steps_max = (u32)min((u64)(SL(s_fin, 0) - L.D), cap_left);     // up to the next completion (the heap's root)
    L.fb0 = (u32)min(L.free_blocks, (u64)0xFFFFFFFFu);
    L.fb = L.fb0; L.it = 0;
    L.hidx = L.Dmod + 1 == L.blk ? 0 : L.blk - (L.Dmod + 1);         // histogram bin of the next iteration's needers
    L.cd = L.csum_d;
    L.ctxd = L.cd + L.dc_nd;
    L.tcur = lane_decode_time<TIME_SUM>(L.ctxd, L.c_f9, L.dc_tha, L.c_kvx, L.c_f10, L.c_b10, L.icA, L.imA, L.dc_fix, L.dc_comm,
                                        L.dc_head, L.Nd, L.tovh, L.lf);
    L.in_run = 1;
    L.mode = LM_RUN;
}

// The pass on a copy of the state in registers (one burst of loads, one of stores), out of line so
// that its register needs do not compete with the run loop's.
template <int TIME_SUM>
__device__ __noinline__ void lane_sched_pass(LaneState *Lp, const LaneEnv *ep) {
    LaneState L = *Lp;
    const LaneEnv e = *ep;
    lane_sched_body<TIME_SUM>(L, e);
    *Lp = L;
}

// Work item w: if it is a config of this launch, set the lane up for it (mode LM_SCHED, or
// LM_FINISHED when it cannot run at all); otherwise leave the lane in LM_NEED.
struct LaneLaunch { Range r; int tp_model, reorder; u64 max_iters_opt; u32 minb, maxb, hist_n; };

__device__ __noinline__ void lane_start_config(LaneState *Lp, const LaneEnv *ep, const LaneLaunch *lp, u64 w) {
    LaneState &L = *Lp;
    const LaneEnv &e = *ep;
    const DSpace &s = *e.s;
    const DTrace &tr = *e.tr;
    const u64 idx = lp->reorder ? work_to_index(s, w, true) : lp->r.first + w;
    const Cfg c = decode_index(s, idx);
    const u32 b = s.batch[c.b];
    if (b < lp->minb || b > lp->maxb) return;                // another launch takes it
    const u32 hf = c.h * s.n_f + c.f;
    const DRate rt = s.rates[hf];
    if (rt.policy != GUIDE_POLICY_PREFILL_FIRST) return;     // k_trace_fuse simulates those
    const DModel m = s.models[c.m];
    const u32 t = s.tp[c.t];
    const uint2 pr = s.pairs[c.l];
    const u32 blk = rt.kv_block;
    const u32 tt = lp->tp_model ? 1u : t;
    const u32 longest = max(tr.max_tokens, tr.any_zero ? pr.x + pr.y : 0u);
    if (!lanes_take(lp->maxb, lp->hist_n, b, blk, lanes_exact(m, tt, b, longest))) return;   // the warp-per-config kernel takes it
    L.hf = hf; L.t = t; L.b = b; L.Lin = pr.x; L.Lout = pr.y; L.blk = blk;
    L.scp = s.stage_consts + (size_t)(lp->tp_model ? s.n_t : c.t) * s.n_m + c.m;
    L.magic = blk > 1 ? (u32)((0x100000000ull + blk - 1) / blk) : 0u;
    const DecodeConst dc = decode_const(m, rt, b, longest, 1.0 / (double)tt);
    L.j = idx - lp->r.first;
    const MemInfo mi = mem_info(m, t);
    L.lf = log2_rule_factor(t, lp->tp_model); L.Nd = (double)m.N;
    L.icA = rt.inv_c[CLS_ATTN]; L.imA = rt.inv_m[CLS_ATTN]; L.tovh = rt.tovh;
    L.c_f9 = dc.c_f9; L.c_kvx = dc.c_kvx; L.c_f10 = dc.c_f10; L.c_b10 = dc.c_b10;
    // ---- what fits (Sec. 3.2 Step 1) ----
    const u64 blocks_total = rt.usable > mi.w_gpu ? floor_div(rt.usable - mi.w_gpu, (u64)blk * mi.kv_tok) : 0;
    const u64 worst = (longest + blk - 1) / blk;
    u32 st = 0;
    if (rt.usable <= mi.w_gpu) st |= GUIDE_ST_WEIGHTS;
    if (worst > blocks_total) st |= GUIDE_ST_KV;
    if ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) st |= GUIDE_ST_HEADS;
    L.st = st;
    L.fit = clamp_u32(blocks_total / worst);
    L.clock = 0.0; L.dec_time = 0.0; L.csum_d = 0.0;
    L.dec_tok = 0; L.n_iters = 0; L.n_req_iters = 0; L.free_blocks = blocks_total; L.csum = 0;
    L.next = 0; L.high_water = 0; L.nheap = 0; L.n_new = 0; L.D = 0; L.Dmod = 0;
    L.dc_n = 0; L.in_run = 0; L.pre_T = 0; L.pre_A = 0;
    L.max_iters = lp->max_iters_opt ? lp->max_iters_opt : 64 * (tr.sum_out + (u64)tr.n_zero * pr.y) + 4 * (u64)tr.n;
    if (st) { L.mode = LM_FINISHED; return; }
    for (u32 i = 0; i < lp->hist_n; i++) SL(s_hist, i) = 0;
    lane_refresh_head(L, e);
    L.mode = LM_SCHED;
}
#undef SL

// write_results(j, st, fit, clock, dec_time, dec_tok, n_iters, n_req_iters, cost_hr, Lout, first, finish): the
// warp-wide reduction of one finished config (supplied by the file that owns the output format).
template <int TIME_SUM, int UNROLL, class WriteResults>
__device__ __forceinline__ void lanes_simulate(const DSpace &s, const DTrace &tr, const Range &r, int tp_model, u64 max_iters_opt,
                                               unsigned long long *counter, unsigned char *scratch, size_t per_lane,
                                               u32 gen_bytes, u32 first_bytes, int reorder, u32 minb, u32 maxb, u32 hist_n,
                                               u32 lanes_used, u32 round_len, unsigned char *wsm, WriteResults &&write_results) {
    const u32 FULL = 0xFFFFFFFFu;
    const u32 lane = threadIdx.x & 31, wib = threadIdx.x >> 5, n_wib = blockDim.x >> 5;
    const u32 lt_mask = (1u << lane) - 1;

    LaneEnv env;
    env.s = &s; env.tr = &tr;
    // shared-memory slots of this warp: slot k of lane l at [k][l]
    env.s_base = (u32 *)wsm + lane;                              // resident: cache - D; admitted, before its prompt pass: prompt + recompute tokens
    env.s_fin = env.s_base + lanes_used * maxb;                  // resident: D at completion; admitted: tokens still to emit
    env.s_rqm = env.s_fin + lanes_used * maxb;                   // request index | phase << 16 | LS_FIRST
    env.s_hist = env.s_rqm + lanes_used * maxb;                  // [hist_n][lanes_used]: residents per (cache - D) mod block
    env.stride = lanes_used;
    unsigned char *warp_ws = scratch + (size_t)(blockIdx.x * n_wib + wib) * lanes_used * per_lane;
    unsigned char *mine = warp_ws + (size_t)lane * per_lane;
    env.gen = (u32 *)mine;
    env.first = (double *)(mine + gen_bytes);
    env.finish = (double *)(mine + gen_bytes + first_bytes);
    LaneLaunch launch;
    launch.r = r; launch.tp_model = tp_model; launch.reorder = reorder; launch.max_iters_opt = max_iters_opt;
    launch.minb = minb; launch.maxb = maxb; launch.hist_n = hist_n;

    LaneState L;
    L.mode = lane < lanes_used ? LM_NEED : LM_OUT;           // small launches spread over more warps, fewer lanes each

    for (;;) {
        // ---- lanes without a config take the next ones from the work counter ----
        for (;;) {
            const u32 want = __ballot_sync(FULL, L.mode == LM_NEED);
            if (want == 0) break;
            unsigned long long w0 = 0;
            if (lane == 0) w0 = atomicAdd(counter, (unsigned long long)__popc(want));
            w0 = __shfl_sync(FULL, w0, 0);
            if (L.mode == LM_NEED) {
                const u64 w = w0 + __popc(want & lt_mask);
                if (w >= r.count) L.mode = LM_OUT;
                else lane_start_config(&L, &env, &launch, w);    // stays LM_NEED when the config is not this launch's
            }
        }
        if (__all_sync(FULL, L.mode == LM_OUT)) break;
        // ---- events ----
        while (__any_sync(FULL, L.mode == LM_SCHED)) {
            if (L.mode == LM_SCHED) lane_sched_pass<TIME_SUM>(&L, &env);
        }
        // ---- run: up to round_len decode iterations, nothing per request is touched.  The next
        // iteration's time is computed before the clock-dependent exit test so that the two
        // dependency chains overlap.  Everything the loop uses sits in registers. ----
        if (L.mode == LM_RUN) {
            double clock = L.clock, dec_time = L.dec_time, tcur = L.tcur, ctxd = L.ctxd, cd = L.cd;
            const double nd = L.dc_nd, tha = L.dc_tha, fix = L.dc_fix, comm = L.dc_comm, head = L.dc_head;
            const double c_f9 = L.c_f9, c_kvx = L.c_kvx, c_f10 = L.c_f10, c_b10 = L.c_b10, icA = L.icA, imA = L.imA;
            const double Nd = L.Nd, tovh = L.tovh, lf = L.lf, arr_next = L.arr_next;
            const u32 steps_max = L.steps_max, blk = L.blk, nheap = L.nheap, need_next = L.need_next;
            const bool room = nheap < L.b;
            const u32 *hist = env.s_hist;
            u32 it = L.it, fb = L.fb, hidx = L.hidx, left = round_len, mode = LM_RUN;
            // One decode iteration of time t at summed context c has just been computed: advance the
            // clock, then see whether an event follows it.
#define LANE_APPLY(t, c)                                                                              \
            clock = clock + (t);                                                                      \
            dec_time = dec_time + (t);                                                                \
            cd = (c);                                                                                 \
            it++;                                                                                     \
            if (it == steps_max) { mode = LM_SCHED; break; }          /* a completion (or the cap) follows */ \
            {                                                                                         \
                const u32 need2 = blk == 1 ? nheap : hist[hidx * lanes_used];                         \
                if (need2 > fb) { mode = LM_SCHED; break; }           /* eviction needed */            \
                if (room && arr_next <= clock && need_next <= fb) { mode = LM_SCHED; break; }   /* the queue head can come in */ \
                fb -= need2;                                                                          \
                hidx = hidx == 0 ? blk - 1 : hidx - 1;                                                \
            }
#define LANE_TIME(c) lane_decode_time<TIME_SUM>((c), c_f9, tha, c_kvx, c_f10, c_b10, icA, imA, fix, comm, head, Nd, tovh, lf)
            if (UNROLL == 4) {
                // Lanes of a warp in step: every lane runs the same loop, four iterations per trip (their
                // times are four independent chains), the exit tests after each clock update.
                for (;;) {
                    const double c1 = ctxd + nd, c2 = c1 + nd, c3 = c2 + nd, c4 = c3 + nd;
                    const double t1 = LANE_TIME(c1), t2 = LANE_TIME(c2), t3 = LANE_TIME(c3), t4 = LANE_TIME(c4);
                    LANE_APPLY(tcur, ctxd)
                    LANE_APPLY(t1, c1)
                    LANE_APPLY(t2, c2)
                    LANE_APPLY(t3, c3)
                    tcur = t4; ctxd = c4;
                    if (left <= 4) break;
                    left -= 4;
                }
            } else if (UNROLL == 1) {
                // the next iteration's time is computed before the clock-dependent exit test
                for (;;) {
                    const double c1 = ctxd + nd;
                    const double t1 = LANE_TIME(c1);
                    LANE_APPLY(tcur, ctxd)
                    tcur = t1; ctxd = c1;
                    if (--left == 0) break;
                }
            }
#undef LANE_APPLY
#undef LANE_TIME
            L.clock = clock; L.dec_time = dec_time; L.tcur = tcur; L.ctxd = ctxd; L.cd = cd;
            L.it = it; L.fb = fb; L.hidx = hidx; L.mode = mode;
        }
        // ---- results of finished configs, one at a time, by the whole warp ----
        u32 fin = __ballot_sync(FULL, L.mode == LM_FINISHED);
        while (fin) {
            const int l = __ffs(fin) - 1;
            fin &= fin - 1;
            const u64 jj = __shfl_sync(FULL, L.j, l);
            const u32 st_l = __shfl_sync(FULL, L.st, l), fit_l = __shfl_sync(FULL, L.fit, l);
            const double clock_l = __shfl_sync(FULL, L.clock, l), dec_time_l = __shfl_sync(FULL, L.dec_time, l);
            const u64 dec_tok_l = __shfl_sync(FULL, L.dec_tok, l), n_iters_l = __shfl_sync(FULL, L.n_iters, l),
                      n_req_iters_l = __shfl_sync(FULL, L.n_req_iters, l);
            const u32 hf_l = __shfl_sync(FULL, L.hf, l), t_l = __shfl_sync(FULL, L.t, l), Lout_l = __shfl_sync(FULL, L.Lout, l);
            unsigned char *theirs = warp_ws + (size_t)l * per_lane;
            write_results(jj, st_l, fit_l, clock_l, dec_time_l, dec_tok_l, n_iters_l, n_req_iters_l,
                          s.rates[hf_l].price * (double)t_l, Lout_l, (double *)(theirs + gen_bytes),
                          (double *)(theirs + gen_bytes + first_bytes));
        }
        if (L.mode == LM_FINISHED) L.mode = LM_NEED;
    }
}

}  // namespace guide
