// Split-and-fuse scheduling for the trace simulation (the FastGen-like framework model: dynamic
// splitting of prompts and fusion with decoding, Sec. 2.3.2 / Sec. 3.1 / Sec. 3.3), one warp per
// config, called by k_trace_sim for configs whose framework has this policy.
//
// Every iteration carries about `budget` tokens: one per resident request past its prompt, the
// rest prompt tokens in arrival order, so a long prompt is spread over several iterations and short
// ones share one.  A chunk of q tokens attends the pdone + q tokens of its request seen so far; a
// request emits its first token in the iteration that finishes its prompt.  Blocks for the whole
// prompt are taken at admission; a decoding request whose last block is full takes one more, and
// when none is free the youngest resident is evicted and recomputed later.
//
// Unlike the prompt-first path little is carried between iterations besides the slots themselves:
// every iteration scans them with all 32 lanes (count the decoders, plan the prompt chunks while
// some request is in its prompt, evaluate one stage time, apply, retire); the non-attention terms
// of the stage time are kept while the iteration's token counts repeat.
#pragma once
#include <cstddef>

#include "guide_internal.cuh"

namespace guide {

static constexpr u32 FUSE_HIST = 64;      // block sizes up to this take the decode-only runs

struct FuseResult {
    double clock, dec_time;
    u64 dec_tok, n_iters, n_req_iters;
};

static_assert(sizeof(DModel) <= 128 && sizeof(DRate) <= 128, "a warp copies each of them with one word per lane");
static_assert(offsetof(DRate, inv_m) == 24 && offsetof(DRate, inv_comm) == 48 && offsetof(DRate, clat) == 56 && offsetof(DRate, tovh) == 64,
              "a rate entry starts like a row of rate10");
struct FuseSlots {
    FuseResult res;                     // what the schedule hands back to the kernel around it
    u32 req[GUIDE_TRACE_MAX_BATCH];     // request index, ascending
    u32 seen[GUIDE_TRACE_MAX_BATCH];    // prompt phase: tokens processed so far; decoding: tokens cached
    u32 todo[GUIDE_TRACE_MAX_BATCH];    // prompt (and recompute) tokens still to process; 0 = decoding
    u32 rem[GUIDE_TRACE_MAX_BATCH];     // tokens still to emit
    unsigned char fresh[GUIDE_TRACE_MAX_BATCH];   // no token emitted yet: the first one sets the TTFT
    u32 hist[FUSE_HIST];                // decode-only runs: residents per (cached tokens mod block size)
    double sc[32];                      // the config's task-table factors as doubles (a StageConst), when its counts stay exact in them
    DModel m;                           // the config's model and (hardware, framework) rates
    DRate rt;
    alignas(16) double tbuf[32];        // decode-only runs: times of the 32 iterations worked out at once
    double dterm[32][3];                // decode-only runs: fixed-task, all-reduce and head terms of 32 neighbouring resident counts
};


// Sum over the warp of 64-bit counts by the integer reduction unit: three pieces of 22, 22 and 20
// bits are summed apart (no piece's sum leaves 32 bits) and put together again modulo 2^64.
__device__ __forceinline__ u64 fuse_warp_sum(u64 v) {
    const u32 a = __reduce_add_sync(0xFFFFFFFFu, (u32)v & 0x3FFFFFu);
    const u32 b = __reduce_add_sync(0xFFFFFFFFu, (u32)(v >> 22) & 0x3FFFFFu);
    const u32 c = __reduce_add_sync(0xFFFFFFFFu, (u32)(v >> 44));
    return ((u64)c << 44) + ((u64)b << 22) + a;
}
__device__ __forceinline__ u32 fuse_warp_sum32(u32 v) { return __reduce_add_sync(0xFFFFFFFFu, v); }
// inclusive prefix sum over the lanes
__device__ __forceinline__ u64 fuse_warp_scan(u64 v, u32 lane) {
    for (int d = 1; d < 32; d <<= 1) {
        const u64 o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= (u32)d) v += o;
    }
    return v;
}

// Runs the whole schedule of one config.  gen / first / tpot: the warp's per-request slices of the
// workspace (tokens generated so far with the done flag in the top bit, first-token time, time of the
// last token).  Returns the status bits (0, or the iteration limit) and leaves the totals in
// sl.res.  The model, the rates and the trace come as pointers to device memory so that the kernel
// around this call keeps its own copies in registers.
struct FuseTrace { const double *arrival; const u32 *in_len, *out_len; };

template <int TIME_SUM>
__device__ __noinline__ u32 fuse_schedule(const DModel *mp, const DRate *rp, const double *arrival, const u32 *in_len,
                                          const u32 *out_len, u32 n, u32 tt, u32 b, u32 Lin, u32 Lout, u64 blocks_total,
                                          double lf, u64 max_iters, FuseSlots &sl, u32 *gen, double *first, double *tpot,
                                          const double *scg) {
    // the model and the pair's rates next to the warp: their fields are read where they are used
    const u32 lane0 = threadIdx.x & 31;
    __syncwarp();
    if (lane0 < sizeof(DModel) / 4) reinterpret_cast<u32 *>(&sl.m)[lane0] = reinterpret_cast<const u32 *>(mp)[lane0];
    if (lane0 < sizeof(DRate) / 4) reinterpret_cast<u32 *>(&sl.rt)[lane0] = reinterpret_cast<const u32 *>(rp)[lane0];
    __syncwarp();
    const DModel &m = sl.m;
    const DRate &rt = sl.rt;
    const FuseTrace tr = {arrival, in_len, out_len};
    const double Nd = (double)m.N;
    const u32 lane = threadIdx.x & 31;
    const u32 lt_mask = (1u << lane) - 1;
    const u32 blk = rt.kv_block, budget = rt.seg;
    const u32 done_flag = 0x80000000u;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    // block sizes are powers of two as a rule: their divisions are shifts
    const u32 blk_shift = (blk & (blk - 1)) == 0 ? (u32)__ffs(blk) - 1 : 0xFFFFFFFFu;
    auto divb = [&](u32 x) { return blk_shift != 0xFFFFFFFFu ? x >> blk_shift : x / blk; };
    auto modb = [&](u32 x) { return blk_shift != 0xFFFFFFFFu ? x & (blk - 1) : x % blk; };
    auto blocks_of = [&](u32 tokens) { return divb(tokens + blk - 1); };

    // scg: the (model, TP degree) factors that turn token counts into a task table, as doubles, when the
    // config's counts stay exact in them (null: the integer table).  Kept next to the warp with the
    // pair's rates and read where they are used.
    const bool sc_ok = scg != nullptr;
    if (sc_ok) {
        sl.sc[lane] = scg[lane];
        __syncwarp();
    }
    const StageConst &sc = *reinterpret_cast<const StageConst *>(sl.sc);
    const double icA = rt.inv_c[CLS_ATTN], imA = rt.inv_m[CLS_ATTN];
    // attention tasks of a stage from doubles: the operations of build_attn_tasks and eval_attn on exact values
    auto attn_d = [&](double Td, double Ad, double Cd) {
        const double xw = rt.flash ? 0.0 : sc.xb;
        const double t9 = task_time<TIME_SUM>(Ad * sc.f9, ((Td * sc.ha + Cd * sc.kv) + Ad * xw) * sc.inv_t, icA, imA);
        const double t10 = task_time<TIME_SUM>(Ad * sc.f10, rt.flash ? 0.0 : (2.0 * (Ad * sc.xb)) * sc.inv_t, icA, imA);
        return (t9 + t10) + t9;
    };
    double clock = 0.0, dec_time = 0.0;
    u64 dec_tok = 0, n_iters = 0, n_req_iters = 0, free_blocks = blocks_total;
    u32 next = 0, high_water = 0, nrun = 0, st = 0;
    u32 n_pre = 0;                                   // residents still in their prompt
    u32 dw0 = 0x80000000u;                           // first resident count of the window of decode terms (none yet)
    u64 dc_T = ~0ull, dc_E = ~0ull;                  // stage terms kept while the token counts repeat
    double dc_fix = 0.0, dc_comm = 0.0, dc_head = 0.0;
    double arr_next = 0.0;
    u32 need_next = 0;
    auto refresh_head = [&]() {
        while (next < high_water && (gen[next] & done_flag)) next++;
        if (next < n) {
            arr_next = __ldg(tr.arrival + next);
            const u32 g = next < high_water ? gen[next] : 0u;
            const u32 in = __ldg(tr.in_len + next);
            need_next = blocks_of((in ? in : Lin) + g);
        } else {
            arr_next = inf; need_next = 0;
        }
    };
    refresh_head();

    // one stage time from (T, E, A, C); everything but attention is kept while T and E repeat
    auto stage_time = [&](u64 T, u64 E, u64 A, u64 C) {
        if (sc_ok) {
            const double Td = (double)(long long)T;
            if (T != dc_T || E != dc_E) {
                const StageFixed sf = stage_fixed<TIME_SUM>(sc, rt.inv_c, Td, (double)(long long)E)   /* a rate entry starts like a row of rate10 */;
                dc_T = T; dc_E = E;
                dc_fix = sf.fix; dc_comm = sf.comm;
                dc_head = E ? sf.head : 0.0;                       // nobody emits a token: no LM head
            }
            return combine_phase(dc_fix, attn_d(Td, (double)(long long)A, (double)(long long)C), dc_comm, dc_head, 1.0, Nd, rt.tovh, lf);
        }
        if (T != dc_T || E != dc_E) {
            TaskTab kf;
            build_fixed_tasks(m, tt, T, E, 1, kf);
            dc_T = T; dc_E = E;
            dc_fix = eval_fixed<TIME_SUM>(kf, rt);
            dc_comm = eval_comm(kf, rt);
            dc_head = E ? eval_head<TIME_SUM>(kf, rt) : 0.0;       // nobody emits a token: no LM head
        }
        TaskTab ka;
        build_attn_tasks(m, tt, T, A, C, ka);
        return combine_phase(dc_fix, eval_attn<TIME_SUM>(ka, rt), dc_comm, dc_head, 1.0, Nd, rt.tovh, lf);
    };
    // retire finished requests, keep the rest in order
    auto retire = [&]() {
        u32 kept = 0;
        u64 freed = 0;
        const u32 n_before = nrun;
        for (u32 base = 0; base < n_before; base += 32) {
            const u32 k = base + lane;
            const bool valid = k < n_before;
            u32 rq = 0, sn = 0, td = 0, rm = 0, fr = 0;
            if (valid) { rq = sl.req[k]; sn = sl.seen[k]; td = sl.todo[k]; rm = sl.rem[k]; fr = sl.fresh[k]; }
            const bool done = valid && td == 0 && rm == 0;
            if (done) {
                gen[rq] = done_flag;
                tpot[rq] = clock;          // time of its last token; the results turn it into time per output token
                freed += blocks_of(sn);
            }
            const bool keep = valid && !done;
            const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);
            __syncwarp();
            if (keep) {
                const u32 d = kept + __popc(ballot & lt_mask);
                sl.req[d] = rq; sl.seen[d] = sn; sl.todo[d] = td; sl.rem[d] = rm; sl.fresh[d] = (unsigned char)fr;
            }
            kept += __popc(ballot);
            __syncwarp();
        }
        free_blocks += fuse_warp_sum(freed);
        nrun = kept;
        refresh_head();
    };

    for (;;) {
        // ---- admit in arrival order, no overtaking ----
        if (nrun < b && arr_next <= clock && need_next <= free_blocks) {
            do {
                const u32 g = next < high_water ? gen[next] : 0u;
                u32 in = __ldg(tr.in_len + next), out = __ldg(tr.out_len + next);
                if (in == 0) { in = Lin; out = Lout; }
                free_blocks -= need_next;
                if (lane == 0) {
                    sl.req[nrun] = next;
                    sl.seen[nrun] = 0;
                    sl.todo[nrun] = in + g;                   // prompt + tokens to recompute
                    sl.rem[nrun] = out - g;
                    sl.fresh[nrun] = g == 0;
                }
                nrun++; next++; n_pre++;
                if (next > high_water) high_water = next;
                refresh_head();
            } while (nrun < b && arr_next <= clock && need_next <= free_blocks);
            __syncwarp();
        }
        if (nrun == 0) {
            if (next >= n) break;
            if (arr_next > clock) { clock = arr_next; continue; }
            st |= GUIDE_ST_ITER;                                   // cannot happen when each request fits alone
            break;
        }
        if (n_iters >= max_iters) { st |= GUIDE_ST_ITER; break; }

        // ---- nobody is in its prompt: a run of decode iterations up to the next event (a completion,
        // a block shortage, room for the head of the queue, the iteration limit).  One pass finds the
        // summed context, the first completion and how many residents sit at each offset within a
        // block; the iterations of the run then touch no slot, and one pass settles them. ----
        if (n_pre == 0 && blk <= FUSE_HIST) {
            for (u32 i = lane; i < blk; i += 32) sl.hist[i] = 0;
            __syncwarp();
            u64 c = 0;
            u32 local_min = 0xFFFFFFFFu;
            for (u32 base = 0; base < nrun; base += 32) {
                const u32 k = base + lane;
                if (k < nrun) {
                    const u32 sn = sl.seen[k];
                    c += (u64)sn + 1;
                    local_min = min(local_min, sl.rem[k]);
                    atomicAdd(&sl.hist[modb(sn)], 1u);
                }
            }
            u64 ctx_i = fuse_warp_sum(c);
            for (int d = 16; d > 0; d >>= 1) local_min = min(local_min, __shfl_xor_sync(0xFFFFFFFFu, local_min, d));
            const u32 min_rem = local_min;
            __syncwarp();
            const u64 cap_left = max_iters - n_iters;
            const bool room = nrun < b;
            const u32 steps_max = (u32)min((u64)min_rem, cap_left);
            const u32 lmod = modb(lane);
            // The terms of a decode iteration that depend on the resident count only are kept for a window
            // of 32 neighbouring counts (worked out one per lane): the count moves by one or two per event.
            if (nrun - dw0 >= 32u) {
                dw0 = nrun > 16 ? nrun - 16 : 1;
                const u32 nl = dw0 + lane;
                TaskTab kf;
                build_fixed_tasks(m, tt, nl, nl, 1, kf);
                __syncwarp();
                sl.dterm[lane][0] = eval_fixed<TIME_SUM>(kf, rt);
                sl.dterm[lane][1] = eval_comm(kf, rt);
                sl.dterm[lane][2] = eval_head<TIME_SUM>(kf, rt);
                __syncwarp();
            }
            const double d_fix = sl.dterm[nrun - dw0][0], d_comm = sl.dterm[nrun - dw0][1], d_head = sl.dterm[nrun - dw0][2];
            u32 it = 0, off = 0;                                   // off = it mod block size
            // The iterations of the run depend on one another through the clock only: the lanes work out
            // the times of 32 consecutive ones at once (summed context ctx_i + k * nrun), a prefix sum
            // over the histogram bins tells which of them finds its blocks, and the clock then advances
            // one iteration after the other, in order, watching for the arrival of the queue head.
            for (;;) {
                const u32 nb = min(32u, steps_max - it);
                const u64 ctx_k = ctx_i + (u64)lane * nrun;
                double s_att;
                if (sc_ok) {
                    const double cd = (double)(long long)ctx_k;
                    s_att = attn_d((double)nrun, cd, cd);
                } else {
                    TaskTab ka;
                    build_attn_tasks(m, tt, nrun, ctx_k, ctx_k, ka);
                    s_att = eval_attn<TIME_SUM>(ka, rt);
                }
                const double t_k = combine_phase(d_fix, s_att, d_comm, d_head, 1.0, Nd, rt.tovh, lf);
                u32 need_k = 0;                                    // residents whose last block is full before lane's iteration
                if (lane < nb) {
                    const u32 o = off + lmod >= blk ? off + lmod - blk : off + lmod;
                    need_k = sl.hist[o == 0 ? 0 : blk - o];
                }
                u32 incl = need_k;
                #pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const u32 up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                    if (lane >= (u32)d) incl += up;
                }
                // free blocks before lane's iteration takes its own (meaningful up to the first shortage)
                const u64 free_k = free_blocks - (incl - need_k);
                const u32 short_at = __ballot_sync(0xFFFFFFFFu, lane < nb && need_k > free_k);   // eviction: the general path below
                const u32 can = short_at ? (u32)__ffs(short_at) - 1 : nb;     // iterations that find their blocks
                if (can == 0) break;
                const u32 last = can - 1;
                const bool counted_out = it + can == steps_max;    // a completion or the cap follows the last one
                const u32 watch = __ballot_sync(0xFFFFFFFFu, room && need_next <= free_k - need_k) & (0xFFFFFFFFu >> (31 - last));
                sl.tbuf[lane] = t_k;
                __syncwarp();
                // the clock, one iteration after the other: four per trip, the arrival tests of a trip taken together
                u32 k = 0;
                bool arrived = false;
                const u32 cnt = last + 1;
                double2 va = *(const double2 *)&sl.tbuf[0], vb = *(const double2 *)&sl.tbuf[2];
                while (k + 4 <= cnt) {
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
                free_blocks -= __shfl_sync(0xFFFFFFFFu, incl, k);
                it += k + 1;
                ctx_i += (u64)(k + 1) * nrun;
                { const u32 adv = modb(k + 1); off = off + adv >= blk ? off + adv - blk : off + adv; }
                __syncwarp();
                if (arrived || counted_out || short_at) break;
            }
            if (it > 0) {
                for (u32 base = 0; base < nrun; base += 32) {
                    const u32 k = base + lane;
                    if (k < nrun) { sl.seen[k] += it; sl.rem[k] -= it; }
                }
                const u64 tok = (u64)it * nrun;
                dec_tok += tok; n_req_iters += tok; n_iters += it;
                __syncwarp();
                if (it == min_rem) retire();
                continue;
            }
        }

        // ---- one pass over the slots: decoding requests (one token each, context = cached + 1) and
        // how many of them need one more block because their last one is full ----
        u32 n_dec, needed;
        u64 ctx;
        auto count_decoders = [&]() {
            u32 packed = 0;                                        // needed << 16 | decoders: both <= 256 per lane sum
            u64 c = 0;
            for (u32 base = 0; base < nrun; base += 32) {
                const u32 k = base + lane;
                if (k < nrun && sl.todo[k] == 0) {
                    const u32 sn = sl.seen[k];
                    packed += 1u + ((modb(sn) == 0) ? 0x10000u : 0u);
                    c += (u64)sn + 1;
                }
            }
            packed = fuse_warp_sum32(packed);
            n_dec = packed & 0xFFFFu; needed = packed >> 16;
            ctx = fuse_warp_sum(c);
        };
        count_decoders();
        if (needed > free_blocks) {                                // evict the youngest, recompute later
            while (needed > free_blocks) {
                const u32 v = nrun - 1;
                const u32 td = sl.todo[v], sn = sl.seen[v], rq = sl.req[v], rm = sl.rem[v];
                free_blocks += blocks_of(sn + td);                 // what it took at admission, plus its decode blocks
                if (td == 0 && modb(sn) == 0) needed--;
                if (td > 0) n_pre--;
                const u32 out = __ldg(tr.in_len + rq) ? __ldg(tr.out_len + rq) : Lout;
                __syncwarp();
                if (lane == 0) gen[rq] = out - rm;
                nrun--;
                next = rq;
            }
            __syncwarp();
            refresh_head();
            count_decoders();
        }
        free_blocks -= needed;

        // ---- plan: the rest of the budget goes to prompts in arrival order ----
        const u64 left0 = budget > n_dec ? budget - n_dec : 0;
        u64 T = n_dec, A = ctx, C = ctx;
        u32 E = n_dec, n_chunk = 0, n_finish = 0;
        const bool chunks = n_pre > 0 && left0 > 0;
        u32 plan_q = 0;                                            // prompt tokens this lane's slot gets (slots 0..31)
        if (chunks) {
            u64 carry = 0, pT = 0, pA = 0, pC = 0;
            u32 pEN = 0;                                           // finishing << 16 | chunks
            plan_q = 0;
            for (u32 base = 0; base < nrun && carry < left0; base += 32) {
                const u32 k = base + lane;
                const u64 td = k < nrun ? sl.todo[k] : 0;
                const u64 incl = fuse_warp_scan(td, lane);
                const u64 start = carry + incl - td;               // prompt tokens asked for by older requests
                if (td > 0 && start < left0) {
                    const u64 q = min(td, left0 - start);
                    const u64 upto = (u64)sl.seen[k] + q;
                    pT += q; pA += q * upto; pC += upto;
                    pEN += 1u + (q == td ? 0x10000u : 0u);
                    plan_q = (u32)q;                               // with at most 32 residents the pass below needs no second scan
                }
                carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            T += fuse_warp_sum(pT); A += fuse_warp_sum(pA); C += fuse_warp_sum(pC);
            pEN = fuse_warp_sum32(pEN);
            n_chunk = pEN & 0xFFFFu; n_finish = pEN >> 16;
            E += n_finish;
        }
        const double t_iter = stage_time(T, E, A, C);
        const double after = clock + t_iter;

        // ---- apply ----
        bool any_done = false;
        if (!chunks) {
            for (u32 base = 0; base < nrun; base += 32) {
                const u32 k = base + lane;
                if (k < nrun && sl.todo[k] == 0) {                  // decoded one token
                    sl.seen[k] += 1;
                    const u32 rm = sl.rem[k] - 1;
                    sl.rem[k] = rm;
                    any_done |= rm == 0;
                }
            }
        } else if (nrun <= 32) {
            // one slot per lane: the chunk sizes are those of the plan
            if (lane < nrun) {
                const u32 td = sl.todo[lane];
                if (td == 0) {                                      // decoded one token
                    sl.seen[lane] += 1;
                    const u32 rm = sl.rem[lane] - 1;
                    sl.rem[lane] = rm;
                    any_done |= rm == 0;
                } else if (plan_q) {
                    sl.seen[lane] += plan_q;
                    sl.todo[lane] = td - plan_q;
                    if (plan_q == td) {                             // prompt finished: first token
                        const u32 rm = sl.rem[lane] - 1;
                        sl.rem[lane] = rm;
                        any_done |= rm == 0;
                        if (sl.fresh[lane]) { first[sl.req[lane]] = after; sl.fresh[lane] = 0; }
                    }
                }
            }
            n_pre -= n_finish;
        } else {
            u64 carry = 0;
            for (u32 base = 0; base < nrun; base += 32) {
                const u32 k = base + lane;
                const bool valid = k < nrun;
                const u64 td = valid ? sl.todo[k] : 0;
                const u64 incl = fuse_warp_scan(td, lane);
                const u64 start = carry + incl - td;
                if (valid) {
                    if (td == 0) {                                  // decoded one token
                        sl.seen[k] += 1;
                        const u32 rm = sl.rem[k] - 1;
                        sl.rem[k] = rm;
                        any_done |= rm == 0;
                    } else if (start < left0) {
                        const u64 q = min(td, left0 - start);
                        sl.seen[k] += (u32)q;
                        sl.todo[k] = (u32)(td - q);
                        if (q == td) {                              // prompt finished: first token
                            const u32 rm = sl.rem[k] - 1;
                            sl.rem[k] = rm;
                            any_done |= rm == 0;
                            if (sl.fresh[k]) { first[sl.req[k]] = after; sl.fresh[k] = 0; }
                        }
                    }
                }
                carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            n_pre -= n_finish;
        }
        any_done = __any_sync(0xFFFFFFFFu, any_done);
        if (n_dec > 0) { dec_time = dec_time + t_iter; dec_tok += n_dec; }
        clock = after;
        n_iters++;
        n_req_iters += (u64)n_dec + n_chunk;
        __syncwarp();

        if (any_done) retire();
    }
    __syncwarp();
    if (lane == 0) {
        sl.res.clock = clock; sl.res.dec_time = dec_time; sl.res.dec_tok = dec_tok; sl.res.n_iters = n_iters;
        sl.res.n_req_iters = n_req_iters;
    }
    __syncwarp();
    return st;
}

}  // namespace guide
