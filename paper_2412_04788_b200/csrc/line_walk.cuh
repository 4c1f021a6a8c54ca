// The walk of the closed-form model over whole lines of the (TP, length) plane: sixteen consecutive
// positions of one (model, batch), 128 bytes of every metric array.  Shared by the kernel that
// stores the metrics (closed_form.cu) and, through other sinks, usable by any consumer of the
// evaluated configs.
//
// A warp takes one line for one (model, batch) and a chunk of the sorted pair walk.  Its 32 lanes
// build the stage tables of the sixteen points (one point and one stage each).  Pairs are taken
// eight at a time; for each of the four foursomes of the line the lanes are four points x eight
// pairs, as in model_walk, with the rates of a lane's pair loaded once for the four passes.
#pragma once
#include "model_walk.cuh"

namespace guide {

static constexpr u32 LINE_CHUNK = 64;           // sorted pairs per work item
static constexpr u32 LINE_TABLE_DOUBLES = 2 * 24 * 16;   // shared memory of one warp's two stage tables

// put(q, fits, pair_live, j, latency, ttft, tpot, thr, cost_hr, cost_tok): every lane, for q = 0..3,
//   its config of point 4 q + u (u = lane & 3) and pair lane >> 2: j is the config index, fits whether
//   it fits (constants otherwise), pair_live whether any config of the line fits for the lane's pair.
// flush(live, fit4, hf, j_line, b_all, lpos0): the whole warp, after the four puts of a group of
//   eight pairs: live = ballot of lanes with a fitting config, fit4 = the lane's four fit bits,
//   hf = the lane's pair, j_line = index of the line's first config for pair 0.
template <int TIME_SUM, class Put, class Flush>
__device__ __forceinline__ void line_walk(const DSpace &s, int tp_model, u32 n_chunks, unsigned *ticket, LineTab &tb_pre,
                                          LineTab &tb_dec, Put &&put, Flush &&flush) {
    const u32 lane = threadIdx.x & 31;
    const u32 u = lane & 3, h = lane >> 2;
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f, n_lines = n_tl >> 4;
    const u32 n_mb = s.n_m * s.n_b;
    const u32 n_items = n_mb * n_lines * n_chunks;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    const u64 stride_hf = (u64)s.n_b * n_tl;
    for (;;) {
        u32 item = 0;
        if (lane == 0) item = atomicAdd(ticket, 1u);
        item = __shfl_sync(0xFFFFFFFFu, item, 0);
        if (item >= n_items) break;
        const u32 mb = item % n_mb, rest = item / n_mb;
        const u32 rank = rest % n_lines, chunk_i = rest / n_lines;
        const u32 bpos = mb % s.n_b, mpos = mb / s.n_b;
        const u32 tl0 = __ldg(s.line_order + (size_t)mpos * n_lines + rank) * 16;
        const u32 tpos = tl0 / s.n_l, lpos0 = tl0 % s.n_l;        // sixteen divides the length axis: one TP degree per line
        const DModel *mp = s.models + mpos;
        const u32 t = s.tp[tpos], b_all = s.batch[bpos];
        const u32 b = replica_batch(b_all, s.dp[tpos]);
        if ((mp->nh & (t - 1)) != 0 || (mp->nkv & (t - 1)) != 0) continue;      // nothing of the line fits
        const u32 log2t = 31 - __clz(t);
        const u64 w_gpu = (mp->wbytes + (u64)(t - 1)) >> log2t;  // as mem_info
        const u64 kv_tok = mp->kv2 >> log2t;
        const u32 p_lo = chunk_i * LINE_CHUNK, p_hi = min(n_hf, p_lo + LINE_CHUNK);
        auto need_of = [&](u64 S, u32 block) {
            const u64 s_blk = block == 1 ? S : ((S + block - 1) / block) * block;
            const u64 bytes = s_blk * kv_tok;
            return __umul64hi((u64)b, bytes) ? ~0ull : (u64)b * bytes;
        };
        // Does anything fit?  Per KV block size the first pair of the chunk has the most memory.
        const uint2 pr16 = s.pairs[lpos0 + (lane & 15)];          // the point this lane builds a table for
        {
            bool any = false;
            const u64 S = (u64)pr16.x + pr16.y;
            for (u32 p0 = p_lo; p0 < p_hi;) {
                const HfSorted e0 = s.hf_sorted[p0];
                any |= e0.usable > w_gpu && e0.usable - w_gpu >= need_of(S, e0.block);
                p0 = e0.seg_end;
            }
            if (!__any_sync(0xFFFFFFFFu, any)) continue;
        }
        __syncwarp();                                 // the previous item's reads of the tables are over
        build_stage_table(mp, tp_model ? 1u : t, b, pr16.x, pr16.y - 1, lane >> 4, (lane >> 4) ? &tb_dec : &tb_pre, lane & 15);
        __syncwarp();
        // the four points this lane evaluates: 4q + u
        u64 S4[4];
        u32 n4[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            const uint2 pr = s.pairs[lpos0 + 4 * q + u];
            S4[q] = (u64)pr.x + pr.y; n4[q] = pr.y - 1;
        }
        const u64 j_line = (u64)mpos * n_hf * stride_hf + (u64)bpos * n_tl + tl0;
        const double lf = log2_rule_factor(t, tp_model);
        const double Nd = (double)mp->N;
        u32 p0 = p_lo;
        while (p0 < p_hi) {
            // one KV block size at a time: within it the pairs are sorted by falling usable memory
            const HfSorted e0 = s.hf_sorted[p0];
            const u32 seg_end = min(e0.seg_end, p_hi);
            u64 need4[4];
#pragma unroll
            for (int q = 0; q < 4; q++) need4[q] = need_of(S4[q], e0.block);
            for (u32 pp = p0; pp < seg_end; pp += 8) {
                const u32 p = pp + h;
                const bool in = p < seg_end;
                const HfSorted e = s.hf_sorted[in ? p : seg_end - 1];
                const bool room = in && e.usable > w_gpu;
                const u64 avail = room ? e.usable - w_gpu : 0;
                u32 fit4 = 0;
#pragma unroll
                for (int q = 0; q < 4; q++) fit4 |= (room && avail >= need4[q]) ? 1u << q : 0u;
                const u32 live = __ballot_sync(0xFFFFFFFFu, fit4 != 0);      // lanes with a config that fits
                if (live == 0) break;                 // nor does any later pair of this block size
                const bool pair_live = ((live >> (lane & ~3u)) & 0xFu) != 0;   // this lane's pair has one in the line
                RateRegs r;
                double c_hr = inf, c_sec = 0.0;
                if (fit4) {
                    const double2 *q = reinterpret_cast<const double2 *>(s.rate10 + (size_t)e.hf * 10);
                    const double2 q0 = __ldg(q), q1 = __ldg(q + 1), q2 = __ldg(q + 2), q3 = __ldg(q + 3), q4 = __ldg(q + 4);
                    r.icL = q0.x; r.icA = q0.y; r.icE = q1.x; r.imL = q1.y; r.imA = q2.x; r.imE = q2.y;
                    r.inv_comm = q3.x; r.clat = q3.y; r.tovh = q4.x; r.flash = q4.y;
                    const u32 ci = e.hf * s.n_t + tpos;
                    c_hr = __ldg(s.cost_hr + ci);
                    c_sec = __ldg(s.cost_sec + ci);
                }
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    double latency = inf, ttft = inf, tpot = inf, thr = 0.0, cost_hr = inf, cost_tok = inf;
                    if (fit4 & (1u << q)) {
                        const u32 n = n4[q];
                        const double t_pre = eval_stage<TIME_SUM>(tb_pre, 4 * q + u, r, Nd, lf);
                        const double t_dec = n > 0 ? eval_stage<TIME_SUM>(tb_dec, 4 * q + u, r, Nd, lf) : 0.0;
                        ttft = t_pre;
                        latency = t_pre + t_dec;
                        cost_hr = c_hr;
                        if (n > 0) {
                            tpot = t_dec / (double)n;
                            thr = cvt((u64)b_all * n) / t_dec;
                            cost_tok = c_sec / thr;
                        } else {
                            tpot = 0.0; thr = 0.0; cost_tok = inf;
                        }
                    }
                    put(q, (fit4 >> q) & 1u, pair_live, j_line + (u64)e.hf * stride_hf + 4 * q + u, latency, ttft, tpot, thr, cost_hr,
                        cost_tok);
                }
                flush(live, fit4, e.hf, j_line, b_all, lpos0);
            }
            p0 = e0.seg_end;
        }
    }
}

}  // namespace guide
