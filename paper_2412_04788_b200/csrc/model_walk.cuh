// The walk of the closed-form model kernel over the configs that fit, shared by the kernel that
// stores the metrics (closed_form.cu) and by the fused selection kernels (select_stream.cu).
#pragma once
#include "model.cuh"

namespace guide {

static constexpr u32 MODEL_THREADS = 128;
static constexpr u32 MODEL_BLOCKS_PER_SM = 8;
static constexpr u32 MODEL_CHUNK = 64;  // sorted pairs per work item

// Stage table of one point in shared memory: the 24 entries of a TaskTab, interleaved over the
// four points of a foursome so that the lanes of a warp read neighbouring 8-byte words (a 64-bit
// shared load of a warp costs two wavefronts, a 128-bit one four, whatever the lanes share).
typedef double StageTab[24][4];
enum { E_F1, E_B1, E_F2, E_B2, E_F3, E_B3, E_F5, E_B5, E_F6, E_B6, E_F7, E_B7, E_F8, E_B8, E_F9, E_B9, E_B9X, E_F10, E_B10X,
       E_F13, E_B13, E_HOPS, E_CBYTES, E_RD };

// A line of the plane (sixteen points, 128 bytes of every metric array) keeps its tables the same way.
typedef double LineTab[24][16];

template <class Tab>
__device__ __forceinline__ void put_stage(Tab &tb, u32 u, const TaskTab &k) {
    tb[E_F1][u] = k.F1; tb[E_B1][u] = k.B1; tb[E_F2][u] = k.F2; tb[E_B2][u] = k.B2; tb[E_F3][u] = k.F3; tb[E_B3][u] = k.B3;
    tb[E_F5][u] = k.F5; tb[E_B5][u] = k.B5; tb[E_F6][u] = k.F6; tb[E_B6][u] = k.B6; tb[E_F7][u] = k.F7; tb[E_B7][u] = k.B7;
    tb[E_F8][u] = k.F8; tb[E_B8][u] = k.B8; tb[E_F9][u] = k.F9; tb[E_B9][u] = k.B9; tb[E_B9X][u] = k.B9x; tb[E_F10][u] = k.F10;
    tb[E_B10X][u] = k.B10x; tb[E_F13][u] = k.F13; tb[E_B13][u] = k.B13; tb[E_HOPS][u] = k.hops; tb[E_CBYTES][u] = k.cbytes;
    tb[E_RD][u] = k.Rd;
}

// One stage table of one point, written to shared memory: stage 0 is the prompt pass, stage 1 the
// aggregated decode steps.  Eight lanes of a warp call it together (four points x two stages): the
// instruction stream is the same for both stages, only the token counts differ.  Kept out of line:
// it runs once per work item and needs far more registers than the walk around it.
template <class Tab>
static __device__ __noinline__ void build_stage_table(const DModel *mp, u32 tt, u32 b, u32 lin, u32 n, u32 stage, Tab *tb, u32 u) {
    const DModel m = *mp;
    TaskTab k;
    const u32 nn = n > 0 ? n : 1;          // a decode table is built either way; unused when n == 0
    const u64 Tp = (u64)b * lin, Td = (u64)b * nn;
    const u64 ctx = (u64)b * ((u64)nn * lin + ((u64)nn * (nn + 1)) / 2);
    const u64 T = stage ? Td : Tp;
    build_fixed_tasks(m, tt, T, stage ? Td : (u64)b, stage ? (u64)nn : 1ull, k);
    build_attn_tasks(m, tt, T, stage ? ctx : Tp * lin, stage ? ctx : Tp, k);
    put_stage(*tb, u, k);
}

// rates of one pair in registers (a row of rate10)
struct RateRegs { double icL, icA, icE, imL, imA, imE, inv_comm, clat, tovh, flash; };

// eval_phase of model.cuh, operation for operation, with the task entries read from a StageTab
template <int TIME_SUM, class Tab>
__device__ __forceinline__ double eval_stage(const Tab &tb, u32 u, const RateRegs &r, double Nd, double log2_factor) {
    const double t2 = task_time<TIME_SUM>(tb[E_F2][u], tb[E_B2][u], r.icL, r.imL);
    double sfix = task_time<TIME_SUM>(tb[E_F1][u], tb[E_B1][u], r.icE, r.imE);
    sfix = sfix + t2;
    sfix = sfix + task_time<TIME_SUM>(tb[E_F3][u], tb[E_B3][u], r.icL, r.imL);
    sfix = sfix + t2;
    sfix = sfix + task_time<TIME_SUM>(tb[E_F5][u], tb[E_B5][u], r.icE, r.imE);
    sfix = sfix + task_time<TIME_SUM>(tb[E_F6][u], tb[E_B6][u], r.icL, r.imL);
    sfix = sfix + task_time<TIME_SUM>(tb[E_F7][u], tb[E_B7][u], r.icE, r.imE);
    sfix = sfix + task_time<TIME_SUM>(tb[E_F8][u], tb[E_B8][u], r.icL, r.imL);
    // without FlashAttention the score matrix adds to the bytes of qk / sv and gives softmax its own
    const double b9 = r.flash != 0.0 ? tb[E_B9][u] : tb[E_B9X][u];
    const double b10 = r.flash != 0.0 ? 0.0 : tb[E_B10X][u];
    const double t9 = task_time<TIME_SUM>(tb[E_F9][u], b9, r.icA, r.imA);
    const double t10 = task_time<TIME_SUM>(tb[E_F10][u], b10, r.icA, r.imA);
    const double satt = (t9 + t10) + t9;
    const double scomm = 2.0 * (tb[E_HOPS][u] * r.clat + tb[E_CBYTES][u] * r.inv_comm);
    const double thead = task_time<TIME_SUM>(tb[E_F13][u], tb[E_B13][u], r.icL, r.imL);
    return combine_phase(sfix, satt, scomm, thead, tb[E_RD][u], Nd, r.tovh, log2_factor);
}

// Performance model for the configs that fit (Sec. 3.2 Step 2, Sec. 3.4.2, Sec. 3.5.1).  A warp takes one foursome of the plane for one
// (model, batch) and a chunk of the sorted pair walk; its lanes are four points x eight pairs, so
// the four lanes that share a pair write one whole sector.  The stage tables of the four points
// sit in shared memory (built once per item by eight lanes), the rates of a lane's pair in
// registers: that is half the registers of a table per thread, hence twice the warps.  Work items
// differ wildly in cost (most have nothing that fits): they are handed out through a counter to a
// persistent grid, heaviest chunks and foursomes first.
//
// emit(fits, vote, lane, j, latency, ttft, tpot, thr, cost_hr, cost_tok, n_iters, n_req_iters) is
// called by all 32 lanes for every group of eight pairs in which some lane's config fits: j is the
// lane's config index, vote the ballot of `fits`; a lane whose config does not fit passes the
// constants of a config that does not fit.
template <int TIME_SUM, class Emit>
__device__ __forceinline__ void model_walk(const DSpace &s, int tp_model, u32 n_chunks, unsigned *ticket, Emit &&emit) {
    __shared__ StageTab s_tab[MODEL_THREADS / 32][2];
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 u = lane & 3, h = lane >> 2;
    StageTab &tb_pre = s_tab[warp][0], &tb_dec = s_tab[warp][1];
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f, n_four = n_tl >> 2;
    const u32 n_mb = s.n_m * s.n_b;
    const u32 n_items = n_mb * n_four * n_chunks;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    const u64 stride_hf = (u64)s.n_b * n_tl;
    for (;;) {
        u32 item = 0;
        if (lane == 0) item = atomicAdd(ticket, 1u);
        item = __shfl_sync(0xFFFFFFFFu, item, 0);
        if (item >= n_items) break;
        const u32 mb = item % n_mb, rest = item / n_mb;
        const u32 rank = rest % n_four, chunk_i = rest / n_four;
        const u32 bpos = mb % s.n_b, mpos = mb / s.n_b;
        const u32 tl = __ldg(s.plane_order + (size_t)mpos * n_four + rank) * 4 + u;
        const u32 tpos = tl / s.n_l, lpos = tl % s.n_l;
        const DModel *mp = s.models + mpos;
        const u32 t = s.tp[tpos], b_all = s.batch[bpos];
        const u32 b = replica_batch(b_all, s.dp[tpos]);
        const u32 nh = mp->nh, nkv = mp->nkv;
        if ((nh & (t - 1)) != 0 || (nkv & (t - 1)) != 0) continue;          // the foursome shares its TP degree: nothing fits
        const uint2 pr = s.pairs[lpos];
        const u32 lin = pr.x, lout = pr.y, n = lout - 1;
        const u32 log2t = 31 - __clz(t);
        const u64 w_gpu = (mp->wbytes + (u64)(t - 1)) >> log2t;            // as mem_info
        const u64 kv_tok = mp->kv2 >> log2t;
        const u64 S = (u64)lin + lout;
        const u32 p_lo = chunk_i * MODEL_CHUNK, p_hi = min(n_hf, p_lo + MODEL_CHUNK);
        // Does anything fit?  Per KV block size the first pair of the chunk has the most memory.
        bool any = false;
        for (u32 p0 = p_lo; p0 < p_hi;) {
            const HfSorted e0 = s.hf_sorted[p0];
            const u64 s_blk = e0.block == 1 ? S : ((S + e0.block - 1) / e0.block) * e0.block;
            const u64 bytes = s_blk * kv_tok;
            const u64 need = __umul64hi((u64)b, bytes) ? ~0ull : (u64)b * bytes;
            any |= e0.usable > w_gpu && e0.usable - w_gpu >= need;
            p0 = e0.seg_end;
        }
        if (!__any_sync(0xFFFFFFFFu, any)) continue;
        __syncwarp();                                 // the previous item's reads of the tables are over
        if (h < 2) build_stage_table(mp, tp_model ? 1u : t, b, lin, n, h, h ? &tb_dec : &tb_pre, u);   // lanes 0-3: prompt stage of point u; 4-7: decode stage
        __syncwarp();
        const u64 j0 = (u64)mpos * n_hf * stride_hf + (u64)bpos * n_tl + tl;
        const double lf = log2_rule_factor(t, tp_model);
        const double Nd = (double)mp->N;
        u32 p0 = p_lo;
        while (p0 < p_hi) {
            // one KV block size at a time: within it the pairs are sorted by falling usable memory
            const HfSorted e0 = s.hf_sorted[p0];
            const u32 seg_end = min(e0.seg_end, p_hi);
            const u64 s_blk = e0.block == 1 ? S : ((S + e0.block - 1) / e0.block) * e0.block;
            const u64 bytes = s_blk * kv_tok;
            const u64 need = __umul64hi((u64)b, bytes) ? ~0ull : (u64)b * bytes;
            for (u32 pp = p0; pp < seg_end; pp += 8) {
                const u32 p = pp + h;
                const bool in = p < seg_end;
                const HfSorted e = s.hf_sorted[in ? p : seg_end - 1];
                // fits <=> usable > weights and b <= floor((usable - weights) / bytes) <=> b x bytes <= usable - weights
                const bool fits = in && e.usable > w_gpu && e.usable - w_gpu >= need;
                const u32 vote = __ballot_sync(0xFFFFFFFFu, fits);
                if (vote == 0) break;                 // nor does any later pair of this block size
                double latency = inf, ttft = inf, tpot = inf, thr = 0.0, cost_hr = inf, cost_tok = inf;
                u64 n_iters = 0, n_req_iters = 0;
                if (fits) {
                    const double2 *q = reinterpret_cast<const double2 *>(s.rate10 + (size_t)e.hf * 10);
                    const double2 q0 = __ldg(q), q1 = __ldg(q + 1), q2 = __ldg(q + 2), q3 = __ldg(q + 3), q4 = __ldg(q + 4);
                    RateRegs r;      // rate10 row: inv_c[LINEAR, ATTN, ELEM], inv_m[LINEAR, ATTN, ELEM], inv_comm, clat, tovh, flash
                    r.icL = q0.x; r.icA = q0.y; r.icE = q1.x; r.imL = q1.y; r.imA = q2.x; r.imE = q2.y;
                    r.inv_comm = q3.x; r.clat = q3.y; r.tovh = q4.x; r.flash = q4.y;
                    const double t_pre = eval_stage<TIME_SUM>(tb_pre, u, r, Nd, lf);
                    const double t_dec = n > 0 ? eval_stage<TIME_SUM>(tb_dec, u, r, Nd, lf) : 0.0;
                    const u32 ci = e.hf * s.n_t + tpos;
                    ttft = t_pre;
                    latency = t_pre + t_dec;
                    cost_hr = __ldg(s.cost_hr + ci);
                    if (n > 0) {
                        tpot = t_dec / (double)n;
                        thr = cvt((u64)b_all * n) / t_dec;
                        cost_tok = __ldg(s.cost_sec + ci) / thr;
                    } else {
                        tpot = 0.0; thr = 0.0; cost_tok = inf;
                    }
                    n_iters = 1 + (u64)n;
                    n_req_iters = (u64)b_all * (1 + (u64)n);
                }
                emit(fits, vote, lane, j0 + (u64)e.hf * stride_hf, latency, ttft, tpot, thr, cost_hr, cost_tok, n_iters, n_req_iters);
            }
            p0 = e0.seg_end;
        }
    }
}

}  // namespace guide
