// Tiled walk over a closed-form space, shared by the evaluation kernel and the fused selection
// kernels.
//
// The integer task table of a config depends on (model, batch, TP, lengths) only, and within one
// (model, batch) the (TP, length) positions are the fastest-running part of the config index.  A
// thread therefore owns one (model, batch, TP, length) point, builds both stage tables once, and
// walks a chunk of the hardware x framework pairs, which are the only things the roofline
// evaluation needs beyond the table.  A warp's 32 threads hold 32 consecutive config indices for
// every pair, so whatever is stored per config goes out as 256-byte runs.
#pragma once
#include "model.cuh"

namespace guide {

struct Range { u64 first, count; };

struct TileGeom {
    u32 threads;        // block size (multiple of 32, <= 256)
    u32 tiles_per_mb;   // blocks along the (TP, length) plane of one (model, batch)
    u32 gx;             // n_models * n_batch * tiles_per_mb
    u32 splits;         // chunks of the hardware x framework axis (grid.y)
    u32 hf_chunk;       // pairs per chunk
};

// emit(valid, j, metrics), j = config index - r.first, is called by every thread of the block exactly
// hf_chunk times, valid or not, so emit may contain block-wide barriers.
template <int TIME_SUM, class Emit>
__device__ __forceinline__ void tiled_visit(const DSpace &s, const Range &r, int tp_model, u32 hf_chunk,
                                            u32 tiles_per_mb, Emit &&emit) {
    const u32 n_tl = s.n_t * s.n_l;
    const u32 n_hf = s.n_h * s.n_f;
    // blockIdx.x -> (model, batch, tile of the (TP, length) plane); blockIdx.y -> chunk of pairs
    const u32 tile = blockIdx.x % tiles_per_mb;
    const u32 mb = blockIdx.x / tiles_per_mb;
    const u32 bpos = mb % s.n_b, mpos = mb / s.n_b;
    const u32 tl_raw = tile * blockDim.x + threadIdx.x;
    const bool active = tl_raw < n_tl;
    const u32 tl = active ? tl_raw : n_tl - 1;
    const u32 tpos = tl / s.n_l, lpos = tl % s.n_l;
    const u32 hf0 = blockIdx.y * hf_chunk;

    const DModel m = s.models[mpos];
    const u32 t = s.tp[tpos], b_all = s.batch[bpos];
    const u32 b = replica_batch(b_all, s.dp[tpos]);
    const uint2 pr = s.pairs[lpos];
    const u32 lin = pr.x, lout = pr.y, n = lout - 1;
    const MemInfo mi = mem_info(m, t);
    const u32 tt = tp_model ? 1u : t;
    const double lf = log2_rule_factor(t, tp_model);
    const double Nd = (double)m.N;

    // The stage tables are built when the first config of this thread turns out to fit: threads
    // whose configs never do (head counts not divisible by the TP degree, lengths too long for
    // every memory in the chunk) skip the integer work altogether.
    TaskTab kp, kd;
    bool built = false;
    auto build_tables = [&]() {
        const u64 Tp = (u64)b * lin;
        build_fixed_tasks(m, tt, Tp, b, 1, kp);
        build_attn_tasks(m, tt, Tp, Tp * lin, Tp, kp);
        const u32 nn = n > 0 ? n : 1;          // a table is built either way; unused when n == 0
        const u64 Td = (u64)b * nn;
        const u64 ctx = (u64)b * ((u64)nn * lin + ((u64)nn * (nn + 1)) / 2);
        build_fixed_tasks(m, tt, Td, Td, nn, kd);
        build_attn_tasks(m, tt, Td, ctx, ctx, kd);
        built = true;
    };
    // index of this thread's config for pair (h, f): ((((m n_h + h) n_f + f) n_b + b) n_t n_l) + tl.
    // j is its offset in the caller's range, kept as a running value; as an unsigned number it is
    // below r.count exactly when the index lies inside [first, first + count).
    const u64 stride_hf = (u64)s.n_b * n_tl;
    u64 j = ((u64)mpos * n_hf + hf0) * stride_hf + (u64)bpos * n_tl + tl - r.first;

    ReqBytes rq;
    rq.block = 0; rq.bytes = 1; rq.inv = 1.0; rq.small = false;
    const u64 S = (u64)lin + lout;
    const double nd = (double)n;
    const double tok = cvt((u64)b_all * n);
    const u32 heads_bad = ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) ? 4u : 0u;   // t is a power of two
    const u32 hf_end = min(hf_chunk, n_hf > hf0 ? n_hf - hf0 : 0u);

#pragma unroll 2
    for (u32 i = 0; i < hf_chunk; i++, j += stride_hf) {
        const u32 hf = hf0 + i;
        const bool valid = active && i < hf_end && j < r.count;
        Metrics out;
        out.status = 0xFF;
        if (valid) {
            // memory check (Sec. 3.2 Step 1, Sec. 3.3.1): one 16-byte load per pair
            const ulonglong2 hm = __ldg(s.hfmem + hf);
            const u32 block = (u32)hm.y;
            if (block != rq.block) req_bytes_for(rq, block, S, mi.kv_tok);
            u64 bmax = 0;
            u32 st = heads_bad;
            if (hm.x > mi.w_gpu) {
                const u64 avail = hm.x - mi.w_gpu;
                bmax = (rq.small && (avail >> 52) == 0) ? floor_div_recip(avail, rq.bytes, rq.inv) : avail / rq.bytes;
            } else st |= 1;
            if ((u64)b > bmax) st |= 2;
            out.status = st;
            out.bmax = clamp_u32(bmax);
            if (st) set_infeasible(out);
            else {
                if (!built) build_tables();
                const DRate &rt = s.rates[hf];
                const double inf = __longlong_as_double(0x7FF0000000000000LL);
                const double t_pre = eval_phase<TIME_SUM>(kp, rt, Nd, lf);
                const double t_dec = n > 0 ? eval_phase<TIME_SUM>(kd, rt, Nd, lf) : 0.0;
                const u32 ci = hf * s.n_t + tpos;
                out.ttft = t_pre;
                out.latency = t_pre + t_dec;
                out.cost_hr = __ldg(s.cost_hr + ci);
                if (n > 0) {
                    out.tpot = t_dec / nd;
                    out.thr = tok / t_dec;
                    out.cost_tok = __ldg(s.cost_sec + ci) / out.thr;
                } else {
                    out.tpot = 0.0; out.thr = 0.0; out.cost_tok = inf;
                }
                out.n_iters = 1 + (u64)n;
                out.n_req_iters = (u64)b_all * (1 + (u64)n);
            }
        }
        emit(valid, j, out);
    }
}

// Host side: block and grid shape.  want_blocks steers how finely the pair axis is split (longer
// chunks amortise the table building over more configs); max_blocks bounds the whole grid.
// Returns false when the space does not suit the tiled walk.
inline bool tiled_geometry(const DSpace &s, u64 want_blocks, u64 max_blocks, TileGeom *g) {
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f;
    if (n_tl < 32 || s.chunked) return false;     // split prompt processing differs per framework: no shared tables
    g->threads = n_tl >= 256 ? 256 : ((n_tl + 31) / 32) * 32;
    g->tiles_per_mb = (n_tl + g->threads - 1) / g->threads;
    const u64 gx = (u64)s.n_m * s.n_b * g->tiles_per_mb;
    if (gx > 0x7FFFFFFFull || gx > max_blocks) return false;
    u64 splits = (want_blocks + gx - 1) / gx;
    if (splits < 1) splits = 1;
    if (splits > n_hf) splits = n_hf;
    if (gx * splits > max_blocks) splits = max_blocks / gx;
    if (splits > 65535) splits = 65535;
    g->hf_chunk = (u32)((n_hf + splits - 1) / splits);
    g->splits = (n_hf + g->hf_chunk - 1) / g->hf_chunk;
    g->gx = (u32)gx;
    return true;
}

}  // namespace guide
