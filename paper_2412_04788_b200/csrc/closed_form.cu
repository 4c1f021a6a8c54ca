// Closed-form evaluation kernels: one prefill stage + one aggregated decode stage per config
// (Sec. 3.2 Steps 1-2, roofline of Sec. 3.4.2, time decomposition of Sec. 3.5.1).
#include <algorithm>

#include "guide_internal.cuh"
#include "model_walk.cuh"
#include "line_walk.cuh"
#include "select_sink.cuh"

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
    if (o.seq_used) __stcs(o.seq_used + j, m.seq_used);
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

// The same in binary32 (model_f32.cuh): the reduced-precision variant, values stored widened.
template <int TIME_SUM>
__global__ void __launch_bounds__(256) k_closed_form_flat_f32(DSpace s, Range r, int tp_model, guide_outputs o) {
    const u64 j = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= r.count) return;
    const Cfg c = decode_index(s, r.first + j);
    Metrics m;
    closed_form_eval_f32<TIME_SUM>(s, s.ratef, c, tp_model, m);
    store_metrics(o, j, m);
}

// Tiled evaluation (see tiled.cuh): every valid config's metrics are stored.
template <int TIME_SUM>
__global__ void __launch_bounds__(256, 2) k_closed_form_tiled(DSpace s, Range r, int tp_model, u32 hf_chunk,
                                                              u32 tiles_per_mb, guide_outputs o) {
    tiled_visit<TIME_SUM>(s, r, tp_model, hf_chunk, tiles_per_mb, [&](bool valid, u64 j, const Metrics &m) {
        if (valid) store_metrics(o, j, m);
    });
}

// ---- split evaluation ----------------------------------------------------------------------------
//
// Most configs of a large sweep do not fit their memory (Sec. 3.2 Step 1) and need no performance
// model at all: a status byte, B_max and constant metrics.  Whole-space calls are therefore served
// by two kernels.  The unit they share out is the foursome: four consecutive length positions, 32
// bytes of every metric array, one memory sector.  A sector is always written whole by one warp
// instruction of one kernel; partly written sectors cost a read-modify-write in memory and were
// measured to halve the write bandwidth.
//
//   memory kernel : every config's status and B_max, and the constant metrics of the foursomes in
//     which no config fits.  A thread takes two neighbouring positions of one (model, pair) and
//     walks the batch axis: B_max does not depend on the batch size, so its exact division is done
//     once per position; a warp's stores are 512 contiguous bytes.  Needs few registers and few
//     warps; bound by the write bandwidth.  A small persistent grid, so that the model kernel finds
//     room beside it.
//   model kernel  : the roofline model (Sec. 3.2 Step 2, Sec. 3.4.2, Sec. 3.5.1) for the configs
//     that fit, and the metrics of every foursome in which at least one does (constants for the
//     others).  A thread owns one (model, batch, TP, length) point, as in the tiled walk, and
//     visits the pairs in the order of hf_sorted: per KV block size, falling usable memory, so the
//     pairs the point fits are a prefix and the walk stops at the first pair no lane of the warp
//     fits.  Whether a config fits is one comparison here:
//     b <= floor(avail / bytes) <=> b x bytes <= avail.  Foursomes are dealt to lanes in
//     plane_order, so the lanes of a warp stop at about the same place.  Small blocks (two warps)
//     let the scheduler refill the slots of warps that had nothing to do.
//
// The model kernel is launched as a programmatic dependent of the memory kernel and waits for it
// only at its very end: the two run side by side, one bound by bandwidth and one by arithmetic,
// and write disjoint sectors.
//
// On large spaces whose length axis divides into sixteens the unit becomes the line (sixteen
// positions, 128 bytes) and k_closed_form_lines takes the model kernel's place: see below.

static constexpr u32 MEM_THREADS = 128;         // x 2 positions = 256 positions of the plane per work item
static constexpr u32 MEM_BLOCKS_PER_SM = 3;       // 12 warps keep the write path busier than 8 (workload 5: 177.4 against 180.6 us for the pair); 16 do not (181 us)
static constexpr int SPLIT_MAX_CONST = 10;

// 8-byte arrays that receive a constant for a config that does not fit (+inf, or 0 for throughput and counters)
struct ConstOut {
    unsigned long long *p[SPLIT_MAX_CONST];
    unsigned long long pat[SPLIT_MAX_CONST];
    int n;
};

// programmatic dependent launch: a kernel launched with the attribute may start while its
// predecessor runs; cf_dep_wait() returns when the predecessor has completed and flushed
__device__ __forceinline__ void cf_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void cf_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Memory check of Sec. 3.2 Step 1 / Sec. 3.3.1 for every config.  Work items: (model, tile of 256
// plane positions, pair), taken in turn by a persistent grid.
// LINE: the unit shared out with the model kernel is the line (sixteen positions, eight lanes)
// instead of the foursome (two lanes).
template <int LINE>
__global__ void __launch_bounds__(MEM_THREADS) k_closed_form_memory(DSpace s, guide_outputs o, ConstOut co, u32 tiles) {
    __shared__ unsigned long long *s_p[SPLIT_MAX_CONST];
    __shared__ unsigned long long s_pat[SPLIT_MAX_CONST];
    cf_dep_launch();
    if (threadIdx.x < SPLIT_MAX_CONST) { s_p[threadIdx.x] = co.p[threadIdx.x]; s_pat[threadIdx.x] = co.pat[threadIdx.x]; }
    __syncthreads();
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f;
    const u32 items = s.n_m * tiles * n_hf;
    const int n_const = co.n;
    for (u32 item = blockIdx.x; item < items; item += gridDim.x) {
        const u32 hf = item % n_hf;
        const u32 mt = item / n_hf;
        const u32 tile = mt % tiles, mpos = mt / tiles;
        const u32 tl_raw = tile * (2 * MEM_THREADS) + 2 * threadIdx.x;
        const bool active = tl_raw < n_tl;                  // n_l is a multiple of 4: a foursome shares its TP degree
        const u32 tl = active ? tl_raw : 0;                  // idle lanes still take part in the exchange below
        const u32 tpos = tl / s.n_l, lpos = tl % s.n_l;
        const DModel m = s.models[mpos];
        const u32 t = s.tp[tpos], dp = s.dp[tpos];
        const MemInfo mi = mem_info(m, t);
        const u32 st_base = ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) ? 4u : 0u;
        const ulonglong2 hm = __ldg(s.hfmem + hf);
        u64 bmax[2] = {0, 0};
        u32 st0 = st_base;
        if (hm.x > mi.w_gpu) {
            const u64 avail = hm.x - mi.w_gpu;
#pragma unroll
            for (int u = 0; u < 2; u++) {
                const uint2 pr = s.pairs[lpos + u];
                ReqBytes rq;
                req_bytes_for(rq, (u32)hm.y, (u64)pr.x + pr.y, mi.kv_tok);
                bmax[u] = (rq.small && (avail >> 52) == 0) ? floor_div_recip(avail, rq.bytes, rq.inv) : avail / rq.bytes;
            }
        } else st0 |= 1;
        const uint2 bm = make_uint2(clamp_u32(bmax[0]), clamp_u32(bmax[1]));
        // the largest batch size either of the two positions takes; the neighbouring lane holds the
        // other half of the foursome
        const u64 mine = st0 ? 0 : (bmax[0] > bmax[1] ? bmax[0] : bmax[1]);
        const u64 other = __shfl_xor_sync(0xFFFFFFFFu, mine, 1);
        u64 four_max = mine > other ? mine : other;         // a config of the foursome fits <=> b <= four_max
        if (LINE) {                                         // ... of the line: six more lanes
            const u64 o2 = __shfl_xor_sync(0xFFFFFFFFu, four_max, 2);
            four_max = four_max > o2 ? four_max : o2;
            const u64 o4 = __shfl_xor_sync(0xFFFFFFFFu, four_max, 4);
            four_max = four_max > o4 ? four_max : o4;
        }
        u64 j = ((u64)mpos * n_hf + hf) * ((u64)s.n_b * n_tl) + tl;
        if (active) {
            for (u32 bi = 0; bi < s.n_b; bi++, j += n_tl) {
                const u64 b = replica_batch(__ldg(s.batch + bi), dp);
                const u32 sa = st0 | (b > bmax[0] ? 2u : 0u), sb = st0 | (b > bmax[1] ? 2u : 0u);
                if (o.status) __stcs(reinterpret_cast<unsigned short *>(o.status + j), (unsigned short)(sa | (sb << 8)));
                if (o.bmax) __stcs(reinterpret_cast<uint2 *>(o.bmax + j), bm);
                if (b > four_max) {                         // nothing in the foursome fits (batch sizes are >= 1)
                    for (int a = 0; a < n_const; a++)
                        __stcs(reinterpret_cast<ulonglong2 *>(s_p[a] + j), make_ulonglong2(s_pat[a], s_pat[a]));
                }
            }
        }
    }
}

// Performance model for the configs that fit: the walk of model_walk.cuh with the metrics stored.
// The four lanes of a pair write the whole foursome (one sector per array) as soon as one of its
// configs fits, constants for the members that do not.
template <int TIME_SUM>
__global__ void __launch_bounds__(MODEL_THREADS, MODEL_BLOCKS_PER_SM)
k_closed_form_model(DSpace s, int tp_model, guide_outputs o, u32 n_chunks, unsigned *ticket) {
    model_walk<TIME_SUM>(s, tp_model, n_chunks, ticket,
                         [&](bool, u32 vote, u32 lane, u64 j, double latency, double ttft, double tpot, double thr, double cost_hr,
                             double cost_tok, u64 n_iters, u64 n_req_iters) {
        if ((vote >> (lane & ~3u)) & 0xFu) {
            if (o.latency) __stcs(o.latency + j, latency);
            if (o.ttft) __stcs(o.ttft + j, ttft);
            if (o.ttft_p50) __stcs(o.ttft_p50 + j, ttft);
            if (o.ttft_p99) __stcs(o.ttft_p99 + j, ttft);
            if (o.tpot) __stcs(o.tpot + j, tpot);
            if (o.thr_decode) __stcs(o.thr_decode + j, thr);
            if (o.cost_per_hr) __stcs(o.cost_per_hr + j, cost_hr);
            if (o.cost_per_token) __stcs(o.cost_per_token + j, cost_tok);
            if (o.n_iters) __stcs(o.n_iters + j, n_iters);
            if (o.n_req_iters) __stcs(o.n_req_iters + j, n_req_iters);
        }
    });
    // the grid must not be complete before the memory kernel is: whatever follows in the stream
    // waits for this one only
    cf_dep_wait();
}

// ---- the model kernel on lines ---------------------------------------------------------------------
//
// Isolated 32-byte stores are dear: next to the memory kernel's contiguous stream, 240 MB written as
// scattered sectors cost as much time as the 650 MB of the stream itself, written as whole 128-byte
// lines a quarter of that.  When the length axis divides into sixteens the unit the two kernels share
// out is therefore the line: sixteen consecutive positions of one (model, pair, batch size), 128
// bytes of every metric array.
//
// A warp takes one line of the plane for one (model, batch) and a chunk of the sorted pair walk.  Its
// 32 lanes build the stage tables of the sixteen points (one point and one stage each).  Pairs are
// taken eight at a time; for each of the four foursomes of the line the lanes are four points x
// eight pairs, as in model_walk, with the rates of a lane's pair loaded once for the four passes.
// Results go to a per-warp staging area in shared memory (constants for configs that do not fit) and
// leave it as whole lines: eight lanes x 16 bytes per (pair, array), for every pair with a config
// that fits anywhere in the line.
static constexpr u32 LINE_BLOCKS_PER_SM = 4;
static constexpr u32 LINE_STAGE_ARRAYS = 6;     // latency, ttft, tpot, throughput, cost per hour, cost per token
static constexpr u32 LINE_STAGE_ROW = 20;       // doubles per (array, pair) row: 16 + 4 of padding against bank conflicts
static constexpr u32 LINE_WARP_DOUBLES = LINE_TABLE_DOUBLES + LINE_STAGE_ARRAYS * 8 * LINE_STAGE_ROW;
static constexpr u32 LINE_SMEM_BYTES = (MODEL_THREADS / 32) * LINE_WARP_DOUBLES * 8;
static constexpr u32 LINE_KILLERS = 64;          // killers the selecting variant keeps in shared memory (1 KB)

// SELECT: the kernel is also the filter pass of a top-k and a Pareto selection whose bound and killers
// were worked out from a sample before the launch: every config that fits is tested while its metrics
// are in registers, and the few that either selection may still want go to its survivor list, so the
// arrays need not be read back.
template <int TIME_SUM, bool SELECT>
__global__ void __launch_bounds__(MODEL_THREADS, LINE_BLOCKS_PER_SM + 1)      // registers: four blocks beside the memory kernel's three (3 x 128 x 32 + 4 x 128 x 96 registers fit the file)
k_closed_form_lines(DSpace s, int tp_model, guide_outputs o, u32 n_chunks, unsigned *ticket, LineSelect sel) {
    extern __shared__ __align__(16) double line_smem[];
    // Four blocks of this kernel fill an SM's shared memory but for a few KB: the filter keeps every
    // fourth killer of the staircase (any subset of it is a valid set of killers; fewer only let more
    // survivors through) and four pivots spread over it, which rule out most configs by themselves.
    __shared__ P2 s_killers[SELECT ? LINE_KILLERS : 1];
    __shared__ ulonglong2 s_pivot[4];
    u64 bkey = 0, bidx = 0;
    KillerSet K;
    K.k = s_killers; K.n = 0;
    if (SELECT) {
        // the kernels that made the bound and the killers completed before the memory kernel started
        const u64 *bp = reinterpret_cast<const u64 *>(sel.header_t + TK_BOUND);
        bkey = __ldcg(bp); bidx = __ldcg(bp + 1);
        const u32 n_all = min(__ldcg(sel.header_p + PH_KILLERS), PA_KILLERS);
        K.n = min(n_all, LINE_KILLERS);
        for (u32 i = threadIdx.x; i < K.n; i += blockDim.x) {
            const ulonglong2 w = __ldcg(reinterpret_cast<const ulonglong2 *>(sel.killers + ((u64)i * n_all) / K.n));
            s_killers[i].x = w.x; s_killers[i].y = w.y;
        }
        if (threadIdx.x < 4) {
            ulonglong2 w = make_ulonglong2(KEY_MAX, KEY_MAX);
            if (n_all > 0) w = __ldcg(reinterpret_cast<const ulonglong2 *>(sel.killers + (n_all * (2 * threadIdx.x + 1)) / 8));
            s_pivot[threadIdx.x] = w;
        }
        __syncthreads();
    }
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 u = lane & 3, h = lane >> 2;
    double *mine = line_smem + (size_t)warp * LINE_WARP_DOUBLES;
    LineTab &tb_pre = *reinterpret_cast<LineTab *>(mine);
    LineTab &tb_dec = *reinterpret_cast<LineTab *>(mine + 24 * 16);
    double *stage = mine + LINE_TABLE_DOUBLES;                    // [array][pair of the group][LINE_STAGE_ROW]
    const u64 stride_hf = (u64)s.n_b * s.n_t * s.n_l;
    double *const arr[LINE_STAGE_ARRAYS] = {o.latency, o.ttft, o.tpot, o.thr_decode, o.cost_per_hr, o.cost_per_token};
    line_walk<TIME_SUM>(s, tp_model, n_chunks, ticket, tb_pre, tb_dec,
        [&](int q, bool fits, bool pair_live, u64 j, double latency, double ttft, double tpot, double thr, double cost_hr, double cost_tok) {
        if (SELECT && fits) {
            // the cheap exclusions first: most configs are beyond the bound and under a pivot
            const u64 k64 = enc(pick_metric(sel.key, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
            if (pair_le(k64, j, bkey, bidx) && meets(sel.ct, latency, ttft, thr, cost_hr)) topk_keep(k64, j, sel.header_t, sel.cand);
            const u64 x = enc(pick_metric(sel.xm, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
            const u64 y = enc(pick_metric(sel.ym, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
            const ulonglong2 p0 = s_pivot[0], p1 = s_pivot[1], p2 = s_pivot[2], p3 = s_pivot[3];
            const bool dead = dominates(p0.x, p0.y, x, y) || dominates(p1.x, p1.y, x, y) || dominates(p2.x, p2.y, x, y) ||
                              dominates(p3.x, p3.y, x, y);
            if (!dead && meets(sel.cp, latency, ttft, thr, cost_hr) && !K.kills_sorted(x, y)) pareto_keep(x, y, j, sel.header_p, sel.surv);
        }
        if (pair_live) {
            double *w = stage + (size_t)h * LINE_STAGE_ROW + u + 4 * q;
            w[0 * 8 * LINE_STAGE_ROW] = latency; w[1 * 8 * LINE_STAGE_ROW] = ttft; w[2 * 8 * LINE_STAGE_ROW] = tpot;
            w[3 * 8 * LINE_STAGE_ROW] = thr; w[4 * 8 * LINE_STAGE_ROW] = cost_hr; w[5 * 8 * LINE_STAGE_ROW] = cost_tok;

        }
        },
        [&](u32 live, u32 fit4, u32 hf, u64 j_line, u32 b_all, u32 lpos0) {
        __syncwarp();
        // whole lines out: eight lanes x 16 bytes per (pair, array), four pairs per store instruction
#pragma unroll
        for (int half = 0; half < 2; half++) {
            const u32 hh = 4 * half + (lane >> 3), piece = lane & 7;
            const u32 src = 4 * hh;                                  // the lane with point 0 of pair hh
            const u32 hf_hh = __shfl_sync(0xFFFFFFFFu, hf, src);
            const u32 fits_hh = (__shfl_sync(0xFFFFFFFFu, fit4, src) & 0xFu) | ((__shfl_sync(0xFFFFFFFFu, fit4, src + 1) & 0xFu) << 4) |
                                ((__shfl_sync(0xFFFFFFFFu, fit4, src + 2) & 0xFu) << 8) | ((__shfl_sync(0xFFFFFFFFu, fit4, src + 3) & 0xFu) << 12);
            // fits_hh: bit 4 * u' + q' = point 4 q' + u' of pair hh fits
            if ((live >> src) & 0xFu) {
                const u64 j = j_line + (u64)hf_hh * stride_hf + 2 * piece;
                const double *rd = stage + (size_t)hh * LINE_STAGE_ROW + 2 * piece;
#pragma unroll
                for (u32 a = 0; a < LINE_STAGE_ARRAYS; a++) {
                    if (arr[a]) {
                        const double2 v = *reinterpret_cast<const double2 *>(rd + (size_t)a * 8 * LINE_STAGE_ROW);
                        __stcs(reinterpret_cast<double2 *>(arr[a] + j), v);
                    }
                }
                if (o.ttft_p50 || o.ttft_p99) {
                    const double2 v = *reinterpret_cast<const double2 *>(rd + (size_t)1 * 8 * LINE_STAGE_ROW);
                    if (o.ttft_p50) __stcs(reinterpret_cast<double2 *>(o.ttft_p50 + j), v);
                    if (o.ttft_p99) __stcs(reinterpret_cast<double2 *>(o.ttft_p99 + j), v);
                }
                if (o.n_iters || o.n_req_iters) {
                    // iteration counts of the two points this lane writes: 1 + n and b (1 + n), 0 when the config does not fit
                    ulonglong2 it, rq;
                    u64 *itp = &it.x, *rqp = &rq.x;
#pragma unroll
                    for (u32 k = 0; k < 2; k++) {
                        const u32 pt = 2 * piece + k;                 // point 4 q' + u'
                        const bool f = (fits_hh >> (4 * (pt & 3) + (pt >> 2))) & 1u;
                        const u64 n1 = 1 + (u64)(s.pairs[lpos0 + pt].y - 1);
                        itp[k] = f ? n1 : 0;
                        rqp[k] = f ? (u64)b_all * n1 : 0;
                    }
                    if (o.n_iters) __stcs(reinterpret_cast<ulonglong2 *>(o.n_iters + j), it);
                    if (o.n_req_iters) __stcs(reinterpret_cast<ulonglong2 *>(o.n_req_iters + j), rq);
                }
            }
        }
        __syncwarp();                         // the staging area is free for the next eight pairs
        });
    // the grid must not be complete before the memory kernel is: whatever follows in the stream
    // waits for this one only
    cf_dep_wait();
}

// Does the call suit the split kernels?  Fills the list of constant-filled arrays.
static bool split_applies(const DSpace &s, Range r, const guide_outputs &o, ConstOut *co) {
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    const u32 n_tl = s.n_t * s.n_l;
    if (r.first != 0 || r.count != total || total < (1u << 16)) return false;       // whole spaces only
    if (s.n_l % 4 != 0 || n_tl < 32 || s.chunked) return false;
    if ((u64)s.n_m * ((n_tl + 255) / 256) * s.n_h * s.n_f > 0x7FFFFFFFull) return false;
    auto al = [](const void *p, uintptr_t a) { return ((uintptr_t)p % a) == 0; };
    const void *wide[] = {o.latency, o.ttft, o.ttft_p50, o.ttft_p99, o.tpot, o.thr_decode, o.cost_per_hr, o.cost_per_token,
                          o.n_iters, o.n_req_iters};
    for (const void *p : wide)
        if (p && !al(p, 32)) return false;                  // foursomes are sectors only if the arrays start on one
    if ((o.bmax && !al(o.bmax, 8)) || (o.status && !al(o.status, 2))) return false;
    const unsigned long long inf = 0x7FF0000000000000ull;
    co->n = 0;
    for (int i = 0; i < SPLIT_MAX_CONST; i++) { co->p[i] = nullptr; co->pat[i] = 0; }
    auto add = [&](void *p, unsigned long long pat) { if (p) { co->p[co->n] = (unsigned long long *)p; co->pat[co->n] = pat; co->n++; } };
    add(o.latency, inf); add(o.ttft, inf); add(o.ttft_p50, inf); add(o.ttft_p99, inf); add(o.tpot, inf);
    add(o.thr_decode, 0); add(o.cost_per_hr, inf); add(o.cost_per_token, inf); add(o.n_iters, 0); add(o.n_req_iters, 0);
    return true;
}

// Can the two kernels share out whole lines?  The length axis must divide into sixteens and every
// 8-byte array start on a 128-byte boundary.
static bool lines_apply(const DSpace &s, const guide_outputs &o) {
    if (s.n_l % 16 != 0) return false;
    // a line is four times the work of a foursome: with fewer than two work items per resident warp
    // the foursome kernel's finer grain fills the machine better
    const u64 n_hf = (u64)s.n_h * s.n_f;
    const u64 items = (u64)s.n_m * s.n_b * (s.n_t * s.n_l / 16) * ((n_hf + LINE_CHUNK - 1) / LINE_CHUNK);
    if (items < 2ull * (u64)num_sms() * LINE_BLOCKS_PER_SM * (MODEL_THREADS / 32)) return false;
    const void *wide[] = {o.latency, o.ttft, o.ttft_p50, o.ttft_p99, o.tpot, o.thr_decode, o.cost_per_hr, o.cost_per_token,
                          o.n_iters, o.n_req_iters};
    for (const void *p : wide)
        if (p && ((uintptr_t)p % 128) != 0) return false;
    return true;
}

template <int TIME_SUM>
static int launch_split(const DSpace &s, int tp_model, const guide_outputs &o, const ConstOut &co, unsigned *ticket,
                        cudaStream_t st, const LineSelect *sel) {
    const u32 n_tl = s.n_t * s.n_l, n_hf = s.n_h * s.n_f;
    const u32 tiles = (n_tl + 2 * MEM_THREADS - 1) / (2 * MEM_THREADS);
    const u32 items = s.n_m * tiles * n_hf;
    const u32 mem_grid = std::min<u32>(items, (u32)num_sms() * MEM_BLOCKS_PER_SM);
    const bool lines = lines_apply(s, o);
    const u32 n_chunks = lines ? (n_hf + LINE_CHUNK - 1) / LINE_CHUNK : (n_hf + MODEL_CHUNK - 1) / MODEL_CHUNK;
    // refuse before anything is queued: a failed call leaves the caller's arrays untouched
    if ((u64)s.n_m * s.n_b * (n_tl / 4) * n_chunks > 0x7FFFFFFFull) return fail(GUIDE_ERR_UNSUPPORTED, "space too large for one launch");
    GUIDE_CUDA(cudaMemsetAsync(ticket, 0, 4, st));           // the model kernel's work counter
    if (lines) k_closed_form_memory<1><<<mem_grid, MEM_THREADS, 0, st>>>(s, o, co, tiles);
    else k_closed_form_memory<0><<<mem_grid, MEM_THREADS, 0, st>>>(s, o, co, tiles);
    GUIDE_CUDA(cudaGetLastError());
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(MODEL_THREADS); cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (lines) {
        // function attributes belong to the device: set them once per device and kernel variant
        static bool opted_in[64][2] = {};
        const auto plain = k_closed_form_lines<TIME_SUM, false>;
        const auto selecting = k_closed_form_lines<TIME_SUM, true>;
        static std::mutex opt_mu;
        int dev = 0;
        GUIDE_CUDA(cudaGetDevice(&dev));
        std::lock_guard<std::mutex> opt_lock(opt_mu);
        if (dev < 0 || dev >= 64 || !opted_in[dev][TIME_SUM]) {
            // more dynamic shared memory than the default limit
            GUIDE_CUDA(cudaFuncSetAttribute(plain, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LINE_SMEM_BYTES));
            GUIDE_CUDA(cudaFuncSetAttribute(selecting, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LINE_SMEM_BYTES));
            // An SM changes its split between L1 and shared memory only when it is empty.  The memory
            // kernel gets there first and needs neither: it asks for the split the line kernel needs,
            // so that the line kernel's blocks find room beside it instead of waiting for it to leave.
            GUIDE_CUDA(cudaFuncSetAttribute(k_closed_form_memory<1>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                            (int)cudaSharedmemCarveoutMaxShared));
            GUIDE_CUDA(cudaFuncSetAttribute(plain, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
            GUIDE_CUDA(cudaFuncSetAttribute(selecting, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
            if (dev >= 0 && dev < 64) opted_in[dev][TIME_SUM] = true;
        }
        cfg.gridDim = dim3((u32)num_sms() * LINE_BLOCKS_PER_SM); cfg.dynamicSmemBytes = LINE_SMEM_BYTES;
        if (sel) GUIDE_CUDA(cudaLaunchKernelEx(&cfg, selecting, s, tp_model, o, n_chunks, ticket, *sel));
        else GUIDE_CUDA(cudaLaunchKernelEx(&cfg, plain, s, tp_model, o, n_chunks, ticket, LineSelect{}));
    } else {
        cfg.gridDim = dim3((u32)num_sms() * MODEL_BLOCKS_PER_SM); cfg.dynamicSmemBytes = 0;
        GUIDE_CUDA(cudaLaunchKernelEx(&cfg, k_closed_form_model<TIME_SUM>, s, tp_model, o, n_chunks, ticket));
    }
    return GUIDE_OK;
}

int launch_closed_form_f32(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o, cudaStream_t st) {
    const u64 blocks = (r.count + 255) / 256;
    if (blocks > 0x7FFFFFFFull) return fail(GUIDE_ERR_UNSUPPORTED, "range too large for one launch");
    if (time_model) k_closed_form_flat_f32<1><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
    else k_closed_form_flat_f32<0><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

// Would launch_closed_form write this call through the memory and line kernels (the pair that can
// also act as the filter pass of a combined simulate-and-select call)?
bool closed_form_by_lines(const DSpace &s, Range r, const guide_outputs &o) {
    ConstOut co;
    return split_applies(s, r, o, &co) && lines_apply(s, o);
}

// sel: non-null only when closed_form_by_lines() holds for the call
int launch_closed_form(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o,
                       unsigned *ticket, cudaStream_t st, const LineSelect *sel) {
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    if (sel && !(ticket && closed_form_by_lines(s, r, o))) return fail(GUIDE_ERR_UNSUPPORTED, "the call does not go through the line kernel");
    // The tiled kernel pays off when a (TP, length) plane fills warps and the range is (most of)
    // the space; slivers of the space go through the flat kernel.
    ConstOut co;
    if (ticket && split_applies(s, r, o, &co))
        return time_model ? launch_split<1>(s, tp_model, o, co, ticket, st, sel) : launch_split<0>(s, tp_model, o, co, ticket, st, sel);
    TileGeom g;
    const bool tiled = r.count * 2 >= total && tiled_geometry(s, (u64)num_sms() * 16, 1ull << 30, &g);
    if (!tiled) {
        const u64 blocks = (r.count + 255) / 256;
        if (blocks > 0x7FFFFFFFull) return fail(GUIDE_ERR_UNSUPPORTED, "range too large for one launch");
        if (time_model) k_closed_form_flat<1><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
        else k_closed_form_flat<0><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
    } else {
        const dim3 grid(g.gx, g.splits);
        if (time_model) k_closed_form_tiled<1><<<grid, g.threads, 0, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, o);
        else k_closed_form_tiled<0><<<grid, g.threads, 0, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, o);
    }
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

}  // namespace guide
