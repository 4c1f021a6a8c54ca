// Trace-driven continuous-batching simulation, one warp per config (dynamic batching of Sec. 3.1;
// prompt-priority scheduling and fixed-granularity paged KV of the vLLM-like framework model,
// Sec. 2.3.2 / 2.4.1 / 2.4.2).
//
// A warp owns one config at a time and pulls the next one from a global counter, so configs
// whose schedules are long do not hold back a whole block.  The clock, counters and the
// iteration time are warp-uniform; the resident requests live in per-warp shared-memory slots,
// kept in ascending request order, which the 32 lanes scan together.  Per-request results that
// must outlive residency (tokens generated so far, first-token time, time per output token) sit
// in a per-warp slice of the workspace.  The request trace itself is the same for every config
// and is read through the read-only path, so it stays cache resident.
#include "guide_internal.cuh"

namespace guide {

static constexpr u32 SIM_WARPS_PER_BLOCK = 8;
static constexpr u32 SIM_THREADS = SIM_WARPS_PER_BLOCK * 32;
static constexpr u32 SIM_MAX_WARPS = 6144;        // workspace is sized for this many resident warps
static constexpr u32 SLOTS = GUIDE_TRACE_MAX_BATCH;
static constexpr u32 F_NEEDS_PREFILL = 0x80000000u, F_FIRST = 0x40000000u, REM_MASK = 0x3FFFFFFFu;
static constexpr u32 GEN_DONE = 0x80000000u;

static u32 pow2_at_least(u32 v) { u32 p = 1; while (p < v) p <<= 1; return p; }

static size_t per_warp_bytes(u32 n_req) {
    // gen u32[n] | first f64[n] | tpot f64[pow2(n)] (reused as the sort buffer)
    const size_t n = n_req, p = pow2_at_least(n_req);
    return ((n * 4 + 255) / 256 * 256) + ((n * 8 + 255) / 256 * 256) + ((p * 8 + 255) / 256 * 256);
}

size_t trace_workspace_bytes(u32 n_req) { return 256 + (size_t)SIM_MAX_WARPS * per_warp_bytes(n_req); }

__device__ __forceinline__ u64 warp_sum(u64 v) {
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}
__device__ __forceinline__ u32 ceil_div32(u32 a, u32 b) { return (a + b - 1) / b; }

// time of a decode iteration's fixed part, cached while the number of running sequences stays
struct DecodeCache {
    u32 n;              // running count the cache was built for (0 = empty)
    double s_fix, s_comm, t_head;
    u64 THa;            // n * H * a_b
};

template <int TIME_SUM>
__global__ void __launch_bounds__(SIM_THREADS)
k_trace_sim(DSpace s, DTrace tr, Range r, int tp_model, u64 max_iters_opt, guide_outputs o, u32 *counter,
            unsigned char *scratch, size_t per_warp, u32 gen_bytes, u32 first_bytes) {
    __shared__ u32 sh_slots[SIM_WARPS_PER_BLOCK][3][SLOTS];
    const u32 lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const u32 warp_global = blockIdx.x * SIM_WARPS_PER_BLOCK + wib;
    u32 *s_req = sh_slots[wib][0], *s_cache = sh_slots[wib][1], *s_rem = sh_slots[wib][2];
    unsigned char *mine = scratch + (size_t)warp_global * per_warp;
    u32 *gen = (u32 *)mine;
    double *first = (double *)(mine + gen_bytes);
    double *tpot = (double *)(mine + gen_bytes + first_bytes);
    const u32 n = tr.n;
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    const u32 lt_mask = (1u << lane) - 1;

    for (;;) {
        u64 j = 0;
        if (lane == 0) j = atomicAdd(counter, 1u);
        j = __shfl_sync(0xFFFFFFFFu, j, 0);
        if (j >= r.count) break;
        const Cfg c = decode_index(s, r.first + j);
        const DModel m = s.models[c.m];
        const DRate rt = s.rates[c.h * s.n_f + c.f];
        const u32 t = s.tp[c.t], b = s.batch[c.b];
        const uint2 pr = s.pairs[c.l];
        const u32 Lin = pr.x, Lout = pr.y, blk = rt.kv_block;
        const MemInfo mi = mem_info(m, t);
        const u32 tt = tp_model ? 1u : t;
        const double lf = log2_rule_factor(t, tp_model), Nd = (double)m.N;

        // ---- what fits (Sec. 3.2 Step 1) ----
        const u64 blocks_total = rt.usable > mi.w_gpu ? floor_div(rt.usable - mi.w_gpu, (u64)blk * mi.kv_tok) : 0;
        const u32 longest = max(tr.max_tokens, tr.any_zero ? Lin + Lout : 0u);
        const u64 worst = ceil_div32(longest, blk);
        u32 st = 0;
        if (rt.usable <= mi.w_gpu) st |= GUIDE_ST_WEIGHTS;
        if (worst > blocks_total) st |= GUIDE_ST_KV;
        if ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) st |= GUIDE_ST_HEADS;
        const u32 fit = clamp_u32(blocks_total / worst);

        double clock = 0.0, dec_time = 0.0;
        u64 dec_tok = 0, n_iters = 0, n_req_iters = 0, free_blocks = blocks_total, csum = 0;
        u32 next = 0, high_water = 0, nrun = 0, n_new = 0;
        const u64 max_iters = max_iters_opt ? max_iters_opt : 64 * (tr.sum_out + (u64)tr.n_zero * Lout) + 4 * (u64)n;
        DecodeCache dc;
        dc.n = 0;

        while (!st) {
            // ---- 1. admit in arrival order, no overtaking ----
            for (;;) {
                while (next < high_water && (gen[next] & GEN_DONE)) next++;
                if (next >= n || nrun >= b) break;
                if (!(__ldg(tr.arrival + next) <= clock)) break;
                const u32 g = next < high_water ? gen[next] : 0u;     // tokens kept from before an eviction
                u32 in = __ldg(tr.in_len + next), out = __ldg(tr.out_len + next);
                if (in == 0) { in = Lin; out = Lout; }
                const u32 q = in + g;                                  // prompt + tokens to recompute
                const u32 need = ceil_div32(q, blk);
                if (need > free_blocks) break;
                free_blocks -= need;
                if (lane == 0) {
                    s_req[nrun] = next;
                    s_cache[nrun] = q;
                    s_rem[nrun] = (out - g) | F_NEEDS_PREFILL | (g == 0 ? F_FIRST : 0u);
                }
                nrun++; n_new++; next++;
                if (next > high_water) high_water = next;
            }
            __syncwarp();
            // ---- 2. nothing to run: finished, or jump to the next arrival ----
            if (nrun == 0) {
                if (next >= n) break;
                const double a = __ldg(tr.arrival + next);
                if (a > clock) { clock = a; continue; }
                st |= GUIDE_ST_ITER;                                   // cannot happen when each request fits alone
                break;
            }
            if (n_iters >= max_iters) { st |= GUIDE_ST_ITER; break; }
            // ---- 3. build the iteration: prompts first, everything else stalls ----
            double t_iter;
            u32 participants;
            bool any_done = false;
            if (n_new > 0) {
                u64 T = 0, A = 0;
                for (u32 base = 0; base < nrun; base += 32) {
                    const u32 k = base + lane;
                    if (k < nrun && (s_rem[k] & F_NEEDS_PREFILL)) {
                        const u64 q = s_cache[k];
                        T += q; A += q * q;
                    }
                }
                T = warp_sum(T); A = warp_sum(A);
                TaskTab kt;
                build_fixed_tasks(m, tt, T, n_new, 1, kt);
                build_attn_tasks(m, tt, T, A, T, kt);
                t_iter = eval_phase<TIME_SUM>(kt, rt, Nd, lf);
                const double after = clock + t_iter;
                for (u32 base = 0; base < nrun; base += 32) {
                    const u32 k = base + lane;
                    if (k < nrun) {
                        const u32 rem = s_rem[k];
                        if (rem & F_NEEDS_PREFILL) {
                            if (rem & F_FIRST) first[s_req[k]] = after;    // first token of this request
                            const u32 left = (rem & REM_MASK) - 1;
                            s_rem[k] = left;
                            any_done |= left == 0;
                        }
                    }
                }
                csum += T;
                participants = n_new;
                n_new = 0;
            } else {
                // every sequence whose last block is full needs one more block
                u32 needed = 0;
                for (u32 base = 0; base < nrun; base += 32) {
                    const u32 k = base + lane;
                    needed += __popc(__ballot_sync(0xFFFFFFFFu, k < nrun && s_cache[k] % blk == 0));
                }
                if (needed > free_blocks) {
                    while (needed > free_blocks) {                     // evict the youngest, recompute later
                        const u32 v = nrun - 1;
                        const u32 cv = s_cache[v], rq = s_req[v], rem = s_rem[v] & REM_MASK;
                        free_blocks += ceil_div32(cv, blk);
                        if (cv % blk == 0) needed--;
                        csum -= cv;
                        u32 out = __ldg(tr.in_len + rq) ? __ldg(tr.out_len + rq) : Lout;
                        if (lane == 0) gen[rq] = out - rem;
                        nrun--;
                        next = rq;
                    }
                    __syncwarp();
                }
                free_blocks -= needed;
                const u64 ctx = csum + nrun;                           // cached tokens + the new one, summed
                if (dc.n != nrun) {
                    TaskTab kt;
                    build_fixed_tasks(m, tt, nrun, nrun, 1, kt);
                    dc.n = nrun;
                    dc.s_fix = eval_fixed<TIME_SUM>(kt, rt);
                    dc.s_comm = eval_comm(kt, rt);
                    dc.t_head = eval_head<TIME_SUM>(kt, rt);
                    dc.THa = (u64)nrun * m.H * m.ab;
                }
                {
                    const double inv_t = 1.0 / (double)tt;
                    const u64 X = rt.flash ? 0ull : (u64)m.nh * ctx * m.ab;
                    const double F9 = cvt(2 * (u64)m.H * ctx) * inv_t;
                    const double B9 = cvt(dc.THa + ctx * m.Dkv * m.kvb + X) * inv_t;
                    const double F10 = cvt(5 * (u64)m.nh * ctx) * inv_t;
                    const double B10 = cvt(2 * X) * inv_t;
                    const double ic = rt.inv_c[CLS_ATTN], im = rt.inv_m[CLS_ATTN];
                    const double t9 = task_time<TIME_SUM>(F9, B9, ic, im);
                    const double t10 = task_time<TIME_SUM>(F10, B10, ic, im);
                    const double s_att = (t9 + t10) + t9;
                    t_iter = combine_phase(dc.s_fix, s_att, dc.s_comm, dc.t_head, 1.0, Nd, rt.tovh, lf);
                }
                for (u32 base = 0; base < nrun; base += 32) {
                    const u32 k = base + lane;
                    if (k < nrun) {
                        s_cache[k] += 1;
                        const u32 left = s_rem[k] - 1;
                        s_rem[k] = left;
                        any_done |= left == 0;
                    }
                }
                csum += nrun;
                dec_time = dec_time + t_iter;
                dec_tok += nrun;
                participants = nrun;
            }
            // ---- 4. advance the clock ----
            clock = clock + t_iter;
            n_iters++;
            n_req_iters += participants;
            // ---- 5. retire finished sequences, keep the rest in order ----
            if (__any_sync(0xFFFFFFFFu, any_done)) {
                __syncwarp();
                u32 kept = 0;
                u64 freed = 0, gone = 0;
                const u32 n_before = nrun;
                for (u32 base = 0; base < n_before; base += 32) {
                    const u32 k = base + lane;
                    const bool valid = k < n_before;
                    u32 rq = 0, cv = 0, rem = 1;
                    if (valid) { rq = s_req[k]; cv = s_cache[k]; rem = s_rem[k]; }
                    const bool done = valid && rem == 0;
                    if (done) {
                        gen[rq] = GEN_DONE;
                        const u32 out = __ldg(tr.in_len + rq) ? __ldg(tr.out_len + rq) : Lout;
                        tpot[rq] = out > 1 ? (clock - first[rq]) / (double)(out - 1) : 0.0;
                        freed += ceil_div32(cv, blk);
                        gone += cv;
                    }
                    const bool keep = valid && !done;
                    const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);
                    __syncwarp();
                    if (keep) {
                        const u32 d = kept + __popc(ballot & lt_mask);
                        s_req[d] = rq; s_cache[d] = cv; s_rem[d] = rem;
                    }
                    kept += __popc(ballot);
                    __syncwarp();
                }
                free_blocks += warp_sum(freed);
                csum -= warp_sum(gone);
                nrun = kept;
            }
        }

        // ---- results ----
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
            }
            for (u32 i = lane; i < n; i += 32) {
                if (rq_ttft) __stcs(rq_ttft + i, inf);
                if (rq_tpot) __stcs(rq_tpot + i, inf);
            }
            continue;
        }
        // means in request order: 32 values at a time, added one after the other
        double s_ttft = 0.0, s_tpot = 0.0;
        for (u32 base = 0; base < n; base += 32) {
            const u32 i = base + lane;
            double vt = 0.0, vp = 0.0;
            if (i < n) {
                vt = first[i] - __ldg(tr.arrival + i);
                vp = tpot[i];
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
            const double cost_hr = rt.price * (double)t;
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
        }
        __syncwarp();
    }
}

int launch_trace_sim(const DSpace &s, const DTrace &t, Range r, int time_model, int tp_model, u64 max_iters,
                     const guide_outputs &o, void *ws, size_t, cudaStream_t st) {
    const size_t pw = per_warp_bytes(t.n);
    const u32 gen_bytes = (u32)(((size_t)t.n * 4 + 255) / 256 * 256);
    const u32 first_bytes = (u32)(((size_t)t.n * 8 + 255) / 256 * 256);
    // resident warps: as many as the SMs hold, never more than the workspace was sized for
    u32 blocks = (u32)num_sms() * 4;
    blocks = std::min<u32>(blocks, SIM_MAX_WARPS / SIM_WARPS_PER_BLOCK);
    blocks = (u32)std::min<u64>(blocks, (r.count + SIM_WARPS_PER_BLOCK - 1) / SIM_WARPS_PER_BLOCK);
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    unsigned char *scratch = (unsigned char *)ws + 256;
    if (time_model)
        k_trace_sim<1><<<blocks, SIM_THREADS, 0, st>>>(s, t, r, tp_model, max_iters, o, (u32 *)ws, scratch, pw, gen_bytes, first_bytes);
    else
        k_trace_sim<0><<<blocks, SIM_THREADS, 0, st>>>(s, t, r, tp_model, max_iters, o, (u32 *)ws, scratch, pw, gen_bytes, first_bytes);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

}  // namespace guide
