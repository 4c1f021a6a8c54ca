// Constraint filter + global top-k + 2-D Pareto front (selection of Sec. 3.2 / Sec. 4.1).
//
// Both reductions are streaming: a block walks its share of the configs, drops on the spot
// whatever its current partial result already beats (a threshold for top-k, the block's current
// front for Pareto) and appends the few survivors to a shared-memory buffer with one atomic and
// no barrier.  Every few rounds the block meets at a checkpoint and, if the buffer could overflow
// before the next one, sorts it and rebuilds the partial result.  Block results go to the
// workspace.  Top-k lists are merged by a second, fully parallel kernel that ranks every surviving
// candidate against all lists; Pareto fronts are folded by the block that finishes last.
// Every comparison is on the total order (value, config index), so the answer does not depend on
// how configs are spread over blocks or in which order they are appended.
//
// The metrics come either from materialised arrays or, fused, from the closed-form evaluation
// itself, walked in the tiled order of tiled.cuh so the integer task tables are built once per
// (model, batch, TP, length) point.
#include "select_sink.cuh"

namespace guide {

static constexpr u32 PARETO_CAP = 4096;          // shared-memory items per block
static constexpr u32 TOPK_CAP = 4096;            // shared-memory candidates per block
static constexpr u32 MAX_BUDGET = 16;            // most appends per thread between two checkpoints

// ---- where the metrics come from --------------------------------------------------------------

// materialised arrays written by guide_simulate
struct MatSource {
    static constexpr int ITEMS = 4;     // a thread fetches four consecutive configs per round
    static constexpr bool CONSEC = true;
    guide_outputs o;
    Cons c;
    int m0, m1;
    int vec;                            // every array in use is 16-byte aligned (status: 4-byte)
    __device__ __forceinline__ const double *metric_ptr(int key) const {
        switch (key) {
        case GUIDE_LATENCY: return o.latency;
        case GUIDE_TTFT: return o.ttft;
        case GUIDE_TTFT_P99: return o.ttft_p99;
        case GUIDE_TPOT: return o.tpot;
        case GUIDE_THROUGHPUT: return o.thr_decode;
        case GUIDE_COST_PER_HR: return o.cost_per_hr;
        default: return o.cost_per_token;
        }
    }
    static __device__ __forceinline__ void load4(const double *p, u64 j0, double v[4]) {
        const double2 lo = __ldg(reinterpret_cast<const double2 *>(p + j0));
        const double2 hi = __ldg(reinterpret_cast<const double2 *>(p + j0 + 2));
        v[0] = lo.x; v[1] = lo.y; v[2] = hi.x; v[3] = hi.y;
    }
    // Four consecutive configs j0..j0+3 (j0 a multiple of 4, all in range, vec set): one 4-byte
    // status load and two 16-byte loads per array in use.
    __device__ __forceinline__ void get4(u64 j0, bool ok[4], double a[4], double b[4]) const {
        const double inf = __longlong_as_double(0x7FF0000000000000LL);
        const u32 st = __ldg(reinterpret_cast<const u32 *>(o.status + j0));
        double v[4];
#pragma unroll
        for (int u = 0; u < 4; u++) ok[u] = ((st >> (8 * u)) & 0xFFu) == 0;
        if (c.max_ttft < inf) {
            const double *p = c.ttft_stat == GUIDE_STAT_MEAN ? o.ttft : c.ttft_stat == GUIDE_STAT_P50 ? o.ttft_p50 : o.ttft_p99;
            load4(p, j0, v);
#pragma unroll
            for (int u = 0; u < 4; u++) ok[u] &= v[u] <= c.max_ttft;
        }
        if (c.max_latency < inf) {
            load4(o.latency, j0, v);
#pragma unroll
            for (int u = 0; u < 4; u++) ok[u] &= v[u] <= c.max_latency;
        }
        if (c.max_cost_hr < inf) {
            load4(o.cost_per_hr, j0, v);
#pragma unroll
            for (int u = 0; u < 4; u++) ok[u] &= v[u] <= c.max_cost_hr;
        }
        if (c.min_thr > 0.0) {
            load4(o.thr_decode, j0, v);
#pragma unroll
            for (int u = 0; u < 4; u++) ok[u] &= v[u] >= c.min_thr;
        }
        load4(metric_ptr(m0), j0, a);
        if (m0 == GUIDE_THROUGHPUT) {
#pragma unroll
            for (int u = 0; u < 4; u++) a[u] = 0.0 - a[u];
        }
        if (m1 >= 0) {
            load4(metric_ptr(m1), j0, b);
            if (m1 == GUIDE_THROUGHPUT) {
#pragma unroll
                for (int u = 0; u < 4; u++) b[u] = 0.0 - b[u];
            }
        } else {
#pragma unroll
            for (int u = 0; u < 4; u++) b[u] = 0.0;
        }
    }
    __device__ __forceinline__ double metric(int key, u64 j) const {
        switch (key) {
        case GUIDE_LATENCY: return __ldg(o.latency + j);
        case GUIDE_TTFT: return __ldg(o.ttft + j);
        case GUIDE_TTFT_P99: return __ldg(o.ttft_p99 + j);
        case GUIDE_TPOT: return __ldg(o.tpot + j);
        case GUIDE_THROUGHPUT: return 0.0 - __ldg(o.thr_decode + j);
        case GUIDE_COST_PER_HR: return __ldg(o.cost_per_hr + j);
        default: return __ldg(o.cost_per_token + j);
        }
    }
    // No data-dependent early exit: every load of a config (and of the other configs a thread
    // fetches in the same round) can be in flight at once.  Branches are on launch constants only.
    __device__ __forceinline__ bool get(u64 j, u64, double &a, double &b) const {
        const double inf = __longlong_as_double(0x7FF0000000000000LL);
        bool ok = __ldg(o.status + j) == 0;
        if (c.max_ttft < inf) {
            const double *p = c.ttft_stat == GUIDE_STAT_MEAN ? o.ttft : c.ttft_stat == GUIDE_STAT_P50 ? o.ttft_p50 : o.ttft_p99;
            ok &= __ldg(p + j) <= c.max_ttft;
        }
        if (c.max_latency < inf) ok &= __ldg(o.latency + j) <= c.max_latency;
        if (c.max_cost_hr < inf) ok &= __ldg(o.cost_per_hr + j) <= c.max_cost_hr;
        if (c.min_thr > 0.0) ok &= __ldg(o.thr_decode + j) >= c.min_thr;
        a = metric(m0, j);
        b = m1 >= 0 ? metric(m1, j) : 0.0;
        return ok;
    }
};

// closed form evaluated on the fly: nothing is written to memory
template <int TIME_SUM>
struct FusedSource {
    static constexpr int ITEMS = 1;     // evaluation is register heavy: one config at a time
    static constexpr bool CONSEC = false;
    __device__ __forceinline__ void get4(u64, bool *, double *, double *) const {}
    static constexpr int vec = 0;
    DSpace s;
    Cons c;
    int m0, m1, tp_model;
    __device__ __forceinline__ bool get(u64, u64 idx, double &a, double &b) const {
        Metrics m;
        closed_form_eval<TIME_SUM>(s, decode_index(s, idx), tp_model, m);
        if (m.status) return false;
        if (!(m.ttft <= c.max_ttft) || !(m.latency <= c.max_latency) || !(m.cost_hr <= c.max_cost_hr) ||
            !(m.thr >= c.min_thr))
            return false;
        a = pick_metric(m0, m.latency, m.ttft, m.ttft, m.tpot, m.thr, m.cost_hr, m.cost_tok);
        b = m1 >= 0 ? pick_metric(m1, m.latency, m.ttft, m.ttft, m.tpot, m.thr, m.cost_hr, m.cost_tok) : 0.0;
        return true;
    }
};

// One round of a scan: ITEMS configs per thread.  Sources with CONSEC give a thread consecutive
// configs (vector loads when aligned and in range); otherwise thread t takes t, t + blockDim, ...
template <class Src>
__device__ __forceinline__ void fetch_round(const Src &src, const Range &r, u64 tile, bool ok[Src::ITEMS],
                                            double a[Src::ITEMS], double b[Src::ITEMS], u64 jj[Src::ITEMS]) {
    constexpr int ITEMS = Src::ITEMS;
    const u64 span = (u64)ITEMS * blockDim.x;
    if (Src::CONSEC) {
        const u64 j0 = tile * span + (u64)ITEMS * threadIdx.x;
#pragma unroll
        for (int u = 0; u < ITEMS; u++) jj[u] = j0 + u;
        if (src.vec && j0 + ITEMS <= r.count) { src.get4(j0, ok, a, b); return; }
    } else {
#pragma unroll
        for (int u = 0; u < ITEMS; u++) jj[u] = tile * span + (u64)u * blockDim.x + threadIdx.x;
    }
#pragma unroll
    for (int u = 0; u < ITEMS; u++) {
        const u64 jc = jj[u] < r.count ? jj[u] : r.count - 1;      // keep the loads in range
        a[u] = 0.0; b[u] = 0.0;
        ok[u] = src.get(jc, r.first + jc, a[u], b[u]) && jj[u] < r.count;
    }
}

// ---- top-k accumulator -------------------------------------------------------------------------------

struct TopKAcc {
    KI *buf;          // shared, TOPK_CAP entries
    u32 *cnt;         // shared append cursor
    u32 k;
    u32 c;            // buffered count at the last checkpoint, identical in every thread
    u32 budget;       // appends each thread may still make before the next checkpoint
    u32 ramp;         // checkpoint spacing: 1, 2, 4, ... MAX_BUDGET appends per thread
    bool has_thr;
    KI thr;

    __device__ void init(KI *b, u32 *cn, u32 k_) {
        buf = b; cnt = cn; k = k_; c = 0; has_thr = false; thr.key = KEY_MAX; thr.idx = KEY_MAX;
        budget = 1; ramp = 1;
        if (threadIdx.x == 0) *cnt = 0;
        __syncthreads();
    }
    // sort what is buffered, keep the k smallest, tighten the threshold
    __device__ void compact() {
        const u32 P = next_pow2(c);
        for (u32 i = c + threadIdx.x; i < P; i += blockDim.x) { buf[i].key = KEY_MAX; buf[i].idx = KEY_MAX; }
        __syncthreads();
        block_bitonic_sort(buf, P, ki_less);
        if (c >= k) { c = k; has_thr = true; thr = buf[k - 1]; }
        __syncthreads();                       // everyone has read the threshold
        if (threadIdx.x == 0) *cnt = c;
        __syncthreads();
    }
    // Collective.  Compacts when the buffer could overflow before the next checkpoint, and early
    // while that is cheap: as soon as k candidates exist (first threshold), then whenever about k
    // more have slipped under the stale threshold.  Checkpoints start one append apart, so the
    // first threshold comes from a small sort, and thin out to MAX_BUDGET appends apart.
    __device__ void checkpoint() {
        __syncthreads();
        c = *cnt;
        __syncthreads();                       // nobody appends before everyone has read the count
        if (ramp < MAX_BUDGET) ramp *= 2;
        const u32 early = has_thr ? 2 * k + blockDim.x : k;
        if (c >= early || c + ramp * blockDim.x > TOPK_CAP) compact();
        budget = min(ramp, (TOPK_CAP - c) / blockDim.x);
    }
    // Collective in the sense that every thread of the block calls it the same number of times; a
    // barrier happens only when the budget runs out.  The slot is always in range because the
    // checkpoint leaves room for budget * blockDim appends.
    __device__ __forceinline__ void push(bool ok, const KI &it) {
        if (ok && (!has_thr || ki_less(it, thr))) buf[atomicAdd(cnt, 1)] = it;
        if (--budget == 0) checkpoint();
    }
    __device__ void finish() {
        __syncthreads();
        c = *cnt;
        __syncthreads();
        compact();
    }
};

// ---- per-warp top-k accumulator (k <= TOPK_WARP_K) -------------------------------------------------
//
// No block barrier on the hot path.  Each warp owns a segment of shared memory with its own sorted
// candidates and its own threshold; takers of a round are placed by ballot, and when the segment
// fills (or about k entries have slipped under a stale threshold) the warp sorts it alone.  A warp
// that holds k candidates publishes its k-th key to a grid-wide word (kept as the complement, so a
// zeroed workspace header means "no bound"; atomicMax tightens it); every warp drops
// anything above that word at once, so once a few warps have found good candidates the rest of
// the grid hardly appends at all.  The word only bounds keys (strictly larger keys are dropped),
// ties on the key are still decided by the index in the exact per-warp test.

static constexpr u32 TOPK_WARP_K = 128;

__host__ __device__ inline u32 warp_seg_cap(u32 k) {
    u32 need = 2 * k + 64, p = 128;
    while (p < need) p <<= 1;
    return p;
}

struct WarpTopK {
    KI *seg;          // this warp's segment, cap entries
    u64 *gptr;        // grid-wide upper bound on the k-th key, stored as its complement (0 = no bound yet)
    u64 gthr;         // cached copy
    u32 cap, k, fill, tick;
    bool has_thr;
    KI thr;

    __device__ void init(KI *smem, u32 k_, u64 *gptr_) {
        k = k_; cap = warp_seg_cap(k_);
        seg = smem + (size_t)(threadIdx.x >> 5) * cap;
        gptr = gptr_; gthr = ~__ldcg(gptr_);
        fill = 0; tick = 0; has_thr = false; thr.key = KEY_MAX; thr.idx = KEY_MAX;
    }
    __device__ void compact() {
        const u32 lane = threadIdx.x & 31;
        const u32 P = next_pow2(fill);
        for (u32 i = fill + lane; i < P; i += 32) { seg[i].key = KEY_MAX; seg[i].idx = KEY_MAX; }
        __syncwarp();
        for (u32 size = 2; size <= P; size <<= 1) {
            for (u32 stride = size >> 1; stride > 0; stride >>= 1) {
                for (u32 i = lane; i < (P >> 1); i += 32) {
                    const u32 lo = ((i & ~(stride - 1)) << 1) | (i & (stride - 1));
                    const u32 hi = lo + stride;
                    const bool up = (lo & size) == 0;
                    const KI a = seg[lo], b = seg[hi];
                    if (ki_less(b, a) == up) { seg[lo] = b; seg[hi] = a; }
                }
                __syncwarp();
            }
        }
        if (fill >= k) {
            fill = k; has_thr = true; thr = seg[k - 1];
            if (lane == 0) atomicMax((unsigned long long *)gptr, (unsigned long long)~thr.key);
            if (thr.key < gthr) gthr = thr.key;
        }
        __syncwarp();
    }
    // largest key that can still matter to this warp
    __device__ __forceinline__ u64 bound() const { return has_thr && thr.key < gthr ? thr.key : gthr; }
    __device__ __forceinline__ void refresh() {
        if ((++tick & 15u) == 0) { const u64 g = ~__ldcg(gptr); if (g < gthr) gthr = g; }
    }
    // all 32 lanes of the warp call it together
    __device__ __forceinline__ void push(bool ok, const KI &it) {
        refresh();
        const bool take = ok && it.key <= gthr && (!has_thr || ki_less(it, thr));
        const u32 ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            if (take) seg[fill + __popc(ballot & ((1u << (threadIdx.x & 31)) - 1))] = it;
            fill += __popc(ballot);
            __syncwarp();
            const u32 early = has_thr ? 2 * k + 32 : k;
            if (fill + 32 > cap || fill >= early) compact();
        }
    }
};

// the block's warps pool their candidates, one sort, the k smallest go to the workspace
__device__ void warp_topk_store(WarpTopK &w, KI *smem, u32 block, u32 k, u32 *counts, KI *lists) {
    __shared__ u32 wfill[SEL_THREADS / 32];
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    if (w.fill > 0) w.compact();                   // sorted, at most k left
    KI mine[TOPK_WARP_K / 32];
#pragma unroll
    for (u32 q = 0; q < TOPK_WARP_K / 32; q++) {
        const u32 i = q * 32 + lane;
        if (i < w.fill) mine[q] = w.seg[i];
    }
    if (lane == 0) wfill[warp] = w.fill;
    __syncthreads();                               // every segment has been read into registers
    u32 off = 0, total = 0;
    for (u32 x = 0; x < n_warps; x++) {
        if (x < warp) off += wfill[x];
        total += wfill[x];
    }
#pragma unroll
    for (u32 q = 0; q < TOPK_WARP_K / 32; q++) {
        const u32 i = q * 32 + lane;
        if (i < w.fill) smem[off + i] = mine[q];
    }
    const u32 P = next_pow2(total);
    __syncthreads();
    for (u32 i = total + threadIdx.x; i < P; i += blockDim.x) { smem[i].key = KEY_MAX; smem[i].idx = KEY_MAX; }
    __syncthreads();
    block_bitonic_sort(smem, P, ki_less);
    const u32 c = min(total, k);
    KI *dst = lists + (size_t)block * k;
    for (u32 i = threadIdx.x; i < c; i += blockDim.x) dst[i] = smem[i];
    if (threadIdx.x == 0) counts[block] = c;
}

// ---- Pareto accumulator ----------------------------------------------------------------------------

struct ParetoAcc {
    P3 *buf;          // shared: [0, nf) current front sorted by x (y strictly falling), then appended survivors
    u32 *cnt;
    u32 *scratch;     // shared, 2 * 32 words
    u32 nf, c;
    u32 cap;          // entries of buf this accumulator may use
    u32 budget, ramp;
    u64 kx[4], ky[4];  // a few front points kept in registers: most configs are beaten by one of them
    bool overflow;
    bool lazy;        // folding fronts: incoming points are mostly keepers, merge only when the buffer fills

    __device__ void init(P3 *b, u32 *cn, u32 *sc, bool lazy_ = false, u32 cap_ = PARETO_CAP) {
        buf = b; cnt = cn; scratch = sc; nf = 0; c = 0; overflow = false; lazy = lazy_; cap = cap_;
        budget = lazy_ ? max(1u, (cap_ / 2) / blockDim.x) : 1; ramp = lazy_ ? min(budget, MAX_BUDGET) : 1;
#pragma unroll
        for (int i = 0; i < 4; i++) { kx[i] = KEY_MAX; ky[i] = KEY_MAX; }
        if (threadIdx.x == 0) *cnt = 0;
        __syncthreads();
    }
    // is `it` beaten by the current front?  Only the front point with the largest x <= it.x can do it.
    __device__ __forceinline__ bool beaten(const P3 &it) const {
        u32 lo = 0, hi = nf;                   // first front point with x > it.x
        while (lo < hi) {
            const u32 mid = (lo + hi) >> 1;
            if (buf[mid].x <= it.x) lo = mid + 1; else hi = mid;
        }
        if (lo == 0) return false;
        const P3 p = buf[lo - 1];
        if (p.y < it.y) return true;
        if (p.y > it.y) return false;
        return p.x < it.x || p.idx < it.idx;
    }
    // sort front + survivors by (x, y, idx); a point stays iff its y is below every earlier y
    __device__ void merge() {
        u64 *wmin = (u64 *)scratch;            // per-warp minima (32 x u64 = 64 words)
        const u32 P = next_pow2(c);
        for (u32 i = c + threadIdx.x; i < P; i += blockDim.x) { buf[i].x = KEY_MAX; buf[i].y = KEY_MAX; buf[i].idx = KEY_MAX; }
        __syncthreads();
        block_bitonic_sort(buf, P, p3_less);
        const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
        u64 carry = KEY_MAX;                   // smallest y seen in earlier rounds
        u32 out = 0;                           // points kept so far
        for (u32 base = 0; base < c; base += blockDim.x) {
            const u32 pos = base + threadIdx.x;
            const bool valid = pos < c;
            P3 it;
            if (valid) it = buf[pos]; else { it.x = KEY_MAX; it.y = KEY_MAX; it.idx = KEY_MAX; }
            // inclusive min-scan of y inside the warp
            u64 incl = it.y;
            for (u32 d = 1; d < 32; d <<= 1) {
                const u64 o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d && o < incl) incl = o;
            }
            u64 before = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
            if (lane == 0) before = KEY_MAX;
            if (lane == 31) wmin[warp] = incl;
            __syncthreads();
            u64 all = carry;
            for (u32 w = 0; w < n_warps; w++) {
                const u64 v = wmin[w];
                if (w < warp && v < before) before = v;
                if (v < all) all = v;
            }
            if (carry < before) before = carry;
            const bool keep = valid && it.y < before;
            const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);
            __syncthreads();                   // wmin has been read by everyone
            u32 *wcnt = scratch;               // reuse as per-warp keep counts
            if (lane == 0) wcnt[warp] = __popc(ballot);
            __syncthreads();
            u32 off = out, total = 0;
            for (u32 w = 0; w < n_warps; w++) {
                const u32 v = wcnt[w];
                if (w < warp) off += v;
                total += v;
            }
            // destinations never run ahead of this round's sources, which are all in registers
            if (keep) buf[off + __popc(ballot & ((1u << lane) - 1))] = it;
            out += total;
            carry = all;
            __syncthreads();
        }
        if (out > GUIDE_PARETO_MAX) { overflow = true; out = GUIDE_PARETO_MAX; }
        if (out + blockDim.x > cap) { overflow = true; out = cap - blockDim.x; }
        nf = out; c = out;
        if (threadIdx.x == 0) *cnt = out;
        __syncthreads();
        // refresh the register copies: four points spread over the front
#pragma unroll
        for (int i = 0; i < 4; i++) {
            if (nf > 0) { const P3 p = buf[(nf * (2 * i + 1)) / 8]; kx[i] = p.x; ky[i] = p.y; }
            else { kx[i] = KEY_MAX; ky[i] = KEY_MAX; }
        }
    }
    // strictly dominated by one of the register points (equal points are left to the exact test)
    __device__ __forceinline__ bool killed(const P3 &it) const {
        bool k = false;
#pragma unroll
        for (int i = 0; i < 4; i++) k |= (kx[i] <= it.x && ky[i] <= it.y) && (kx[i] < it.x || ky[i] < it.y);
        return k;
    }
    // Collective.  Merges when the buffer could overflow before the next checkpoint and, unless
    // lazy, as soon as there is anything while no front exists yet (until then nothing is
    // filtered) and whenever a block's worth of points has slipped past the stale front.
    __device__ void checkpoint() {
        __syncthreads();
        c = min(*cnt, cap);
        __syncthreads();
        if (ramp < MAX_BUDGET && 4 * ramp * blockDim.x <= cap) ramp *= 2;
        const bool early = !lazy && ((nf == 0 && c > 0) || c >= nf + blockDim.x);
        if (early || c + ramp * blockDim.x > cap) merge();
        // a front that leaves no room for one more round of appends cannot be handled in this buffer
        if (c + blockDim.x > cap) { overflow = true; nf = c = cap - blockDim.x; if (threadIdx.x == 0) *cnt = c; __syncthreads(); }
        budget = max(1u, min(ramp, (cap - c) / blockDim.x));
    }
    // every thread of the block calls it the same number of times; a barrier only when the budget runs out
    __device__ __forceinline__ void push(bool ok, const P3 &it) {
        if (ok && !killed(it) && !beaten(it)) {
            const u32 pos = atomicAdd(cnt, 1);
            if (pos < cap) buf[pos] = it;      // always true by the checkpoint rule; kept as a guard
        }
        if (--budget == 0) checkpoint();
    }
    __device__ void finish() {
        __syncthreads();
        c = min(*cnt, cap);
        __syncthreads();
        merge();
    }
};

// ---- per-warp Pareto accumulator ---------------------------------------------------------------
//
// The barrier-free counterpart of ParetoAcc for the common case of small fronts.  Each warp keeps
// its own front, sorted by x, in a small segment of shared memory; survivors of a round are placed
// behind it by ballot, and when a warp-load of them has gathered the warp sorts and sweeps its
// segment alone.  A front that outgrows the segment raises a flag and the caller's general
// (block-level) kernel redoes the work.

static constexpr u32 WSEG = 128;                 // entries per warp segment

struct WarpPareto {
    P3 *seg;
    u32 nf, fill;
    u64 kx[4], ky[4];
    bool overflow;

    __device__ void init(P3 *smem) {
        seg = smem + (size_t)(threadIdx.x >> 5) * WSEG;
        nf = 0; fill = 0; overflow = false;
#pragma unroll
        for (int i = 0; i < 4; i++) { kx[i] = KEY_MAX; ky[i] = KEY_MAX; }
    }
    __device__ __forceinline__ bool killed(const P3 &it) const {
        bool k = false;
#pragma unroll
        for (int i = 0; i < 4; i++) k |= (kx[i] <= it.x && ky[i] <= it.y) && (kx[i] < it.x || ky[i] < it.y);
        return k;
    }
    __device__ __forceinline__ bool beaten(const P3 &it) const {
        u32 lo = 0, hi = nf;                   // first front point with x > it.x
        while (lo < hi) {
            const u32 mid = (lo + hi) >> 1;
            if (seg[mid].x <= it.x) lo = mid + 1; else hi = mid;
        }
        if (lo == 0) return false;
        const P3 p = seg[lo - 1];
        if (p.y < it.y) return true;
        if (p.y > it.y) return false;
        return p.x < it.x || p.idx < it.idx;
    }
    // sort the segment by (x, y, idx); a point stays iff its y is below every earlier y
    __device__ void merge() {
        const u32 lane = threadIdx.x & 31;
        const u32 P = next_pow2(fill);
        for (u32 i = fill + lane; i < P; i += 32) { seg[i].x = KEY_MAX; seg[i].y = KEY_MAX; seg[i].idx = KEY_MAX; }
        __syncwarp();
        for (u32 size = 2; size <= P; size <<= 1) {
            for (u32 stride = size >> 1; stride > 0; stride >>= 1) {
                for (u32 i = lane; i < (P >> 1); i += 32) {
                    const u32 lo = ((i & ~(stride - 1)) << 1) | (i & (stride - 1));
                    const u32 hi = lo + stride;
                    const bool up = (lo & size) == 0;
                    const P3 a = seg[lo], b = seg[hi];
                    if (p3_less(b, a) == up) { seg[lo] = b; seg[hi] = a; }
                }
                __syncwarp();
            }
        }
        u64 carry = KEY_MAX;
        u32 out = 0;
        for (u32 base = 0; base < fill; base += 32) {
            const u32 pos = base + lane;
            const bool valid = pos < fill;
            P3 it;
            if (valid) it = seg[pos]; else { it.x = KEY_MAX; it.y = KEY_MAX; it.idx = KEY_MAX; }
            u64 incl = it.y;
            for (u32 d = 1; d < 32; d <<= 1) {
                const u64 o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d && o < incl) incl = o;
            }
            const u64 prev = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
            const u64 before = lane == 0 ? carry : (prev < carry ? prev : carry);   // smallest y before this point
            const bool keep = valid && it.y < before;
            const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);      // also orders this round's reads before its writes
            if (keep) seg[out + __popc(ballot & ((1u << lane) - 1))] = it;
            out += __popc(ballot);
            const u64 last = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (last < carry) carry = last;
            __syncwarp();
        }
        if (out + 32 > WSEG) { overflow = true; out = WSEG - 32; }     // no room for another round: flag it
        nf = out; fill = out;
#pragma unroll
        for (int i = 0; i < 4; i++) {
            if (nf > 0) { const P3 p = seg[(nf * (2 * i + 1)) / 8]; kx[i] = p.x; ky[i] = p.y; }
            else { kx[i] = KEY_MAX; ky[i] = KEY_MAX; }
        }
        __syncwarp();
    }
    // all 32 lanes of the warp call it together
    __device__ __forceinline__ void push(bool ok, const P3 &it) {
        const bool take = ok && !killed(it) && !beaten(it);
        const u32 ballot = __ballot_sync(0xFFFFFFFFu, take);
        if (ballot) {
            if (take) seg[fill + __popc(ballot & ((1u << (threadIdx.x & 31)) - 1))] = it;
            fill += __popc(ballot);
            __syncwarp();
            if (nf == 0 || fill >= nf + 32 || fill + 32 > WSEG) merge();
        }
    }
};

// ---- top-k kernels -----------------------------------------------------------------------------------

// a block's sorted candidates and their number go to the workspace
__device__ __forceinline__ void topk_store(TopKAcc &acc, u32 block, u32 k, u32 *counts, KI *lists) {
    acc.finish();
    KI *mine = lists + (size_t)block * k;
    for (u32 i = threadIdx.x; i < acc.c; i += blockDim.x) mine[i] = acc.buf[i];
    if (threadIdx.x == 0) counts[block] = acc.c;
}

// WARP: per-warp accumulators (no barrier while scanning); otherwise one accumulator per block.
template <bool WARP> struct TopKPick { typedef TopKAcc type; };
template <> struct TopKPick<true> { typedef WarpTopK type; };
// cheap necessary condition for an item to be taken (exact for neither: push decides)
__device__ __forceinline__ bool topk_maybe(const TopKAcc &, u64) { return true; }
__device__ __forceinline__ bool topk_maybe(const WarpTopK &acc, u64 key) { return key <= acc.bound(); }
// may a whole warp skip its pushes when no lane has a candidate?  Only the per-warp mode: the
// block accumulator counts pushes towards its checkpoints.
__device__ __forceinline__ bool topk_can_skip(const TopKAcc &) { return false; }
__device__ __forceinline__ bool topk_can_skip(WarpTopK &acc) { acc.refresh(); return true; }
__device__ __forceinline__ void topk_begin(TopKAcc &acc, KI *smem, u32 *cnt, u32 k, u64 *) { acc.init(smem, cnt, k); }
__device__ __forceinline__ void topk_begin(WarpTopK &acc, KI *smem, u32 *, u32 k, u64 *gthr) { acc.init(smem, k, gthr); }
__device__ __forceinline__ void topk_end(TopKAcc &acc, KI *, u32 block, u32 k, u32 *counts, KI *lists) {
    topk_store(acc, block, k, counts, lists);
}
__device__ __forceinline__ void topk_end(WarpTopK &acc, KI *smem, u32 block, u32 k, u32 *counts, KI *lists) {
    warp_topk_store(acc, smem, block, k, counts, lists);
}

template <class Src, bool WARP>
__global__ void __launch_bounds__(SEL_THREADS) k_topk_scan(Src src, Range r, u32 k, u32 *counts, KI *lists, u64 *gthr,
                                                           const u32 *gate) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 cnt;
    grid_dep_launch();
    grid_dep_wait();                            // a gated launch may have started before its predecessor finished
    if (gate && __ldcg(gate) == 0) return;
    typename TopKPick<WARP>::type acc;
    topk_begin(acc, (KI *)smem_raw, &cnt, k, gthr);
    constexpr int ITEMS = Src::ITEMS;
    const u64 span = (u64)ITEMS * blockDim.x;
    const u64 tiles = (r.count + span - 1) / span;
    for (u64 tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        bool ok[ITEMS];
        double a[ITEMS], b[ITEMS];
        u64 jj[ITEMS];
        KI it[ITEMS];
        fetch_round(src, r, tile, ok, a, b, jj);
        bool any = false;
#pragma unroll
        for (int u = 0; u < ITEMS; u++) {
            it[u].key = enc(a[u]); it[u].idx = r.first + jj[u];
            ok[u] = ok[u] && topk_maybe(acc, it[u].key);
            any |= ok[u];
        }
        // almost always nobody in the warp has a candidate: one vote instead of ITEMS pushes
        if (topk_can_skip(acc) && !__any_sync(0xFFFFFFFFu, any)) continue;
#pragma unroll
        for (int u = 0; u < ITEMS; u++) acc.push(ok[u], it[u]);
    }
    topk_end(acc, (KI *)smem_raw, blockIdx.x, k, counts, lists);
}

template <int TIME_SUM, bool WARP>
__global__ void __launch_bounds__(SEL_THREADS, 2)
k_topk_tiled(DSpace s, Range r, int tp_model, u32 hf_chunk, u32 tiles_per_mb, Cons c, int key, u32 k, u32 *counts, KI *lists,
             u64 *gthr, const u32 *gate) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 cnt;
    grid_dep_launch();
    grid_dep_wait();                            // a gated launch may have started before its predecessor finished
    if (gate && __ldcg(gate) == 0) return;
    typename TopKPick<WARP>::type acc;
    topk_begin(acc, (KI *)smem_raw, &cnt, k, gthr);
    tiled_visit<TIME_SUM>(s, r, tp_model, hf_chunk, tiles_per_mb, [&](bool valid, u64 j, const Metrics &m) {
        double a = 0.0, b;
        const bool ok = valid && fused_pick(m, c, key, -1, a, b);
        KI it;
        it.key = enc(a); it.idx = r.first + j;
        acc.push(ok, it);
    });
    topk_end(acc, (KI *)smem_raw, blockIdx.y * gridDim.x + blockIdx.x, k, counts, lists);
}

// Merge of the per-block lists.  One warp per candidate: its rank in the union is its position in
// its own list plus, for every other list, the number of entries smaller than it (binary search,
// the lanes sharing out the lists; entries are unique because config indices are).  Candidates
// above the smallest k-th entry of any full list cannot be among the k smallest and are skipped.
// Ranks below k are distinct, so every output slot has one writer.
__global__ void __launch_bounds__(SEL_THREADS) k_topk_merge(u32 nblk, u32 k, const u32 *counts, const KI *lists,
                                                            int negate_out, u64 *idx_out, double *key_out, u32 *count_out,
                                                            const u32 *gate) {
    __shared__ KI s_best[SEL_THREADS / 32];
    __shared__ u32 s_tot[SEL_THREADS / 32];
    grid_dep_wait();
    if (gate && __ldcg(gate) == 0) return;
    KI best; best.key = KEY_MAX; best.idx = KEY_MAX;
    u32 tot = 0;
    for (u32 b = threadIdx.x; b < nblk; b += blockDim.x) {
        const u32 cb = counts[b];
        tot += min(cb, k);          // saturating: only min(total, k) matters
        if (cb >= k) {
            const KI e = lists[(size_t)b * k + k - 1];
            if (ki_less(e, best)) best = e;
        }
    }
    for (int d = 16; d > 0; d >>= 1) {
        KI o;
        o.key = __shfl_xor_sync(0xFFFFFFFFu, best.key, d);
        o.idx = __shfl_xor_sync(0xFFFFFFFFu, best.idx, d);
        if (ki_less(o, best)) best = o;
        const u32 t2 = __shfl_xor_sync(0xFFFFFFFFu, tot, d);
        tot = min(tot + t2, k);
    }
    if ((threadIdx.x & 31) == 0) { s_best[threadIdx.x >> 5] = best; s_tot[threadIdx.x >> 5] = tot; }
    __syncthreads();
    best = s_best[0]; tot = s_tot[0];
    for (u32 w = 1; w < SEL_THREADS / 32; w++) {
        if (ki_less(s_best[w], best)) best = s_best[w];
        tot = min(tot + s_tot[w], k);
    }
    const u32 found = min(tot, k);
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) *count_out = found;
        for (u32 i = found + threadIdx.x; i < k; i += blockDim.x) {
            idx_out[i] = KEY_MAX;
            key_out[i] = __longlong_as_double(0x7FF0000000000000LL);
        }
    }
    // candidates, one warp each: the lanes split the lists
    const u32 lane = threadIdx.x & 31;
    const u64 n_warps = (u64)gridDim.x * (blockDim.x >> 5);
    const u64 n_cand = (u64)nblk * k;
    for (u64 g = (u64)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); g < n_cand; g += n_warps) {
        const u32 b = (u32)(g / k), p = (u32)(g % k);
        if (p >= counts[b]) continue;
        const KI me = lists[g];
        if (ki_less(best, me)) continue;
        u32 part = 0;
        for (u32 b2 = lane; b2 < nblk; b2 += 32) {
            if (b2 == b) continue;
            const u32 cb = counts[b2];
            if (cb == 0) continue;
            const KI *L = lists + (size_t)b2 * k;
            if (!ki_less(L[0], me)) continue;              // nothing smaller in that list
            u32 lo = 1, hi = cb;                           // number of entries smaller than me
            while (lo < hi) {
                const u32 mid = (lo + hi) >> 1;
                if (ki_less(L[mid], me)) lo = mid + 1; else hi = mid;
            }
            part += lo;
        }
        for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, d);
        const u32 rank = p + part;
        if (lane == 0 && rank < k) {
            const double v = dec(me.key);
            idx_out[rank] = me.idx;
            key_out[rank] = negate_out ? 0.0 - v : v;
        }
    }
}

// ---- Pareto kernels --------------------------------------------------------------------------------

// Store this block's front; the block that arrives last folds all fronts into the answer.  A prefix
// sum over the front sizes turns them into one flat list, so the number of collective steps
// depends on the number of points, not on the number of blocks.
__device__ void pareto_store_and_fold(ParetoAcc &acc, u32 block, u32 nblk, u32 *ticket, u32 *sizes, P3 *partial,
                                      u64 *idx_out, u32 out_cap, u32 *count_out, u32 *redo_flag = nullptr) {
    __shared__ u32 last_flag;
    __shared__ u32 pre[SEL_MAX_BLOCKS + 1];
    __shared__ u32 wsum[SEL_THREADS / 32];
    acc.finish();
    P3 *mine = partial + (size_t)block * GUIDE_PARETO_MAX;
    for (u32 i = threadIdx.x; i < acc.nf; i += blockDim.x) mine[i] = acc.buf[i];
    if (threadIdx.x == 0) sizes[block] = acc.nf | (acc.overflow ? 0x80000000u : 0u);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_flag = (atomicAdd(ticket, 1) == nblk - 1);
    __syncthreads();
    if (!last_flag) return;
    __threadfence();
    // exclusive prefix sum of the front sizes (up to SEL_MAX_BLOCKS of them) with any block size
    const u32 per = (SEL_MAX_BLOCKS + blockDim.x - 1) / blockDim.x;
    u32 local = 0;
    bool ovf = false;
    for (u32 u = 0; u < per; u++) {
        const u32 bi = threadIdx.x * per + u;
        const u32 sz = bi < nblk ? __ldcg(sizes + bi) : 0u;
        ovf |= (sz >> 31) != 0;
        local += sz & 0x7FFFFFFFu;
    }
    u32 incl = local;
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (u32 d = 1; d < 32; d <<= 1) {
        const u32 v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
    }
    if (lane == 31) wsum[warp] = incl;
    bool overflow = __syncthreads_or(ovf) != 0;
    u32 run = incl - local;
    for (u32 w2 = 0; w2 < warp; w2++) run += wsum[w2];
    for (u32 u = 0; u < per; u++) {
        const u32 bi = threadIdx.x * per + u;
        if (bi < SEL_MAX_BLOCKS) pre[bi] = run;
        run += bi < nblk ? (__ldcg(sizes + bi) & 0x7FFFFFFFu) : 0u;
    }
    if (threadIdx.x == blockDim.x - 1) pre[SEL_MAX_BLOCKS] = run;
    acc.init(acc.buf, acc.cnt, acc.scratch, true, acc.cap);   // includes a barrier: pre[] is complete
    const u32 total = pre[SEL_MAX_BLOCKS];
    for (u32 base = 0; base < total; base += blockDim.x) {
        const u32 i = base + threadIdx.x;
        P3 it; it.x = KEY_MAX; it.y = KEY_MAX; it.idx = KEY_MAX;
        if (i < total) {
            u32 lo = 0, hi = SEL_MAX_BLOCKS;            // last block index whose offset is <= i
            while (lo < hi) {
                const u32 mid = (lo + hi + 1) >> 1;
                if (pre[mid] <= i) lo = mid; else hi = mid - 1;
            }
            // written by other blocks: read through L2
            const u64 *w = reinterpret_cast<const u64 *>(partial + (size_t)lo * GUIDE_PARETO_MAX + (i - pre[lo]));
            it.x = __ldcg(w); it.y = __ldcg(w + 1); it.idx = __ldcg(w + 2);
        }
        acc.push(i < total, it);
    }
    acc.finish();
    overflow |= acc.overflow;
    for (u32 i = threadIdx.x; i < acc.nf && i < out_cap; i += blockDim.x) idx_out[i] = acc.buf[i].idx;
    if (threadIdx.x == 0) {
        *count_out = overflow ? 0xFFFFFFFFu : acc.nf;
        if (overflow && redo_flag) *redo_flag = 1;       // the general kernel, queued behind, redoes the work
    }
}

// Block end of the per-warp mode: the warps' fronts are pooled into one block accumulator (its
// buffer is the segments' own shared memory), which then goes the usual way.
__device__ void warp_pareto_pool(WarpPareto &w, ParetoAcc &acc, P3 *smem, u32 *cnt, u32 *scratch) {
    __shared__ u32 wfill[SEL_THREADS / 32];
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    if (w.fill > w.nf) w.merge();
    P3 mine[WSEG / 32];
#pragma unroll
    for (u32 q = 0; q < WSEG / 32; q++) {
        const u32 i = q * 32 + lane;
        if (i < w.nf) mine[q] = w.seg[i];
    }
    if (lane == 0) wfill[warp] = w.nf;
    const bool any_overflow = __syncthreads_or(w.overflow) != 0;     // also: every segment is in registers
    u32 off = 0, total = 0;
    for (u32 x = 0; x < n_warps; x++) {
        if (x < warp) off += wfill[x];
        total += wfill[x];
    }
#pragma unroll
    for (u32 q = 0; q < WSEG / 32; q++) {
        const u32 i = q * 32 + lane;
        if (i < w.nf) smem[off + i] = mine[q];
    }
    acc.init(smem, cnt, scratch, false, n_warps * WSEG);            // barrier inside: the pool is complete
    if (threadIdx.x == 0) *cnt = total;
    acc.overflow = any_overflow;
}

// Workspace header of a Pareto call: word 0 = ticket of the per-warp (fast) kernel, word 1 = redo
// flag it raises when a front outgrew a warp segment, word 2 = ticket of the general kernel.
// The general kernel with `gate` set does nothing unless the redo flag is up.

template <class Src, bool WARP>
__global__ void __launch_bounds__(SEL_THREADS) k_pareto_scan(Src src, Range r, u32 *header, const u32 *gate, u32 *sizes,
                                                             P3 *partial, u64 *idx_out, u32 out_cap, u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 cnt;
    __shared__ __align__(8) u32 scratch[64];
    grid_dep_wait();                            // a gated launch may have started before its predecessor finished
    if (gate && __ldcg(gate) == 0) return;
    ParetoAcc acc;
    WarpPareto wacc;
    if (WARP) wacc.init((P3 *)smem_raw); else acc.init((P3 *)smem_raw, &cnt, scratch);
    constexpr int ITEMS = Src::ITEMS;
    const u64 span = (u64)ITEMS * blockDim.x;
    const u64 tiles = (r.count + span - 1) / span;
    for (u64 tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        bool ok[ITEMS];
        double a[ITEMS], b[ITEMS];
        u64 jj[ITEMS];
        fetch_round(src, r, tile, ok, a, b, jj);
#pragma unroll
        for (int u = 0; u < ITEMS; u++) {
            P3 it;
            it.x = enc(a[u]); it.y = enc(b[u]); it.idx = r.first + jj[u];
            if (WARP) wacc.push(ok[u], it); else acc.push(ok[u], it);
        }
    }
    if (WARP) warp_pareto_pool(wacc, acc, (P3 *)smem_raw, &cnt, scratch);
    pareto_store_and_fold(acc, blockIdx.x, gridDim.x, header + (WARP ? 0 : 2), sizes, partial, idx_out, out_cap, count_out,
                          WARP ? header + 1 : nullptr);
}

template <int TIME_SUM, bool WARP>
__global__ void __launch_bounds__(SEL_THREADS, 2)
k_pareto_tiled(DSpace s, Range r, int tp_model, u32 hf_chunk, u32 tiles_per_mb, Cons c, int xm, int ym, u32 *header,
               const u32 *gate, u32 *sizes, P3 *partial, u64 *idx_out, u32 out_cap, u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 cnt;
    __shared__ __align__(8) u32 scratch[64];
    grid_dep_wait();                            // a gated launch may have started before its predecessor finished
    if (gate && __ldcg(gate) == 0) return;
    ParetoAcc acc;
    WarpPareto wacc;
    if (WARP) wacc.init((P3 *)smem_raw); else acc.init((P3 *)smem_raw, &cnt, scratch);
    tiled_visit<TIME_SUM>(s, r, tp_model, hf_chunk, tiles_per_mb, [&](bool valid, u64 j, const Metrics &m) {
        double a = 0.0, b = 0.0;
        const bool ok = valid && fused_pick(m, c, xm, ym, a, b);
        P3 it;
        it.x = enc(a); it.y = enc(b); it.idx = r.first + j;
        if (WARP) wacc.push(ok, it); else acc.push(ok, it);
    });
    if (WARP) warp_pareto_pool(wacc, acc, (P3 *)smem_raw, &cnt, scratch);
    pareto_store_and_fold(acc, blockIdx.y * gridDim.x + blockIdx.x, gridDim.x * gridDim.y, header + (WARP ? 0 : 2), sizes,
                          partial, idx_out, out_cap, count_out, WARP ? header + 1 : nullptr);
}

// ---- host side -----------------------------------------------------------------------------------------

// top-k workspace: 256 B header | counts u32[max_blocks] | lists KI[max_blocks][k]
static size_t topk_lists_offset(u32 max_blocks) { return 256 + ((size_t)max_blocks * 4 + 255) / 256 * 256; }

// ... followed by the streaming path's region (sample results and survivor list)
static size_t topk_stream_offset(u32 k) {
    return (topk_lists_offset(SEL_MAX_BLOCKS) + (size_t)SEL_MAX_BLOCKS * k * sizeof(KI) + 255) / 256 * 256;
}
static size_t pareto_stream_offset() {
    return (256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32) + (size_t)SEL_MAX_BLOCKS * GUIDE_PARETO_MAX * sizeof(P3) + 255) / 256 * 256;
}
size_t topk_workspace_bytes(u32 k) { return topk_stream_offset(k) + topk_stream_bytes(); }
size_t pareto_workspace_bytes() { return pareto_stream_offset() + pareto_stream_bytes(); }

static u32 grid_for(u64 count, u32 items, u32 blocks_per_sm, u32 max_blocks) {
    // every block has fixed costs (first sorts, final sort, its list in the merge): give each at
    // least eight rounds of tiles
    const u64 tiles = (count + (u64)SEL_THREADS * items - 1) / ((u64)SEL_THREADS * items);
    u64 g = std::min<u64>((u64)num_sms() * blocks_per_sm, max_blocks);
    g = std::min<u64>(g, std::max<u64>(tiles / 8, 1));
    return (u32)g;
}

// can the fused selection walk the space in tiled order (grid bounded by the workspace's block count)?
static bool fused_tiled(const DSpace &s, Range r, TileGeom *g) {
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    return r.count * 2 >= total && tiled_geometry(s, SEL_MAX_BLOCKS, SEL_MAX_BLOCKS, g);
}

template <class K>
static int allow_smem(K kernel, size_t bytes) {
    GUIDE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    return GUIDE_OK;
}

static int run_topk_merge(u32 nblk, u32 k, int negate, u32 *counts, KI *lists, u64 *idx_out, double *key_out,
                          u32 *count_out, const u32 *gate, cudaStream_t st) {
    const u64 cand = (u64)nblk * k;                      // one warp per candidate, a few candidates per warp
    const u64 want = (cand + (SEL_THREADS / 32) * 4 - 1) / ((SEL_THREADS / 32) * 4);
    const u32 grid = (u32)std::min<u64>(std::max<u64>(want, 1), (u64)num_sms() * 8);
    if (gate) {
        GUIDE_CUDA(launch_dependent(k_topk_merge, grid, SEL_THREADS, 0, st, nblk, k, (const u32 *)counts, (const KI *)lists, negate,
                                    idx_out, key_out, count_out, gate));
    } else {
        k_topk_merge<<<grid, SEL_THREADS, 0, st>>>(nblk, k, counts, lists, negate, idx_out, key_out, count_out, gate);
        GUIDE_CUDA(cudaGetLastError());
    }
    return GUIDE_OK;
}

// The first 256 bytes of a top-k workspace are its header (select.cuh); every word starts at zero.
static int topk_reset_header(unsigned char *ws, cudaStream_t st) {
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    return GUIDE_OK;
}

template <class Src, bool WARP>
static int run_topk_scan_mode(const Src &src, Range r, u32 k, int negate, u32 max_blocks, unsigned char *ws, u64 *idx_out,
                              double *key_out, u32 *count_out, const u32 *gate, cudaStream_t st) {
    u32 *counts = (u32 *)(ws + 256);
    KI *lists = (KI *)(ws + topk_lists_offset(max_blocks));
    const size_t smem = WARP ? (size_t)(SEL_THREADS / 32) * warp_seg_cap(k) * sizeof(KI) : (size_t)TOPK_CAP * sizeof(KI);
    int rc = allow_smem(k_topk_scan<Src, WARP>, smem);
    if (rc) return rc;
    // a gated launch runs behind the streaming path, which has reset the header for the whole call
    if (!gate && (rc = topk_reset_header(ws, st))) return rc;
    const u32 grid = grid_for(r.count, Src::ITEMS, gate ? 1 : (WARP ? 4 : 3), max_blocks);   // gated: rarely runs, keep the launch small
    if (gate) {
        GUIDE_CUDA(launch_dependent(k_topk_scan<Src, WARP>, grid, SEL_THREADS, smem, st, src, r, k, counts, lists, (u64 *)ws, gate));
    } else {
        k_topk_scan<Src, WARP><<<grid, SEL_THREADS, smem, st>>>(src, r, k, counts, lists, (u64 *)ws, gate);
        GUIDE_CUDA(cudaGetLastError());
    }
    return run_topk_merge(grid, k, negate, counts, lists, idx_out, key_out, count_out, gate, st);
}

template <class Src>
static int run_topk_scan(const Src &src, Range r, u32 k, int negate, u32 max_blocks, unsigned char *ws, u64 *idx_out,
                         double *key_out, u32 *count_out, cudaStream_t st, const u32 *gate = nullptr) {
    return k <= TOPK_WARP_K
               ? run_topk_scan_mode<Src, true>(src, r, k, negate, max_blocks, ws, idx_out, key_out, count_out, gate, st)
               : run_topk_scan_mode<Src, false>(src, r, k, negate, max_blocks, ws, idx_out, key_out, count_out, gate, st);
}

template <int TIME_SUM, bool WARP>
static int run_topk_tiled_mode(const DSpace &s, Range r, const TileGeom &g, int tp_model, const Cons &c, int key, u32 k,
                               unsigned char *ws, u64 *idx_out, double *key_out, u32 *count_out, const u32 *gate,
                               cudaStream_t st) {
    u32 *counts = (u32 *)(ws + 256);
    KI *lists = (KI *)(ws + topk_lists_offset(SEL_MAX_BLOCKS));
    const size_t smem = WARP ? (size_t)(SEL_THREADS / 32) * warp_seg_cap(k) * sizeof(KI) : (size_t)TOPK_CAP * sizeof(KI);
    int rc = allow_smem(k_topk_tiled<TIME_SUM, WARP>, smem);
    if (rc) return rc;
    // a gated launch runs behind the fused streaming path, which has reset the header for the whole call
    if (!gate && (rc = topk_reset_header(ws, st))) return rc;
    const dim3 grid(g.gx, g.splits);
    if (gate) {
        GUIDE_CUDA(launch_dependent(k_topk_tiled<TIME_SUM, WARP>, grid, g.threads, smem, st, s, r, tp_model, g.hf_chunk,
                                    g.tiles_per_mb, c, key, k, counts, lists, (u64 *)ws, gate));
    } else {
        k_topk_tiled<TIME_SUM, WARP><<<grid, g.threads, smem, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, c, key, k,
                                                                   counts, lists, (u64 *)ws, gate);
        GUIDE_CUDA(cudaGetLastError());
    }
    return run_topk_merge(g.gx * g.splits, k, key == GUIDE_THROUGHPUT, counts, lists, idx_out, key_out, count_out, gate, st);
}

template <int TIME_SUM>
static int run_topk_tiled(const DSpace &s, Range r, const TileGeom &g, int tp_model, const Cons &c, int key, u32 k,
                          unsigned char *ws, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st,
                          const u32 *gate = nullptr) {
    return k <= TOPK_WARP_K
               ? run_topk_tiled_mode<TIME_SUM, true>(s, r, g, tp_model, c, key, k, ws, idx_out, key_out, count_out, gate, st)
               : run_topk_tiled_mode<TIME_SUM, false>(s, r, g, tp_model, c, key, k, ws, idx_out, key_out, count_out, gate, st);
}

int launch_topk(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                const guide_constraints &c, int key, u32 k, u64 *idx_out, double *key_out, u32 *count_out,
                void *ws, unsigned *ticket, cudaStream_t st) {
    const int negate = key == GUIDE_THROUGHPUT;
    unsigned char *w = (unsigned char *)ws;
    if (mat) {
        MatSource src{*mat, make_cons(c), key, -1, mat_vec_ok(*mat)};
        if (k <= STREAM_TOPK_MAX_K && stream_eligible(*mat, r)) {
            // streaming path first; the accumulator kernels are queued behind it and return at once
            // unless it raised the redo flag
            int rc;
            u32 *header = (u32 *)w;                         // reset by the streaming path itself
            if ((rc = launch_topk_stream(r, *mat, c, key, k, header, w + topk_stream_offset(k), idx_out, key_out, count_out, st)))
                return rc;
            return run_topk_scan(src, r, k, negate, SEL_MAX_BLOCKS, w, idx_out, key_out, count_out, st, header + TK_REDO);
        }
        return run_topk_scan(src, r, k, negate, SEL_MAX_BLOCKS, w, idx_out, key_out, count_out, st);
    }
    TileGeom g;
    if (fused_tiled(s, r, &g)) {
        const u32 *gate = nullptr;
        if (!mat && ticket && k <= STREAM_TOPK_MAX_K && fused_stream_eligible(s, r)) {
            // fused streaming path first (sampled bound, model walk as the filter); the tiled kernels
            // are queued behind it and return at once unless it raised the redo flag
            int rc;
            u32 *header = (u32 *)w;                         // reset by the streaming path itself
            if ((rc = launch_topk_fused(s, time_model, tp_model, c, key, k, header, w + topk_stream_offset(k), ticket, idx_out,
                                        key_out, count_out, st)))
                return rc;
            gate = header + TK_REDO;
        }
        return time_model ? run_topk_tiled<1>(s, r, g, tp_model, make_cons(c), key, k, w, idx_out, key_out, count_out, st, gate)
                          : run_topk_tiled<0>(s, r, g, tp_model, make_cons(c), key, k, w, idx_out, key_out, count_out, st, gate);
    }
    if (time_model) {
        FusedSource<1> src{s, make_cons(c), key, -1, tp_model};
        return run_topk_scan(src, r, k, negate, SEL_MAX_BLOCKS, w, idx_out, key_out, count_out, st);
    }
    FusedSource<0> src{s, make_cons(c), key, -1, tp_model};
    return run_topk_scan(src, r, k, negate, SEL_MAX_BLOCKS, w, idx_out, key_out, count_out, st);
}

// Per-warp kernel first; the general kernel is queued right behind it and returns at once unless
// the first one raised the redo flag (a front too large for a warp segment).
template <class Src>
static int run_pareto_scan(const Src &src, Range r, u64 *idx_out, u32 cap, u32 *count_out, void *ws, cudaStream_t st) {
    const size_t smem_fast = (size_t)(SEL_THREADS / 32) * WSEG * sizeof(P3);
    const size_t smem_gen = (size_t)PARETO_CAP * sizeof(P3);
    int rc = allow_smem(k_pareto_scan<Src, false>, smem_gen);
    if (rc) return rc;
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    u32 *header = (u32 *)ws;
    u32 *sizes = (u32 *)((char *)ws + 256);
    P3 *partial = (P3 *)((char *)ws + 256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32));
    const u32 grid_fast = grid_for(r.count, Src::ITEMS, 4, SEL_MAX_BLOCKS);
    k_pareto_scan<Src, true><<<grid_fast, SEL_THREADS, smem_fast, st>>>(src, r, header, nullptr, sizes, partial, idx_out, cap,
                                                                         count_out);
    GUIDE_CUDA(cudaGetLastError());
    const u32 grid_gen = grid_for(r.count, Src::ITEMS, 2, SEL_MAX_BLOCKS);
    k_pareto_scan<Src, false><<<grid_gen, SEL_THREADS, smem_gen, st>>>(src, r, header, header + 1, sizes, partial, idx_out, cap,
                                                                        count_out);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

// The general kernel alone, gated on the redo flag a preceding kernel of the same call may have raised.
template <class Src>
static int run_pareto_general(const Src &src, Range r, u64 *idx_out, u32 cap, u32 *count_out, void *ws, cudaStream_t st) {
    const size_t smem_gen = (size_t)PARETO_CAP * sizeof(P3);
    int rc = allow_smem(k_pareto_scan<Src, false>, smem_gen);
    if (rc) return rc;
    u32 *header = (u32 *)ws;
    u32 *sizes = (u32 *)((char *)ws + 256);
    P3 *partial = (P3 *)((char *)ws + 256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32));
    const u32 grid_gen = grid_for(r.count, Src::ITEMS, 1, SEL_MAX_BLOCKS);      // rarely runs: keep the launch small
    GUIDE_CUDA(launch_dependent(k_pareto_scan<Src, false>, grid_gen, SEL_THREADS, smem_gen, st, src, r, header,
                                (const u32 *)(header + 1), sizes, partial, idx_out, cap, count_out));
    return GUIDE_OK;
}

template <int TIME_SUM>
static int run_pareto_tiled(const DSpace &s, Range r, const TileGeom &g, int tp_model, const Cons &c, int xm, int ym,
                            u64 *idx_out, u32 cap, u32 *count_out, void *ws, cudaStream_t st, bool general_only = false) {
    const size_t smem_fast = (size_t)(SEL_THREADS / 32) * WSEG * sizeof(P3);
    const size_t smem_gen = (size_t)PARETO_CAP * sizeof(P3);
    int rc = allow_smem(k_pareto_tiled<TIME_SUM, false>, smem_gen);
    if (rc) return rc;
    u32 *header = (u32 *)ws;
    u32 *sizes = (u32 *)((char *)ws + 256);
    P3 *partial = (P3 *)((char *)ws + 256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32));
    const dim3 grid(g.gx, g.splits);
    if (general_only) {
        // behind the fused streaming path, which has reset the header: the general kernel alone, gated on the redo flag
        GUIDE_CUDA(launch_dependent(k_pareto_tiled<TIME_SUM, false>, grid, g.threads, smem_gen, st, s, r, tp_model, g.hf_chunk,
                                    g.tiles_per_mb, c, xm, ym, header, (const u32 *)(header + 1), sizes, partial, idx_out, cap,
                                    count_out));
        return GUIDE_OK;
    }
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    k_pareto_tiled<TIME_SUM, true><<<grid, g.threads, smem_fast, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, c, xm, ym,
                                                                      header, nullptr, sizes, partial, idx_out, cap, count_out);
    GUIDE_CUDA(cudaGetLastError());
    k_pareto_tiled<TIME_SUM, false><<<grid, g.threads, smem_gen, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, c, xm, ym,
                                                                      header, header + 1, sizes, partial, idx_out, cap,
                                                                      count_out);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

int launch_pareto(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                  const guide_constraints &c, int xm, int ym, u64 *idx_out, u32 cap, u32 *count_out, void *ws,
                  unsigned *ticket, cudaStream_t st) {
    if (mat) {
        MatSource src{*mat, make_cons(c), xm, ym, mat_vec_ok(*mat)};
        if (stream_eligible(*mat, r)) {
            // streaming path, then the general kernel gated on the redo flag (header word 1)
            GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
            u32 *header = (u32 *)ws;
            int rc = launch_pareto_stream(r, *mat, c, xm, ym, header, (unsigned char *)ws + pareto_stream_offset(), idx_out, cap,
                                          count_out, st);
            if (rc) return rc;
            return run_pareto_general(src, r, idx_out, cap, count_out, ws, st);
        }
        return run_pareto_scan(src, r, idx_out, cap, count_out, ws, st);
    }
    TileGeom g;
    if (fused_tiled(s, r, &g)) {
        bool behind = false;
        if (!mat && ticket && fused_stream_eligible(s, r)) {
            GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
            int rc = launch_pareto_fused(s, time_model, tp_model, c, xm, ym, (u32 *)ws, (unsigned char *)ws + pareto_stream_offset(),
                                         ticket, idx_out, cap, count_out, st);
            if (rc) return rc;
            behind = true;
        }
        return time_model ? run_pareto_tiled<1>(s, r, g, tp_model, make_cons(c), xm, ym, idx_out, cap, count_out, ws, st, behind)
                          : run_pareto_tiled<0>(s, r, g, tp_model, make_cons(c), xm, ym, idx_out, cap, count_out, ws, st, behind);
    }
    if (time_model) {
        FusedSource<1> src{s, make_cons(c), xm, ym, tp_model};
        return run_pareto_scan(src, r, idx_out, cap, count_out, ws, st);
    }
    FusedSource<0> src{s, make_cons(c), xm, ym, tp_model};
    return run_pareto_scan(src, r, idx_out, cap, count_out, ws, st);
}

// ---- simulate and select in one call ---------------------------------------------------------------
//
// A whole closed-form space, its metrics written out, and a top-k and a Pareto selection over it.
// Where the space goes through the memory and line kernels, the selections cost no pass of their own:
// their bound and killers come from a sample of configs evaluated first (the fused selection's first
// half), the line kernel tests every config it evaluates against them while it stores the metrics, and
// the rank kernels finish on the two short survivor lists.  The answers are those of the separate
// calls (bound and killers only ever exclude configs that cannot be part of them); a survivor list
// that overflows raises the redo flag, and the tiled fused kernels queued behind redo that selection.
// Anything else runs the three calls one after the other on the stream.
int launch_simulate_select(const DSpace &s, Range r, const guide_outputs &o, int time_model, int tp_model,
                           const guide_constraints &ct, int key, u32 k, u64 *tk_idx, double *tk_key, u32 *tk_count, void *ws_t,
                           const guide_constraints &cp, int xm, int ym, u64 *pf_idx, u32 cap, u32 *pf_count, void *ws_p,
                           unsigned *ticket, cudaStream_t st, cudaEvent_t sweep_begin, cudaEvent_t sweep_end) {
    int rc;
    TileGeom g;
    if (!(ticket && k <= STREAM_TOPK_MAX_K && fused_tiled(s, r, &g) && fused_stream_eligible(s, r) && closed_form_by_lines(s, r, o))) {
        if (sweep_begin) GUIDE_CUDA(cudaEventRecord(sweep_begin, st));
        if ((rc = launch_closed_form(s, r, time_model, tp_model, o, ticket, st))) return rc;
        if (sweep_end) GUIDE_CUDA(cudaEventRecord(sweep_end, st));
        if ((rc = launch_topk(s, r, &o, time_model, tp_model, ct, key, k, tk_idx, tk_key, tk_count, ws_t, nullptr, st))) return rc;
        return launch_pareto(s, r, &o, time_model, tp_model, cp, xm, ym, pf_idx, cap, pf_count, ws_p, nullptr, st);
    }
    unsigned char *wt = (unsigned char *)ws_t, *wp = (unsigned char *)ws_p;
    u32 *ht = (u32 *)wt, *hp = (u32 *)wp;                   // the top-k header is reset by its bound kernel
    unsigned char *rt = wt + topk_stream_offset(k), *rp = wp + pareto_stream_offset();
    // the two samples side by side, then the two bound kernels
    GUIDE_CUDA(cudaMemsetAsync(wp, 0, 256, st));
    if ((rc = launch_topk_fused(s, time_model, tp_model, ct, key, k, ht, rt, ticket, tk_idx, tk_key, tk_count, st, FUSED_SAMPLE))) return rc;
    if ((rc = launch_pareto_fused(s, time_model, tp_model, cp, xm, ym, hp, rp, ticket, pf_idx, cap, pf_count, st, FUSED_SAMPLE_BESIDE)))
        return rc;
    if ((rc = launch_topk_fused(s, time_model, tp_model, ct, key, k, ht, rt, ticket, tk_idx, tk_key, tk_count, st, FUSED_BOUND_ONLY)))
        return rc;
    if ((rc = launch_pareto_fused(s, time_model, tp_model, cp, xm, ym, hp, rp, ticket, pf_idx, cap, pf_count, st, FUSED_BOUND_ONLY)))
        return rc;
    LineSelect sel;
    sel.ct = make_cons(ct); sel.key = key; sel.header_t = ht;
    sel.cp = make_cons(cp); sel.xm = xm; sel.ym = ym; sel.header_p = hp;
    fused_lists(rt, rp, &sel);
    if (sweep_begin) GUIDE_CUDA(cudaEventRecord(sweep_begin, st));
    if ((rc = launch_closed_form(s, r, time_model, tp_model, o, ticket, st, &sel))) return rc;
    if (sweep_end) GUIDE_CUDA(cudaEventRecord(sweep_end, st));
    // both rank kernels, then the gated fallbacks (they return at once unless a survivor list overflowed)
    if ((rc = launch_topk_fused(s, time_model, tp_model, ct, key, k, ht, rt, ticket, tk_idx, tk_key, tk_count, st, FUSED_RANK))) return rc;
    if ((rc = launch_pareto_fused(s, time_model, tp_model, cp, xm, ym, hp, rp, ticket, pf_idx, cap, pf_count, st, FUSED_RANK))) return rc;
    rc = time_model ? run_topk_tiled<1>(s, r, g, tp_model, sel.ct, key, k, wt, tk_idx, tk_key, tk_count, st, ht + TK_REDO)
                    : run_topk_tiled<0>(s, r, g, tp_model, sel.ct, key, k, wt, tk_idx, tk_key, tk_count, st, ht + TK_REDO);
    if (rc) return rc;
    return time_model ? run_pareto_tiled<1>(s, r, g, tp_model, sel.cp, xm, ym, pf_idx, cap, pf_count, wp, st, true)
                      : run_pareto_tiled<0>(s, r, g, tp_model, sel.cp, xm, ym, pf_idx, cap, pf_count, wp, st, true);
}

// ---- top-k over materialised metrics with library-owned scratch ----------------------------------
//
// Same kernels as launch_topk, but the per-block candidate lists live in a fixed device array that
// is part of the library image instead of a caller-supplied workspace, for callers that are not
// allowed to allocate device memory.  The array bounds k and the grid; every call reuses it.

static constexpr u32 NOALLOC_BLOCKS = 256;                     // grid cap of this variant
static constexpr size_t NOALLOC_SCRATCH_BYTES = 256 + (size_t)NOALLOC_BLOCKS * 4 + (size_t)NOALLOC_BLOCKS * GUIDE_NOALLOC_TOPK_MAX * sizeof(KI);

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

// Device address of the scratch array on the current device.  The array's name is only a handle
// on the host, so the address is asked for once per device and cached.
static int noalloc_scratch_address(unsigned char **out) {
    static std::mutex mu;
    static unsigned char *cached[64] = {};
    int dev = 0;
    GUIDE_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return fail(GUIDE_ERR_UNSUPPORTED, "device ordinal %d is outside 0..63", dev);
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void *p = nullptr;
        GUIDE_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) return fail(GUIDE_ERR_CUDA, "the scratch array has no device address");
        cached[dev] = (unsigned char *)p;
    }
    *out = cached[dev];
    return GUIDE_OK;
}

int launch_topk_noalloc(Range r, const guide_outputs &mat, const guide_constraints &c, int key, u32 k,
                        u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st) {
    unsigned char *scratch = nullptr;
    const int rc = noalloc_scratch_address(&scratch);
    if (rc) return rc;
    static_assert(256 + NOALLOC_BLOCKS * 4 == 1280, "list offset below assumes a 256-byte multiple");
    MatSource src{mat, make_cons(c), key, -1, mat_vec_ok(mat)};
    // The array still holds the previous call's bound, counts and lists.  The bound word is reset
    // on this stream before the scan; counts and lists need no clearing: every block of this
    // launch writes its own before the merge kernel, which follows on the same stream and reads
    // only this launch's blocks.
    return run_topk_scan(src, r, k, key == GUIDE_THROUGHPUT, NOALLOC_BLOCKS, scratch, idx_out, key_out, count_out, st);
}

}  // namespace guide
