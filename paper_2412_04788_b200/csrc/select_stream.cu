// Streaming selection over materialised metrics (constraint filter + top-k / Pareto front of
// Sec. 3.2 / Sec. 4.1 on arrays written by guide_simulate).
//
// A selection keeps a handful of configs out of millions, so the work is reading the arrays once at
// memory speed; what has to be avoided is every warp of the grid building its own partial answer
// before it can reject anything.  Three small steps do that:
//
//   sample : rows of 64 consecutive configs, one row out of every r at a hashed position, are read
//            by a small grid.  Top-k: every block reports the smallest passing (key, index) pair it
//            saw; the k-th smallest of those block minima is a pair that at least k passing configs
//            reach, hence an upper bound of the k-th pair of the whole range.  A second pass over the
//            same rows gathers the sample pairs within that bound and replaces it by their k-th
//            smallest, the exact k-th pair of the sample.  Pareto: every block reduces its sample to
//            its own front; the last block to finish merges those into one staircase of real points
//            ("killers"), sorted by x.
//   filter : one pass over everything.  A config survives if it passes the constraints and its
//            pair is within the bound (top-k), or no killer strictly dominates it (Pareto).
//            Survivors go to a list in the workspace through one atomic counter; there are few.
//   finish : every survivor is ranked against all others by one warp (the list staged in shared
//            memory): top-k writes the pairs of rank < k in place; Pareto keeps the survivors no
//            other survivor rules out and orders them by x.
//
// The bound and the killers only ever exclude configs that cannot be part of the answer, whatever
// the sample looked like, so the result is exact; a poor sample only means more survivors.  If they
// outgrow the list, the redo flag in the workspace header is raised and the accumulator-based
// kernels queued behind this path (select.cu) redo the call.
//
// Loads are laid out so that a warp reads 512 contiguous bytes of each array per instruction (a
// thread takes two consecutive configs, 16 bytes), two such rows per thread and round.
#include <algorithm>
#include <cmath>
#include <cstdlib>

#include <cooperative_groups.h>

#include "model_walk.cuh"
#include "select_sink.cuh"

namespace guide {

static constexpr u32 ROW = 64;                  // configs per warp-wide load (32 lanes x 2)
static constexpr u32 TILE = 1024;               // configs per block and round of the filter pass
static constexpr int MAX_ARR = 6;               // distinct arrays a call can touch

static constexpr u32 SAMPLE_BATCH = 4;          // rows a warp has in flight at once

static constexpr u32 TK_SAMPLE_BLOCKS = 256;    // block minima of the coarse bound (must stay >= 2 x STREAM_TOPK_MAX_K)
static constexpr u32 TK_SAMPLE_ROWS = 8192;     // rows the sample aims at
static constexpr u32 TK_SAMPLE_MAX_R = 32;
static constexpr u32 TK_SKEYS_CAP = 8192;       // sample pairs within the coarse bound the workspace holds
static constexpr u32 TK_SKEYS_SMEM = 2048;      // ... and how many the last block of the refinement sorts at once
static constexpr u32 TK_CAND_SMEM = 8192;       // ... of which the rank kernel stages this many in shared memory

static constexpr u32 PA_SAMPLE_BLOCKS = 128;
static constexpr u32 PA_ROWS_PER_WARP = 4;
static constexpr u32 PA_SAMPLE_ROWS = PA_SAMPLE_BLOCKS * (SEL_THREADS / 32) * PA_ROWS_PER_WARP;   // 4096
static constexpr u32 PA_LOCAL_CAP = 1024;       // per-block list of sample points that survive the two seeds
static constexpr u32 PA_PER_BLOCK = 2;          // front points a sample block hands on
static_assert(PA_KILLERS == PA_SAMPLE_BLOCKS * PA_PER_BLOCK, "every sample block hands on its share of the killers");

// one metric array with the role it plays in this call
struct Arr {
    const double *p;
    double bound;
    int cmp;          // 0: no bound, 1: value <= bound, 2: value >= bound
    int neg;          // used as a metric through its negation (throughput)
};
// arrays in use: entry 0 is the key (top-k) or x (Pareto), entry 1 is y (Pareto only)
template <int NA>
struct Src {
    Arr a[NA];
    const uint8_t *status;
    const u64 *row_base;   // null: entry j is config first + j.  Else the arrays hold sampled rows of 64 configs
                           // back to back and row_base[j / 64] is the index of the row's first config.
};

template <int NA>
__device__ __forceinline__ u64 cfg_index(const Src<NA> &s, u64 first, u64 j) {
    return s.row_base ? __ldg(s.row_base + (j >> 6)) + (j & 63) : first + j;
}

// region layout, top-k: pairs minima[TK_SAMPLE_BLOCKS] | pairs spairs[TK_SKEYS_CAP] | KI cand[TK_CAND_CAP]
static constexpr size_t TK_OFF_SKEYS = (size_t)TK_SAMPLE_BLOCKS * 16;
static constexpr size_t TK_OFF_CAND = TK_OFF_SKEYS + (size_t)TK_SKEYS_CAP * 16;
// ... | fused form only: u64 row_base[FUSED_ROWS] | u8 pass[FUSED_ROWS][64] | f64 a0[FUSED_ROWS][64] | f64 a1[FUSED_ROWS][64]
static constexpr u32 FUSED_ROWS = 8192;         // sample rows the compact scratch holds
static constexpr size_t FU_OFF_PASS = (size_t)FUSED_ROWS * 8;
static constexpr size_t FU_OFF_A0 = FU_OFF_PASS + (size_t)FUSED_ROWS * 64;
static constexpr size_t FU_OFF_A1 = FU_OFF_A0 + (size_t)FUSED_ROWS * 64 * 8;
static constexpr size_t FU_BYTES = FU_OFF_A1 + (size_t)FUSED_ROWS * 64 * 8;
static constexpr size_t TK_OFF_FUSED = (TK_OFF_CAND + (size_t)TK_CAND_CAP * sizeof(KI) + 255) / 256 * 256;
size_t topk_stream_bytes() { return TK_OFF_FUSED + FU_BYTES; }
// region layout, Pareto: P2 local[PA_KILLERS] | P2 killers[PA_KILLERS] | u32 local_n[PA_SAMPLE_BLOCKS] (padded to 256 B)
//                        | P3 surv[PA_SURV_CAP] | KI front[PA_SURV_CAP]
static constexpr size_t PA_OFF_KILLERS = (size_t)PA_KILLERS * sizeof(P2);
static constexpr size_t PA_OFF_LOCAL_N = 2 * PA_OFF_KILLERS;
static constexpr size_t PA_OFF_SURV = PA_OFF_LOCAL_N + 512;
static constexpr size_t PA_OFF_FRONT = PA_OFF_SURV + (size_t)PA_SURV_CAP * sizeof(P3);
static_assert(PA_SAMPLE_BLOCKS * 4 <= 512, "local_n fits its slot");
static constexpr size_t PA_OFF_FUSED = (PA_OFF_FRONT + (size_t)PA_SURV_CAP * sizeof(KI) + 255) / 256 * 256;
size_t pareto_stream_bytes() { return PA_OFF_FUSED + FU_BYTES; }

bool stream_eligible(const guide_outputs &mat, Range r) { return r.count >= STREAM_MIN_COUNT && mat_vec_ok(mat) != 0; }

// ---- loads and the constraint filter ----------------------------------------------------------------

// two consecutive configs j, j+1 (j even): status bytes and one 16-byte load per array
template <int NA>
__device__ __forceinline__ void load_pair(const Src<NA> &s, u64 j, u32 &st, double2 (&v)[NA]) {
    st = __ldcs(reinterpret_cast<const unsigned short *>(s.status + j));
#pragma unroll
    for (int a = 0; a < NA; a++) v[a] = __ldcs(reinterpret_cast<const double2 *>(s.a[a].p + j));
}

__device__ __forceinline__ bool within(const Arr &a, double v) {
    // no bound, value <= bound, or value >= bound; written so that a NaN fails an active bound
    return a.cmp == 0 || (a.cmp == 1 ? v <= a.bound : v >= a.bound);
}

// The two pairs of a thread in a filter tile (a warp: 64 consecutive configs at j0, 64 at j1).  The
// status bytes come first; the metric values of a 64-config group are loaded only when some config of
// the group passed its memory check, which most groups of a large sweep do not: whole runs of the
// length axis do not fit, and their 512 bytes per array are never read.  Returns false when both
// groups are dead.
template <int NA>
__device__ __forceinline__ bool load_live_pairs(const Src<NA> &s, u64 j0, u64 j1, u32 &st0, u32 &st1, double2 (&v0)[NA],
                                                double2 (&v1)[NA]) {
    st0 = __ldcs(reinterpret_cast<const unsigned short *>(s.status + j0));
    st1 = __ldcs(reinterpret_cast<const unsigned short *>(s.status + j1));
    const bool g0 = __any_sync(0xFFFFFFFFu, (st0 & 0xFFu) == 0 || (st0 >> 8) == 0);
    const bool g1 = __any_sync(0xFFFFFFFFu, (st1 & 0xFFu) == 0 || (st1 >> 8) == 0);
    if (!g0 && !g1) return false;
#pragma unroll
    for (int a = 0; a < NA; a++) {
        v0[a] = g0 ? __ldcs(reinterpret_cast<const double2 *>(s.a[a].p + j0)) : make_double2(0.0, 0.0);
        v1[a] = g1 ? __ldcs(reinterpret_cast<const double2 *>(s.a[a].p + j1)) : make_double2(0.0, 0.0);
    }
    return true;
}

template <int NA>
__device__ __forceinline__ void eval_pair(const Src<NA> &s, u32 st, const double2 (&v)[NA], bool &ok0, bool &ok1) {
    ok0 = (st & 0xFFu) == 0;
    ok1 = (st >> 8) == 0;
#pragma unroll
    for (int a = 0; a < NA; a++) {
        ok0 &= within(s.a[a], v[a].x);
        ok1 &= within(s.a[a], v[a].y);
    }
}

__device__ __forceinline__ u64 metric_key(const Arr &a, double v) { return enc(a.neg ? 0.0 - v : v); }

// one config through scalar loads (ragged tail of the range)
template <int NA>
__device__ __forceinline__ bool eval_one(const Src<NA> &s, u64 j, u64 &k0, u64 &k1) {
    bool ok = s.status[j] == 0;
    double v[NA];
#pragma unroll
    for (int a = 0; a < NA; a++) { v[a] = s.a[a].p[j]; ok &= within(s.a[a], v[a]); }
    k0 = metric_key(s.a[0], v[0]);
    k1 = NA > 1 ? metric_key(s.a[NA > 1 ? 1 : 0], v[NA > 1 ? 1 : 0]) : 0;
    return ok;
}

// The sample: the range is cut into groups of r consecutive rows and one row per group is read, at
// a hashed offset so that the sample does not lock onto a period of the config index (an axis whose
// length divides r).  Warps do not walk the groups in index order either: slot c of the walk is
// group (c x mul) mod n_groups, a bijection (mul is a prime that does not divide n_groups), so the
// rows one block sees are spread over the whole range instead of sharing a model or a hardware profile.
struct Sample {
    u64 n_groups;   // groups in the range
    u64 n_slots;    // slots walked (<= n_groups)
    u64 mul;
    u32 r;
    __device__ __forceinline__ u64 row(u64 slot) const {
        const u64 g = (slot * mul) % n_groups;
        const u32 h = (u32)(g * 2654435761ull) >> 7;
        return g * r + h % r;
    }
};

// SAMPLE_BATCH rows of a warp's walk at once: slots c0, c0 + stride, ...; j[u] is the first config of
// this lane's pair in row u.  Loads past the end of the walk are redirected to the last slot and
// marked j[u] = all-ones, so that every load can be issued before any is used.
template <int NA>
__device__ __forceinline__ void load_batch(const Src<NA> &s, const Sample &sm, u64 c0, u64 stride, u32 lane,
                                           u32 (&st)[SAMPLE_BATCH], double2 (&v)[SAMPLE_BATCH][NA], u64 (&j)[SAMPLE_BATCH]) {
#pragma unroll
    for (u32 u = 0; u < SAMPLE_BATCH; u++) {
        const u64 c = c0 + u * stride;
        const bool live = c < sm.n_slots;
        const u64 jj = sm.row(live ? c : sm.n_slots - 1) * ROW + 2 * lane;
        load_pair(s, jj, st[u], v[u]);
        j[u] = live ? jj : KEY_MAX;
    }
}

// ---- top-k ---------------------------------------------------------------------------------------
//
__device__ __forceinline__ void pair_min(u64 &key, u64 &idx, u64 okey, u64 oidx) {
    if (okey < key || (okey == key && oidx < idx)) { key = okey; idx = oidx; }
}

// k-th smallest (k >= 1) of the n <= blockDim.x * PER pairs in shared memory, by counting: entry i
// has rank #{entries before it in the total order}; indices are distinct, so ranks are.  The thread
// that finds rank k-1 writes the bound.  All-ones pairs are padding and sort last.
template <u32 PER>
__device__ __forceinline__ void write_kth_pair(const ulonglong2 *sl, u32 n, u32 k, u32 *header) {
#pragma unroll
    for (u32 u = 0; u < PER; u++) {
        const u32 i = threadIdx.x + u * blockDim.x;
        if (i >= n) continue;
        const ulonglong2 me = sl[i];
        u32 ahead = 0;
        for (u32 q = 0; q < n; q++) {
            const ulonglong2 o = sl[q];
            ahead += (o.x < me.x || (o.x == me.x && (o.y < me.y || (o.y == me.y && q < i)))) ? 1u : 0u;
        }
        if (ahead == k - 1) {
            u64 *b = reinterpret_cast<u64 *>(header + TK_BOUND);
            b[0] = me.x; b[1] = me.y;
        }
    }
}

// Coarse bound: every block's smallest passing sample pair, then (last block) the k-th smallest of
// those.  At least k passing configs, one per block, are within it.  All-ones (nothing excluded)
// when fewer than k blocks saw a passing config.
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS) k_topk_sample(Src<NA> s, Sample sm, u64 first, u32 k, u32 *header,
                                                             ulonglong2 *minima) {
    __shared__ ulonglong2 sl[TK_SAMPLE_BLOCKS];
    __shared__ u32 last;
    static_assert(TK_SAMPLE_BLOCKS == SEL_THREADS, "one block minimum per thread in the last block");
    grid_dep_launch();
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = SEL_THREADS / 32;
    u64 bk = KEY_MAX, bi = KEY_MAX;
    const u64 stride = (u64)gridDim.x * n_warps;
    for (u64 c0 = (u64)warp * gridDim.x + blockIdx.x; c0 < sm.n_slots; c0 += SAMPLE_BATCH * stride) {
        u32 st[SAMPLE_BATCH];
        double2 v[SAMPLE_BATCH][NA];
        u64 j[SAMPLE_BATCH];
        load_batch(s, sm, c0, stride, lane, st, v, j);
#pragma unroll
        for (u32 u = 0; u < SAMPLE_BATCH; u++) {
            bool ok0, ok1;
            eval_pair(s, st[u], v[u], ok0, ok1);
            if (j[u] != KEY_MAX && ok0) pair_min(bk, bi, metric_key(s.a[0], v[u][0].x), cfg_index(s, first, j[u]));
            if (j[u] != KEY_MAX && ok1) pair_min(bk, bi, metric_key(s.a[0], v[u][0].y), cfg_index(s, first, j[u]) + 1);
        }
    }
    for (int d = 16; d > 0; d >>= 1)
        pair_min(bk, bi, __shfl_xor_sync(0xFFFFFFFFu, bk, d), __shfl_xor_sync(0xFFFFFFFFu, bi, d));
    if (lane == 0) { sl[warp].x = bk; sl[warp].y = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (u32 w = 1; w < n_warps; w++) pair_min(bk, bi, sl[w].x, sl[w].y);
        ulonglong2 m; m.x = bk; m.y = bi;
        minima[blockIdx.x] = m;
        __threadfence();
        last = atomicAdd(header + TK_TICKET, 1) == gridDim.x - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    {
        ulonglong2 m; m.x = KEY_MAX; m.y = KEY_MAX;
        if (threadIdx.x < gridDim.x) m = __ldcg(minima + threadIdx.x);
        sl[threadIdx.x] = m;
    }
    __syncthreads();
    // padding entries are equal pairs; write_kth_pair orders them by position, so rank k-1 exists
    write_kth_pair<1>(sl, TK_SAMPLE_BLOCKS, k, header);
}

// Refinement: the sample's pairs within the coarse bound are gathered (few: the coarse bound is at
// worst the k-th best row of the sample) and the last block replaces the bound by their k-th
// smallest, the exact k-th pair of the sample (of the stored part of it, if they do not all fit).
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS) k_topk_refine(Src<NA> s, Sample sm, u64 first, u32 k, u32 *header,
                                                             ulonglong2 *spairs) {
    constexpr u32 PER = TK_SKEYS_SMEM / SEL_THREADS;
    __shared__ ulonglong2 sl[TK_SKEYS_SMEM];
    __shared__ u32 s_n;
    __shared__ u32 last;
    grid_dep_launch();
    grid_dep_wait();
    const u64 *bp = reinterpret_cast<const u64 *>(header + TK_BOUND);
    const u64 bkey = __ldcg(bp), bidx = __ldcg(bp + 1);
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = SEL_THREADS / 32;
    const u64 stride = (u64)gridDim.x * n_warps;
    for (u64 c0 = (u64)warp * gridDim.x + blockIdx.x; c0 < sm.n_slots; c0 += SAMPLE_BATCH * stride) {
        u32 st[SAMPLE_BATCH];
        double2 v[SAMPLE_BATCH][NA];
        u64 j[SAMPLE_BATCH];
        load_batch(s, sm, c0, stride, lane, st, v, j);
#pragma unroll
        for (u32 u = 0; u < SAMPLE_BATCH; u++) {
            bool ok[2];
            eval_pair(s, st[u], v[u], ok[0], ok[1]);
            const u64 key[2] = {metric_key(s.a[0], v[u][0].x), metric_key(s.a[0], v[u][0].y)};
#pragma unroll
            for (u32 h = 0; h < 2; h++) {
                if (j[u] != KEY_MAX && ok[h] && pair_le(key[h], cfg_index(s, first, j[u]) + h, bkey, bidx)) {
                    const u32 p = atomicAdd(header + TK_SAMPLED, 1);
                    if (p < TK_SKEYS_CAP) { ulonglong2 e; e.x = key[h]; e.y = cfg_index(s, first, j[u]) + h; spairs[p] = e; }
                }
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(header + TK_TICKET2, 1) == gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    // More pairs than the workspace holds: the ones that were stored are still real configs within
    // the coarse bound, so their k-th smallest is a valid (if looser) bound.  Fewer than k happens
    // only when the coarse bound is all-ones: it stays.
    const u32 n = min(__ldcg(header + TK_SAMPLED), TK_SKEYS_CAP);
    if (n < k) return;
    auto pair_before = [](const ulonglong2 &a, const ulonglong2 &b) { return a.x < b.x || (a.x == b.x && a.y < b.y); };
    u64 *bound = reinterpret_cast<u64 *>(header + TK_BOUND);
    if (n <= 2 * SEL_THREADS) {                      // a short list: counting is quicker than sorting
#pragma unroll
        for (u32 u = 0; u < 2; u++) {
            const u32 i = threadIdx.x + u * blockDim.x;
            if (i < n) sl[i] = __ldcg(spairs + i);
        }
        __syncthreads();
        write_kth_pair<2>(sl, n, k, header);
        return;
    }
    // Longer lists are sorted in shared memory, at most TK_SKEYS_SMEM pairs at a time.  A list above
    // that goes in two steps: every step-th pair first, whose k-th smallest bounds the k-th of the
    // whole list from above; then all pairs within that bound (about k x step of them).
    const u32 step = (n + TK_SKEYS_SMEM - 1) / TK_SKEYS_SMEM;
    const u32 m = (n + step - 1) / step;
    u32 P = next_pow2(m);
#pragma unroll
    for (u32 u = 0; u < PER; u++) {
        const u32 i = threadIdx.x + u * blockDim.x;
        ulonglong2 e; e.x = KEY_MAX; e.y = KEY_MAX;
        if (i < m) e = __ldcg(spairs + (size_t)i * step);
        if (i < P) sl[i] = e;
    }
    __syncthreads();
    block_bitonic_sort(sl, P, pair_before);
    const ulonglong2 b1 = sl[k - 1];                 // m >= k: n > 512 >= 2k and step <= 4
    __syncthreads();
    if (step == 1) {
        if (threadIdx.x == 0) { bound[0] = b1.x; bound[1] = b1.y; }
        return;
    }
    if (threadIdx.x == 0) s_n = 0;
    __syncthreads();
    for (u32 i = threadIdx.x; i < n; i += blockDim.x) {
        const ulonglong2 e = __ldcg(spairs + i);
        if (!pair_before(b1, e)) {                   // e <= b1
            const u32 pos = atomicAdd(&s_n, 1u);
            if (pos < TK_SKEYS_SMEM) sl[pos] = e;
        }
    }
    __syncthreads();
    const u32 c = s_n;                               // >= k: the k pairs that put b1 at rank k-1 of its subset are among them
    if (c > TK_SKEYS_SMEM) {                         // does not fit (heavy ties): the first bound stands
        if (threadIdx.x == 0) { bound[0] = b1.x; bound[1] = b1.y; }
        return;
    }
    P = next_pow2(c);
    for (u32 i = c + threadIdx.x; i < P; i += blockDim.x) { sl[i].x = KEY_MAX; sl[i].y = KEY_MAX; }
    __syncthreads();
    block_bitonic_sort(sl, P, pair_before);
    if (threadIdx.x == 0) { bound[0] = sl[k - 1].x; bound[1] = sl[k - 1].y; }
}

// The two kernels above as one cooperative launch: the same steps, with grid-wide barriers in place
// of the kernel boundary and of the "last block" selections, which here are spread over the whole
// grid (one warp ranks one pair).  A dependent chain of short latencies, so every hand-over it
// saves counts.  Used when the device supports cooperative launches.
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS) k_topk_bound(Src<NA> s, Sample sm, u64 first, u32 k, u32 *header,
                                                            ulonglong2 *minima, ulonglong2 *spairs) {
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    __shared__ ulonglong2 sl[SEL_THREADS / 32];
    // the call's header is reset here rather than by a memset in front: nothing reads it before the
    // first grid barrier, and the kernels queued behind wait for this grid to complete
    if (blockIdx.x == 0 && threadIdx.x < 64) header[threadIdx.x] = 0;
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = SEL_THREADS / 32;
    const u32 gwarp = blockIdx.x * n_warps + warp, total_warps = gridDim.x * n_warps;
    const u64 stride = (u64)gridDim.x * n_warps;
    u64 *bound = reinterpret_cast<u64 *>(header + TK_BOUND);
    // 1: block minima of the passing sample pairs
    u64 bk = KEY_MAX, bi = KEY_MAX;
    for (u64 c0 = (u64)warp * gridDim.x + blockIdx.x; c0 < sm.n_slots; c0 += SAMPLE_BATCH * stride) {
        u32 st[SAMPLE_BATCH];
        double2 v[SAMPLE_BATCH][NA];
        u64 j[SAMPLE_BATCH];
        load_batch(s, sm, c0, stride, lane, st, v, j);
#pragma unroll
        for (u32 u = 0; u < SAMPLE_BATCH; u++) {
            bool ok0, ok1;
            eval_pair(s, st[u], v[u], ok0, ok1);
            if (j[u] != KEY_MAX && ok0) pair_min(bk, bi, metric_key(s.a[0], v[u][0].x), cfg_index(s, first, j[u]));
            if (j[u] != KEY_MAX && ok1) pair_min(bk, bi, metric_key(s.a[0], v[u][0].y), cfg_index(s, first, j[u]) + 1);
        }
    }
    for (int d = 16; d > 0; d >>= 1)
        pair_min(bk, bi, __shfl_xor_sync(0xFFFFFFFFu, bk, d), __shfl_xor_sync(0xFFFFFFFFu, bi, d));
    if (lane == 0) { sl[warp].x = bk; sl[warp].y = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (u32 w = 1; w < n_warps; w++) pair_min(bk, bi, sl[w].x, sl[w].y);
        ulonglong2 m; m.x = bk; m.y = bi;
        minima[blockIdx.x] = m;
    }
    grid.sync();
    // 2: coarse bound = k-th smallest block minimum (equal all-ones entries ordered by position)
    if (gwarp < gridDim.x) {
        const ulonglong2 me = __ldcg(minima + gwarp);
        u32 ahead = 0;
        for (u32 q = lane; q < gridDim.x; q += 32) {
            const ulonglong2 o = __ldcg(minima + q);
            ahead += (o.x < me.x || (o.x == me.x && (o.y < me.y || (o.y == me.y && q < gwarp)))) ? 1u : 0u;
        }
        for (int d = 16; d > 0; d >>= 1) ahead += __shfl_xor_sync(0xFFFFFFFFu, ahead, d);
        if (lane == 0 && ahead == k - 1) { bound[0] = me.x; bound[1] = me.y; }
    }
    grid.sync();
    // 3: the sample pairs within the coarse bound (the rows come from L2 this time)
    const u64 bkey = __ldcg(bound), bidx = __ldcg(bound + 1);
    for (u64 c0 = (u64)warp * gridDim.x + blockIdx.x; c0 < sm.n_slots; c0 += SAMPLE_BATCH * stride) {
        u32 st[SAMPLE_BATCH];
        double2 v[SAMPLE_BATCH][NA];
        u64 j[SAMPLE_BATCH];
        load_batch(s, sm, c0, stride, lane, st, v, j);
#pragma unroll
        for (u32 u = 0; u < SAMPLE_BATCH; u++) {
            bool ok[2];
            eval_pair(s, st[u], v[u], ok[0], ok[1]);
            const u64 key[2] = {metric_key(s.a[0], v[u][0].x), metric_key(s.a[0], v[u][0].y)};
#pragma unroll
            for (u32 h = 0; h < 2; h++) {
                if (j[u] != KEY_MAX && ok[h] && pair_le(key[h], cfg_index(s, first, j[u]) + h, bkey, bidx)) {
                    const u32 p = atomicAdd(header + TK_SAMPLED, 1);
                    if (p < TK_SKEYS_CAP) { ulonglong2 e; e.x = key[h]; e.y = cfg_index(s, first, j[u]) + h; spairs[p] = e; }
                }
            }
        }
    }
    grid.sync();
    grid_dep_launch();              // late: a dependent that starts early only sits on registers other streams could use
    // 4: their k-th smallest (of the stored ones, if they did not all fit: still a valid bound);
    // fewer than k only when the coarse bound is all-ones, which then stays
    const u32 n = min(__ldcg(header + TK_SAMPLED), TK_SKEYS_CAP);
    if (n < k) return;
    for (u32 g = gwarp; g < n; g += total_warps) {
        const ulonglong2 me = __ldcg(spairs + g);
        u32 ahead = 0;
        for (u32 q = lane; q < n; q += 32) {
            const ulonglong2 o = __ldcg(spairs + q);
            ahead += (o.x < me.x || (o.x == me.x && o.y < me.y)) ? 1u : 0u;
        }
        for (int d = 16; d > 0; d >>= 1) ahead += __shfl_xor_sync(0xFFFFFFFFu, ahead, d);
        if (lane == 0 && ahead == k - 1) { bound[0] = me.x; bound[1] = me.y; }
    }
}

// Filter pass: passing configs within the bound go to the candidate list.
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS, 4) k_topk_filter(Src<NA> s, Range r, u32 *header, KI *cand) {
    grid_dep_wait();
    const u64 *bp = reinterpret_cast<const u64 *>(header + TK_BOUND);
    const u64 bkey = __ldcg(bp), bidx = __ldcg(bp + 1);
    const u64 tiles = r.count / TILE;
    // from the end of the range backwards: when the metrics were written just before this call the
    // end of the arrays is what the L2 still holds
    for (u64 back = blockIdx.x; back < tiles; back += gridDim.x) {
        const u64 tile = tiles - 1 - back;
        const u64 j0 = tile * TILE + 2 * threadIdx.x, j1 = j0 + TILE / 2;
        u32 st0, st1;
        double2 v0[NA], v1[NA];
        if (!load_live_pairs(s, j0, j1, st0, st1, v0, v1)) continue;
        bool ok[4];
        eval_pair(s, st0, v0, ok[0], ok[1]);
        eval_pair(s, st1, v1, ok[2], ok[3]);
        const u64 key[4] = {metric_key(s.a[0], v0[0].x), metric_key(s.a[0], v0[0].y), metric_key(s.a[0], v1[0].x),
                            metric_key(s.a[0], v1[0].y)};
        bool any = false;
#pragma unroll
        for (int u = 0; u < 4; u++) { ok[u] = ok[u] && key[u] <= bkey; any |= ok[u]; }
        if (!__any_sync(0xFFFFFFFFu, any)) continue;        // the usual case: nothing in this warp's 128 configs
#pragma unroll
        for (int u = 0; u < 4; u++) {
            const u64 idx = r.first + (u < 2 ? j0 : j1) + (u & 1);
            if (ok[u] && pair_le(key[u], idx, bkey, bidx)) topk_keep(key[u], idx, header, cand);
        }
    }
    grid_dep_launch();              // late: the rank kernel needs this block's registers only now
    if (blockIdx.x == gridDim.x - 1) {                      // ragged tail, scalar loads
        for (u64 j = tiles * TILE + threadIdx.x; j < r.count; j += blockDim.x) {
            u64 k0, k1;
            if (eval_one(s, j, k0, k1) && pair_le(k0, r.first + j, bkey, bidx)) topk_keep(k0, r.first + j, header, cand);
        }
    }
}

// Finish: every block stages the candidate list in shared memory; one warp per candidate counts
// the candidates ahead of it.  Ranks are distinct (config indices are), so every output slot has
// one writer.
__global__ void __launch_bounds__(SEL_THREADS) k_topk_rank(u32 *header, const KI *cand, u32 k, int negate_out, u64 *idx_out,
                                                           double *key_out, u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ulonglong2 *sl = reinterpret_cast<ulonglong2 *>(smem_raw);
    grid_dep_launch();
    grid_dep_wait();
    const u32 n = __ldcg(header + TK_COUNT);
    if (n > TK_CAND_CAP) {                                   // the list overflowed: hand the call to the fallback
        if (blockIdx.x == 0 && threadIdx.x == 0) header[TK_REDO] = 1;
        return;
    }
    const u32 found = min(n, k);
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) *count_out = found;
        for (u32 i = found + threadIdx.x; i < k; i += blockDim.x) {
            idx_out[i] = KEY_MAX;
            key_out[i] = __longlong_as_double(0x7FF0000000000000LL);
        }
    }
    const u32 n_warps = gridDim.x * (blockDim.x >> 5);
    if (blockIdx.x * (blockDim.x >> 5) >= n) return;         // no candidate for this block
    const ulonglong2 *list = reinterpret_cast<const ulonglong2 *>(cand);
    const u32 ns = min(n, TK_CAND_SMEM);             // a longer list is read past this point straight from memory
    for (u32 i = threadIdx.x; i < ns; i += blockDim.x) sl[i] = __ldcg(list + i);
    __syncthreads();
    const u32 lane = threadIdx.x & 31;
    for (u32 g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); g < n; g += n_warps) {
        const ulonglong2 me = g < ns ? sl[g] : __ldcg(list + g);
        u32 ahead = 0;
        for (u32 i = lane; i < ns; i += 32) {
            const ulonglong2 o = sl[i];
            ahead += (o.x < me.x || (o.x == me.x && o.y < me.y)) ? 1u : 0u;
        }
        for (u32 i = ns + lane; i < n; i += 32) {
            const ulonglong2 o = __ldcg(list + i);
            ahead += (o.x < me.x || (o.x == me.x && o.y < me.y)) ? 1u : 0u;
        }
        for (int d = 16; d > 0; d >>= 1) ahead += __shfl_xor_sync(0xFFFFFFFFu, ahead, d);
        if (lane == 0 && ahead < k) {
            const double v = dec(me.x);
            idx_out[ahead] = me.y;
            key_out[ahead] = negate_out ? 0.0 - v : v;
        }
    }
}

// ---- Pareto ----------------------------------------------------------------------------------------

// lexicographic minimum of (p, q) pairs over the block; every thread gets the result
__device__ __forceinline__ void block_lex_min(u64 &p, u64 &q, u64 (*scratch)[2]) {
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    for (int d = 16; d > 0; d >>= 1) {
        const u64 op = __shfl_xor_sync(0xFFFFFFFFu, p, d), oq = __shfl_xor_sync(0xFFFFFFFFu, q, d);
        if (op < p || (op == p && oq < q)) { p = op; q = oq; }
    }
    if (lane == 0) { scratch[warp][0] = p; scratch[warp][1] = q; }
    __syncthreads();
    p = scratch[0][0]; q = scratch[0][1];
    for (u32 w = 1; w < n_warps; w++) {
        const u64 op = scratch[w][0], oq = scratch[w][1];
        if (op < p || (op == p && oq < q)) { p = op; q = oq; }
    }
    __syncthreads();
}

// Sample pass.  Each block: its sample points that survive four of the block's own points (the
// seeds below) are gathered in shared memory and compared all against all; up to PA_PER_BLOCK of
// the block's front, spread over it, go to the workspace.  The last block sorts the union and
// sweeps it into the killer staircase: real points, ascending x, strictly falling y.
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS) k_pareto_sample(Src<NA> s, Sample sm, u32 *header, P2 *local, u32 *local_n,
                                                               P2 *killers) {
    constexpr u32 N_PTS = 2 * PA_ROWS_PER_WARP;
    __shared__ P2 list[PA_LOCAL_CAP];               // also the last block's sort buffer (PA_KILLERS entries)
    __shared__ P2 front[32];
    __shared__ u64 scratch[SEL_THREADS / 32][2];
    __shared__ u32 wkeep[SEL_THREADS / 32];
    __shared__ u32 n_list, n_front, last;
    static_assert(PA_LOCAL_CAP >= PA_KILLERS && PA_KILLERS == SEL_THREADS, "one killer candidate per thread in the merge");
    static_assert(PA_ROWS_PER_WARP % SAMPLE_BATCH == 0, "whole batches");
    const u32 lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = SEL_THREADS / 32;
    if (threadIdx.x == 0) { n_list = 0; n_front = 0; }
    u64 px[N_PTS], py[N_PTS];
    const u64 stride = (u64)gridDim.x * n_warps;
#pragma unroll
    for (u32 b = 0; b < PA_ROWS_PER_WARP / SAMPLE_BATCH; b++) {
        u32 st[SAMPLE_BATCH];
        double2 v[SAMPLE_BATCH][NA];
        u64 j[SAMPLE_BATCH];
        load_batch(s, sm, (u64)warp * gridDim.x + blockIdx.x + (u64)b * SAMPLE_BATCH * stride, stride, lane, st, v, j);
#pragma unroll
        for (u32 u = 0; u < SAMPLE_BATCH; u++) {
            const u32 i = 2 * (b * SAMPLE_BATCH + u);
            bool ok0, ok1;
            eval_pair(s, st[u], v[u], ok0, ok1);
            px[i] = py[i] = px[i + 1] = py[i + 1] = KEY_MAX;            // "no point"
            if (j[u] != KEY_MAX && ok0) { px[i] = metric_key(s.a[0], v[u][0].x); py[i] = metric_key(s.a[1 % NA], v[u][1 % NA].x); }
            if (j[u] != KEY_MAX && ok1) { px[i + 1] = metric_key(s.a[0], v[u][0].y); py[i + 1] = metric_key(s.a[1 % NA], v[u][1 % NA].y); }
        }
    }
    // four seeds, all real points of this block: smallest (x, y), smallest (y, x), and between them
    // the lowest point of the left half (x up to the midpoint of the two, in encoded order) and the
    // leftmost point of the lower half
    u64 ax = KEY_MAX, ay = KEY_MAX, by = KEY_MAX, bx = KEY_MAX;
#pragma unroll
    for (u32 i = 0; i < N_PTS; i++) {
        if (px[i] < ax || (px[i] == ax && py[i] < ay)) { ax = px[i]; ay = py[i]; }
        if (py[i] < by || (py[i] == by && px[i] < bx)) { by = py[i]; bx = px[i]; }
    }
    block_lex_min(ax, ay, scratch);
    block_lex_min(by, bx, scratch);
    const u64 xm = ax + (bx - ax) / 2, ym = by + (ay - by) / 2;     // bx >= ax and ay >= by
    u64 cy = KEY_MAX, cx = KEY_MAX, dx = KEY_MAX, dy = KEY_MAX;
#pragma unroll
    for (u32 i = 0; i < N_PTS; i++) {
        if (px[i] <= xm && (py[i] < cy || (py[i] == cy && px[i] < cx))) { cy = py[i]; cx = px[i]; }
        if (py[i] <= ym && (px[i] < dx || (px[i] == dx && py[i] < dy))) { dx = px[i]; dy = py[i]; }
    }
    block_lex_min(cy, cx, scratch);
    block_lex_min(dx, dy, scratch);
    // points no seed rules out (the seeds themselves included)
#pragma unroll
    for (u32 i = 0; i < N_PTS; i++) {
        if (px[i] == KEY_MAX && py[i] == KEY_MAX) continue;
        if (dominates(ax, ay, px[i], py[i]) || dominates(bx, by, px[i], py[i]) || dominates(cx, cy, px[i], py[i]) ||
            dominates(dx, dy, px[i], py[i]))
            continue;
        const u32 pos = atomicAdd(&n_list, 1);
        if (pos < PA_LOCAL_CAP) { list[pos].x = px[i]; list[pos].y = py[i]; }     // beyond the cap: dropped, any subset will do
    }
    __syncthreads();
    const u32 nl = min(n_list, PA_LOCAL_CAP);
    // all against all, four list entries per step; of equal points the first in the list stays
    for (u32 i = threadIdx.x; i < nl; i += blockDim.x) {
        const P2 me = list[i];
        bool out = false;
        for (u32 q0 = 0; q0 < nl && !out; q0 += 4) {
#pragma unroll
            for (u32 u = 0; u < 4; u++) {
                const u32 q = min(q0 + u, nl - 1);
                const P2 o = list[q];
                out |= dominates(o.x, o.y, me.x, me.y) || (o.x == me.x && o.y == me.y && q < i);
            }
        }
        if (!out) {
            const u32 pos = atomicAdd(&n_front, 1);
            if (pos < 32) front[pos] = me;
        }
    }
    grid_dep_launch();              // late, as in k_topk_bound
    __syncthreads();
    const u32 nf = min(n_front, 32u);
    // hand on up to PA_PER_BLOCK of them, evenly spaced by rank in x
    if (threadIdx.x < nf) {
        const P2 me = front[threadIdx.x];
        u32 rank = 0;
        for (u32 q = 0; q < nf; q++) rank += front[q].x < me.x ? 1u : 0u;        // x values of a front are distinct
        const u32 slot = rank * PA_PER_BLOCK / nf;
        const bool first_of_slot = rank == 0 || (rank - 1) * PA_PER_BLOCK / nf != slot;
        if (nf <= PA_PER_BLOCK) local[(size_t)blockIdx.x * PA_PER_BLOCK + rank] = me;
        else if (first_of_slot) local[(size_t)blockIdx.x * PA_PER_BLOCK + slot] = me;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        local_n[blockIdx.x] = min(nf, PA_PER_BLOCK);
        __threadfence();
        last = atomicAdd(header + PH_TICKET, 1) == gridDim.x - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    // union of the block fronts (one per thread) -> sorted by (x, y) -> strictly falling y
    {
        const u32 i = threadIdx.x, b = i / PA_PER_BLOCK, q = i % PA_PER_BLOCK;
        P2 p; p.x = KEY_MAX; p.y = KEY_MAX;
        if (b < gridDim.x && q < __ldcg(local_n + b)) {
            const ulonglong2 w = __ldcg(reinterpret_cast<const ulonglong2 *>(local + i));
            p.x = w.x; p.y = w.y;
        }
        list[i] = p;
    }
    __syncthreads();
    block_bitonic_sort(list, PA_KILLERS, [](const P2 &a, const P2 &b) { return a.x < b.x || (a.x == b.x && a.y < b.y); });
    const P2 it = list[threadIdx.x];
    const bool real = !(it.x == KEY_MAX && it.y == KEY_MAX);
    u64 incl = it.y;                                 // smallest y up to and including this point
    for (u32 d = 1; d < 32; d <<= 1) {
        const u64 o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d && o < incl) incl = o;
    }
    u64 before = __shfl_up_sync(0xFFFFFFFFu, incl, 1);
    if (lane == 0) before = KEY_MAX;
    if (lane == 31) scratch[warp][0] = incl;
    __syncthreads();
    for (u32 w = 0; w < warp; w++) before = scratch[w][0] < before ? scratch[w][0] : before;
    const bool keep = real && it.y < before;
    const u32 ballot = __ballot_sync(0xFFFFFFFFu, keep);
    if (lane == 0) wkeep[warp] = __popc(ballot);
    __syncthreads();
    u32 off = 0, total = 0;
    for (u32 w = 0; w < n_warps; w++) { if (w < warp) off += wkeep[w]; total += wkeep[w]; }
    if (keep) {
        ulonglong2 w; w.x = it.x; w.y = it.y;
        *reinterpret_cast<ulonglong2 *>(killers + off + __popc(ballot & ((1u << lane) - 1))) = w;
    }
    if (threadIdx.x == 0) header[PH_KILLERS] = total;
}

// Filter pass: passing configs no killer strictly dominates go to the survivor list.
template <int NA>
__global__ void __launch_bounds__(SEL_THREADS, 4) k_pareto_filter(Src<NA> s, Range r, u32 *header, const P2 *killers, P3 *surv) {
    __shared__ P2 ks[PA_KILLERS];
    grid_dep_wait();
    KillerSet K;
    K.k = ks;
    K.n = min(__ldcg(header + PH_KILLERS), PA_KILLERS);
    for (u32 i = threadIdx.x; i < K.n; i += blockDim.x) {
        const ulonglong2 w = __ldcg(reinterpret_cast<const ulonglong2 *>(killers + i));
        ks[i].x = w.x; ks[i].y = w.y;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; i++) {
        if (K.n > 0) { const P2 p = ks[(K.n * (2 * i + 1)) / 8]; K.rx[i] = p.x; K.ry[i] = p.y; }
        else { K.rx[i] = KEY_MAX; K.ry[i] = KEY_MAX; }
    }
    const u64 tiles = r.count / TILE;
    // from the end of the range backwards: when the metrics were written just before this call the
    // end of the arrays is what the L2 still holds
    for (u64 back = blockIdx.x; back < tiles; back += gridDim.x) {
        const u64 tile = tiles - 1 - back;
        const u64 j0 = tile * TILE + 2 * threadIdx.x, j1 = j0 + TILE / 2;
        u32 st0, st1;
        double2 v0[NA], v1[NA];
        if (!load_live_pairs(s, j0, j1, st0, st1, v0, v1)) continue;
        bool ok[4];
        eval_pair(s, st0, v0, ok[0], ok[1]);
        eval_pair(s, st1, v1, ok[2], ok[3]);
        if (!__any_sync(0xFFFFFFFFu, ok[0] | ok[1] | ok[2] | ok[3])) continue;
        const Arr &ax = s.a[0], &ay = s.a[1 % NA];
        const u64 x[4] = {metric_key(ax, v0[0].x), metric_key(ax, v0[0].y), metric_key(ax, v1[0].x), metric_key(ax, v1[0].y)};
        const u64 y[4] = {metric_key(ay, v0[1 % NA].x), metric_key(ay, v0[1 % NA].y), metric_key(ay, v1[1 % NA].x),
                          metric_key(ay, v1[1 % NA].y)};
#pragma unroll
        for (int u = 0; u < 4; u++)
            if (ok[u] && !K.kills(x[u], y[u])) pareto_keep(x[u], y[u], r.first + (u < 2 ? j0 : j1) + (u & 1), header, surv);
    }
    grid_dep_launch();              // late: the rank kernel needs this block's registers only now
    if (blockIdx.x == gridDim.x - 1) {                      // ragged tail, scalar loads
        for (u64 j = tiles * TILE + threadIdx.x; j < r.count; j += blockDim.x) {
            u64 x, y;
            if (eval_one(s, j, x, y) && !K.kills(x, y)) pareto_keep(x, y, r.first + j, header, surv);
        }
    }
}

// Finish.  Every block stages the survivors in shared memory; one warp per survivor looks for a
// survivor that rules it out (a dominating point, or an equal point with a lower index); those left
// are the front and go to a second list.  The block that finishes last places each front point at
// its rank in x (x values of a front are distinct).
__global__ void __launch_bounds__(SEL_THREADS) k_pareto_rank(u32 *header, const P3 *surv, KI *front, u64 *idx_out, u32 out_cap,
                                                             u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 last;
    grid_dep_launch();
    grid_dep_wait();
    const u32 n = __ldcg(header + PH_COUNT);
    if (n > PA_SURV_CAP) {                                   // the list overflowed: the general kernel redoes the call
        if (blockIdx.x == 0 && threadIdx.x == 0) header[1] = 1;
        return;
    }
    u64 *sx = reinterpret_cast<u64 *>(smem_raw), *sy = sx + n;      // x and y staged; the index is read only for equal points
    const u32 lane = threadIdx.x & 31;
    const u32 n_warps = gridDim.x * (blockDim.x >> 5);
    const u64 *w = reinterpret_cast<const u64 *>(surv);
    if (blockIdx.x * (blockDim.x >> 5) < n) {               // this block has survivors to judge
        for (u32 i = threadIdx.x; i < 3 * n; i += blockDim.x) {
            const u32 e = i / 3, f = i % 3;
            if (f < 2) (f == 0 ? sx : sy)[e] = __ldcg(w + i);
        }
        __syncthreads();
        for (u32 g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); g < n; g += n_warps) {
            const u64 mx = sx[g], my = sy[g], mi = __ldcg(w + 3 * (size_t)g + 2);
            bool out = false;
            for (u32 i = lane; i < n; i += 32) {
                const u64 ox = sx[i], oy = sy[i];
                out |= dominates(ox, oy, mx, my) || (ox == mx && oy == my && __ldcg(w + 3 * (size_t)i + 2) < mi);
            }
            if (!__any_sync(0xFFFFFFFFu, out) && lane == 0) {
                const u32 pos = atomicAdd(header + PH_FRONT, 1);   // pos < n <= PA_SURV_CAP
                front[pos].key = mx; front[pos].idx = mi;
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = atomicAdd(header + PH_TICKET2, 1) == gridDim.x - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    const u32 nf = __ldcg(header + PH_FRONT);
    const ulonglong2 *f = reinterpret_cast<const ulonglong2 *>(front);
    const u32 lim = min(out_cap, GUIDE_PARETO_MAX);
    for (u32 i = threadIdx.x; i < nf; i += blockDim.x) sx[i] = __ldcg(f + i).x;      // nf <= n: fits
    __syncthreads();
    for (u32 g = threadIdx.x >> 5; g < nf; g += blockDim.x >> 5) {
        const ulonglong2 me = __ldcg(f + g);
        u32 ahead = 0;
        for (u32 i = lane; i < nf; i += 32) ahead += sx[i] < me.x ? 1u : 0u;
        for (int d = 16; d > 0; d >>= 1) ahead += __shfl_xor_sync(0xFFFFFFFFu, ahead, d);
        if (lane == 0 && ahead < lim) idx_out[ahead] = me.y;
    }
    if (threadIdx.x == 0) *count_out = nf > GUIDE_PARETO_MAX ? 0xFFFFFFFFu : nf;
}

// ---- host side -----------------------------------------------------------------------------------------

// The arrays a call touches, each once: metric(s) first, then the bounded ones not yet listed.
static int collect_arrays(const guide_outputs &o, const guide_constraints &c, int m0, int m1, Arr *arr) {
    int n = 0;
    auto add_metric = [&](int key) { arr[n++] = Arr{metric_array_of(o, key), 0.0, 0, key == GUIDE_THROUGHPUT ? 1 : 0}; };
    add_metric(m0);
    if (m1 >= 0) add_metric(m1);
    auto add_bound = [&](const double *p, double bound, int cmp) {
        for (int i = 0; i < n; i++)
            if (arr[i].p == p && arr[i].cmp == 0) { arr[i].bound = bound; arr[i].cmp = cmp; return; }
        arr[n++] = Arr{p, bound, cmp, 0};
    };
    if (c.max_ttft < INFINITY)
        add_bound(c.ttft_stat == GUIDE_STAT_MEAN ? o.ttft : c.ttft_stat == GUIDE_STAT_P50 ? o.ttft_p50 : o.ttft_p99, c.max_ttft, 1);
    if (c.max_latency < INFINITY) add_bound(o.latency, c.max_latency, 1);
    if (c.max_cost_per_hr < INFINITY) add_bound(o.cost_per_hr, c.max_cost_per_hr, 1);
    if (c.min_throughput > 0.0) add_bound(o.thr_decode, c.min_throughput, 2);
    return n;
}

static u32 filter_grid(u64 count) {
    const u64 tiles = std::max<u64>(count / TILE, 1);
    return (u32)std::min<u64>((u64)num_sms() * 4, tiles);
}

// The walk over the sample (see Sample): groups of r rows, n_slots of them visited.
static Sample make_sample(u64 n_rows, u32 want_rows, u32 max_r) {
    Sample sm;
    sm.r = (u32)std::min<u64>(std::max<u64>(n_rows / want_rows, 1), max_r);
    sm.n_groups = n_rows / sm.r;
    sm.n_slots = std::min<u64>(sm.n_groups, want_rows);
    sm.mul = 1;
    for (u64 p : {1000003ull, 999983ull, 1299709ull, 15485863ull})
        if (sm.n_groups % p != 0) { sm.mul = p; break; }
    return sm;
}

// Can the bound kernel's grid (TK_SAMPLE_BLOCKS blocks of SEL_THREADS threads) be resident at once on
// the current device, and does the device launch cooperatively?  Asked once per device.  Setting
// GUIDE_NO_COOPERATIVE in the environment forces the two-kernel form (the tests use it to cover both).
template <int NA>
static bool cooperative_ok() {
    static int cached[64] = {};                      // 0 unknown, 1 yes, 2 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (!cached[dev]) {
        int coop = 0, per_sm = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_topk_bound<NA>, SEL_THREADS, 0);
        if (getenv("GUIDE_NO_COOPERATIVE")) coop = 0;
        cached[dev] = (coop && (u64)per_sm * num_sms() >= TK_SAMPLE_BLOCKS) ? 1 : 2;
    }
    return cached[dev] == 1;
}

template <int NA>
static int topk_stream_na(const Arr *arr, Range r, const guide_outputs &mat, u32 k, int negate, u32 *header,
                          unsigned char *region, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st) {
    Src<NA> s;
    for (int i = 0; i < NA; i++) s.a[i] = arr[i];
    s.status = mat.status;
    s.row_base = nullptr;
    ulonglong2 *minima = reinterpret_cast<ulonglong2 *>(region);
    ulonglong2 *spairs = reinterpret_cast<ulonglong2 *>(region + TK_OFF_SKEYS);
    KI *cand = reinterpret_cast<KI *>(region + TK_OFF_CAND);
    // the coarse bound needs every block to see rows: the walk covers the whole sample (all groups)
    Sample sm = make_sample(r.count / ROW, TK_SAMPLE_ROWS, TK_SAMPLE_MAX_R);
    sm.n_slots = sm.n_groups;
    if (cooperative_ok<NA>()) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(TK_SAMPLE_BLOCKS); cfg.blockDim = dim3(SEL_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeCooperative;
        at[0].val.cooperative = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        GUIDE_CUDA(cudaLaunchKernelEx(&cfg, k_topk_bound<NA>, s, sm, r.first, k, header, minima, spairs));
    } else {
        GUIDE_CUDA(cudaMemsetAsync(header, 0, 256, st));
        k_topk_sample<NA><<<TK_SAMPLE_BLOCKS, SEL_THREADS, 0, st>>>(s, sm, r.first, k, header, minima);
        GUIDE_CUDA(cudaGetLastError());
        GUIDE_CUDA(launch_dependent(k_topk_refine<NA>, TK_SAMPLE_BLOCKS, SEL_THREADS, 0, st, s, sm, r.first, k, header, spairs));
    }
    GUIDE_CUDA(launch_dependent(k_topk_filter<NA>, filter_grid(r.count), SEL_THREADS, 0, st, s, r, header, cand));
    const size_t smem = (size_t)TK_CAND_SMEM * sizeof(KI);
    GUIDE_CUDA(cudaFuncSetAttribute(k_topk_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    GUIDE_CUDA(launch_dependent(k_topk_rank, num_sms(), SEL_THREADS, smem, st, header, (const KI *)cand, k, negate, idx_out,
                                key_out, count_out));
    return GUIDE_OK;
}

int launch_topk_stream(Range r, const guide_outputs &mat, const guide_constraints &c, int key, u32 k, u32 *header,
                       unsigned char *region, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st) {
    Arr arr[MAX_ARR];
    const int na = collect_arrays(mat, c, key, -1, arr);
    const int negate = key == GUIDE_THROUGHPUT;
    switch (na) {
    case 1: return topk_stream_na<1>(arr, r, mat, k, negate, header, region, idx_out, key_out, count_out, st);
    case 2: return topk_stream_na<2>(arr, r, mat, k, negate, header, region, idx_out, key_out, count_out, st);
    case 3: return topk_stream_na<3>(arr, r, mat, k, negate, header, region, idx_out, key_out, count_out, st);
    case 4: return topk_stream_na<4>(arr, r, mat, k, negate, header, region, idx_out, key_out, count_out, st);
    case 5: return topk_stream_na<5>(arr, r, mat, k, negate, header, region, idx_out, key_out, count_out, st);
    default: return fail(GUIDE_ERR_UNSUPPORTED, "a top-k call touches at most five arrays");
    }
}

template <int NA>
static int pareto_stream_na(const Arr *arr, Range r, const guide_outputs &mat, u32 *header, unsigned char *region, u64 *idx_out,
                            u32 cap, u32 *count_out, cudaStream_t st) {
    Src<NA> s;
    for (int i = 0; i < NA; i++) s.a[i] = arr[i];
    s.status = mat.status;
    s.row_base = nullptr;
    P2 *local = reinterpret_cast<P2 *>(region);
    P2 *killers = reinterpret_cast<P2 *>(region + PA_OFF_KILLERS);
    u32 *local_n = reinterpret_cast<u32 *>(region + PA_OFF_LOCAL_N);
    P3 *surv = reinterpret_cast<P3 *>(region + PA_OFF_SURV);
    KI *front = reinterpret_cast<KI *>(region + PA_OFF_FRONT);
    const Sample sm = make_sample(r.count / ROW, PA_SAMPLE_ROWS, 1u << 20);
    k_pareto_sample<NA><<<PA_SAMPLE_BLOCKS, SEL_THREADS, 0, st>>>(s, sm, header, local, local_n, killers);
    GUIDE_CUDA(cudaGetLastError());
    GUIDE_CUDA(launch_dependent(k_pareto_filter<NA>, filter_grid(r.count), SEL_THREADS, 0, st, s, r, header, (const P2 *)killers,
                                surv));
    const size_t smem = (size_t)PA_SURV_CAP * 16;
    GUIDE_CUDA(cudaFuncSetAttribute(k_pareto_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    GUIDE_CUDA(launch_dependent(k_pareto_rank, num_sms(), SEL_THREADS, smem, st, header, (const P3 *)surv, front, idx_out, cap,
                                count_out));
    return GUIDE_OK;
}

int launch_pareto_stream(Range r, const guide_outputs &mat, const guide_constraints &c, int xm, int ym, u32 *header,
                         unsigned char *region, u64 *idx_out, u32 cap, u32 *count_out, cudaStream_t st) {
    Arr arr[MAX_ARR];
    const int na = collect_arrays(mat, c, xm, ym, arr);
    switch (na) {
    case 2: return pareto_stream_na<2>(arr, r, mat, header, region, idx_out, cap, count_out, st);
    case 3: return pareto_stream_na<3>(arr, r, mat, header, region, idx_out, cap, count_out, st);
    case 4: return pareto_stream_na<4>(arr, r, mat, header, region, idx_out, cap, count_out, st);
    case 5: return pareto_stream_na<5>(arr, r, mat, header, region, idx_out, cap, count_out, st);
    case 6: return pareto_stream_na<6>(arr, r, mat, header, region, idx_out, cap, count_out, st);
    default: return fail(GUIDE_ERR_UNSUPPORTED, "a Pareto call touches two to six arrays");
    }
}

// ---- fused form: nothing materialised ---------------------------------------------------------------

// The sample rows of a whole closed-form space, evaluated config by config into the compact
// scratch: pass flag (0 = fits and meets the constraints), the metric(s) of the call, and where
// each row starts.  One thread per config; 64 consecutive configs of a row share everything but
// the length pair.
template <int TIME_SUM>
__global__ void __launch_bounds__(SEL_THREADS) k_fused_sample(DSpace s, int tp_model, Sample sm, Cons c, int m0, int m1,
                                                              u64 *row_base, uint8_t *pass, double *a0, double *a1, int beside) {
    grid_dep_launch();
    const u64 slot = (u64)blockIdx.x * (SEL_THREADS / ROW) + threadIdx.x / ROW;
    if (slot >= sm.n_slots) { if (beside) grid_dep_wait(); return; }
    const u32 l = threadIdx.x % ROW;
    const u64 first = sm.row(slot) * ROW;
    Metrics m;
    closed_form_eval<TIME_SUM>(s, decode_index(s, first + l), tp_model, m);
    double a = 0.0, b = 0.0;
    const bool ok = fused_pick(m, c, m0, m1, a, b);
    const u64 q = slot * ROW + l;
    pass[q] = ok ? 0 : 1;
    a0[q] = a;
    if (m1 >= 0) a1[q] = b;
    if (l == 0) row_base[slot] = first;
    // Launched beside its predecessor in the stream (another sample), the grid must not be complete
    // before that one is: whatever follows in the stream waits for this grid only.
    if (beside) grid_dep_wait();
}

// Filter pass of the fused top-k: the model walk, with the configs that fit, meet the constraints
// and are within the bound going to the candidate list.
template <int TIME_SUM>
__global__ void __launch_bounds__(MODEL_THREADS, MODEL_BLOCKS_PER_SM)
k_topk_model(DSpace s, int tp_model, u32 n_chunks, unsigned *ticket, Cons c, int key, u32 *header, KI *cand) {
    grid_dep_launch();
    grid_dep_wait();
    const u64 *bp = reinterpret_cast<const u64 *>(header + TK_BOUND);
    const u64 bkey = __ldcg(bp), bidx = __ldcg(bp + 1);
    model_walk<TIME_SUM>(s, tp_model, n_chunks, ticket,
                         [&](bool fits, u32, u32, u64 j, double latency, double ttft, double tpot, double thr, double cost_hr,
                             double cost_tok, u64, u64) {
        if (!fits || !meets(c, latency, ttft, thr, cost_hr)) return;
        const u64 k64 = enc(pick_metric(key, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
        if (pair_le(k64, j, bkey, bidx)) topk_keep(k64, j, header, cand);
    });
}

// Filter pass of the fused Pareto front: configs no killer strictly dominates go to the survivor list.
template <int TIME_SUM>
__global__ void __launch_bounds__(MODEL_THREADS, MODEL_BLOCKS_PER_SM)
k_pareto_model(DSpace s, int tp_model, u32 n_chunks, unsigned *ticket, Cons c, int xm, int ym, u32 *header, const P2 *killers,
               P3 *surv) {
    __shared__ P2 ks[PA_KILLERS];
    grid_dep_launch();
    grid_dep_wait();
    KillerSet K;
    K.k = ks;
    K.n = min(__ldcg(header + PH_KILLERS), PA_KILLERS);
    for (u32 i = threadIdx.x; i < K.n; i += blockDim.x) {
        const ulonglong2 w = __ldcg(reinterpret_cast<const ulonglong2 *>(killers + i));
        ks[i].x = w.x; ks[i].y = w.y;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; i++) {
        if (K.n > 0) { const P2 p = ks[(K.n * (2 * i + 1)) / 8]; K.rx[i] = p.x; K.ry[i] = p.y; }
        else { K.rx[i] = KEY_MAX; K.ry[i] = KEY_MAX; }
    }
    model_walk<TIME_SUM>(s, tp_model, n_chunks, ticket,
                         [&](bool fits, u32, u32, u64 j, double latency, double ttft, double tpot, double thr, double cost_hr,
                             double cost_tok, u64, u64) {
        if (!fits || !meets(c, latency, ttft, thr, cost_hr)) return;
        const u64 x = enc(pick_metric(xm, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
        const u64 y = enc(pick_metric(ym, latency, ttft, ttft, tpot, thr, cost_hr, cost_tok));
        if (!K.kills(x, y)) pareto_keep(x, y, j, header, surv);
    });
}

// Whole closed-form spaces whose (TP, length) plane divides into foursomes (what model_walk needs),
// large enough for the sampled bound to pay.
bool fused_stream_eligible(const DSpace &s, Range r) {
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    const u32 n_tl = s.n_t * s.n_l;
    if (r.first != 0 || r.count != total || total < STREAM_MIN_COUNT) return false;
    if (s.n_l % 4 != 0 || n_tl < 32 || s.chunked) return false;
    const u64 n_hf = (u64)s.n_h * s.n_f;
    return (u64)s.n_m * s.n_b * (n_tl / 4) * ((n_hf + MODEL_CHUNK - 1) / MODEL_CHUNK) <= 0x7FFFFFFFull;
}

// the compact scratch as the arrays of a selection source
struct FusedScratch {
    u64 *row_base;
    uint8_t *pass;
    double *a0, *a1;
};
static FusedScratch fused_scratch(unsigned char *base) {
    return FusedScratch{reinterpret_cast<u64 *>(base), base + FU_OFF_PASS, reinterpret_cast<double *>(base + FU_OFF_A0),
                        reinterpret_cast<double *>(base + FU_OFF_A1)};
}

// sample rows of the space -> compact scratch; returns the walk over the scratch (row c of it is slot c)
template <int TIME_SUM>
static int fused_sample(const DSpace &s, int tp_model, const Cons &c, int m0, int m1, u32 want_rows, u32 max_r, const FusedScratch &f,
                        Sample *compact, cudaStream_t st, int phase) {
    const bool beside = phase == FUSED_SAMPLE_BESIDE;
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    Sample sm = make_sample(total / ROW, want_rows, max_r);
    sm.n_slots = std::min<u64>(sm.n_groups, FUSED_ROWS);
    const u32 grid = (u32)((sm.n_slots + SEL_THREADS / ROW - 1) / (SEL_THREADS / ROW));
    if (phase == FUSED_BOUND_ONLY) {
        // the rows were evaluated by an earlier call with the same arguments
    } else if (beside) {
        // the stream's previous kernel is the other selection's sample, which lets its dependents start at once
        GUIDE_CUDA(launch_dependent(k_fused_sample<TIME_SUM>, grid, SEL_THREADS, 0, st, s, tp_model, sm, c, m0, m1, f.row_base, f.pass,
                                    f.a0, f.a1, 1));
    } else {
        k_fused_sample<TIME_SUM><<<grid, SEL_THREADS, 0, st>>>(s, tp_model, sm, c, m0, m1, f.row_base, f.pass, f.a0, f.a1, 0);
        GUIDE_CUDA(cudaGetLastError());
    }
    compact->n_groups = sm.n_slots; compact->n_slots = sm.n_slots; compact->mul = 1; compact->r = 1;
    return GUIDE_OK;
}

static cudaError_t launch_model_dependent_cfg(cudaLaunchConfig_t *cfg, cudaLaunchAttribute *at, cudaStream_t st) {
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((u32)num_sms() * MODEL_BLOCKS_PER_SM); cfg->blockDim = dim3(MODEL_THREADS); cfg->dynamicSmemBytes = 0;
    cfg->stream = st;
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg->attrs = at; cfg->numAttrs = 1;
    return cudaSuccess;
}

template <int TIME_SUM>
static int topk_fused_t(const DSpace &s, int tp_model, const guide_constraints &gc, int key, u32 k, u32 *header,
                        unsigned char *region, unsigned *ticket, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st,
                        int phase) {
    const Cons c = make_cons(gc);
    const FusedScratch f = fused_scratch(region + TK_OFF_FUSED);
    ulonglong2 *minima = reinterpret_cast<ulonglong2 *>(region);
    ulonglong2 *spairs = reinterpret_cast<ulonglong2 *>(region + TK_OFF_SKEYS);
    KI *cand = reinterpret_cast<KI *>(region + TK_OFF_CAND);
    const size_t smem = (size_t)TK_CAND_SMEM * sizeof(KI);
    if (phase == FUSED_RANK) {
        GUIDE_CUDA(cudaFuncSetAttribute(k_topk_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GUIDE_CUDA(launch_dependent(k_topk_rank, num_sms(), SEL_THREADS, smem, st, header, (const KI *)cand, k,
                                    key == GUIDE_THROUGHPUT ? 1 : 0, idx_out, key_out, count_out));
        return GUIDE_OK;
    }
    if (phase == FUSED_ALL) GUIDE_CUDA(cudaMemsetAsync(ticket, 0, 4, st));           // the model walk's work counter
    Sample sm;
    // Half the rows of the materialised path's sample: here a row costs an evaluation of 64 configs, not a
    // read, and the filter pass behind it tolerates the wider bound (workload 5: 3,542 survivors instead
    // of 2,465, the call 10 us shorter).
    int rc = fused_sample<TIME_SUM>(s, tp_model, c, key, -1, TK_SAMPLE_ROWS / 2, TK_SAMPLE_MAX_R * 2, f, &sm, st, phase);
    if (rc) return rc;
    if (phase == FUSED_SAMPLE || phase == FUSED_SAMPLE_BESIDE) return GUIDE_OK;
    Src<1> src;
    src.a[0] = Arr{f.a0, 0.0, 0, 0};                         // pick_metric has negated the throughput already
    src.status = f.pass;
    src.row_base = f.row_base;
    if (cooperative_ok<1>()) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(TK_SAMPLE_BLOCKS); cfg.blockDim = dim3(SEL_THREADS); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeCooperative;
        at[0].val.cooperative = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        GUIDE_CUDA(cudaLaunchKernelEx(&cfg, k_topk_bound<1>, src, sm, (u64)0, k, header, minima, spairs));
    } else {
        GUIDE_CUDA(cudaMemsetAsync(header, 0, 256, st));
        k_topk_sample<1><<<TK_SAMPLE_BLOCKS, SEL_THREADS, 0, st>>>(src, sm, (u64)0, k, header, minima);
        GUIDE_CUDA(cudaGetLastError());
        GUIDE_CUDA(launch_dependent(k_topk_refine<1>, TK_SAMPLE_BLOCKS, SEL_THREADS, 0, st, src, sm, (u64)0, k, header, spairs));
    }
    if (phase == FUSED_BOUND || phase == FUSED_BOUND_ONLY) return GUIDE_OK;
    const u32 n_chunks = (s.n_h * s.n_f + MODEL_CHUNK - 1) / MODEL_CHUNK;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute at[1];
    launch_model_dependent_cfg(&cfg, at, st);
    GUIDE_CUDA(cudaLaunchKernelEx(&cfg, k_topk_model<TIME_SUM>, s, tp_model, n_chunks, ticket, c, key, header, cand));
    GUIDE_CUDA(cudaFuncSetAttribute(k_topk_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    GUIDE_CUDA(launch_dependent(k_topk_rank, num_sms(), SEL_THREADS, smem, st, header, (const KI *)cand, k,
                                key == GUIDE_THROUGHPUT ? 1 : 0, idx_out, key_out, count_out));
    return GUIDE_OK;
}

int launch_topk_fused(const DSpace &s, int time_model, int tp_model, const guide_constraints &c, int key, u32 k, u32 *header,
                      unsigned char *region, unsigned *ticket, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st,
                      int phase) {
    return time_model ? topk_fused_t<1>(s, tp_model, c, key, k, header, region, ticket, idx_out, key_out, count_out, st, phase)
                      : topk_fused_t<0>(s, tp_model, c, key, k, header, region, ticket, idx_out, key_out, count_out, st, phase);
}

// Where the filter pass of a combined call finds the lists of the two selections' workspaces.
void fused_lists(unsigned char *topk_region, unsigned char *pareto_region, LineSelect *sel) {
    sel->cand = reinterpret_cast<KI *>(topk_region + TK_OFF_CAND);
    sel->killers = reinterpret_cast<const P2 *>(pareto_region + PA_OFF_KILLERS);
    sel->surv = reinterpret_cast<P3 *>(pareto_region + PA_OFF_SURV);
}

template <int TIME_SUM>
static int pareto_fused_t(const DSpace &s, int tp_model, const guide_constraints &gc, int xm, int ym, u32 *header,
                          unsigned char *region, unsigned *ticket, u64 *idx_out, u32 cap, u32 *count_out, cudaStream_t st,
                          int phase) {
    const Cons c = make_cons(gc);
    const FusedScratch f = fused_scratch(region + PA_OFF_FUSED);
    P2 *local = reinterpret_cast<P2 *>(region);
    P2 *killers = reinterpret_cast<P2 *>(region + PA_OFF_KILLERS);
    u32 *local_n = reinterpret_cast<u32 *>(region + PA_OFF_LOCAL_N);
    P3 *surv = reinterpret_cast<P3 *>(region + PA_OFF_SURV);
    KI *front = reinterpret_cast<KI *>(region + PA_OFF_FRONT);
    const size_t smem = (size_t)PA_SURV_CAP * 16;
    if (phase == FUSED_RANK) {
        GUIDE_CUDA(cudaFuncSetAttribute(k_pareto_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GUIDE_CUDA(launch_dependent(k_pareto_rank, num_sms(), SEL_THREADS, smem, st, header, (const P3 *)surv, front, idx_out, cap,
                                    count_out));
        return GUIDE_OK;
    }
    if (phase == FUSED_ALL) GUIDE_CUDA(cudaMemsetAsync(ticket, 0, 4, st));
    Sample sm;
    int rc = fused_sample<TIME_SUM>(s, tp_model, c, xm, ym, PA_SAMPLE_ROWS, 1u << 20, f, &sm, st, phase);
    if (rc) return rc;
    if (phase == FUSED_SAMPLE || phase == FUSED_SAMPLE_BESIDE) return GUIDE_OK;
    Src<2> src;
    src.a[0] = Arr{f.a0, 0.0, 0, 0};
    src.a[1] = Arr{f.a1, 0.0, 0, 0};
    src.status = f.pass;
    src.row_base = f.row_base;
    k_pareto_sample<2><<<PA_SAMPLE_BLOCKS, SEL_THREADS, 0, st>>>(src, sm, header, local, local_n, killers);
    GUIDE_CUDA(cudaGetLastError());
    if (phase == FUSED_BOUND || phase == FUSED_BOUND_ONLY) return GUIDE_OK;
    const u32 n_chunks = (s.n_h * s.n_f + MODEL_CHUNK - 1) / MODEL_CHUNK;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute at[1];
    launch_model_dependent_cfg(&cfg, at, st);
    GUIDE_CUDA(cudaLaunchKernelEx(&cfg, k_pareto_model<TIME_SUM>, s, tp_model, n_chunks, ticket, c, xm, ym, header,
                                  (const P2 *)killers, surv));
    GUIDE_CUDA(cudaFuncSetAttribute(k_pareto_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    GUIDE_CUDA(launch_dependent(k_pareto_rank, num_sms(), SEL_THREADS, smem, st, header, (const P3 *)surv, front, idx_out, cap,
                                count_out));
    return GUIDE_OK;
}

int launch_pareto_fused(const DSpace &s, int time_model, int tp_model, const guide_constraints &c, int xm, int ym, u32 *header,
                        unsigned char *region, unsigned *ticket, u64 *idx_out, u32 cap, u32 *count_out, cudaStream_t st,
                        int phase) {
    return time_model ? pareto_fused_t<1>(s, tp_model, c, xm, ym, header, region, ticket, idx_out, cap, count_out, st, phase)
                      : pareto_fused_t<0>(s, tp_model, c, xm, ym, header, region, ticket, idx_out, cap, count_out, st, phase);
}

}  // namespace guide
