// What a kernel that has just evaluated a config needs in order to decide whether a selection can
// still want it: the sampled bound of a top-k call, the dominating points ("killers") of a Pareto
// call, and the lists the survivors go to.  Shared by the streaming selection kernels
// (select_stream.cu) and by the closed-form line kernel when it runs as the filter pass of a
// combined simulate-and-select call (closed_form.cu).
#pragma once
#include "select.cuh"

namespace guide {

static constexpr u32 TK_CAND_CAP = 16384;       // top-k survivors the workspace can hold
static constexpr u32 PA_KILLERS = 256;          // staircase points a Pareto sample hands to the filter pass
static constexpr u32 PA_SURV_CAP = 8192;        // Pareto survivors the workspace can hold

struct P2 { u64 x, y; };

// Bounds are (key, index) pairs in the same total order as the answer, so that a key shared by
// many configs (a metric with few distinct values) does not let them all through: of equal keys
// only the indices up to the bound's survive.
__device__ __forceinline__ bool pair_le(u64 key, u64 idx, u64 bkey, u64 bidx) {
    return key < bkey || (key == bkey && idx <= bidx);
}

// does b rule a out?  strictly better in one coordinate and not worse in the other
__device__ __forceinline__ bool dominates(u64 bx, u64 by, u64 ax, u64 ay) {
    return bx <= ax && by <= ay && (bx < ax || by < ay);
}

__device__ __forceinline__ void topk_keep(u64 key, u64 idx, u32 *header, KI *cand) {
    const u32 pos = atomicAdd(header + TK_COUNT, 1);
    if (pos < TK_CAND_CAP) { cand[pos].key = key; cand[pos].idx = idx; }
}

__device__ __forceinline__ void pareto_keep(u64 x, u64 y, u64 idx, u32 *header, P3 *surv) {
    const u32 pos = atomicAdd(header + PH_COUNT, 1);
    if (pos < PA_SURV_CAP) { surv[pos].x = x; surv[pos].y = y; surv[pos].idx = idx; }
}

struct KillerSet {
    const P2 *k;      // shared: sorted by x, y strictly falling
    u32 n;
    u64 rx[4], ry[4]; // four of them in registers
    // strictly dominated by a killer of the sorted list?  Only the killer with the largest x <= it.x can do it.
    __device__ __forceinline__ bool kills_sorted(u64 x, u64 y) const {
        u32 lo = 0, hi = n;                           // first killer with x > it.x
        while (lo < hi) {
            const u32 mid = (lo + hi) >> 1;
            if (k[mid].x <= x) lo = mid + 1; else hi = mid;
        }
        if (lo == 0) return false;
        const P2 p = k[lo - 1];
        return p.y < y || (p.y == y && p.x < x);
    }
    __device__ __forceinline__ bool kills(u64 x, u64 y) const {
        bool dead = false;
#pragma unroll
        for (int i = 0; i < 4; i++) dead |= dominates(rx[i], ry[i], x, y);
        return dead || kills_sorted(x, y);
    }
};

__device__ __forceinline__ bool meets(const Cons &c, double latency, double ttft, double thr, double cost_hr) {
    return ttft <= c.max_ttft && latency <= c.max_latency && cost_hr <= c.max_cost_hr && thr >= c.min_thr;
}

// Both selections of a combined call, as the line kernel sees them: constraints and metric choice,
// the workspace headers (bound pair, killer count, survivor counters) and the lists.
struct LineSelect {
    Cons ct; int key; u32 *header_t; KI *cand;
    Cons cp; int xm, ym; u32 *header_p; const P2 *killers; P3 *surv;
};

}  // namespace guide
