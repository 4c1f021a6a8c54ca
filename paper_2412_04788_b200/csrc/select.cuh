// Shared by the selection kernels (select.cu: accumulator-based scans and the fused kernels;
// select_stream.cu: the sampled-bound streaming path over materialised metrics).
#pragma once
#include "guide_internal.cuh"

namespace guide {

static constexpr u32 SEL_THREADS = 256;
static constexpr u32 SEL_MAX_BLOCKS = 1024;
static constexpr u64 KEY_MAX = ~0ull;

// order-preserving map double -> u64 (after -0.0 -> +0.0)
__device__ __forceinline__ u64 enc(double v) {
    const u64 b = (u64)__double_as_longlong(v + 0.0);
    return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ __forceinline__ double dec(u64 k) {
    const u64 b = (k >> 63) ? (k ^ 0x8000000000000000ull) : ~k;
    return __longlong_as_double((long long)b);
}

struct Cons {
    double max_ttft, max_latency, max_cost_hr, min_thr;
    int ttft_stat;
};

__device__ __forceinline__ double pick_metric(int key, double latency, double ttft, double ttft_p99, double tpot,
                                              double thr, double cost_hr, double cost_tok) {
    switch (key) {
    case GUIDE_LATENCY: return latency;
    case GUIDE_TTFT: return ttft;
    case GUIDE_TTFT_P99: return ttft_p99;
    case GUIDE_TPOT: return tpot;
    case GUIDE_THROUGHPUT: return 0.0 - thr;      // larger is better
    case GUIDE_COST_PER_HR: return cost_hr;
    default: return cost_tok;
    }
}

// constraint filter and metric choice on freshly evaluated closed-form metrics
__device__ __forceinline__ bool fused_pick(const Metrics &m, const Cons &c, int m0, int m1, double &a, double &b) {
    if (m.status) return false;
    if (!(m.ttft <= c.max_ttft) || !(m.latency <= c.max_latency) || !(m.cost_hr <= c.max_cost_hr) || !(m.thr >= c.min_thr))
        return false;
    a = pick_metric(m0, m.latency, m.ttft, m.ttft, m.tpot, m.thr, m.cost_hr, m.cost_tok);
    b = m1 >= 0 ? pick_metric(m1, m.latency, m.ttft, m.ttft, m.tpot, m.thr, m.cost_hr, m.cost_tok) : 0.0;
    return true;
}

inline Cons make_cons(const guide_constraints &c) {
    Cons k;
    k.max_ttft = c.max_ttft; k.max_latency = c.max_latency; k.max_cost_hr = c.max_cost_per_hr;
    k.min_thr = c.min_throughput; k.ttft_stat = c.ttft_stat;
    return k;
}

inline const double *metric_array_of(const guide_outputs &o, int key) {
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

// Are all metric arrays aligned for 16-byte loads (status: 4-byte)?
inline int mat_vec_ok(const guide_outputs &o) {
    auto al = [](const void *p, uintptr_t a) { return ((uintptr_t)p % a) == 0; };
    const double *arrs[] = {o.latency, o.ttft, o.ttft_p50, o.ttft_p99, o.tpot, o.thr_decode, o.cost_per_hr, o.cost_per_token};
    for (const double *p : arrs)
        if (p && !al(p, 16)) return 0;
    return al(o.status, 4) ? 1 : 0;
}

struct KI { u64 key, idx; };
__device__ __forceinline__ bool ki_less(const KI &a, const KI &b) {
    return a.key < b.key || (a.key == b.key && a.idx < b.idx);
}
struct P3 { u64 x, y, idx; };
__device__ __forceinline__ bool p3_less(const P3 &a, const P3 &b) {
    if (a.x != b.x) return a.x < b.x;
    if (a.y != b.y) return a.y < b.y;
    return a.idx < b.idx;
}

__device__ __forceinline__ u32 next_pow2(u32 v) { return v <= 1 ? 1 : 1u << (32 - __clz(v - 1)); }

// in-place ascending bitonic sort of buf[0..P), P a power of two; ends with a barrier
template <class T, class Less>
__device__ void block_bitonic_sort(T *buf, u32 P, Less less) {
    for (u32 size = 2; size <= P; size <<= 1) {
        for (u32 stride = size >> 1; stride > 0; stride >>= 1) {
            for (u32 i = threadIdx.x; i < (P >> 1); i += blockDim.x) {
                const u32 lo = ((i & ~(stride - 1)) << 1) | (i & (stride - 1));
                const u32 hi = lo + stride;
                const bool up = (lo & size) == 0;
                const T a = buf[lo], b = buf[hi];
                if (less(b, a) == up) { buf[lo] = b; buf[hi] = a; }
            }
            __syncthreads();
        }
    }
}

// ---- programmatic dependent launch ---------------------------------------------------------------
// The kernels of one selection call form a chain of short launches.  A kernel launched with
// launch_dependent() may start (and sit in grid_dep_wait()) while its predecessor in the stream is
// still running, which hides its launch latency; it must call grid_dep_wait() before touching
// anything the predecessor writes.  grid_dep_wait() returns only when the predecessor grid has
// completed and its writes are visible, and is a no-op in a kernel launched the ordinary way.
// grid_dep_launch() in the predecessor lets the dependent start early; without it the dependent
// starts when the predecessor's blocks have exited.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <class... KArgs, class... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- workspace headers (first 256 bytes of a selection workspace, zeroed at the start of a call) ----
// top-k:  u64 at word 0: complement of the grid-wide key bound of the per-warp accumulators (0 = none);
//         words 2..: the streaming path's tickets, candidate and sample counts, redo flag and (two u64 at word 6) its bound pair.
// Pareto: word 0 ticket of the per-warp kernel, word 1 redo flag, word 2 ticket of the general kernel;
//         words 4..: the streaming path's tickets, survivor count, killer count and front count.
enum { TK_TICKET = 2, TK_COUNT = 3, TK_REDO = 4, TK_SAMPLED = 5, TK_BOUND = 6, TK_TICKET2 = 10 };
enum { PH_TICKET = 4, PH_COUNT = 5, PH_KILLERS = 6, PH_FRONT = 7, PH_TICKET2 = 8 };

// ---- streaming path (select_stream.cu) -----------------------------------------------------------
// Materialised metrics only.  A strided sample gives a bound (top-k) or a small set of dominating
// points (Pareto); one pass at memory speed then keeps the few configs the bound cannot exclude and
// a last small kernel finishes exactly.  When the survivors do not fit the workspace the redo flag
// goes up and the accumulator-based kernels, queued behind and gated on that flag, redo the call.
static constexpr u64 STREAM_MIN_COUNT = 1ull << 18;      // below this the accumulator kernels are as fast
static constexpr u32 STREAM_TOPK_MAX_K = 128;
size_t topk_stream_bytes();
size_t pareto_stream_bytes();
bool stream_eligible(const guide_outputs &mat, Range r);
// Both leave *redo_flag pointing at the device word the fallback kernels must be gated on.
int launch_topk_stream(Range r, const guide_outputs &mat, const guide_constraints &c, int key, u32 k, u32 *header,
                       unsigned char *region, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st);
int launch_pareto_stream(Range r, const guide_outputs &mat, const guide_constraints &c, int xm, int ym, u32 *header,
                         unsigned char *region, u64 *idx_out, u32 cap, u32 *count_out, cudaStream_t st);


// Fused form (nothing materialised, whole closed-form spaces): the sample rows are evaluated into a
// compact scratch in the workspace, the same bound / killer kernels run on that, and the filter pass
// is the model walk of model_walk.cuh with a sink that keeps candidates instead of storing metrics.
// phase: the whole call, or a part of it around a filter pass that somebody else runs (the line
// kernel of a combined simulate-and-select call): up to the bound / the killers (FUSED_BOUND; or in
// two steps: the sample rows, possibly beside the stream's previous kernel when that is the other
// selection's sample, then the bound kernels alone), or the ranking of what that pass left in the
// lists (fused_lists() tells it where they are).
enum { FUSED_ALL = 0, FUSED_BOUND = 1, FUSED_RANK = 2, FUSED_SAMPLE = 3, FUSED_SAMPLE_BESIDE = 4, FUSED_BOUND_ONLY = 5 };
bool fused_stream_eligible(const DSpace &s, Range r);
int launch_topk_fused(const DSpace &s, int time_model, int tp_model, const guide_constraints &c, int key, u32 k, u32 *header,
                      unsigned char *region, unsigned *ticket, u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st,
                      int phase = FUSED_ALL);
int launch_pareto_fused(const DSpace &s, int time_model, int tp_model, const guide_constraints &c, int xm, int ym, u32 *header,
                        unsigned char *region, unsigned *ticket, u64 *idx_out, u32 cap, u32 *count_out, cudaStream_t st,
                        int phase = FUSED_ALL);
struct LineSelect;
void fused_lists(unsigned char *topk_region, unsigned char *pareto_region, LineSelect *sel);

}  // namespace guide
