// Constraint filter + global top-k + 2-D Pareto front (selection of Sec. 3.2 / Sec. 4.1).
//
// Both reductions are streaming: a block walks its share of the configs, drops on the spot
// whatever its current partial result already beats (a threshold for top-k, the block's current
// front for Pareto), appends the few survivors to a shared-memory buffer and, when that fills,
// sorts the buffer and rebuilds the partial result.  Block results go to the workspace; the block
// that finishes last streams them through the same routine to produce the global answer.
// Every comparison is on the total order (value, config index), so the answer does not depend on
// how configs are spread over blocks or in which order they are appended.
#include "guide_internal.cuh"

namespace guide {

static constexpr u32 SEL_THREADS = 256;
static constexpr u32 SEL_MAX_BLOCKS = 1024;
static constexpr u32 PARETO_CAP = 4096;          // shared-memory items per block
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

// ---- where the metrics come from --------------------------------------------------------------

// materialised arrays written by guide_simulate
struct MatSource {
    guide_outputs o;
    Cons c;
    int m0, m1;
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
    __device__ __forceinline__ bool get(u64 j, u64, double &a, double &b) const {
        if (__ldg(o.status + j)) return false;
        const double inf = __longlong_as_double(0x7FF0000000000000LL);
        if (c.max_ttft < inf) {
            const double *p = c.ttft_stat == GUIDE_STAT_MEAN ? o.ttft : c.ttft_stat == GUIDE_STAT_P50 ? o.ttft_p50 : o.ttft_p99;
            if (!(__ldg(p + j) <= c.max_ttft)) return false;
        }
        if (c.max_latency < inf && !(__ldg(o.latency + j) <= c.max_latency)) return false;
        if (c.max_cost_hr < inf && !(__ldg(o.cost_per_hr + j) <= c.max_cost_hr)) return false;
        if (c.min_thr > 0.0 && !(__ldg(o.thr_decode + j) >= c.min_thr)) return false;
        a = metric(m0, j);
        b = m1 >= 0 ? metric(m1, j) : 0.0;
        return true;
    }
};

// closed form evaluated on the fly: nothing is written to memory
template <int TIME_SUM>
struct FusedSource {
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

// ---- block-wide helpers ---------------------------------------------------------------------------

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

// ---- top-k accumulator -------------------------------------------------------------------------------

struct TopKAcc {
    KI *buf;          // shared, cap entries
    u32 *cnt;         // shared append cursor
    u32 cap, k;
    u32 c;            // mirror of *cnt, identical in every thread
    bool has_thr;
    KI thr;

    __device__ void init(KI *b, u32 *cn, u32 cap_, u32 k_) {
        buf = b; cnt = cn; cap = cap_; k = k_; c = 0; has_thr = false; thr.key = KEY_MAX; thr.idx = KEY_MAX;
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
    // collective: every thread of the block calls it once per tile
    __device__ void push(bool ok, KI it) {
        const bool take = ok && (!has_thr || ki_less(it, thr));
        if (take) buf[atomicAdd(cnt, 1)] = it;
        c += __syncthreads_count(take);        // same count in every thread
        if (c + blockDim.x > cap) compact();
    }
};

// ---- Pareto accumulator ----------------------------------------------------------------------------

struct ParetoAcc {
    P3 *buf;          // shared: [0, nf) current front sorted by x (y strictly falling), then appended survivors
    u32 *cnt;
    u32 *scratch;     // shared, 2 * 32 words
    u32 nf, c;
    bool overflow;

    __device__ void init(P3 *b, u32 *cn, u32 *sc) {
        buf = b; cnt = cn; scratch = sc; nf = 0; c = 0; overflow = false;
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
        nf = out; c = out;
        if (threadIdx.x == 0) *cnt = out;
        __syncthreads();
    }
    __device__ void push(bool ok, P3 it) {
        const bool take = ok && !beaten(it);
        if (take) buf[atomicAdd(cnt, 1)] = it;
        c += __syncthreads_count(take);
        if (c + blockDim.x > PARETO_CAP) merge();
    }
};

// ---- kernels ----------------------------------------------------------------------------------------

// workspace: [0] ticket, then per block k candidates
template <class Src>
__global__ void __launch_bounds__(SEL_THREADS) k_topk(Src src, Range r, u32 k, u32 cap, u32 *ticket, KI *partial,
                                                      int negate_out, u64 *idx_out, double *key_out, u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    KI *buf = (KI *)smem_raw;
    __shared__ u32 cnt;
    __shared__ u32 last_flag;
    TopKAcc acc;
    acc.init(buf, &cnt, cap, k);
    const u64 tiles = (r.count + blockDim.x - 1) / blockDim.x;
    for (u64 tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const u64 j = tile * blockDim.x + threadIdx.x;
        double a = 0.0, b;
        const bool ok = j < r.count && src.get(j, r.first + j, a, b);
        KI it;
        it.key = enc(a); it.idx = r.first + j;
        acc.push(ok, it);
    }
    acc.compact();
    KI *mine = partial + (size_t)blockIdx.x * k;
    for (u32 i = threadIdx.x; i < k; i += blockDim.x) {
        KI v; v.key = KEY_MAX; v.idx = KEY_MAX;
        if (i < acc.c) v = buf[i];
        mine[i] = v;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_flag = (atomicAdd(ticket, 1) == gridDim.x - 1);
    __syncthreads();
    if (!last_flag) return;
    __threadfence();
    // the last block folds every block's candidates
    acc.init(buf, &cnt, cap, k);
    const u64 total = (u64)gridDim.x * k;
    for (u64 base = 0; base < total; base += blockDim.x) {
        const u64 i = base + threadIdx.x;
        KI it; it.key = KEY_MAX; it.idx = KEY_MAX;
        if (i < total) {      // written by other blocks: read through L2
            const ulonglong2 v = __ldcg(reinterpret_cast<const ulonglong2 *>(partial) + i);
            it.key = v.x; it.idx = v.y;
        }
        acc.push(i < total && it.idx != KEY_MAX, it);
    }
    acc.compact();
    for (u32 i = threadIdx.x; i < k; i += blockDim.x) {
        if (i < acc.c) {
            const double v = dec(buf[i].key);
            idx_out[i] = buf[i].idx;
            key_out[i] = negate_out ? 0.0 - v : v;
        } else {
            idx_out[i] = KEY_MAX;
            key_out[i] = __longlong_as_double(0x7FF0000000000000LL);
        }
    }
    if (threadIdx.x == 0) *count_out = acc.c;
}

// workspace: ticket, per-block front sizes and overflow flags, per-block fronts
template <class Src>
__global__ void __launch_bounds__(SEL_THREADS) k_pareto(Src src, Range r, u32 *ticket, u32 *sizes, P3 *partial,
                                                        u64 *idx_out, u32 out_cap, u32 *count_out) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    P3 *buf = (P3 *)smem_raw;
    __shared__ u32 cnt;
    __shared__ u32 last_flag;
    __shared__ __align__(8) u32 scratch[64];
    ParetoAcc acc;
    acc.init(buf, &cnt, scratch);
    const u64 tiles = (r.count + blockDim.x - 1) / blockDim.x;
    for (u64 tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const u64 j = tile * blockDim.x + threadIdx.x;
        double a = 0.0, b = 0.0;
        const bool ok = j < r.count && src.get(j, r.first + j, a, b);
        P3 it;
        it.x = enc(a); it.y = enc(b); it.idx = r.first + j;
        acc.push(ok, it);
    }
    acc.merge();
    P3 *mine = partial + (size_t)blockIdx.x * GUIDE_PARETO_MAX;
    for (u32 i = threadIdx.x; i < acc.nf; i += blockDim.x) mine[i] = buf[i];
    if (threadIdx.x == 0) sizes[blockIdx.x] = acc.nf | (acc.overflow ? 0x80000000u : 0u);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last_flag = (atomicAdd(ticket, 1) == gridDim.x - 1);
    __syncthreads();
    if (!last_flag) return;
    __threadfence();
    acc.init(buf, &cnt, scratch);
    bool overflow = false;
    for (u32 blk = 0; blk < gridDim.x; blk++) {
        const u32 sz = __ldcg(sizes + blk);
        overflow |= (sz >> 31) != 0;
        const u32 n = sz & 0x7FFFFFFFu;
        const P3 *theirs = partial + (size_t)blk * GUIDE_PARETO_MAX;
        for (u32 base = 0; base < n; base += blockDim.x) {
            const u32 i = base + threadIdx.x;
            P3 it; it.x = KEY_MAX; it.y = KEY_MAX; it.idx = KEY_MAX;
            if (i < n) {      // written by other blocks: read through L2
                const u64 *w = reinterpret_cast<const u64 *>(theirs + i);
                it.x = __ldcg(w); it.y = __ldcg(w + 1); it.idx = __ldcg(w + 2);
            }
            acc.push(i < n, it);
        }
    }
    acc.merge();
    overflow |= acc.overflow;
    for (u32 i = threadIdx.x; i < acc.nf && i < out_cap; i += blockDim.x) idx_out[i] = buf[i].idx;
    if (threadIdx.x == 0) *count_out = overflow ? 0xFFFFFFFFu : acc.nf;
}

// ---- host side -----------------------------------------------------------------------------------------

static u32 topk_cap(u32 k) { return k <= 256 ? 512u : 2048u; }

size_t topk_workspace_bytes(u32 k) { return 256 + (size_t)SEL_MAX_BLOCKS * k * sizeof(KI); }
size_t pareto_workspace_bytes() {
    return 256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32) + (size_t)SEL_MAX_BLOCKS * GUIDE_PARETO_MAX * sizeof(P3);
}

static Cons make_cons(const guide_constraints &c) {
    Cons k;
    k.max_ttft = c.max_ttft; k.max_latency = c.max_latency; k.max_cost_hr = c.max_cost_per_hr;
    k.min_thr = c.min_throughput; k.ttft_stat = c.ttft_stat;
    return k;
}

static u32 grid_for(u64 count, u32 blocks_per_sm) {
    const u64 tiles = (count + SEL_THREADS - 1) / SEL_THREADS;
    u64 g = std::min<u64>((u64)num_sms() * blocks_per_sm, SEL_MAX_BLOCKS);
    g = std::min<u64>(g, std::max<u64>(tiles, 1));
    return (u32)g;
}

template <class Src>
static int run_topk(const Src &src, Range r, u32 k, int negate, u64 *idx_out, double *key_out, u32 *count_out,
                    void *ws, cudaStream_t st) {
    const u32 cap = topk_cap(k);
    const u32 grid = grid_for(r.count, 4);
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    k_topk<Src><<<grid, SEL_THREADS, cap * sizeof(KI), st>>>(src, r, k, cap, (u32 *)ws, (KI *)((char *)ws + 256), negate,
                                                             idx_out, key_out, count_out);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

template <class Src>
static int run_pareto(const Src &src, Range r, u64 *idx_out, u32 cap, u32 *count_out, void *ws, cudaStream_t st) {
    const size_t smem = (size_t)PARETO_CAP * sizeof(P3);
    static bool configured[64] = {};      // per kernel instantiation and device
    int dev = 0;
    GUIDE_CUDA(cudaGetDevice(&dev));
    if (dev >= 64 || !configured[dev]) {
        GUIDE_CUDA(cudaFuncSetAttribute(k_pareto<Src>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        if (dev < 64) configured[dev] = true;
    }
    const u32 grid = grid_for(r.count, 2);
    GUIDE_CUDA(cudaMemsetAsync(ws, 0, 256, st));
    u32 *sizes = (u32 *)((char *)ws + 256);
    P3 *partial = (P3 *)((char *)ws + 256 + (size_t)SEL_MAX_BLOCKS * sizeof(u32));
    k_pareto<Src><<<grid, SEL_THREADS, smem, st>>>(src, r, (u32 *)ws, sizes, partial, idx_out, cap, count_out);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

int launch_topk(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                const guide_constraints &c, int key, u32 k, u64 *idx_out, double *key_out, u32 *count_out,
                void *ws, cudaStream_t st) {
    const int negate = key == GUIDE_THROUGHPUT;
    if (mat) {
        MatSource src{*mat, make_cons(c), key, -1};
        return run_topk(src, r, k, negate, idx_out, key_out, count_out, ws, st);
    }
    if (time_model) {
        FusedSource<1> src{s, make_cons(c), key, -1, tp_model};
        return run_topk(src, r, k, negate, idx_out, key_out, count_out, ws, st);
    }
    FusedSource<0> src{s, make_cons(c), key, -1, tp_model};
    return run_topk(src, r, k, negate, idx_out, key_out, count_out, ws, st);
}

int launch_pareto(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                  const guide_constraints &c, int xm, int ym, u64 *idx_out, u32 cap, u32 *count_out, void *ws,
                  cudaStream_t st) {
    if (mat) {
        MatSource src{*mat, make_cons(c), xm, ym};
        return run_pareto(src, r, idx_out, cap, count_out, ws, st);
    }
    if (time_model) {
        FusedSource<1> src{s, make_cons(c), xm, ym, tp_model};
        return run_pareto(src, r, idx_out, cap, count_out, ws, st);
    }
    FusedSource<0> src{s, make_cons(c), xm, ym, tp_model};
    return run_pareto(src, r, idx_out, cap, count_out, ws, st);
}

// ---- top-k over materialised metrics with library-owned scratch ----------------------------------
//
// Same kernel as launch_topk, but the per-block partial results live in a fixed device array that
// is part of the library image instead of a caller-supplied workspace, for callers that are not
// allowed to allocate device memory.  The array bounds k and the grid; every call reuses it.

static constexpr u32 NOALLOC_BLOCKS = 256;                     // grid cap of this variant
static constexpr size_t NOALLOC_SCRATCH_BYTES = 256 + (size_t)NOALLOC_BLOCKS * GUIDE_NOALLOC_TOPK_MAX * sizeof(KI);

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
    MatSource src{mat, make_cons(c), key, -1};
    const u32 cap = topk_cap(k);
    const u32 grid = std::min<u32>(grid_for(r.count, 4), NOALLOC_BLOCKS);
    // the array still holds the previous call's ticket and candidates: the ticket must restart at 0,
    // the candidate slots are all rewritten by the blocks of this launch before they are read
    GUIDE_CUDA(cudaMemsetAsync(scratch, 0, 256, st));
    k_topk<MatSource><<<grid, SEL_THREADS, cap * sizeof(KI), st>>>(src, r, k, cap, (u32 *)scratch, (KI *)(scratch + 256),
                                                                   key == GUIDE_THROUGHPUT, idx_out, key_out, count_out);
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

}  // namespace guide
