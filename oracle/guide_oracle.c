/*
 * CPU oracle for GUIDE's deployment-space evaluation (arXiv 2412.04788).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step restatement of what the
 * hot path computes, written from the paper; the library never calls it and it shares no code
 * with the CUDA path.  Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC guide_oracle.c -lm
 * All floating point is IEEE binary64, round-to-nearest-even, no contraction, and every sum is
 * taken in the order written here.
 *
 * What follows the paper directly:
 *   - memory model: Sec. 3.2 "Step 1" (available memory = GPU memory - model slice memory;
 *     max batch = available / KV per request) and Sec. 3.3.1 "Dynamic Batch Size Adjustment"
 *     (kv bytes per request = 2 N H S kv; B_max = floor(C_available / kv_per_request)).
 *   - task list of a prefill and a decode stage, each task with a compute load and a data
 *     size: Sec. 3.2 "Step 2", Sec. 3.4.1 "Task and GPU Models".
 *   - per-task time from the roofline: Sec. 3.4.2; the alternative literal sum of compute
 *     time and read/write time: Sec. 3.5.1 "Time Calculation"; the transfer term of
 *     Sec. 3.5.1 is the tensor-parallel all-reduce.
 *   - throughput 1/TPOT and the N*T_single/(1+log2 P_TP) scaling rule: Sec. 3.2 (throughput
 *     formulas); TTFT = prefill time: Sec. 3.2.
 *   - prefill-priority scheduling and fixed-granularity paged KV of the vLLM-like framework
 *     model: Sec. 2.3.2 "Inference Frameworks", Sec. 2.4.1, Sec. 2.4.2; iteration-level
 *     dynamic batching: Sec. 3.1 "Overview".
 *   - metrics TTFT / decode throughput / batch latency: Sec. 5.1 "Experimental Setup".
 *   - top-k selection by time or throughput under a budget: Sec. 3.2, Sec. 4.1.
 *
 * The paper prints no per-operator FLOP/byte counts; the task table below is first-principles
 * dense-decoder arithmetic (attention counted as the full query x context rectangle).
 *
 * Parity unpinned: absolute accuracy against real GPU runs (the paper's Tables 1-2) cannot be
 * checked here; everything else is pinned by the CPU tests (worked toy example, closed forms,
 * invariants, brute force).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef uint64_t u64;
typedef uint32_t u32;

/* The arithmetic type of the performance model: binary64, or binary32 when built with -DREAL=float
 * (the reduced-precision variant the library offers for the closed form; same operations, same
 * order, every value rounded to binary32; results are handed back widened to double). */
#ifndef REAL
#define REAL double
#endif
typedef REAL real;

enum { CLS_LINEAR = 0, CLS_ATTN = 1, CLS_ELEM = 2 };
enum { TIME_MAX = 0, TIME_SUM = 1 };
enum { TP_EXPLICIT = 0, TP_PAPER_LOG2 = 1 };
enum { ST_WEIGHTS = 1, ST_KV = 2, ST_HEADS = 4, ST_ITER = 8 };

/* flat views of the generator's arrays */
typedef struct {
    const u32 *models; u32 n_m;            /* [n_m][10]: N H n_h n_kv I V g w_b a_b kv_b */
    const double *hw; const u64 *hw_mem; u32 n_h;   /* [n_h][5]: P BW CBW CLAT PRICE */
    const double *fw_f; const u32 *fw_i; u32 n_f;   /* [n_f][8], [n_f][4] */
    const u32 *batch; u32 n_b;
    const u32 *tp; u32 n_t;
    const u32 *pairs; u32 n_l;             /* [n_l][2]: Lin Lout */
    const u32 *dp;                         /* [n_t] data-parallel degree of each entry of the parallelism axis; NULL = all 1 */
    const u32 *fw_chunk;                   /* [n_f][2]: split_size (requests per prompt sub-batch), seg_tokens (prompt
                                              segment length); 0 = no splitting; NULL = none anywhere */
    const u32 *fw_keep;                    /* [n_f]: thousandths of the KV cache that the framework's cache-eviction policy
                                              keeps (H2O, Sec. 3.2 Step 1 / Sec. 3.3); 0 or 1000 = everything; NULL = all 1000 */
} ospace;

typedef struct {
    const double *arrival; const u32 *in_len; const u32 *out_len; u64 n;
} otrace;

typedef struct {
    double *latency, *ttft, *ttft_p50, *ttft_p99, *tpot, *thr_decode, *cost_per_hr, *cost_per_token;
    uint8_t *status; u32 *bmax; u64 *n_iters, *n_req_iters;
    double *req_ttft, *req_tpot;           /* optional [count][n_req] */
    u64 *n_preempt;                        /* optional: preemptions per config (diagnostic) */
    u32 *seq_used;                         /* optional: tokens per request the metrics were computed for (Lin + Lout, less
                                              when the sequence was cut to fit, Sec. 3.3.2); 0 for configs that do not fit */
} oout;

enum { POLICY_PREFILL_FIRST = 0, POLICY_SPLIT_FUSE = 1 };
typedef struct { u64 N, H, nh, nkv, I, V, g, wb, ab, kvb, d, Dkv; } model_t;

typedef struct {
    real inv_c[3], inv_m[3], inv_comm, clat, tovh, price;
    int flash;
} rates_t;

static int g_overflow; /* set when a 64-bit product would wrap */
#pragma omp threadprivate(g_overflow)

static u64 mul(u64 a, u64 b) {
    unsigned __int128 p = (unsigned __int128)a * b;
    if (p >> 64) g_overflow = 1;
    return (u64)p;
}
static u64 add(u64 a, u64 b) {
    u64 s = a + b;
    if (s < a) g_overflow = 1;
    return s;
}
static u64 ceil_div(u64 a, u64 b) { return a / b + (a % b != 0); }

static model_t load_model(const u32 *r) {
    model_t m;
    m.N = r[0]; m.H = r[1]; m.nh = r[2]; m.nkv = r[3]; m.I = r[4]; m.V = r[5]; m.g = r[6];
    m.wb = r[7]; m.ab = r[8]; m.kvb = r[9];
    m.d = m.H / m.nh;
    m.Dkv = m.nkv * m.d;
    return m;
}

/* reciprocal rates of one (hardware, framework) pair: product first, then one reciprocal */
static rates_t load_rates(const double *hw, const double *ff, const u32 *fi) {
    rates_t r;
    for (int k = 0; k < 3; k++) {
        r.inv_c[k] = (real)1 / ((real)hw[0] * (real)ff[k]);
        r.inv_m[k] = (real)1 / ((real)hw[1] * (real)ff[3 + k]);
    }
    r.inv_comm = (real)1 / ((real)hw[2] * (real)ff[6]);
    r.clat = (real)hw[3];
    r.price = (real)hw[4];
    r.tovh = (real)ff[7];
    r.flash = (int)fi[0];
    return r;
}

/* ---- memory model (Sec. 3.2 Step 1, Sec. 3.3.1) -------------------------------------------- */

/* parameters: N (2H^2 + 2 H Dkv + (2+g) H I) + 2 V H  (attention + FFN + embedding + head) */
static u64 weight_params(const model_t *m) {
    u64 per_layer = add(add(mul(2, mul(m->H, m->H)), mul(2, mul(m->H, m->Dkv))),
                        mul(2 + m->g, mul(m->H, m->I)));
    return add(mul(m->N, per_layer), mul(2, mul(m->V, m->H)));
}
static u64 weight_bytes_per_gpu(const model_t *m, u64 t) { return ceil_div(mul(weight_params(m), m->wb), t); }
/* KV bytes of one token on one GPU: 2 N H kv with H -> Dkv for grouped-query attention, / t */
static u64 kv_bytes_per_token(const model_t *m, u64 t) { return mul(2, mul(m->N, mul(m->Dkv, m->kvb))) / t; }
static u64 usable_bytes(u64 mem, u64 reserve_permille) { return mem - (mem / 1000) * reserve_permille; }

/* ---- one task: compute load, data size -> time (Sec. 3.4.1, 3.4.2, 3.5.1) ------------------ */

static real task_time(u64 F_sh, u64 F_rp, u64 B_sh, u64 B_rp, real t, real inv_c, real inv_m,
                      int time_model) {
    real F = (real)F_sh / t + (real)F_rp;         /* sharded part splits over t GPUs */
    real B = (real)B_sh / t + (real)B_rp;
    real tc = F * inv_c;                          /* compute time = load / compute power */
    real tm = B * inv_m;                          /* read/write time = data / memory bandwidth */
    if (time_model == TIME_SUM) return tc + tm;   /* literal sum of Sec. 3.5.1 */
    return tc > tm ? tc : tm;                     /* roofline: the slower resource binds */
}

/*
 * Time of one phase (a prefill pass, one decode iteration, or an aggregated decode stage).
 *   T new tokens, E sequences emitting a token, A = sum q_i c_i, C = sum c_i, R repeats.
 * detail (optional, 16 doubles): t1..t8 with multiplicity, t9, t10, t11, S_comm, t13, S_fix,
 * S_att, T_phase.
 */
static real phase_time(const model_t *m, const rates_t *r, u64 tp, u64 T, u64 E, u64 A, u64 C, u64 R,
                       int time_model, int tp_model, double *detail) {
    u64 tt = (tp_model == TP_PAPER_LOG2) ? 1 : tp;   /* log2 rule: single-GPU formulas, scaled below */
    real t = (real)tt;
    const real *ic = r->inv_c, *im = r->inv_m;
    u64 H = m->H, I = m->I, Dkv = m->Dkv, V = m->V, ab = m->ab, wb = m->wb, kvb = m->kvb;
    u64 TH = mul(T, H), THa = mul(TH, ab), TI = mul(T, I), TIa = mul(TI, ab);
    u64 X = r->flash ? 0 : mul(mul(m->nh, A), ab);  /* score-matrix traffic, gone with FlashAttention */
    real tk[14];

    tk[1] = (real)2 * task_time(0, mul(4, TH), 0, mul(2, THa), t, ic[CLS_ELEM], im[CLS_ELEM], time_model);
    tk[2] = task_time(mul(2, mul(TH, H)), 0, add(mul(R, mul(mul(H, H), wb)), THa), THa, t,
                      ic[CLS_LINEAR], im[CLS_LINEAR], time_model);
    tk[3] = (real)2 * task_time(mul(2, mul(TH, Dkv)), 0,
                            add(mul(R, mul(mul(H, Dkv), wb)), mul(mul(T, Dkv), kvb)), THa, t,
                            ic[CLS_LINEAR], im[CLS_LINEAR], time_model);
    tk[4] = task_time(mul(2, mul(TH, H)), 0, add(mul(R, mul(mul(H, H), wb)), THa), THa, t,
                      ic[CLS_LINEAR], im[CLS_LINEAR], time_model);
    tk[5] = (real)2 * task_time(0, TH, 0, mul(3, THa), t, ic[CLS_ELEM], im[CLS_ELEM], time_model);
    tk[6] = (real)(1 + m->g) * task_time(mul(2, mul(TH, I)), 0, add(mul(R, mul(mul(H, I), wb)), TIa), THa, t,
                                           ic[CLS_LINEAR], im[CLS_LINEAR], time_model);
    tk[7] = task_time(mul(4, TI), 0, mul(2 + m->g, TIa), 0, t, ic[CLS_ELEM], im[CLS_ELEM], time_model);
    tk[8] = task_time(mul(2, mul(TI, H)), 0, add(mul(R, mul(mul(I, H), wb)), TIa), THa, t,
                      ic[CLS_LINEAR], im[CLS_LINEAR], time_model);
    u64 kv_read = mul(mul(C, Dkv), kvb);
    tk[9] = task_time(mul(2, mul(H, A)), 0, add(add(THa, kv_read), X), 0, t, ic[CLS_ATTN], im[CLS_ATTN], time_model);
    tk[10] = task_time(mul(5, mul(m->nh, A)), 0, mul(2, X), 0, t, ic[CLS_ATTN], im[CLS_ATTN], time_model);
    tk[11] = task_time(mul(2, mul(H, A)), 0, add(add(kv_read, THa), X), 0, t, ic[CLS_ATTN], im[CLS_ATTN], time_model);
    /* no sequence emits a token (a prompt segment that is not the last one): no LM head at all */
    tk[13] = E == 0 ? (real)0
                    : task_time(mul(2, mul(mul(E, H), V)), 0, add(mul(R, mul(mul(H, V), wb)), mul(mul(E, V), ab)),
                                mul(mul(E, H), ab), t, ic[CLS_LINEAR], im[CLS_LINEAR], time_model);

    real S_fix = tk[1];
    for (int k = 2; k <= 8; k++) S_fix = S_fix + tk[k];
    real S_att = tk[9] + tk[10];
    S_att = S_att + tk[11];

    /* ring all-reduce of the T x H activations, twice per layer; only when really sharded */
    real S_comm = 0;
    if (tt > 1) {
        u64 M = THa;
        real t12 = (real)mul(R, 2 * (tt - 1)) * r->clat + ((real)mul(2 * (tt - 1), M) / t) * r->inv_comm;
        S_comm = (real)2 * t12;
    }
    real T_layer = (S_fix + S_att) + S_comm;
    real T_phase = (real)R * r->tovh + ((real)m->N * T_layer + tk[13]);
    if (tp_model == TP_PAPER_LOG2) {
        /* throughput N T_single / (1 + log2 P_TP) with N = P_TP GPUs: time scales by (1+log2 t)/t */
        u64 lg = 0;
        while (((u64)1 << (lg + 1)) <= tp) lg++;
        T_phase = T_phase * ((real)(1 + lg) / (real)tp);
    }
    if (detail) {
        for (int k = 1; k <= 11; k++) detail[k - 1] = tk[k];
        detail[11] = S_comm; detail[12] = tk[13]; detail[13] = S_fix; detail[14] = S_att; detail[15] = T_phase;
    }
    return T_phase;
}

/* ---- index decoding: length pair fastest, model slowest ------------------------------------- */

typedef struct { u32 m, h, f, b, t, l; } pos_t;
static pos_t decode(const ospace *s, u64 idx) {
    pos_t p;
    p.l = (u32)(idx % s->n_l); idx /= s->n_l;
    p.t = (u32)(idx % s->n_t); idx /= s->n_t;
    p.b = (u32)(idx % s->n_b); idx /= s->n_b;
    p.f = (u32)(idx % s->n_f); idx /= s->n_f;
    p.h = (u32)(idx % s->n_h); idx /= s->n_h;
    p.m = (u32)idx;
    return p;
}

static void write_infeasible(const oout *o, u64 j) {
    o->latency[j] = INFINITY; o->ttft[j] = INFINITY; o->ttft_p50[j] = INFINITY; o->ttft_p99[j] = INFINITY;
    o->tpot[j] = INFINITY; o->thr_decode[j] = 0.0; o->cost_per_hr[j] = INFINITY; o->cost_per_token[j] = INFINITY;
    o->n_iters[j] = 0; o->n_req_iters[j] = 0;
}

/* ---- closed form: one prefill pass + an aggregated decode stage ----------------------------- */

/*
 * Prompt processing of one sub-batch of sb requests whose prompts are cut into segments of seg
 * tokens (Sec. 3.3.2: number of splits = ceil(Lin / split size), the last one short): one pass per
 * segment; its q tokens attend the done + q tokens of their own prompt seen so far, and only the
 * last segment emits a token.  Every pass reads the weights and pays the iteration overhead.
 */
static real segmented_prefill(const model_t *m, const rates_t *r, u64 t, u64 sb, u64 Lin, u64 seg,
                              int time_model, int tp_model) {
    real sum = 0;
    for (u64 done = 0; done < Lin; done += seg) {
        u64 q = Lin - done < seg ? Lin - done : seg;
        u64 T = mul(sb, q);
        u64 E = done + q == Lin ? sb : 0;
        sum = sum + phase_time(m, r, t, T, E, mul(T, done + q), mul(sb, done + q), 1, time_model, tp_model, NULL);
    }
    return sum;
}

/* Tokens of a cache of c tokens that stay when the eviction policy keeps p thousandths of it (H2O, named
 * in Sec. 3.2 Step 1 and Sec. 3.3 among the optimisations that shrink the KV cache; the paper gives
 * no rule, so: the kept share of the length, rounded up to a whole token). */
static u64 kept_tokens(u64 c, u64 p) { return p >= 1000 ? c : ceil_div(mul(p, c), 1000); }

static void closed_form_one(const ospace *s, u64 idx, u64 j, int time_model, int tp_model, int clamp_seq, const oout *o) {
    pos_t p = decode(s, idx);
    model_t m = load_model(s->models + 10 * p.m);
    rates_t r = load_rates(s->hw + 5 * p.h, s->fw_f + 8 * p.f, s->fw_i + 4 * p.f);
    u64 t = s->tp[p.t], b_all = s->batch[p.b], Lin = s->pairs[2 * p.l], Lout = s->pairs[2 * p.l + 1];
    u64 kv_block = s->fw_i[4 * p.f + 1], reserve = s->fw_i[4 * p.f + 2];
    u64 keep = s->fw_keep && s->fw_keep[p.f] ? s->fw_keep[p.f] : 1000;
    /* Hybrid parallelism (Sec. 3.5.2, Sec. 3.5.3): the batch is split over dp replicas of t GPUs each;
     * a stage lasts as long as its slowest replica, the one with ceil(b / dp) requests.  The memory
     * bound is per replica: Sec. 3.2 Step 1 obtains the largest batch by dividing the largest number of
     * requests in flight by the data-parallel degree. */
    u64 dp = s->dp ? s->dp[p.t] : 1;
    u64 b = ceil_div(b_all, dp);

    /* Step 1: what fits */
    u64 usable = usable_bytes(s->hw_mem[p.h], reserve);
    u64 W_gpu = weight_bytes_per_gpu(&m, t);
    u64 kv_tok = kv_bytes_per_token(&m, t);
    u64 S = Lin + Lout;
    if (clamp_seq && usable > W_gpu) {
        /* Dynamic sequence length adjustment (Sec. 3.3.2): S_max = floor(C_available / KV bytes of one
         * token of all B requests); a longer sequence is cut to it.  Whole blocks only; with a cache that
         * keeps p thousandths, the longest sequence whose kept part fits.  The prompt is what gets cut:
         * every output token is still generated. */
        u64 cap_tok = (usable - W_gpu) / mul(kv_tok, b);
        u64 cap_blk = (cap_tok / kv_block) * kv_block;
        u64 S_max = keep >= 1000 ? cap_blk : mul(1000, cap_blk) / keep;
        if (S > S_max && S_max > Lout) { Lin = S_max - Lout; S = S_max; }
    }
    u64 S_blk = mul(ceil_div(kept_tokens(S, keep), kv_block), kv_block);   /* fixed-granularity allocation of what is kept */
    u64 bmax = usable > W_gpu ? (usable - W_gpu) / mul(S_blk, kv_tok) : 0;
    uint8_t st = 0;
    if (usable <= W_gpu) st |= ST_WEIGHTS;
    if (b > bmax) st |= ST_KV;
    if (m.nh % t != 0 || m.nkv % t != 0) st |= ST_HEADS;
    o->status[j] = st;
    o->bmax[j] = bmax > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)bmax;
    if (o->seq_used) o->seq_used[j] = st ? 0 : (u32)S;
    if (st) { write_infeasible(o, j); return; }

    /* Step 2: the two stages.  Prompt processing (Sec. 3.3.1): the batch goes through in sub-batches
     * of split_size requests and what is left over goes through as one more, smaller sub-batch;
     * equal sub-batches take equal time.  Without splitting this is one pass over b x Lin tokens. */
    u64 split = s->fw_chunk ? s->fw_chunk[2 * p.f] : 0, seg = s->fw_chunk ? s->fw_chunk[2 * p.f + 1] : 0;
    if (split == 0 || split > b) split = b;
    if (seg == 0 || seg > Lin) seg = Lin;
    u64 n_full = b / split, rest = b % split, n_seg = ceil_div(Lin, seg);
    real T_pre = (real)n_full * segmented_prefill(&m, &r, t, split, Lin, seg, time_model, tp_model);
    if (rest) T_pre = T_pre + segmented_prefill(&m, &r, t, rest, Lin, seg, time_model, tp_model);
    u64 n = Lout - 1;                 /* the prefill pass emits token 1 */
    real T_dec = 0;
    if (n > 0) {
        u64 ctx = mul(b, add(mul(n, Lin), mul(n, n + 1) / 2));   /* step j attends Lin + j */
        ctx = kept_tokens(ctx, keep);                            /* ... of which the cache still holds this many: less work, less KV read */
        T_dec = phase_time(&m, &r, t, mul(b, n), mul(b, n), ctx, ctx, n, time_model, tp_model, NULL);
    }
    o->ttft[j] = T_pre; o->ttft_p50[j] = T_pre; o->ttft_p99[j] = T_pre;
    real lat = T_pre + T_dec;
    o->latency[j] = lat;
    real cost_hr = r.price * (real)mul(t, dp);               /* every GPU of every replica is paid for */
    o->cost_per_hr[j] = cost_hr;
    if (n > 0) {
        real tpot = T_dec / (real)n;
        real thr = (real)mul(b_all, n) / T_dec;               /* all replicas decode at once (Sec. 3.2: N x T_single) */
        real cost_tok = (cost_hr / (real)3600) / thr;
        o->tpot[j] = tpot; o->thr_decode[j] = thr; o->cost_per_token[j] = cost_tok;
    } else {
        o->tpot[j] = 0.0; o->thr_decode[j] = 0.0; o->cost_per_token[j] = INFINITY;
    }
    o->n_iters[j] = add(mul(n_full + (rest != 0), n_seg), n);   /* passes of one replica */
    o->n_req_iters[j] = mul(b_all, add(n_seg, n));
}

/* ---- trace-driven continuous batching with paged KV and preempt-and-recompute --------------- */

static int cmp_double(const void *a, const void *b) {
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

typedef struct {
    u32 *gen, *cache, *held, *running, *todo, *pdone;
    uint8_t *done, *needs_prefill, *has_first;
    double *first, *finish, *sorted;
} simbuf;

static void simbuf_alloc(simbuf *w, u64 n) {
    w->gen = malloc(n * sizeof(u32)); w->cache = malloc(n * sizeof(u32)); w->held = malloc(n * sizeof(u32));
    w->running = malloc(n * sizeof(u32)); w->todo = malloc(n * sizeof(u32)); w->pdone = malloc(n * sizeof(u32));
    w->done = malloc(n); w->needs_prefill = malloc(n); w->has_first = malloc(n);
    w->first = malloc(n * sizeof(double)); w->finish = malloc(n * sizeof(double)); w->sorted = malloc(n * sizeof(double));
}
static void simbuf_free(simbuf *w) {
    free(w->gen); free(w->cache); free(w->held); free(w->running); free(w->todo); free(w->pdone); free(w->done); free(w->needs_prefill);
    free(w->has_first); free(w->first); free(w->finish); free(w->sorted);
}

static void trace_sim_one(const ospace *s, const otrace *tr, u64 idx, u64 j, int time_model, int tp_model,
                          u64 max_iters_opt, const oout *o, simbuf *w) {
    pos_t p = decode(s, idx);
    model_t m = load_model(s->models + 10 * p.m);
    rates_t r = load_rates(s->hw + 5 * p.h, s->fw_f + 8 * p.f, s->fw_i + 4 * p.f);
    u64 t = s->tp[p.t], b = s->batch[p.b], Lin = s->pairs[2 * p.l], Lout = s->pairs[2 * p.l + 1];
    u64 blk = s->fw_i[4 * p.f + 1], reserve = s->fw_i[4 * p.f + 2];
    int fuse = s->fw_i[4 * p.f + 3] == POLICY_SPLIT_FUSE;
    u64 budget_tokens = fuse ? s->fw_chunk[2 * p.f + 1] : 0;   /* tokens per iteration (checked > 0 by the caller) */
    u64 n = tr->n;
#define IN(i)  ((u64)(tr->in_len[i] ? tr->in_len[i] : Lin))
#define OUT(i) ((u64)(tr->in_len[i] ? tr->out_len[i] : Lout))

    u64 usable = usable_bytes(s->hw_mem[p.h], reserve);
    u64 W_gpu = weight_bytes_per_gpu(&m, t);
    u64 kv_tok = kv_bytes_per_token(&m, t);
    u64 blocks_total = usable > W_gpu ? (usable - W_gpu) / mul(blk, kv_tok) : 0;
    u64 worst = 0, sum_out = 0;
    for (u64 i = 0; i < n; i++) {
        u64 need = ceil_div(IN(i) + OUT(i), blk);
        if (need > worst) worst = need;
        sum_out += OUT(i);
        if (fuse) sum_out += IN(i);      /* prompt chunks take iterations too: the backstop counts them */
    }
    u64 fit = worst ? blocks_total / worst : 0;      /* worst-case requests resident at once */
    uint8_t st = 0;
    if (usable <= W_gpu) st |= ST_WEIGHTS;
    if (worst > blocks_total) st |= ST_KV;           /* the largest single request cannot fit */
    if (m.nh % t != 0 || m.nkv % t != 0) st |= ST_HEADS;
    o->bmax[j] = fit > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)fit;
    double *rq_ttft = o->req_ttft ? o->req_ttft + j * n : NULL;
    double *rq_tpot = o->req_tpot ? o->req_tpot + j * n : NULL;
    if (o->n_preempt) o->n_preempt[j] = 0;
    if (st) goto infeasible;

    u64 max_iters = max_iters_opt ? max_iters_opt : 64 * sum_out + 4 * n;
    memset(w->gen, 0, n * sizeof(u32)); memset(w->cache, 0, n * sizeof(u32)); memset(w->held, 0, n * sizeof(u32));
    memset(w->done, 0, n); memset(w->needs_prefill, 0, n); memset(w->has_first, 0, n);
    u32 *run = w->running;
    u64 nrun = 0, next = 0, free_blocks = blocks_total;
    u64 n_iters = 0, n_req_iters = 0, dec_tok = 0, n_preempt = 0;
    double clock = 0.0, dec_time = 0.0;

    for (;;) {
        /* 1. admit in arrival order, no overtaking */
        for (;;) {
            while (next < n && w->done[next]) next++;
            if (!(next < n && tr->arrival[next] <= clock && nrun < b)) break;
            u64 need = ceil_div(IN(next) + w->gen[next], blk);   /* prompt + tokens to recompute */
            if (need > free_blocks) break;
            free_blocks -= need;
            w->held[next] = (u32)need;
            w->needs_prefill[next] = 1;
            w->todo[next] = (u32)(IN(next) + w->gen[next]);      /* split-fuse: prompt tokens still to process */
            w->pdone[next] = 0;
            run[nrun++] = (u32)next;
            next++;
        }
        /* 2. nothing to run: finished, or jump to the next arrival */
        if (nrun == 0) {
            if (next == n) break;
            if (tr->arrival[next] > clock) { clock = tr->arrival[next]; continue; }
            st |= ST_ITER; break;                     /* cannot happen when every request fits alone */
        }
        /* 3. build the iteration: prompts first, everything else stalls */
        if (n_iters >= max_iters) { st |= ST_ITER; break; }   /* backstop against a runaway schedule */
        double T_iter;
        u64 participants;
        if (fuse) {
            /*
             * Dynamic split and fuse (the FastGen-like framework model, Sec. 2.3.2 / Sec. 3.1): every
             * iteration carries about budget_tokens tokens.  Each resident past its prompt decodes one
             * token; what is left of the budget goes to prompts in arrival order, a long prompt
             * spread over several iterations, short ones sharing one.  A prompt chunk of q tokens
             * attends the pdone + q tokens of its request seen so far; the request emits its first
             * token in the iteration that finishes its prompt.
             */
            u64 needed = 0;
            for (u64 k = 0; k < nrun; k++) needed += (!w->needs_prefill[run[k]] && w->cache[run[k]] % blk == 0);
            while (needed > free_blocks) {            /* preempt the youngest, recompute later */
                u32 v = run[nrun - 1];
                free_blocks += w->held[v];
                if (!w->needs_prefill[v] && w->cache[v] % blk == 0) needed--;
                w->cache[v] = 0; w->held[v] = 0; w->needs_prefill[v] = 0;
                nrun--; next = v; n_preempt++;
            }
            free_blocks -= needed;
            u64 n_dec = 0, n_chunk = 0, T = 0, E = 0, A = 0, C = 0;
            for (u64 k = 0; k < nrun; k++) {
                u32 i = run[k];
                if (w->needs_prefill[i]) continue;
                if (w->cache[i] % blk == 0) w->held[i] += 1;
                u64 c = IN(i) + w->gen[i];
                n_dec++; A = add(A, c); C = add(C, c);
            }
            T = n_dec; E = n_dec;
            u64 left = budget_tokens > n_dec ? budget_tokens - n_dec : 0;
            double after;
            for (u64 k = 0; k < nrun && left > 0; k++) {          /* plan the chunks */
                u32 i = run[k];
                if (!w->needs_prefill[i]) continue;
                u64 q = w->todo[i] < left ? w->todo[i] : left;
                T = add(T, q); A = add(A, mul(q, w->pdone[i] + q)); C = add(C, w->pdone[i] + q);
                if (q == w->todo[i]) E++;
                left -= q; n_chunk++;
            }
            T_iter = phase_time(&m, &r, t, T, E, A, C, 1, time_model, tp_model, NULL);
            after = clock + T_iter;
            for (u64 k = 0; k < nrun; k++) {                      /* decodes advance */
                u32 i = run[k];
                if (!w->needs_prefill[i]) { w->cache[i] += 1; w->gen[i] += 1; }
            }
            left = budget_tokens > n_dec ? budget_tokens - n_dec : 0;
            for (u64 k = 0; k < nrun && left > 0; k++) {          /* the planned chunks are processed */
                u32 i = run[k];
                if (!w->needs_prefill[i] || w->todo[i] == 0) continue;
                u64 q = w->todo[i] < left ? w->todo[i] : left;
                w->pdone[i] += (u32)q; w->todo[i] -= (u32)q; left -= q;
                if (w->todo[i] == 0) {                            /* prompt finished: first token */
                    w->cache[i] = (u32)(IN(i) + w->gen[i]);
                    w->gen[i] += 1;
                    w->needs_prefill[i] = 0;
                    if (!w->has_first[i]) { w->has_first[i] = 1; w->first[i] = after; }
                }
            }
            if (n_dec > 0) { dec_time = dec_time + T_iter; dec_tok += n_dec; }
            participants = n_dec + n_chunk;
            goto advance;
        }
        u64 n_pre = 0;
        for (u64 k = 0; k < nrun; k++) n_pre += w->needs_prefill[run[k]];
        if (n_pre > 0) {
            u64 T = 0, A = 0;
            for (u64 k = 0; k < nrun; k++) {
                u32 i = run[k];
                if (!w->needs_prefill[i]) continue;
                u64 q = IN(i) + w->gen[i];
                T = add(T, q); A = add(A, mul(q, q));
            }
            T_iter = phase_time(&m, &r, t, T, n_pre, A, T, 1, time_model, tp_model, NULL);
            double after = clock + T_iter;
            for (u64 k = 0; k < nrun; k++) {
                u32 i = run[k];
                if (!w->needs_prefill[i]) continue;
                w->cache[i] = (u32)(IN(i) + w->gen[i]);
                w->gen[i] += 1;
                w->needs_prefill[i] = 0;
                if (!w->has_first[i]) { w->has_first[i] = 1; w->first[i] = after; }
            }
            participants = n_pre;
        } else {
            /* every sequence whose last block is full needs one more block */
            u64 needed = 0;
            for (u64 k = 0; k < nrun; k++) needed += (w->cache[run[k]] % blk == 0);
            while (needed > free_blocks) {            /* preempt the youngest, recompute later */
                u32 v = run[nrun - 1];
                free_blocks += w->held[v];
                if (w->cache[v] % blk == 0) needed--;
                w->cache[v] = 0; w->held[v] = 0;
                nrun--; next = v; n_preempt++;
            }
            free_blocks -= needed;
            u64 ctx = 0;
            for (u64 k = 0; k < nrun; k++) {
                u32 i = run[k];
                if (w->cache[i] % blk == 0) w->held[i] += 1;
                ctx = add(ctx, IN(i) + w->gen[i]);
            }
            T_iter = phase_time(&m, &r, t, nrun, nrun, ctx, ctx, 1, time_model, tp_model, NULL);
            for (u64 k = 0; k < nrun; k++) { u32 i = run[k]; w->cache[i] += 1; w->gen[i] += 1; }
            dec_time = dec_time + T_iter;
            dec_tok += nrun;
            participants = nrun;
        }
        /* 4. advance the clock */
advance:
        clock = clock + T_iter;
        n_iters++; n_req_iters += participants;
        /* 5. retire finished sequences, keep the rest in order */
        u64 keep = 0;
        for (u64 k = 0; k < nrun; k++) {
            u32 i = run[k];
            if (w->gen[i] == OUT(i)) {
                w->done[i] = 1; w->finish[i] = clock; free_blocks += w->held[i]; w->held[i] = 0;
            } else run[keep++] = i;
        }
        nrun = keep;
    }
    if (st) goto infeasible;

    o->status[j] = 0;
    o->latency[j] = clock;                            /* makespan of the whole trace */
    double s_ttft = 0.0, s_tpot = 0.0;
    for (u64 i = 0; i < n; i++) {
        double ttft = w->first[i] - tr->arrival[i];
        double tpot = OUT(i) > 1 ? (w->finish[i] - w->first[i]) / (double)(OUT(i) - 1) : 0.0;
        s_ttft = s_ttft + ttft; s_tpot = s_tpot + tpot;
        w->sorted[i] = ttft;
        if (rq_ttft) rq_ttft[i] = ttft;
        if (rq_tpot) rq_tpot[i] = tpot;
    }
    o->ttft[j] = s_ttft / (double)n;
    o->tpot[j] = s_tpot / (double)n;
    qsort(w->sorted, n, sizeof(double), cmp_double);
    o->ttft_p50[j] = w->sorted[(50 * n + 99) / 100 - 1];   /* nearest rank */
    o->ttft_p99[j] = w->sorted[(99 * n + 99) / 100 - 1];
    o->thr_decode[j] = dec_time > 0.0 ? (double)dec_tok / dec_time : 0.0;
    o->cost_per_hr[j] = r.price * (double)t;
    o->cost_per_token[j] = o->thr_decode[j] > 0.0 ? (o->cost_per_hr[j] / 3600.0) / o->thr_decode[j] : INFINITY;
    o->n_iters[j] = n_iters; o->n_req_iters[j] = n_req_iters;
    if (o->n_preempt) o->n_preempt[j] = n_preempt;
    if (o->seq_used) o->seq_used[j] = 0;                 /* closed form only */
    return;

infeasible:
    o->status[j] = st;
    write_infeasible(o, j);
    if (o->seq_used) o->seq_used[j] = 0;
    if (rq_ttft) for (u64 i = 0; i < n; i++) rq_ttft[i] = INFINITY;
    if (rq_tpot) for (u64 i = 0; i < n; i++) rq_tpot[i] = INFINITY;
#undef IN
#undef OUT
}

/* ---- exported entry points ------------------------------------------------------------------ */

/* Evaluate configs first, first+stride, ... (count of them); output slot j for the j-th.
 * trace == NULL: closed form.  Returns 0, or -2 when a 64-bit product overflowed. */
int oracle_simulate(const ospace *s, const otrace *tr, u64 first, u64 count, u64 stride,
                    int time_model, int tp_model, u64 max_iters, const oout *o, int threads, int clamp_seq) {
    int bad = 0;
    /* reject shapes the model is not defined for: zero sizes, KV bytes per token rounding to 0 */
    u64 t_max = 0;
    for (u32 i = 0; i < s->n_t; i++) { if (s->tp[i] == 0 || (s->tp[i] & (s->tp[i] - 1))) return -1; if (s->tp[i] > t_max) t_max = s->tp[i]; }
    for (u32 i = 0; i < s->n_m; i++) {
        const u32 *r = s->models + 10 * i;
        for (int c = 0; c < 10; c++) if (c != 6 && r[c] == 0) return -1;
        if (r[6] > 1 || r[1] % r[2] != 0) return -1;
        model_t m = load_model(r);
        if (2 * m.N * m.Dkv * m.kvb < t_max) return -1;
    }
    for (u32 i = 0; i < s->n_f; i++) if (s->fw_i[4 * i + 1] == 0 || s->fw_i[4 * i + 2] > 1000) return -1;
    for (u32 i = 0; i < s->n_b; i++) if (s->batch[i] == 0) return -1;
    if (s->dp) for (u32 i = 0; i < s->n_t; i++) {
        if (s->dp[i] == 0) return -1;
        if (tr && s->dp[i] != 1) return -3;      /* the trace simulation models one replica */
    }
    for (u32 i = 0; i < s->n_f; i++) {
        u32 policy = s->fw_i[4 * i + 3];
        u32 split = s->fw_chunk ? s->fw_chunk[2 * i] : 0, seg = s->fw_chunk ? s->fw_chunk[2 * i + 1] : 0;
        if (policy > POLICY_SPLIT_FUSE) return -1;
        if (!tr) continue;
        if (policy == POLICY_PREFILL_FIRST && (split || seg)) return -3;   /* prompt-first passes take whole prompts */
        if (policy == POLICY_SPLIT_FUSE && (seg == 0 || split != 0)) return -1;   /* needs its token budget, and only that */
    }
    for (u32 i = 0; i < s->n_l; i++) if (s->pairs[2 * i] == 0 || s->pairs[2 * i + 1] == 0) return -1;
    if (s->fw_keep) for (u32 i = 0; i < s->n_f; i++) {
        if (s->fw_keep[i] > 1000) return -1;
        if (tr && s->fw_keep[i] != 0 && s->fw_keep[i] != 1000) return -3;   /* cache eviction is modelled in the closed form only */
    }
    if (tr && clamp_seq) return -3;                                         /* a trace fixes the lengths of its requests */
    if (tr) for (u64 i = 0; i < tr->n; i++) {
        if (i && tr->arrival[i] < tr->arrival[i - 1]) return -1;
        if (tr->in_len[i] && !tr->out_len[i]) return -1;
    }
#ifdef _OPENMP
    if (threads > 0) omp_set_num_threads(threads);
#endif
#pragma omp parallel reduction(| : bad)
    {
        simbuf w;
        g_overflow = 0;
        if (tr) simbuf_alloc(&w, tr->n ? tr->n : 1);
#pragma omp for schedule(dynamic, 16)
        for (long long j = 0; j < (long long)count; j++) {
            u64 idx = first + (u64)j * stride;
            if (tr) trace_sim_one(s, tr, idx, (u64)j, time_model, tp_model, max_iters, o, &w);
            else closed_form_one(s, idx, (u64)j, time_model, tp_model, clamp_seq, o);
        }
        if (tr) simbuf_free(&w);
        bad |= g_overflow;
    }
    return bad ? -2 : 0;
}

int oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* pieces exposed so the pins can look inside */
u64 oracle_weight_params(const u32 *model) { model_t m = load_model(model); return weight_params(&m); }
u64 oracle_weight_bytes_per_gpu(const u32 *model, u64 t) { model_t m = load_model(model); return weight_bytes_per_gpu(&m, t); }
u64 oracle_kv_bytes_per_token(const u32 *model, u64 t) { model_t m = load_model(model); return kv_bytes_per_token(&m, t); }
u64 oracle_usable_bytes(u64 mem, u64 reserve_permille) { return usable_bytes(mem, reserve_permille); }

double oracle_phase_time(const u32 *model, const double *hw, const double *fw_f, const u32 *fw_i, u64 t,
                         u64 T, u64 E, u64 A, u64 C, u64 R, int time_model, int tp_model, double *detail16) {
    model_t m = load_model(model);
    rates_t r = load_rates(hw, fw_f, fw_i);
    return phase_time(&m, &r, t, T, E, A, C, R, time_model, tp_model, detail16);
}

/* ---- selection (Sec. 3.2: best configurations by time or throughput; Sec. 4.1: under budget) - */

typedef struct {
    double max_ttft; int ttft_stat;   /* 0 mean, 1 p50, 2 p99 */
    double max_latency, max_cost_per_hr, min_throughput;
} ocons;

typedef struct {
    const double *latency, *ttft, *ttft_p50, *ttft_p99, *tpot, *thr_decode, *cost_per_hr, *cost_per_token;
    const uint8_t *status;
} ometrics;

enum { K_LATENCY = 0, K_TTFT, K_TTFT_P99, K_TPOT, K_THROUGHPUT, K_COST_PER_HR, K_COST_PER_TOKEN };

static int passes(const ometrics *mt, const ocons *c, u64 i) {
    if (mt->status[i] != 0) return 0;
    double tt = c->ttft_stat == 0 ? mt->ttft[i] : c->ttft_stat == 1 ? mt->ttft_p50[i] : mt->ttft_p99[i];
    return tt <= c->max_ttft && mt->latency[i] <= c->max_latency && mt->cost_per_hr[i] <= c->max_cost_per_hr
           && mt->thr_decode[i] >= c->min_throughput;
}
static double metric_value(const ometrics *mt, int key, u64 i) {
    switch (key) {
    case K_LATENCY: return mt->latency[i];
    case K_TTFT: return mt->ttft[i];
    case K_TTFT_P99: return mt->ttft_p99[i];
    case K_TPOT: return mt->tpot[i];
    case K_THROUGHPUT: return mt->thr_decode[i];
    case K_COST_PER_HR: return mt->cost_per_hr[i];
    default: return mt->cost_per_token[i];
    }
}
/* smaller is better everywhere: throughput is compared negated */
static double ordered_value(const ometrics *mt, int key, u64 i) {
    double v = metric_value(mt, key, i);
    return key == K_THROUGHPUT ? 0.0 - v : v;
}

typedef struct { double x, y; u64 idx; } item_t;
static int cmp_item(const void *a, const void *b) {
    const item_t *p = a, *q = b;
    if (p->x != q->x) return p->x < q->x ? -1 : 1;
    if (p->y != q->y) return p->y < q->y ? -1 : 1;
    return (p->idx > q->idx) - (p->idx < q->idx);
}

/* k smallest passing configs under (key, index); metric arrays hold n entries, entry i is config
 * first + i.  Unused slots: index UINT64_MAX, key +inf.  Returns the number found. */
u32 oracle_select_topk(const ometrics *mt, u64 n, u64 first, const ocons *c, int key, u32 k,
                       u64 *idx_out, double *key_out) {
    item_t *it = malloc((n ? n : 1) * sizeof(item_t));
    u64 cnt = 0;
    for (u64 i = 0; i < n; i++)
        if (passes(mt, c, i)) { it[cnt].x = ordered_value(mt, key, i); it[cnt].y = 0.0; it[cnt].idx = first + i; cnt++; }
    qsort(it, cnt, sizeof(item_t), cmp_item);
    u32 found = cnt < k ? (u32)cnt : k;
    for (u32 r = 0; r < k; r++) {
        if (r < found) { idx_out[r] = it[r].idx; key_out[r] = metric_value(mt, key, it[r].idx - first); }
        else { idx_out[r] = UINT64_MAX; key_out[r] = INFINITY; }
    }
    free(it);
    return found;
}

/* Non-dominated passing configs (minimise both), duplicates of (x, y) keep the lowest index,
 * ascending x.  Writes at most cap indices, returns the size of the whole front. */
u32 oracle_pareto(const ometrics *mt, u64 n, u64 first, const ocons *c, int x_metric, int y_metric,
                  u64 *idx_out, u32 cap) {
    item_t *it = malloc((n ? n : 1) * sizeof(item_t));
    u64 cnt = 0;
    for (u64 i = 0; i < n; i++)
        if (passes(mt, c, i)) {
            it[cnt].x = ordered_value(mt, x_metric, i); it[cnt].y = ordered_value(mt, y_metric, i);
            it[cnt].idx = first + i; cnt++;
        }
    qsort(it, cnt, sizeof(item_t), cmp_item);
    u32 found = 0;
    double best_y = INFINITY;
    int any = 0;
    for (u64 r = 0; r < cnt; r++) {
        /* sorted by (x, y, idx): a point survives iff its y beats every earlier one */
        if (!any || it[r].y < best_y) {
            if (found < cap) idx_out[found] = it[r].idx;
            found++; best_y = it[r].y; any = 1;
        }
    }
    free(it);
    return found;
}
