/*
 * guide.h - C ABI of the B200 deployment-space evaluator for GUIDE (arXiv 2412.04788).
 *
 * The library evaluates the paper's performance model over a space of candidate deployments
 * (model shape x hardware profile x framework profile x batch size x modelled tensor-parallel
 * degree x input/output length), in closed form or by simulating iteration-level continuous
 * batching over a request trace, and reduces the results to a top-k and a 2-D Pareto front.
 * Every step runs in CUDA kernels for sm_100a; there is no CPU fallback.
 *
 * Conventions
 *   - Every function returns GUIDE_OK (0) or a negative guide_status; nothing aborts or throws.
 *     guide_last_error() gives a thread-local message for the last failure on this thread.
 *   - "host" / "device" in a parameter comment says where the pointer must point.
 *   - Handles (guide_space, guide_trace) are owned by the library and freed by their destroy
 *     call.  On first use on a device a handle allocates its own small device tables (under 1 MB:
 *     the axis tables, a rate table per hardware x framework pair, the trace); every large
 *     buffer (outputs, workspace) is caller-owned device memory.
 *   - Kernel launches are asynchronous on the given CUDA stream (a cudaStream_t passed as
 *     void*; NULL is the default stream).  Results are valid once that stream has been
 *     synchronised.  The one exception is the first use of a handle on a device, which uploads
 *     its tables on the given stream and waits for that stream (no other stream is touched).
 *   - A config index enumerates the axes in mixed radix, length pair fastest, model slowest:
 *       idx = ((((m*n_hw + h)*n_fw + f)*n_batch + b)*n_tp + t)*n_pairs + l
 *   - All floating point is IEEE binary64, round to nearest even, no fused multiply-add, in a
 *     fixed operation order, so results do not depend on launch shape.
 */
#ifndef GUIDE_H
#define GUIDE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum guide_status {
    GUIDE_OK = 0,
    GUIDE_ERR_INVALID = -1,      /* NULL where a pointer is required, zero-length axis, bad value */
    GUIDE_ERR_OVERFLOW = -2,     /* an axis maximum could wrap a 64-bit FLOP or byte count */
    GUIDE_ERR_UNSUPPORTED = -3,  /* valid request outside what the kernels implement */
    GUIDE_ERR_CUDA = -4,         /* a CUDA call failed; guide_last_error() carries its message */
    GUIDE_ERR_WORKSPACE = -5,    /* workspace NULL, misaligned (256 B) or smaller than required */
    GUIDE_ERR_ITER_LIMIT = -6    /* reserved: per-config overruns are reported in status bit 3 */
} guide_status;

/* ---- axis entries ------------------------------------------------------------------------- */

/* A dense decoder: the quantities the memory equations of Sec. 3.3.1 (N layers, hidden size H,
 * bytes per KV element) and the per-layer task list of Sec. 3.2 Step 2 need. */
typedef struct guide_model {
    uint32_t n_layers, hidden, n_heads, n_kv_heads, ffn, vocab;
    uint32_t gated;                       /* 1: gate+up+down FFN, 0: up+down */
    uint32_t w_bytes, a_bytes, kv_bytes;  /* bytes per weight / activation / KV element */
} guide_model;

/* The GPU model of Sec. 3.4.1: compute performance, memory bandwidth, communication
 * bandwidth and latency; plus capacity (Sec. 3.2 Step 1) and price (budget, Sec. 4.1). */
typedef struct guide_hw {
    double peak_flops;      /* FLOP/s */
    double mem_bw;          /* B/s */
    double comm_bw;         /* B/s, interconnect used by tensor parallelism */
    double comm_lat;        /* s per hop */
    double price_per_hr;    /* $ per GPU-hour */
    uint64_t mem_bytes;     /* device memory */
} guide_hw;

/* An inference-framework profile (Sec. 3.1: the framework's influence is abstracted):
 * achieved fractions of peak per task class, scheduling overhead, KV paging granularity. */
typedef struct guide_fw {
    double e_c[3];          /* compute efficiency for LINEAR, ATTENTION, ELEMENTWISE tasks */
    double e_m[3];          /* memory-bandwidth efficiency, same classes */
    double e_comm;          /* interconnect efficiency */
    double t_ovh;           /* s added per iteration */
    uint32_t flash;         /* 1: FlashAttention (no score-matrix traffic), Sec. 3.2 Step 1 */
    uint32_t kv_block;      /* tokens per KV block (fixed-granularity paging, Sec. 2.4.1); 1 = unpaged */
    uint32_t reserve_permille; /* thousandths of device memory kept back */
    uint32_t policy;        /* GUIDE_POLICY_*: how the trace simulation composes an iteration */
    /* Prompt processing in pieces (closed form; with a trace: GUIDE_ERR_UNSUPPORTED under the prompt-first
     * policy, and seg_tokens is the per-iteration token budget under GUIDE_POLICY_SPLIT_FUSE):
     * split_size: requests per prompt sub-batch (Sec. 3.3.1: the batch is divided into sub-batches of
     *   split_size, the remainder forming one more); 0 or >= the batch = the whole batch at once.
     * seg_tokens: tokens per prompt segment (Sec. 3.3.2: ceil(Lin / segment) splits, base value times
     *   tuning factor supplied as one number); 0 or >= Lin = the whole prompt at once.
     * Every (sub-batch, segment) pass reads the weights and pays t_ovh; a segment's tokens attend
     * their prompt up to the end of that segment; only the last segment runs the LM head.  TTFT is
     * the time of all passes, n_iters counts them, n_req_iters = batch x (segments + Lout - 1). */
    uint32_t split_size;
    uint32_t seg_tokens;
    /* KV-cache eviction (H2O; Sec. 3.2 Step 1 and Sec. 3.3 name it among the optimisations that shrink
     * the cache, without a rule): thousandths of a request's cache that the policy keeps; a cache of c
     * tokens holds ceil(kv_keep_permille * c / 1000).  Used by the memory check (per request, then whole
     * blocks) and by the decode stage (attention work and KV read of the stage total); the prompt pass
     * attends its prompt in full.  0 or 1000 = nothing is evicted.  Closed form only: with a trace,
     * any other value gives GUIDE_ERR_UNSUPPORTED. */
    uint32_t kv_keep_permille;
    uint32_t reserved;
} guide_fw;

typedef struct guide_len_pair { uint32_t lin, lout; } guide_len_pair;

enum { GUIDE_POLICY_PREFILL_FIRST = 0,  /* an iteration is either all waiting prompts, whole, or one decode step (Sec. 2.4.2) */
       /* Dynamic split and fuse (the FastGen-like framework model, Sec. 2.3.2 / Sec. 3.1): every iteration
        * carries seg_tokens tokens, one per request past its prompt, the rest prompt tokens in arrival
        * order (long prompts spread over iterations, short ones sharing one).  Trace simulation only;
        * needs seg_tokens >= 1 and split_size == 0 there.  The closed form ignores the policy. */
       GUIDE_POLICY_SPLIT_FUSE = 1 };

/* The candidate space of Sec. 3.1.  All pointers: host; copied by guide_space_create. */
typedef struct guide_space_desc {
    const guide_model *models;   uint32_t n_models;   /* <= 4096 */
    const guide_hw *hw;          uint32_t n_hw;       /* n_hw * n_fw <= 65536 */
    const guide_fw *fw;          uint32_t n_fw;
    const uint32_t *batch;       uint32_t n_batch;    /* batch size (closed form) / max batch (trace) */
    const uint32_t *tp;          uint32_t n_tp;       /* modelled tensor-parallel degree, powers of two */
    const guide_len_pair *pairs; uint32_t n_pairs;    /* (input length, output length) */
    /* Hybrid parallelism (Sec. 3.5.2, Sec. 3.5.3): dp[i] is the data-parallel degree that goes with
     * tp[i], so entry i of the parallelism axis is the pair (dp[i], tp[i]) on dp[i] * tp[i] GPUs;
     * enumerating the pairs under a GPU budget is the caller's get_configurations step.  The batch is
     * split over the dp replicas and a stage lasts as long as the replica with ceil(batch / dp)
     * requests; B_max and the memory check are per replica (Sec. 3.2 Step 1), throughput counts all
     * replicas, the hourly cost all dp * tp GPUs.  NULL = every dp is 1.  Closed form only: with any
     * dp > 1, guide_simulate on a trace returns GUIDE_ERR_UNSUPPORTED. */
    const uint32_t *dp;
} guide_space_desc;

typedef struct guide_config {
    uint32_t model, hw, fw, batch_pos, tp_pos, pair_pos;   /* axis positions */
    uint32_t batch, tp, lin, lout;                         /* axis values */
    uint32_t dp;                                           /* data-parallel degree of the tp_pos entry */
} guide_config;

typedef struct guide_space guide_space;
typedef struct guide_trace guide_trace;

/* ---- evaluation options, outputs, constraints --------------------------------------------- */

enum { GUIDE_TIME_MAX = 0,        /* per-task roofline: the slower of compute and memory (Sec. 3.4.2) */
       GUIDE_TIME_SUM = 1 };      /* literal sum of compute time and read/write time (Sec. 3.5.1) */
enum { GUIDE_PREC_F64 = 0, GUIDE_PREC_F32 = 1 };
enum { GUIDE_TP_EXPLICIT = 0,     /* sharded work / t plus a ring all-reduce transfer term (Sec. 3.5.1) */
       GUIDE_TP_PAPER_LOG2 = 1 }; /* single-GPU time x (1 + log2 t) / t (throughput rule of Sec. 3.2) */

typedef struct guide_sim_opts {
    uint64_t first;       /* first config index */
    uint64_t count;       /* number of consecutive configs; 0 = through the end of the space */
    int32_t time_model;   /* GUIDE_TIME_* */
    int32_t tp_model;     /* GUIDE_TP_* */
    uint64_t max_iters;   /* trace simulation: iteration cap per config; 0 = 64*sum(out_len) + 4*n_req */
    /* Dynamic sequence length adjustment (Sec. 3.3.2), closed form only (with a trace:
     * GUIDE_ERR_UNSUPPORTED).  1: a config whose sequence Lin + Lout is longer than
     * S_max = floor(C_available / (KV bytes per token x B)) - in whole KV blocks, and with cache
     * eviction the longest sequence whose kept part fits - is evaluated with its prompt cut so that
     * Lin + Lout = S_max, provided at least one prompt token remains; bmax is then that of the length
     * used.  outputs->seq_used tells which configs were cut.  0 (default): every config is judged
     * with its own lengths. */
    int32_t clamp_seq;
    /* GUIDE_PREC_F64 (default): every operation of the model in binary64.  GUIDE_PREC_F32: the closed
     * form with every operation in binary32 - each integer FLOP / byte count rounded once, then the
     * same operations in the same order; results are written to the same double arrays, widened (so a
     * materialised selection works on them unchanged) and agree with the binary64 results to 1e-5
     * relative; status, bmax and the counters are identical.  guide_simulate without a trace only:
     * GUIDE_ERR_UNSUPPORTED with a trace (a clock summed over 10^5 iterations in binary32 flips
     * admission decisions) and for the fused selection. */
    int32_t precision;
} guide_sim_opts;

/* status bits */
enum { GUIDE_ST_WEIGHTS = 1,   /* the weight slice does not leave any usable memory */
       GUIDE_ST_KV = 2,        /* closed form: batch x KV per request exceeds capacity (Sec. 3.3.1);
                                  trace: the largest single request cannot fit */
       GUIDE_ST_HEADS = 4,     /* TP degree does not divide the head counts */
       GUIDE_ST_ITER = 8 };    /* trace simulation hit max_iters */

/* Struct of caller-owned DEVICE arrays, entry j for config first + j; any pointer may be NULL
 * (that output is skipped).  Infeasible configs (status != 0) get +inf times and costs and 0
 * throughput. */
typedef struct guide_outputs {
    double *latency;         /* closed form: prefill + decode time of the batch; trace: makespan */
    double *ttft;            /* closed form: prefill time (Sec. 3.2); trace: mean over requests */
    double *ttft_p50;        /* nearest-rank percentiles over requests (closed form: = ttft) */
    double *ttft_p99;
    double *tpot;            /* time per output token after the first */
    double *thr_decode;      /* decode tokens per second (Sec. 5.1) */
    double *cost_per_hr;     /* price x TP degree */
    double *cost_per_token;  /* (cost_per_hr / 3600) / thr_decode */
    uint8_t *status;         /* GUIDE_ST_* bits, 0 = feasible */
    uint32_t *bmax;          /* closed form: B_max of Sec. 3.3.1; trace: worst-case requests resident at once */
    uint64_t *n_iters;       /* iterations simulated (closed form: 1 + decode steps) */
    uint64_t *n_req_iters;   /* sum over iterations of participating requests */
    double *req_ttft;        /* trace only, [count][n_req]: per-request TTFT */
    double *req_tpot;        /* trace only, [count][n_req]: per-request mean time per output token */
    uint32_t *seq_used;      /* closed form: tokens per request the metrics were computed for: Lin + Lout, less when
                                clamp_seq cut the prompt, 0 for configs that do not fit; trace: 0.  Asking for it
                                sends a closed-form call through the one-thread-per-config kernel. */
} guide_outputs;

enum { GUIDE_STAT_MEAN = 0, GUIDE_STAT_P50 = 1, GUIDE_STAT_P99 = 2 };

/* User constraints (Sec. 4.1 budget; Sec. 4.2 throughput requirement, latency preference).
 * +inf / 0 disable a bound.  A config passes when status == 0 and every bound holds. */
typedef struct guide_constraints {
    double max_ttft;         /* on the statistic chosen by ttft_stat */
    int32_t ttft_stat;       /* GUIDE_STAT_* */
    int32_t reserved;
    double max_latency;
    double max_cost_per_hr;
    double min_throughput;   /* on thr_decode */
} guide_constraints;

typedef enum guide_metric {
    GUIDE_LATENCY = 0, GUIDE_TTFT = 1, GUIDE_TTFT_P99 = 2, GUIDE_TPOT = 3,
    GUIDE_THROUGHPUT = 4,    /* larger is better: ordered by its negation */
    GUIDE_COST_PER_HR = 5, GUIDE_COST_PER_TOKEN = 6
} guide_metric;

#define GUIDE_TOPK_MAX 1024u
#define GUIDE_PARETO_MAX 2048u
#define GUIDE_TRACE_MAX_BATCH 256u   /* largest max-batch the trace kernel keeps resident */

/* ---- calls -------------------------------------------------------------------------------- */

const char *guide_last_error(void);

/* Build the candidate space (Sec. 3.1; enumeration as in Sec. 3.5.3's get_configurations).
 * desc and its arrays: host, copied.  Validates: non-empty axes, non-zero sizes, hidden divisible
 * by n_heads, TP degrees powers of two, kv_block >= 1, reserve <= 1000, and that no FLOP or byte
 * count of the model can wrap 64 bits at the axis maxima (GUIDE_ERR_OVERFLOW).  Touches no GPU. */
int guide_space_create(const guide_space_desc *desc, guide_space **out);
void guide_space_destroy(guide_space *space);             /* frees host and device tables; NULL ok */
uint64_t guide_space_size(const guide_space *space);      /* product of the axis lengths; 0 for NULL */
/* Mixed-radix decode of a config index (host side, for reports). */
int guide_space_decode(const guide_space *space, uint64_t idx, guide_config *out);

/* Load a request trace (iteration-level dynamic batching, Sec. 3.1).  Arrays: host, n_req
 * entries, copied; arrival_s non-decreasing and >= 0.  in_len[i] == 0 means "request i takes the
 * config's (lin, lout)"; otherwise out_len[i] >= 1.  n_req in 1..65536.  Touches no GPU. */
int guide_trace_load(const double *arrival_s, const uint32_t *in_len, const uint32_t *out_len,
                     uint64_t n_req, guide_trace **out);
void guide_trace_destroy(guide_trace *trace);
uint64_t guide_trace_size(const guide_trace *trace);

/* Bytes of device workspace guide_simulate needs (0 for the closed form; the trace kernel keeps
 * per-warp request state there).  Depends only on the trace length, not on opts. */
size_t guide_workspace_bytes(const guide_space *space, const guide_trace *trace, const guide_sim_opts *opts);

/* Evaluate configs [first, first+count).
 *   trace == NULL: closed form, one prefill stage + one aggregated decode stage per config
 *     (memory check of Sec. 3.2 Step 1 / Sec. 3.3.1, task list of Step 2, roofline of Sec. 3.4.2,
 *     time decomposition of Sec. 3.5.1, metrics of Sec. 3.2 and 5.1).
 *   trace != NULL: one warp per config steps the trace through prompt-priority continuous
 *     batching with paged KV and evict-youngest + recompute; batch sizes above
 *     GUIDE_TRACE_MAX_BATCH give GUIDE_ERR_UNSUPPORTED.
 * out: host struct of device pointers.  workspace: device, 256-byte aligned, at least
 * guide_workspace_bytes(); may be NULL when that is 0.  opts NULL = whole space, defaults. */
int guide_simulate(const guide_space *space, const guide_trace *trace, const guide_sim_opts *opts,
                   const guide_outputs *out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Bytes of device workspace for guide_select_topk / guide_pareto (per-block partial results). */
size_t guide_select_workspace_bytes(const guide_space *space, uint32_t k);
size_t guide_pareto_workspace_bytes(const guide_space *space);

/* Constraint filter + global top-k (the "top three configurations" of Sec. 3.2, generalised):
 * the k passing configs that are smallest under (key value, config index), ascending.
 *   outputs != NULL: reads materialised metrics of configs [first, first+count) (opts gives the
 *     range the arrays cover; the metric arrays the key and the constraints need must be non-NULL).
 *   outputs == NULL: fused - evaluates the closed form on the fly, nothing is materialised;
 *     trace must be NULL (GUIDE_ERR_UNSUPPORTED otherwise).
 * idx_out_dev[k], key_out_dev[k], count_out_dev[1]: device.  Fewer than k passing configs is not
 * an error: count < k, unused slots hold UINT64_MAX and +inf.  1 <= k <= GUIDE_TOPK_MAX. */
int guide_select_topk(const guide_space *space, const guide_trace *trace, const guide_outputs *outputs,
                      const guide_sim_opts *opts, const guide_constraints *cons, int key, uint32_t k,
                      uint64_t *idx_out_dev, double *key_out_dev, uint32_t *count_out_dev,
                      void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Constraint filter + 2-D Pareto front, both metrics minimised (throughput by its negation):
 * passing configs not dominated by another passing config; of several configs with equal (x, y)
 * the lowest index stays.  Written in ascending x.  The paper has no Pareto step; it is the
 * two-objective form of its selection of the fastest and the highest-throughput deployment that a
 * budget allows (Sec. 3.2, Sec. 4.1).  idx_out_dev[cap], count_out_dev[1]: device.  count is the full size of
 * the front even when cap is smaller; a front above GUIDE_PARETO_MAX points sets count to
 * UINT32_MAX.  outputs / opts / trace as for guide_select_topk. */
int guide_pareto(const guide_space *space, const guide_trace *trace, const guide_outputs *outputs,
                 const guide_sim_opts *opts, const guide_constraints *cons, int x_metric, int y_metric,
                 uint64_t *idx_out_dev, uint32_t cap, uint32_t *count_out_dev,
                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* guide_simulate (closed form), guide_select_topk and guide_pareto of the same space in one call:
 * the steps of Sec. 3.2 (memory check, performance model, selection under the constraints of Sec. 4.1)
 * as one pass.  out receives the metrics exactly as guide_simulate writes them; the two answers are
 * exactly those of the separate calls on those arrays.  What the call saves is the read-back: for a
 * whole space that goes through the line-wise kernels, a sample of configs evaluated first gives the
 * top-k bound and a set of dominating points, every config is tested against them while its metrics
 * are being stored, and only the few survivors are ranked.  Other spaces, sub-ranges and k above 128
 * run the three steps one after the other on the stream, with the same results.
 *   sel->topk_cons / pareto_cons, key, k, x_metric, y_metric: as for guide_select_topk / guide_pareto;
 *   both selections are required.  The metric arrays that the keys and the active constraints need
 *   must be present in out (as for a selection on materialised metrics).
 *   sel->topk_idx_dev[k], topk_key_dev[k], topk_count_dev[1], front_idx_dev[front_cap],
 *   front_count_dev[1]: device, written as by the separate calls.
 *   topk_workspace: device, 256-byte aligned, at least guide_select_workspace_bytes(space, k);
 *   pareto_workspace: likewise, guide_pareto_workspace_bytes(space).  The caller keeps ownership.
 * opts: time_model and tp_model as for guide_simulate; a sub-range is allowed; clamp_seq and the
 * binary32 variant give GUIDE_ERR_UNSUPPORTED (use the separate calls).  Errors as for the three
 * calls; nothing is queued when an argument is refused. */
typedef struct guide_selection {
    const guide_constraints *topk_cons;
    int32_t key;
    uint32_t k;
    uint64_t *topk_idx_dev;
    double *topk_key_dev;
    uint32_t *topk_count_dev;
    const guide_constraints *pareto_cons;
    int32_t x_metric, y_metric;
    uint64_t *front_idx_dev;
    uint32_t front_cap;
    uint32_t *front_count_dev;
    void *sweep_begin_event;      /* optional cudaEvent_t pair (NULL: none), recorded on the stream right before and   */
    void *sweep_end_event;        /* right after the kernels that evaluate and store the metrics: for callers that time them */
} guide_selection;
int guide_simulate_select(const guide_space *space, const guide_sim_opts *opts, const guide_outputs *out,
                          const guide_selection *sel, void *topk_workspace, size_t topk_workspace_bytes,
                          void *pareto_workspace, size_t pareto_workspace_bytes, void *cuda_stream);

/* Top-k over materialised metrics for callers that must not allocate device memory.  (The paper
 * has no counterpart: this is a packaging variant of guide_select_topk, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving loop whose memory
 * pool was sized up front and must not grow, in a plug-in whose host application owns every
 * allocation, or after start-up in a process that has promised a fixed device footprint.  Such a
 * caller cannot supply the workspace guide_select_topk asks for.  Here the per-block partial
 * results live in a fixed array compiled into the library (about 257 KB of device memory on every
 * GPU that loads the library, held until the process exits), and the call makes no cudaMalloc,
 * cudaFree or other allocating call.
 *
 * It selects among count configs whose metrics were written by guide_simulate: entry j of each
 * array belongs to config first + j.  outputs: host struct of DEVICE pointers; status, the key's
 * array and the array of every enabled bound must be non-NULL.  idx_out_dev[k], key_out_dev[k],
 * count_out_dev[1]: device, caller-owned.  Results, order, tie-break and unused slots are exactly
 * those of guide_select_topk.
 *
 * Limits: 1 <= k <= GUIDE_NOALLOC_TOPK_MAX and 1 <= count <= GUIDE_NOALLOC_COUNT_MAX; anything
 * larger returns GUIDE_ERR_UNSUPPORTED with a message naming the limit.
 *
 * The first call on each device looks up the array's device address (no allocation, but a
 * one-time set-up step): make that first call before starting any stream capture.  All calls on a
 * device share the one array, which keeps the previous call's contents; the call resets, on the
 * given stream, the one word that has to start from a known value, and its kernels write every
 * other word before they read it.  Two calls whose kernels could overlap on the GPU (different
 * streams, or different threads, without ordering between them) race on it: order them. */
#define GUIDE_NOALLOC_TOPK_MAX 64u
#define GUIDE_NOALLOC_COUNT_MAX (1ull << 40)
int guide_select_topk_noalloc(const guide_outputs *outputs, uint64_t first, uint64_t count,
                              const guide_constraints *cons, int key, uint32_t k,
                              uint64_t *idx_out_dev, double *key_out_dev, uint32_t *count_out_dev,
                              void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* GUIDE_H */
