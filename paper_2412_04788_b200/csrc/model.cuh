// Device-side performance model: task table, roofline, stage time, memory check.
//
// Everything here is written so that the same values come out regardless of how a kernel
// arranges its loops: integer FLOP/byte counts are exact 64-bit integers, converted to double
// once, combined in one fixed order, and the file is compiled with -fmad=false so no
// multiply-add is ever fused.  Scaling by a power of two (the tensor-parallel degree, the
// task multiplicities 2 and 1+g) is exact in binary64 and commutes with rounding, which is
// what lets a kernel fold those factors into a cached table without changing a bit.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace guide {

typedef unsigned long long u64;
typedef unsigned int u32;

enum { CLS_LINEAR = 0, CLS_ATTN = 1, CLS_ELEM = 2 };

// per-model table entry (built on the device by k_build_tables)
struct DModel {
    u32 N, H, nh, nkv, I, V, g, wb, ab, kvb;
    u32 Dkv;      // n_kv * (H / n_h)
    u32 pad;
    u64 wbytes;   // all weights in bytes: (N (2H^2 + 2 H Dkv + (2+g) H I) + 2 V H) * w_b
    u64 kv2;      // KV bytes per token over all GPUs: 2 N Dkv kv_b   (Sec. 3.3.1 with H -> Dkv)
};

// per (hardware, framework) entry: reciprocal rates (product first, then one reciprocal)
struct DRate {
    double inv_c[3], inv_m[3], inv_comm, clat, tovh, price;
    u64 usable;   // MEM - (MEM/1000) * reserve_permille
    u32 flash, kv_block;
    u32 split, seg;   // requests per prompt sub-batch, tokens per prompt segment (0: whole batch / prompt)
    u32 policy;       // trace scheduling: GUIDE_POLICY_*; with SPLIT_FUSE seg is the token budget of an iteration
    u32 keep;         // thousandths of a request's KV cache the eviction policy keeps (1000: all of it)
};

// one hardware x framework pair in the sorted walk of the model kernel
struct HfSorted {
    u64 usable;
    u32 block;        // KV block size
    u32 hf;           // pair index h * n_f + f
    u32 seg_end;      // sorted position one past the last pair with this block size
    u32 pad;
};

struct StageConst;
struct RateF;

struct DSpace {
    const DModel *models;
    const DRate *rates;          // [n_h * n_f]
    const u32 *batch, *tp;
    const u32 *dp;               // [n_t]: data-parallel degree that goes with tp[i] (Sec. 3.5.2)
    const uint2 *pairs;          // (lin, lout)
    const double *cost_hr;       // [n_h * n_f][n_t]: price x TP degree
    const double *cost_sec;      // [n_h * n_f][n_t]: (price x TP degree) / 3600
    const ulonglong2 *hfmem;     // [n_h * n_f]: x = usable bytes, y = KV block size (what the memory check reads)
    const StageConst *stage_consts;   // [n_t + 1][n_m]: the task-table factors per (TP degree, model); the last group is t = 1
    const RateF *ratef;          // [n_h * n_f]: the rates in binary32 (reduced-precision variant of the closed form)
    const double *rate10;        // [n_h * n_f][10]: inv_c[3], inv_m[3], inv_comm, clat, tovh, flash (0.0 or 1.0); 16-byte aligned rows
    // Orders that only steer which thread does what (any permutation gives the same results):
    const HfSorted *hf_sorted;   // [n_h * n_f]: the pairs grouped by KV block size, largest usable memory first
    const u32 *plane_order;      // [n_m][n_t * n_l / 4]: foursomes of the (TP, length) plane by growing memory need
    const u32 *line_order;       // [n_m][n_t * n_l / 16]: the same for lines of sixteen positions
    u32 n_m, n_h, n_f, n_b, n_t, n_l;
    u32 chunked;                 // per-framework prompt splitting or cache eviction, or a per-call option below: only the
                                 // one-thread-per-config evaluation handles those (no tables shared between frameworks)
    u32 clamp_seq;               // cut sequences that do not fit to S_max (Sec. 3.3.2); set per call
};

struct DTrace {
    const double *arrival;
    const u32 *in_len, *out_len;
    u32 n;
    u32 max_tokens;              // max over requests of in+out (0-length requests excluded)
    u32 any_zero;                // some request takes the config's lengths
    u64 sum_out;                 // sum of out_len over requests with explicit lengths
    u64 sum_in;                  // sum of in_len over the same requests
    u32 n_zero;                  // number of requests taking the config's lengths
};

struct Cfg { u32 m, h, f, b, t, l; };

__device__ __forceinline__ Cfg decode_index(const DSpace &s, u64 idx) {
    Cfg c;
    c.l = (u32)(idx % s.n_l); idx /= s.n_l;
    c.t = (u32)(idx % s.n_t); idx /= s.n_t;
    c.b = (u32)(idx % s.n_b); idx /= s.n_b;
    c.f = (u32)(idx % s.n_f); idx /= s.n_f;
    c.h = (u32)(idx % s.n_h); idx /= s.n_h;
    c.m = (u32)idx;
    return c;
}

// ---- task table --------------------------------------------------------------------------------
// Compute load F and data size B of every distinct task of one layer, for a stage with T new
// tokens, E sequences emitting a token, A = sum(query x context), C = sum(context), R repeats.
// Values are per GPU (sharded part / t + replicated part) with the task multiplicity folded in.
// o_proj has the same F and B as q_proj, and sv the same as qk, so each pair shares an entry.
struct TaskTab {
    double F1, B1;      // norm x2 (ELEM)
    double F2, B2;      // q_proj, o_proj (LINEAR)
    double F3, B3;      // k_proj + v_proj (LINEAR)
    double F5, B5;      // residual x2 (ELEM)
    double F6, B6;      // up (+ gate) (LINEAR)
    double F7, B7;      // activation (ELEM)
    double F8, B8;      // down (LINEAR)
    double F9, B9;      // qk = sv (ATTN), B9 with FlashAttention
    double B9x;         // ... without: + score matrix
    double F10, B10x;   // softmax (ATTN); with FlashAttention its B is 0
    double F13, B13;    // lm_head (LINEAR), once per stage
    double hops, cbytes; // all-reduce: latency hops R*2(t-1), bytes 2(t-1) M / t
    double Rd;
};

__device__ __forceinline__ double cvt(u64 x) { return __ull2double_rn(x); }

// sharded / t + replicated, one rounding in the add
__device__ __forceinline__ double per_gpu(u64 sh, u64 rp, double inv_t) { return cvt(sh) * inv_t + cvt(rp); }

// The part of the table that does not depend on A or C (everything but attention).
__device__ __forceinline__ void build_fixed_tasks(const DModel &m, u32 t, u64 T, u64 E, u64 R, TaskTab &k) {
    const double inv_t = 1.0 / (double)t;      // t is a power of two: exact
    const u64 H = m.H, I = m.I, Dkv = m.Dkv, V = m.V, ab = m.ab, wb = m.wb, kvb = m.kvb;
    const u64 TH = T * H, THa = TH * ab, TI = T * I, TIa = TI * ab;
    k.F1 = 2.0 * cvt(4 * TH);
    k.B1 = 2.0 * cvt(2 * THa);
    k.F2 = cvt(2 * TH * H) * inv_t;
    k.B2 = per_gpu(R * (H * H * wb) + THa, THa, inv_t);
    k.F3 = 2.0 * (cvt(2 * TH * Dkv) * inv_t);
    k.B3 = 2.0 * per_gpu(R * (H * Dkv * wb) + T * Dkv * kvb, THa, inv_t);
    k.F5 = 2.0 * cvt(TH);
    k.B5 = 2.0 * cvt(3 * THa);
    const double mult6 = (double)(1 + m.g);
    k.F6 = mult6 * (cvt(2 * TH * I) * inv_t);
    k.B6 = mult6 * per_gpu(R * (H * I * wb) + TIa, THa, inv_t);
    k.F7 = cvt(4 * TI) * inv_t;
    k.B7 = cvt((2 + m.g) * TIa) * inv_t;
    k.F8 = cvt(2 * TI * H) * inv_t;
    k.B8 = per_gpu(R * (I * H * wb) + TIa, THa, inv_t);
    k.F13 = cvt(2 * (E * H) * V) * inv_t;
    k.B13 = per_gpu(R * (H * V * wb) + E * V * ab, E * H * ab, inv_t);
    k.Rd = cvt(R);
    if (t > 1) {
        k.hops = cvt(R * (u64)(2 * (t - 1)));
        k.cbytes = cvt((u64)(2 * (t - 1)) * THa) * inv_t;
    } else {
        k.hops = 0.0; k.cbytes = 0.0;
    }
}

// Attention entries: query x context work A, KV read of C context tokens, score matrix X.
__device__ __forceinline__ void build_attn_tasks(const DModel &m, u32 t, u64 T, u64 A, u64 C, TaskTab &k) {
    const double inv_t = 1.0 / (double)t;
    const u64 THa = T * m.H * m.ab;
    const u64 kv_read = C * m.Dkv * m.kvb;
    const u64 X = (u64)m.nh * A * m.ab;
    k.F9 = cvt(2 * m.H * A) * inv_t;
    k.B9 = cvt(THa + kv_read) * inv_t;
    k.B9x = cvt(THa + kv_read + X) * inv_t;
    k.F10 = cvt(5 * (u64)m.nh * A) * inv_t;
    k.B10x = cvt(2 * X) * inv_t;
}

template <int TIME_SUM>
__device__ __forceinline__ double task_time(double F, double B, double ic, double im) {
    const double tc = F * ic;          // compute time (Sec. 3.5.1)
    const double tm = B * im;          // read/write time
    return TIME_SUM ? tc + tm : (tc > tm ? tc : tm);   // Sec. 3.5.1 literal sum, or the roofline of Sec. 3.4.2
}

// ---- the same table in doubles ---------------------------------------------------------------------
// Per (model, tensor-parallel degree): the factors that turn the token counts of a stage into the
// entries of its task table.  Products and sums of integers stay exact in binary64 below 2^53, and
// scaling by 1/t (a power of two) and by the multiplicities commutes with rounding, so
//   T x factor  ==  (double)(T * integer factor) x 1/t
// bit for bit whenever the integer count is below 2^53.  A kernel that has checked that bound for a
// config can build its tables without integer products and conversions.
struct StageConst {
    double f1, b1;        // norm x2:        8 H, 4 H a_b                   (per new token)
    double f2, w2;        // q_proj, o_proj: 2 H H / t;  H H w_b
    double ha;            // activations of one token: H a_b
    double f3, w3, dk;    // k/v_proj x2:    4 H Dkv / t;  H Dkv w_b;  Dkv kv_b
    double f5, b5;        // residual x2:    2 H, 6 H a_b
    double f6, w6, ia;    // up (+ gate):    (1+g) 2 H I / t;  H I w_b;  I a_b
    double mult6;         // 1 + g
    double f7, b7;        // activation:     4 I / t, (2+g) I a_b / t
    double f8;            // down:           2 I H / t  (weights and activations as up)
    double f13, w13, va;  // lm_head:        2 H V / t;  H V w_b;  V a_b      (per emitting sequence)
    double hops, cb;      // all-reduce:     2 (t-1);  2 (t-1) H a_b / t
    double inv_t;
    double f9, kv, f10, xb;   // attention:  2 H / t;  Dkv kv_b;  5 n_h / t;  n_h a_b (score bytes per unit of A)
    double pad[5];        // 256 bytes
};

__device__ __forceinline__ StageConst stage_const(const DModel &m, u32 t) {
    StageConst c;
    const double inv_t = 1.0 / (double)t;
    const u64 H = m.H, I = m.I, Dkv = m.Dkv, V = m.V, ab = m.ab, wb = m.wb, kvb = m.kvb;
    c.f1 = cvt(8 * H); c.b1 = cvt(4 * H * ab);
    c.f2 = cvt(2 * H * H) * inv_t; c.w2 = cvt(H * H * wb);
    c.ha = cvt(H * ab);
    c.f3 = cvt(4 * H * Dkv) * inv_t; c.w3 = cvt(H * Dkv * wb); c.dk = cvt(Dkv * kvb);
    c.f5 = cvt(2 * H); c.b5 = cvt(6 * H * ab);
    c.mult6 = (double)(1 + m.g);
    c.f6 = c.mult6 * (cvt(2 * H * I) * inv_t); c.w6 = cvt(H * I * wb); c.ia = cvt(I * ab);
    c.f7 = cvt(4 * I) * inv_t; c.b7 = cvt((2 + m.g) * I * ab) * inv_t;
    c.f8 = cvt(2 * I * H) * inv_t;
    c.f13 = cvt(2 * H * V) * inv_t; c.w13 = cvt(H * V * wb); c.va = cvt(V * ab);
    c.hops = cvt((u64)(2 * (t - 1))); c.cb = cvt((u64)(2 * (t - 1)) * H * ab) * inv_t;
    c.inv_t = inv_t;
    c.f9 = cvt(2 * H) * inv_t; c.kv = cvt(Dkv * kvb); c.f10 = cvt(5 * (u64)m.nh) * inv_t; c.xb = cvt((u64)m.nh * ab);
    for (int i = 0; i < 5; i++) c.pad[i] = 0.0;
    return c;
}

// Upper bound (as a double: no wrap-around, rounding far below the margin) of the largest integer
// count a stage of at most T new tokens, E emitting sequences, attention work A and context C
// produces for this model (R = 1).  While it is below 2^52 the doubles above reproduce the integer
// table exactly (the limit is 2^53; the factor of two covers this bound's own rounding).
__device__ __forceinline__ double stage_count_bound(const DModel &m, u32 t, double T, double E, double A, double C) {
    const double H = m.H, I = m.I, Dkv = m.Dkv, V = m.V, ab = m.ab, wb = m.wb, kvb = m.kvb, nh = m.nh, g = m.g;
    const double big = fmax(fmax(H, I), Dkv), bytes = fmax(ab, kvb);
    double v = 8.0 * T * H;
    v = fmax(v, 6.0 * T * H * ab);
    v = fmax(v, 4.0 * T * big * big);                    // 2 T H H, 4 T H Dkv, (1+g) 2 T H I, 2 T I H
    v = fmax(v, big * big * wb + T * big * bytes);       // weights of one matrix + its activations / KV written
    v = fmax(v, (2.0 + g) * T * I * ab);
    v = fmax(v, 2.0 * E * H * V);
    v = fmax(v, H * V * wb + E * V * ab + E * H * ab);
    v = fmax(v, 2.0 * (double)t * T * H * ab);
    v = fmax(v, 2.0 * H * A);
    v = fmax(v, 5.0 * nh * A);
    v = fmax(v, T * H * ab + C * Dkv * kvb + 2.0 * nh * A * ab);
    return v;
}

// One stage time (R = 1) from the doubles: the same operations in the same order as
// build_fixed_tasks / build_attn_tasks followed by eval_phase.  rate: a row of rate10
// (inv_c[LINEAR, ATTN, ELEM], inv_m[LINEAR, ATTN, ELEM], inv_comm, clat, tovh, flash).
struct StageFixed { double fix, comm, head, tha; };

template <int TIME_SUM>
__device__ __forceinline__ StageFixed stage_fixed(const StageConst &c, const double *rate, double Td, double Ed) {
    const double icL = rate[0], icE = rate[2], imL = rate[3], imE = rate[5];
    const double tha = Td * c.ha;
    const double t2 = task_time<TIME_SUM>(Td * c.f2, (c.w2 + tha) * c.inv_t + tha, icL, imL);
    double s = task_time<TIME_SUM>(Td * c.f1, Td * c.b1, icE, imE);
    s = s + t2;
    s = s + task_time<TIME_SUM>(Td * c.f3, 2.0 * ((c.w3 + Td * c.dk) * c.inv_t + tha), icL, imL);
    s = s + t2;
    s = s + task_time<TIME_SUM>(Td * c.f5, Td * c.b5, icE, imE);
    const double up = (c.w6 + Td * c.ia) * c.inv_t + tha;        // bytes of one FFN matrix pass
    s = s + task_time<TIME_SUM>(Td * c.f6, c.mult6 * up, icL, imL);
    s = s + task_time<TIME_SUM>(Td * c.f7, Td * c.b7, icE, imE);
    s = s + task_time<TIME_SUM>(Td * c.f8, up, icL, imL);
    StageFixed o;
    o.fix = s;
    o.comm = 2.0 * (c.hops * rate[7] + (Td * c.cb) * rate[6]);
    o.head = task_time<TIME_SUM>(Ed * c.f13, (c.w13 + Ed * c.va) * c.inv_t + Ed * c.ha, icL, imL);
    o.tha = tha * c.inv_t;
    return o;
}

// Sum of the eight non-attention layer tasks in their fixed order.
template <int TIME_SUM>
__device__ __forceinline__ double eval_fixed(const TaskTab &k, const DRate &r) {
    const double icL = r.inv_c[CLS_LINEAR], imL = r.inv_m[CLS_LINEAR];
    const double icE = r.inv_c[CLS_ELEM], imE = r.inv_m[CLS_ELEM];
    const double t2 = task_time<TIME_SUM>(k.F2, k.B2, icL, imL);
    double s = task_time<TIME_SUM>(k.F1, k.B1, icE, imE);
    s = s + t2;
    s = s + task_time<TIME_SUM>(k.F3, k.B3, icL, imL);
    s = s + t2;
    s = s + task_time<TIME_SUM>(k.F5, k.B5, icE, imE);
    s = s + task_time<TIME_SUM>(k.F6, k.B6, icL, imL);
    s = s + task_time<TIME_SUM>(k.F7, k.B7, icE, imE);
    s = s + task_time<TIME_SUM>(k.F8, k.B8, icL, imL);
    return s;
}

template <int TIME_SUM>
__device__ __forceinline__ double eval_attn(const TaskTab &k, const DRate &r) {
    const double ic = r.inv_c[CLS_ATTN], im = r.inv_m[CLS_ATTN];
    const double t9 = task_time<TIME_SUM>(k.F9, r.flash ? k.B9 : k.B9x, ic, im);
    const double t10 = task_time<TIME_SUM>(k.F10, r.flash ? 0.0 : k.B10x, ic, im);
    return (t9 + t10) + t9;
}

__device__ __forceinline__ double eval_comm(const TaskTab &k, const DRate &r) {
    // two ring all-reduces per layer; both terms are exactly 0 when t == 1
    return 2.0 * (k.hops * r.clat + k.cbytes * r.inv_comm);
}

template <int TIME_SUM>
__device__ __forceinline__ double eval_head(const TaskTab &k, const DRate &r) {
    return task_time<TIME_SUM>(k.F13, k.B13, r.inv_c[CLS_LINEAR], r.inv_m[CLS_LINEAR]);
}

// T_phase = R t_ovh + (N ((S_fix + S_att) + S_comm) + t_head), then the optional log2 rule.
__device__ __forceinline__ double combine_phase(double s_fix, double s_att, double s_comm, double t_head,
                                                double Rd, double Nd, double tovh, double log2_factor) {
    const double layer = (s_fix + s_att) + s_comm;
    double tp = Rd * tovh + (Nd * layer + t_head);
    if (log2_factor != 1.0) tp = tp * log2_factor;   // x1.0 would be exact anyway
    return tp;
}

// Time of a prompt pass over T new tokens of E requests with attention work A = sum of squared
// lengths (the context is the new tokens themselves), from the doubles; out of line: events are
// rare next to decode iterations and the call keeps their registers apart.
struct AttnRates { double c_f9, c_f10, c_b10, icA, imA, Nd, tovh, lf; };
template <int TIME_SUM>
__device__ __noinline__ double stage_prompt_pass(const StageConst *scp, const double *rate, double Td, double Ed, double Ad,
                                                 const AttnRates *ar) {
    const StageConst c = *scp;
    const StageFixed sf = stage_fixed<TIME_SUM>(c, rate, Td, Ed);
    const double xw = rate[9] != 0.0 ? 0.0 : c.xb;           // FlashAttention: no score-matrix traffic
    const double t9 = task_time<TIME_SUM>(Ad * ar->c_f9, ((Td * c.ha + Td * c.kv) + Ad * xw) * c.inv_t, ar->icA, ar->imA);
    const double t10 = task_time<TIME_SUM>(Ad * ar->c_f10, Ad * ar->c_b10, ar->icA, ar->imA);
    return combine_phase(sf.fix, (t9 + t10) + t9, sf.comm, sf.head, 1.0, ar->Nd, ar->tovh, ar->lf);
}
// The terms of a decode iteration that depend on the number of residents only.
template <int TIME_SUM>
__device__ __noinline__ StageFixed stage_decode_terms(const StageConst *scp, const double *rate, double nd) {
    return stage_fixed<TIME_SUM>(*scp, rate, nd, nd);
}

template <int TIME_SUM>
__device__ __forceinline__ double eval_phase(const TaskTab &k, const DRate &r, double Nd, double log2_factor) {
    return combine_phase(eval_fixed<TIME_SUM>(k, r), eval_attn<TIME_SUM>(k, r), eval_comm(k, r),
                         eval_head<TIME_SUM>(k, r), k.Rd, Nd, r.tovh, log2_factor);
}

// (1 + log2 t) / t for the throughput rule of Sec. 3.2; 1.0 when the explicit TP model is used.
__device__ __forceinline__ double log2_rule_factor(u32 t, int tp_model) {
    if (tp_model == 0) return 1.0;
    const u32 lg = 31 - __clz(t);
    return (double)(1 + lg) / (double)t;
}

// ---- memory model (Sec. 3.2 Step 1, Sec. 3.3.1) ---------------------------------------------

// floor(num / den) for den >= 1, by one double division plus a correction when both fit 2^53
__device__ __forceinline__ u64 floor_div(u64 num, u64 den) {
    if ((num | den) >> 53) return num / den;
    u64 q = __double2ull_rz(__ull2double_rn(num) / __ull2double_rn(den));
    // the rounded quotient is within 1 of the true one
    if (q * den > num) q--;
    else if ((q + 1) * den <= num) q++;
    return q;
}

__device__ __forceinline__ u32 clamp_u32(u64 v) { return v > 0xFFFFFFFFull ? 0xFFFFFFFFu : (u32)v; }

// floor(num / den) with a precomputed reciprocal inv = 1 / (double)den, for num, den < 2^52:
// the product is within one unit of the quotient, two integer checks make it exact.
__device__ __forceinline__ u64 floor_div_recip(u64 num, u64 den, double inv) {
    u64 q = __double2ull_rz(__ull2double_rn(num) * inv);
    if (q * den > num) q--;
    else if ((q + 1) * den <= num) q++;
    return q;
}

struct MemInfo { u64 w_gpu, kv_tok; u32 log2t; };

// KV bytes of one request of S tokens under a block size, and the reciprocal used to divide by it;
// depends on the thread's (model, TP, lengths) and on the framework's block size only, so a loop
// over hardware x framework pairs recomputes it just when the block size changes.
struct ReqBytes {
    u64 bytes;        // ceil(S / block) * block * kv_tok
    double inv;       // 1 / bytes, valid when small is set
    u32 block;        // block size this was computed for (0 = not yet)
    bool small;       // bytes < 2^52: the reciprocal path is exact
};
__device__ __forceinline__ void req_bytes_for(ReqBytes &q, u32 block, u64 S, u64 kv_tok) {
    const u64 s_blk = block == 1 ? S : ((S + block - 1) / block) * block;
    q.bytes = s_blk * kv_tok;
    q.small = (q.bytes >> 52) == 0;
    q.inv = 1.0 / __ull2double_rn(q.bytes);
    q.block = block;
}
// status and B_max with the request bytes already known
__device__ __forceinline__ u32 feasibility_cached(const DModel &m, u64 usable, const MemInfo &mi, u32 t, u32 b,
                                                  const ReqBytes &q, u32 &bmax_out) {
    u64 bmax = 0;
    if (usable > mi.w_gpu) {
        const u64 avail = usable - mi.w_gpu;
        bmax = (q.small && (avail >> 52) == 0) ? floor_div_recip(avail, q.bytes, q.inv) : avail / q.bytes;
    }
    u32 st = 0;
    if (usable <= mi.w_gpu) st |= 1;
    if ((u64)b > bmax) st |= 2;
    if ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) st |= 4;   // t is a power of two
    bmax_out = clamp_u32(bmax);
    return st;
}

__device__ __forceinline__ MemInfo mem_info(const DModel &m, u32 t) {
    MemInfo mi;
    mi.log2t = 31 - __clz(t);
    mi.w_gpu = (m.wbytes + (u64)(t - 1)) >> mi.log2t;   // ceil(W w_b / t)
    mi.kv_tok = m.kv2 >> mi.log2t;
    return mi;
}


// ---- one config in closed form -------------------------------------------------------------------

struct Metrics {
    double latency, ttft, tpot, thr, cost_hr, cost_tok;
    u64 n_iters, n_req_iters;
    u32 bmax;
    u32 status;
    u32 seq_used;      // tokens per request the metrics were computed for; 0 when the config does not fit
};

__device__ __forceinline__ void set_infeasible(Metrics &o) {
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    o.latency = inf; o.ttft = inf; o.tpot = inf; o.thr = 0.0; o.cost_hr = inf; o.cost_tok = inf;
    o.n_iters = 0; o.n_req_iters = 0;
}

// status and B_max of a closed-form config
// Sec. 3.2 Step 1: with data parallelism the batch is shared out over dp replicas; the slowest one
// (the one with the rounded-up share) sets the time and the memory need.
__device__ __forceinline__ u32 replica_batch(u32 b, u32 dp) { return dp == 1 ? b : (b + dp - 1) / dp; }

// Tokens of a cache of c tokens that stay when the eviction policy keeps p thousandths of it.
__device__ __forceinline__ u64 kept_tokens(u64 c, u32 p) { return p >= 1000 ? c : (c * p + 999) / 1000; }

__device__ __forceinline__ u32 closed_form_feasibility(const DModel &m, const DRate &r, const MemInfo &mi, u32 t,
                                                       u32 b, u32 lin, u32 lout, u32 &bmax_out) {
    const u64 S = kept_tokens((u64)lin + lout, r.keep);
    const u64 s_blk = r.kv_block == 1 ? S : ((S + r.kv_block - 1) / r.kv_block) * r.kv_block;
    const u64 bmax = r.usable > mi.w_gpu ? floor_div(r.usable - mi.w_gpu, s_blk * mi.kv_tok) : 0;
    u32 st = 0;
    if (r.usable <= mi.w_gpu) st |= 1;
    if ((u64)b > bmax) st |= 2;
    if ((m.nh & (t - 1)) != 0 || (m.nkv & (t - 1)) != 0) st |= 4;   // t is a power of two
    bmax_out = clamp_u32(bmax);
    return st;
}

// final metrics from the two stage times (Sec. 3.2: TTFT = prefill time, throughput; Sec. 5.1)
__device__ __forceinline__ void closed_form_metrics(double t_pre, double t_dec, u32 b, u32 n, double cost_hr,
                                                    double cost_sec, Metrics &o, u64 n_pass = 1, u64 n_seg = 1) {
    const double inf = __longlong_as_double(0x7FF0000000000000LL);
    o.ttft = t_pre;
    o.latency = t_pre + t_dec;
    o.cost_hr = cost_hr;                 // price x TP degree x DP degree
    if (n > 0) {
        o.tpot = t_dec / (double)n;
        o.thr = cvt((u64)b * n) / t_dec;
        o.cost_tok = cost_sec / o.thr;   // (cost_hr / 3600) / throughput
    } else {
        o.tpot = 0.0; o.thr = 0.0; o.cost_tok = inf;
    }
    o.n_iters = n_pass + (u64)n;                    // prompt passes of one replica + decode steps
    o.n_req_iters = (u64)b * (n_seg + (u64)n);
}

// Prompt processing of one sub-batch of sb requests in segments of seg tokens (Sec. 3.3.2): one pass
// per segment, its tokens attending the prompt up to the end of the segment; the LM head runs with
// the last segment only.  Passes are summed in order from 0.0.
template <int TIME_SUM>
__device__ __noinline__ double segmented_prefill(const DModel &m, const DRate &r, u32 tt, u32 sb, u32 lin, u32 seg,
                                                 double Nd, double lf) {
    TaskTab k;
    double sum = 0.0;
    for (u32 done = 0; done < lin; done += seg) {
        const u32 q = min(seg, lin - done);
        const bool last = done + q == lin;
        const u64 T = (u64)sb * q;
        build_fixed_tasks(m, tt, T, last ? sb : 0, 1, k);
        build_attn_tasks(m, tt, T, T * (done + q), (u64)sb * (done + q), k);
        const double head = last ? eval_head<TIME_SUM>(k, r) : 0.0;
        sum = sum + combine_phase(eval_fixed<TIME_SUM>(k, r), eval_attn<TIME_SUM>(k, r), eval_comm(k, r), head, k.Rd, Nd,
                                  r.tovh, lf);
    }
    return sum;
}

// Whole closed-form evaluation of one config, nothing cached (used where configs arrive in
// arbitrary order; the tiled kernels hoist the table building out of the hardware x framework loop).
template <int TIME_SUM>
__device__ __forceinline__ void closed_form_eval(const DSpace &s, const Cfg &c, int tp_model, Metrics &o) {
    const DModel m = s.models[c.m];
    const DRate &r = s.rates[c.h * s.n_f + c.f];
    const u32 t = s.tp[c.t], b_all = s.batch[c.b];
    const u32 b = replica_batch(b_all, s.dp[c.t]);   // each of the dp replicas serves its share of the batch
    const uint2 pr = s.pairs[c.l];
    u32 lin = pr.x;
    const u32 lout = pr.y;
    const MemInfo mi = mem_info(m, t);
    if (s.clamp_seq && r.usable > mi.w_gpu) {
        // Sec. 3.3.2: S_max = floor(C_available / (KV bytes per token x B)), in whole blocks; with cache
        // eviction the longest sequence whose kept part fits.  The prompt is what gets cut.
        const u64 cap_tok = floor_div(r.usable - mi.w_gpu, mi.kv_tok * b);
        const u64 cap_blk = (cap_tok / r.kv_block) * r.kv_block;
        // room for 2^40 tokens or more is room for any sequence (lengths are 32-bit): no product that could wrap
        const u64 s_max = (r.keep >= 1000 || cap_blk >= (1ull << 40)) ? cap_blk : (1000 * cap_blk) / r.keep;
        if ((u64)lin + lout > s_max && s_max > lout) lin = (u32)(s_max - lout);
    }
    o.status = closed_form_feasibility(m, r, mi, t, b, lin, lout, o.bmax);
    o.seq_used = o.status ? 0u : lin + lout;
    if (o.status) { set_infeasible(o); return; }
    const u32 tt = tp_model ? 1u : t;
    const double lf = log2_rule_factor(t, tp_model);
    const double Nd = (double)m.N;
    TaskTab k;
    double t_pre;
    u64 n_pass = 1, n_seg = 1;
    if (r.split | r.seg) {
        // Sec. 3.3.1: sub-batches of split requests, the remainder as one more; equal ones take equal time
        const u32 split = (r.split == 0 || r.split > b) ? b : r.split;
        const u32 seg = (r.seg == 0 || r.seg > lin) ? lin : r.seg;
        const u32 n_full = b / split, rest = b % split;
        t_pre = (double)n_full * segmented_prefill<TIME_SUM>(m, r, tt, split, lin, seg, Nd, lf);
        if (rest) t_pre = t_pre + segmented_prefill<TIME_SUM>(m, r, tt, rest, lin, seg, Nd, lf);
        n_seg = (lin + seg - 1) / seg;
        n_pass = (u64)(n_full + (rest != 0)) * n_seg;
    } else {
        const u64 Tp = (u64)b * lin;
        build_fixed_tasks(m, tt, Tp, b, 1, k);
        build_attn_tasks(m, tt, Tp, Tp * lin, Tp, k);
        t_pre = eval_phase<TIME_SUM>(k, r, Nd, lf);
    }
    const u32 n = lout - 1;
    double t_dec = 0.0;
    if (n > 0) {
        const u64 Td = (u64)b * n;
        // step j attends lin + j tokens, of which the cache still holds the kept share
        const u64 ctx = kept_tokens((u64)b * ((u64)n * lin + ((u64)n * (n + 1)) / 2), r.keep);
        build_fixed_tasks(m, tt, Td, Td, n, k);
        build_attn_tasks(m, tt, Td, ctx, ctx, k);
        t_dec = eval_phase<TIME_SUM>(k, r, Nd, lf);
    }
    const u32 ci = (c.h * s.n_f + c.f) * s.n_t + c.t;
    closed_form_metrics(t_pre, t_dec, b_all, n, s.cost_hr[ci], s.cost_sec[ci], o, n_pass, n_seg);
}

}  // namespace guide
