// Library-internal declarations: handles, device views, launch entry points of each kernel file.
#pragma once
#include <cstdarg>
#include <cstdio>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/guide.h"
#include "model.cuh"
#include "model_f32.cuh"
#include "tiled.cuh"

namespace guide {

int fail(int code, const char *fmt, ...);          // records the message, returns code
int cuda_fail(cudaError_t e, const char *what);

#define GUIDE_CUDA(call)                                            \
    do {                                                            \
        cudaError_t e__ = (call);                                   \
        if (e__ != cudaSuccess) return guide::cuda_fail(e__, #call); \
    } while (0)

// Work counters of the persistent closed-form model kernel: one 128-byte slot per stream that uses
// the handle, so that calls on different streams never share one.
static constexpr unsigned TICKET_SLOTS = 64;

struct DeviceTables {
    int device = -1;
    void *blob = nullptr;
    DSpace view{};
    unsigned *tickets = nullptr;     // TICKET_SLOTS slots, 32 words apart
    std::vector<void *> ticket_streams;   // slot i belongs to the calls on ticket_streams[i]
};

struct DeviceTrace {
    int device = -1;
    void *blob = nullptr;
    DTrace view{};
};

}  // namespace guide

struct guide_space {
    std::vector<guide_model> models;
    std::vector<guide_hw> hw;
    std::vector<guide_fw> fw;
    std::vector<uint32_t> batch, tp, dp;          // dp[i] goes with tp[i]; all 1 when the caller gave none
    std::vector<guide_len_pair> pairs;
    uint64_t size = 0;
    uint32_t max_batch = 0, max_tp = 0, max_lin = 0, max_lout = 0, max_dp = 1, chunked = 0, evicting = 0;
    std::mutex mu;
    std::vector<guide::DeviceTables> dev;
};

struct guide_trace {
    std::vector<double> arrival;
    std::vector<uint32_t> in_len, out_len;
    uint32_t max_in = 0, max_out = 0, max_tokens = 0, n_zero = 0;
    uint64_t sum_out = 0, sum_in = 0;
    std::mutex mu;
    std::vector<guide::DeviceTrace> dev;
};

namespace guide {

// device views for the current device (uploads on first use)
int space_on_device(guide_space *s, DSpace *out, unsigned **ticket, cudaStream_t st);
int trace_on_device(guide_trace *t, DTrace *out, cudaStream_t st);

// closed_form.cu
struct LineSelect;           // select_sink.cuh: both selections of a combined simulate-and-select call
bool closed_form_by_lines(const DSpace &s, Range r, const guide_outputs &o);
int launch_closed_form(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o,
                       unsigned *ticket, cudaStream_t st, const LineSelect *sel = nullptr);
int launch_closed_form_f32(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o, cudaStream_t st);
// trace_sim.cu
// What the host knows about the configs the one-lane-per-config kernel would take: per class of max
// batch, how many configs of the whole space have a prompt-first framework with a block size the
// phase histogram covers (an upper bound: the kernel itself also checks that the config's integer
// counts stay below 2^53), and the largest such block size.
static constexpr unsigned LANE_N_CLASSES = 3;
struct LaneHints { u64 class_configs[LANE_N_CLASSES]; u32 hist_n; };
LaneHints lane_hints(const guide_space &s);
size_t trace_workspace_bytes(u32 n_req, const LaneHints &hints);
int launch_trace_sim(const DSpace &s, const DTrace &t, Range r, int time_model, int tp_model, u64 max_iters,
                     const guide_outputs &o, void *ws, size_t ws_bytes, cudaStream_t st, u32 policies,
                     const LaneHints &hints);
// select.cu
size_t topk_workspace_bytes(u32 k);
size_t pareto_workspace_bytes();
int launch_topk(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                const guide_constraints &c, int key, u32 k, u64 *idx_out, double *key_out, u32 *count_out,
                void *ws, unsigned *ticket, cudaStream_t st);
int launch_pareto(const DSpace &s, Range r, const guide_outputs *mat, int time_model, int tp_model,
                  const guide_constraints &c, int xm, int ym, u64 *idx_out, u32 cap, u32 *count_out,
                  void *ws, unsigned *ticket, cudaStream_t st);
int launch_simulate_select(const DSpace &s, Range r, const guide_outputs &o, int time_model, int tp_model,
                           const guide_constraints &ct, int key, u32 k, u64 *tk_idx, double *tk_key, u32 *tk_count, void *ws_t,
                           const guide_constraints &cp, int xm, int ym, u64 *pf_idx, u32 cap, u32 *pf_count, void *ws_p,
                           unsigned *ticket, cudaStream_t st, cudaEvent_t sweep_begin, cudaEvent_t sweep_end);
int launch_topk_noalloc(Range r, const guide_outputs &mat, const guide_constraints &c, int key, u32 k,
                        u64 *idx_out, double *key_out, u32 *count_out, cudaStream_t st);

int num_sms();

}  // namespace guide
