// Closed-form evaluation kernels: one prefill stage + one aggregated decode stage per config
// (Sec. 3.2 Steps 1-2, roofline of Sec. 3.4.2, time decomposition of Sec. 3.5.1).
#include "guide_internal.cuh"

namespace guide {

__device__ __forceinline__ void store_metrics(const guide_outputs &o, u64 j, const Metrics &m) {
    if (o.latency) __stcs(o.latency + j, m.latency);
    if (o.ttft) __stcs(o.ttft + j, m.ttft);
    if (o.ttft_p50) __stcs(o.ttft_p50 + j, m.ttft);
    if (o.ttft_p99) __stcs(o.ttft_p99 + j, m.ttft);
    if (o.tpot) __stcs(o.tpot + j, m.tpot);
    if (o.thr_decode) __stcs(o.thr_decode + j, m.thr);
    if (o.cost_per_hr) __stcs(o.cost_per_hr + j, m.cost_hr);
    if (o.cost_per_token) __stcs(o.cost_per_token + j, m.cost_tok);
    if (o.status) o.status[j] = (uint8_t)m.status;
    if (o.bmax) __stcs(o.bmax + j, m.bmax);
    if (o.n_iters) __stcs(o.n_iters + j, m.n_iters);
    if (o.n_req_iters) __stcs(o.n_req_iters + j, m.n_req_iters);
}

// One thread per config, nothing shared between configs.
template <int TIME_SUM>
__global__ void __launch_bounds__(256) k_closed_form_flat(DSpace s, Range r, int tp_model, guide_outputs o) {
    const u64 j = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= r.count) return;
    const Cfg c = decode_index(s, r.first + j);
    Metrics m;
    closed_form_eval<TIME_SUM>(s, c, tp_model, m);
    store_metrics(o, j, m);
}

// Tiled evaluation (see tiled.cuh): every valid config's metrics are stored.
template <int TIME_SUM>
__global__ void __launch_bounds__(256, 2) k_closed_form_tiled(DSpace s, Range r, int tp_model, u32 hf_chunk,
                                                              u32 tiles_per_mb, guide_outputs o) {
    tiled_visit<TIME_SUM>(s, r, tp_model, hf_chunk, tiles_per_mb, [&](bool valid, u64 j, const Metrics &m) {
        if (valid) store_metrics(o, j, m);
    });
}

int launch_closed_form(const DSpace &s, Range r, int time_model, int tp_model, const guide_outputs &o,
                       cudaStream_t st) {
    const u64 total = (u64)s.n_m * s.n_h * s.n_f * s.n_b * s.n_t * s.n_l;
    // The tiled kernel pays off when a (TP, length) plane fills warps and the range is (most of)
    // the space; slivers of the space go through the flat kernel.
    TileGeom g;
    const bool tiled = r.count * 2 >= total && tiled_geometry(s, (u64)num_sms() * 16, 1ull << 30, &g);
    if (!tiled) {
        const u64 blocks = (r.count + 255) / 256;
        if (blocks > 0x7FFFFFFFull) return fail(GUIDE_ERR_UNSUPPORTED, "range too large for one launch");
        if (time_model) k_closed_form_flat<1><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
        else k_closed_form_flat<0><<<(u32)blocks, 256, 0, st>>>(s, r, tp_model, o);
    } else {
        const dim3 grid(g.gx, g.splits);
        if (time_model) k_closed_form_tiled<1><<<grid, g.threads, 0, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, o);
        else k_closed_form_tiled<0><<<grid, g.threads, 0, st>>>(s, r, tp_model, g.hf_chunk, g.tiles_per_mb, o);
    }
    GUIDE_CUDA(cudaGetLastError());
    return GUIDE_OK;
}

}  // namespace guide
