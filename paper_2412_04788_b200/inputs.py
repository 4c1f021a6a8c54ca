"""Seeded synthetic inputs: deployment spaces and request traces.

This module only *draws numbers*: it holds none of the performance model's
arithmetic, so that the CUDA path and the CPU oracle (which share no code with
each other) can both be fed from it.  Everything is plain numpy arrays:

  space = {
    "models": uint32 [n_m, 10]  columns N, H, n_h, n_kv, I, V, g, w_b, a_b, kv_b
    "hw":     float64 [n_h, 5]  columns P (FLOP/s), BW (B/s), CBW (B/s), CLAT (s), PRICE ($/h/GPU)
    "hw_mem": uint64 [n_h]      device memory in bytes (1 GB = 10**9 B)
    "fw_f":   float64 [n_f, 8]  columns e_c[LINEAR,ATTN,ELEM], e_m[LINEAR,ATTN,ELEM], e_comm, t_ovh (s)
    "fw_i":   uint32 [n_f, 4]   columns flash, kv_block, reserve_permille, policy
    "batch":  uint32 [n_b]
    "tp":     uint32 [n_t]
    "pairs":  uint32 [n_l, 2]   (Lin, Lout)
  }
  trace = {"arrival": float64 [n], "in_len": uint32 [n], "out_len": uint32 [n]}

A config index enumerates the axes in mixed radix with the length pair fastest
and the model slowest: idx = ((((m*n_h + h)*n_f + f)*n_b + b)*n_t + t)*n_l + l.

Random numbers come from SplitMix64 used as a counter-based generator
(Steele, Lea & Flood 2014): the i-th draw of stream s under seed k is
mix(k*GAMMA + s*STREAM + (i+1)*GAMMA) and u = (x >> 11) * 2**-53.
"""
from __future__ import annotations

import numpy as np

SEED_BASE = 20241204
_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_STREAM = np.uint64(0xD1B54A32D192ED03)

GB = 10**9


def _mix(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def raw_u64(seed: int, stream: int, n: int) -> np.ndarray:
    """n 64-bit draws of (seed, stream)."""
    with np.errstate(over="ignore"):
        base = np.uint64(seed) * _GAMMA + np.uint64(stream) * _STREAM
        ctr = (np.arange(1, n + 1, dtype=np.uint64)) * _GAMMA + base
        return _mix(ctr)


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    """n doubles in [0, 1) with 53 random bits."""
    return (raw_u64(seed, stream, n) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)


def uniform(seed: int, stream: int, n: int, lo: float, hi: float) -> np.ndarray:
    return lo + (hi - lo) * uniform01(seed, stream, n)


def randint(seed: int, stream: int, n: int, lo: int, hi: int) -> np.ndarray:
    """n integers in [lo, hi] (inclusive)."""
    span = hi - lo + 1
    return (lo + np.floor(uniform01(seed, stream, n) * span)).astype(np.int64)


def normal01(seed: int, stream: int, n: int) -> np.ndarray:
    """Box-Muller from two uniform streams."""
    u1 = uniform01(seed, stream, n)
    u2 = uniform01(seed, stream + 1, n)
    return np.sqrt(-2.0 * np.log1p(-u1)) * np.cos(2.0 * np.pi * u2)


# ----------------------------------------------------------------------------------------------
# axis builders
# ----------------------------------------------------------------------------------------------

# the eight decoder shapes (N, H, n_h, n_kv, I, V, gated) spanning ~1.4B to ~69B parameters
SHAPES_8 = [
    (24, 2048, 16, 16, 8192, 50272, 0),
    (32, 2560, 32, 32, 10240, 50272, 0),
    (32, 4096, 32, 32, 11008, 32000, 1),
    (32, 4096, 32, 8, 14336, 128256, 1),
    (40, 5120, 40, 40, 13824, 32000, 1),
    (48, 6144, 48, 8, 16384, 32000, 1),
    (60, 7168, 56, 8, 20480, 32000, 1),
    (80, 8192, 64, 8, 28672, 32000, 1),
]

BATCHES_16 = [1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64, 96, 128, 192, 256]
LEN_GRID_8 = [64, 128, 256, 512, 1024, 2048, 4096, 8192]


def models_from_shapes(shapes, w_b=2, a_b=2, kv_b=2) -> np.ndarray:
    out = np.zeros((len(shapes), 10), dtype=np.uint32)
    for i, s in enumerate(shapes):
        out[i, :7] = s
        out[i, 7:] = (w_b, a_b, kv_b)
    return out


def seeded_models(seed: int, n: int) -> np.ndarray:
    """N~U{24..80}, H=128*U{16..64}, n_h=H/128, n_kv in {8, n_h}, I=256*round(U[2.5,4]*H/256),
    V in {32000, 128256}, gated, fp16 everywhere."""
    N = randint(seed, 10, n, 24, 80)
    hm = randint(seed, 11, n, 16, 64)
    H = 128 * hm
    n_h = hm
    gqa = raw_u64(seed, 12, n) & np.uint64(1)
    n_kv = np.where(gqa == 1, 8, n_h)
    ratio = uniform(seed, 13, n, 2.5, 4.0)
    I = 256 * np.rint(ratio * H / 256.0).astype(np.int64)
    big_v = raw_u64(seed, 14, n) & np.uint64(1)
    V = np.where(big_v == 1, 128256, 32000)
    out = np.zeros((n, 10), dtype=np.uint32)
    out[:, 0], out[:, 1], out[:, 2], out[:, 3] = N, H, n_h, n_kv
    out[:, 4], out[:, 5], out[:, 6] = I, V, 1
    out[:, 7:] = 2
    return out


def seeded_hw(seed: int, n: int, mem_gb=None, mem_choices=None, mem_range=None):
    """P~U[100,1000] TFLOP/s, BW~U[1,8] TB/s, CBW~U[50,900] GB/s, CLAT~U[1,10] us, PRICE~U[1,40] $/h.
    Memory: explicit list `mem_gb`, seeded pick from `mem_choices`, or whole GB ~U{lo..hi}."""
    hw = np.zeros((n, 5), dtype=np.float64)
    hw[:, 0] = uniform(seed, 20, n, 100.0, 1000.0) * 1e12
    hw[:, 1] = uniform(seed, 21, n, 1.0, 8.0) * 1e12
    hw[:, 2] = uniform(seed, 22, n, 50.0, 900.0) * 1e9
    hw[:, 3] = uniform(seed, 23, n, 1.0, 10.0) * 1e-6
    hw[:, 4] = uniform(seed, 24, n, 1.0, 40.0)
    if mem_gb is not None:
        gb = np.asarray(mem_gb, dtype=np.int64)
        assert gb.shape == (n,)
    elif mem_choices is not None:
        pick = randint(seed, 25, n, 0, len(mem_choices) - 1)
        gb = np.asarray(mem_choices, dtype=np.int64)[pick]
    else:
        lo, hi = mem_range
        gb = randint(seed, 25, n, lo, hi)
    return hw, (gb * GB).astype(np.uint64)


def seeded_fw(seed: int, n: int, kv_block: int = 16, reserve_permille: int = 100):
    """Per-class efficiencies and e_comm ~U[0.4,0.9], t_ovh~U[0,500] us, flash a seeded bit
    (profile 0 always has flash on), PREFILL_FIRST policy."""
    fw_f = np.zeros((n, 8), dtype=np.float64)
    for c in range(7):
        fw_f[:, c] = uniform(seed, 30 + c, n, 0.4, 0.9)
    fw_f[:, 7] = uniform(seed, 37, n, 0.0, 500.0) * 1e-6
    fw_i = np.zeros((n, 4), dtype=np.uint32)
    fw_i[:, 0] = (raw_u64(seed, 38, n) & np.uint64(1)).astype(np.uint32)
    fw_i[0, 0] = 1
    fw_i[:, 1] = kv_block
    fw_i[:, 2] = reserve_permille
    fw_i[:, 3] = 0
    return fw_f, fw_i


def pairs_grid(lins, louts) -> np.ndarray:
    """All (Lin, Lout) with Lout fastest."""
    return np.array([(a, b) for a in lins for b in louts], dtype=np.uint32)


def space_size(space) -> int:
    n = 1
    for k in ("models", "hw", "fw_f", "batch", "tp", "pairs"):
        n *= len(space[k])
    return n


def decode_index(space, idx: int):
    """(m, h, f, b, t, l) axis positions of a config index."""
    dims = [len(space[k]) for k in ("models", "hw", "fw_f", "batch", "tp", "pairs")]
    pos = []
    for d in reversed(dims):
        pos.append(idx % d)
        idx //= d
    return tuple(reversed(pos))


def hybrid_axis(n_gpus: int):
    """Every (dp, tp) with tp a power of two and dp * tp <= n_gpus, dp slowest: the candidate
    parallel configurations of the hybrid enumeration.  Returns (dp list, tp list)."""
    dps, tps = [], []
    for dp in range(1, n_gpus + 1):
        tp = 1
        while dp * tp <= n_gpus:
            dps.append(dp)
            tps.append(tp)
            tp *= 2
    return dps, tps


def _space(models, hw, hw_mem, fw_f, fw_i, batch, tp, pairs, dp=None, fw_chunk=None, fw_keep=None):
    """dp (optional): data-parallel degree per entry of the TP axis.  fw_chunk (optional): per
    framework (split_size, seg_tokens) = requests per prompt sub-batch, tokens per prompt segment;
    0 = whole batch / whole prompt.  fw_keep (optional): per framework, thousandths of the KV cache
    its eviction policy keeps (0 or 1000 = all of it)."""
    extra = {} if dp is None else {"dp": np.ascontiguousarray(dp, dtype=np.uint32)}
    if fw_keep is not None:
        extra["fw_keep"] = np.ascontiguousarray(fw_keep, dtype=np.uint32).reshape(len(fw_f))
    assert dp is None or len(dp) == len(tp)
    if fw_chunk is not None:
        extra["fw_chunk"] = np.ascontiguousarray(fw_chunk, dtype=np.uint32).reshape(len(fw_f), 2)
    return {**extra,
        "models": np.ascontiguousarray(models, dtype=np.uint32),
        "hw": np.ascontiguousarray(hw, dtype=np.float64),
        "hw_mem": np.ascontiguousarray(hw_mem, dtype=np.uint64),
        "fw_f": np.ascontiguousarray(fw_f, dtype=np.float64),
        "fw_i": np.ascontiguousarray(fw_i, dtype=np.uint32),
        "batch": np.ascontiguousarray(batch, dtype=np.uint32),
        "tp": np.ascontiguousarray(tp, dtype=np.uint32),
        "pairs": np.ascontiguousarray(pairs, dtype=np.uint32).reshape(-1, 2),
    }


# ----------------------------------------------------------------------------------------------
# traces
# ----------------------------------------------------------------------------------------------

def poisson_arrivals(seed: int, n: int, rate: float) -> np.ndarray:
    """Cumulative sum of exponential gaps -ln(1-u)/rate; non-decreasing by construction."""
    gaps = -np.log1p(-uniform01(seed, 40, n)) / rate
    return np.cumsum(gaps)


def lognormal_lengths(seed: int, stream: int, n: int, mu: float, sigma: float, clip: int) -> np.ndarray:
    z = normal01(seed, stream, n)
    x = np.rint(np.exp(mu + sigma * z))
    return np.clip(x, 1, clip).astype(np.uint32)


def make_trace(seed: int, n: int, rate: float, lengths: bool,
               in_clip: int = 8192, out_clip: int = 2048):
    """Poisson arrivals; lengths LogN(6,1) / LogN(5,1) clipped, or zeros (= take the config's pair)."""
    arrival = poisson_arrivals(seed, n, rate)
    if lengths:
        in_len = lognormal_lengths(seed, 50, n, 6.0, 1.0, in_clip)
        out_len = lognormal_lengths(seed, 60, n, 5.0, 1.0, out_clip)
    else:
        in_len = np.zeros(n, dtype=np.uint32)
        out_len = np.zeros(n, dtype=np.uint32)
    return {"arrival": np.ascontiguousarray(arrival, dtype=np.float64),
            "in_len": in_len, "out_len": out_len}


# ----------------------------------------------------------------------------------------------
# the five workloads
# ----------------------------------------------------------------------------------------------

def workload(k: int, scale: float = 1.0, trace_scale: float | None = None):
    """Workload k in 1..5 -> dict(space, trace or None, constraints, topk, name).

    `scale` < 1 shrinks the hardware axis and `trace_scale` (default: = scale) the trace, for
    quick parity cases that keep every other axis, value law and seed; 1 is the full size.
    """
    seed = SEED_BASE + k
    if trace_scale is None:
        trace_scale = scale
    if k == 1:
        models = models_from_shapes([SHAPES_8[2]])
        hw, mem = seeded_hw(seed, 4, mem_gb=[24, 48, 80, 192])
        fw_f, fw_i = seeded_fw(seed, 1)
        space = _space(models, hw, mem, fw_f, fw_i, [1, 2, 4, 8, 16, 32, 64], [1, 2, 4],
                       pairs_grid([128, 512, 2048], [128, 512]))
        trace = make_trace(seed, max(8, int(256 * trace_scale)), 4.0, lengths=False)
        cons = {"max_ttft": 0.5, "ttft_stat": "p99"}
        return {"name": "C1", "space": space, "trace": trace, "constraints": cons,
                "topk": {"key": "cost_per_token", "k": 8}}
    if k == 2:
        models = models_from_shapes(SHAPES_8)
        n_hw = max(1, int(16 * scale))
        hw, mem = seeded_hw(seed, n_hw, mem_choices=[24, 48, 80, 192])
        fw_f, fw_i = seeded_fw(seed, 3)
        space = _space(models, hw, mem, fw_f, fw_i, [1 << i for i in range(10)], [1, 2, 4, 8],
                       pairs_grid(LEN_GRID_8, LEN_GRID_8))
        return {"name": "C2", "space": space, "trace": None, "constraints": {},
                "topk": {"key": "cost_per_token", "k": 8}}
    if k == 3:
        models = models_from_shapes(SHAPES_8)
        n_hw = max(1, int(32 * scale))
        hw, mem = seeded_hw(seed, n_hw, mem_gb=[192] * n_hw)
        fw_f, fw_i = seeded_fw(seed, 4)
        space = _space(models, hw, mem, fw_f, fw_i, BATCHES_16, [1, 2, 4, 8], [(1, 1)])
        trace = make_trace(seed, max(8, int(4096 * trace_scale)), 16.0, lengths=True)
        return {"name": "C3", "space": space, "trace": trace, "constraints": {},
                "topk": {"key": "ttft_p99", "k": 8}}
    if k == 4:
        models = seeded_models(seed, 16)
        n_hw = max(1, int(256 * scale))
        hw, mem = seeded_hw(seed, n_hw, mem_range=(16, 192))
        fw_f, fw_i = seeded_fw(seed, 4)
        space = _space(models, hw, mem, fw_f, fw_i, BATCHES_16, [1, 2, 4, 8], [(1, 1)])
        trace = make_trace(seed, max(8, int(1024 * trace_scale)), 32.0, lengths=True)
        return {"name": "C4", "space": space, "trace": trace, "constraints": {},
                "topk": {"key": "ttft_p99", "k": 8}}
    if k == 5:
        models = seeded_models(seed, 16)
        n_hw = max(1, int(64 * scale))
        hw, mem = seeded_hw(seed, n_hw, mem_choices=[24, 48, 80, 192])
        fw_f, fw_i = seeded_fw(seed, 4)
        # 16 distinct sorted batch sizes in 1..512
        draws = randint(seed, 70, 4096, 1, 512)
        seen = []
        for v in draws.tolist():
            if v not in seen:
                seen.append(v)
            if len(seen) == 16:
                break
        batch = sorted(seen)
        space = _space(models, hw, mem, fw_f, fw_i, batch, [1, 2, 4, 8],
                       pairs_grid(LEN_GRID_8, LEN_GRID_8))
        slo = float(uniform(seed, 71, 1, 20.0, 120.0)[0])
        cons = {"max_latency": slo}
        return {"name": "C5", "space": space, "trace": None, "constraints": cons,
                "topk": {"key": "cost_per_token", "k": 64},
                "pareto": {"x": "latency", "y": "cost_per_hr"}}
    raise ValueError("workload must be 1..5")


def hybrid_workload(n_gpus: int = 8, n_hw: int = 8, n_fw: int = 3, seed_offset: int = 20):
    """Closed-form sweep whose parallelism axis is every (dp, tp) pair under a budget of n_gpus:
    the eight model shapes, seeded hardware and frameworks, batch sizes that are and are not
    multiples of the replica counts, the 8 x 8 length grid."""
    seed = SEED_BASE + seed_offset
    models = models_from_shapes(SHAPES_8)
    hw, mem = seeded_hw(seed, n_hw, mem_choices=[24, 48, 80, 192])
    fw_f, fw_i = seeded_fw(seed, n_fw)
    dp, tp = hybrid_axis(n_gpus)
    space = _space(models, hw, mem, fw_f, fw_i, [1, 2, 3, 5, 8, 16, 31, 64, 100, 256, 509, 1024], tp,
                   pairs_grid(LEN_GRID_8, LEN_GRID_8), dp=dp)
    return {"name": f"hybrid-{n_gpus}", "space": space, "trace": None, "constraints": {},
            "topk": {"key": "cost_per_token", "k": 64},
            "pareto": {"x": "latency", "y": "cost_per_hr"}}


def chunked_workload(scale: float = 0.5, n_gpus: int = 1):
    """Workload 2's sweep with frameworks that process prompts in pieces: profile 0 whole batches and
    prompts, profile 1 sub-batches of 4 requests and 512-token segments, profile 2 sub-batches of
    16 requests.  n_gpus > 1 replaces the TP axis by the (dp, tp) pairs under that budget."""
    w = workload(2, scale=scale)
    sp = dict(w["space"])
    sp["fw_chunk"] = np.array([[0, 0], [4, 512], [16, 0]], dtype=np.uint32)
    if n_gpus > 1:
        dp, tp = hybrid_axis(n_gpus)
        sp["dp"] = np.array(dp, dtype=np.uint32)
        sp["tp"] = np.array(tp, dtype=np.uint32)
    return {"name": "C2-chunked", "space": sp, "trace": None, "constraints": {},
            "topk": {"key": "cost_per_token", "k": 8}, "pareto": {"x": "latency", "y": "cost_per_hr"}}
