"""The seeded generator: published SplitMix64 outputs, determinism, workload shapes."""
import numpy as np

from paper_2412_04788_b200 import inputs as I


def test_splitmix64_known_answer():
    # first outputs of the published SplitMix64 for state 1234567 (state += gamma, then mix)
    want = [6457827717110365317, 3203168211198807973, 9817491932198370423]
    s = np.uint64(1234567)
    got = []
    with np.errstate(over="ignore"):
        for _ in range(3):
            s = s + I._GAMMA
            got.append(int(I._mix(np.array([s]))[0]))
    assert got == want


def test_uniform_range_and_determinism():
    u = I.uniform01(7, 3, 10000)
    assert u.min() >= 0.0 and u.max() < 1.0
    assert abs(u.mean() - 0.5) < 0.02
    assert np.array_equal(u, I.uniform01(7, 3, 10000))
    assert not np.array_equal(u, I.uniform01(7, 4, 10000))
    # counter based: a prefix of a longer draw is the shorter draw
    assert np.array_equal(u[:100], I.uniform01(7, 3, 100))


def test_workload_sizes():
    sizes = {1: 504, 2: 983040, 3: 65536, 4: 1048576, 5: 16777216}
    reqs = {1: 256, 2: None, 3: 4096, 4: 1024, 5: None}
    for k in range(1, 6):
        w = I.workload(k)
        assert I.space_size(w["space"]) == sizes[k]
        assert (None if w["trace"] is None else len(w["trace"]["arrival"])) == reqs[k]


def test_trace_laws():
    tr = I.workload(3)["trace"]
    assert np.all(np.diff(tr["arrival"]) >= 0)
    assert 1 <= tr["in_len"].min() and tr["in_len"].max() <= 8192
    assert 1 <= tr["out_len"].min() and tr["out_len"].max() <= 2048
    # lognormal(6,1) has mean exp(6.5) ~ 665 before clipping, lognormal(5,1) ~ 245
    assert 550 < tr["in_len"].mean() < 750
    assert 200 < tr["out_len"].mean() < 280
    rate = len(tr["arrival"]) / tr["arrival"][-1]
    assert 14.0 < rate < 18.0


def test_decode_index_order():
    sp = I.workload(1)["space"]
    assert I.decode_index(sp, 0) == (0, 0, 0, 0, 0, 0)
    assert I.decode_index(sp, 1) == (0, 0, 0, 0, 0, 1)          # length pair fastest
    assert I.decode_index(sp, 6) == (0, 0, 0, 0, 1, 0)          # then TP
    assert I.decode_index(sp, 503) == (0, 3, 0, 6, 2, 5)
    w5 = I.workload(5)
    assert len(set(w5["space"]["batch"].tolist())) == 16
    assert list(w5["space"]["batch"]) == sorted(w5["space"]["batch"])


def test_hybrid_axis_enumerates_the_gpu_budget():
    dp, tp = I.hybrid_axis(8)
    pairs = set(zip(dp, tp))
    assert len(pairs) == len(dp) == 15
    want = {(d, t) for d in range(1, 9) for t in (1, 2, 4, 8) if d * t <= 8}
    assert pairs == want
    assert I.hybrid_axis(1) == ([1], [1])
    w = I.hybrid_workload(8)["space"]
    assert w["dp"].dtype == np.uint32 and len(w["dp"]) == len(w["tp"])
    assert (len(w["tp"]) * len(w["pairs"])) % 4 == 0
