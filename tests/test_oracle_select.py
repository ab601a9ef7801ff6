"""Pins for the oracle's accumulation, selection, gather and clearing (fp32, exact)."""
import os

import numpy as np
import pytest

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "layout_counts.txt")


def golden():
    return {l.split()[0]: int(l.split()[1]) for l in open(GOLDEN) if l.strip() and not l.startswith("#")}


def brute_topk(v, k):
    """Independent definition: python sort on (-|v| as integer key, index)."""
    keys = (v.view(np.uint32) & 0x7FFFFFFF).tolist()
    order = sorted(range(len(keys)), key=lambda j: (-keys[j], j))
    return np.array(sorted(order[:k]), dtype=np.int32)


def test_keep_count_rounding():
    g = golden()
    assert O.keep_count(1 << 20, 1000) == g["k_tiny"]
    assert O.keep_count(1 << 30, 100) == g["k_stress"]
    assert O.keep_count(64, 1000) == 1            # never zero
    assert O.keep_count(1499, 1000) == 1 and O.keep_count(1500, 1000) == 2   # half up
    assert O.keep_count(10, 2_000_000) == 10      # never above n
    assert O.innovation_count(1049, 100) == 105 and O.innovation_count(3, 100) == 1


@pytest.mark.parametrize("n,k", [(1, 1), (7, 3), (64, 1), (257, 9), (1000, 1000), (4096, 41)])
@pytest.mark.parametrize("method", ["sort", "select"])
def test_topk_against_brute_force(n, k, method):
    rng = np.random.default_rng(n * 31 + k)
    v = rng.standard_normal(n).astype(np.float32)
    assert np.array_equal(O.topk(v, k, method=method), brute_topk(v, k))
    assert np.array_equal(O.topk(v, k, base=100, method=method), brute_topk(v, k) + 100)


@pytest.mark.parametrize("method", ["sort", "select"])
def test_topk_ties_go_to_lower_index(method):
    v = np.full(50, -2.5, dtype=np.float32)
    assert O.topk(v, 7, method=method).tolist() == list(range(7))         # all equal
    v = np.array([1, -3, 3, 2, -3, 3, 0, 3], dtype=np.float32)
    assert O.topk(v, 3, method=method).tolist() == [1, 2, 4]              # |.| ties, sign ignored
    assert O.topk(v, 5, method=method).tolist() == [1, 2, 4, 5, 7]
    z = np.array([0.0, -0.0, 0.0, -0.0], dtype=np.float32)                # -0 and +0 tie
    assert O.topk(z, 2, method=method).tolist() == [0, 1]
    # few distinct values, many ties: against brute force
    rng = np.random.default_rng(5)
    v = rng.integers(-3, 4, size=3000).astype(np.float32)
    for k in (1, 10, 500, 2999):
        assert np.array_equal(O.topk(v, k, method=method), brute_topk(v, k))


def test_topk_denormals_and_order_by_bits():
    v = np.array([1e-45, -3e-45, 0.0, 1e-38, -1e-39], dtype=np.float32)
    assert O.topk(v, 2, method="sort").tolist() == [3, 4]
    assert O.topk(v, 3, method="select").tolist() == [1, 3, 4]


def test_topk_select_equals_sort_large_random():
    rng = np.random.default_rng(11)
    v = (rng.laplace(size=300_000) * 1e-3).astype(np.float32)
    v[rng.integers(0, v.size, 5000)] = v[0]       # a block of ties somewhere
    for k in (1, 300, 30_000):
        assert np.array_equal(O.topk(v, k, method="select"), O.topk(v, k, method="sort"))


def test_topk_properties_permutation_and_sign():
    rng = np.random.default_rng(2)
    v = rng.standard_normal(5000).astype(np.float32)
    k = 37
    idx = O.topk(v, k)
    assert idx.size == k and np.all(np.diff(idx) > 0)
    mask = np.zeros(v.size, bool)
    mask[idx] = True
    assert np.abs(v[mask]).min() >= np.abs(v[~mask]).max()
    assert np.array_equal(O.topk(-v, k), idx)                       # sign flip
    perm = rng.permutation(v.size)
    idx_p = O.topk(v[perm], k)
    assert set(perm[idx_p].tolist()) == set(idx.tolist())           # no ties: same set


def test_accumulate_closed_form_and_m0():
    n, m, steps = 1000, np.float32(0.9), 12
    rng = np.random.default_rng(0)
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    u = np.zeros(n, np.float32)
    v = np.zeros(n, np.float32)
    for t in range(1, steps + 1):
        O.accumulate(u, v, g, float(m))
        md = float(m)                                   # the fp32 momentum, as a real number
        u_exact = g.astype(np.float64) * (1 - md**t) / (1 - md)
        v_exact = g.astype(np.float64) * (t - md * (1 - md**t) / (1 - md)) / (1 - md)
        assert np.allclose(u, u_exact, rtol=1e-5, atol=0)
        assert np.allclose(v, v_exact, rtol=1e-5, atol=0)
    # m = 0: plain error feedback, v is the running sum of gradients, u the last gradient
    u[:] = 0
    v[:] = 0
    total = np.zeros(n, np.float32)
    for t in range(5):
        gt = (rng.standard_normal(n)).astype(np.float32)
        O.accumulate(u, v, gt, 0.0)
        total = total + gt
        assert np.array_equal(u, gt) and np.array_equal(v, total)


def test_accumulate_is_single_rounding_fma():
    # m*u + g with one rounding differs from two roundings for these operands
    m = np.float32(0.9)
    u0 = np.float32(1.0 + 2**-23)
    g = np.float32(-0.9)
    u = np.array([u0], np.float32)
    v = np.zeros(1, np.float32)
    O.accumulate(u, v, np.array([g], np.float32), float(m))
    fused = np.float32(np.float64(m) * np.float64(u0) + np.float64(g))   # exact product, one rounding
    two_step = np.float32(np.float32(m * u0) + g)
    assert fused != two_step, "operands must separate the two evaluation orders"
    assert u[0] == fused and v[0] == fused


def test_sent_plus_kept_equals_accumulated():
    rng = np.random.default_rng(4)
    n, k = 20_000, 20
    u = rng.standard_normal(n).astype(np.float32)
    v = rng.standard_normal(n).astype(np.float32)
    before = v.copy()
    idx = O.topk(v, k)
    val = O.gather(v, idx)
    O.clear(u, v, idx)
    sent = np.zeros(n, np.float32)
    sent[idx] = val
    assert np.array_equal((sent + v).view(np.uint32), before.view(np.uint32))   # bitwise
    assert np.all(v[idx] == 0) and np.all(u[idx] == 0)
    untouched = np.ones(n, bool)
    untouched[idx] = False
    assert np.array_equal(v[untouched], before[untouched])


def test_innovation_keeps_top_values_in_place():
    val = np.array([0.1, -5.0, 2.0, 5.0, -0.2, 3.0], dtype=np.float32)
    assert O.innovation(val, 2).tolist() == [0.0, -5.0, 0.0, 5.0, 0.0, 0.0]
    assert O.innovation(val, 1).tolist() == [0.0, -5.0, 0.0, 0.0, 0.0, 0.0]      # tie: lower position
    rng = np.random.default_rng(9)
    val = rng.standard_normal(500).astype(np.float32)
    inn = O.innovation(val, 50)
    keep = brute_topk(val, 50)
    ref = np.zeros_like(val)
    ref[keep] = val[keep]
    assert np.array_equal(inn, ref)
