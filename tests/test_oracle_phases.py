"""Pins for the phase / layer-mode composition of the oracle (oracle/phases.py)."""
import numpy as np

from oracle import OracleLGC
from oracle.phases import OraclePhased, dense_mean
from paper_2103_08870_b200 import workloads as W

NUMEL = [9408, 20000, 4096, 70000, 5000]


def grads(K, t, scale=1.0):
    src = W.GradientSource(W.LayerTable("ph", NUMEL, [1, 2, 3, 1, 2]), K, seed=17)
    return src.step(t).numpy() * np.float32(scale)


def test_raw_phase_and_dense_layers_are_the_mean():
    K = 4
    g = grads(K, 0)
    params = {0: W.ae_init_params(8, 4, "rar", K, 3).numpy()}
    o = OraclePhased(NUMEL, ["ae"] * 5, K, params)
    upd, _ = o.step(g, "raw")
    assert np.abs(upd - g.astype(np.float64).mean(0)).max() <= 2e-7 * np.abs(g).max()      # fp32 sum of 4 terms
    assert np.array_equal(dense_mean(np.stack([g[0]] * 4)), g[0])                          # K a power of two: exact
    o = OraclePhased(NUMEL, ["dense", "ae", "ae", "ae", "topk"], K, {1: params[0]})
    upd, _ = o.step(g, "compressed", 1)
    assert np.array_equal(upd[:9408], dense_mean(g[:, :9408]))


def test_all_layers_through_the_autoencoder_equals_the_single_pipeline():
    K = 2
    params = W.ae_init_params(8, 4, "rar", K, 3).numpy()
    whole = OracleLGC(NUMEL, K, params=params.copy())
    comp = OraclePhased(NUMEL, ["ae"] * 5, K, {0: params.copy()})
    for t in range(3):
        g = grads(K, t)
        ref = whole.step(g, t % K)
        upd, _ = comp.step(g, "compressed", t % K)
        assert np.array_equal(upd, ref)


def test_topk_only_layer_sends_the_mean_of_the_kept_values_and_keeps_the_rest():
    K = 2
    params = W.ae_init_params(8, 4, "rar", K, 3).numpy()
    o = OraclePhased(NUMEL, ["dense", "ae", "ae", "ae", "topk"], K, {1: params})
    g = grads(K, 0)
    upd, _ = o.step(g, "compressed", 0)
    a = sum(NUMEL[:4])
    last = o.groups[-1]["o"]
    sent = np.flatnonzero(upd[a:])
    assert len(sent) == last.k_l[0] == 5
    # momentum correction on a first step: v = g; the kept entries are the leader's 5 largest |g| of the layer
    lead = np.sort(np.argsort(-np.abs(g[0, a:]), kind="stable")[:5])
    assert np.array_equal(sent, lead)
    assert np.allclose(upd[a:][lead], g[:, a:][:, lead].mean(0), rtol=1e-6)
    assert not last.v[:, lead].any() and np.array_equal(np.delete(last.v[1], lead), np.delete(g[1, a:], lead))
    # second phase: the autoencoder trains, the update of its layers is the sparse mean of the kept values
    upd2, losses = o.step(grads(K, 1), "topk_train", 1)
    assert len(losses) == 1 and losses[0] > 0
    ae = o.groups[1]["o"]
    assert np.count_nonzero(upd2[9408:a]) == ae.mu


def test_one_group_per_mode_equals_runs_when_the_modes_come_in_runs():
    # Section VI-A's table (first layer dense, last layer top-k only): every mode is one run, so grouping by
    # mode and grouping by run are the same pipelines: identical bits, both variants
    K = 3
    modes = ["dense", "ae", "ae", "ae", "topk"]
    for variant in ("rar", "ps"):
        params = W.ae_init_params(8, 4, variant, K, 3).numpy()
        runs = OraclePhased(NUMEL, modes, K, {1: params.copy()}, variant=variant)
        whole = OraclePhased(NUMEL, modes, K, {0: params.copy()}, grouping="modes", variant=variant)
        for t, phase in enumerate(["raw", "topk_train", "compressed", "compressed"]):
            g = grads(K, t, 300.0)
            a, la = runs.step(g, phase, t % K)
            b, lb = whole.step(g, phase, t % K)
            assert np.array_equal(a, b) and la == lb, (variant, t)
        assert np.array_equal(runs.groups[1]["o"].get_params(), whole.groups[1]["o"].get_params())


def test_layers_of_a_mode_that_are_apart_share_one_pipeline():
    # modes (ae, topk, ae, dense, ae): the three "ae" layers feed ONE autoencoder in layer order.  Moving the
    # layers so that each mode is a run (a permutation of the gradient's columns) gives the pinned case
    # above; the update must be the same numbers at the moved places, and the indices the same entries.
    K = 2
    modes = ["ae", "topk", "ae", "dense", "ae"]
    order = [0, 2, 4, 1, 3]                                   # ae, ae, ae, topk, dense
    off = np.concatenate([[0], np.cumsum(NUMEL)])
    cols = np.concatenate([np.arange(off[l], off[l + 1]) for l in order])
    params = W.ae_init_params(8, 4, "rar", K, 3).numpy()
    apart = OraclePhased(NUMEL, modes, K, {0: params.copy()}, grouping="modes")
    moved = OraclePhased([NUMEL[l] for l in order], [modes[l] for l in order], K, {0: params.copy()})
    assert [gr["mode"] for gr in apart.groups] == ["ae", "topk", "dense"] and apart.groups[0]["layers"] == [0, 2, 4]
    for t, phase in enumerate(["topk_train", "compressed", "compressed"]):
        g = grads(K, t, 300.0)
        a, la = apart.step(g, phase, t % K)
        b, lb = moved.step(np.ascontiguousarray(g[:, cols]), phase, t % K)
        assert np.array_equal(a[cols], b) and la == lb, t
        full = apart.full_row_indices(apart.groups[0])            # offsets inside the whole row
        assert np.array_equal(full[0], cols[moved.groups[0]["o"].idx[0]])
    ae = apart.groups[0]["o"]
    assert ae.mu == sum(ae.k_l) and len(ae.k_l) == 3
