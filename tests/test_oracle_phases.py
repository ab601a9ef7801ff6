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
