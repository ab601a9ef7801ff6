"""Pins for the oracle of the paper's full-size autoencoder (oracle/full_ae.py): the parameter
counts the two layer tables of Section IV-C imply, torch's CPU convolutions as the library
special case of every layer, direct loops on a tiny case, and the length chain."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import full_ae as A


def rand_params(seed=0):
    rng = np.random.default_rng(seed)
    return rng.uniform(-0.3, 0.3, size=A.param_count())


def test_parameter_counts_follow_the_layer_tables():
    # encoder: filters 64, 128, 256, 64 with kernels of 3 taps, then 4 filters of 1 tap
    enc = (64 * 1 * 3 + 64) + (128 * 64 * 3 + 128) + (256 * 128 * 3 + 256) + (64 * 256 * 3 + 64) + (4 * 64 + 4)
    # decoder: filters 4, 32, 64, 128, 32 with 3 taps (inputs 4, 4, 32, 64, 128), then one 1-tap filter
    dec = (4 * 4 * 3 + 4) + (4 * 32 * 3 + 32) + (32 * 64 * 3 + 64) + (64 * 128 * 3 + 128) + (128 * 32 * 3 + 32) + (32 + 1)
    assert (enc, dec) == (172_996, 43_733)
    assert A.param_count() == enc + dec
    names = [n for n, _ in A.param_shapes()]
    assert names[:2] == ["enc.w1", "enc.b1"] and names[-2:] == ["dec.w6", "dec.b6"]


@pytest.mark.parametrize("mu", [31, 32, 33, 34, 61, 100, 257, 1049])
def test_lengths_return_to_mu(mu):
    ln = A.lengths(mu)
    assert ln[0] == mu and all(ln[i + 1] == (ln[i] - 3) // 2 + 1 for i in range(4))
    p = A.unpack(rand_params())
    z = np.zeros((4, ln[4]))
    assert A.decode(z, p, mu).shape == (mu,)


def test_lengths_of_the_benchmark_shapes():
    assert A.lengths(25_617) == [25_617, 12_808, 6_403, 3_201, 1_600]
    assert A.lengths(107_374) == [107_374, 53_686, 26_842, 13_420, 6_709]


def torch_forward(val, flat):
    p = {k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in A.unpack(flat).items()}
    K, mu = val.shape
    ln = A.lengths(mu)
    zs = []
    for k in range(K):
        h = torch.from_numpy(val[k].astype(np.float64)).reshape(1, 1, -1)
        for i in range(1, 5):
            h = F.leaky_relu(F.conv1d(h, p[f"enc.w{i}"], p[f"enc.b{i}"], stride=2), 0.01)
        zs.append(F.conv1d(h, p["enc.w5"], p["enc.b5"]))
    zbar = sum(zs[1:], zs[0]) / K
    d = F.leaky_relu(F.conv_transpose1d(zbar, p["dec.w1"], p["dec.b1"], stride=1, padding=1), 0.01)
    for i in range(2, 6):
        op = (ln[5 - i] - 3) % 2
        d = F.leaky_relu(F.conv_transpose1d(d, p[f"dec.w{i}"], p[f"dec.b{i}"], stride=2, output_padding=op), 0.01)
    r = F.conv1d(d, p["dec.w6"], p["dec.b6"])
    return torch.cat(zs).numpy(), zbar[0].numpy(), r.reshape(-1).numpy()


@pytest.mark.parametrize("mu, K", [(61, 1), (100, 3), (257, 2), (1049, 2)])
def test_whole_autoencoder_against_torch_cpu(mu, K):
    rng = np.random.default_rng(mu)
    val = rng.standard_normal((K, mu)).astype(np.float32)
    flat = rand_params(mu)
    z, zbar, r = A.rar_forward(val, A.unpack(flat))
    tz, tzbar, tr = torch_forward(val, flat)
    for a, b in ((z, tz), (zbar, tzbar), (r, tr)):
        assert a.shape == b.shape
        assert np.abs(a - b).max() <= 1e-12 * max(1.0, np.abs(b).max())


def test_each_layer_kind_against_direct_loops():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((3, 11))
    w = rng.standard_normal((2, 3, 3))          # conv: [co][ci][tau]
    b = rng.standard_normal(2)
    y = A.conv_k3s2(x, w, b)
    assert y.shape == (2, 5)
    for co in range(2):
        for t in range(5):
            ref = b[co] + sum(w[co, ci, tau] * x[ci, 2 * t + tau] for ci in range(3) for tau in range(3))
            assert abs(y[co, t] - ref) < 1e-12
    wt = rng.standard_normal((3, 2, 3))         # transposed conv: [ci][co][tau]
    for op in (0, 1):
        y = A.convt_k3s2(x, wt, b, op)
        ref = np.tile(b.reshape(2, 1), (1, 2 * 10 + 3 + op))
        for ci in range(3):
            for co in range(2):
                for j in range(11):
                    for tau in range(3):
                        ref[co, 2 * j + tau] += wt[ci, co, tau] * x[ci, j]
        assert np.abs(y - ref).max() < 1e-12
    y = A.convt_k3s1p1(x, wt, b)
    ref = np.tile(b.reshape(2, 1), (1, 11))
    for ci in range(3):
        for co in range(2):
            for j in range(11):
                for tau in range(3):
                    s = j + tau - 1
                    if 0 <= s < 11:
                        ref[co, s] += wt[ci, co, tau] * x[ci, j]
    assert np.abs(y - ref).max() < 1e-12
    assert np.array_equal(A.leaky(np.array([-2.0, 0.0, 3.0])), np.array([-0.02, 0.0, 3.0]))


def test_identical_nodes_average_to_their_own_code():
    rng = np.random.default_rng(9)
    x = rng.standard_normal(200).astype(np.float32)
    p = A.unpack(rand_params(9))
    z, zbar, r = A.rar_forward(np.stack([x] * 4), p)
    assert np.array_equal(zbar, z[0])                       # K a power of two: exact
    assert np.array_equal(r, A.decode(A.encode(x, p), p, 200))
