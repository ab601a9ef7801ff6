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


# ---- training step (ring-allreduce reconstruction loss of Section IV-B on the full-size autoencoder) ----

def flat_grads(g):
    return np.concatenate([g[name].reshape(-1) for name, _ in A.param_shapes()])


@pytest.mark.parametrize("mu, K", [(61, 1), (100, 3), (130, 2)])
def test_training_gradients_against_torch_autograd(mu, K):
    # the same graph built from torch's CPU convolutions, differentiated by autograd
    rng = np.random.default_rng(mu + K)
    val = rng.standard_normal((K, mu)).astype(np.float32)
    flat = rand_params(mu)
    loss, g = A.rar_loss_and_grads(val, A.unpack(flat))
    tp = {k: torch.from_numpy(np.ascontiguousarray(v)).requires_grad_(True) for k, v in A.unpack(flat).items()}
    ln = A.lengths(mu)
    zs = []
    for k in range(K):
        h = torch.from_numpy(val[k].astype(np.float64)).reshape(1, 1, -1)
        for i in range(1, 5):
            h = F.leaky_relu(F.conv1d(h, tp[f"enc.w{i}"], tp[f"enc.b{i}"], stride=2), 0.01)
        zs.append(F.conv1d(h, tp["enc.w5"], tp["enc.b5"]))
    zbar = sum(zs[1:], zs[0]) / K
    d = F.leaky_relu(F.conv_transpose1d(zbar, tp["dec.w1"], tp["dec.b1"], stride=1, padding=1), 0.01)
    for i in range(2, 6):
        d = F.leaky_relu(F.conv_transpose1d(d, tp[f"dec.w{i}"], tp[f"dec.b{i}"], stride=2,
                                            output_padding=(ln[5 - i] - 3) % 2), 0.01)
    r = F.conv1d(d, tp["dec.w6"], tp["dec.b6"]).reshape(-1)
    target = torch.from_numpy(val.astype(np.float64)).sum(0) / K
    tl = ((r - target) ** 2).sum() / mu
    tl.backward()
    assert abs(loss - tl.item()) <= 1e-12 * max(1.0, abs(tl.item()))
    for name, _ in A.param_shapes():
        ref = tp[name].grad.numpy()
        assert np.abs(g[name] - ref).max() <= 1e-10 * max(1e-3, np.abs(ref).max()), name


def test_training_gradients_against_finite_differences():
    # central differences of the loss itself, on parameters drawn from every tensor
    rng = np.random.default_rng(17)
    mu, K = 75, 2
    val = rng.standard_normal((K, mu)).astype(np.float32)
    flat = rand_params(17)
    _, g = A.rar_loss_and_grads(val, A.unpack(flat))
    gf = flat_grads(g)
    pos, picks = 0, []
    for _, shape in A.param_shapes():
        n = int(np.prod(shape))
        picks += list(pos + rng.choice(n, size=min(3, n), replace=False))
        pos += n
    eps = 1e-6
    for i in picks:
        hi, lo = flat.copy(), flat.copy()
        hi[i] += eps
        lo[i] -= eps
        fd = (A.rar_loss_and_grads(val, A.unpack(hi))[0] - A.rar_loss_and_grads(val, A.unpack(lo))[0]) / (2 * eps)
        assert abs(fd - gf[i]) <= 1e-5 * max(1e-3, abs(gf[i])) + 1e-8, (i, fd, gf[i])


def test_training_loss_is_the_forward_pass_error_and_vanishes_for_a_perfect_decoder():
    rng = np.random.default_rng(4)
    val = rng.standard_normal((3, 90)).astype(np.float32)
    p = A.unpack(rand_params(4))
    loss, _ = A.rar_loss_and_grads(val, p)
    _, _, r = A.rar_forward(val, p)
    target = (val[0].astype(np.float64) + val[1] + val[2]) / 3.0
    assert abs(loss - np.sum((r - target) ** 2) / 90) <= 1e-15 * max(1.0, loss)
    # zero weights in the last layer and a target that equals its bias: loss 0, and only the
    # last layer's weights can have a gradient (which is zero too, the error being zero)
    flat = rand_params(5)
    q = A.unpack(flat)
    q["dec.w6"][...] = 0.0
    q["dec.b6"][...] = 0.25
    same = np.full((2, 90), 0.25, dtype=np.float32)
    loss, g = A.rar_loss_and_grads(same, q)
    assert loss == 0.0 and all(not g[name].any() for name, _ in A.param_shapes())


def test_training_step_moves_every_parameter_against_its_gradient():
    from oracle import OracleLGC
    numel = [60_000, 30_000]
    ora = OracleLGC(numel, 2, ae_kind="conv5", params=rand_params(8) * 0.5)
    rng = np.random.default_rng(8)
    ora.accumulate(rng.standard_normal((2, ora.N)).astype(np.float32))
    ora.topk(0)
    before = ora.get_params()
    _, g = ora.ae_loss_and_grads()
    loss = ora.ae_train_step()
    after = ora.get_params()
    gf = flat_grads(g)
    big = np.abs(gf) > 1e-5                    # |g| >> eps: the first Adam step is lr * sign(g)
    assert big.sum() > 1000
    assert np.allclose(after[big] - before[big], -1e-3 * np.sign(gf[big]), rtol=2e-3, atol=0)
    assert ora.ae_train_step() < loss          # and the loss goes down
