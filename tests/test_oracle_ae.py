"""Pins for the oracle's autoencoder arithmetic: library routines, adjointness, special kernels."""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "layout_counts.txt")


def golden():
    return {l.split()[0]: int(l.split()[1]) for l in open(GOLDEN) if l.strip() and not l.startswith("#")}


def rnd(rng, *shape):
    return np.ascontiguousarray(rng.standard_normal(shape))


def test_lengths_mirror_back_to_mu():
    g = golden()
    mu = g["ae_len_mu"]
    l1 = O.conv_len(mu)
    l2 = O.conv_len(l1)
    assert (l1, l2) == (g["ae_len_l1"], g["ae_len_l2"])
    op1, op2 = (l1 - 3) % 2, (mu - 3) % 2
    assert O.convt_len(l2, op1) == l1 and O.convt_len(l1, op2) == mu
    for mu in range(7, 200):
        l1 = O.conv_len(mu)
        l2 = O.conv_len(l1)
        assert O.convt_len(O.convt_len(l2, (l1 - 3) % 2), (mu - 3) % 2) == mu


@pytest.mark.parametrize("cin,cout,lin", [(1, 8, 1049), (8, 4, 524), (3, 5, 3), (2, 2, 4), (16, 8, 77)])
def test_conv1d_equals_torch(cin, cout, lin):
    rng = np.random.default_rng(lin)
    x, w, b = rnd(rng, cin, lin), rnd(rng, cout, cin, 3), rnd(rng, cout)
    ref = F.conv1d(torch.from_numpy(x)[None], torch.from_numpy(w), torch.from_numpy(b), stride=2)[0].numpy()
    got = O.conv1d(x, w, b)
    assert got.shape == ref.shape
    assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("cin,cout,lin,op", [(4, 8, 261, 1), (8, 1, 524, 0), (2, 3, 1, 0), (3, 2, 5, 1)])
def test_convt1d_equals_torch(cin, cout, lin, op):
    rng = np.random.default_rng(lin + op)
    x, w, b = rnd(rng, cin, lin), rnd(rng, cin, cout, 3), rnd(rng, cout)
    ref = F.conv_transpose1d(torch.from_numpy(x)[None], torch.from_numpy(w), torch.from_numpy(b),
                             stride=2, output_padding=op)[0].numpy()
    got = O.convt1d(x, w, b, op)
    assert got.shape == ref.shape
    assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_delta_kernels():
    x = np.arange(1.0, 12.0).reshape(1, 11)
    for tau in range(3):
        w = np.zeros((1, 1, 3))
        w[0, 0, tau] = 1.0
        assert O.conv1d(x, w, np.zeros(1))[0].tolist() == x[0, tau::2][:5].tolist()      # strided subsample
        y = O.convt1d(x, w, np.zeros(1), 0)[0]
        ref = np.zeros(2 * 10 + 3)
        ref[tau:tau + 2 * 11:2] = x[0]                                                   # zero stuffing
        assert y.tolist() == ref.tolist()
    # the padded tail of a transposed convolution only sees the bias
    y = O.convt1d(x, np.ones((1, 1, 3)), np.array([0.25]), 1)[0]
    assert y[-1] == 0.25 and y.size == 24


def test_adjointness():
    rng = np.random.default_rng(3)
    cin, cout, lin = 3, 5, 41
    w = rnd(rng, cout, cin, 3)
    x = rnd(rng, cin, lin)
    y = rnd(rng, cout, O.conv_len(lin))
    # <conv(x), y> == <x, convT(y)> with the same weight tensor read as [cin_T=cout][cout_T=cin][3]
    lhs = np.sum(O.conv1d(x, w, np.zeros(cout)) * y)
    rhs = np.sum(x * O.convt1d(y, w, np.zeros(cin), (lin - 3) % 2))
    assert abs(lhs - rhs) <= 1e-12 * abs(lhs)


def test_conv_gradients_equal_autograd():
    rng = np.random.default_rng(8)
    cin, cout, lin = 3, 4, 30
    x, w, b = rnd(rng, cin, lin), rnd(rng, cout, cin, 3), rnd(rng, cout)
    dy = rnd(rng, cout, O.conv_len(lin))
    xt, wt, bt = (torch.from_numpy(a).clone().requires_grad_(True) for a in (x, w, b))
    (F.conv1d(xt[None], wt, bt, stride=2)[0] * torch.from_numpy(dy)).sum().backward()
    dw, db = np.zeros_like(w), np.zeros_like(b)
    dx = O.conv1d_bwd(x, w, dy, dw, db)
    for got, ref in ((dx, xt.grad), (dw, wt.grad), (db, bt.grad)):
        assert np.abs(got - ref.numpy()).max() <= 1e-12 * max(1.0, ref.abs().max().item())
    # accumulation: calling again doubles dw/db, dx is overwritten
    dx2 = O.conv1d_bwd(x, w, dy, dw, db)
    assert np.allclose(dw, 2 * wt.grad.numpy()) and np.allclose(dx2, dx)


@pytest.mark.parametrize("op", [0, 1])
def test_convt_gradients_equal_autograd(op):
    rng = np.random.default_rng(18 + op)
    cin, cout, lin = 4, 3, 17
    x, w, b = rnd(rng, cin, lin), rnd(rng, cin, cout, 3), rnd(rng, cout)
    dy = rnd(rng, cout, O.convt_len(lin, op))
    xt, wt, bt = (torch.from_numpy(a).clone().requires_grad_(True) for a in (x, w, b))
    (F.conv_transpose1d(xt[None], wt, bt, stride=2, output_padding=op)[0] * torch.from_numpy(dy)).sum().backward()
    dw, db = np.zeros_like(w), np.zeros_like(b)
    dx = O.convt1d_bwd(x, w, op, dy, dw, db)
    for got, ref in ((dx, xt.grad), (dw, wt.grad), (db, bt.grad)):
        assert np.abs(got - ref.numpy()).max() <= 1e-12 * max(1.0, ref.abs().max().item())


def test_relu_and_fuse():
    x = np.array([-1.0, 0.0, 2.0, -0.0])
    assert O.relu(x).tolist() == [0.0, 0.0, 2.0, 0.0]
    assert O.relu_bwd(np.array([0.0, 3.0, -1.0]), np.array([5.0, 6.0, 7.0])).tolist() == [0.0, 6.0, 0.0]
    y = np.array([1.0, 2.0])
    inn = np.array([0.5, 0.0], dtype=np.float32)
    assert O.ps_fuse(y, inn, 2.0, 4.0, 0.25).tolist() == [4.25, 4.25]


def test_adam_equals_torch_optim():
    rng = np.random.default_rng(21)
    p0 = rnd(rng, 50)
    p = p0.copy()
    m, v = np.zeros(50), np.zeros(50)
    pt = torch.from_numpy(p0.copy()).requires_grad_(True)
    opt = torch.optim.Adam([pt], lr=1e-3, betas=(0.9, 0.999), eps=1e-8)
    for t in range(1, 8):
        g = rnd(rng, 50) * 10.0 ** rng.integers(-6, 0)
        O.adam(p, m, v, g, t, 1e-3, 0.9, 0.999, 1e-8)
        pt.grad = torch.from_numpy(g.copy())
        opt.step()
        assert np.abs(p - pt.detach().numpy()).max() <= 1e-12
    # first step moves every parameter by lr * sign(g) (up to eps)
    p = np.zeros(3)
    O.adam(p, np.zeros(3), np.zeros(3), np.array([1e-3, -2.0, 5.0]), 1, 1e-3, 0.9, 0.999, 1e-8)
    assert np.allclose(p, [-1e-3, 1e-3, -1e-3], rtol=1e-4)
