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


# ---- parameter-server form (Section IV-A): one decoder per node, the innovation as a 33rd channel ----

def rand_params_ps(K, seed=0):
    rng = np.random.default_rng(seed)
    n = sum(int(np.prod(s)) for _, s in A.param_shapes_ps(K))
    return rng.uniform(-0.3, 0.3, size=n)


def unpack_ps(flat, K):
    out, pos = {}, 0
    for name, shape in A.param_shapes_ps(K):
        n = int(np.prod(shape))
        out[name] = flat[pos:pos + n].reshape(shape)
        pos += n
    assert pos == flat.size
    return out


def test_ps_parameter_count_one_encoder_and_one_decoder_per_node():
    shapes = A.param_shapes_ps(3)
    assert sum(int(np.prod(s)) for _, s in shapes) == 172_996 + 3 * (43_733 + 1)    # the last filter has one more tap
    assert [n for n, _ in shapes if n.endswith(".w6")] == ["dec0.w6", "dec1.w6", "dec2.w6"]


def test_ps_decoder_against_torch_concatenation():
    # the definition itself with torch's CPU ops: transposed convolutions, then torch.cat of the 32
    # feature channels with the innovation, then a 1-tap convolution over 33 channels
    rng = np.random.default_rng(21)
    mu, K = 130, 2
    p = unpack_ps(rand_params_ps(K, 21), K)
    z = rng.standard_normal((4, A.lengths(mu)[4]))
    inn = np.where(rng.random((K, mu)) < 0.1, rng.standard_normal((K, mu)), 0.0).astype(np.float32)
    ln = A.lengths(mu)
    for k in range(K):
        tp = {n[len(f"dec{k}."):]: torch.from_numpy(np.ascontiguousarray(v)) for n, v in p.items() if n.startswith(f"dec{k}.")}
        d = F.leaky_relu(F.conv_transpose1d(torch.from_numpy(z)[None], tp["w1"], tp["b1"], stride=1, padding=1), 0.01)
        for i in range(2, 6):
            d = F.leaky_relu(F.conv_transpose1d(d, tp[f"w{i}"], tp[f"b{i}"], stride=2, output_padding=(ln[5 - i] - 3) % 2), 0.01)
        cat = torch.cat([d, torch.from_numpy(inn[k].astype(np.float64))[None, None]], dim=1)
        ref = F.conv1d(cat, tp["w6"], tp["b6"]).reshape(-1).numpy()
        got = A.decode(z, p, mu, prefix=f"dec{k}", inn=inn[k])
        assert np.abs(got - ref).max() <= 1e-12 * max(1.0, np.abs(ref).max())


def test_ps_special_last_filters():
    from oracle import OracleLGC
    numel = [60_000, 30_000]
    K = 3
    flat = rand_params_ps(K, 3)
    p = unpack_ps(flat, K)
    rng = np.random.default_rng(3)
    g = rng.standard_normal((K, sum(numel))).astype(np.float32)

    def run(params):
        ora = OracleLGC(numel, K, variant="ps", ae_kind="conv5", params=params)
        ora.accumulate(g)
        ora.topk()
        ora.encode()
        ora.combine(1)
        ora.decode()
        return ora

    # (a) last filter = the innovation channel alone: every node reconstructs exactly its innovation
    for k in range(K):
        p[f"dec{k}.w6"][...] = 0.0
        p[f"dec{k}.w6"][0, 32, 0] = 1.0
        p[f"dec{k}.b6"][...] = 0.0
    ora = run(flat)
    assert np.array_equal(ora.r, ora.inn.astype(np.float64))
    # (b) the innovation channel switched off and all decoders alike: every node gets the ring-allreduce
    # decoder's output for the common node's code
    flat2 = rand_params_ps(K, 4)
    q = unpack_ps(flat2, K)
    for k in range(K):
        for name in ("w1", "b1", "w2", "b2", "w3", "b3", "w4", "b4", "w5", "b5", "w6", "b6"):
            q[f"dec{k}.{name}"][...] = q[f"dec0.{name}"]
        q[f"dec{k}.w6"][0, 32, 0] = 0.0
    ora = run(flat2)
    rar = {n.replace("dec0.", "dec."): v for n, v in q.items() if n.startswith("dec0.") or n.startswith("enc.")}
    rar["dec.w6"] = rar["dec.w6"][:, :32, :]
    ref = A.decode(ora.z[1], rar, ora.mu)
    for k in range(K):
        assert np.array_equal(ora.r[k], ref)
    assert np.array_equal(ora.zc, ora.z[1])


def ps_flat_grads(g, K):
    return np.concatenate([g[name].reshape(-1) for name, _ in A.param_shapes_ps(K)])


def test_ps_training_gradients_against_torch_autograd():
    rng = np.random.default_rng(31)
    mu, K, common = 100, 3, 1
    val = rng.standard_normal((K, mu)).astype(np.float32)
    inn = np.where(rng.random((K, mu)) < 0.1, val, 0.0).astype(np.float32)
    flat = rand_params_ps(K, 31)
    loss, rec, sim, g = A.ps_loss_and_grads(val, inn, unpack_ps(flat, K), common, 0.7, 0.3)
    tp = {k: torch.from_numpy(np.ascontiguousarray(v)).requires_grad_(True) for k, v in unpack_ps(flat, K).items()}
    ln = A.lengths(mu)
    zs = []
    for k in range(K):
        h = torch.from_numpy(val[k].astype(np.float64)).reshape(1, 1, -1)
        for i in range(1, 5):
            h = F.leaky_relu(F.conv1d(h, tp[f"enc.w{i}"], tp[f"enc.b{i}"], stride=2), 0.01)
        zs.append(F.conv1d(h, tp["enc.w5"], tp["enc.b5"]))
    tsim = sum(((zs[k] - zs[m]) ** 2).sum() for k in range(K) for m in range(K) if m != k) / zs[0].numel()
    trec = 0.0
    for k in range(K):
        d = F.leaky_relu(F.conv_transpose1d(zs[common], tp[f"dec{k}.w1"], tp[f"dec{k}.b1"], stride=1, padding=1), 0.01)
        for i in range(2, 6):
            d = F.leaky_relu(F.conv_transpose1d(d, tp[f"dec{k}.w{i}"], tp[f"dec{k}.b{i}"], stride=2,
                                                output_padding=(ln[5 - i] - 3) % 2), 0.01)
        cat = torch.cat([d, torch.from_numpy(inn[k].astype(np.float64))[None, None]], dim=1)
        r = F.conv1d(cat, tp[f"dec{k}.w6"], tp[f"dec{k}.b6"]).reshape(-1)
        trec = trec + ((r - torch.from_numpy(val[k].astype(np.float64))) ** 2).sum() / mu
    tl = 0.7 * trec + 0.3 * tsim
    tl.backward()
    assert abs(loss - tl.item()) <= 1e-12 * abs(tl.item()) and abs(rec - trec.item()) <= 1e-12 * rec
    assert abs(sim - tsim.item()) <= 1e-12 * sim
    for name, _ in A.param_shapes_ps(K):
        ref = tp[name].grad.numpy()
        assert np.abs(g[name] - ref).max() <= 1e-10 * max(1e-3, np.abs(ref).max()), name


def test_ps_training_similarity_term_vanishes_for_one_node_and_for_identical_nodes():
    rng = np.random.default_rng(33)
    mu = 80
    x = rng.standard_normal(mu).astype(np.float32)
    inn = np.where(rng.random(mu) < 0.1, x, 0.0).astype(np.float32)
    _, _, sim, _ = A.ps_loss_and_grads(x[None], inn[None], unpack_ps(rand_params_ps(1, 1), 1), 0)
    assert sim == 0.0
    _, _, sim, g = A.ps_loss_and_grads(np.stack([x] * 3), np.stack([inn] * 3), unpack_ps(rand_params_ps(3, 2), 3), 2, 0.0, 1.0)
    assert sim == 0.0 and not any(v.any() for v in g.values())        # lam_rec = 0: nothing else contributes


def test_ps_training_gradients_against_finite_differences():
    rng = np.random.default_rng(35)
    mu, K = 70, 2
    val = rng.standard_normal((K, mu)).astype(np.float32)
    inn = np.where(rng.random((K, mu)) < 0.1, val, 0.0).astype(np.float32)
    flat = rand_params_ps(K, 35)
    _, _, _, g = A.ps_loss_and_grads(val, inn, unpack_ps(flat, K), 0, 1.0, 0.5)
    gf = ps_flat_grads(g, K)
    pos, picks = 0, []
    for _, shape in A.param_shapes_ps(K):
        n = int(np.prod(shape))
        picks += list(pos + rng.choice(n, size=min(2, n), replace=False))
        pos += n
    eps = 1e-6
    for i in picks:
        hi, lo = flat.copy(), flat.copy()
        hi[i] += eps
        lo[i] -= eps
        fd = (A.ps_loss_and_grads(val, inn, unpack_ps(hi, K), 0, 1.0, 0.5)[0]
              - A.ps_loss_and_grads(val, inn, unpack_ps(lo, K), 0, 1.0, 0.5)[0]) / (2 * eps)
        assert abs(fd - gf[i]) <= 1e-5 * max(1e-3, abs(gf[i])) + 1e-8, (i, fd, gf[i])


def test_layer_shapes_follow_the_tables_of_the_paper():
    # tests/golden/full_ae_layers.txt restates the two tables of Section IV-C; every tensor of the oracle, and of
    # the seeded initialiser the tests and the benchmark use, must have the filters and taps printed there, each
    # layer taking as many input channels as the layer before it has filters (1 for conv1, 4 = the code for deconv1)
    import os
    from paper_2103_08870_b200 import workloads as W
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "full_ae_layers.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                side, layer, filters, taps, stride = line.split()
                rows.append((side, layer, int(filters), int(taps), int(stride)))
    assert len(rows) == 11
    shapes = dict(A.param_shapes())
    init_shapes = {n: s for n, s, _ in W.ae5_param_shapes()}
    prev = {"enc": 1, "dec": 4}
    for i, (side, layer, filters, taps, stride) in enumerate(rows):
        n = i + 1 if side == "enc" else i - 4
        w = shapes[f"{side}.w{n}"]
        transposed = layer.startswith("deconv")
        want = (prev[side], filters, taps) if transposed else (filters, prev[side], taps)
        assert w == want and shapes[f"{side}.b{n}"] == (filters,), (layer, w, want)
        assert init_shapes[f"{side}.w{n}"] == want
        prev[side] = filters
    assert rows[4][2] == 4                                   # the code the decoder starts from has conv5's 4 channels
    assert [r[4] for r in rows if r[3] == 3] == [2] * 9      # as printed; deconv1's stride is the documented reading


def test_one_dimensional_kernels_save_about_sixty_per_cent_of_the_parameters():
    # Section IV-C: 1-D kernels reduce the number of network parameters "by approximately 60 %" against
    # conventional 2-D (3 x 3) kernels.  With the tables' layers: 216,729 against 648,057 parameters, 66.6 % fewer.
    one_d = A.param_count()
    two_d = sum(int(np.prod(s)) * (3 if len(s) == 3 and s[2] == 3 else 1) for _, s in A.param_shapes())
    assert (one_d, two_d) == (216_729, 648_057)
    assert 0.55 < 1.0 - one_d / two_d < 0.70
