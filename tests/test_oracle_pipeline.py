"""Pins for the oracle's pipeline: invariants and special cases of the whole step."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as O
from oracle import OracleLGC
from paper_2103_08870_b200 import workloads as W

TOY = [4096, 64, 1500, 9000, 65, 127, 20000]     # ragged toy layer table


def grads(numel, K, steps, seed=5):
    src = W.GradientSource(W.LayerTable("toy", list(numel), [1] * len(numel)), K, seed=seed)
    return [src.step(t).numpy() for t in range(steps)]


def params(c1, c2, variant, K, seed=3):
    return W.ae_init_params(c1, c2, variant, K, seed).numpy()


def test_layout_counts():
    o = OracleLGC(TOY, 2)
    assert o.k_l == [4, 1, 2, 9, 1, 1, 20] and o.mu == 38
    assert o.ki_l == [1, 1, 1, 1, 1, 1, 2]


def test_identity_rar_round_trip_exact():
    K = 4
    gs = grads(TOY, K, 3)
    o = OracleLGC(TOY, K, ae_kind="identity")
    for t, g in enumerate(gs):
        o.accumulate(g)
        v_before = o.v.copy()
        o.topk(leader=t % K)
        idx = o.idx[0].copy()
        assert all(np.array_equal(o.idx[k], idx) for k in range(K))          # shared indices
        o.encode()
        o.combine()
        upd = o.decode_scatter()
        mean = v_before[:, idx].astype(np.float64).sum(0) / K
        assert np.array_equal(upd[idx], mean.astype(np.float32))
        rest = np.ones(o.N, bool)
        rest[idx] = False
        assert not upd[rest].any()
        assert not o.v[:, idx].any() and not o.u[:, idx].any()
        assert np.array_equal(o.v[:, rest], v_before[:, rest])


def test_identity_single_node_update_plus_residual_is_accumulated():
    gs = grads(TOY, 1, 4)
    for variant in ("rar", "ps"):
        o = OracleLGC(TOY, 1, variant=variant, ae_kind="identity", innovation_permille=0)
        for g in gs:
            o.accumulate(g)
            before = o.v[0].copy()
            o.topk(0)
            o.encode()
            o.combine(0)
            upd = o.decode_scatter()
            if variant == "rar":
                assert np.array_equal((upd + o.v[0]).view(np.uint32), before.view(np.uint32))


def test_ps_identity_k1_counts_value_twice_only_where_innovation():
    # K = 1, identity trunk, fusion (1,1,0): reconstruction = value + innovation at kept positions
    g = grads(TOY, 1, 1)[0]
    o = OracleLGC(TOY, 1, variant="ps", ae_kind="identity")
    o.accumulate(g)
    before = o.v[0].copy()
    o.topk()
    o.encode()
    o.combine(0)
    upd = o.decode_scatter()
    idx = o.idx[0]
    assert np.allclose(upd[idx], before[idx].astype(np.float64) + o.inn[0], rtol=1e-7)
    assert np.count_nonzero(o.inn[0]) == sum(o.ki_l)


def test_k_identical_nodes_mean_is_each_latent():
    K = 4
    g1 = grads(TOY, 1, 1)[0]
    g = np.repeat(g1, K, axis=0)
    o = OracleLGC(TOY, K, params=params(8, 4, "rar", K))
    o.accumulate(g)
    o.topk(2)
    o.encode()
    o.combine()
    assert np.array_equal(o.zbar, o.z[0])          # K a power of two: exact


def test_linear_autoencoder_commutes_with_mean():
    # bias-free and without the ReLU clipping (all pre-activations kept positive by a large
    # positive first-layer response) the encoder is linear: mean of latents = latent of mean.
    K, mu = 3, 57
    rng = np.random.default_rng(1)
    xs = rng.random((K, mu)) + 0.5                       # positive inputs
    w1 = np.abs(rng.standard_normal((8, 1, 3)))          # positive weights -> ReLU inactive
    w2 = rng.standard_normal((4, 8, 3))
    z = [O.conv1d(O.relu(O.conv1d(x[None], w1, np.zeros(8))), w2, np.zeros(4)) for x in xs]
    zm = O.conv1d(O.relu(O.conv1d(xs.mean(0)[None], w1, np.zeros(8))), w2, np.zeros(4))
    assert np.abs(sum(z) / K - zm).max() <= 1e-12 * np.abs(zm).max()


def test_rar_forward_equals_torch_modules():
    K = 3
    gs = grads(TOY, K, 2)
    p = params(8, 4, "rar", K)
    o = OracleLGC(TOY, K, params=p)
    for t, g in enumerate(gs):
        o.accumulate(g)
        o.topk(t)
        val, idx = o.val.copy(), o.idx[0].copy()
        o.encode()
        o.combine()
        upd = o.decode_scatter()
    tp = {k: torch.from_numpy(v) for k, v in o.p.items()}
    x = torch.from_numpy(val.astype(np.float64))[:, None, :]
    z = F.conv1d(F.relu(F.conv1d(x, tp["enc.w1"], tp["enc.b1"], stride=2)), tp["enc.w2"], tp["enc.b2"], stride=2)
    zbar = z.mean(0, keepdim=True)
    d = F.relu(F.conv_transpose1d(zbar, tp["dec.w1"], tp["dec.b1"], stride=2, output_padding=o.op1))
    r = F.conv_transpose1d(d, tp["dec.w2"], tp["dec.b2"], stride=2, output_padding=o.op2)[0, 0].numpy()
    assert r.shape == (o.mu,)
    assert np.abs(upd[idx] - r).max() <= 2e-7 * np.abs(r).max()            # fp32 rounding of the update


def test_ps_special_weights():
    K = 3
    g = grads(TOY, K, 1)[0]
    base = params(8, 4, "ps", K)

    def run(w0, w1, b):
        p = base.copy()
        o = OracleLGC(TOY, K, variant="ps", params=p)
        for k in range(K):
            o.p[f"dec{k}.fuse"][:] = (w0, w1, b)
        o.accumulate(g)
        o.topk()
        o.encode()
        o.combine(common_node=1)
        v_sel = [o.v[k, o.idx[k]].copy() for k in range(K)]
        upd = o.decode_scatter()
        return o, upd, v_sel

    # (0,1,0): the update is the node-ordered average of the innovations alone
    o, upd, _ = run(0.0, 1.0, 0.0)
    ref = np.zeros(o.N)
    for k in range(K):
        np.add.at(ref, o.idx[k], o.inn[k].astype(np.float64) / K)
    assert np.array_equal(upd, ref.astype(np.float32))
    assert np.count_nonzero(o.inn) == K * sum(o.ki_l)
    # (1,0,0): every node decodes the common code of node 1 with its own decoder
    o, upd, _ = run(1.0, 0.0, 0.0)
    ref = np.zeros(o.N)
    for k in range(K):
        d = O.relu(O.convt1d(o.z[1], o.p[f"dec{k}.w1"], o.p[f"dec{k}.b1"], o.op1))
        y = O.convt1d(d, o.p[f"dec{k}.w2"], o.p[f"dec{k}.b2"], o.op2)[0]
        np.add.at(ref, o.idx[k], y / K)
    assert np.allclose(upd, ref.astype(np.float32), rtol=1e-6, atol=1e-12)
    # per-node index sets differ but overlap (shared heavy-tailed component)
    s0, s1 = set(o.idx[0].tolist()), set(o.idx[1].tolist())
    assert s0 != s1 and len(s0 & s1) > 0
    # every node cleared its own positions
    for k in range(K):
        assert not o.v[k, o.idx[k]].any() and not o.u[k, o.idx[k]].any()


def test_ps_two_layer_decoder_fusion_is_a_concatenation_and_a_one_tap_convolution():
    # Section IV-C: the innovation is "concatenated ... before the final convolutional layer".  For the
    # two-layer decoders that reading is: decoder stack -> 1 channel, torch.cat with the innovation -> 2
    # channels -> Conv1d(2 -> 1, one tap) whose weights are the node's (w0, w1) and whose bias is b.
    # Built here from torch's own modules with random per-node scalars, none of the oracle's formula.
    K = 3
    g = grads(TOY, K, 1)[0] * 1e3
    o = OracleLGC(TOY, K, variant="ps", params=params(8, 4, "ps", K))
    rng = np.random.default_rng(17)
    for k in range(K):
        o.p[f"dec{k}.fuse"][:] = rng.uniform(-2.0, 2.0, 3)
    o.accumulate(g)
    o.topk()
    o.encode()
    o.combine(common_node=2)
    idx = o.idx.copy()
    upd = o.decode_scatter()
    tp = {k: torch.from_numpy(v.copy()) for k, v in o.p.items()}
    zc = torch.from_numpy(o.z[2])[None]
    ref = np.zeros(o.N)
    for k in range(K):
        d = F.relu(F.conv_transpose1d(zc, tp[f"dec{k}.w1"], tp[f"dec{k}.b1"], stride=2, output_padding=o.op1))
        y = F.conv_transpose1d(d, tp[f"dec{k}.w2"], tp[f"dec{k}.b2"], stride=2, output_padding=o.op2)     # [1][1][mu]
        two = torch.cat([y, torch.from_numpy(o.inn[k].astype(np.float64))[None, None]], dim=1)            # [1][2][mu]
        f = tp[f"dec{k}.fuse"]
        r = F.conv1d(two, f[:2].reshape(1, 2, 1), f[2:3])[0, 0].numpy()
        assert np.abs(o.r[k] - r).max() <= 1e-12 * np.abs(r).max(), k
        np.add.at(ref, idx[k], r / K)
    assert np.count_nonzero(o.inn) == K * sum(o.ki_l)                  # the second channel is not empty
    assert np.allclose(upd, ref.astype(np.float32), rtol=1e-6, atol=1e-12)


def test_training_gradients_by_finite_differences():
    K = 2
    g = grads(TOY, K, 1)[0] * 1e3                    # O(1) values: well-scaled differences
    o = OracleLGC(TOY, K, params=params(8, 4, "rar", K, seed=12))
    o.accumulate(g)
    o.topk(0)
    loss, gr = o.ae_loss_and_grads()
    flat_g = np.concatenate([gr[n].reshape(-1) for n, _ in o.order])
    flat_p = o.get_params()
    rng = np.random.default_rng(0)
    h = 1e-6
    for j in rng.choice(flat_p.size, 40, replace=False):
        pp, pm = flat_p.copy(), flat_p.copy()
        pp[j] += h
        pm[j] -= h
        o.set_params(pp)
        lp = o.ae_loss_and_grads()[0]
        o.set_params(pm)
        lm = o.ae_loss_and_grads()[0]
        fd = (lp - lm) / (2 * h)
        assert abs(fd - flat_g[j]) <= 1e-6 * max(1.0, abs(flat_g[j])) + 1e-7 * np.abs(flat_g).max(), j
    o.set_params(flat_p)


def test_training_gradients_equal_autograd_and_loss_falls():
    K = 2
    g = grads(TOY, K, 1)[0] * 1e3
    o = OracleLGC(TOY, K, params=params(8, 4, "rar", K, seed=12))
    o.accumulate(g)
    o.topk(1)
    loss, gr = o.ae_loss_and_grads()
    tp = {k: torch.from_numpy(v.copy()).requires_grad_(True) for k, v in o.p.items()}
    x = torch.from_numpy(o.val.astype(np.float64))[:, None, :]
    z = F.conv1d(F.relu(F.conv1d(x, tp["enc.w1"], tp["enc.b1"], stride=2)), tp["enc.w2"], tp["enc.b2"], stride=2)
    d = F.relu(F.conv_transpose1d(z.mean(0, keepdim=True), tp["dec.w1"], tp["dec.b1"], stride=2, output_padding=o.op1))
    r = F.conv_transpose1d(d, tp["dec.w2"], tp["dec.b2"], stride=2, output_padding=o.op2)
    tl = ((r[0, 0] - x[:, 0].mean(0)) ** 2).mean()
    tl.backward()
    assert abs(loss - tl.item()) <= 1e-12 * tl.item()
    for name, _ in o.order:
        ref = tp[name].grad.numpy()
        assert np.abs(gr[name] - ref).max() <= 1e-10 * max(1e-3, np.abs(ref).max()), name
    # zero training steps leave inference untouched; training lowers the loss
    losses = [o.ae_train_step() for _ in range(50)]
    assert losses[0] == loss
    assert losses[-1] < 0.95 * losses[0]
    assert all(b < a for a, b in zip(losses, losses[1:]))          # falls at every step
    assert o.adam_t == 50


def ps_training_oracle(K=3, seed=12):
    g = grads(TOY, K, 1)[0] * 1e3
    o = OracleLGC(TOY, K, variant="ps", params=params(8, 4, "ps", K, seed=seed))
    for k in range(K):                                # fusion scalars away from their (1, 1, 0) start
        o.p[f"dec{k}.fuse"][:] = (0.8 + 0.1 * k, 0.6 - 0.1 * k, 0.05 * k)
    o.accumulate(g)
    o.topk()
    return o


def test_ps_training_gradients_by_finite_differences():
    o = ps_training_oracle()
    loss, rec, sim, gr = o.ae_loss_and_grads_ps(1, 0.7, 0.3)
    assert abs(loss - (0.7 * rec + 0.3 * sim)) <= 1e-12 * loss
    flat_g = np.concatenate([gr[n].reshape(-1) for n, _ in o.order])
    flat_p = o.get_params()
    rng = np.random.default_rng(1)
    h = 1e-6
    fuse = [i for i in range(flat_p.size - 3, flat_p.size)]          # the last node's fusion scalars
    for j in list(rng.choice(flat_p.size, 60, replace=False)) + fuse:
        pp, pm = flat_p.copy(), flat_p.copy()
        pp[j] += h
        pm[j] -= h
        o.set_params(pp)
        lp = o.ae_loss_and_grads_ps(1, 0.7, 0.3)[0]
        o.set_params(pm)
        lm = o.ae_loss_and_grads_ps(1, 0.7, 0.3)[0]
        fd = (lp - lm) / (2 * h)
        assert abs(fd - flat_g[j]) <= 1e-6 * max(1.0, abs(flat_g[j])) + 1e-7 * np.abs(flat_g).max(), j
    o.set_params(flat_p)


def test_ps_training_loss_and_gradients_equal_autograd():
    K = 3
    o = ps_training_oracle(K)
    c = 2
    loss, rec, sim, gr = o.ae_loss_and_grads_ps(c, 1.0, 1.0)
    tp = {k: torch.from_numpy(v.copy()).requires_grad_(True) for k, v in o.p.items()}
    x = torch.from_numpy(o.val.astype(np.float64))[:, None, :]
    z = F.conv1d(F.relu(F.conv1d(x, tp["enc.w1"], tp["enc.b1"], stride=2)), tp["enc.w2"], tp["enc.b2"], stride=2)
    t_sim = sum(((z[k] - z[m]) ** 2).sum() for k in range(K) for m in range(K) if m != k) / z[0].numel()
    t_rec = 0.0
    for k in range(K):
        inn = np.zeros(o.mu)
        for l in range(o.L):
            a, b = int(o.koff[l]), int(o.koff[l + 1])
            inn[a:b] = O.innovation(o.val[k, a:b], o.ki_l[l])
        d = F.relu(F.conv_transpose1d(z[c:c + 1], tp[f"dec{k}.w1"], tp[f"dec{k}.b1"], stride=2, output_padding=o.op1))
        y = F.conv_transpose1d(d, tp[f"dec{k}.w2"], tp[f"dec{k}.b2"], stride=2, output_padding=o.op2)[0, 0]
        f = tp[f"dec{k}.fuse"]
        r = f[0] * y + f[1] * torch.from_numpy(inn) + f[2]
        t_rec = t_rec + ((r - x[k, 0]) ** 2).sum() / o.mu
    tl = t_rec + t_sim
    tl.backward()
    assert abs(rec - t_rec.item()) <= 1e-12 * t_rec.item() and abs(sim - t_sim.item()) <= 1e-12 * t_sim.item()
    for name, _ in o.order:
        ref = tp[name].grad.numpy()
        assert np.abs(gr[name] - ref).max() <= 1e-10 * max(1e-3, np.abs(ref).max()), name


def test_ps_training_special_cases():
    # one node: no pairs, L_sim = 0 and the loss is the reconstruction term alone
    g = grads(TOY, 1, 1)[0] * 1e3
    o = OracleLGC(TOY, 1, variant="ps", params=params(8, 4, "ps", 1, seed=3))
    o.accumulate(g)
    o.topk()
    loss, rec, sim, _ = o.ae_loss_and_grads_ps(0, 1.0, 5.0)
    assert sim == 0.0 and loss == rec
    # identical nodes: all codes coincide, L_sim = 0 and its gradient vanishes: with lam_rec = 0 nothing moves
    K = 3
    o = OracleLGC(TOY, K, variant="ps", params=params(8, 4, "ps", K, seed=3))
    o.accumulate(np.repeat(g, K, axis=0))
    o.topk()
    loss, rec, sim, gr = o.ae_loss_and_grads_ps(1, 0.0, 1.0)
    assert sim == 0.0 and loss == 0.0 and all(not v.any() for v in gr.values())
    # training lowers the loss
    o = ps_training_oracle()
    losses = [o.ae_train_step_ps(t % 3) for t in range(40)]
    assert losses[-1] < 0.95 * losses[0] and o.adam_t == 40


def test_momentum_zero_is_plain_error_feedback():
    K = 2
    gs = grads(TOY, K, 3)
    o = OracleLGC(TOY, K, momentum=0.0, ae_kind="identity")
    resid = np.zeros((K, o.N), np.float32)
    for t, g in enumerate(gs):
        acc = resid + g                               # g_l = grad + g_acc
        o.accumulate(g)
        assert np.array_equal(o.v, acc)
        o.topk(t % K)
        o.encode(); o.combine(); o.decode_scatter()
        resid = acc.copy()
        resid[:, o.idx[0]] = 0                        # only the unsent part stays
        assert np.array_equal(o.v, resid)


def test_ps_innovation_positions_are_the_slots_of_the_nonzero_innovation_entries():
    # the innovation keeps, per layer, the kI_l kept values of largest magnitude: its positions list
    # is ascending inside each layer, has kI_l entries per layer, and names exactly the slots where
    # the innovation vector is non-zero (random values: no kept value is zero)
    from oracle import OracleLGC
    numel = [3000, 800, 64, 5000]
    rng = np.random.default_rng(12)
    ora = OracleLGC(numel, 2, density_ppm=20000, variant="ps", ae_kind="identity")
    ora.accumulate(rng.standard_normal((2, ora.N)).astype(np.float32))
    ora.topk()
    ora.encode()
    ora.combine(0)
    kioff = np.concatenate([[0], np.cumsum(ora.ki_l)])
    for k in range(2):
        assert np.array_equal(np.flatnonzero(ora.inn[k]), np.sort(ora.inn_pos[k]))
        for l in range(len(numel)):
            seg = ora.inn_pos[k, kioff[l]:kioff[l + 1]]
            assert len(seg) == ora.ki_l[l] and np.all(np.diff(seg) > 0)
            assert ora.koff[l] <= seg[0] and seg[-1] < ora.koff[l + 1]
            kept = np.abs(ora.val[k, ora.koff[l]:ora.koff[l + 1]])
            assert np.sort(kept)[::-1][:ora.ki_l[l]].min() == np.abs(ora.val[k, seg]).min()
