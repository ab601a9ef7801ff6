"""The three phases of Section V-B with the layer treatment of Section VI-A (first layer dense, last
layer top-k only, autoencoder in between): the composed CUDA path against the composed oracle."""
import numpy as np
import pytest
import torch

from oracle.phases import OraclePhased
from paper_2103_08870_b200 import lgc
from paper_2103_08870_b200 import workloads as W
from paper_2103_08870_b200.phases import PhasedLGC, layer_runs

from parity import assert_bitwise, assert_close

pytestmark = pytest.mark.gpu

NUMEL = [9408, 20000, 4096, 70000, 65, 127, 5000]
MODES = ["dense", "ae", "ae", "ae", "ae", "ae", "topk"]      # the runs start at multiples of 4 elements


def test_layer_runs():
    runs = layer_runs(NUMEL, MODES)
    assert [(r.mode, r.first, r.last, r.begin, r.end) for r in runs] == [
        ("dense", 0, 1, 0, 9408), ("ae", 1, 6, 9408, 103696), ("topk", 6, 7, 103696, 108696)]


def compare_state_and_slots(gpu, ora, what):
    """Residuals, velocities and index slots of a context with per-layer modes against the oracle's groups."""
    c = gpu.ctx if hasattr(gpu, "ctx") else gpu
    u, v, idx = c.u.cpu().numpy(), c.v.cpu().numpy(), c.idx.cpu().numpy()
    for gr in ora.groups:
        cols = np.concatenate([np.arange(a, b) for a, b in gr["ranges"]])
        if gr["mode"] == "dense":
            assert not u[:, cols].any() and not v[:, cols].any(), f"{what}: a dense layer holds state"
            continue
        o = gr["o"]
        assert_bitwise(v[:, cols], o.v, f"{what}: residual of the {gr['mode']} layers")
        assert_bitwise(u[:, cols], o.u, f"{what}: velocity of the {gr['mode']} layers")
        full = ora.full_row_indices(gr)
        at = 0
        for l, k in zip(gr["layers"], o.k_l):
            s0 = c.first_slot[l]
            assert c.k_l[l] == k
            assert_bitwise(idx[:, s0:s0 + k], full[:idx.shape[0], at:at + k], f"{what}: indices of layer {l}")
            at += k


@pytest.mark.parametrize("variant, K", [("rar", 4), ("ps", 3)])
def test_three_phases_against_the_oracle(variant, K):
    c1, c2 = 8, 4
    params = W.ae_init_params(c1, c2, variant, K, 5)
    gpu = PhasedLGC(NUMEL, MODES, K, variant=variant, c1=c1, c2=c2)
    gpu.ctx.set_ae_params(params)
    assert gpu.ctx.first_slot[0] == -1 and gpu.ctx.k_l[0] == 0 and gpu.ctx.mu_t == 5
    ora = OraclePhased(NUMEL, MODES, K, {1: params.numpy()}, variant=variant, c1=c1, c2=c2)
    src = W.GradientSource(W.LayerTable("ph", NUMEL, [1, 2, 3, 1, 2, 3, 1]), K, seed=23)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, device="cuda")
    schedule = ["raw"] * 2 + ["topk_train"] * 4 + ["compressed"] * 4
    for t, phase in enumerate(schedule):
        g = src.step(t) * 300.0
        choice = W.choice_for_step(5, t, K)
        upd.fill_(float("nan"))
        gpu.step(g.cuda(), upd, phase, choice, loss)
        ref, losses = ora.step(g.numpy(), phase, choice)
        got = upd.cpu().numpy()
        if phase == "raw":
            assert_bitwise(got, ref, f"step {t} ({phase}): dense mean")
            continue
        assert_bitwise(got[:9408], ref[:9408], f"step {t}: dense first layer")
        assert_close(got, ref, f"step {t} ({phase}): update")
        if losses:
            assert_close(np.array([loss.item()]), np.array(losses), f"step {t}: training loss")
        compare_state_and_slots(gpu, ora, f"step {t}")
    assert_close(gpu.ctx.get_ae_params().numpy(), ora.groups[1]["o"].get_params(), "trained parameters")
    gpu.check()


@pytest.mark.parametrize("variant", ["rar", "ps"])
def test_three_phases_with_the_full_size_autoencoder(variant):
    # the same schedule with Section IV-C's autoencoder on the middle layers (mu = 96 kept values there).
    # eps = 1e-2 keeps Adam's step well conditioned, so that the two sides' parameters stay together
    # through the training phase (see test_full_size_autoencoder_training_phase in test_gpu_parity.py).
    K = 2
    params = W.ae5_init_params(5, variant, K)
    gpu = PhasedLGC(NUMEL, MODES, K, variant=variant, ae_kind="conv5", eps=1e-2)
    gpu.ctx.set_ae_params(params)
    ora = OraclePhased(NUMEL, MODES, K, {1: params.numpy()}, variant=variant, ae_kind="conv5", eps=1e-2)
    src = W.GradientSource(W.LayerTable("ph", NUMEL, [1, 2, 3, 1, 2, 3, 1]), K, seed=29)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    loss = torch.zeros(1, device="cuda")
    for t, phase in enumerate(["raw"] + ["topk_train"] * 3 + ["compressed"] * 2):
        g = src.step(t) * 300.0
        choice = W.choice_for_step(5, t, K)
        upd.fill_(float("nan"))
        gpu.step(g.cuda(), upd, phase, choice, loss)
        ref, losses = ora.step(g.numpy(), phase, choice)
        assert_close(upd.cpu().numpy(), ref, f"step {t} ({phase}): update")
        if losses:
            assert_close(np.array([loss.item()]), np.array(losses), f"step {t}: training loss")
    # parameter server: the similarity gradient is a difference of nearly equal codes, known to ~1e-4 of its
    # scale in fp32 (test_full_size_autoencoder_parameter_server_training), and three Adam steps carry that on
    assert_close(gpu.ctx.get_ae_params().numpy(), ora.groups[1]["o"].get_params(), "trained parameters",
                 rel=1e-5 if variant == "rar" else 2e-4)
    gpu.check()


# layers of one mode that lie apart, sizes that are no multiple of four (dense runs start and end inside a
# 16-byte group), a dense layer that covers whole 4096-element tiles, large and small layers of every mode
APART = [9001, 20003, 5000, 70000, 4097, 13000, 127, 30000, 64, 8193, 4100, 3]
APART_MODES = ["dense", "ae", "topk", "ae", "dense", "ae", "topk", "dense", "ae", "topk", "ae", "dense"]


@pytest.mark.parametrize("variant, K, extra", [("rar", 3, []), ("ps", 3, []), ("rar", 2, [2]), ("ps", 2, [2])])
def test_layer_modes_inside_one_context(variant, K, extra):
    # Section VI-A's three treatments in one context, with the layers of a mode apart from one another: one
    # autoencoder over the kept values of all "ae" layers, stage by stage against the oracle's pipelines.
    # extra = [2]: N % 4 != 0, the rows do not start 16-byte aligned (row-wise accumulation, no fused candidates).
    numel, modes = APART + extra, APART_MODES + ["ae"] * len(extra)
    assert (sum(numel) % 4 == 0) == (not extra)
    params = W.ae_init_params(8, 4, variant, K, 5)
    gpu = lgc.LGC(numel, K, variant=variant, layer_mode=modes)
    gpu.set_ae_params(params)
    ora = OraclePhased(numel, modes, K, {0: params.numpy()}, grouping="modes", variant=variant)
    ae = next(gr["o"] for gr in ora.groups if gr["mode"] == "ae")
    assert gpu.mu == ae.mu and gpu.mu_all == gpu.mu + gpu.mu_t and gpu.mu_t == 5 + 1 + 8
    src = W.GradientSource(W.LayerTable("apart", numel, [1 + (i % 3) for i in range(len(numel))]), K, seed=61)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    dense_cols = np.concatenate([np.arange(a, b) for gr in ora.groups if gr["mode"] == "dense" for a, b in gr["ranges"]])
    for t in range(7):
        g = src.step(t) * 300.0
        gd = g.cuda()
        choice = W.choice_for_step(9, t, K)
        announce = t % 3 != 1
        upd.fill_(float("nan"))
        gpu.accumulate(gd, choice if t % 4 != 3 else -1)               # now and then without the leader's name
        gpu.topk(choice, upd if announce else None)
        if t == 2:                                                        # a step of the second phase in between
            ref, _ = ora.step(g.numpy(), "topk_train", choice)
            gpu.ae_train_step() if variant == "rar" else gpu.ae_train_step_ps(choice, 1.0, 1.0)
            gpu.topk_scatter(upd)
            gpu.set_ae_params(torch.from_numpy(ae.get_params().astype(np.float32)))     # both sides go on from the oracle's
            ae.set_params(ae.get_params().astype(np.float32).astype(np.float64))
        else:
            ref, _ = ora.step(g.numpy(), "compressed", choice)
            gpu.encode()
            assert_bitwise(gpu.val.cpu().numpy(), ae.val, f"step {t}: kept values of the autoencoder's layers")
            assert_close(gpu.code.cpu().numpy(), ae.z.reshape(K, -1), f"step {t}: codes")
            gpu.combine(choice)
            if variant == "ps":
                assert_bitwise(gpu.inn.cpu().numpy(), ae.inn, f"step {t}: innovation")
            gpu.decode_scatter(upd)
            assert_close(gpu.recon.cpu().numpy(), ae.r, f"step {t}: reconstruction")
        got = upd.cpu().numpy()
        assert_bitwise(got[dense_cols], ref[dense_cols], f"step {t}: dense layers")
        assert_close(got, ref, f"step {t}: update")
        compare_state_and_slots(gpu, ora, f"step {t}")
        gpu.check()
    if variant == "ps":
        top = next(gr["o"] for gr in ora.groups if gr["mode"] == "topk")
        # (the last step was a compression step: lgc_topk gathered the top-k-only layers' values too)
        assert gpu.val_topk_only.shape == (K, gpu.mu_t) and top.mu == gpu.mu_t


@pytest.mark.parametrize("variant", ["rar", "ps"])
def test_index_stream_and_host_step_with_layer_modes(variant):
    # the DEFLATE stream of an index row covers the autoencoder's layers and then the top-k-only ones (slot order),
    # each layer's gaps counted from the layer's own start; and lgc_step_host serves a context with modes (the dense
    # layers are read from the device copy of the gradients at the scatter)
    from oracle import index_coding as IC
    K = 3
    numel, modes = APART, APART_MODES
    params = W.ae_init_params(8, 4, variant, K, 5)
    gpu = lgc.LGC(numel, K, variant=variant, layer_mode=modes)
    gpu.set_ae_params(params)
    ora = OraclePhased(numel, modes, K, {0: params.numpy()}, grouping="modes", variant=variant)
    src = W.GradientSource(W.LayerTable("apart", numel, [1 + (i % 3) for i in range(len(numel))]), K, seed=71)
    hu = torch.empty(gpu.N, dtype=torch.float32).pin_memory()
    dg = torch.empty(K, gpu.N, device="cuda")
    du = torch.empty(gpu.N, device="cuda")
    for t in range(4):
        g = src.step(t) * 300.0
        choice = W.choice_for_step(11, t, K)
        gpu.step_host(g.clone().pin_memory(), dg, du, hu, choice)
        torch.cuda.synchronize()
        ref, _ = ora.step(g.numpy(), "compressed", choice)
        assert_close(hu.numpy(), ref, f"step {t}: update through host buffers")
        compare_state_and_slots(gpu, ora, f"step {t}")
    # the stream of the last selection: slot-ordered layer starts and slot offsets
    g = src.step(4) * 300.0
    choice = W.choice_for_step(11, 4, K)
    gpu.accumulate(g.cuda(), choice)
    gpu.topk(choice, None)
    order = [l for l, m in enumerate(modes) if m == "ae"] + [l for l, m in enumerate(modes) if m == "topk"]
    off = np.concatenate([[0], np.cumsum(numel)])
    layer_off = [int(off[l]) for l in order]
    koff = np.concatenate([[0], np.cumsum([gpu.k_l[l] for l in order])])
    assert [gpu.first_slot[l] for l in order] == [int(x) for x in koff[:-1]] and koff[-1] == gpu.mu_all
    for node in range(K if variant == "ps" else 1):
        row = gpu.idx[node].cpu().numpy()
        ref_bytes = IC.varint_bytes(row, layer_off, koff)
        out = torch.full((8 * gpu.mu_all + 1024,), 0xEE, dtype=torch.uint8, device="cuda")
        sizes = torch.zeros(2, dtype=torch.int64, device="cuda")
        gpu.encode_indices(node, out, sizes)
        torch.cuda.synchronize()
        n_stream, n_bytes = (int(x) for x in sizes.cpu())
        assert n_bytes == len(ref_bytes)
        assert IC.inflate(out[:n_stream].cpu().numpy().tobytes()) == ref_bytes
        assert np.array_equal(IC.indices_from_varint(ref_bytes, layer_off, koff), row)
    gpu.abort_step()
    gpu.check()


def test_a_context_needs_a_layer_for_the_autoencoder_and_known_modes():
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        lgc.LGC([5000, 6000], 2, layer_mode=["dense", "topk"])
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        lgc.LGC([5000, 6000], 2, layer_mode=[0, 7])


def test_a_context_on_a_slice_of_a_longer_gradient():
    # lgc_config.grad_row_stride: the context's rows are slices of rows that are a whole model apart
    K, numel, before, after = 3, [20000, 4096, 70001, 127], 5000, 300
    total = before + sum(numel) + after
    from oracle import OracleLGC
    params = W.ae_init_params(8, 4, "rar", K, 5)
    gpu = lgc.LGC(numel, K, grad_row_stride=total)
    gpu.set_ae_params(params)
    ora = OracleLGC(numel, K, params=params.numpy())
    src = W.GradientSource(W.LayerTable("wide", [total], [1]), K, seed=67)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(4):
        g = src.step(t)
        gd = g.cuda()
        gpu.step(gd[:, before:before + gpu.N], upd, t % K)
        ref = ora.step(np.ascontiguousarray(g.numpy()[:, before:before + gpu.N]), t % K)
        assert_close(upd.cpu().numpy(), ref, f"step {t}: update")
        assert_bitwise(gpu.v.cpu().numpy(), ora.v, f"step {t}: v")
    gpu.check()


def test_dense_mean_on_ragged_and_strided_rows():
    rng = np.random.default_rng(2)
    g = torch.from_numpy(rng.standard_normal((5, 10007)).astype(np.float32)).cuda()
    for a, b in ((0, 10007), (3, 9001), (4, 4100), (17, 18)):
        view = g[:, a:b]
        out = torch.empty(b - a, device="cuda")
        lgc.dense_mean(view, out)
        acc = view[0].cpu().numpy().copy()
        for k in range(1, 5):
            acc = acc + view[k].cpu().numpy()
        assert_bitwise(out.cpu().numpy(), acc / np.float32(5), f"slice {a}:{b}")
