"""CUDA path vs CPU oracle, element by element, on cases the oracle finishes in seconds."""
import numpy as np
import pytest
import torch

from paper_2103_08870_b200 import lgc
from paper_2103_08870_b200 import workloads as W

from parity import assert_bitwise, assert_close, compare_step, make_pair

pytestmark = pytest.mark.gpu

# ragged toy table: tiny layers, sizes that are no multiple of four, chunk edges (4096, 4097,
# 8193), several chunks with a ragged tail (20000, 70001)
TOY = [4096, 64, 1500, 9000, 65, 127, 20000, 5001, 4097, 8193, 1, 3, 70001, 1000]


def toy_source(numel, K, seed=5):
    return W.GradientSource(W.LayerTable("toy", list(numel), [1 + (i % 3) for i in range(len(numel))]), K, seed=seed)


def run_steps(numel, K, steps, hints=("leader",), **kw):
    seed = kw.get("seed", W.DEFAULT_SEED)
    ora, gpu = make_pair(numel, K, **kw)
    src = toy_source(numel, K)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(steps):
        g = src.step(t)
        compare_step(ora, gpu, g, g.cuda(), W.choice_for_step(seed, t, K), upd, hint=hints[t % len(hints)],
                     announce_update=(t % 3 != 1))
    return ora, gpu


def test_tiny_config_ring_allreduce():
    # one flat tensor of 2^20 elements, K = 2, density 0.1 % (k = 1049), AE 8/4, 3 steps
    w = W.workload("tiny")
    ora, gpu = make_pair(w.table.numel, w.num_nodes)
    assert gpu.mu == 1049 and (gpu.L1, gpu.L2) == (524, 261)
    src = W.GradientSource(w.table, w.num_nodes, seed=w.seed)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(w.steps):
        g = src.step(t)
        compare_step(ora, gpu, g, g.cuda(), W.choice_for_step(w.seed, t, w.num_nodes), upd)


@pytest.mark.parametrize("K", [1, 3])
def test_ragged_layers_ring_allreduce(K):
    assert sum(TOY) % 4 == 0                      # rows start 16-byte aligned: the fused accumulation runs
    run_steps(TOY, K, 6)


def test_leader_hint_never_changes_a_result():
    # candidates collected while accumulating are used only when the hint was right; a missing or
    # wrong hint, and hints that come and go, give the same bits
    run_steps(TOY, 3, 8, hints=("none", "leader", "leader", "wrong", "leader", "none", "leader", "leader"))


def test_rows_that_do_not_start_aligned():
    numel = TOY + [2]                             # N % 4 == 2: the plain accumulation kernel is used
    assert sum(numel) % 4 != 0
    run_steps(numel, 3, 4)
    run_steps(numel, 2, 3, variant="ps")


def test_prediction_survives_a_collapse_of_the_gradient_scale():
    # the predicted bucket comes from the previous step; when the residual's large entries vanish
    # (scale drops by 1e4) the prediction is too high and the selection must fall back
    numel = [200000, 3000, 50000]
    K = 2
    ora, gpu = make_pair(numel, K, momentum=0.0, density_ppm=5000)
    src = toy_source(numel, K)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t, scale in enumerate([1.0, 1.0, 1e-4, 1e-4, 1.0, 10.0, 1e-6]):
        g = src.step(t) * scale
        if t in (2, 6):                           # wipe the residual: only the tiny gradient remains
            gpu.v.zero_(); gpu.u.zero_(); ora.v[:] = 0; ora.u[:] = 0
        compare_step(ora, gpu, g, g.cuda(), t % K, upd)


def test_prediction_a_little_too_high():
    # the k-th key drops by a tenth from one step to the next (the residual is wiped and the gradient
    # scaled by 0.9): fewer than k entries pass the predicted key, and the layers are finished from one read
    # of the data with a lowered key; a drop by a third (last but one step) is beyond that and takes the full search
    numel = [300000, 3000, 70000]
    K = 2
    ora, gpu = make_pair(numel, K, momentum=0.0, density_ppm=5000)
    src = toy_source(numel, K)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    from_data = []
    for t, scale in enumerate([1.0, 1.0, 0.9, 0.9, 0.8, 0.8, 0.55, 1.0]):
        g = src.step(t % 2) * scale
        gpu.v.zero_(); gpu.u.zero_(); ora.v[:] = 0; ora.u[:] = 0
        compare_step(ora, gpu, g, g.cuda(), t % K, upd)
        stats = gpu.selection_stats()
        from_data.append(stats[4])
        if t in (2, 4):
            assert stats[3] < numel[0], stats         # a handful of candidates, not the whole layer
        if t == 6:
            assert stats[3] == numel[0], stats
    assert from_data[2] == 2 and from_data[4] == 2 and from_data[6] == 2, from_data


def test_ragged_layers_parameter_server():
    ora, gpu = run_steps(TOY, 3, 3, variant="ps")
    assert gpu.idx.shape == (3, gpu.mu)


def test_parameter_server_large_innovation_segments():
    # dense selection so that a layer keeps more than one chunk of values: the innovation
    # selection then runs through the chunked path as well
    run_steps([60000, 300, 5000], 2, 2, variant="ps", density_ppm=100000, innovation_permille=300)


@pytest.mark.parametrize("variant", ["rar", "ps"])
def test_identity_autoencoder(variant):
    run_steps(TOY, 2, 3, variant=variant, ae_kind="identity")


def test_wide_autoencoder_and_small_channels():
    run_steps(TOY, 2, 2, c1=16, c2=8)
    run_steps(TOY, 2, 1, c1=3, c2=2)
    run_steps(TOY, 2, 1, c1=16, c2=8, variant="ps")


def test_momentum_zero_and_other_densities():
    run_steps(TOY, 2, 3, momentum=0.0)
    run_steps(TOY, 2, 2, density_ppm=50000)
    run_steps([50000, 777], 2, 2, density_ppm=1000000, ae_kind="identity")     # everything is kept


def test_layer_spanning_several_compaction_groups():
    # more than 2048 chunks in one layer: its selection is completed group by group, one CTA per group
    numel = [9_000_000, 5000]
    ora, gpu = make_pair(numel, 2, topk_method="select")
    src = W.GradientSource(W.LayerTable("big", numel, [1, 1]), 2, seed=11, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(5):
        g = src.step(t)
        compare_step(ora, gpu, g.cpu(), g, t % 2, upd)
    assert gpu.selection_stats()[1] == 2          # both layers served from the accumulation by now


@pytest.mark.parametrize("levels, first_from_data", [(200, 0), (3, 2)])
def test_layer_of_several_groups_with_ties(levels, first_from_data):
    # integer-valued gradients: the k-th magnitude is shared by many entries of the 9 M layer, which
    # is finished group by group (401 levels: ~45 k entries tie for 9000 places in the first step, and
    # the candidates, nine levels, are 4.5 % of the layer) or, when the tied entries exceed the layer's
    # compact capacity or a chunk's list (7 levels: 2.6 M of the large layer, 1400 of the small one), from the data
    numel = [9_000_000, 5000]
    K = 2
    ora, gpu = make_pair(numel, K, momentum=0.0, topk_method="select")
    rng = np.random.default_rng(levels)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    from_data = []
    for t in range(4):
        g = rng.integers(-levels, levels + 1, size=(K, gpu.N)).astype(np.float32)
        gt = torch.from_numpy(g)
        compare_step(ora, gpu, gt, gt.cuda(), t % K, upd)
        from_data.append(gpu.selection_stats()[4])
    assert from_data[0] == first_from_data


@pytest.mark.parametrize("numel, K, scale", [([300_000, 5000, 120_000], 2, 1.0), ([300_000, 5000, 120_000], 2, 500.0),
                                             ([2_000_000, 700_000, 300_001], 3, 1.0)])
def test_full_size_autoencoder(numel, K, scale):
    # the autoencoder of Section IV-C (filters 64/128/256/64/4 and 4/32/64/128/32 + 1x1): mu = 425
    # (every GEMM tile ragged) and mu = 3000 (several tiles per layer and node, ragged tails).
    # scale 500 makes the kept values O(1), so that the data, not the biases, dominate every layer.
    ora, gpu = make_pair(numel, K, ae_kind="conv5")
    src = W.GradientSource(W.LayerTable("ae5", numel, [1 + i for i in range(len(numel))]), K, seed=21)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(3):
        g = src.step(t) * scale
        compare_step(ora, gpu, g, g.cuda(), t % K, upd)


@pytest.mark.parametrize("c1, c2, K", [(8, 4, 3), (16, 8, 4)])
def test_parameter_server_autoencoder_training(c1, c2, K):
    # Section IV-A: reconstruction loss through the K decoders (innovation fused in) + similarity loss
    # between the nodes' codes; 12 Adam steps with a changing common node, then a compression step
    numel = [70001, 9000, 20000, 4097, 127]
    ora, gpu = make_pair(numel, K, variant="ps", c1=c1, c2=c2)
    src = toy_source(numel, K, seed=31)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    loss_dev = torch.zeros(1, device="cuda")
    losses, losses_ref = [], []
    for t in range(12):
        g = src.step(t) * 300.0                       # kept values of O(1): well-conditioned gradients
        ora.accumulate(g.numpy())
        gpu.accumulate(g.cuda())
        ora.topk()
        gpu.topk(0)
        common = (5 * t + 1) % K
        losses_ref.append(ora.ae_train_step_ps(common, 0.7, 0.3))
        gpu.ae_train_step_ps(common, 0.7, 0.3, loss_dev)
        losses.append(loss_dev.item())
        ref = ora.topk_scatter()
        gpu.topk_scatter(upd)
        assert_close(upd.cpu().numpy(), ref, f"sparse update at training step {t}")
    assert_close(np.array(losses), np.array(losses_ref), "training losses")
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "trained parameters")
    gpu.check()
    g = src.step(12) * 300.0
    compare_step(ora, gpu, g, g.cuda(), 1, upd)


def test_dense_selection_uses_the_global_compact_arrays():
    # k = 40,000 of 2,000,000: more candidates than the finishing CTA keeps in shared memory
    numel = [2_000_000]
    ora, gpu = make_pair(numel, 2, density_ppm=20000, topk_method="select")
    src = W.GradientSource(W.LayerTable("dense", numel, [1]), 2, seed=12, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(5):
        g = src.step(t)
        compare_step(ora, gpu, g.cpu(), g, t % 2, upd)
    assert gpu.selection_stats()[3] > 20480


def test_a_chunk_with_more_candidates_than_its_list_holds():
    # 3000 large entries side by side land in one or two 4096-element tiles: their lists (1024
    # records) overflow and the layer is finished from the data; the layer next to it is not affected
    numel = [400_000, 100_000]
    K = 2
    ora, gpu = make_pair(numel, K, density_ppm=20000, momentum=0.0)
    rng = np.random.default_rng(5)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(6):
        g = (rng.standard_normal((K, gpu.N)) * 1e-3).astype(np.float32)
        g[:, 10_000:13_000] += np.float32(1.0) * rng.choice([-1, 1], size=(K, 3000)).astype(np.float32)
        gt = torch.from_numpy(g)
        compare_step(ora, gpu, gt, gt.cuda(), t % K, upd)
    large, served, _, _, from_data = gpu.selection_stats()
    assert (large, served, from_data) == (2, 1, 1)


@pytest.mark.parametrize("fill", ["zeros", "equal", "few_values", "denormal"])
def test_degenerate_values(fill):
    numel = [9000, 130, 4097, 33000, 300001]      # the last two exceed the candidate capacity when all tie
    K = 2
    ora, gpu = make_pair(numel, K, density_ppm=20000)
    N = gpu.N
    rng = np.random.default_rng(3)
    upd = torch.empty(N, dtype=torch.float32, device="cuda")
    for t in range(3):
        if fill == "zeros":
            g = np.zeros((K, N), np.float32)
        elif fill == "equal":
            g = np.full((K, N), -0.25, np.float32)
        elif fill == "few_values":
            g = rng.integers(-2, 3, size=(K, N)).astype(np.float32)
        else:
            g = (rng.integers(-5, 6, size=(K, N)) * 1e-45).astype(np.float32)
        gt = torch.from_numpy(g)
        compare_step(ora, gpu, gt, gt.cuda(), t % K, upd)


def test_same_inputs_same_bits_twice():
    outs = []
    for _ in range(2):
        w = lgc.LGC(TOY, 3, variant="ps")
        w.set_ae_params(W.ae_init_params(8, 4, "ps", 3))
        src = toy_source(TOY, 3)
        upd = torch.empty(w.N, dtype=torch.float32, device="cuda")
        for t in range(3):
            w.step(src.step(t).cuda(), upd, t % 3)
        w.check()
        outs.append((upd.cpu().numpy().copy(), w.v.cpu().numpy().copy(), w.idx.cpu().numpy().copy()))
    for a, b in zip(*outs):
        assert_bitwise(a, b, "repeat run")


def test_call_order_and_argument_errors():
    w = lgc.LGC(TOY, 2)
    g = torch.zeros(2, w.N, device="cuda")
    upd = torch.empty(w.N, device="cuda")
    with pytest.raises(lgc.LGCError, match="BAD_STATE"):
        w.topk(0)
    with pytest.raises(lgc.LGCError, match="BAD_STATE"):
        w.decode_scatter(upd)
    w.accumulate(g)
    with pytest.raises(lgc.LGCError, match="BAD_STATE"):
        w.accumulate(g)
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        w.topk(5)
    w.topk(1)
    with pytest.raises(lgc.LGCError, match="BAD_STATE"):
        w.combine(0)
    with pytest.raises(ValueError):
        w.decode_scatter(upd[:-1])
    w.encode()
    w.combine(0)
    w.decode_scatter(upd)
    w.check()
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        w.set_ae_params(torch.zeros(5))


def test_topk_scatter_phase_two():
    for variant in ("rar", "ps"):
        ora, gpu = make_pair(TOY, 3, variant=variant)
        src = toy_source(TOY, 3)
        upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
        for t in range(2):
            g = src.step(t)
            ora.accumulate(g.numpy())
            gpu.accumulate(g.cuda(), t)
            ora.topk(t)
            gpu.topk(t)
            ref = ora.topk_scatter()
            gpu.topk_scatter(upd)
            assert_close(upd.cpu().numpy(), ref, "sparse mean update")
            assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v")
            assert_bitwise(gpu.u.cpu().numpy(), ora.u, "u")
        gpu.check()


def test_autoencoder_training_matches_oracle():
    numel = [300000, 5000, 64, 120000]
    K = 3
    ora, gpu = make_pair(numel, K)
    src = toy_source(numel, K)
    g = src.step(0) * 1e3                       # O(1) values
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda())
    ora.topk(0)
    gpu.topk(0)
    loss_dev = torch.zeros(1, device="cuda")
    losses_ref, losses = [], []
    for _ in range(50):
        losses_ref.append(ora.ae_train_step())
        gpu.ae_train_step(loss_dev)
        losses.append(loss_dev.item())
    assert_close(np.array(losses), np.array(losses_ref), "training losses", rel=1e-5)
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "trained parameters")
    assert losses[-1] < losses[0]
    # the trained autoencoder then compresses
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    ora.encode(); ora.combine(0); ref = ora.decode_scatter()
    gpu.encode(); gpu.combine(0); gpu.decode_scatter(upd)
    assert_close(upd.cpu().numpy(), ref, "update with the trained autoencoder")
    gpu.check()


def test_step_from_host_buffers():
    ora, gpu = make_pair(TOY, 2)
    src = toy_source(TOY, 2)
    g = src.step(0)
    hg = g.clone().pin_memory()
    hu = torch.empty(gpu.N, dtype=torch.float32).pin_memory()
    dg = torch.empty(2, gpu.N, device="cuda")
    du = torch.empty(gpu.N, device="cuda")
    gpu.step_host(hg, dg, du, hu, 1)
    torch.cuda.synchronize()
    ref = ora.step(g.numpy(), 1)
    assert_close(hu.numpy(), ref, "update through host buffers")
    assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v")


@pytest.mark.parametrize("variant", ["rar", "ps"])
def test_a_refused_host_step_leaves_state_and_context_untouched(variant):
    # every argument of lgc_step_host is checked before anything is copied or enqueued: a leader / common
    # node outside 0 .. K-1 (for both variants), a misaligned device buffer or a NULL pointer returns
    # INVALID_ARG, u and v keep their bits, and the context still accepts the next step
    K = 3
    ora, gpu = make_pair(TOY, K, variant=variant)
    src = toy_source(TOY, K)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g0 = src.step(0)
    compare_step(ora, gpu, g0, g0.cuda(), 1, upd)
    u0, v0 = gpu.u.clone(), gpu.v.clone()
    g1 = src.step(1)
    hg = g1.clone().pin_memory()
    hu = torch.empty(gpu.N, dtype=torch.float32).pin_memory()
    dg = torch.empty(K * gpu.N + 4, device="cuda")
    du = torch.empty(gpu.N + 4, device="cuda")
    for choice in (-1, K, 1000):
        with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
            gpu.step_host(hg, dg[:K * gpu.N], du[:gpu.N], hu, choice)
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        gpu.step_host(hg, dg[1:K * gpu.N + 1], du[:gpu.N], hu, 0)          # dev_grads off by one float
    with pytest.raises(lgc.LGCError, match="INVALID_ARG"):
        gpu.step_host(hg, dg[:K * gpu.N], du[1:gpu.N + 1], hu, 0)          # dev_update off by one float
    torch.cuda.synchronize()
    assert torch.equal(gpu.u.view(torch.int32), u0.view(torch.int32)) and torch.equal(gpu.v.view(torch.int32), v0.view(torch.int32))
    gpu.step_host(hg, dg[:K * gpu.N], du[:gpu.N], hu, 2)                   # the context is idle: a good call runs
    torch.cuda.synchronize()
    assert_close(hu.numpy(), ora.step(g1.numpy(), 2), "update of the step after the refused calls")
    assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v")
    gpu.check()


def test_abort_step_returns_the_context_to_idle():
    # a step given up after its accumulation: nothing was sent, so the gradient stays in the residual
    # (Algorithm 1/2 after a step that transmitted nothing) and the next step starts from there
    K = 2
    ora, gpu = make_pair(TOY, K)
    src = toy_source(TOY, K)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g0, g1 = src.step(0), src.step(1)
    gpu.accumulate(g0.cuda(), 0)
    gpu.topk(0, upd)
    gpu.abort_step()
    ora.accumulate(g0.numpy())
    with pytest.raises(lgc.LGCError, match="BAD_STATE"):
        gpu.encode()
    compare_step(ora, gpu, g1, g1.cuda(), 1, upd)


def test_contexts_on_two_devices_in_one_process():
    # kernel attributes (the opt-in to more dynamic shared memory) and the SM count are per device
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible GPUs")
    numel = [300_000, 5000, 120_000]          # a layer above 4096 elements: finish_kernel with its 80 KB of shared memory
    src = toy_source(numel, 2)
    g = src.step(0)
    outs = []
    for dev in ("cuda:0", "cuda:1"):
        w = lgc.LGC(numel, 2, device=dev)
        w.set_ae_params(W.ae_init_params(8, 4, "rar", 2))
        upd = torch.empty(w.N, dtype=torch.float32, device=dev)
        w.step(g.to(dev), upd, 0)
        w.check()
        outs.append((w.idx.cpu().numpy().copy(), upd.cpu().numpy().copy()))
    assert_bitwise(outs[0][0], outs[1][0], "indices on the two devices")
    assert_bitwise(outs[0][1], outs[1][1], "update on the two devices")


@pytest.mark.parametrize("variant,K,extra", [("rar", 3, []), ("ps", 2, []), ("rar", 2, [2])])
def test_steps_from_host_buffers_back_to_back(variant, K, extra):
    # Six calls queued without waiting in between: each node's row is accumulated as it arrives
    # (from the third step on by the kernel that also collects the selection candidates), the
    # upload of one call overlaps the download of the one before.  extra = [2]: N % 4 != 0, rows
    # do not start 16-byte aligned and the step falls back to one accumulation of all rows.
    numel = TOY + extra
    steps = 6
    ora, gpu = make_pair(numel, K, variant=variant)
    src = toy_source(numel, K)
    gs = [src.step(t) for t in range(steps)]
    hg = [g.clone().pin_memory() for g in gs]
    hu = [torch.full((gpu.N,), float("nan"), dtype=torch.float32).pin_memory() for _ in range(steps)]
    dg = torch.empty(K, gpu.N, device="cuda")
    du = torch.empty(gpu.N, device="cuda")
    choices = [W.choice_for_step(7, t, K) for t in range(steps)]
    for t in range(steps):
        gpu.step_host(hg[t], dg, du, hu[t], choices[t])
    torch.cuda.synchronize()
    for t in range(steps):
        ref = ora.step(gs[t].numpy(), choices[t])
        assert_close(hu[t].numpy(), ref, f"update of step {t} through host buffers")
    assert_bitwise(gpu.u.cpu().numpy(), ora.u, "u")
    assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v")
    idx_ref = ora.idx if variant == "ps" else ora.idx[:1]
    assert_bitwise(gpu.idx.cpu().numpy(), idx_ref, "selected indices of the last step")
    if (gpu.N % 4) == 0:
        large, served, _, _, _ = gpu.selection_stats()
        assert large > 0 and served > 0, "the row-by-row accumulation did not collect any candidates"
    gpu.check()


def per_tensor(flat, shapes):
    pos = 0
    for name, shape in shapes:
        n = int(np.prod(shape))
        yield name, np.asarray(flat[pos:pos + n], dtype=np.float64)
        pos += n


def adam_moments(gpu):
    """Adam's two moment vectors as the library keeps them behind the parameters (caller-owned buffer)."""
    pad = (gpu.P + 3) // 4 * 4
    return gpu.params_buf[pad:pad + gpu.P], gpu.params_buf[2 * pad:2 * pad + gpu.P]


@pytest.mark.parametrize("numel, K", [([300_000, 5000, 120_000], 2), ([2_000_000, 700_000, 300_001], 3)])
def test_full_size_autoencoder_gradients_and_first_steps(numel, K):
    # Section IV-C's autoencoder, loss of Section IV-B.  mu = 425 (every GEMM tile ragged, a single chunk
    # per gradient sum) and mu = 3000.  After the first step Adam's first moment is (1 - beta1) times the
    # gradient, so every tensor's gradient is compared with the oracle's directly, at its own scale;
    # then the parameters after that step, and the losses of two more steps on the same kept values.
    from oracle import full_ae as A5
    ora, gpu = make_pair(numel, K, ae_kind="conv5")
    src = toy_source(numel, K, seed=41)
    g = src.step(0) * 300.0                           # kept values of O(1)
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda(), 0)
    ora.topk(0)
    gpu.topk(0)
    loss_dev = torch.zeros(1, device="cuda")
    _, grads_ref = ora.ae_loss_and_grads()
    losses_ref, losses = [ora.ae_train_step()], []
    gpu.ae_train_step(loss_dev)
    losses.append(loss_dev.item())
    m = adam_moments(gpu)[0].cpu().numpy().astype(np.float64)
    for name, got in per_tensor(m / 0.1, A5.param_shapes()):
        assert_close(got, grads_ref[name], f"gradient of {name}")
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "parameters after the first step")
    for _ in range(2):
        losses_ref.append(ora.ae_train_step())
        gpu.ae_train_step(loss_dev)
        losses.append(loss_dev.item())
    assert_close(np.array(losses), np.array(losses_ref), "training losses")
    assert losses[2] < losses[0]
    assert_bitwise(gpu.val.cpu().numpy(), ora.val, "kept values")
    gpu.check()


def test_full_size_autoencoder_training_phase():
    # Section V-B's second phase: fresh gradients every step, selection, one training step on the kept
    # values, the sparse mean as the update; then a compression step with the trained autoencoder.
    # Adam's step lr m^ / (sqrt(v^) + eps) amplifies a gradient's rounding error by up to lr / eps, so
    # two correct runs in different precisions drift apart over the steps.  Each step is therefore
    # compared from the same state: the oracle's parameters and moments, rounded to fp32, are given to
    # both sides before every step (nothing of the library's flows into the oracle), and eps = 1e-2
    # (above most gradients: close to the plain SGD the paper trains with) keeps the step itself well
    # conditioned.  Per step: loss, every tensor's gradient (from the change of the first moment),
    # the parameters after the step, the sparse update.
    from oracle import full_ae as A5
    numel, K = [2_000_000, 700_000, 300_001], 3
    ora, gpu = make_pair(numel, K, ae_kind="conv5", lr=1e-3, eps=1e-2)
    src = toy_source(numel, K, seed=41)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    loss_dev = torch.zeros(1, device="cuda")
    m_dev, v_dev = adam_moments(gpu)
    ora.adam_m = np.zeros(ora.get_params().size)
    ora.adam_v = np.zeros(ora.get_params().size)
    for t in range(4):
        p32, m32, v32 = (x.astype(np.float32) for x in (ora.get_params(), ora.adam_m, ora.adam_v))
        ora.set_params(p32.astype(np.float64))
        ora.adam_m, ora.adam_v = m32.astype(np.float64), v32.astype(np.float64)
        gpu.set_ae_params(torch.from_numpy(p32))
        m_dev.copy_(torch.from_numpy(m32))
        v_dev.copy_(torch.from_numpy(v32))
        g = src.step(t) * 300.0
        ora.accumulate(g.numpy())
        gpu.accumulate(g.cuda(), t % K)
        ora.topk(t % K)
        gpu.topk(t % K, upd)
        _, grads_ref = ora.ae_loss_and_grads()
        loss_ref = ora.ae_train_step()
        gpu.ae_train_step(loss_dev)
        assert abs(loss_dev.item() - loss_ref) <= 1e-5 * loss_ref, f"loss at step {t}"
        got = (m_dev.cpu().numpy().astype(np.float64) - 0.9 * m32) / 0.1
        for name, gg in per_tensor(got, A5.param_shapes()):
            # The leaky ReLU's derivative jumps at zero: a unit whose pre-activation lies within rounding of
            # zero (about one in a million, so about one per step here) takes the other slope in fp32 than in
            # fp64, which moves the gradient entries that pass through it by up to about 1e-2 of their
            # tensor's scale (one row of a few hundred in a sum).  The test above holds the gradients to
            # 1e-5 on two selections where no unit does.
            assert_close(gg, grads_ref[name], f"gradient of {name} at step {t}", rel=3e-2)
        assert_close(gpu.get_ae_params().numpy(), ora.get_params(), f"parameters after step {t}")
        ref = ora.topk_scatter()
        gpu.topk_scatter(upd)
        assert_close(upd.cpu().numpy(), ref, f"sparse update at training step {t}")
    gpu.check()
    p32 = ora.get_params().astype(np.float32)
    ora.set_params(p32.astype(np.float64))
    gpu.set_ae_params(torch.from_numpy(p32))
    g = src.step(4) * 300.0
    compare_step(ora, gpu, g, g.cuda(), 1, upd)


@pytest.mark.parametrize("numel, K", [([300_000, 5000, 120_000], 2), ([2_000_000, 700_000, 300_001], 3)])
def test_full_size_autoencoder_parameter_server(numel, K):
    # Section IV-A with Section IV-C's layers: every node encodes, the common node's code goes through
    # every node's own decoder, whose last convolution also sees the node's innovation (33rd channel);
    # node-ordered average at each node's own indices.  Every stage compared, three steps.
    ora, gpu = make_pair(numel, K, variant="ps", ae_kind="conv5")
    assert gpu.P == 172_996 + K * 43_734
    src = toy_source(numel, K, seed=43)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(3):
        g = src.step(t) * 300.0
        compare_step(ora, gpu, g, g.cuda(), (2 * t + 1) % K, upd)
    gpu.check()


@pytest.mark.parametrize("numel, K", [([300_000, 5000, 120_000], 2), ([2_000_000, 700_000, 300_001], 3)])
def test_full_size_autoencoder_parameter_server_training(numel, K):
    # Section IV-A's loss on Section IV-C's layers: reconstruction through the K decoders (each with its
    # node's innovation as 33rd channel) + similarity of the codes.  After the first step Adam's first
    # moment is (1 - beta1) times the gradient: every tensor's gradient (encoder and all decoders) against
    # the oracle's, the loss, the parameters after that step; then the losses of two more steps on the
    # same kept values with other common nodes, and the sparse update of the second training phase.
    from oracle import full_ae as A5
    ora, gpu = make_pair(numel, K, variant="ps", ae_kind="conv5")
    src = toy_source(numel, K, seed=53)
    g = src.step(0) * 300.0
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda())
    ora.topk()
    gpu.topk(0)
    loss_dev = torch.zeros(1, device="cuda")
    _, _, _, grads_ref = ora.ae_loss_and_grads_ps(1, 0.7, 0.3)
    losses_ref, losses = [ora.ae_train_step_ps(1, 0.7, 0.3)], []
    gpu.ae_train_step_ps(1, 0.7, 0.3, loss_dev)
    losses.append(loss_dev.item())
    m = adam_moments(gpu)[0].cpu().numpy().astype(np.float64)
    # The similarity term's gradient at a code, 4 lam_sim (K z_k - sum_m z_m) / n, is a difference of codes that
    # agree in their leading digits (the nodes share most of their signal), so the codes' own error (1e-6 of
    # their scale, fp32 against fp64) shows up several times larger in it and in what the encoder makes of it.
    for name, got in per_tensor(m / 0.1, A5.param_shapes_ps(K)):
        assert_close(got, grads_ref[name], f"gradient of {name}", rel=1e-4)
    # Adam's first step is lr g / (|g| + eps): where |g| is near eps = 1e-8 a gradient error of 1e-10 moves it by 1e-5 lr / eps
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "parameters after the first step", rel=1e-4)
    for common in (0, K - 1):
        losses_ref.append(ora.ae_train_step_ps(common, 0.7, 0.3))
        gpu.ae_train_step_ps(common, 0.7, 0.3, loss_dev)
        losses.append(loss_dev.item())
    assert_close(np.array(losses), np.array(losses_ref), "training losses")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    assert_close(upd_of(gpu, upd), ora.topk_scatter(), "sparse update")
    gpu.check()


def upd_of(gpu, upd):
    gpu.topk_scatter(upd)
    return upd.cpu().numpy()


@pytest.mark.parametrize("variant", ["rar", "ps"])
@pytest.mark.parametrize("numel", [[31_000], [16_000, 17_000], [34_000, 64]])
def test_full_size_autoencoder_at_its_shortest_inputs(variant, numel):
    # mu = 31 (the code is one position of four channels), 33 and 35: every layer of the autoencoder is a
    # single ragged tile, the transposed convolutions' output paddings take both values
    K = 2
    ora, gpu = make_pair(numel, K, variant=variant, ae_kind="conv5")
    assert gpu.mu in (31, 33, 35)
    src = toy_source(numel, K, seed=47)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(2):
        g = src.step(t) * 300.0
        compare_step(ora, gpu, g, g.cuda(), t % K, upd)
    if variant == "rar":                               # and one training step: loss and every tensor's gradient
        from oracle import full_ae as A5
        g = src.step(2) * 300.0
        ora.accumulate(g.numpy())
        gpu.accumulate(g.cuda(), 0)
        ora.topk(0)
        gpu.topk(0)
        loss_dev = torch.zeros(1, device="cuda")
        _, grads_ref = ora.ae_loss_and_grads()
        loss_ref = ora.ae_train_step()
        gpu.ae_train_step(loss_dev)
        assert abs(loss_dev.item() - loss_ref) <= 1e-5 * loss_ref
        m = adam_moments(gpu)[0].cpu().numpy().astype(np.float64)
        for name, got in per_tensor(m / 0.1, A5.param_shapes()):
            assert_close(got, grads_ref[name], f"gradient of {name}", rel=2e-5)
    gpu.check()


def test_parameter_server_with_five_nodes():
    # five index sets that overlap in part: the node-ordered average looks an index up in the other nodes' lists
    # eight nodes at a time (one batch here, with idle slots), with and without the update buffer announced
    numel = [70001, 9000, 20000, 4097, 127, 300_000]
    K = 5
    ora, gpu = make_pair(numel, K, variant="ps", c1=16, c2=8)
    src = toy_source(numel, K, seed=59)
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    for t in range(4):
        g = src.step(t)
        compare_step(ora, gpu, g, g.cuda(), (3 * t + 1) % K, upd, announce_update=(t % 2 == 0))
    g = src.step(4)                                   # and the second training phase's sparse mean
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda())
    ora.topk()
    gpu.topk(0)
    assert_close(upd_of(gpu, upd), ora.topk_scatter(), "sparse update")
    assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v")
    gpu.check()
