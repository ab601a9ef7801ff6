"""The five workload configurations at full size, in the launch configuration bench.py times.

Configs 1-3 run the whole oracle beside the CUDA path (they fit in host memory and finish in
tens of seconds per step); the stress config (2^30 elements per node) does too when the host has
the memory for the oracle's state (32 GiB), and otherwise compares the elementwise stages on sampled
positions, the selection on the leader's full row, and the autoencoder stages in full.
"""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import OracleLGC
from paper_2103_08870_b200 import lgc
from paper_2103_08870_b200 import workloads as W

from parity import assert_bitwise, assert_close, compare_step, make_pair

pytestmark = pytest.mark.gpu


def run_workload(name, steps, state_every=1):
    w = W.workload(name)
    ora, gpu = make_pair(w.table.numel, w.num_nodes, variant=w.variant, ae_kind=w.ae_kind, c1=w.ae_c1, c2=w.ae_c2,
                         density_ppm=w.density_ppm, momentum=w.momentum,
                         innovation_permille=w.innovation_permille, seed=w.seed)
    src = W.GradientSource(w.table, w.num_nodes, seed=w.seed, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g = torch.empty((w.num_nodes, gpu.N), dtype=torch.float32, device="cuda")
    for t in range(steps):
        src.step_into(t, g)
        check = (t % state_every == 0) or t == steps - 1
        compare_step(ora, gpu, g.cpu(), g, W.choice_for_step(w.seed, t, w.num_nodes), upd, check_state=check)
    return ora, gpu


def test_resnet50_config():
    ora, gpu = run_workload("resnet50", 10, state_every=3)
    assert gpu.L == 161 and gpu.N == 25_557_032 and gpu.mu == sum(ora.k_l)


def test_resnet50_config_with_the_full_size_autoencoder():
    # the ResNet-50-shaped case, K = 8, with the autoencoder of Section IV-C: mu = 25,617, code 4 x 1600
    ora, gpu = run_workload("resnet50_ae5", 3, state_every=2)
    assert gpu.mu == 25_617 and gpu.code_len == 4 * 1600 and gpu.P == 216_729
    # one training step of that autoencoder at this size (every gradient sum cut into 48 chunks): the
    # loss, every tensor's gradient (Adam's first moment after a first step is a tenth of it) and the
    # sparse update.  About eight of the 7 million leaky-ReLU units lie within rounding of zero here and
    # take the other slope in fp32 than in fp64, hence the tolerance on the gradients (see
    # test_full_size_autoencoder_training_phase in test_gpu_parity.py).
    from oracle import full_ae as A5
    w = W.workload("resnet50_ae5")
    src = W.GradientSource(w.table, w.num_nodes, seed=w.seed, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g = torch.empty((w.num_nodes, gpu.N), dtype=torch.float32, device="cuda")
    loss_dev = torch.zeros(1, device="cuda")
    src.step_into(3, g)
    leader = W.choice_for_step(w.seed, 3, w.num_nodes)
    ora.accumulate(g.cpu().numpy())
    gpu.accumulate(g, leader)
    ora.topk(leader)
    gpu.topk(leader, None)
    _, grads_ref = ora.ae_loss_and_grads()
    ref_loss = ora.ae_train_step()
    gpu.ae_train_step(loss_dev)
    assert_close(np.array([loss_dev.item()]), np.array([ref_loss]), "training loss")
    pad = (gpu.P + 3) // 4 * 4
    m = gpu.params_buf[pad:pad + gpu.P].cpu().numpy().astype(np.float64) / 0.1
    pos = 0
    for name, shape in A5.param_shapes():
        n = int(np.prod(shape))
        assert_close(m[pos:pos + n], grads_ref[name], f"gradient of {name}", rel=3e-2)
        pos += n
    assert_close(upd_after(gpu, upd), ora.topk_scatter(), "sparse update after the training step")
    gpu.check()


def test_resnet101_parameter_server_config():
    ora, gpu = run_workload("resnet101_ps", 4, state_every=3)
    assert gpu.L == 314 and gpu.N == 44_549_160 and gpu.idx.shape[0] == 16
    # two training steps of the parameter-server autoencoder (Section IV-A) at this size
    w = W.workload("resnet101_ps")
    src = W.GradientSource(w.table, w.num_nodes, seed=w.seed, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g = torch.empty((w.num_nodes, gpu.N), dtype=torch.float32, device="cuda")
    loss_dev = torch.zeros(1, device="cuda")
    for t in range(4, 6):
        src.step_into(t, g)
        ora.accumulate(g.cpu().numpy())
        gpu.accumulate(g)
        ora.topk()
        gpu.topk(0)
        common = W.choice_for_step(w.seed, t, w.num_nodes)
        ref_loss = ora.ae_train_step_ps(common)
        gpu.ae_train_step_ps(common, 1.0, 1.0, loss_dev)
        assert_close(np.array([loss_dev.item()]), np.array([ref_loss]), f"training loss at step {t}")
        assert_close(upd_after(gpu, upd), ora.topk_scatter(), f"sparse update at step {t}")
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "trained parameters")
    gpu.check()


def test_resnet101_parameter_server_config_with_the_full_size_autoencoder():
    # K = 16 decoders of Section IV-C's size, each with its node's innovation: mu = 44,657, code 4 x 2789
    ora, gpu = run_workload("resnet101_ps_ae5", 2, state_every=1)
    assert gpu.mu == 44_657 and gpu.P == 172_996 + 16 * 43_734


def upd_after(gpu, upd):
    gpu.topk_scatter(upd)
    return upd.cpu().numpy()


def test_segnet_config_with_autoencoder_training():
    w = W.workload("segnet")
    K = w.num_nodes
    ora, gpu = make_pair(w.table.numel, K, seed=w.seed)
    src = W.GradientSource(w.table, K, seed=w.seed, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g = torch.empty((K, gpu.N), dtype=torch.float32, device="cuda")
    loss_dev = torch.zeros(1, device="cuda")
    losses, losses_ref = [], []
    for t in range(w.ae_train_steps):                      # second phase: top-k updates while the AE trains
        src.step_into(t, g)
        choice = W.choice_for_step(w.seed, t, K)
        ora.accumulate(g.cpu().numpy())
        gpu.accumulate(g, choice)
        ora.topk(choice)
        gpu.topk(choice)
        losses_ref.append(ora.ae_train_step())
        gpu.ae_train_step(loss_dev)
        losses.append(loss_dev.item())
        if t % 10 == 0:
            assert_bitwise(gpu.idx.cpu().numpy(), ora.idx[:1], f"indices at training step {t}")
            assert_bitwise(gpu.val.cpu().numpy(), ora.val, f"values at training step {t}")
        ref = ora.topk_scatter()
        gpu.topk_scatter(upd)
        if t % 10 == 0 or t == w.ae_train_steps - 1:
            assert_close(upd.cpu().numpy(), ref, f"sparse update at training step {t}")
            assert_bitwise(gpu.v.cpu().numpy(), ora.v, f"v at training step {t}")
    assert_close(np.array(losses), np.array(losses_ref), "training losses")
    assert_close(gpu.get_ae_params().numpy(), ora.get_params(), "trained parameters")
    gpu.check()
    for t in range(w.ae_train_steps, w.ae_train_steps + 3):  # third phase: compressed updates
        src.step_into(t, g)
        compare_step(ora, gpu, g.cpu(), g, W.choice_for_step(w.seed, t, K), upd, check_state=(t == w.ae_train_steps + 2))


def rows_equal_bitwise(dev_row: torch.Tensor, host_row: np.ndarray, what: str, piece: int = 1 << 28):
    """Whole-row bitwise comparison of a device row with the oracle's host row, a GiB at a time."""
    n = dev_row.numel()
    assert host_row.size == n
    for a in range(0, n, piece):
        b = min(n, a + piece)
        ref = torch.from_numpy(host_row[a:b]).cuda().view(torch.int32)
        got = dev_row[a:b].view(torch.int32)
        if not torch.equal(got, ref):
            bad = torch.nonzero(got != ref).flatten()
            raise AssertionError(f"{what}: {bad.numel()} entries of [{a}, {b}) differ bitwise; first at {a + int(bad[0])}")
        del ref


def host_memory_available() -> int:
    import psutil
    return int(psutil.virtual_memory().available)


def test_stress_config():
    # 2^30 elements per node, K = 4.  With enough host memory the oracle carries the WHOLE state (u, v of all
    # four nodes, 32 GiB): every step its accumulation is compared with the device rows bit for bit over
    # the full length, the selection is the oracle's on the leader's full row, and the rows are compared
    # again in full after the sent entries have been cleared.  The autoencoder stages work on mu values
    # and are compared in full in either mode.  With less host memory the elementwise stages are compared
    # on two million sampled positions plus the row edges instead.
    w = W.workload("stress")
    K, N = w.num_nodes, w.table.total
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2**30:
        pytest.skip("needs about 70 GiB of free device memory")
    whole = host_memory_available() >= 56 * 2**30
    print(f"stress config: host memory available {host_memory_available() / 2**30:.0f} GiB -> "
          + ("whole-row comparison" if whole else "sampled comparison"))
    gpu = lgc.LGC(w.table.numel, K, density_ppm=w.density_ppm, momentum=w.momentum, c1=w.ae_c1, c2=w.ae_c2)
    params = W.ae_init_params(w.ae_c1, w.ae_c2, "rar", K, w.seed)
    gpu.set_ae_params(params)
    assert gpu.mu == 107_374 and (gpu.L1, gpu.L2) == (53_686, 26_842)
    # the oracle of the autoencoder stages works on mu-sized vectors in full
    ora = OracleLGC([gpu.mu * 1000], K, density_ppm=1000, c1=w.ae_c1, c2=w.ae_c2, params=params.numpy())
    assert ora.mu == gpu.mu
    m = float(np.float32(w.momentum))
    rng = np.random.default_rng(7)
    pos = np.unique(np.concatenate([rng.integers(0, N, 2_000_000), np.arange(0, 4096), np.arange(N - 4099, N)]))
    pos_dev = torch.from_numpy(pos).cuda()
    if whole:
        u_o = np.zeros((K, N), np.float32)
        v_o = np.zeros((K, N), np.float32)
    else:
        u_s = np.zeros((K, pos.size), np.float32)
        v_s = np.zeros((K, pos.size), np.float32)
    src = W.GradientSource(w.table, K, seed=w.seed, device="cuda", chunk=1 << 26)
    g = torch.empty((K, N), dtype=torch.float32, device="cuda")
    upd = torch.empty(N, dtype=torch.float32, device="cuda")
    for t in range(w.steps):
        src.step_into(t, g)
        leader = W.choice_for_step(w.seed, t, K)
        edge = t in (0, w.steps - 1)
        if not whole:
            g_s = g[:, pos_dev].cpu().numpy()
        gpu.accumulate(g, leader)
        for k in range(K):
            if whole:
                g_k = g[k].cpu().numpy()
                O.accumulate(u_o[k], v_o[k], g_k, m)
                del g_k
                if edge or k == leader:
                    rows_equal_bitwise(gpu.v[k], v_o[k], f"v of node {k} after the accumulation of step {t}")
                if edge:
                    rows_equal_bitwise(gpu.u[k], u_o[k], f"u of node {k} after the accumulation of step {t}")
            else:
                O.accumulate(u_s[k], v_s[k], np.ascontiguousarray(g_s[k]), m)
        if whole:
            assert_bitwise(gpu.u[:, pos_dev].cpu().numpy(), u_o[:, pos], f"sampled u, step {t}")
            assert_bitwise(gpu.v[:, pos_dev].cpu().numpy(), v_o[:, pos], f"sampled v, step {t}")
        else:
            assert_bitwise(gpu.u[:, pos_dev].cpu().numpy(), u_s, f"sampled u, step {t}")
            assert_bitwise(gpu.v[:, pos_dev].cpu().numpy(), v_s, f"sampled v, step {t}")
        gpu.topk(leader, upd)
        idx = gpu.idx.cpu().numpy()[0]
        ref_idx = leader_vals = None
        if whole or edge:                                  # the selection against the oracle, whole row
            v_leader = v_o[leader] if whole else gpu.v[leader].cpu().numpy()
            ref_idx = O.topk(v_leader, gpu.mu, method="select")
            assert_bitwise(idx, ref_idx, f"selected indices, step {t}")
            leader_vals = O.gather(v_leader, ref_idx)
            del v_leader
        assert np.all(np.diff(idx) > 0)
        idx_dev = gpu.idx[0].long()
        gpu.encode()
        val = gpu.val.cpu().numpy()
        if whole:                                          # the oracle's gather on its own rows
            assert_bitwise(val, np.stack([O.gather(v_o[k], ref_idx) for k in range(K)]), "gathered values")
        else:
            assert_bitwise(val, gpu.v[:, idx_dev].cpu().numpy(), "gathered values")  # same bits as v at idx
            if leader_vals is not None:
                assert_bitwise(val[leader], leader_vals, "leader values against the oracle's gather")
        ora.idx = np.broadcast_to(idx, (K, gpu.mu)).copy()
        ora.val = val.copy()
        ora.encode()
        assert_close(gpu.code.cpu().numpy(), ora.z.reshape(K, -1), "codes")
        ora.combine()
        gpu.combine(leader)
        assert_close(gpu.combined.cpu().numpy(), ora.zbar, "mean code")
        ora.decode()
        gpu.decode_scatter(upd)
        assert_close(gpu.recon.cpu().numpy(), ora.r, "reconstruction")
        assert_close(upd[idx_dev].cpu().numpy(), ora.r[0], "update at the scatter positions")
        assert int(torch.count_nonzero(upd).item()) <= gpu.mu
        assert float(upd.abs().sum().item()) == pytest.approx(float(np.abs(ora.r[0].astype(np.float32)).sum()), rel=1e-4)
        if whole:
            for k in range(K):
                O.clear(u_o[k], v_o[k], ref_idx)
                if edge:
                    rows_equal_bitwise(gpu.u[k], u_o[k], f"u of node {k} after the clearing of step {t}")
                    rows_equal_bitwise(gpu.v[k], v_o[k], f"v of node {k} after the clearing of step {t}")
            assert_bitwise(gpu.v[:, pos_dev].cpu().numpy(), v_o[:, pos], f"sampled v after clearing, step {t}")
        else:
            sent = np.isin(pos, idx)
            u_s[:, sent] = 0
            v_s[:, sent] = 0
            assert_bitwise(gpu.v[:, pos_dev].cpu().numpy(), v_s, f"sampled v after clearing, step {t}")
        assert not gpu.v[:, idx_dev].any().item() and not gpu.u[:, idx_dev].any().item()
        gpu.check()


def test_resnet50_config_with_the_layer_treatment_of_the_paper():
    # Section VI-A on the ResNet-50-shaped table: first tensor dense, the classifier's two tensors top-k only,
    # everything in between through the autoencoder; one step of each phase of Section V-B and two more compressed
    from oracle.phases import OraclePhased
    from paper_2103_08870_b200.phases import PhasedLGC
    w = W.workload("resnet50")
    K, numel = w.num_nodes, w.table.numel
    modes = ["dense"] + ["ae"] * (len(numel) - 3) + ["topk", "topk"]
    params = W.ae_init_params(w.ae_c1, w.ae_c2, "rar", K, w.seed)
    gpu = PhasedLGC(numel, modes, K, density_ppm=w.density_ppm, momentum=w.momentum)
    gpu.ctx.set_ae_params(params)
    ora = OraclePhased(numel, modes, K, {1: params.numpy()}, density_ppm=w.density_ppm, momentum=w.momentum)
    src = W.GradientSource(w.table, K, seed=w.seed, device="cuda")
    upd = torch.empty(gpu.N, dtype=torch.float32, device="cuda")
    g = torch.empty((K, gpu.N), dtype=torch.float32, device="cuda")
    for t, phase in enumerate(["raw", "topk_train", "compressed", "compressed", "compressed"]):
        src.step_into(t, g)
        choice = W.choice_for_step(w.seed, t, K)
        gpu.step(g, upd, phase, choice)
        ref, _ = ora.step(g.cpu().numpy(), phase, choice)
        assert_close(upd.cpu().numpy(), ref, f"step {t} ({phase}): update")
    v = gpu.ctx.v.cpu().numpy()
    for gr in ora.groups:
        if gr["mode"] == "dense":
            assert not v[:, gr["a"]:gr["b"]].any(), "the dense layer holds state"
        else:
            assert_bitwise(v[:, gr["a"]:gr["b"]], gr["o"].v, f"residual of the {gr['mode']} layers")
    large, served, _, _, _ = gpu.ctx.selection_stats()
    assert served > 0, "the accumulation collected no candidates for the one context"
    gpu.check()
