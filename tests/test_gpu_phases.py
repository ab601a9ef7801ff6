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


@pytest.mark.parametrize("variant, K", [("rar", 4), ("ps", 3)])
def test_three_phases_against_the_oracle(variant, K):
    c1, c2 = 8, 4
    params = W.ae_init_params(c1, c2, variant, K, 5)
    gpu = PhasedLGC(NUMEL, MODES, K, variant=variant, c1=c1, c2=c2)
    gpu.ae_runs()[0].ctx.set_ae_params(params)
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
        for r, gr in zip(gpu.runs, ora.groups):
            if r.ctx is not None:
                assert_bitwise(r.ctx.v.cpu().numpy(), gr["o"].v, f"step {t}: residual of run {r.mode}")
                assert_bitwise(r.ctx.u.cpu().numpy(), gr["o"].u, f"step {t}: velocity of run {r.mode}")
    assert_close(gpu.ae_runs()[0].ctx.get_ae_params().numpy(), ora.groups[1]["o"].get_params(), "trained parameters")
    gpu.check()


@pytest.mark.parametrize("variant", ["rar", "ps"])
def test_three_phases_with_the_full_size_autoencoder(variant):
    # the same schedule with Section IV-C's autoencoder on the middle layers (mu = 96 kept values there).
    # eps = 1e-2 keeps Adam's step well conditioned, so that the two sides' parameters stay together
    # through the training phase (see test_full_size_autoencoder_training_phase in test_gpu_parity.py).
    K = 2
    params = W.ae5_init_params(5, variant, K)
    gpu = PhasedLGC(NUMEL, MODES, K, variant=variant, ae_kind="conv5", eps=1e-2)
    gpu.ae_runs()[0].ctx.set_ae_params(params)
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
    assert_close(gpu.ae_runs()[0].ctx.get_ae_params().numpy(), ora.groups[1]["o"].get_params(), "trained parameters",
                 rel=1e-5 if variant == "rar" else 2e-4)
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
