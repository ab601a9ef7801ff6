"""Stage-by-stage comparison of the CUDA path (through the C ABI) with the CPU oracle."""
import numpy as np
import torch

from oracle import OracleLGC
from paper_2103_08870_b200 import lgc
from paper_2103_08870_b200 import workloads as W

REL_TOL = 1e-5      # autoencoder outputs: max|a - b| <= REL_TOL * max|ref|  (fp32 against the fp64 oracle)


def bits(a):
    a = np.ascontiguousarray(a)
    return a.view(np.uint32) if a.dtype == np.float32 else a


def assert_bitwise(got, ref, what):
    got, ref = np.asarray(got), np.asarray(ref)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    if not np.array_equal(bits(got), bits(ref)):
        bad = np.flatnonzero(bits(got).reshape(-1) != bits(ref).reshape(-1))
        raise AssertionError(f"{what}: {bad.size} of {got.size} entries differ bitwise; first at {bad[:5]}: "
                             f"{got.reshape(-1)[bad[:5]]} vs {ref.reshape(-1)[bad[:5]]}")


def assert_close(got, ref, what, rel=REL_TOL):
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    ref = np.asarray(ref, dtype=np.float64).reshape(-1)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    scale = max(np.abs(ref).max(), 1e-30)
    err = np.abs(got - ref).max()
    assert err <= rel * scale, f"{what}: max error {err:.3e} > {rel:.0e} * {scale:.3e}"


def assert_close_elementwise(got, ref, what, rel=REL_TOL, floor=2e-6):
    """Entry by entry: |a - b| <= rel * |ref| + floor * max|ref|.  The floor is the rounding of the fp32
    sums themselves (up to 49 terms at the vector's scale); above it every entry is held to `rel` of its
    own magnitude, so small entries are not covered by the largest one."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    ref = np.asarray(ref, dtype=np.float64).reshape(-1)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    scale = max(np.abs(ref).max(), 1e-30)
    excess = np.abs(got - ref) - (rel * np.abs(ref) + floor * scale)
    worst = int(np.argmax(excess))
    assert excess[worst] <= 0, (f"{what}: entry {worst}: {got[worst]!r} vs {ref[worst]!r} "
                                f"(allowed {rel:.0e} of the entry + {floor:.0e} of {scale:.3e})")


def make_pair(numel, K, variant="rar", ae_kind="conv2", c1=8, c2=4, density_ppm=1000, momentum=0.9,
              innovation_permille=100, seed=W.DEFAULT_SEED, topk_method="auto", **adam):
    """`adam`: lr, beta1, beta2, eps for both sides (defaults 1e-3, 0.9, 0.999, 1e-8)."""
    params = None
    if ae_kind == "conv2":
        params = W.ae_init_params(c1, c2, variant, K, seed)
    elif ae_kind == "conv5":
        params = W.ae5_init_params(seed, variant, K)
    ora = OracleLGC(numel, K, density_ppm=density_ppm, momentum=momentum, variant=variant, ae_kind=ae_kind,
                    c1=c1, c2=c2, params=None if params is None else params.numpy(),
                    innovation_permille=innovation_permille, topk_method=topk_method, **adam)
    gpu = lgc.LGC(numel, K, density_ppm=density_ppm, momentum=momentum, variant=variant, ae_kind=ae_kind,
                  c1=c1, c2=c2, innovation_permille=innovation_permille, **adam)
    if params is not None:
        gpu.set_ae_params(params)
    assert (gpu.N, gpu.mu) == (ora.N, ora.mu) and gpu.k_l == ora.k_l
    if ae_kind == "conv2":
        assert (gpu.L1, gpu.L2) == (ora.L1, ora.L2)
    return ora, gpu


def compare_step(ora, gpu, g_cpu: torch.Tensor, g_dev: torch.Tensor, choice: int, update_dev: torch.Tensor,
                 check_state=True, hint="leader", announce_update=True, rel=REL_TOL):
    """One full compression step on both sides, compared after every stage.  `hint`: what
    lgc_accumulate is told about the coming leader ("leader", "none", or "wrong");
    `announce_update`: whether lgc_topk is told the update buffer (and clears it early)."""
    K = ora.K
    ora.accumulate(g_cpu.numpy())
    gpu.accumulate(g_dev, {"leader": choice, "none": -1, "wrong": (choice + 1) % K}[hint])
    if check_state:
        assert_bitwise(gpu.u.cpu().numpy(), ora.u, "u after accumulate")
        assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v after accumulate")
    ora.topk(choice)
    if announce_update:
        update_dev.fill_(float("nan"))           # whatever is there must be overwritten
    gpu.topk(choice, update_dev if announce_update else None)
    idx_ref = ora.idx if ora.variant == "ps" else ora.idx[:1]
    assert_bitwise(gpu.idx.cpu().numpy(), idx_ref, "selected indices")
    ora.encode()
    gpu.encode()
    assert_bitwise(gpu.val.cpu().numpy(), ora.val, "gathered values")     # valid once the encoder has run
    if ora.ae_kind == "conv5":               # the library keeps these codes position-major: [K][L4][4]
        assert_close(gpu.code.cpu().numpy(), ora.z.transpose(0, 2, 1).reshape(K, -1), "codes", rel=rel)
    else:
        assert_close(gpu.code.cpu().numpy(), ora.z.reshape(K, -1), "codes")
        if ora.ae_kind == "conv2":
            assert_close_elementwise(gpu.code.cpu().numpy(), ora.z.reshape(K, -1), "codes, entry by entry")
    ora.combine(choice)
    gpu.combine(choice)
    if ora.variant == "rar":
        zbar = ora.zbar.T if ora.ae_kind == "conv5" else ora.zbar
        assert_close(gpu.combined.cpu().numpy(), zbar, "mean code", rel=rel)
    else:
        assert_close(gpu.combined.cpu().numpy(), ora.zc.T if ora.ae_kind == "conv5" else ora.zc, "common code", rel=rel)
        assert_bitwise(gpu.inn.cpu().numpy(), ora.inn, "innovation")
    upd_ref = ora.decode_scatter()
    gpu.decode_scatter(update_dev)
    if not (ora.variant == "rar" and ora.ae_kind == "identity"):
        assert_close(gpu.recon.cpu().numpy(), ora.r, "reconstruction", rel=rel)
        if ora.ae_kind == "conv2":
            assert_close_elementwise(gpu.recon.cpu().numpy(), ora.r, "reconstruction, entry by entry")
    upd = update_dev.cpu().numpy()
    assert_close(upd, upd_ref, "dense update", rel=rel)
    touched = np.zeros(ora.N, bool)
    touched[ora.idx.reshape(-1)] = True
    assert not upd[~touched].any(), "update is non-zero outside the scatter positions"
    if check_state:
        assert_bitwise(gpu.u.cpu().numpy(), ora.u, "u after clearing")
        assert_bitwise(gpu.v.cpu().numpy(), ora.v, "v after clearing")
    gpu.check()
