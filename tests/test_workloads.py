"""The seeded input generators: layer tables, the counter-based stream, value model."""
import math
import os

import numpy as np
import torch

from paper_2103_08870_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "layout_counts.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = int(v)
    return out


def test_resnet_tables_match_published_counts():
    g = golden()
    t50, t101 = W.resnet50_table(), W.resnet101_table()
    assert len(t50.numel) == g["resnet50_tensors"] and t50.total == g["resnet50_elements"]
    assert len(t101.numel) == g["resnet101_tensors"] and t101.total == g["resnet101_elements"]
    assert min(t50.numel) == 64 and max(t50.numel) == 2359296
    assert t50.numel[0] == 64 * 3 * 7 * 7 and t50.fan_in[0] == 147
    assert t50.numel[-2:] == [2048 * 1000, 1000] and t50.fan_in[-2:] == [2048, 1]


def test_segnet_table():
    t = W.segnet_table()
    assert len(t.numel) == 220 and t.total == 65_000_000
    assert min(t.numel) >= 64 and max(t.numel) <= 2_400_000
    assert W.segnet_table().numel == t.numel          # deterministic
    logs = np.log(np.array(t.numel, dtype=np.float64))
    assert logs.std() > 1.5                            # spread over orders of magnitude


def test_torch_stream_equals_python_stream():
    key = W.stream_key(123, 4, 5)
    c = torch.tensor([0, 1, 2, 1000, 2**31, 2**40 + 7], dtype=torch.int64)
    got = [x & W.MASK64 for x in W.hash_counters(key, c).tolist()]
    assert got == [W.hash_counter_int(key, int(i)) for i in c.tolist()]
    # splitmix64 reference value: first output of the generator seeded with 0
    assert W.splitmix64(0) == 0xE220A8397B1DCDAF


def test_gradient_value_model():
    src = W.GradientSource(W.flat_table(1 << 18), 3, seed=7)
    g = src.step(0)
    assert g.shape == (3, 1 << 18) and g.dtype == torch.float32
    # random access: a chunked evaluation gives the same bytes
    src2 = W.GradientSource(W.flat_table(1 << 18), 3, seed=7, chunk=4099)
    assert torch.equal(g, src2.step(0))
    assert not torch.equal(g, src.step(1))
    # s ~ Laplace(0,b): var 2 b^2 ; 0.3 n: var 0.09 b^2 ; correlation between nodes 2/2.09
    b = 1e-3
    assert abs(g.var().item() / (2.09 * b * b) - 1) < 0.05
    c = torch.corrcoef(g)[0, 1].item()
    assert abs(c - 2 / 2.09) < 0.01
    # heavy tail: kurtosis well above the Gaussian 3
    x = g[0].double()
    assert (x**4).mean() / (x**2).mean() ** 2 > 4.5


def test_per_layer_scale():
    t = W.LayerTable("toy", [4096, 4096], [1, 64])
    g = W.GradientSource(t, 1, seed=3).step(0)[0]
    ratio = g[:4096].std() / g[4096:].std()
    assert abs(ratio.item() - 8.0) < 0.8


def test_ae_params():
    g = golden()
    assert W.ae_param_count(8, 4, "rar", 2) == g["ae_params_8_4"]
    assert W.ae_param_count(16, 8, "rar", 4) == g["ae_params_16_8"]
    p = W.ae_init_params(8, 4, "rar", 2)
    assert p.numel() == 261 and p.dtype == torch.float32
    assert p[:24].abs().max() <= 1 / math.sqrt(3) and p[:24].abs().max() > 0.4
    ps = W.ae_init_params(8, 4, "ps", 3)
    assert ps.numel() == W.ae_param_count(8, 4, "ps", 3)
    assert ps[-3:].tolist() == [1.0, 1.0, 0.0]


def test_workload_definitions():
    for name in W.WORKLOAD_NAMES:
        w = W.workload(name)
        assert w.table.total > 0 and w.num_nodes >= 2
    assert W.workload("stress").table.total == 1 << 30
    assert 0 <= W.choice_for_step(1, 2, 8) < 8
