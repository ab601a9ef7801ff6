"""Seeded synthetic inputs for the LGC compression path.

This module only *makes inputs*: layer tables shaped like the networks the paper trains
(ResNet-50 / ResNet-101 parameter shapes, a segmentation-net-like size mix), per-step node
gradients ``g_k = s + 0.3 n_k`` with a heavy-tailed part ``s`` shared by all nodes and a
Gaussian part ``n_k`` private to node ``k`` (the "common + innovation" structure of Section
III / Section IV-A of the paper), and uniformly initialised autoencoder parameters.  It holds
none of the method's arithmetic (no accumulation, selection, convolution or optimiser code) and
is used both by the CUDA path's tests/benchmark and by the CPU oracle's tests.

Randomness is counter based: every value is a pure function of ``(seed, step, stream,
element)`` through the published splitmix64 finaliser, so any element can be produced on its
own and the CPU and a CUDA device evaluate the same integer stream.  The float transforms
(``log``, ``cos``) may differ in the last bit between devices, so a comparison always
generates a tensor ONCE and hands the same bytes to both sides.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import torch

MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
DEFAULT_SEED = 20210308

STREAM_SHARED = 0x5348          # the shared component s
STREAM_NODE = 0x4E4F0000        # + node index: the private component n_k
STREAM_AE = 0x41450000          # autoencoder parameter draws
STREAM_SIZES = 0x53495A45       # segmentation-net size draws
STREAM_CHOICE = 0x43484F49      # per-step leader / common-node choice


# --------------------------------------------------------------------------------------
# splitmix64: python-int version (tables, keys) and torch int64 version (bulk draws)
# --------------------------------------------------------------------------------------
def splitmix64(x: int) -> int:
    """The splitmix64 output function (Steele, Lea, Flood 2014) on a python int."""
    z = (x + _GOLDEN) & MASK64
    z = ((z ^ (z >> 30)) * _M1) & MASK64
    z = ((z ^ (z >> 27)) * _M2) & MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, step: int, stream: int) -> int:
    """One 64-bit key per (seed, step, stream)."""
    k = splitmix64(seed & MASK64)
    k = splitmix64(k ^ ((step & MASK64) * 0xD1342543DE82EF95 & MASK64))
    k = splitmix64(k ^ ((stream & MASK64) * 0xA0761D6478BD642F & MASK64))
    return k


def _s64(x: int) -> int:
    """Reinterpret an unsigned 64-bit python int as the signed value torch.int64 stores."""
    x &= MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 tensors (torch's ``>>`` is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def hash_counters(key: int, counters: torch.Tensor) -> torch.Tensor:
    """splitmix64(key ^ (counter * golden)) elementwise; int64 in, int64 (bit pattern) out."""
    z = counters * _s64(_GOLDEN)
    z = z ^ _s64(key)
    z = z + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def hash_counter_int(key: int, counter: int) -> int:
    """Python-int twin of :func:`hash_counters` for one counter."""
    return splitmix64((key ^ ((counter * _GOLDEN) & MASK64)) & MASK64)


def _uniform23(bits: torch.Tensor) -> torch.Tensor:
    """23-bit integers -> fp32 in (0,1), exactly representable: (x + 0.5) / 2^23."""
    return (bits.to(torch.float32) + 0.5) * (1.0 / 8388608.0)


def unit_laplace(key: int, start: int, count: int, device) -> torch.Tensor:
    """Laplace(0,1) draws for counters start..start+count-1 (inverse CDF), fp32."""
    c = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = hash_counters(key, c)
    u = _uniform23(_lsr(h, 41)) - 0.5                      # exact, in (-0.5, 0.5)
    mag = -torch.log(1.0 - 2.0 * u.abs())
    return torch.where(u < 0, -mag, mag)


def unit_gauss(key: int, start: int, count: int, device) -> torch.Tensor:
    """N(0,1) draws for counters start..start+count-1 (Box-Muller, cosine branch), fp32."""
    c = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = hash_counters(key, c)
    u1 = _uniform23(_lsr(h, 41))
    u2 = _uniform23(_lsr(h, 18) & 0x7FFFFF)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


# --------------------------------------------------------------------------------------
# layer tables
# --------------------------------------------------------------------------------------
@dataclass
class LayerTable:
    """Per-tensor element counts n_l and fan-in (for the value scale b_l = base/sqrt(fan_in))."""
    name: str
    numel: List[int]
    fan_in: List[int]
    labels: List[str] = field(default_factory=list)

    @property
    def total(self) -> int:
        return sum(self.numel)

    def offsets(self) -> List[int]:
        out, acc = [], 0
        for n in self.numel:
            out.append(acc)
            acc += n
        return out


def _resnet_bottleneck_table(name: str, blocks: Sequence[int], num_classes: int = 1000) -> LayerTable:
    """Parameter tensors of a bottleneck ResNet in definition order.

    Stem 7x7 conv + BN; four stages of bottleneck blocks (1x1 -> 3x3 -> 1x1 with expansion 4,
    each followed by a BN weight and bias), a 1x1 projection + BN on the first block of every
    stage; a fully connected classifier with bias.  Only shapes are produced.
    """
    numel: List[int] = []
    fan: List[int] = []
    labels: List[str] = []

    def conv(label, cout, cin, kh, kw):
        numel.append(cout * cin * kh * kw)
        fan.append(cin * kh * kw)
        labels.append(label)

    def bn(label, c):
        for part in ("weight", "bias"):
            numel.append(c)
            fan.append(1)
            labels.append(f"{label}.{part}")

    conv("conv1", 64, 3, 7, 7)
    bn("bn1", 64)
    inplanes = 64
    for stage, (planes, nblk) in enumerate(zip((64, 128, 256, 512), blocks), start=1):
        for b in range(nblk):
            p = f"layer{stage}.{b}"
            conv(f"{p}.conv1", planes, inplanes, 1, 1)
            bn(f"{p}.bn1", planes)
            conv(f"{p}.conv2", planes, planes, 3, 3)
            bn(f"{p}.bn2", planes)
            conv(f"{p}.conv3", planes * 4, planes, 1, 1)
            bn(f"{p}.bn3", planes * 4)
            if b == 0:
                conv(f"{p}.downsample.0", planes * 4, inplanes, 1, 1)
                bn(f"{p}.downsample.1", planes * 4)
            inplanes = planes * 4
    numel.append(num_classes * inplanes)
    fan.append(inplanes)
    labels.append("fc.weight")
    numel.append(num_classes)
    fan.append(1)
    labels.append("fc.bias")
    return LayerTable(name, numel, fan, labels)


def resnet50_table() -> LayerTable:
    return _resnet_bottleneck_table("resnet50", (3, 4, 6, 3))


def resnet101_table() -> LayerTable:
    return _resnet_bottleneck_table("resnet101", (3, 4, 23, 3))


def flat_table(n: int, name: str = "flat") -> LayerTable:
    return LayerTable(name, [int(n)], [1], ["flat"])


def segnet_table(seed: int = DEFAULT_SEED, count: int = 220, total: int = 65_000_000,
                 lo: int = 64, hi: int = 2_400_000) -> LayerTable:
    """``count`` tensor sizes, log-uniform in [lo, hi], rescaled so that they sum to ``total``.

    Draw r_l = exp(U(ln lo, ln hi)); find by bisection the factor c with
    sum(clamp(floor(c r_l), lo, hi)) <= total as large as possible; hand the remaining elements
    out one at a time, round robin in tensor order, to tensors still below ``hi``.  No tensor
    shapes exist for this stand-in, so fan_in_l = max(1, floor(3 sqrt(n_l))): what a square
    3x3 convolution with n_l weights would have.
    """
    key = stream_key(seed, 0, STREAM_SIZES)
    raw = []
    for l in range(count):
        u = ((hash_counter_int(key, l) >> 11) + 0.5) / float(1 << 53)
        raw.append(math.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))))

    def sizes_for(c: float) -> List[int]:
        return [min(hi, max(lo, int(c * r))) for r in raw]

    lo_c, hi_c = 0.0, 1.0
    while sum(sizes_for(hi_c)) <= total and hi_c < 1e9:
        hi_c *= 2.0
    for _ in range(200):
        mid = 0.5 * (lo_c + hi_c)
        if sum(sizes_for(mid)) <= total:
            lo_c = mid
        else:
            hi_c = mid
    sizes = sizes_for(lo_c)
    rest = total - sum(sizes)
    if rest < 0 or all(s >= hi for s in sizes) and rest > 0:
        raise ValueError("segnet_table: total not reachable within [lo, hi]")
    l = 0
    while rest > 0:
        if sizes[l] < hi:
            sizes[l] += 1
            rest -= 1
        l = (l + 1) % count
    fan = [max(1, int(3.0 * math.sqrt(n))) for n in sizes]
    return LayerTable("segnet", sizes, fan, [f"t{l}" for l in range(count)])


# --------------------------------------------------------------------------------------
# gradients
# --------------------------------------------------------------------------------------
class GradientSource:
    """Per-step node gradients ``g_k = b_l (s + 0.3 n_k)`` on a layer table.

    ``s`` ~ Laplace(0,1) is drawn once per step and shared by every node, ``n_k`` ~ N(0,1) is
    private to node k; b_l = base_scale / sqrt(fan_in_l) is constant inside a tensor.  Values
    are fp32.  ``device`` chooses where the draws are evaluated; ``chunk`` bounds temporaries.
    """

    def __init__(self, table: LayerTable, num_nodes: int, seed: int = DEFAULT_SEED,
                 base_scale: float = 1e-3, device="cpu", chunk: int = 1 << 24):
        self.table = table
        self.K = int(num_nodes)
        self.N = table.total
        self.seed = int(seed)
        self.device = torch.device(device)
        self.chunk = int(chunk)
        scales = [base_scale / math.sqrt(f) for f in table.fan_in]
        if len(scales) == 1:
            self._scale = float(torch.tensor(scales[0], dtype=torch.float32).item())
            self._scale_vec = None
        else:
            sv = torch.tensor(scales, dtype=torch.float32)
            reps = torch.tensor(table.numel, dtype=torch.int64)
            self._scale_vec = torch.repeat_interleave(sv, reps).to(self.device)
            self._scale = None

    def _scaled(self, x: torch.Tensor, start: int) -> torch.Tensor:
        if self._scale_vec is None:
            return x * self._scale
        return x * self._scale_vec[start:start + x.numel()]

    def step_into(self, step: int, out: torch.Tensor) -> torch.Tensor:
        """Fill ``out`` ([K, N] fp32 on self.device) with the gradients of ``step``."""
        assert out.shape == (self.K, self.N) and out.dtype == torch.float32
        ks = stream_key(self.seed, step, STREAM_SHARED)
        for start in range(0, self.N, self.chunk):
            cnt = min(self.chunk, self.N - start)
            s = unit_laplace(ks, start, cnt, self.device)
            for k in range(self.K):
                kn = stream_key(self.seed, step, STREAM_NODE + k)
                n = unit_gauss(kn, start, cnt, self.device)
                out[k, start:start + cnt] = self._scaled(s + 0.3 * n, start)
        return out

    def step(self, step: int) -> torch.Tensor:
        out = torch.empty((self.K, self.N), dtype=torch.float32, device=self.device)
        return self.step_into(step, out)


def choice_for_step(seed: int, step: int, num_nodes: int) -> int:
    """The node that leads the selection (ring-allreduce) or sends the common code
    (parameter server) at ``step``: a hash of (seed, step) modulo K."""
    return int(hash_counter_int(stream_key(seed, step, STREAM_CHOICE), 0) % num_nodes)


# --------------------------------------------------------------------------------------
# autoencoder parameters (flat fp32 vector; tensor order documented in include/lgc.h)
# --------------------------------------------------------------------------------------
def ae_param_shapes(c1: int, c2: int, variant: str, num_nodes: int) -> List[Tuple[str, Tuple[int, ...], int]]:
    """(name, shape, fan_in) of every tensor of the flat parameter vector, in order.

    fan_in 0 marks the parameter-server fusion scalars, which start at (1, 1, 0).
    """
    enc = [("enc.w1", (c1, 1, 3), 3), ("enc.b1", (c1,), 3),
           ("enc.w2", (c2, c1, 3), 3 * c1), ("enc.b2", (c2,), 3 * c1)]

    def dec(prefix: str):
        return [(f"{prefix}.w1", (c2, c1, 3), 3 * c2), (f"{prefix}.b1", (c1,), 3 * c2),
                (f"{prefix}.w2", (c1, 1, 3), 3 * c1), (f"{prefix}.b2", (1,), 3 * c1)]

    if variant == "rar":
        return enc + dec("dec")
    if variant == "ps":
        out = list(enc)
        for k in range(num_nodes):
            out += dec(f"dec{k}") + [(f"dec{k}.fuse", (3,), 0)]
        return out
    raise ValueError(variant)


def ae_param_count(c1: int, c2: int, variant: str, num_nodes: int) -> int:
    return sum(math.prod(s) for _, s, _ in ae_param_shapes(c1, c2, variant, num_nodes))


def ae_init_params(c1: int, c2: int, variant: str, num_nodes: int, seed: int = DEFAULT_SEED) -> torch.Tensor:
    """U(-1/sqrt(fan_in), +1/sqrt(fan_in)) for every weight and bias (fan_in = C_in * 3),
    fusion scalars (w0, w1, b) = (1, 1, 0); flat fp32 CPU tensor."""
    key = stream_key(seed, 0, STREAM_AE)
    parts = []
    ctr = 0
    for _, shape, fan in ae_param_shapes(c1, c2, variant, num_nodes):
        n = math.prod(shape)
        if fan == 0:
            parts.append(torch.tensor([1.0, 1.0, 0.0], dtype=torch.float32))
        else:
            c = torch.arange(ctr, ctr + n, dtype=torch.int64)
            u = _uniform23(_lsr(hash_counters(key, c), 41))
            bound = 1.0 / math.sqrt(fan)
            parts.append(((2.0 * u - 1.0) * bound).to(torch.float32))
        ctr += n
    return torch.cat(parts)


def ae5_param_shapes(variant: str = "rar", num_nodes: int = 1) -> List[Tuple[str, Tuple[int, ...], int]]:
    """(name, shape, fan_in) of the full-size autoencoder's tensors (Section IV-C: encoder filters
    64/128/256/64 of 3 taps and 4 of 1 tap; decoder filters 4/32/64/128/32 of 3 taps and one 1-tap
    filter), in the order of the flat parameter vector.  Convolutions: w[co][ci][tap]; transposed
    convolutions: w[ci][co][tap].  Parameter server: one decoder per node, whose last filter has a
    33rd tap on the node's innovation (Section IV-A)."""
    enc_ch, dec_ch = [1, 64, 128, 256, 64], [4, 4, 32, 64, 128, 32]
    out = []
    for i in range(4):
        fan = 3 * enc_ch[i]
        out += [(f"enc.w{i + 1}", (enc_ch[i + 1], enc_ch[i], 3), fan), (f"enc.b{i + 1}", (enc_ch[i + 1],), fan)]
    out += [("enc.w5", (4, 64, 1), 64), ("enc.b5", (4,), 64)]
    ps = variant == "ps"
    for k in range(num_nodes if ps else 1):
        pre = f"dec{k}" if ps else "dec"
        for i in range(5):
            fan = 3 * dec_ch[i]
            out += [(f"{pre}.w{i + 1}", (dec_ch[i], dec_ch[i + 1], 3), fan), (f"{pre}.b{i + 1}", (dec_ch[i + 1],), fan)]
        taps = 33 if ps else 32
        out += [(f"{pre}.w6", (1, taps, 1), taps), (f"{pre}.b6", (1,), taps)]
    return out


def ae5_init_params(seed: int = DEFAULT_SEED, variant: str = "rar", num_nodes: int = 1) -> torch.Tensor:
    """U(-1/sqrt(fan_in), +1/sqrt(fan_in)) for every tensor of the full-size autoencoder; flat
    fp32 CPU tensor."""
    key = stream_key(seed, 1, STREAM_AE)
    parts = []
    ctr = 0
    for _, shape, fan in ae5_param_shapes(variant, num_nodes):
        n = math.prod(shape)
        c = torch.arange(ctr, ctr + n, dtype=torch.int64)
        u = _uniform23(_lsr(hash_counters(key, c), 41))
        parts.append(((2.0 * u - 1.0) * (1.0 / math.sqrt(fan))).to(torch.float32))
        ctr += n
    return torch.cat(parts)


# --------------------------------------------------------------------------------------
# the five workload configurations
# --------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    table: LayerTable
    num_nodes: int
    density_ppm: int
    variant: str            # "rar" | "ps"
    ae_c1: int
    ae_c2: int
    steps: int
    ae_train_steps: int = 0
    momentum: float = 0.9
    innovation_permille: int = 100
    seed: int = DEFAULT_SEED
    ae_kind: str = "conv2"    # "conv2": two layers each way with (ae_c1, ae_c2) channels; "conv5": the full-size one

    def init_params(self) -> torch.Tensor:
        """The autoencoder's seeded initial parameters, flat fp32 on the CPU."""
        if self.ae_kind == "conv5":
            return ae5_init_params(self.seed, self.variant, self.num_nodes)
        return ae_init_params(self.ae_c1, self.ae_c2, self.variant, self.num_nodes, self.seed)


def workload(name: str) -> Workload:
    if name == "tiny":
        return Workload("tiny", flat_table(1 << 20), 2, 1000, "rar", 8, 4, 3)
    if name == "resnet50":
        return Workload("resnet50", resnet50_table(), 8, 1000, "rar", 8, 4, 10)
    if name == "resnet101_ps":
        return Workload("resnet101_ps", resnet101_table(), 16, 1000, "ps", 16, 8, 10)
    if name == "segnet":
        return Workload("segnet", segnet_table(), 4, 1000, "rar", 8, 4, 10, ae_train_steps=50)
    if name == "stress":
        return Workload("stress", flat_table(1 << 30), 4, 100, "rar", 16, 8, 5)
    if name == "resnet50_ae5":      # the ResNet-50-shaped case with the paper's full-size autoencoder
        return Workload("resnet50_ae5", resnet50_table(), 8, 1000, "rar", 64, 4, 10, ae_kind="conv5")
    if name == "resnet101_ps_ae5":  # the ResNet-101-shaped parameter-server case with the full-size autoencoder
        return Workload("resnet101_ps_ae5", resnet101_table(), 16, 1000, "ps", 64, 4, 10, ae_kind="conv5")
    raise KeyError(name)


WORKLOAD_NAMES = ("tiny", "resnet50", "resnet101_ps", "segnet", "stress", "resnet50_ae5", "resnet101_ps_ae5")
