"""The three training phases of Section V-B of the paper and the per-layer treatment of
Section VI-A, composed from the C-ABI entry points.

Section V-B: (1) the first iterations exchange the original gradients; (2) then the weights are
updated with the top-magnitude gradients while the autoencoder trains on them; (3) from then on
the compressed path runs.  Section VI-A: the first layer's gradient is sent as it is, the last
layer's top-magnitude values are sent without the autoencoder, every layer in between goes
through top-k selection and the autoencoder.

One context serves the whole model: lgc_config.layer_mode gives every layer its treatment
("dense": the mean of the nodes' gradients, no state; "topk": accumulated and selected, the kept
values sent without the autoencoder; "ae": top-k selection and the autoencoder, whose input is the
concatenation of the kept values of all such layers).  The first phase is lgc_dense_mean over the
whole gradient.  This module only sequences calls and passes pointers: every step of the path runs
in the library's kernels.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import lgc

MODES = ("dense", "topk", "ae")
PHASES = ("raw", "topk_train", "compressed")


class Run:
    def __init__(self, mode: str, first: int, last: int, begin: int, end: int):
        self.mode, self.first, self.last, self.begin, self.end = mode, first, last, begin, end
        self.ctx: Optional[lgc.LGC] = None


def layer_runs(layer_numel: Sequence[int], layer_mode: Sequence[str]) -> List[Run]:
    """Maximal runs of consecutive layers with the same mode, with their element ranges."""
    if len(layer_numel) != len(layer_mode) or any(m not in MODES for m in layer_mode):
        raise ValueError("layer_mode: one of 'dense', 'topk', 'ae' per layer")
    runs: List[Run] = []
    at = 0
    for i, (n, m) in enumerate(zip(layer_numel, layer_mode)):
        if runs and runs[-1].mode == m:
            runs[-1].last, runs[-1].end = i + 1, at + int(n)
        else:
            runs.append(Run(m, i, i + 1, at, at + int(n)))
        at += int(n)
    return runs


class PhasedLGC:
    def __init__(self, layer_numel: Sequence[int], layer_mode: Sequence[str], num_nodes: int, density_ppm: int = 1000,
                 momentum: float = 0.9, variant: str = "rar", ae_kind: str = "conv2", c1: int = 8, c2: int = 4,
                 innovation_permille: int = 100, device: Optional[torch.device] = None, **adam):
        """`adam`: lr, beta1, beta2, eps of the autoencoder's training steps (defaults 1e-3, 0.9, 0.999, 1e-8)."""
        self.numel = [int(n) for n in layer_numel]
        self.N, self.K, self.variant = sum(self.numel), int(num_nodes), variant
        self.runs = layer_runs(self.numel, layer_mode)          # for callers that want the element ranges
        self.ctx = lgc.LGC(self.numel, num_nodes, density_ppm=density_ppm, momentum=momentum, variant=variant,
                           ae_kind=ae_kind, c1=c1, c2=c2, innovation_permille=innovation_permille, device=device,
                           layer_mode=list(layer_mode), **adam)

    def step(self, grads: torch.Tensor, update: torch.Tensor, phase: str, choice: int = 0,
             loss_out: Optional[torch.Tensor] = None) -> None:
        """One iteration: grads [K][N] fp32 CUDA (contiguous), update [N] fully written.
        choice: the ring-allreduce leader / the parameter server's common node of this iteration.
        `grads` must stay as it is until the step has run on the stream (the dense layers are read last)."""
        if phase not in PHASES:
            raise ValueError(phase)
        if tuple(grads.shape) != (self.K, self.N) or not grads.is_contiguous() or update.numel() != self.N:
            raise ValueError("grads must be a contiguous [K][N] tensor and update hold N elements")
        if phase == "raw":
            lgc.dense_mean(grads, update)
            return
        c = self.ctx
        c.accumulate(grads, choice)
        c.topk(choice, update)
        if phase == "topk_train":
            if c.ae_kind != "identity":
                if self.variant == "rar":
                    c.ae_train_step(loss_out)
                else:
                    c.ae_train_step_ps(choice, 1.0, 1.0, loss_out)
            c.topk_scatter(update)
        else:
            c.encode()
            c.combine(choice)
            c.decode_scatter(update)

    def check(self) -> None:
        self.ctx.check()
