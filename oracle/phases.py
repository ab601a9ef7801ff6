"""The phases of Section V-B and the per-layer treatment of Section VI-A on the CPU oracle.

TEST INFRASTRUCTURE ONLY.  Written from the definitions, layer by layer: a "dense" layer's update
is the node-ordered fp32 mean of its gradients and it keeps no residual; a "topk" layer is
accumulated and selected and its update is the mean over nodes of the kept values; "ae" layers in
a row share one autoencoder whose input is the concatenation of their kept values.
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from .pipeline import OracleLGC


def dense_mean(g: np.ndarray) -> np.ndarray:
    acc = g[0].astype(np.float32).copy()
    for k in range(1, g.shape[0]):
        acc = acc + g[k]                      # fp32, node order
    return acc / np.float32(g.shape[0])


class OraclePhased:
    def __init__(self, layer_numel: Sequence[int], layer_mode: Sequence[str], num_nodes: int, ae_params: Dict[int, np.ndarray],
                 **kw):
        self.numel = [int(n) for n in layer_numel]
        self.mode = list(layer_mode)
        self.K, self.N = num_nodes, sum(self.numel)
        self.off = np.concatenate([[0], np.cumsum(self.numel)]).astype(np.int64)
        self.groups: List[dict] = []          # consecutive layers of one mode
        for i, m in enumerate(self.mode):
            if self.groups and self.groups[-1]["mode"] == m:
                self.groups[-1]["last"] = i + 1
            else:
                self.groups.append({"mode": m, "first": i, "last": i + 1})
        for j, gr in enumerate(self.groups):
            gr["a"], gr["b"] = int(self.off[gr["first"]]), int(self.off[gr["last"]])
            if gr["mode"] != "dense":
                sub = dict(kw)
                if gr["mode"] == "topk":
                    sub["ae_kind"] = "identity"
                gr["o"] = OracleLGC(self.numel[gr["first"]:gr["last"]], num_nodes, params=ae_params.get(j) if gr["mode"] == "ae" else None, **sub)

    def step(self, g: np.ndarray, phase: str, choice: int = 0):
        upd = np.zeros(self.N, dtype=np.float32)
        losses = []
        if phase == "raw":
            return dense_mean(g), losses
        for gr in self.groups:
            a, b = gr["a"], gr["b"]
            gs = np.ascontiguousarray(g[:, a:b])
            if gr["mode"] == "dense":
                upd[a:b] = dense_mean(gs)
                continue
            o = gr["o"]
            o.accumulate(gs)
            o.topk(choice)
            if gr["mode"] == "topk" or phase == "topk_train":
                if gr["mode"] == "ae" and o.ae_kind != "identity":
                    losses.append(o.ae_train_step() if o.variant == "rar" else o.ae_train_step_ps(choice, 1.0, 1.0))
                upd[a:b] = o.topk_scatter()
            else:
                o.encode()
                o.combine(choice)
                upd[a:b] = o.decode_scatter()
        return upd, losses
