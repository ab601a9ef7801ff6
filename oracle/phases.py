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
    """grouping = "runs": consecutive layers of one mode form a group with a pipeline (and, for "ae",
    an autoencoder) of its own.  grouping = "modes": ALL layers of a mode form one group, wherever they
    lie: one autoencoder whose input is the concatenation, in layer order, of the kept values of every
    "ae" layer (Section VI-A: the layers in between the first and the last share the autoencoder), one
    top-k pipeline for every "topk" layer.  A group works on the concatenation of its layers' slices of
    the gradient; its update is cut back to those slices."""

    def __init__(self, layer_numel: Sequence[int], layer_mode: Sequence[str], num_nodes: int, ae_params: Dict[int, np.ndarray],
                 grouping: str = "runs", **kw):
        assert grouping in ("runs", "modes")
        self.numel = [int(n) for n in layer_numel]
        self.mode = list(layer_mode)
        self.K, self.N = num_nodes, sum(self.numel)
        self.off = np.concatenate([[0], np.cumsum(self.numel)]).astype(np.int64)
        self.groups: List[dict] = []
        for i, m in enumerate(self.mode):
            if grouping == "runs":
                same = self.groups[-1] if self.groups and self.groups[-1]["mode"] == m else None
            else:
                same = next((gr for gr in self.groups if gr["mode"] == m and m != "dense"), None)
            if same is not None:
                same["layers"].append(i)
            else:
                self.groups.append({"mode": m, "layers": [i]})
        for j, gr in enumerate(self.groups):
            gr["first"], gr["last"] = gr["layers"][0], gr["layers"][-1] + 1
            gr["ranges"] = [(int(self.off[l]), int(self.off[l + 1])) for l in gr["layers"]]
            gr["a"], gr["b"] = gr["ranges"][0][0], gr["ranges"][-1][1]
            if gr["mode"] != "dense":
                sub = dict(kw)
                if gr["mode"] == "topk":
                    sub["ae_kind"] = "identity"
                key = j if grouping == "runs" else 0
                gr["o"] = OracleLGC([self.numel[l] for l in gr["layers"]], num_nodes,
                                    params=ae_params.get(key) if gr["mode"] == "ae" else None, **sub)

    @staticmethod
    def _slices(g: np.ndarray, ranges) -> np.ndarray:
        return np.ascontiguousarray(np.concatenate([g[:, a:b] for a, b in ranges], axis=1))

    @staticmethod
    def _put(upd: np.ndarray, ranges, values: np.ndarray) -> None:
        at = 0
        for a, b in ranges:
            upd[a:b] = values[at:at + (b - a)]
            at += b - a

    def full_row_indices(self, gr: dict) -> np.ndarray:
        """The group's selected indices as offsets inside a whole row of the model, [rows][mu of the group]."""
        o = gr["o"]
        starts = np.concatenate([[0], np.cumsum([b - a for a, b in gr["ranges"]])])
        shift = np.zeros(int(starts[-1]), dtype=np.int64)
        for (a, _), s0, s1 in zip(gr["ranges"], starts[:-1], starts[1:]):
            shift[s0:s1] = a - s0
        return (o.idx + shift[o.idx]).astype(np.int32)

    def step(self, g: np.ndarray, phase: str, choice: int = 0):
        upd = np.zeros(self.N, dtype=np.float32)
        losses = []
        if phase == "raw":
            return dense_mean(g), losses
        for gr in self.groups:
            gs = self._slices(g, gr["ranges"])
            if gr["mode"] == "dense":
                self._put(upd, gr["ranges"], dense_mean(gs))
                continue
            o = gr["o"]
            o.accumulate(gs)
            o.topk(choice)
            if gr["mode"] == "topk" or phase == "topk_train":
                if gr["mode"] == "ae" and o.ae_kind != "identity":
                    losses.append(o.ae_train_step() if o.variant == "rar" else o.ae_train_step_ps(choice, 1.0, 1.0))
                self._put(upd, gr["ranges"], o.topk_scatter())
            else:
                o.encode()
                o.combine(choice)
                self._put(upd, gr["ranges"], o.decode_scatter())
        return upd, losses
