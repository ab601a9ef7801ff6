"""The LGC per-step path on the CPU oracle, stage by stage in the paper's order.

TEST INFRASTRUCTURE ONLY (see ``lgc_oracle.c``).  K nodes are K rows of the state arrays.

Stages (Algorithm 1 = parameter server "ps", Algorithm 2 = ring-allreduce "rar"):
  accumulate      u <- m u + g ; v <- v + u                       (Alg. 1/2 accumulation; Sec. V-A)
  topk            per layer, the k_l largest |v| (ties: lower index); rar: the leader's indices
                  serve every node, ps: every node selects on its own (Sec. V-A)
                  followed by the gather of the kept values into g~_k in R^mu
  encode          g~^c_k = E_c(g~_k)                              (Sec. IV-A/IV-B)
  combine         rar: g~^avg = (1/K) sum_k g~^c_k                 (Sec. IV-B / V-B.2)
                  ps : common code of one node + every node's innovation (Alg. 1, Sec. V-B.1)
  decode_scatter  rar: g~^rec = D_c(g~^avg); ps: g~^rec_k = D_c^k(g~^c, g~^I_k), averaged over k
                  (Sec. V-B.1); written back to dense positions; sent entries leave u and v
  ae_train_step   ring-allreduce reconstruction loss (Sec. IV-B), mean over mu, one Adam step
  ae_train_step_ps  parameter-server loss lam_rec L_rec + lam_sim L_sim (Sec. IV-A), one Adam step
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np

import oracle as O
from oracle import full_ae as A5


def _param_order(c1: int, c2: int, variant: str, K: int):
    enc = [("enc.w1", (c1, 1, 3)), ("enc.b1", (c1,)), ("enc.w2", (c2, c1, 3)), ("enc.b2", (c2,))]

    def dec(p):
        return [(p + ".w1", (c2, c1, 3)), (p + ".b1", (c1,)), (p + ".w2", (c1, 1, 3)), (p + ".b2", (1,))]

    if variant == "rar":
        return enc + dec("dec")
    out = list(enc)
    for k in range(K):
        out += dec(f"dec{k}") + [(f"dec{k}.fuse", (3,))]
    return out


class OracleLGC:
    def __init__(self, layer_numel: Sequence[int], num_nodes: int, density_ppm: int = 1000,
                 momentum: float = 0.9, variant: str = "rar", ae_kind: str = "conv2",
                 c1: int = 8, c2: int = 4, params: Optional[np.ndarray] = None,
                 innovation_permille: int = 100, lr: float = 1e-3, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, topk_method: str = "auto"):
        assert variant in ("rar", "ps") and ae_kind in ("conv2", "identity", "conv5")
        self.numel = [int(n) for n in layer_numel]
        self.L = len(self.numel)
        self.K = int(num_nodes)
        self.N = sum(self.numel)
        self.off = np.concatenate([[0], np.cumsum(self.numel)]).astype(np.int64)
        self.k_l = [O.keep_count(n, density_ppm) for n in self.numel]
        self.koff = np.concatenate([[0], np.cumsum(self.k_l)]).astype(np.int64)
        self.mu = int(self.koff[-1])
        self.ki_l = [O.innovation_count(k, innovation_permille) for k in self.k_l]
        self.m = np.float32(momentum)
        self.variant, self.ae_kind, self.c1, self.c2 = variant, ae_kind, c1, c2
        self.topk_method = topk_method
        self.u = np.zeros((self.K, self.N), dtype=np.float32)
        self.v = np.zeros((self.K, self.N), dtype=np.float32)
        # autoencoder geometry: mu -> L1 -> L2 and back, output paddings mirror the encoder
        self.L1 = O.conv_len(self.mu)
        self.L2 = O.conv_len(self.L1)
        self.op1 = (self.L1 - 3) % 2 if self.L1 >= 3 else 0   # decoder layer 1: L2 -> L1
        self.op2 = (self.mu - 3) % 2 if self.mu >= 3 else 0   # decoder layer 2: L1 -> mu
        self.p: Dict[str, np.ndarray] = {}
        if ae_kind == "conv5":
            self.order = A5.param_shapes() if variant == "rar" else A5.param_shapes_ps(self.K)
        else:
            self.order = _param_order(c1, c2, variant, self.K)
        if params is not None:
            self.set_params(params)
        self.adam_m = self.adam_v = None
        self.adam_t = 0
        self.lr, self.beta1, self.beta2, self.eps = lr, beta1, beta2, eps
        self.idx = self.val = self.z = self.zbar = self.zc = self.inn = self.r = None

    # -- parameters ---------------------------------------------------------------------
    def set_params(self, flat: np.ndarray) -> None:
        flat = np.asarray(flat, dtype=np.float64).reshape(-1)
        pos = 0
        for name, shape in self.order:
            n = int(np.prod(shape))
            self.p[name] = np.ascontiguousarray(flat[pos:pos + n].reshape(shape))
            pos += n
        assert pos == flat.size, "parameter vector has the wrong length"

    def get_params(self) -> np.ndarray:
        return np.concatenate([self.p[name].reshape(-1) for name, _ in self.order])

    # -- stage 1 ------------------------------------------------------------------------
    def accumulate(self, g: np.ndarray) -> None:
        assert g.shape == (self.K, self.N) and g.dtype == np.float32
        for k in range(self.K):
            O.accumulate(self.u[k], self.v[k], np.ascontiguousarray(g[k]), float(self.m))

    # -- stages 2 + 3 -------------------------------------------------------------------
    def _select(self, k: int) -> np.ndarray:
        out = np.empty(self.mu, dtype=np.int32)
        for l in range(self.L):
            a, b = int(self.off[l]), int(self.off[l + 1])
            out[self.koff[l]:self.koff[l + 1]] = O.topk(self.v[k, a:b], self.k_l[l], base=a,
                                                        method=self.topk_method)
        return out

    def topk(self, leader: int = 0) -> None:
        if self.variant == "rar":
            sel = self._select(leader)
            self.idx = np.broadcast_to(sel, (self.K, self.mu)).copy()
        else:
            self.idx = np.stack([self._select(k) for k in range(self.K)])
        self.val = np.stack([O.gather(self.v[k], self.idx[k]) for k in range(self.K)])

    # -- stage 4 ------------------------------------------------------------------------
    def _enc(self, x: np.ndarray):
        h = O.relu(O.conv1d(x.reshape(1, -1), self.p["enc.w1"], self.p["enc.b1"]))
        return h, O.conv1d(h, self.p["enc.w2"], self.p["enc.b2"])

    def encode(self) -> None:
        if self.ae_kind == "identity":
            self.z = self.val.astype(np.float64).reshape(self.K, 1, self.mu)
            return
        if self.ae_kind == "conv5":          # the paper's full-size encoder (Section IV-C)
            self.z = np.stack([A5.encode(self.val[k], self.p) for k in range(self.K)])
            return
        self.z = np.stack([self._enc(self.val[k].astype(np.float64))[1] for k in range(self.K)])

    def combine(self, common_node: int = 0) -> None:
        if self.variant == "rar":
            acc = np.zeros_like(self.z[0])
            for k in range(self.K):
                acc = acc + self.z[k]
            self.zbar = acc / float(self.K)
            return
        self.zc = self.z[common_node].copy()
        self.inn = np.zeros((self.K, self.mu), dtype=np.float32)
        self.inn_pos = np.zeros((self.K, int(sum(self.ki_l))), dtype=np.int32)    # the kept slots the innovation holds
        for k in range(self.K):
            at = 0
            for l in range(self.L):
                a, b = int(self.koff[l]), int(self.koff[l + 1])
                self.inn[k, a:b] = O.innovation(self.val[k, a:b], self.ki_l[l])
                self.inn_pos[k, at:at + self.ki_l[l]] = O.topk(self.val[k, a:b], self.ki_l[l], base=a, method="sort")
                at += self.ki_l[l]

    # -- stage 5 ------------------------------------------------------------------------
    def _dec(self, z: np.ndarray, prefix: str):
        d = O.relu(O.convt1d(z, self.p[prefix + ".w1"], self.p[prefix + ".b1"], self.op1))
        return d, O.convt1d(d, self.p[prefix + ".w2"], self.p[prefix + ".b2"], self.op2)

    def decode(self) -> None:
        if self.variant == "rar":
            if self.ae_kind == "identity":
                self.r = self.zbar.reshape(1, self.mu).copy()
            elif self.ae_kind == "conv5":
                self.r = A5.decode(self.zbar, self.p, self.mu).reshape(1, self.mu)
            else:
                self.r = self._dec(self.zbar, "dec")[1].reshape(1, self.mu)
            return
        self.r = np.empty((self.K, self.mu), dtype=np.float64)
        for k in range(self.K):
            if self.ae_kind == "conv5":      # full-size decoder of node k, its innovation as the 33rd channel
                self.r[k] = A5.decode(self.zc, self.p, self.mu, prefix=f"dec{k}", inn=self.inn[k])
                continue
            if self.ae_kind == "identity":
                y = self.zc.reshape(-1)
                w0, w1, b = 1.0, 1.0, 0.0
            else:
                y = self._dec(self.zc, f"dec{k}")[1].reshape(-1)
                w0, w1, b = (float(t) for t in self.p[f"dec{k}.fuse"])
            self.r[k] = O.ps_fuse(y, self.inn[k], w0, w1, b)

    def _clear_sent(self) -> None:
        for k in range(self.K):
            O.clear(self.u[k], self.v[k], self.idx[k])

    def decode_scatter(self) -> np.ndarray:
        self.decode()
        upd = np.zeros(self.N, dtype=np.float64)
        if self.variant == "rar":
            upd[self.idx[0]] = self.r[0]
        else:
            for k in range(self.K):                      # node order, each term divided by K
                np.add.at(upd, self.idx[k], self.r[k] / float(self.K))
        self._clear_sent()
        return upd.astype(np.float32)

    def topk_scatter(self) -> np.ndarray:
        """Second training phase (weights updated with the plain top-magnitude gradients while
        the autoencoder trains, Sec. V-B): dense mean over nodes of the kept values."""
        upd = np.zeros(self.N, dtype=np.float64)
        if self.variant == "rar":
            acc = np.zeros(self.mu, dtype=np.float64)
            for k in range(self.K):
                acc = acc + self.val[k].astype(np.float64)
            upd[self.idx[0]] = acc / float(self.K)
        else:
            for k in range(self.K):
                np.add.at(upd, self.idx[k], self.val[k].astype(np.float64) / float(self.K))
        self._clear_sent()
        return upd.astype(np.float32)

    # -- autoencoder training (ring-allreduce loss, Sec. IV-B) ----------------------------
    def ae_loss_and_grads(self):
        """loss = (1/mu) || D_c(mean_k E_c(g~_k)) - mean_k g~_k ||^2 and its parameter gradients."""
        assert self.variant == "rar" and self.ae_kind in ("conv2", "conv5")
        if self.ae_kind == "conv5":          # the paper's full-size autoencoder (Section IV-C)
            return A5.rar_loss_and_grads(self.val, self.p)
        K, mu = self.K, self.mu
        xs = [self.val[k].astype(np.float64).reshape(1, -1) for k in range(K)]
        hs, zs = [], []
        for k in range(K):
            h, z = self._enc(xs[k][0])
            hs.append(h)
            zs.append(z)
        zbar = sum(zs[1:], zs[0].copy()) / float(K)
        d, r = self._dec(zbar, "dec")
        target = sum(xs[1:], xs[0].copy()) / float(K)
        diff = r - target
        loss = float(np.sum(diff * diff) / mu)
        g = {name: np.zeros(shape, dtype=np.float64) for name, shape in self.order}
        dr = 2.0 * diff / mu
        dd = O.convt1d_bwd(d, self.p["dec.w2"], self.op2, dr, g["dec.w2"], g["dec.b2"])
        dd = O.relu_bwd(d, dd)
        dzbar = O.convt1d_bwd(zbar, self.p["dec.w1"], self.op1, dd, g["dec.w1"], g["dec.b1"])
        for k in range(K):
            dz = dzbar / float(K)
            dh = O.conv1d_bwd(hs[k], self.p["enc.w2"], dz, g["enc.w2"], g["enc.b2"])
            dh = O.relu_bwd(hs[k], dh)
            O.conv1d_bwd(xs[k], self.p["enc.w1"], dh, g["enc.w1"], g["enc.b1"], want_dx=False)
        return loss, g

    # -- autoencoder training (parameter-server loss, Sec. IV-A) ----------------------------
    def ae_loss_and_grads_ps(self, common_node: int, lam_rec: float = 1.0, lam_sim: float = 1.0):
        """L = lam_rec L_rec + lam_sim L_sim (Sec. IV-A): every node's kept values go through the
        encoder; L_sim sums ||E_c(g~_k) - E_c(g~_m)||^2 over all ordered pairs k != m; the code of
        `common_node` is decoded by every node's decoder together with that node's innovation and
        L_rec sums ||g~_k - g~^rec_k||^2 over the nodes.  Reading: L_rec is divided by mu and L_sim
        by the number of code entries (c2 L2), so that lam_rec = lam_sim = 1 weighs an average
        entry of either kind alike.  Returns (loss, L_rec / mu, L_sim / (c2 L2), gradients)."""
        assert self.variant == "ps" and self.ae_kind in ("conv2", "conv5")
        K, mu = self.K, self.mu
        if self.ae_kind == "conv5":          # the full-size autoencoder: innovation as the 33rd channel
            inn = np.zeros((K, mu), dtype=np.float64)
            for k in range(K):
                for l in range(self.L):
                    a, b = int(self.koff[l]), int(self.koff[l + 1])
                    inn[k, a:b] = O.innovation(self.val[k, a:b], self.ki_l[l])
            return A5.ps_loss_and_grads(self.val, inn, self.p, common_node, lam_rec, lam_sim)
        xs = [self.val[k].astype(np.float64).reshape(1, -1) for k in range(K)]
        hs, zs = [], []
        for k in range(K):
            h, z = self._enc(xs[k][0])
            hs.append(h)
            zs.append(z)
        nz = zs[0].size
        sim = 0.0
        for k in range(K):
            for m in range(K):
                if m != k:
                    sim += float(np.sum((zs[k] - zs[m]) ** 2))
        sim /= nz
        zc = zs[common_node]
        g = {name: np.zeros(shape, dtype=np.float64) for name, shape in self.order}
        dzs = [np.zeros_like(zc) for _ in range(K)]
        rec = 0.0
        for k in range(K):
            inn = np.zeros(mu, dtype=np.float64)
            for l in range(self.L):
                a, b = int(self.koff[l]), int(self.koff[l + 1])
                inn[a:b] = O.innovation(self.val[k, a:b], self.ki_l[l])
            d, y = self._dec(zc, f"dec{k}")
            w0, w1, b = (float(t) for t in self.p[f"dec{k}.fuse"])
            r = w0 * y + w1 * inn.reshape(1, -1) + b
            diff = r - xs[k]
            rec += float(np.sum(diff * diff)) / mu
            dr = lam_rec * 2.0 * diff / mu
            g[f"dec{k}.fuse"] += np.array([np.sum(dr * y), np.sum(dr * inn), np.sum(dr)])
            dy = w0 * dr
            dd = O.convt1d_bwd(d, self.p[f"dec{k}.w2"], self.op2, dy, g[f"dec{k}.w2"], g[f"dec{k}.b2"])
            dd = O.relu_bwd(d, dd)
            dzs[common_node] = dzs[common_node] + O.convt1d_bwd(zc, self.p[f"dec{k}.w1"], self.op1, dd,
                                                                 g[f"dec{k}.w1"], g[f"dec{k}.b1"])
        zsum = sum(zs[1:], zs[0].copy())
        for k in range(K):
            # d/dz_k of sum over ordered pairs: every unordered pair appears twice
            dz = dzs[k] + lam_sim * 4.0 * (K * zs[k] - zsum) / nz
            dh = O.conv1d_bwd(hs[k], self.p["enc.w2"], dz, g["enc.w2"], g["enc.b2"])
            dh = O.relu_bwd(hs[k], dh)
            O.conv1d_bwd(xs[k], self.p["enc.w1"], dh, g["enc.w1"], g["enc.b1"], want_dx=False)
        return lam_rec * rec + lam_sim * sim, rec, sim, g

    def _adam_step(self, g) -> None:
        flat_p = self.get_params()
        flat_g = np.concatenate([g[name].reshape(-1) for name, _ in self.order])
        if self.adam_m is None:
            self.adam_m = np.zeros_like(flat_p)
            self.adam_v = np.zeros_like(flat_p)
        self.adam_t += 1
        O.adam(flat_p, self.adam_m, self.adam_v, flat_g, self.adam_t, self.lr, self.beta1,
               self.beta2, self.eps)
        self.set_params(flat_p)

    def ae_train_step_ps(self, common_node: int, lam_rec: float = 1.0, lam_sim: float = 1.0) -> float:
        loss, _, _, g = self.ae_loss_and_grads_ps(common_node, lam_rec, lam_sim)
        self._adam_step(g)
        return loss

    def ae_train_step(self) -> float:
        loss, g = self.ae_loss_and_grads()
        flat_p = self.get_params()
        flat_g = np.concatenate([g[name].reshape(-1) for name, _ in self.order])
        if self.adam_m is None:
            self.adam_m = np.zeros_like(flat_p)
            self.adam_v = np.zeros_like(flat_p)
        self.adam_t += 1
        O.adam(flat_p, self.adam_m, self.adam_v, flat_g, self.adam_t, self.lr, self.beta1,
               self.beta2, self.eps)
        self.set_params(flat_p)
        return loss

    # -- one whole compression step -------------------------------------------------------
    def step(self, g: np.ndarray, choice: int = 0) -> np.ndarray:
        self.accumulate(g)
        self.topk(choice)
        self.encode()
        self.combine(choice)
        return self.decode_scatter()
