"""The paper's full-size autoencoder (Section IV-C, the two tables of layer hyper-parameters) on
the CPU, in float64, for the ring-allreduce form (Section IV-B): every node's kept values go
through the encoder, the codes are averaged, one decoder reconstructs.

TEST INFRASTRUCTURE ONLY: nothing in the product path may import this module.

Encoder E_c (table of the encoder's layers): five 1-D convolutions,
    conv1 1->64, conv2 64->128, conv3 128->256, conv4 256->64   kernel 3, stride 2, no padding
    conv5 64->4                                                  kernel 1, stride 1
Decoder D_c (table of the decoder's layers): five transposed convolutions and a final 1x1
convolution,
    deconv1 4->4, deconv2 4->32, deconv3 32->64, deconv4 64->128, deconv5 128->32   kernel 3
    conv 32->1                                                                        kernel 1
Leaky ReLU after every layer but the last of each side (Section IV-C names the activation and
gives no slope).

Readings where the paper is silent or at odds with itself:
 * the decoder's table lists stride 2 for all five transposed convolutions, which would upsample
   by 32 against the encoder's 16.  deconv1 is taken with stride 1 and padding 1 (length
   preserved); deconv2..5 have stride 2, no padding, and the output padding that returns each
   length exactly to the length the mirrored encoder layer saw: op = (L_enc_in - 3) mod 2;
 * leaky-ReLU slope 0.01;
 * weight layouts: conv w[co][ci][tau], transposed conv w[ci][co][tau] (the usual ones).

Every function is the layer's defining sum written out with numpy slices; no blocking, no
reordering.  Pinned in tests/test_oracle_full_ae.py against torch's CPU convolutions, the
parameter counts the tables imply, and the length chain.  The training step (loss of Section
IV-B, derivative of every layer, written the same way) is pinned there against torch's autograd
on the same graph, central differences of the loss, and the cases where loss and gradients vanish.
The parameter-server form (Section IV-A: one decoder per node, the node's innovation concatenated
with the decoder's 32 feature channels in front of the last convolution) is pinned against the
same construction with torch.cat and torch's convolutions and by the last filters that reduce it
to the innovation alone and to the ring-allreduce decoder; its training loss (reconstruction through
the K decoders + similarity of the codes) against torch's autograd, central differences and the
cases where the similarity term vanishes.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np

SLOPE = 0.01
ENC_CH = [1, 64, 128, 256, 64]      # channels through conv1..conv4; conv5 maps 64 -> 4
CODE_CH = 4
DEC_CH = [4, 4, 32, 64, 128, 32]    # channels through deconv1..deconv5; the 1x1 conv maps 32 -> 1


def param_shapes() -> List[Tuple[str, Tuple[int, ...]]]:
    out: List[Tuple[str, Tuple[int, ...]]] = []
    for i in range(4):
        out += [(f"enc.w{i + 1}", (ENC_CH[i + 1], ENC_CH[i], 3)), (f"enc.b{i + 1}", (ENC_CH[i + 1],))]
    out += [("enc.w5", (CODE_CH, ENC_CH[4], 1)), ("enc.b5", (CODE_CH,))]
    for i in range(5):
        out += [(f"dec.w{i + 1}", (DEC_CH[i], DEC_CH[i + 1], 3)), (f"dec.b{i + 1}", (DEC_CH[i + 1],))]
    out += [("dec.w6", (1, DEC_CH[5], 1)), ("dec.b6", (1,))]
    return out


def param_shapes_ps(K: int) -> List[Tuple[str, Tuple[int, ...]]]:
    """Parameter-server form (Section IV-A): one encoder, one decoder per node; the node's innovation
    joins its decoder as a 33rd channel in front of the last convolution."""
    out = [t for t in param_shapes() if t[0].startswith("enc.")]
    for k in range(K):
        for i in range(5):
            out += [(f"dec{k}.w{i + 1}", (DEC_CH[i], DEC_CH[i + 1], 3)), (f"dec{k}.b{i + 1}", (DEC_CH[i + 1],))]
        out += [(f"dec{k}.w6", (1, DEC_CH[5] + 1, 1)), (f"dec{k}.b6", (1,))]
    return out


def param_count() -> int:
    return sum(int(np.prod(s)) for _, s in param_shapes())


def unpack(flat: np.ndarray) -> Dict[str, np.ndarray]:
    flat = np.asarray(flat, dtype=np.float64).reshape(-1)
    p, pos = {}, 0
    for name, shape in param_shapes():
        n = int(np.prod(shape))
        p[name] = flat[pos:pos + n].reshape(shape)
        pos += n
    assert pos == flat.size, "parameter vector has the wrong length"
    return p


def lengths(mu: int) -> List[int]:
    """[mu, L1, L2, L3, L4]: lengths after conv1..conv4 (kernel 3, stride 2, no padding)."""
    out = [int(mu)]
    for _ in range(4):
        assert out[-1] >= 3, "input too short for the encoder"
        out.append((out[-1] - 3) // 2 + 1)
    return out


def leaky(x: np.ndarray) -> np.ndarray:
    return np.where(x > 0, x, SLOPE * x)


def conv_k3s2(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y[co][t] = b[co] + sum_ci sum_tau w[co][ci][tau] x[ci][2t + tau]."""
    lout = (x.shape[1] - 3) // 2 + 1
    y = np.repeat(b.reshape(-1, 1), lout, axis=1).astype(np.float64)
    for tau in range(3):
        y += w[:, :, tau] @ x[:, tau:tau + 2 * (lout - 1) + 1:2]
    return y


def conv_k1(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y[co][t] = b[co] + sum_ci w[co][ci][0] x[ci][t]."""
    return w[:, :, 0] @ x + b.reshape(-1, 1)


def convt_k3s2(x: np.ndarray, w: np.ndarray, b: np.ndarray, out_pad: int) -> np.ndarray:
    """y[co][2j + tau] += w[ci][co][tau] x[ci][j]; length 2 (L - 1) + 3 + out_pad."""
    lin = x.shape[1]
    lout = 2 * (lin - 1) + 3 + out_pad
    y = np.repeat(b.reshape(-1, 1), lout, axis=1).astype(np.float64)
    for tau in range(3):
        y[:, tau:tau + 2 * (lin - 1) + 1:2] += w[:, :, tau].T @ x
    return y


def convt_k3s1p1(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Stride 1, padding 1: y[co][j + tau - 1] += w[ci][co][tau] x[ci][j] where the target exists."""
    lin = x.shape[1]
    y = np.repeat(b.reshape(-1, 1), lin, axis=1).astype(np.float64)
    for tau in range(3):
        contrib = w[:, :, tau].T @ x                  # lands at positions j + tau - 1
        lo, hi = max(0, 1 - tau), min(lin, lin + 1 - tau)
        y[:, lo + tau - 1:hi + tau - 1] += contrib[:, lo:hi]
    return y


def encode(x: np.ndarray, p: Dict[str, np.ndarray]) -> np.ndarray:
    """x[mu] -> code[4][L4]."""
    h = np.asarray(x, dtype=np.float64).reshape(1, -1)
    for i in range(1, 5):
        h = leaky(conv_k3s2(h, p[f"enc.w{i}"], p[f"enc.b{i}"]))
    return conv_k1(h, p["enc.w5"], p["enc.b5"])


def decode(z: np.ndarray, p: Dict[str, np.ndarray], mu: int, prefix: str = "dec", inn: np.ndarray = None) -> np.ndarray:
    """code[4][L4] -> reconstruction[mu].  With `inn` (parameter server, Section IV-A: the innovation is
    concatenated with the decoder's features before the last convolution) the last convolution sees
    33 channels, the 33rd being the innovation vector."""
    ln = lengths(mu)
    d = leaky(convt_k3s1p1(z, p[f"{prefix}.w1"], p[f"{prefix}.b1"]))
    for i in range(2, 6):                     # deconv2..5 undo conv4..conv1
        enc_in = ln[5 - i]                    # length the mirrored encoder layer saw
        d = convt_k3s2(d, p[f"{prefix}.w{i}"], p[f"{prefix}.b{i}"], (enc_in - 3) % 2)
        assert d.shape[1] == enc_in
        d = leaky(d)
    if inn is not None:
        d = np.concatenate([d, np.asarray(inn, dtype=np.float64).reshape(1, -1)], axis=0)
    return conv_k1(d, p[f"{prefix}.w6"], p[f"{prefix}.b6"]).reshape(-1)


def rar_forward(val: np.ndarray, p: Dict[str, np.ndarray]):
    """val[K][mu] -> (codes[K][4][L4], mean code, reconstruction[mu]); the mean is the
    node-ordered sum divided by K (Section IV-B)."""
    K, mu = val.shape
    z = np.stack([encode(val[k], p) for k in range(K)])
    acc = np.zeros_like(z[0])
    for k in range(K):
        acc = acc + z[k]
    zbar = acc / float(K)
    return z, zbar, decode(zbar, p, mu)


# ---- training step of the ring-allreduce form (Section IV-B: the reconstruction of the averaged
# code is compared with the average of the nodes' vectors; Section V-B trains on the kept values) ----
#
# Each *_bwd function is the derivative of the layer's defining sum above, written the same way:
# given dL/dy it adds dL/dw and dL/db into gw / gb and returns dL/dx.

def leaky_bwd(pre: np.ndarray, dy: np.ndarray) -> np.ndarray:
    return np.where(pre > 0, dy, SLOPE * dy)


def conv_k3s2_bwd(x, w, dy, gw, gb, want_dx=True):
    lout = dy.shape[1]
    gb += dy.sum(axis=1)
    dx = np.zeros_like(x) if want_dx else None
    for tau in range(3):
        xs = x[:, tau:tau + 2 * (lout - 1) + 1:2]
        gw[:, :, tau] += dy @ xs.T
        if want_dx:
            dx[:, tau:tau + 2 * (lout - 1) + 1:2] += w[:, :, tau].T @ dy
    return dx


def conv_k1_bwd(x, w, dy, gw, gb):
    gb += dy.sum(axis=1)
    gw[:, :, 0] += dy @ x.T
    return w[:, :, 0].T @ dy


def convt_k3s2_bwd(x, w, dy, gw, gb):
    lin = x.shape[1]
    gb += dy.sum(axis=1)
    dx = np.zeros_like(x)
    for tau in range(3):
        dys = dy[:, tau:tau + 2 * (lin - 1) + 1:2]
        gw[:, :, tau] += x @ dys.T
        dx += w[:, :, tau] @ dys
    return dx


def convt_k3s1p1_bwd(x, w, dy, gw, gb):
    lin = x.shape[1]
    gb += dy.sum(axis=1)
    dx = np.zeros_like(x)
    for tau in range(3):
        lo, hi = max(0, 1 - tau), min(lin, lin + 1 - tau)      # inputs j whose target j + tau - 1 exists
        dys = dy[:, lo + tau - 1:hi + tau - 1]
        gw[:, :, tau] += x[:, lo:hi] @ dys.T
        dx[:, lo:hi] += w[:, :, tau] @ dys
    return dx


def rar_loss_and_grads(val: np.ndarray, p: Dict[str, np.ndarray]):
    """loss = (1/mu) || D_c((1/K) sum_k E_c(val_k)) - (1/K) sum_k val_k ||^2 and dloss/dparameter
    for every tensor of param_shapes()."""
    val = np.asarray(val, dtype=np.float64)
    K, mu = val.shape
    ln = lengths(mu)
    g = {name: np.zeros(shape, dtype=np.float64) for name, shape in param_shapes()}
    # forward, keeping every layer's input and pre-activation
    enc_in, enc_pre, codes = [], [], []
    for k in range(K):
        h = val[k].reshape(1, -1)
        ins, pres = [], []
        for i in range(1, 5):
            ins.append(h)
            pre = conv_k3s2(h, p[f"enc.w{i}"], p[f"enc.b{i}"])
            pres.append(pre)
            h = leaky(pre)
        ins.append(h)
        codes.append(conv_k1(h, p["enc.w5"], p["enc.b5"]))
        enc_in.append(ins)
        enc_pre.append(pres)
    acc = np.zeros_like(codes[0])
    for k in range(K):
        acc = acc + codes[k]
    zbar = acc / float(K)
    dec_in, dec_pre = [zbar], []
    pre = convt_k3s1p1(zbar, p["dec.w1"], p["dec.b1"])
    dec_pre.append(pre)
    d = leaky(pre)
    for i in range(2, 6):
        dec_in.append(d)
        pre = convt_k3s2(d, p[f"dec.w{i}"], p[f"dec.b{i}"], (ln[5 - i] - 3) % 2)
        dec_pre.append(pre)
        d = leaky(pre)
    dec_in.append(d)
    r = conv_k1(d, p["dec.w6"], p["dec.b6"]).reshape(-1)
    target = np.zeros(mu)
    for k in range(K):
        target = target + val[k]
    target = target / float(K)
    diff = r - target
    loss = float(np.sum(diff * diff) / mu)
    # backward
    dy = (2.0 * diff / mu).reshape(1, -1)
    dd = conv_k1_bwd(dec_in[5], p["dec.w6"], dy, g["dec.w6"], g["dec.b6"])
    for i in range(5, 1, -1):
        dd = leaky_bwd(dec_pre[i - 1], dd)
        dd = convt_k3s2_bwd(dec_in[i - 1], p[f"dec.w{i}"], dd, g[f"dec.w{i}"], g[f"dec.b{i}"])
    dd = leaky_bwd(dec_pre[0], dd)
    dzbar = convt_k3s1p1_bwd(dec_in[0], p["dec.w1"], dd, g["dec.w1"], g["dec.b1"])
    for k in range(K):
        dh = conv_k1_bwd(enc_in[k][4], p["enc.w5"], dzbar / float(K), g["enc.w5"], g["enc.b5"])
        for i in range(4, 0, -1):
            dh = leaky_bwd(enc_pre[k][i - 1], dh)
            dh = conv_k3s2_bwd(enc_in[k][i - 1], p[f"enc.w{i}"], dh, g[f"enc.w{i}"], g[f"enc.b{i}"], want_dx=i > 1)
    return loss, g


def ps_loss_and_grads(val: np.ndarray, inn: np.ndarray, p: Dict[str, np.ndarray], common: int,
                      lam_rec: float = 1.0, lam_sim: float = 1.0):
    """Parameter-server training loss of Section IV-A on the full-size autoencoder and its gradients:
        loss = lam_rec (1/mu) sum_k || val_k - D_k(E(val_common), inn_k) ||^2
             + lam_sim (1/(4 L4)) sum_k sum_{m != k} || E(val_k) - E(val_m) ||^2
    (each term divided by the entries it sums per node, as for the two-layer autoencoders).
    Returns (loss, rec term, sim term, gradients by tensor name of param_shapes_ps(K))."""
    val = np.asarray(val, dtype=np.float64)
    inn = np.asarray(inn, dtype=np.float64)
    K, mu = val.shape
    ln = lengths(mu)
    g = {name: np.zeros(shape, dtype=np.float64) for name, shape in param_shapes_ps(K)}
    enc_in, enc_pre, codes = [], [], []
    for k in range(K):
        h = val[k].reshape(1, -1)
        ins, pres = [], []
        for i in range(1, 5):
            ins.append(h)
            pre = conv_k3s2(h, p[f"enc.w{i}"], p[f"enc.b{i}"])
            pres.append(pre)
            h = leaky(pre)
        ins.append(h)
        codes.append(conv_k1(h, p["enc.w5"], p["enc.b5"]))
        enc_in.append(ins)
        enc_pre.append(pres)
    nz = codes[0].size
    sim = 0.0
    for k in range(K):
        for m in range(K):
            if m != k:
                sim += float(np.sum((codes[k] - codes[m]) ** 2))
    sim /= nz
    zc = codes[common]
    dzs = [np.zeros_like(zc) for _ in range(K)]
    rec = 0.0
    for k in range(K):
        pre_name = f"dec{k}"
        dec_in, dec_pre = [zc], []
        pre = convt_k3s1p1(zc, p[f"{pre_name}.w1"], p[f"{pre_name}.b1"])
        dec_pre.append(pre)
        d = leaky(pre)
        for i in range(2, 6):
            dec_in.append(d)
            pre = convt_k3s2(d, p[f"{pre_name}.w{i}"], p[f"{pre_name}.b{i}"], (ln[5 - i] - 3) % 2)
            dec_pre.append(pre)
            d = leaky(pre)
        cat = np.concatenate([d, inn[k].reshape(1, -1)], axis=0)          # 32 features + the innovation
        r = conv_k1(cat, p[f"{pre_name}.w6"], p[f"{pre_name}.b6"]).reshape(-1)
        diff = r - val[k]
        rec += float(np.sum(diff * diff)) / mu
        dy = (lam_rec * 2.0 * diff / mu).reshape(1, -1)
        dcat = conv_k1_bwd(cat, p[f"{pre_name}.w6"], dy, g[f"{pre_name}.w6"], g[f"{pre_name}.b6"])
        dd = dcat[:32]                                                     # the innovation is data: no gradient kept
        for i in range(5, 1, -1):
            dd = leaky_bwd(dec_pre[i - 1], dd)
            dd = convt_k3s2_bwd(dec_in[i - 1], p[f"{pre_name}.w{i}"], dd, g[f"{pre_name}.w{i}"], g[f"{pre_name}.b{i}"])
        dd = leaky_bwd(dec_pre[0], dd)
        dzs[common] = dzs[common] + convt_k3s1p1_bwd(zc, p[f"{pre_name}.w1"], dd, g[f"{pre_name}.w1"], g[f"{pre_name}.b1"])
    zsum = np.zeros_like(zc)
    for k in range(K):
        zsum = zsum + codes[k]
    for k in range(K):
        # d/dz_k of the sum over ordered pairs: every unordered pair appears twice
        dz = dzs[k] + lam_sim * 4.0 * (K * codes[k] - zsum) / nz
        dh = conv_k1_bwd(enc_in[k][4], p["enc.w5"], dz, g["enc.w5"], g["enc.b5"])
        for i in range(4, 0, -1):
            dh = leaky_bwd(enc_pre[k][i - 1], dh)
            dh = conv_k3s2_bwd(enc_in[k][i - 1], p[f"enc.w{i}"], dh, g[f"enc.w{i}"], g[f"enc.b{i}"], want_dx=i > 1)
    return lam_rec * rec + lam_sim * sim, rec, sim, g
