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
parameter counts the tables imply, and the length chain.
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


def decode(z: np.ndarray, p: Dict[str, np.ndarray], mu: int) -> np.ndarray:
    """code[4][L4] -> reconstruction[mu]."""
    ln = lengths(mu)
    d = leaky(convt_k3s1p1(z, p["dec.w1"], p["dec.b1"]))
    for i in range(2, 6):                     # deconv2..5 undo conv4..conv1
        enc_in = ln[5 - i]                    # length the mirrored encoder layer saw
        d = convt_k3s2(d, p[f"dec.w{i}"], p[f"dec.b{i}"], (enc_in - 3) % 2)
        assert d.shape[1] == enc_in
        d = leaky(d)
    return conv_k1(d, p["dec.w6"], p["dec.b6"]).reshape(-1)


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
