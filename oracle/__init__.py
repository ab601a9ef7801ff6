"""CPU oracle for the LGC compression path: ctypes binding of ``lgc_oracle.c``.

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU-baseline leg import
this package; the product path never does.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lgc_oracle.c")
_LIB = os.path.join(_HERE, "liblgc_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction of separate operations)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _declare(_lib)
    return _lib


_f32p = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(dtype=np.int32, flags="C_CONTIGUOUS")


def _declare(l: C.CDLL) -> None:
    i64, u32, i32, f32, f64 = C.c_int64, C.c_uint32, C.c_int32, C.c_float, C.c_double
    vp = C.c_void_p
    sig = {
        "lgc_oracle_keep_count": (i64, [i64, u32]),
        "lgc_oracle_innovation_count": (i64, [i64, u32]),
        "lgc_oracle_accumulate": (None, [_f32p, _f32p, _f32p, i64, f32]),
        "lgc_oracle_topk_sort": (C.c_int, [_f32p, i64, i64, i32, _i32p]),
        "lgc_oracle_topk_select": (C.c_int, [_f32p, i64, i64, i32, _i32p]),
        "lgc_oracle_gather": (None, [_f32p, _i32p, i64, _f32p]),
        "lgc_oracle_clear": (None, [_f32p, _f32p, _i32p, i64]),
        "lgc_oracle_innovation": (C.c_int, [_f32p, i64, i64, _f32p]),
        "lgc_oracle_conv_len": (i64, [i64]),
        "lgc_oracle_convt_len": (i64, [i64, C.c_int]),
        "lgc_oracle_conv1d": (None, [_f64p, C.c_int, i64, _f64p, _f64p, C.c_int, _f64p]),
        "lgc_oracle_conv1d_bwd": (None, [_f64p, C.c_int, i64, _f64p, C.c_int, _f64p, vp, vp, vp]),
        "lgc_oracle_convt1d": (None, [_f64p, C.c_int, i64, _f64p, _f64p, C.c_int, C.c_int, _f64p]),
        "lgc_oracle_convt1d_bwd": (None, [_f64p, C.c_int, i64, _f64p, C.c_int, C.c_int, _f64p, vp, vp, vp]),
        "lgc_oracle_relu": (None, [_f64p, i64]),
        "lgc_oracle_relu_bwd": (None, [_f64p, _f64p, i64]),
        "lgc_oracle_ps_fuse": (None, [_f64p, _f32p, i64, f64, f64, f64, _f64p]),
        "lgc_oracle_adam": (None, [_f64p, _f64p, _f64p, _f64p, i64, i64, f64, f64, f64, f64]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(l, name)
        fn.restype = res
        fn.argtypes = args


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


# ------------------------------------------------------------------------------------------
# thin numpy-level wrappers (one per C function)
# ------------------------------------------------------------------------------------------
def keep_count(n: int, density_ppm: int) -> int:
    return int(lib().lgc_oracle_keep_count(n, density_ppm))


def innovation_count(k_l: int, permille: int) -> int:
    return int(lib().lgc_oracle_innovation_count(k_l, permille))


def accumulate(u: np.ndarray, v: np.ndarray, g: np.ndarray, m: float) -> None:
    assert u.shape == v.shape == g.shape and u.ndim == 1
    lib().lgc_oracle_accumulate(u, v, g, u.size, m)


def topk(v: np.ndarray, k: int, base: int = 0, method: str = "auto") -> np.ndarray:
    """Indices (ascending, plus ``base``) of the k largest |v|, ties to the lower index."""
    out = np.empty(k, dtype=np.int32)
    if method == "auto":
        method = "sort" if v.size <= 65536 else "select"
    fn = lib().lgc_oracle_topk_sort if method == "sort" else lib().lgc_oracle_topk_select
    rc = fn(np.ascontiguousarray(v), v.size, k, base, out)
    if rc != 0:
        raise RuntimeError(f"oracle topk failed rc={rc}")
    return out


def gather(v: np.ndarray, idx: np.ndarray) -> np.ndarray:
    out = np.empty(idx.size, dtype=np.float32)
    lib().lgc_oracle_gather(v, idx, idx.size, out)
    return out


def clear(u: np.ndarray, v: np.ndarray, idx: np.ndarray) -> None:
    lib().lgc_oracle_clear(u, v, idx, idx.size)


def innovation(val: np.ndarray, ki: int) -> np.ndarray:
    out = np.empty(val.size, dtype=np.float32)
    rc = lib().lgc_oracle_innovation(np.ascontiguousarray(val), val.size, ki, out)
    if rc != 0:
        raise RuntimeError(f"oracle innovation failed rc={rc}")
    return out


def conv_len(lin: int) -> int:
    return int(lib().lgc_oracle_conv_len(lin))


def convt_len(lin: int, out_pad: int) -> int:
    return int(lib().lgc_oracle_convt_len(lin, out_pad))


def conv1d(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """x [cin][lin], w [cout][cin][3], b [cout] -> [cout][lout]; three taps, stride 2."""
    cin, lin = x.shape
    cout = w.shape[0]
    assert w.shape == (cout, cin, 3) and b.shape == (cout,)
    y = np.empty((cout, conv_len(lin)), dtype=np.float64)
    lib().lgc_oracle_conv1d(x, cin, lin, w, b, cout, y)
    return y


def conv1d_bwd(x, w, dy, dw=None, db=None, want_dx=True):
    cin, lin = x.shape
    cout = w.shape[0]
    dx = np.empty_like(x) if want_dx else None
    lib().lgc_oracle_conv1d_bwd(x, cin, lin, w, cout, np.ascontiguousarray(dy), _ptr(dx), _ptr(dw), _ptr(db))
    return dx


def convt1d(x: np.ndarray, w: np.ndarray, b: np.ndarray, out_pad: int) -> np.ndarray:
    """x [cin][lin], w [cin][cout][3], b [cout] -> [cout][2(lin-1)+3+out_pad]."""
    cin, lin = x.shape
    cout = w.shape[1]
    assert w.shape == (cin, cout, 3) and b.shape == (cout,)
    y = np.empty((cout, convt_len(lin, out_pad)), dtype=np.float64)
    lib().lgc_oracle_convt1d(x, cin, lin, w, b, cout, out_pad, y)
    return y


def convt1d_bwd(x, w, out_pad, dy, dw=None, db=None, want_dx=True):
    cin, lin = x.shape
    cout = w.shape[1]
    dx = np.empty_like(x) if want_dx else None
    lib().lgc_oracle_convt1d_bwd(x, cin, lin, w, cout, out_pad, np.ascontiguousarray(dy), _ptr(dx), _ptr(dw), _ptr(db))
    return dx


def relu(x: np.ndarray) -> np.ndarray:
    y = np.array(x, dtype=np.float64, order="C", copy=True)
    lib().lgc_oracle_relu(y.reshape(-1), y.size)
    return y


def relu_bwd(y: np.ndarray, d: np.ndarray) -> np.ndarray:
    out = np.array(d, dtype=np.float64, order="C", copy=True)
    lib().lgc_oracle_relu_bwd(np.ascontiguousarray(y).reshape(-1), out.reshape(-1), out.size)
    return out


def ps_fuse(y: np.ndarray, inn: np.ndarray, w0: float, w1: float, b: float) -> np.ndarray:
    r = np.empty(y.size, dtype=np.float64)
    lib().lgc_oracle_ps_fuse(np.ascontiguousarray(y).reshape(-1), inn, y.size, w0, w1, b, r)
    return r


def adam(p, m, v, g, t, lr, beta1, beta2, eps) -> None:
    lib().lgc_oracle_adam(p, m, v, np.ascontiguousarray(g), p.size, t, lr, beta1, beta2, eps)


from .pipeline import OracleLGC  # noqa: E402,F401
