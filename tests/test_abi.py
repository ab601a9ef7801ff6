"""The C-ABI library: loads without a GPU, exports what include/lgc.h declares, and refuses bad
configurations on the host (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

from paper_2103_08870_b200 import build as B
from paper_2103_08870_b200 import lgc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return lgc.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lgc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lgc_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"lgc_init", "lgc_accumulate", "lgc_topk", "lgc_encode", "lgc_combine", "lgc_decode_scatter",
            "lgc_ae_train_step"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(lgc.EXPORTS)


def cfg(numel, **kw):
    arr = (C.c_int64 * len(numel))(*numel)
    base = dict(num_nodes=2, num_layers=len(numel), layer_numel=arr, density_ppm=1000,
                innovation_permille=100, momentum=0.9, variant=0, ae_kind=0, ae_c1=8, ae_c2=4)
    base.update(kw)
    c = lgc.lgc_config(**base)
    c._keep = arr
    return c


def sizes(lib, c):
    a, b, d = C.c_size_t(), C.c_size_t(), C.c_size_t()
    st = lib.lgc_workspace_bytes(C.byref(c), C.byref(a), C.byref(b), C.byref(d))
    return st, a.value, b.value, d.value


def test_workspace_sizes(lib):
    st, state, scratch, params = sizes(lib, cfg([1 << 20]))
    assert st == 0
    assert state == 2 * 2 * (1 << 20) * 4
    assert params == 3 * 264 * 4          # 261 parameters, padded to a multiple of four
    assert scratch > 0 and scratch % 256 == 0
    st, state, _, params = sizes(lib, cfg([1 << 20], variant=1, ae_c1=16, ae_c2=8, num_nodes=4))
    assert st == 0 and params == 3 * (16 * 4 + 8 * 48 + 8 + 4 * (384 + 16 + 48 + 1 + 3)) * 4


def test_bad_configurations_are_refused_on_the_host(lib):
    INVALID, UNSUPPORTED = 1, 4
    assert lib.lgc_workspace_bytes(None, None, None, None) == INVALID
    assert sizes(lib, cfg([100], num_nodes=0))[0] == INVALID
    assert sizes(lib, cfg([100, 0]))[0] == INVALID
    assert sizes(lib, cfg([100], density_ppm=0))[0] == INVALID
    assert sizes(lib, cfg([100], momentum=1.0))[0] == INVALID
    assert sizes(lib, cfg([100], variant=7))[0] == INVALID
    assert sizes(lib, cfg([2**31 - 1, 1]))[0] == INVALID            # N would need more than int32 offsets
    assert sizes(lib, cfg([1 << 20], ae_c1=5, ae_c2=5))[0] == UNSUPPORTED
    assert sizes(lib, cfg([100]))[0] == UNSUPPORTED                  # mu = 1: too short for the autoencoder
    assert sizes(lib, cfg([100], ae_kind=1))[0] == 0                 # identity has no length limit
    # lgc_init refuses before touching the device
    out = C.c_void_p()
    assert lib.lgc_init(C.byref(cfg([1 << 20])), None, 0, None, 0, None, 0, C.byref(out)) == INVALID
    assert not out.value
    assert lib.lgc_init(C.byref(cfg([1 << 20])), 16, 0, 16, 0, 16, 0, C.byref(out)) == 3   # workspace too small


def test_status_strings_and_null_context(lib):
    assert lib.lgc_status_string(0) == b"LGC_OK"
    assert lib.lgc_status_string(2) == b"LGC_ERR_BAD_STATE"
    assert lib.lgc_status_string(99) == b"LGC_ERR_UNKNOWN"
    assert lib.lgc_accumulate(None, None, 0) == 1
    assert lib.lgc_destroy(None) == 0
    assert lib.lgc_abort_step(None) == 1
    assert lib.lgc_step_host(None, None, None, None, None, 0) == 1
    assert isinstance(lib.lgc_last_error(None), bytes)


def test_binding_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(RuntimeError, match="no CPU path"):
        lgc.LGC([1 << 12], 2)
