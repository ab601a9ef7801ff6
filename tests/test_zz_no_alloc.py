"""lgc_topk_noalloc -- the entry point for callers that cannot allocate device memory or pass
scratch (fixed-footprint regions, plugins that only receive inputs and outputs, a full device).

Called through the C ABI twice in a row (the calls share the library's built-in work space, and
the second must not see what the first left there) and compared, bit for bit as for every index
set in this suite, with what the regular entry point lgc_topk selects for the same vector.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import ctypes as C

import pytest
import torch

from paper_2103_08870_b200 import lgc

pytestmark = pytest.mark.gpu


def reference_indices(v: torch.Tensor, ppm: int) -> torch.Tensor:
    """The existing path: one node, one layer; the first accumulation makes the residual equal v."""
    ctx = lgc.LGC([v.numel()], 1, density_ppm=ppm, momentum=0.0, ae_kind="identity")
    ctx.accumulate(v.view(1, -1))
    ctx.topk(0)
    out = ctx.idx[0].clone()
    ctx.check()
    return out


def test_two_calls_in_a_row_match_the_regular_entry_point():
    lib = lgc.lib()
    gen = torch.Generator(device="cuda").manual_seed(11)
    cases = [(3_000_001, 1000), (70_001, 50_000), (1_500, 20_000)]     # chunked, chunked + dense, single CTA
    for n, ppm in cases:
        v = torch.randn(n, generator=gen, device="cuda") * 1e-3
        v[n // 3: n // 3 + 500] = v[0]                     # a run of equal magnitudes
        ref = reference_indices(v, ppm)
        k = ref.numel()
        out = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        stream = torch.cuda.current_stream()
        st = lib.lgc_topk_noalloc(v.data_ptr(), n, k, out.data_ptr(), C.c_void_p(stream.cuda_stream))
        assert st == 0, lib.lgc_last_error(None)
        torch.cuda.synchronize()
        assert torch.equal(out, ref), f"n={n}, k={k}"
    # the same through the binding, with a different vector right after
    v2 = torch.rand(1_000_003, generator=gen, device="cuda") - 0.5
    ref2 = reference_indices(v2, 1000)
    out2 = torch.empty(ref2.numel(), dtype=torch.int32, device="cuda")
    lgc.topk_noalloc(v2, ref2.numel(), out2)
    torch.cuda.synchronize()
    assert torch.equal(out2, ref2)


def test_sizes_beyond_the_built_in_work_space_are_refused():
    lib = lgc.lib()
    v = torch.zeros(16, device="cuda")
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = lib.lgc_topk_noalloc(v.data_ptr(), lgc.NOALLOC_MAX_N + 1, 4, out.data_ptr(), None)
    assert lgc.status_string(st) == "LGC_ERR_UNSUPPORTED"
    assert b"LGC_NOALLOC_MAX_N" in lib.lgc_last_error(None)
    assert lib.lgc_topk_noalloc(v.data_ptr(), 16, 17, out.data_ptr(), None) == 1      # k > n
    assert lib.lgc_topk_noalloc(None, 16, 4, out.data_ptr(), None) == 1
    with pytest.raises(lgc.LGCError, match="UNSUPPORTED"):          # the binding raises on the same refusal
        lgc.topk_noalloc(torch.empty(lgc.NOALLOC_MAX_N + 4, device="cuda"), 4, out)
