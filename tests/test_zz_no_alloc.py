"""lgc_topk_noalloc -- the entry point for callers that cannot allocate device memory or pass
scratch (fixed-footprint regions, plugins that only receive inputs and outputs, a full device).

Called through the C ABI, calls in a row (they share the library's built-in work space, and a
call must not see what the one before left there), and compared bit for bit, as every index set
in this suite, with the CPU oracle's selection (Section V-A: the k entries of largest magnitude,
ties to the lower index, ascending) and with what the regular entry point lgc_topk selects for
the same vector.  Collected last on purpose: a run that stops at the first failure has then run
everything else.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle as O
from paper_2103_08870_b200 import lgc

pytestmark = pytest.mark.gpu


def regular_entry_point(v: torch.Tensor, k: int) -> torch.Tensor:
    """The existing path: one node, one layer; the first accumulation makes the residual equal v."""
    n = v.numel()
    ppm = None
    for cand in range(max(1, k * 1_000_000 // n - 2), k * 1_000_000 // n + 3):      # a density that gives exactly k
        if min(max((n * cand + 500_000) // 1_000_000, 1), n) == k:
            ppm = cand
            break
    if ppm is None or ppm > 1_000_000:
        return None
    ctx = lgc.LGC([n], 1, density_ppm=ppm, momentum=0.0, ae_kind="identity")
    assert ctx.mu == k
    g = v.clone().view(1, -1)                          # the context wants a 16-byte aligned gradient
    ctx.accumulate(g)
    ctx.topk(0)
    out = ctx.idx[0].clone()
    ctx.check()
    return out


def noalloc(lib, v: torch.Tensor, k: int) -> torch.Tensor:
    out = torch.full((k,), -1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    st = lib.lgc_topk_noalloc(v.data_ptr(), v.numel(), k, out.data_ptr(), C.c_void_p(stream.cuda_stream))
    assert st == 0, lib.lgc_last_error(None)
    assert lib.lgc_topk_noalloc_check(C.c_void_p(stream.cuda_stream)) == 0, lib.lgc_last_error(None)
    return out


def check_case(lib, v: torch.Tensor, k: int, what: str, against_regular=True):
    ref = torch.from_numpy(O.topk(v.cpu().numpy(), k)).cuda()
    out = noalloc(lib, v, k)
    assert torch.equal(out, ref), f"{what}: differs from the oracle's selection"
    if against_regular:
        reg = regular_entry_point(v, k)
        if reg is not None:
            assert torch.equal(out, reg), f"{what}: differs from lgc_topk"


def test_two_calls_in_a_row_match_the_oracle_and_the_regular_entry_point():
    lib = lgc.lib()
    gen = torch.Generator(device="cuda").manual_seed(11)
    cases = [(3_000_001, 3000), (70_001, 3500), (1_500, 30)]           # chunked, chunked + dense, single CTA
    for n, k in cases:
        v = torch.randn(n, generator=gen, device="cuda") * 1e-3
        v[n // 3: n // 3 + 500] = v[0]                     # a run of equal magnitudes
        check_case(lib, v, k, f"n={n}, k={k}")
    # the same through the binding, with a different vector right after
    v2 = torch.rand(1_000_003, generator=gen, device="cuda") - 0.5
    ref2 = torch.from_numpy(O.topk(v2.cpu().numpy(), 1000)).cuda()
    out2 = torch.empty(1000, dtype=torch.int32, device="cuda")
    lgc.topk_noalloc(v2, 1000, out2)
    lgc.topk_noalloc_check()
    assert torch.equal(out2, ref2)


def test_chunk_edges_ties_across_chunks_and_unaligned_vectors():
    lib = lgc.lib()
    gen = torch.Generator(device="cuda").manual_seed(12)
    # one chunk exactly, one element into the second chunk
    for n in (4096, 4097):
        v = torch.randn(n, generator=gen, device="cuda")
        check_case(lib, v, 41, f"n={n}")
    # everything is kept
    v = torch.randn(10_001, generator=gen, device="cuda")
    check_case(lib, v, 10_001, "k = n")
    # a run of equal magnitudes (both signs) that crosses the boundary between chunks 1 and 2, and the
    # k-th place falls inside it: ties must go to the lower indices across the boundary
    v = torch.randn(20_000, generator=gen, device="cuda") * 0.1
    v[8000:8400] = 7.0
    v[8100:8300] = -7.0
    v[100] = 9.0
    check_case(lib, v, 251, "ties across a chunk boundary")
    # a vector that starts one float past a 16-byte boundary
    base = torch.randn(300_004, generator=gen, device="cuda")
    check_case(lib, base[1:300_002], 300, "unaligned v", against_regular=False)
    # all entries equal: the first k indices
    v = torch.full((50_000,), -0.5, device="cuda")
    out = noalloc(lib, v, 77)
    assert torch.equal(out, torch.arange(77, dtype=torch.int32, device="cuda"))


def test_largest_supported_vector():
    lib = lgc.lib()
    gen = torch.Generator(device="cuda").manual_seed(13)
    n = lgc.NOALLOC_MAX_N
    v = torch.randn(n, generator=gen, device="cuda")
    check_case(lib, v, 16_777, "n = LGC_NOALLOC_MAX_N")
    # and a small one right after it: nothing of the large call's tables may survive
    w = torch.randn(5000, generator=gen, device="cuda")
    check_case(lib, w, 5, "small vector after the largest")


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
