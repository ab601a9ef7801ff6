"""The index stream of the CUDA path: a raw DEFLATE block that the library's inflate must decode
to exactly the varint bytes of the oracle, with a size between the order-0 entropy of those bytes
and a small factor of the library's own deflate."""
import numpy as np
import pytest
import torch

from oracle import index_coding as IC
from paper_2103_08870_b200 import workloads as W

from parity import make_pair

pytestmark = pytest.mark.gpu


def encode(gpu, node, capacity):
    out = torch.full((capacity,), 0xEE, dtype=torch.uint8, device="cuda")
    sizes = torch.zeros(2, dtype=torch.int64, device="cuda")
    gpu.encode_indices(node, out, sizes)
    torch.cuda.synchronize()
    gpu.check()
    return out.cpu().numpy(), [int(x) for x in sizes.cpu()]


def check_stream(ora, gpu, node, row):
    ref_bytes = IC.varint_bytes(ora.idx[row], ora.off[:-1], ora.koff)
    out, (n_stream, n_bytes) = encode(gpu, node, 8 * gpu.mu + 1024)
    assert n_bytes == len(ref_bytes)
    stream = out[:n_stream].tobytes()
    assert not out[n_stream:].any(), "bytes beyond the stream must be zero"
    assert IC.inflate(stream) == ref_bytes                                   # a valid DEFLATE stream of the right content
    assert np.array_equal(IC.indices_from_varint(IC.inflate(stream), ora.off[:-1], ora.koff), ora.idx[row])
    lib = len(IC.deflate(ref_bytes))
    assert IC.entropy_bytes(ref_bytes) <= n_stream <= 1.05 * lib + 160, (n_stream, lib, IC.entropy_bytes(ref_bytes))
    return n_stream, lib


def test_ring_allreduce_leader_list():
    numel = [300_000, 5000, 120_000, 64, 1, 70_001]
    ora, gpu = make_pair(numel, 2)
    src = W.GradientSource(W.LayerTable("ic", numel, [1] * len(numel)), 2, seed=5)
    for t in range(2):
        g = src.step(t)
        ora.accumulate(g.numpy())
        gpu.accumulate(g.cuda(), t)
        ora.topk(t)
        gpu.topk(t)
        check_stream(ora, gpu, 0, t)
        ora.topk_scatter()
        gpu.topk_scatter(torch.empty(gpu.N, device="cuda"))


def test_parameter_server_lists_and_small_capacity():
    numel = [400_000, 9000, 50_000]
    K = 3
    ora, gpu = make_pair(numel, K, variant="ps", density_ppm=5000)
    g = W.GradientSource(W.LayerTable("ic", numel, [1, 2, 3]), K, seed=6).step(0)
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda())
    ora.topk()
    gpu.topk(0)
    sizes = [check_stream(ora, gpu, k, k)[0] for k in range(K)]
    # a buffer that is too small: only the sizes come back, nothing is written past the capacity
    out, (n_stream, _) = encode(gpu, 1, 64)
    assert n_stream == sizes[1] and n_stream > 64


def test_resnet50_shaped_list_and_compression_ratio():
    w = W.workload("resnet50")
    ora, gpu = make_pair(w.table.numel, 2, seed=w.seed)
    g = W.GradientSource(w.table, 2, seed=w.seed).step(0)
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda(), 0)
    ora.topk(0)
    gpu.topk(0)
    n_stream, lib = check_stream(ora, gpu, 0, 0)
    # Section VI-A's ratio for the ring-allreduce leader (code + index stream) and for the other nodes (code only)
    code_floats = gpu.code_len
    leader = IC.compression_ratio(gpu.N, code_floats, n_stream)
    others = IC.compression_ratio(gpu.N, code_floats, 0)
    assert 300 < leader < others == 4.0 * gpu.N / (4.0 * code_floats)


def test_parameter_server_innovation_positions_and_ratio():
    # Algorithm 1: besides its code (one node) every node sends the top tenth of each layer's kept
    # values; the receiver needs their slots.  The stream of those slots (counted inside each layer's
    # run of kept values) must inflate to the oracle's varint bytes and decode to the oracle's slots.
    numel = [400_000, 9000, 50_000, 64]
    K = 3
    ora, gpu = make_pair(numel, K, variant="ps", density_ppm=5000)
    g = W.GradientSource(W.LayerTable("ic", numel, [1, 2, 3, 1]), K, seed=8).step(0)
    ora.accumulate(g.numpy())
    gpu.accumulate(g.cuda())
    ora.topk()
    gpu.topk(0)
    ora.encode()
    gpu.encode()
    ora.combine(1)
    gpu.combine(1)
    kioff = np.concatenate([[0], np.cumsum(ora.ki_l)])
    for k in range(K):
        ref_bytes = IC.varint_bytes(ora.inn_pos[k], ora.koff[:-1], kioff)
        out = torch.full((8 * gpu.mu + 1024,), 0xEE, dtype=torch.uint8, device="cuda")
        sizes = torch.zeros(2, dtype=torch.int64, device="cuda")
        gpu.encode_innovation_positions(k, out, sizes)
        n_stream, n_bytes = (int(x) for x in sizes.cpu())
        gpu.check()
        assert n_bytes == len(ref_bytes)
        stream = out[:n_stream].cpu().numpy().tobytes()
        assert IC.inflate(stream) == ref_bytes
        assert np.array_equal(IC.indices_from_varint(IC.inflate(stream), ora.koff[:-1], kioff), ora.inn_pos[k])
        assert IC.entropy_bytes(ref_bytes) <= n_stream <= 1.05 * len(IC.deflate(ref_bytes)) + 160
    # Section VI-A's ratio for a node that is not the common one: innovation values + both streams
    idx_sizes = torch.zeros(2, dtype=torch.int64, device="cuda")
    gpu.encode_indices(0, out, idx_sizes)
    ratio = IC.compression_ratio(gpu.N, 0, int(idx_sizes[0]) + n_stream, extra_floats=int(kioff[-1]))
    assert ratio > 100
    upd = torch.empty(gpu.N, device="cuda")
    gpu.decode_scatter(upd)
    ora.decode_scatter()
    with pytest.raises(Exception):                       # the innovations belong to the step that made them
        gpu.encode_innovation_positions(0, out, sizes)
