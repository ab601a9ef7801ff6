"""Pins for the index-list byte form and the rate arithmetic (oracle/index_coding.py)."""
import numpy as np

from oracle import index_coding as IC


def test_varint_worked_example():
    # gaps 0, 127, 128, 300, 16384 in one layer that starts at 1000: base-128, low group first
    idx = np.array([1000, 1128, 1257, 1558, 17943], dtype=np.int32)
    data = IC.varint_bytes(idx, [1000], [0, 5])
    assert data == bytes([0x00, 0x7F, 0x80, 0x01, 0xAC, 0x02, 0x80, 0x80, 0x01])
    assert np.array_equal(IC.indices_from_varint(data, [1000], [0, 5]), idx)


def test_round_trip_over_layers_and_through_deflate():
    rng = np.random.default_rng(4)
    numel = [5000, 1, 300000, 64, 2_000_000]
    off = np.concatenate([[0], np.cumsum(numel)])
    k = [5, 1, 300, 1, 2000]
    koff = np.concatenate([[0], np.cumsum(k)])
    idx = np.concatenate([np.sort(rng.choice(n, kk, replace=False)) + o for n, kk, o in zip(numel, k, off)]).astype(np.int32)
    data = IC.varint_bytes(idx, off[:-1], koff)
    assert np.array_equal(IC.indices_from_varint(data, off[:-1], koff), idx)
    stream = IC.deflate(data)
    assert IC.inflate(stream) == data
    assert IC.entropy_bytes(data) <= len(data)
    # a first offset equal to the layer start and adjacent offsets give zero gaps: one zero byte each
    dense = np.arange(100, 110, dtype=np.int32)
    assert IC.varint_bytes(dense, [100], [0, 10]) == bytes(10)


def test_entropy_and_ratio_closed_forms():
    assert IC.entropy_bytes(bytes([7]) * 100) == 0.0
    assert abs(IC.entropy_bytes(bytes(range(256)) * 4) - 1024.0) < 1e-9      # uniform bytes: 8 bits each
    # N = 1000 values against 10 code floats and a 60-byte index stream: 4000 / 100
    assert IC.compression_ratio(1000, 10, 60) == 40.0
    assert IC.compression_ratio(1000, 10, 60, extra_floats=15) == 4000.0 / 160.0
