"""Index-list coding on the CPU (Section V-A of the paper: the transferred indices are entropy
coded with DEFLATE and their rate counts in the compression ratio; Section VI-A defines the
ratio as size(original) / size(compressed)).

TEST INFRASTRUCTURE ONLY: nothing in the product path may import this module.

The byte form is plain: per layer the ascending offsets become gaps (the first counted from the
layer's start, the others from the previous offset + 1); every gap is a little-endian base-128
varint (7 bits per byte, top bit set while more bytes follow).  DEFLATE itself is the library
routine (zlib, raw stream) -- here it serves both as the reference rate and as the decoder that
any stream of the CUDA path must satisfy.
"""
from __future__ import annotations

import math
import zlib
from typing import Sequence

import numpy as np


def varint_bytes(idx: np.ndarray, layer_off: Sequence[int], koff: Sequence[int]) -> bytes:
    out = bytearray()
    for l in range(len(koff) - 1):
        prev = None
        for p in range(int(koff[l]), int(koff[l + 1])):
            i = int(idx[p])
            gap = i - int(layer_off[l]) if prev is None else i - prev - 1
            assert gap >= 0, "offsets must ascend inside a layer"
            prev = i
            while True:
                b = gap & 0x7F
                gap >>= 7
                if gap:
                    out.append(b | 0x80)
                else:
                    out.append(b)
                    break
    return bytes(out)


def indices_from_varint(data: bytes, layer_off: Sequence[int], koff: Sequence[int]) -> np.ndarray:
    out = np.empty(int(koff[-1]), dtype=np.int32)
    pos = 0
    for l in range(len(koff) - 1):
        prev = None
        for p in range(int(koff[l]), int(koff[l + 1])):
            gap, shift = 0, 0
            while True:
                b = data[pos]
                pos += 1
                gap |= (b & 0x7F) << shift
                shift += 7
                if not b & 0x80:
                    break
            i = int(layer_off[l]) + gap if prev is None else prev + 1 + gap
            out[p] = i
            prev = i
    assert pos == len(data), "trailing bytes"
    return out


def deflate(data: bytes) -> bytes:
    """Raw DEFLATE stream (RFC 1951) of the library, best compression."""
    c = zlib.compressobj(9, zlib.DEFLATED, -15)
    return c.compress(data) + c.flush()


def inflate(stream: bytes) -> bytes:
    return zlib.decompress(stream, -15)


def entropy_bytes(data: bytes) -> float:
    """Order-0 entropy of the byte string, in bytes: no literal-only code can do better."""
    if not data:
        return 0.0
    counts = np.bincount(np.frombuffer(data, dtype=np.uint8), minlength=256).astype(np.float64)
    p = counts[counts > 0] / len(data)
    return float(-(p * np.log2(p)).sum() * len(data) / 8.0)


def compression_ratio(num_elements: int, code_floats: int, index_stream_bytes: int, extra_floats: int = 0) -> float:
    """size(original) / size(compressed) for one node and step (Section VI-A): N fp32 values against
    its code (fp32), any further fp32 values it sends (innovation), and its index stream."""
    return 4.0 * num_elements / (4.0 * (code_floats + extra_floats) + index_stream_bytes)
