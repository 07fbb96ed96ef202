"""Chunk shapes for tensors whose dimensions are not multiples of the wanted chunk size.

The method assumes n_i = c_i * s_i on every axis (appendix, "Multilinear Transforms and Chunk-wise
Tensor Blocking") and says nothing about remainders.  The way to stay inside that assumption is to
let each axis use an extent that divides it: ``divisor_chunk_shape`` picks, per axis, the largest
divisor of n_i that does not exceed the target, and shrinks the largest extents further while the
chunk would hold more elements than ``demo_init_nd`` accepts.  Host-side planning only; the result
is what ``DemoTransform(..., chunk_shapes=...)`` takes.
"""
from __future__ import annotations

import math
from typing import Sequence, Tuple

MAX_EXTENT = 128        # DEMO_ND_MAX_EXTENT
MAX_CHUNK_ELEMS = 16384  # DEMO_ND_MAX_CHUNK_ELEMS


def largest_divisor_at_most(n: int, limit: int) -> int:
    """Largest d with d | n and 1 <= d <= limit."""
    if n < 1 or limit < 1:
        raise ValueError("n and limit must be positive")
    for d in range(min(n, limit), 0, -1):
        if n % d == 0:
            return d
    return 1


def divisor_chunk_shape(shape: Sequence[int], target: int, max_extent: int = MAX_EXTENT,
                        max_elems: int = MAX_CHUNK_ELEMS) -> Tuple[int, ...]:
    """Per axis the largest divisor of the dimension that is <= min(target, max_extent); while the chunk
    holds more than ``max_elems`` elements the largest extent is replaced by its next smaller divisor."""
    chunk = [largest_divisor_at_most(int(n), min(int(target), max_extent)) for n in shape]
    while math.prod(chunk) > max_elems:
        a = max(range(len(chunk)), key=lambda i: chunk[i])
        if chunk[a] == 1:
            break
        chunk[a] = largest_divisor_at_most(int(shape[a]), chunk[a] - 1)
    return tuple(chunk)
