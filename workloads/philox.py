"""Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC 2011), written
from the published definition, for the uniforms a verify step consumes.

The uniforms are inputs of the step (both the CUDA path and the oracle read the same tensors), so the generator
holds none of the method's arithmetic; what it buys is that a config's uniforms are the same numbers whether the
workload is generated on the CPU or on the GPU (torch's own CPU and CUDA generators give different streams).

A block is philox(counter = (i, 0, 0, 0), key = (seed, stream)); its four 32-bit words give four uniforms
u = (word >> 8) * 2^-24 in [0, 1), exactly representable in fp32.
"""
from __future__ import annotations

import numpy as np

_M0, _M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)      # the two round multipliers
_W0, _W1 = 0x9E3779B9, 0xBB67AE85                            # key increments (golden ratio, sqrt(3) - 1)
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter: np.ndarray, key) -> np.ndarray:
    """counter: uint32 array [..., 4]; key: two 32-bit integers.  Returns uint32 [..., 4]."""
    c = [counter[..., i].astype(np.uint64) for i in range(4)]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0, p1 = _M0 * c[0], _M1 * c[2]                      # 32 x 32 -> 64-bit products
        hi0, lo0, hi1, lo1 = p0 >> np.uint64(32), p0 & _MASK, p1 >> np.uint64(32), p1 & _MASK
        c = [hi1 ^ c[1] ^ np.uint64(k0), lo1, hi0 ^ c[3] ^ np.uint64(k1), lo0]
        k0, k1 = (k0 + _W0) & 0xFFFFFFFF, (k1 + _W1) & 0xFFFFFFFF
    return np.stack([x.astype(np.uint32) for x in c], axis=-1)


def uniforms(n: int, seed: int, stream: int) -> np.ndarray:
    """n fp32 uniforms in [0, 1) from the blocks 0, 1, ... of (seed, stream)."""
    blocks = (n + 3) // 4
    counter = np.zeros((blocks, 4), dtype=np.uint32)
    counter[:, 0] = np.arange(blocks, dtype=np.uint32)
    words = philox4x32_10(counter, (seed, stream)).reshape(-1)[:n]
    return ((words >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)
