"""Philox4x32-10 counter-based generator (Salmon et al., "Parallel random numbers: as easy as
1, 2, 3", SC'11), written out in numpy from the published round function.

This module only produces the uniforms that the sampler consumes; it holds none of the sampler's
arithmetic.  Both the CPU checker and the CUDA library receive the SAME pre-generated buffer, so
the generator itself is not parity-critical; it is pinned by the published known-answer vectors in
the CPU test-suite.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint32(0x9E3779B9)
_W1 = np.uint32(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter: np.ndarray, key: np.ndarray) -> np.ndarray:
    """Ten Philox-4x32 rounds.

    counter: uint32 array [..., 4]; key: uint32 array [..., 2] (broadcastable over the leading
    dimensions).  Returns uint32 [..., 4].
    """
    c = np.array(counter, dtype=np.uint32, copy=True)
    k = np.array(np.broadcast_to(np.asarray(key, dtype=np.uint32), c.shape[:-1] + (2,)), copy=True)
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = k[..., 0].copy(), k[..., 1].copy()
    for rnd in range(10):
        if rnd > 0:
            k0 = ((k0.astype(np.uint64) + np.uint64(_W0)) & _MASK32).astype(np.uint32)
            k1 = ((k1.astype(np.uint64) + np.uint64(_W1)) & _MASK32).astype(np.uint32)
        p0 = c0.astype(np.uint64) * _M0
        p1 = c2.astype(np.uint64) * _M1
        hi0 = (p0 >> np.uint64(32)).astype(np.uint32)
        lo0 = (p0 & _MASK32).astype(np.uint32)
        hi1 = (p1 >> np.uint64(32)).astype(np.uint32)
        lo1 = (p1 & _MASK32).astype(np.uint32)
        n0 = hi1 ^ c1 ^ k0
        n1 = lo1
        n2 = hi0 ^ c3 ^ k1
        n3 = lo0
        c0, c1, c2, c3 = n0, n1, n2, n3
    return np.stack([c0, c1, c2, c3], axis=-1)


def uniforms(seed: int, rows: int, trials: int) -> np.ndarray:
    """float32 uniforms in [0, 1), shape [rows, trials, 4].

    One Philox block per (row, trial): counter = (row, trial, 0, 0), key = (seed low, seed high).
    A 32-bit word x becomes (x >> 8) * 2**-24, which is exact in float32 and never reaches 1.
    Lane 0 drives the draft draw, lane 1 the acceptance test, lane 2 the residual draw, lane 3 is
    spare.
    """
    r = np.arange(rows, dtype=np.uint32)[:, None]
    t = np.arange(trials, dtype=np.uint32)[None, :]
    ctr = np.zeros((rows, trials, 4), dtype=np.uint32)
    ctr[..., 0] = r
    ctr[..., 1] = t
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    words = philox4x32_10(ctr, key)
    return ((words >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)
