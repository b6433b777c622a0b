"""Counter-based Philox4x32-10 generator (Salmon et al., "Parallel random numbers: as easy
as 1, 2, 3", SC'11) in vectorised numpy.

This module only produces random *inputs* (the uniforms a verify call consumes, test
tensors); it holds none of the verification method's arithmetic.  The uniforms handed to
the verify step are passed in as plain arrays, so the CPU oracle and the CUDA library see
the same bits.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint32(0x9E3779B9)
_W1 = np.uint32(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter: np.ndarray, key: np.ndarray) -> np.ndarray:
    """counter: uint32 [..., 4]; key: uint32 [..., 2] (broadcastable).  Returns uint32 [..., 4]."""
    c = np.asarray(counter, dtype=np.uint32)
    k = np.broadcast_to(np.asarray(key, dtype=np.uint32), c.shape[:-1] + (2,))
    c0, c1, c2, c3 = (c[..., i].astype(np.uint64) for i in range(4))
    k0 = k[..., 0].copy()
    k1 = k[..., 1].copy()
    for _ in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        n0 = hi1 ^ c1 ^ k0.astype(np.uint64)
        n2 = hi0 ^ c3 ^ k1.astype(np.uint64)
        c0, c1, c2, c3 = n0, lo1, n2, lo0
        with np.errstate(over="ignore"):
            k0 = (k0 + _W0).astype(np.uint32)
            k1 = (k1 + _W1).astype(np.uint32)
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def uniform_open01(bits: np.ndarray) -> np.ndarray:
    """Map uint32 words to float32 uniforms strictly inside (0, 1): (x >> 8 + 0.5) * 2^-24."""
    x = (np.asarray(bits, dtype=np.uint32) >> np.uint32(8)).astype(np.float64)
    return ((x + 0.5) * (2.0 ** -24)).astype(np.float32)


def verify_uniforms(seed: int, call_id: int, n_images: int, n_draft_max: int) -> np.ndarray:
    """float32 [B, K+1] uniforms for one verify call.

    Word 0 of Philox(counter=(b, i, call_id, 0), key=(seed_lo, seed_hi)).  Column i < K drives
    the acceptance test of draft i, column K the single residual / bonus sample.
    """
    b = np.arange(n_images, dtype=np.uint32)[:, None]
    i = np.arange(n_draft_max + 1, dtype=np.uint32)[None, :]
    ctr = np.zeros((n_images, n_draft_max + 1, 4), dtype=np.uint32)
    ctr[..., 0] = b
    ctr[..., 1] = i
    ctr[..., 2] = np.uint32(call_id & 0xFFFFFFFF)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    return uniform_open01(philox4x32_10(ctr, key)[..., 0])
