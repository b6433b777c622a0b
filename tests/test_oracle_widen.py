"""Pin of the oracle's exact widening of stored bits (every bf16 parity result rests on it): random
and special bfloat16 bit patterns against torch's own bfloat16 -> float64 conversion."""
import numpy as np
import torch

from oracle import vvs_oracle as O


def _torch_widen(bits: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def test_widen_bf16_bit_patterns_match_torch_exactly():
    rng = np.random.default_rng(20251113)
    rand = rng.integers(0, 1 << 16, size=20000, dtype=np.uint16)
    special = np.array([0x0000, 0x8000,            # +0, -0
                        0x0001, 0x8001, 0x007F,    # smallest / largest subnormals
                        0x0080, 0x8080,            # smallest normals
                        0x3F80, 0xBF80,            # +1, -1
                        0x7F7F, 0xFF7F,            # largest finite
                        0x7F80, 0xFF80,            # infinities
                        0x3DCD, 0x4049], dtype=np.uint16)
    bits = np.concatenate([special, rand])
    got, want = O.widen(bits), _torch_widen(bits)
    assert got.dtype == np.float64
    finite = np.isfinite(want)
    # bit-for-bit on every non-NaN pattern (signed zeros included), NaN where torch says NaN
    assert np.array_equal(got[finite].view(np.uint64), want[finite].view(np.uint64))
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want)) and np.array_equal(np.signbit(got[~np.isnan(got)]), np.signbit(want[~np.isnan(want)]))


def test_widen_keeps_shape_and_passes_floats_through():
    a = np.arange(12, dtype=np.uint16).reshape(3, 4) + np.uint16(0x3F80)
    assert O.widen(a).shape == (3, 4)
    f = np.array([[1.5, -2.25]], dtype=np.float32)
    assert np.array_equal(O.widen(f), f.astype(np.float64))
