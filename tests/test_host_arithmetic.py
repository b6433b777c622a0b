"""Arithmetic identities the CUDA path relies on, checked exhaustively on the CPU in the same
precision (numpy float32 operations are correctly rounded, like the device's)."""
import numpy as np


def test_float_reciprocal_division_is_exact_in_its_range():
    """The whole-chain kernel divides ring positions and unit indices (below 2^21) by small runtime
    values as int((float(x) + 0.5f) * rcp(float(d))): the result must be x // d for every x of the
    range, for every ring depth and every k-block / tile count a supported shape can have."""
    x = np.arange(0, 1 << 21, dtype=np.int64)
    xf = x.astype(np.float32) + np.float32(0.5)
    for d in list(range(1, 65)) + [86, 96, 128, 172, 224, 256, 448, 512, 1000, 1024]:
        r = np.float32(1.0) / np.float32(d)
        q = (xf * r).astype(np.int64)
        assert np.array_equal(q, x // d), d
