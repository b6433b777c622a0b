"""Pins of the oracle's token-level feature cache (Sec. 4.3: cache the features of every
verified token, retrieve "the exact number of most recent token-level features"; Sec. 4.1:
post verification writes features back to their positions; Supp. "Memory Overhead": the
latest 5 features of 1280 bf16 values stay under 100 kB).  CPU only."""
import numpy as np

from oracle import vvs_oracle as O


def _feat(r, pos, d=4):
    return np.full(d, 1000.0 * r + pos)


def test_store_then_fetch_returns_most_recent_rows():
    fc = O.FeatureCache(n_rows=2, cap=8, d=4)
    hidden = np.stack([np.stack([_feat(r, 10 + t) for t in range(5)]) for r in range(2)])
    fc.store(hidden, np.array([10, 10]), np.array([5, 3]))
    out, pos = fc.fetch(np.array([1, 1]), np.array([3, 2]), 0, 4)
    np.testing.assert_array_equal(pos[0], [12, 13, 14, -1])
    np.testing.assert_array_equal(pos[1], [11, 12, -1, -1])
    for r in range(2):
        for j in range(4):
            want = _feat(r, pos[r, j]) if pos[r, j] >= 0 else np.zeros(4)
            np.testing.assert_array_equal(out[r, j], want)


def test_staleness_shifts_the_window_back():
    """Supp. Table 5: s = 0 is the most recent cached feature, s = +i is i tokens older."""
    fc = O.FeatureCache(1, 16, 4)
    hidden = np.stack([_feat(0, t) for t in range(9)])[None]
    fc.store(hidden, np.array([0]), np.array([9]))
    for s in range(4):
        _, pos = fc.fetch(np.array([1]), np.array([2]), s, 2)
        np.testing.assert_array_equal(pos[0], [7 - s, 8 - s])


def test_ring_overwrite_skip_mask_and_write_back():
    fc = O.FeatureCache(2, 5, 4)
    for base in (0, 4, 8):                                    # 12 positions into 5 slots
        hidden = np.stack([np.stack([_feat(r, base + t) for t in range(4)]) for r in range(2)])
        fc.store(hidden, np.array([base, base]), np.array([4, 4]))
    out, pos = fc.fetch(np.array([1, 0]), np.array([5, 5]), 0, 6)
    np.testing.assert_array_equal(pos[0], [7, 8, 9, 10, 11, -1])
    assert (pos[1] == -1).all() and not out[1].any()          # image 1 not skip-masked
    _, pos = fc.fetch(np.array([1, 1]), np.array([4, 4]), 3, 4)
    np.testing.assert_array_equal(pos[0], [-1, -1, 7, 8])     # 5, 6 were overwritten
    # post verification: positions 10, 11 re-stored with fresh features; newest unchanged
    fresh = np.stack([np.stack([_feat(r, 500 + t) for t in range(2)]) for r in range(2)])
    fc.store(fresh, np.array([10, 10]), np.array([2, 0]))
    out, pos = fc.fetch(np.array([1, 1]), np.array([3, 3]), 0, 3)
    np.testing.assert_array_equal(pos[0], [9, 10, 11])
    np.testing.assert_array_equal(out[0, 1], _feat(0, 500))
    np.testing.assert_array_equal(out[1, 1], _feat(1, 10))    # n_store = 0: untouched
    assert fc.newest[0] == 11


def test_empty_cache_and_footprint():
    fc = O.FeatureCache(1, 5, 1280)
    _, pos = fc.fetch(np.array([1]), np.array([3]), 0, 3)
    assert (pos == -1).all()
    assert 5 * 1280 * 2 == 12800 < 100_000                    # bf16 bytes per sequence
