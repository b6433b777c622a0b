"""Pins of the oracle's dynamic-skip decision (paper Sec. 4.4, Eq. 2, Alg. 1): closed forms,
special cases and a library routine, chosen so that a wrong weight, a dropped pair, a missing
normalisation or a wrong stride fails one of them."""
import numpy as np
import torch

from oracle import vvs_oracle as O


def _cb(seed, v=50, dim=8):
    return np.random.default_rng(seed).standard_normal((v, dim))


def test_identical_paths_have_similarity_one_and_orthogonal_ones_zero():
    cb = np.eye(8)
    same = np.tile(np.array([[3, 1, 4]]), (6, 1))
    assert abs(O.path_similarity(same, np.full(6, 3), cb, 0.7) - 1.0) < 1e-15
    ortho = np.array([[0, 1, 2], [9, 9, 9], [3, 4, 5], [9, 9, 9], [6, 7, 0]])   # kept: rows 0, 2, 4
    ortho[ortho == 9] = 0                                                        # dropped rows may hold anything
    assert abs(O.path_similarity(ortho, np.full(5, 3), cb, 0.7)) < 1e-15


def test_two_paths_one_level_is_the_plain_cosine_scaled_inputs_do_not_matter():
    cb = _cb(1)
    paths = np.array([[5], [0], [17]])                    # stride 2 keeps tokens 5 and 17
    x, y = cb[5], cb[17]
    want = float(torch.nn.functional.cosine_similarity(torch.tensor(x), torch.tensor(y), dim=0))
    assert abs(O.path_similarity(paths, np.ones(3, int), cb, 0.5) - want) < 1e-12
    cb2 = cb.copy(); cb2[5] *= 7.5; cb2[17] *= 0.01        # cosine ignores the norms
    assert abs(O.path_similarity(paths, np.ones(3, int), cb2, 0.5) - want) < 1e-12


def test_weights_follow_alpha_and_sum_to_one():
    # level similarities 1, 0, 1 (two kept paths): S_bar = (1 + a^2) / (1 + a + a^2)
    cb = np.eye(4)
    paths = np.array([[0, 1, 3], [2, 2, 2], [0, 2, 3]])
    for a in (0.3, 0.9, 1.0):
        got = O.path_similarity(paths, np.full(3, 3), cb, a)
        assert abs(got - (1 + a * a) / (1 + a + a * a)) < 1e-14
    # alpha = 1 is the plain mean over depth; depth is cut at the shortest kept path
    assert abs(O.path_similarity(paths, np.array([3, 1, 2]), cb, 1.0) - 0.5) < 1e-14


def test_pair_mean_equals_torch_pairwise_cosine_matrix():
    cb = _cb(2, 200, 8)
    rng = np.random.default_rng(3)
    paths = rng.integers(0, 200, size=(9, 4))
    keep = paths[::2]
    alpha = 0.8
    w = alpha ** np.arange(4); w /= w.sum()
    want = 0.0
    for l in range(4):
        e = torch.nn.functional.normalize(torch.tensor(cb[keep[:, l]]), dim=1)
        m = (e @ e.T).numpy()
        iu = np.triu_indices(len(keep), 1)
        want += w[l] * m[iu].mean()
    assert abs(O.path_similarity(paths, np.full(9, 4), cb, alpha) - want) < 1e-12


def test_guard_threshold_and_degenerate_inputs():
    cb = _cb(4)
    paths = np.array([[1, 2], [3, 4], [1, 2]])
    s = O.path_similarity(paths, np.full(3, 2), cb, 0.5)
    assert abs(s - 1.0) < 1e-15                               # kept paths 0 and 2 are identical
    assert O.skip_decision(paths, np.full(3, 2), cb, 0.5, 0.95, True) == (True, s)
    assert O.skip_decision(paths, np.full(3, 2), cb, 0.5, 0.95, False) == (False, 0.0)   # never twice in a row
    assert O.skip_decision(paths, np.full(3, 2), cb, 0.5, 1.0 + 1e-9, True)[0] is False  # below the threshold
    assert O.path_similarity(paths[:1], np.array([2]), cb, 0.5) == 1.0                    # a single path
    assert O.path_similarity(paths, np.array([0, 2, 2]), cb, 0.5) == 0.0                  # depth 0
    cb0 = cb.copy(); cb0[1] = 0.0                                                          # zero embedding: cosine 0
    assert abs(O.path_similarity(paths, np.full(3, 2), cb0, 1.0) - 0.5) < 1e-15
    assert O.downsample_paths(7, 2) == [0, 2, 4, 6] and O.downsample_paths(4, 3) == [0, 3]


def test_uniform_path_selection_and_truncation():
    """Sec. 4.2 / Eq. 3: every path is drawn on an interval of width 1/N; gamma = min(L_s, floor(mean))."""
    paths = np.arange(5 * 6).reshape(5, 6)
    lens = np.array([6, 2, 5, 3, 4])                        # mean 4.0
    hits = np.zeros(5, int)
    for k in range(1000):
        i, g, toks = O.select_unverified(paths, lens, (k + 0.5) / 1000)
        hits[i] += 1
        assert g == min(lens[i], 4) and list(toks) == list(paths[i][:g])
    assert (hits == 200).all()
    assert O.select_unverified(paths, lens, 0.999999)[0] == 4 and O.select_unverified(paths, lens, 1e-9)[0] == 0
    # the floor: lengths 3, 4 -> mean 3.5 -> at most 3 tokens even from the longer path
    assert O.select_unverified(paths[:2], np.array([3, 4]), 0.75)[1] == 3
    assert O.select_unverified(paths[:2], np.array([1, 6]), 0.75)[1] == 3     # mean 3.5, L_s = 6
    assert O.select_unverified(paths[:2], np.array([1, 6]), 0.25)[1] == 1     # L_s = 1
