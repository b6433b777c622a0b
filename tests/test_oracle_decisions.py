"""Pins of the oracle's decision stage against what the paper and the mathematics fix
(Sec. 2 "Speculative Decoding": acceptance min(1, p/q), residual resampling, bonus token,
stop at the first rejection; Sec. 6: strict verification is lossless; Sec. 2 LANTERN rule:
relaxed acceptance pools neighbour mass under a threshold delta).  CPU only."""
import itertools

import numpy as np
import pytest

from oracle import vvs_oracle as O


def _rand_dist(rng, v, sharp=1.5):
    z = rng.standard_normal(v) * sharp
    e = np.exp(z - z.max())
    return (e / e.sum()).astype(np.float32)


def _grid(n):
    return ((np.arange(n) + 0.5) / n).astype(np.float32)


def _first_token_law(p_rows, q_rows, n_forced, pos, prefix, n_grid=400):
    """Law of the token emitted at draft position `pos`, given drafts prefix (all accepted):
    integrates the oracle's own outputs over the draft q(x) and fine grids of both uniforms."""
    v = p_rows.shape[1]
    k = q_rows.shape[0]
    law = np.zeros(v)
    for x in range(v):
        if q_rows[pos, x] == 0:
            continue
        drafts = np.array(list(prefix) + [x] + [0] * (k - pos - 1), dtype=np.int32)
        acc = 0
        for u in _grid(n_grid):
            us = np.full(k + 1, 1e-7, dtype=np.float32)      # earlier drafts: accept
            us[pos] = u
            acc += O.decide(p_rows, drafts, pos + 1, n_forced, q_rows, us)["accept_len"] == pos + 1
        a = acc / n_grid
        law[x] += q_rows[pos, x] * a
        if a < 1.0:
            res = np.zeros(v)
            us = np.full(k + 1, 1e-7, dtype=np.float32)
            us[pos] = np.float32(1.0 - 1e-7)                  # force the rejection
            for u in _grid(n_grid):
                us[k] = u
                d = O.decide(p_rows, drafts, pos + 1, n_forced, q_rows, us)
                assert d["accept_len"] == pos
                res[d["next_token"]] += 1.0 / n_grid
            law += q_rows[pos, x] * (1.0 - a) * res
    return law


@pytest.mark.parametrize("v,k,n_forced", [(2, 1, 1), (4, 2, 1), (5, 3, 2), (6, 3, 1)])
def test_strict_verification_is_lossless_by_enumeration(v, k, n_forced):
    """Sec. 6 ("lossless") with Sec. 2's rules: at every draft position the emitted token is
    distributed exactly as the target row, whatever the draft distribution.  A wrong residual
    sign, a missing normalisation, a wrong row / column index or an off-by-one in the inverse
    CDF all break this identity."""
    rng = np.random.default_rng(100 + v * 10 + k)
    t = n_forced + k
    p_rows = np.stack([_rand_dist(rng, v) for _ in range(t)])
    q_rows = np.stack([_rand_dist(rng, v) for _ in range(k)])
    for pos in range(k):
        support = [x for x in range(v) if p_rows[n_forced - 1 + 0, x] > 0]
        prefix = [support[(3 * j + 1) % len(support)] for j in range(pos)]
        law = _first_token_law(p_rows, q_rows, n_forced, pos, prefix)
        np.testing.assert_allclose(law, p_rows[n_forced - 1 + pos], atol=2.5 / 400)


def test_acceptance_probability_is_min_1_p_over_q():
    """Sec. 2: P(accept x) = min(1, p(x)/q(x)), measured as the accepted fraction of a fine
    uniform grid, against hand-computed ratios."""
    p = np.array([[0.5, 0.3, 0.2]], dtype=np.float32)
    q = np.array([[0.25, 0.6, 0.15]], dtype=np.float32)
    want = [1.0, 0.5, 1.0]
    for x in range(3):
        acc = np.mean([O.decide(p, [x], 1, 1, q, np.array([u, 0.5], np.float32))["accept_len"]
                       for u in _grid(1000)])
        assert abs(acc - want[x]) <= 1e-3
    # q(x) = 0: accepted iff the target gives the token any mass
    q0 = np.array([[0.0, 1.0, 0.0]], dtype=np.float32)
    p0 = np.array([[0.5, 0.5, 0.0]], dtype=np.float32)
    assert O.decide(p0, [0], 1, 1, q0, np.array([0.999, 0.5], np.float32))["accept_len"] == 1
    assert O.decide(p0, [2], 1, 1, q0, np.array([0.001, 0.5], np.float32))["accept_len"] == 0


def test_residual_is_zero_where_draft_dominates_and_bonus_comes_from_target():
    """Sec. 2: a rejected position resamples from the part of the target the draft
    under-covers; if all drafts pass, one more token comes from the next target row."""
    p = np.array([[0.1, 0.6, 0.3], [0.7, 0.2, 0.1]], dtype=np.float32)
    q = np.array([[0.8, 0.1, 0.1]], dtype=np.float32)
    seen = set()
    for u in _grid(500):
        d = O.decide(p, [0], 1, 1, q, np.array([0.99, u], np.float32))
        assert d["accept_len"] == 0
        seen.add(d["next_token"])
    assert seen == {1, 2}                                  # never token 0, where q > p
    # residual mass (0.5, 0.2)/0.7: boundary between tokens 1 and 2 at u = 5/7
    assert O.decide(p, [0], 1, 1, q, np.array([0.99, 0.71], np.float32))["next_token"] == 1
    assert O.decide(p, [0], 1, 1, q, np.array([0.99, 0.72], np.float32))["next_token"] == 2
    # bonus: all accepted -> row 1 = (0.7, 0.2, 0.1)
    got = [O.decide(p, [0], 1, 1, q, np.array([0.01, u], np.float32))["next_token"]
           for u in (0.69, 0.71, 0.89, 0.91)]
    assert got == [0, 1, 1, 2]
    # no row after the last draft -> no bonus token
    assert O.decide(p[:1], [0], 1, 1, q, np.array([0.01, 0.3], np.float32))["next_token"] == -1


def test_accepted_prefix_invariant_and_n_draft_limit():
    """Sec. 2: verification is sequential and stops at the first rejection."""
    rng = np.random.default_rng(7)
    v, k = 6, 5
    for trial in range(200):
        p = np.stack([_rand_dist(rng, v) for _ in range(k + 1)])
        q = np.stack([_rand_dist(rng, v) for _ in range(k)])
        drafts = rng.integers(0, v, k)
        u = rng.random(k + 1).astype(np.float32)
        nd = int(rng.integers(0, k + 1))
        d = O.decide(p, drafts, nd, 1, q, u)
        n = d["accept_len"]
        assert 0 <= n <= nd
        assert list(d["accept_mask"]) == [1] * n + [0] * (k - n)
        for i in range(n):
            assert u[i] < min(1.0, float(p[i, drafts[i]]) / float(q[i, drafts[i]]))
        if n < nd:
            assert not u[n] < min(1.0, float(p[n, drafts[n]]) / float(q[n, drafts[n]]))
            assert p[n, d["next_token"]] > q[n, d["next_token"]]
        assert 0 <= d["next_token"] < v


def test_inverse_cdf_matches_searchsorted_and_frequencies():
    rng = np.random.default_rng(3)
    r = rng.random(37).astype(np.float32)
    r[[0, 5, 36]] = 0.0
    cdf = np.cumsum(r.astype(np.float64))
    counts = np.zeros(37)
    for u in _grid(20000):
        j, margin = O.inverse_cdf(r, u)
        assert j == np.searchsorted(cdf, float(u) * cdf[-1], side="right")
        assert margin >= 0
        counts[j] += 1
    np.testing.assert_allclose(counts / 20000, r / r.sum(), atol=2e-4)
    assert counts[0] == counts[5] == counts[36] == 0


# ---------------------------------------------------------------------------------------
# relaxed acceptance


def _hand_table(v, k, rng):
    rows = []
    for x in range(v):
        others = [y for y in range(v) if y != x]
        rng.shuffle(others)
        rows.append([x] + others[:k - 1])
    col = np.array(rows, dtype=np.int32).reshape(-1)
    row_ptr = (np.arange(v + 1) * k).astype(np.int32)
    return row_ptr, col


def test_relaxed_reduces_to_strict_for_k1_or_delta0():
    """k = 1 (neighbourhood = the token itself) or delta = 0 must reproduce strict
    verification bit for bit."""
    rng = np.random.default_rng(11)
    v, k = 8, 4
    row_ptr, col = _hand_table(v, 5, rng)
    for trial in range(100):
        p = np.stack([_rand_dist(rng, v) for _ in range(k + 1)])
        q = np.stack([_rand_dist(rng, v) for _ in range(k)])
        drafts = rng.integers(0, v, k)
        u = rng.random(k + 1).astype(np.float32)
        s = O.decide(p, drafts, k, 1, q, u)
        for kw in (dict(k=1, delta=float("inf")), dict(k=5, delta=0.0)):
            r = O.decide(p, drafts, k, 1, q, u, O.MODE_RELAXED, row_ptr, col, **kw)
            assert r["accept_len"] == s["accept_len"] and r["next_token"] == s["next_token"]
            np.testing.assert_array_equal(r["ratios"], s["ratios"])


def test_pooled_mass_against_brute_force_prefix_search():
    """The accepted set is {x} plus the longest distance-ordered prefix of neighbours whose
    total target mass is <= delta: found here by trying every prefix length and keeping the
    largest admissible one; plus the bounds and monotonicity the rule implies."""
    rng = np.random.default_rng(5)
    v = 8
    for trial in range(300):
        kk = int(rng.integers(1, v + 1))
        row_ptr, col = _hand_table(v, kk, rng)
        p = _rand_dist(rng, v)
        x = int(rng.integers(0, v))
        delta = float(rng.choice([0.0, 0.05, 0.1, 0.2, 0.6, np.inf]))
        k_use = int(rng.integers(1, kk + 1))
        got = O.pooled_mass(p, x, row_ptr, col, k_use, delta)
        nb = col[row_ptr[x]:row_ptr[x + 1]][1:k_use]
        best = 0.0
        for m in range(len(nb) + 1):
            s = float(np.sum(p[nb[:m]].astype(np.float64)))
            if s <= delta:
                best = s
        assert got == pytest.approx(float(p[x]) + best, abs=1e-15)
        assert float(p[x]) <= got <= float(p[x]) + min(delta, 1.0) + 1e-12
        if k_use < kk:
            assert O.pooled_mass(p, x, row_ptr, col, k_use + 1, delta) >= got
        assert O.pooled_mass(p, x, row_ptr, col, k_use, delta * 2 + 0.01) >= got


def test_relaxed_acceptance_probability_by_enumeration():
    """P(accept | x ~ q) = sum_x min(q(x), P_A(x)) with P_A computed by hand for a 4-token
    codebook whose neighbour rows are written out explicitly."""
    p = np.array([[0.4, 0.3, 0.2, 0.1]], dtype=np.float32)
    q = np.array([[0.1, 0.2, 0.3, 0.4]], dtype=np.float32)
    col = np.array([0, 1, 2, 1, 0, 3, 2, 3, 0, 3, 2, 1], dtype=np.int32)
    row_ptr = np.array([0, 3, 6, 9, 12], dtype=np.int32)
    # delta = 0.35, k = 3: A(0) = {0,1} (adding 2 would give 0.5 > 0.35) -> 0.7
    # A(1) = {1} (p(0) = 0.4 > 0.35) -> 0.3; A(2) = {2,3} then +0 -> 0.1 + 0.4 > 0.35 -> 0.3
    # A(3) = {3,2} (0.2) then +1 (0.5 > 0.35) -> 0.3
    pa = [0.7, 0.3, 0.3, 0.3]
    for x in range(4):
        assert O.pooled_mass(p[0], x, row_ptr, col, 3, 0.35) == pytest.approx(pa[x], abs=1e-7)
    total = 0.0
    for x in range(4):
        acc = np.mean([O.decide(p, [x], 1, 1, q, np.array([u, 0.5], np.float32), O.MODE_RELAXED,
                                row_ptr, col, 3, 0.35)["accept_len"] for u in _grid(2000)])
        total += q[0, x] * acc
    assert total == pytest.approx(sum(min(float(q[0, x]), pa[x]) for x in range(4)), abs=2e-3)


def test_decision_margins_and_uniform_columns():
    """Column i of the uniforms judges draft i; the last column alone drives the sample."""
    p = np.array([[0.5, 0.5], [0.5, 0.5], [0.25, 0.75]], dtype=np.float32)
    q = np.array([[1.0, 0.0], [1.0, 0.0]], dtype=np.float32)
    u = np.array([0.4, 0.6, 0.2], dtype=np.float32)
    d = O.decide(p, [0, 0], 2, 1, q, u)
    assert d["accept_len"] == 1                       # 0.4 < 0.5 accepted, 0.6 >= 0.5 rejected
    assert d["next_token"] == 1                       # residual of row 1 = (0, 0.5)
    np.testing.assert_allclose(d["margins"][:2], [0.1, 0.1], atol=1e-6)
    u2 = np.array([0.4, 0.3, 0.2], dtype=np.float32)
    d2 = O.decide(p, [0, 0], 2, 1, q, u2)
    assert d2["accept_len"] == 2 and d2["next_token"] == 0   # bonus from row 2: 0.2 < 0.25


def test_boundary_conventions():
    """Ties: a neighbour that brings the running mass exactly to delta is still pooled; the
    sampled index is the smallest j whose cumulative mass strictly exceeds u * total."""
    p = np.array([0.5, 0.25, 0.25], dtype=np.float32)
    col = np.array([0, 1, 2, 1, 0, 2, 2, 0, 1], dtype=np.int32)
    row_ptr = np.array([0, 3, 6, 9], dtype=np.int32)
    assert O.pooled_mass(p, 0, row_ptr, col, 3, 0.25) == 0.75
    assert O.pooled_mass(p, 0, row_ptr, col, 3, 0.5) == 1.0
    assert O.pooled_mass(p, 0, row_ptr, col, 3, 0.2499) == 0.5
    assert O.inverse_cdf(np.array([0.5, 0.5], np.float32), 0.5)[0] == 1
    assert O.inverse_cdf(np.array([0.0, 0.5, 0.0, 0.5], np.float32), 0.5)[0] == 3
    assert O.inverse_cdf(np.array([0.0, 1.0, 0.0], np.float32), 1e-9)[0] == 1
