"""Pins of the oracle's tree verification: a tree that is a chain reproduces the chain rule bit for
bit; the multi-round rule over sibling candidates is lossless (exact enumeration on a 4-token
vocabulary whose ratios fall on the uniform grid); tree attention equals chain attention on every
root path."""
import numpy as np

from oracle import vvs_oracle as O
from vvs_synth import gen
from vvs_synth.configs import TINY


def test_chain_shaped_tree_is_the_chain_rule():
    rng = np.random.default_rng(5)
    for trial in range(200):
        v, k, f = 7, 4, int(rng.integers(1, 3))
        p = rng.random((f + k, v)).astype(np.float32); p /= p.sum(-1, keepdims=True)
        q = rng.random((k, v)).astype(np.float32); q /= q.sum(-1, keepdims=True)
        drafts = rng.integers(0, v, k)
        u = rng.random(k + 1).astype(np.float32)
        parent = np.arange(-1, f + k - 1)
        a = O.decide(p, drafts, k, f, q, u)
        b = O.tree_decide(p, drafts, parent, f, q, u)
        assert b["accept_len"] == a["accept_len"] and b["next_token"] == a["next_token"]
        assert b["accept_path"] == list(range(f, f + a["accept_len"]))
        n = min(a["accept_len"] + 1, k)
        np.testing.assert_allclose(b["margins"][:n], a["margins"][:n])
        assert b["margins"][k] == a["margins"][k]


def test_two_sibling_candidates_are_lossless_by_enumeration():
    """Root with two children drawn independently from q: the first emitted token (an accepted child
    or the residual sample) is distributed as p.  p, q chosen so that every ratio is a multiple of
    1/4 and the last residual has masses 17/24, 7/24 (15/20, 5/20 if the first residual were not
    normalised, which would break the identity): the midpoint grids integrate exactly."""
    p = np.array([[0.5, 0.3, 0.1, 0.1]] * 3, dtype=np.float32)
    q = np.array([0.1, 0.1, 0.4, 0.4], dtype=np.float32)
    parent = np.array([-1, 0, 0])
    g, gs = 20, 120
    out = np.zeros(4)
    for x1 in range(4):
        for x2 in range(4):
            w = float(q[x1]) * float(q[x2])
            for i1 in range(g):
                for i2 in range(g):
                    u = [(i1 + 0.5) / g, (i2 + 0.5) / g, 0.5]
                    d = O.tree_decide(p, [x1, x2], parent, 1, np.stack([q, q]), np.array(u))
                    if d["accept_len"] == 1:
                        out[[x1, x2][d["accept_path"][0] - 1]] += w / (g * g)
                    else:
                        for js in range(gs):
                            u[2] = (js + 0.5) / gs
                            d2 = O.tree_decide(p, [x1, x2], parent, 1, np.stack([q, q]), np.array(u))
                            out[d2["next_token"]] += w / (g * g * gs)
    np.testing.assert_allclose(out, p[0], atol=1e-6)


def test_tree_rows_equal_chain_rows_on_every_root_path():
    ms = TINY
    w = gen.make_weights(ms, 3)
    kv_k, kv_v = gen.make_kv_cache(ms, 3, 1)
    kc, vc = O.widen(kv_k[:, 0]), O.widen(kv_v[:, 0])
    tokens = np.array([5, 17, 99, 23, 512, 7])
    parent = np.array([-1, 0, 0, 1, 1, 2])          # root 0; children 1, 2; 3, 4 under 1; 5 under 2
    h, k_node, v_node = O.tree_forward(ms, w, tokens, parent, kc, vc, 20)
    for leaf in (3, 4, 5):
        path = O.tree_ancestors(parent, leaf)
        kc2, vc2 = kc.copy(), vc.copy()
        hc = O.target_forward(ms, w, tokens[path], kc2, vc2, 20)
        np.testing.assert_allclose(h[path], hc, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(k_node[:, :, path], kc2[:, :, 20:20 + len(path)], rtol=1e-12, atol=1e-12)
    assert O.tree_ancestors(parent, 4) == [0, 1, 4]
    # siblings share their ancestors but not each other: node 4's features do not depend on node 3's token
    tokens2 = tokens.copy(); tokens2[3] = 1000
    h2, _, _ = O.tree_forward(ms, w, tokens2, parent, kc, vc, 20)
    np.testing.assert_array_equal(h2[4], h[4])
    assert np.abs(h2[3] - h[3]).max() > 1e-6


# ---------------------------------------------------------------------------------------
# relaxed acceptance on trees and the adjusted-residual flag


def _ragged_csr(rng, v, k_max):
    """Neighbour rows of uneven length (the code itself first, then distinct other codes)."""
    row_ptr, col = [0], []
    for x in range(v):
        n = int(rng.integers(1, k_max + 1))
        others = [int(c) for c in rng.permutation(v) if c != x][:n - 1]
        col += [x] + others
        row_ptr.append(len(col))
    return np.array(row_ptr, np.int32), np.array(col, np.int32)


def test_relaxed_chain_shaped_tree_is_the_relaxed_chain_rule_with_and_without_the_flag():
    rng = np.random.default_rng(11)
    hits = 0
    for trial in range(300):
        v, k, f = 9, 4, int(rng.integers(1, 3))
        p = rng.random((f + k, v)).astype(np.float32); p /= p.sum(-1, keepdims=True)
        q = rng.random((k, v)).astype(np.float32); q /= q.sum(-1, keepdims=True)
        drafts = rng.integers(0, v, k)
        u = rng.random(k + 1).astype(np.float32)
        rp, col = _ragged_csr(rng, v, 5)
        nk, delta = int(rng.integers(1, 6)), [float("inf"), 0.3, 0.1][trial % 3]
        parent = np.arange(-1, f + k - 1)
        for flag in (False, True):
            a = O.decide(p, drafts, k, f, q, u, O.MODE_RELAXED, rp, col, nk, delta, flag)
            b = O.tree_decide(p, drafts, parent, f, q, u, O.MODE_RELAXED, rp, col, nk, delta, flag)
            assert b["accept_len"] == a["accept_len"] and b["next_token"] == a["next_token"]
            assert b["margins"][k] == a["margins"][k]
        s = O.decide(p, drafts, k, f, q, u)
        hits += a["accept_len"] != s["accept_len"] or a["next_token"] != s["next_token"]
    assert hits > 30          # the relaxed cases are not the strict ones in disguise


def test_relaxed_tree_with_one_neighbour_is_the_strict_walk():
    rng = np.random.default_rng(12)
    parent = np.array([-1, 0, 0, 1, 1, 2, 3])
    for trial in range(100):
        v = 8
        p = rng.random((7, v)).astype(np.float32); p /= p.sum(-1, keepdims=True)
        q = rng.random((6, v)).astype(np.float32); q /= q.sum(-1, keepdims=True)
        q[1], q[3], q[5] = q[0], q[2], q[2]                   # siblings share their parent's row
        drafts = rng.integers(0, v, 6)
        u = rng.random(7).astype(np.float32)
        rp, col = _ragged_csr(rng, v, 4)
        s = O.tree_decide(p, drafts, parent, 1, q, u)
        for flag in (False, True):
            r = O.tree_decide(p, drafts, parent, 1, q, u, O.MODE_RELAXED, rp, col, 1, float("inf"), flag)
            assert r["accept_path"] == s["accept_path"] and r["next_token"] == s["next_token"]
            np.testing.assert_array_equal(r["margins"], s["margins"])
            r0 = O.tree_decide(p, drafts, parent, 1, q, u, O.MODE_RELAXED, rp, col, 4, 0.0, flag)
            assert r0["accept_path"] == s["accept_path"] and r0["next_token"] == s["next_token"]


def test_adjusted_target_moves_the_pooled_mass_onto_the_draft():
    p = np.array([0.2, 0.1, 0.3, 0.25, 0.15], dtype=np.float32)
    rp, col = np.array([0, 3, 4, 5, 6, 7], np.int32), np.array([0, 1, 3, 1, 2, 3, 4], np.int32)
    np.testing.assert_allclose(O.adjusted_target(p, 0, rp, col, 3, float("inf")), [0.55, 0, 0.3, 0, 0.15], atol=1e-7)
    # delta = 0.2: neighbour 1 (0.1) fits, neighbour 3 (0.25) would take the pooled mass to 0.35
    np.testing.assert_allclose(O.adjusted_target(p, 0, rp, col, 3, 0.2), [0.3, 0, 0.3, 0.25, 0.15], atol=1e-7)
    np.testing.assert_allclose(O.adjusted_target(p, 0, rp, col, 2, float("inf")), [0.3, 0, 0.3, 0.25, 0.15], atol=1e-7)
    np.testing.assert_array_equal(O.adjusted_target(p, 2, rp, col, 3, float("inf")), p)   # no neighbours: unchanged
    rng = np.random.default_rng(13)
    for _ in range(50):                                        # the total mass never changes
        pr = rng.random(12); pr /= pr.sum()
        rp2, col2 = _ragged_csr(rng, 12, 6)
        x = int(rng.integers(0, 12))
        a = O.adjusted_target(pr, x, rp2, col2, 6, [float("inf"), 0.2][_ % 2])
        assert abs(a.sum() - 1.0) < 1e-12 and a[x] == O.pooled_mass(pr, x, rp2, col2, 6, [float("inf"), 0.2][_ % 2])
        assert all(a[c] == 0 for c in O.pooled_neighbours(pr, x, rp2, col2, 6, [float("inf"), 0.2][_ % 2]))


def test_adjusted_residual_hand_example():
    """p = (.1,.2,.3,.4), neighbours of code 0 = {0, 1}, q = (.5,.1,.2,.2), draft 0 rejected
    (ratio .3/.5 = .6 < u).  Plain residual max(0, p - q) = (0,.1,.1,.2): the point .2 of its CDF
    falls on code 1.  Adjusted target (.3,0,.3,.4), residual (0,0,.1,.2): the same point falls on
    code 2."""
    p = np.array([[0.1, 0.2, 0.3, 0.4]] * 2, dtype=np.float32)
    q = np.array([[0.5, 0.1, 0.2, 0.2]], dtype=np.float32)
    rp, col = np.array([0, 2, 3, 4, 5], np.int32), np.array([0, 1, 1, 2, 3], np.int32)
    u = np.array([0.7, 0.2], dtype=np.float32)
    plain = O.decide(p, [0], 1, 1, q, u, O.MODE_RELAXED, rp, col, 2, float("inf"))
    adj = O.decide(p, [0], 1, 1, q, u, O.MODE_RELAXED, rp, col, 2, float("inf"), True)
    assert plain["accept_len"] == 0 and adj["accept_len"] == 0
    assert abs(plain["ratios"][0] - 0.6) < 1e-6
    assert plain["next_token"] == 1 and adj["next_token"] == 2
    parent = np.array([-1, 0])
    assert O.tree_decide(p, [0], parent, 1, q, u, O.MODE_RELAXED, rp, col, 2, float("inf"))["next_token"] == 1
    assert O.tree_decide(p, [0], parent, 1, q, u, O.MODE_RELAXED, rp, col, 2, float("inf"), True)["next_token"] == 2


def test_adjusted_residual_emits_the_adjusted_target_when_the_drafter_is_certain():
    """A drafter that always proposes code 0 (q = point mass): speculative sampling is lossless for
    whatever distribution its ratio and residual are built from, and with the flag on both are
    built from the adjusted target of code 0 - here (.55, 0, .3, 0, .15), typed by hand.  Exact
    enumeration over the uniforms, for the chain rule and for a root with two children (both code
    0: the second round finds no mass left on the pooled codes and passes the residual on)."""
    p = np.array([[0.2, 0.1, 0.3, 0.25, 0.15]] * 3, dtype=np.float32)
    q1 = np.array([1.0, 0, 0, 0, 0], dtype=np.float32)
    rp, col = np.array([0, 3, 4, 5, 6, 7], np.int32), np.array([0, 1, 3, 1, 2, 3, 4], np.int32)
    want = np.array([0.55, 0.0, 0.3, 0.0, 0.15])
    g, gs = 20, 30
    chain, tree, plain = np.zeros(5), np.zeros(5), np.zeros(5)
    for i1 in range(g):
        for js in range(gs):
            u = np.array([(i1 + 0.5) / g, (js + 0.5) / gs])
            for out, flag in ((chain, True), (plain, False)):
                d = O.decide(p[:2], [0], 1, 1, q1[None], u, O.MODE_RELAXED, rp, col, 3, float("inf"), flag)
                out[0 if d["accept_len"] else d["next_token"]] += 1.0 / (g * gs)
            for i2 in range(4):
                u3 = np.array([(i1 + 0.5) / g, (i2 + 0.5) / 4, (js + 0.5) / gs])
                d = O.tree_decide(p, [0, 0], np.array([-1, 0, 0]), 1, np.stack([q1, q1]), u3, O.MODE_RELAXED,
                                  rp, col, 3, float("inf"), True)
                tree[0 if d["accept_len"] else d["next_token"]] += 1.0 / (g * gs * 4)
    np.testing.assert_allclose(chain, want, atol=1e-9)
    np.testing.assert_allclose(tree, want, atol=1e-9)
    # without the flag the pooled codes 1 and 3 can still be emitted after a rejection
    np.testing.assert_allclose(plain, [0.55, 0.45 * 0.1 / 0.8, 0.45 * 0.3 / 0.8, 0.45 * 0.25 / 0.8, 0.45 * 0.15 / 0.8],
                               atol=0.02)
    assert plain[1] > 0.03 and plain[3] > 0.1
