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
