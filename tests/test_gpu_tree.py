"""Tree calls of vvs_verify (candidate token trees, Sec. 5) against the fp64 oracle.

Forward: every node's features and keys/values equal those of the plain chain forward over its
root path (oracle: tree_forward).  Decisions: the oracle's walk re-run on the float32
probabilities the GPU emitted must reproduce accept_len / accept_path / next_token exactly
(decisions within 1e-4 of their threshold excluded).  Cache: after the call the forced rows
and the accepted nodes sit contiguously behind the old fill level, everything else below the
old fill and above the block is untouched."""
import numpy as np
import pytest

import helpers as H
from oracle import vvs_oracle as O
from test_gpu_verify import _tols
from vvs_synth import gen
from vvs_synth.configs import B7_SMALL, MODE_RELAXED, XL_SMALL

pytestmark = pytest.mark.gpu

# F = 1, K = 8: two children of the root, a three-way split below the first, chains below
TREE_A = [-1, 0, 0, 1, 1, 1, 2, 3, 7]
# F = 2, K = 7: siblings directly under the last forced row, one deep branch
TREE_B = [-1, 0, 1, 1, 1, 2, 5, 6, 3]
# F = 1, K = 6 (two images with guidance stay within the 32 block tokens of a tree call)
TREE_C = [-1, 0, 0, 1, 1, 2, 4]


def _replay(case, gpu):
    c, ms = case, case["ms"]
    out = []
    for b in range(c["n_images"]):
        out.append(O.tree_decide(gpu["target_probs"][b].astype(np.float32),
                                 c["block"][b, c["n_forced"]:] - ms.vocab_offset, c["parent"][b],
                                 c["n_forced"], c["draft_probs"][b], c["uniforms"][b],
                                 c.get("mode", 0), c.get("row_ptr"), c.get("col"), c.get("nbr_k", 1),
                                 c.get("delta", float("inf")), c.get("adjusted_residual", False)))
    return out


def _check_tree(case, gpu, ora):
    c, ms = case, case["ms"]
    tol = _tols(ms)
    f, k = c["n_forced"], c["n_draft_max"]
    t_len = f + k
    assert gpu["status"] == 0
    assert H.rel_err_rows(gpu["hidden"], ora["hidden"]) < tol["h_rel"]
    dp = np.abs(gpu["target_probs"] - ora["target_probs"])
    assert (dp < np.maximum(tol["p_abs"], tol["p_rel"] * ora["target_probs"])).all()
    np.testing.assert_allclose(gpu["target_probs"].sum(-1), 1.0, atol=1e-4)
    # decisions: replay of the oracle's walk on the GPU's probabilities
    rep = _replay(case, gpu)
    excluded = 0
    for b in range(c["n_images"]):
        r = rep[b]
        n = int(gpu["accept_len"][b])
        path = [int(x) for x in gpu["accept_path"][b][:n]]
        if np.any(r["margins"][:k] < 1e-4) and (n != r["accept_len"] or path != r["accept_path"]):
            excluded += 1
            continue
        assert n == r["accept_len"] and path == r["accept_path"], (b, path, r["accept_path"])
        assert (gpu["accept_path"][b][n:k] == -1).all()
        mask = np.zeros(k, np.uint8)
        mask[[p - f for p in path]] = 1
        np.testing.assert_array_equal(gpu["accept_mask"][b][:k], mask)
        np.testing.assert_allclose(np.minimum(gpu["margins"][b][:k], 1e30), np.minimum(r["margins"][:k], 1e30),
                                   atol=1e-6)
        if r["margins"][k] < 1e-9 and gpu["next_token"][b] != r["next_token"] + ms.vocab_offset:
            excluded += 1
            continue
        assert gpu["next_token"][b] == r["next_token"] + ms.vocab_offset
        # every accepted node is a child of the one before it
        prev = f - 1
        for p in path:
            assert c["parent"][b][p] == prev
            prev = p
    # cache: forced rows, then the accepted nodes, contiguous; the rest untouched
    k0, v0 = O.widen(c["kv_k"]), O.widen(c["kv_v"])
    rtol = tol["h_rel"] * (2.0 if ms.n_layers > 3 else 1.0)
    for r in range(c["n_images"] * c["n_cfg"]):
        b = r % c["n_images"]
        fill, n = int(c["cache_len"][r]), int(gpu["accept_len"][b])
        assert gpu["new_len"][r] == fill + f + n and gpu["n_commit"][r] == f + n
        rows = list(range(f)) + [int(x) for x in gpu["accept_path"][b][:n]]
        for got, ref, orig in ((gpu["kv_k"], ora["k_node"], k0), (gpu["kv_v"], ora["v_node"], v0)):
            new = got[:, r, :, fill:fill + f + n]
            assert H.rel_err_rows(new, ref[:, r][:, :, rows]) < rtol, r
            np.testing.assert_array_equal(got[:, r, :, :fill], orig[:, r, :, :fill])
            np.testing.assert_array_equal(got[:, r, :, fill + t_len:], orig[:, r, :, fill + t_len:])
    return excluded


@pytest.mark.parametrize("parent,n_forced,n_images,fills,q_noise",
                         [(TREE_A, 1, 1, [130], 0.5), (TREE_C, 1, 2, [17, 300], 1.0),
                          (TREE_B, 2, 1, [124], 0.5)])
def test_tree_parity_xl_small(parent, n_forced, n_images, fills, q_noise):
    """Fill 124 + 9 block rows puts the block across a 128-key chunk boundary."""
    ms = XL_SMALL
    case = H.build_tree_case(ms, 41 + n_images + n_forced, n_images, 2, n_forced, parent, fills, q_noise=q_noise)
    run = H.GpuRunner(ms, case["w"], 2 * n_images, len(parent))
    gpu = H.run_tree_gpu(run, case)
    ora = H.run_tree_oracle(case)
    _check_tree(case, gpu, ora)
    print("tree accept paths", [list(g[:n]) for g, n in zip(gpu["accept_path"], gpu["accept_len"])],
          "oracle", ora["accept_path"])
    run.close()


@pytest.mark.parametrize("nbr_k,delta,adjusted", [(64, float("inf"), False), (16, 0.05, True), (64, float("inf"), True)])
def test_relaxed_tree_parity_xl_small(nbr_k, delta, adjusted):
    """Relaxed acceptance on a candidate tree (the pooled mass is taken in the current residual),
    with and without the adjusted-residual flag, through vvs_verify against the oracle's walk."""
    ms = XL_SMALL
    case = H.build_tree_case(ms, 52, 2, 2, 1, TREE_C, [40, 311], q_noise=1.5)
    case.update(mode=MODE_RELAXED, nbr_k=nbr_k, delta=delta, adjusted_residual=adjusted)
    case["row_ptr"], case["col"] = gen.neighbour_csr(gen.make_codebook(52, ms.vocab), nbr_k)
    run = H.GpuRunner(ms, case["w"], 4, len(TREE_C), max_nbr_k=nbr_k)
    gpu = H.run_tree_gpu(run, case)
    ora = H.run_tree_oracle(case)
    _check_tree(case, gpu, ora)
    strict = _replay(dict(case, mode=0), gpu)
    print("relaxed tree paths", [list(g[:n]) for g, n in zip(gpu["accept_path"], gpu["accept_len"])],
          "strict walk on the same rows", [r["accept_path"] for r in strict])
    run.close()


def test_tree_parity_7b_small_1d_rope():
    """1-D rope: a node's position is fill + depth, not fill + index."""
    ms = B7_SMALL
    case = H.build_tree_case(ms, 77, 1, 2, 1, TREE_A, [201], q_noise=0.5)
    run = H.GpuRunner(ms, case["w"], 2, 9)
    gpu = H.run_tree_gpu(run, case)
    ora = H.run_tree_oracle(case)
    _check_tree(case, gpu, ora)
    run.close()


def test_chain_shaped_tree_equals_chain_call():
    """parent[t] = t - 1: same decisions, probabilities and cache rows as the plain call."""
    ms = XL_SMALL
    case = H.build_case(ms, 12, 2, 2, 1, 6, [288, 33], q_noise=0.7)
    run = H.GpuRunner(ms, case["w"], 4, 7)
    chain = run.verify(case)
    tcase = dict(case, parent=np.tile(np.arange(-1, 6, dtype=np.int32), (2, 1)))
    tree = H.run_tree_gpu(run, tcase)
    # split-K sums arrive in any order, so two runs of the same call already differ by bf16
    # rounding flips of intermediate rows: a few 1e-3 relative on single probabilities
    np.testing.assert_allclose(tree["target_probs"], chain["target_probs"], rtol=3e-2, atol=1e-5)
    rep = H.replay_decisions(case, tree["target_probs"])
    for b in range(2):
        if np.any(rep["margins"][b][:6] < 1e-4):
            continue
        n = int(tree["accept_len"][b])
        assert n == rep["accept_len"][b]
        np.testing.assert_array_equal(tree["accept_path"][b][:n], 1 + np.arange(n))
        if rep["margins"][b][6] >= 1e-9:
            assert tree["next_token"][b] == rep["next_token"][b]
    t_len = 7
    for r in range(4):
        fill = int(case["cache_len"][r])
        for a, b_ in ((tree["kv_k"], chain["kv_k"]), (tree["kv_v"], chain["kv_v"])):
            assert H.rel_err_rows(a[:, r, :, fill:fill + t_len], b_[:, r, :, fill:fill + t_len]) < 1e-2
    run.close()


def test_tree_argument_errors():
    import torch
    ms = XL_SMALL
    case = H.build_tree_case(ms, 5, 1, 2, 1, TREE_A, [50])
    run = H.GpuRunner(ms, case["w"], 2, 9)
    vb = run.vb
    bad = dict(case, parent=np.array([[-1, 0, 0, 1, 1, 1, 2, 8, 7]], dtype=np.int32))   # parent after child
    gpu = H.run_tree_gpu(run, bad)
    assert gpu["status"] & vb.VVS_DEV_BAD_ARG
    # a missing probability buffer, a relaxed call without a neighbour table and a flag value other
    # than 0 / 1 are refused before any launch
    b, r, k, t_len = 1, 2, 8, 9
    common = dict(n_images=b, n_cfg=2, n_forced=1, n_draft_max=k, block=H.to_dev(case["block"]),
                  kv_k=H.to_dev(case["kv_k"]), kv_v=H.to_dev(case["kv_v"]), kv_rows=case["kv_rows"],
                  cache_len=H.to_dev(case["cache_len"]), draft_probs=H.to_dev(case["draft_probs"]),
                  uniforms=H.to_dev(case["uniforms"]), tree_parent=H.to_dev(case["parent"]),
                  accept_len=torch.zeros(b, dtype=torch.int32, device="cuda"),
                  next_token=torch.zeros(b, dtype=torch.int32, device="cuda"),
                  new_len=torch.zeros(r, dtype=torch.int32, device="cuda"))
    with pytest.raises(vb.VvsError):
        vb.vvs_verify(run.ctx, **common)
    probs = torch.zeros((b, t_len, ms.vocab), dtype=torch.float32, device="cuda")
    with pytest.raises(vb.VvsError):
        vb.vvs_verify(run.ctx, mode=MODE_RELAXED, nbr_k=2, target_probs=probs, **common)
    with pytest.raises(vb.VvsError):
        vb.vvs_verify(run.ctx, adjusted_residual=2, target_probs=probs, **common)
    run.close()


@pytest.mark.parametrize("name,seed,parent,n_forced,n_cfg,q_noise",
                         [("seven siblings, all rejected", 407, [-1, 0, 0, 0, 0, 0, 0, 0], 1, 2, 3.0),
                          ("seven siblings, the last accepted", 400, [-1, 0, 0, 0, 0, 0, 0, 0], 1, 2, 3.0),
                          ("chain ending in three leaves", 308, [-1, 0, 1, 2, 3, 4, 4, 4], 1, 2, 0.3),
                          ("17 block rows, no guidance", 317, [-1, 0, 1, 2, 2, 3, 3, 4, 4, 5, 6, 7, 8, 9, 10, 11, 12], 3, 1, 1.0),
                          ("forced rows only", 303, [-1, 0, 1], 3, 2, 1.0)])
def test_tree_shapes(name, seed, parent, n_forced, n_cfg, q_noise):
    """Wide, deep, long and degenerate trees.  A drafter far from the target (noise 3.0) makes
    siblings fail one after the other, so the walk goes through one residual update per rejected
    sibling (the float64 rounds) before it accepts or samples; a tree without draft nodes samples
    from the last forced row."""
    ms = XL_SMALL
    case = H.build_tree_case(ms, seed, 1, n_cfg, n_forced, parent, [77], q_noise=q_noise)
    run = H.GpuRunner(ms, case["w"], n_cfg, len(parent))
    gpu = H.run_tree_gpu(run, case)
    ora = H.run_tree_oracle(case)
    assert _check_tree(case, gpu, ora) == 0
    np.testing.assert_array_equal(gpu["accept_len"], ora["accept_len"])
    print(name, "accepted", gpu["accept_path"][0][:gpu["accept_len"][0]], "oracle", ora["accept_path"][0])
    run.close()


@pytest.mark.parametrize("n_images,parent,n_forced,fills",
                         [(2, TREE_A, 1, [130, 17]),                     # 36 tokens: QKV epilogue with rotation tables
                          (4, TREE_B, 2, [124, 300, 5, 511]),            # 72 tokens: split-K sums + rotate/append kernel
                          (3, [-1, 0, 1, 2, 2, 3, 3, 4, 4, 5, 6, 7, 8, 9, 10, 11, 12, 12, 12, 13, 14], 3, [60, 400, 222])])
def test_tree_parity_per_projection_kernels(n_images, parent, n_forced, fills):
    """More than 32 block tokens: the per-projection tensor-core kernels (attention with the same
    visibility masks, rotation by depth from the step's tables)."""
    ms = XL_SMALL
    case = H.build_tree_case(ms, 900 + n_images, n_images, 2, n_forced, parent, fills, q_noise=0.7)
    run = H.GpuRunner(ms, case["w"], 2 * n_images, len(parent))
    gpu = H.run_tree_gpu(run, case)
    assert gpu["launches"] > 20            # not the whole-chain kernel
    ora = H.run_tree_oracle(case)
    _check_tree(case, gpu, ora)
    print("accept paths", [list(g[:n]) for g, n in zip(gpu["accept_path"], gpu["accept_len"])], "oracle", ora["accept_path"])
    run.close()
