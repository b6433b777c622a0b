"""vvs_decide (the paper's Verify(logits, C_t), Alg. 2 line 10, on given target probabilities)
against the oracle's decision stage: same float32 inputs on both sides, so accept_len,
accept_mask and next_token must be bit-exact (a sample whose CDF margin is below 1e-12 of the
total mass may differ by float64 summation order and is excluded)."""
import numpy as np
import pytest

import helpers as H
from oracle import vvs_oracle as O
from vvs_synth import gen, philox
from vvs_synth.configs import DTYPE_BF16, MODE_RELAXED, MODE_STRICT, ModelShape

pytestmark = pytest.mark.gpu


def decide_case(seed, v, n_images, k, rows, first_row, mode, nbr_k, delta, tau, gumbel, off=0):
    rng = gen.rng_for(seed, "decide")
    t_logits = rng.standard_normal((n_images, rows, v)) * 2.0
    p = gen.softmax_rows_f32(t_logits)
    q = np.zeros((n_images, k, v), np.float32)
    drafts = np.zeros((n_images, k), np.int32)
    for b in range(n_images):
        for i in range(k):
            q[b, i], drafts[b, i] = gen.perturbed_draft_row(seed, f"q.{b}.{i}", t_logits[b, first_row + i],
                                                            0.0, tau, gumbel)
    n_draft = rng.integers(0, k + 1, size=n_images).astype(np.int32)
    n_draft[0] = k
    case = dict(ms=ModelShape("dec", 0, 64, 0, 0, 0, v, vocab_offset=off, dtype=DTYPE_BF16),
                probs=p, draft_probs=q, drafts=drafts + off, n_draft=n_draft,
                uniforms=philox.verify_uniforms(seed, 3, n_images, k), n_images=n_images,
                n_draft_max=k, rows=rows, first_row=first_row, mode=mode, nbr_k=nbr_k, delta=delta,
                row_ptr=None, col=None)
    if mode == MODE_RELAXED:
        case["row_ptr"], case["col"] = gen.neighbour_csr(gen.make_codebook(seed, v), nbr_k)
    return case


def oracle_decide(c):
    res = dict(accept_len=[], next_token=[], accept_mask=[], margins=[])
    off = c["ms"].vocab_offset
    for b in range(c["n_images"]):
        d = O.decide(c["probs"][b], c["drafts"][b] - off, int(c["n_draft"][b]), c["first_row"] + 1,
                     c["draft_probs"][b], c["uniforms"][b], c["mode"], c["row_ptr"], c["col"],
                     c["nbr_k"], c["delta"], c.get("adjusted_residual", False))
        res["accept_len"].append(d["accept_len"])
        res["next_token"].append(d["next_token"] + off if d["next_token"] >= 0 else -1)
        res["accept_mask"].append(d["accept_mask"])
        res["margins"].append(d["margins"])
    return {k: np.array(v) for k, v in res.items()}


def gpu_decide(c, call):
    """`call(ctx_or_None, vb, dev_inputs, outs)` issues the entry point under test."""
    import torch
    b, k = c["n_images"], c["n_draft_max"]
    o = dict(accept_len=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             next_token=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             accept_mask=torch.full((b, k), 9, dtype=torch.uint8, device="cuda"),
             margins=torch.zeros((b, k + 1), dtype=torch.float32, device="cuda"))
    d = dict(target_probs=H.to_dev(c["probs"]), drafts=H.to_dev(c["drafts"]),
             n_draft=H.to_dev(c["n_draft"]), draft_probs=H.to_dev(c["draft_probs"]),
             uniforms=H.to_dev(c["uniforms"]))
    if c["row_ptr"] is not None:
        d["row_ptr"], d["col"] = H.to_dev(c["row_ptr"]), H.to_dev(c["col"])
    call(d, o)
    torch.cuda.synchronize()
    return {k_: H.to_host(t) for k_, t in o.items()}


def compare_exact(c, got, want):
    k = c["n_draft_max"]
    np.testing.assert_array_equal(got["accept_len"], want["accept_len"])
    np.testing.assert_array_equal(got["accept_mask"], want["accept_mask"])
    for b in range(c["n_images"]):
        if want["margins"][b][k] < 1e-12:
            continue
        assert got["next_token"][b] == want["next_token"][b], b
    m = np.minimum(want["margins"][:, :k], 1e30)
    np.testing.assert_allclose(np.minimum(got["margins"][:, :k], 1e30), m, atol=1e-6)


CASES = [
    (1000, 3, 4, 5, 0, MODE_STRICT, 1, float("inf"), 1.0, 0.5, 0),
    (4096 + 40, 17, 8, 8, 0, MODE_RELAXED, 64, float("inf"), 0.5, 1.0, 100),
    (16384, 64, 16, 17, 0, MODE_RELAXED, 1000, 0.1, 1.5, 0.3, 0),
    (16384, 5, 8, 10, 1, MODE_RELAXED, 16, 0.2, 1.0, 2.0, 0),
    (65536, 2, 4, 5, 0, MODE_STRICT, 1, float("inf"), 1.0, 1.0, 0),
]


@pytest.mark.parametrize("v,n_images,k,rows,first_row,mode,nbr_k,delta,tau,gumbel,off", CASES)
def test_decide_is_bit_exact_with_oracle(v, n_images, k, rows, first_row, mode, nbr_k, delta, tau, gumbel, off):
    from paper_2511_13587_b200 import binding as vb
    c = decide_case(v + k, v, n_images, k, rows, first_row, mode, nbr_k, delta, tau, gumbel, off)
    ctx = vb.vvs_create(vb.make_desc(c["ms"], n_images, rows, nbr_k))

    def call(d, o):
        if "row_ptr" in d:
            vb.vvs_bind_neighbors(ctx, d["row_ptr"], d["col"])
        vb.vvs_decide(ctx, target_probs=d["target_probs"], n_rows_per_seq=rows, first_row=first_row,
                      drafts=d["drafts"], n_images=n_images, n_draft_max=k, n_draft=d["n_draft"],
                      draft_probs=d["draft_probs"], uniforms=d["uniforms"], mode=mode, nbr_k=nbr_k,
                      delta=delta, **o)
    got = gpu_decide(c, call)
    assert vb.vvs_device_status(ctx) == 0
    want = oracle_decide(c)
    compare_exact(c, got, want)
    rate = want["accept_len"].sum() / max(1, c["n_draft"].sum())
    assert 0.0 <= rate <= 1.0
    vb.vvs_destroy(ctx)


@pytest.mark.parametrize("v,n_images,k,rows,first_row,mode,nbr_k,delta,tau,gumbel,off",
                         [c for c in CASES if c[5] == MODE_RELAXED])
def test_adjusted_residual_is_bit_exact_with_oracle(v, n_images, k, rows, first_row, mode, nbr_k, delta, tau,
                                                    gumbel, off):
    """The adjusted-residual flag: same acceptances as the plain relaxed call, the sample drawn
    from the adjusted target's residual; on some image the two samples must differ."""
    from paper_2511_13587_b200 import binding as vb
    c = decide_case(v + k, v, n_images, k, rows, first_row, mode, nbr_k, delta, tau, gumbel, off)
    ctx = vb.vvs_create(vb.make_desc(c["ms"], n_images, rows, nbr_k))

    def call(flag):
        def run(d, o):
            vb.vvs_bind_neighbors(ctx, d["row_ptr"], d["col"])
            vb.vvs_decide(ctx, target_probs=d["target_probs"], n_rows_per_seq=rows, first_row=first_row,
                          drafts=d["drafts"], n_images=n_images, n_draft_max=k, n_draft=d["n_draft"],
                          draft_probs=d["draft_probs"], uniforms=d["uniforms"], mode=mode, nbr_k=nbr_k,
                          delta=delta, adjusted_residual=flag, **o)
        return run
    plain = gpu_decide(c, call(False))
    adj = gpu_decide(c, call(True))
    assert vb.vvs_device_status(ctx) == 0
    want = oracle_decide(dict(c, adjusted_residual=True))
    compare_exact(c, adj, want)
    np.testing.assert_array_equal(adj["accept_len"], plain["accept_len"])
    rejected = adj["accept_len"] < c["n_draft"]
    print("rejections", int(rejected.sum()), "of", n_images)
    if rejected.sum() >= 3:
        assert (adj["next_token"][rejected] != plain["next_token"][rejected]).any()
    np.testing.assert_array_equal(adj["next_token"][~rejected], plain["next_token"][~rejected])
    vb.vvs_destroy(ctx)


# ---------------------------------------------------------------------------------------
# candidate trees: the walk of vvs_verify's tree calls on given probabilities


def tree_decide_case(seed, v, n_images, k, n_forced, tau, gumbel, off=0):
    """Random trees (every draft node hangs below a uniformly drawn earlier node or the last
    forced row), target rows softmax(2 N(0,1)), one drafter row per parent node (its target
    logits cooled / perturbed), siblings drawn independently from it."""
    rng = gen.rng_for(seed, "tree_decide")
    rows = n_forced + k
    t_logits = rng.standard_normal((n_images, rows, v)) * 2.0
    p = gen.softmax_rows_f32(t_logits)
    parent = np.zeros((n_images, rows), np.int32)
    parent[:, :n_forced] = np.arange(-1, n_forced - 1)
    q = np.zeros((n_images, k, v), np.float32)
    drafts = np.zeros((n_images, k), np.int32)
    for b in range(n_images):
        for c in range(n_forced, rows):
            parent[b, c] = rng.integers(n_forced - 1, c)
        for pn in range(n_forced - 1, rows):
            kids = [c for c in range(n_forced, rows) if parent[b, c] == pn]
            if not kids:
                continue
            q_row, _ = gen.perturbed_draft_row(seed, f"tq.{b}.{pn}", t_logits[b, pn], 0.0, tau, gumbel)
            for c in kids:
                q[b, c - n_forced] = q_row
                drafts[b, c - n_forced] = gen.sample_rows(q_row[None, :], gen.rng_for(seed, f"tc.{b}.{c}").random(1))[0]
    return dict(ms=ModelShape("tdec", 0, 64, 0, 0, 0, v, vocab_offset=off, dtype=DTYPE_BF16), probs=p,
                draft_probs=q, drafts=drafts + off, parent=parent,
                uniforms=philox.verify_uniforms(seed, 5, n_images, k), n_images=n_images, n_draft_max=k,
                rows=rows, n_forced=n_forced)


@pytest.mark.parametrize("mode,nbr_k,delta,adjusted", [(MODE_STRICT, 1, float("inf"), False),
                                                       (MODE_RELAXED, 16, float("inf"), False),
                                                       (MODE_RELAXED, 64, 0.1, True),
                                                       (MODE_RELAXED, 8, float("inf"), True)])
@pytest.mark.parametrize("v,n_images,k,n_forced,tau,gumbel,off",
                         [(1000, 64, 12, 1, 1.0, 0.5, 0), (16384, 32, 15, 3, 0.5, 1.5, 100),
                          (4096 + 40, 16, 31, 1, 1.0, 2.5, 0), (512, 64, 6, 2, 2.0, 3.0, 7)])
def test_tree_walk_is_exact_on_random_trees(v, n_images, k, n_forced, tau, gumbel, off, mode, nbr_k, delta,
                                            adjusted):
    """Same float32 inputs on both sides: accepted paths and sampled tokens must be equal; only
    decisions within 1e-12 of their threshold (float64 summation order of a later-round
    normaliser, or of the sampling CDF) are left out."""
    import torch
    from paper_2511_13587_b200 import binding as vb
    c = tree_decide_case(v + k, v, n_images, k, n_forced, tau, gumbel, off)
    rows = c["rows"]
    ctx = vb.vvs_create(vb.make_desc(c["ms"], n_images, rows, nbr_k))
    row_ptr = col = None
    if mode == MODE_RELAXED:
        row_ptr, col = gen.neighbour_csr(gen.make_codebook(v + k, v), nbr_k)
        rp_d, col_d = H.to_dev(row_ptr), H.to_dev(col)
        vb.vvs_bind_neighbors(ctx, rp_d, col_d)
    o = dict(accept_len=torch.full((n_images,), -7, dtype=torch.int32, device="cuda"),
             next_token=torch.full((n_images,), -7, dtype=torch.int32, device="cuda"),
             accept_mask=torch.full((n_images, k), 9, dtype=torch.uint8, device="cuda"),
             accept_path=torch.full((n_images, k), -7, dtype=torch.int32, device="cuda"),
             margins=torch.zeros((n_images, k + 1), dtype=torch.float32, device="cuda"))
    vb.vvs_decide(ctx, target_probs=H.to_dev(c["probs"]), n_rows_per_seq=rows, first_row=n_forced - 1,
                  drafts=H.to_dev(c["drafts"]), n_images=n_images, n_draft_max=k,
                  draft_probs=H.to_dev(c["draft_probs"]), uniforms=H.to_dev(c["uniforms"]),
                  tree_parent=H.to_dev(c["parent"]), mode=mode, nbr_k=nbr_k, delta=delta,
                  adjusted_residual=adjusted, **o)
    torch.cuda.synchronize()
    assert vb.vvs_device_status(ctx) == 0
    got = {k_: H.to_host(t) for k_, t in o.items()}
    judged = rejected_rounds = 0
    for b in range(n_images):
        d = O.tree_decide(c["probs"][b], c["drafts"][b] - off, c["parent"][b], n_forced, c["draft_probs"][b],
                          c["uniforms"][b], mode, row_ptr, col, nbr_k, delta, adjusted)
        if np.any(d["margins"][:k] < 1e-12):
            continue
        n = int(got["accept_len"][b])
        assert n == d["accept_len"], b
        assert [int(x) for x in got["accept_path"][b][:n]] == d["accept_path"], b
        assert (got["accept_path"][b][n:] == -1).all()
        mask = np.zeros(k, np.uint8)
        mask[[x - n_forced for x in d["accept_path"]]] = 1
        np.testing.assert_array_equal(got["accept_mask"][b], mask)
        np.testing.assert_allclose(np.minimum(got["margins"][b][:k], 1e30), np.minimum(d["margins"][:k], 1e30), atol=1e-6)
        if d["margins"][k] >= 1e-12:
            assert got["next_token"][b] == d["next_token"] + off, b
        judged += int(np.isfinite(d["margins"][:k]).sum())
        rejected_rounds += int(np.isfinite(d["margins"][:k]).sum()) - d["accept_len"]
    assert judged > n_images and rejected_rounds > 0      # the cases exercise both outcomes
    vb.vvs_destroy(ctx)
