"""Parity of vvs_epilogue (LM head + guidance + softmax + decisions on given features) and of
the feature-cache store / fetch calls with the oracle, through the C ABI."""
from dataclasses import replace

import numpy as np
import pytest

import helpers as H
from oracle import vvs_oracle as O
from vvs_synth import gen, philox
from vvs_synth.configs import DTYPE_BF16, DTYPE_FP32, MODE_RELAXED, MODE_STRICT, ModelShape

pytestmark = pytest.mark.gpu


def _epilogue_case(d, v, n_images, n_cfg, k, rows, first_row, mode, nbr_k, delta, seed, tau=1.0,
                   gumbel=0.5, dtype=DTYPE_BF16, cfg_scale=2.0, temperature=1.0):
    """Features ~ N(0,1); LM head scaled so logits have a standard deviation near 2; drafter =
    target logits / tau + Gumbel noise (skewed draft/target pairs spanning acceptance rates)."""
    ms = ModelShape("epi", 0, d, 0, 0, 0, v, dtype=dtype)
    w = {"w_lm": gen.make_tensor(ms, seed, "w_lm", lm_std=2.0 / np.sqrt(d)), "layers": {}}
    hidden = gen.store(gen.rng_for(seed, "hidden").standard_normal((n_images * n_cfg, rows, d),
                                                                  dtype=np.float32), dtype)
    base = O.epilogue(ms, w, hidden, np.zeros((n_images, k), np.int32), np.zeros(n_images, np.int32),
                      first_row + 1, np.zeros((n_images, k, v), np.float32),
                      np.full((n_images, k + 1), 0.5, np.float32), n_cfg, cfg_scale, temperature)
    q = np.zeros((n_images, k, v), np.float32)
    drafts = np.zeros((n_images, k), np.int32)
    for b in range(n_images):
        for i in range(k):
            q[b, i], drafts[b, i] = gen.perturbed_draft_row(
                seed, f"q.{b}.{i}", base["logits"][b, first_row + i] / temperature, 0.0, tau, gumbel)
    u = philox.verify_uniforms(seed, 0, n_images, k)
    case = dict(ms=ms, w=w, hidden_in=hidden, rows=rows, first_row=first_row, drafts=drafts,
                draft_probs=q, uniforms=u, n_images=n_images, n_cfg=n_cfg, n_draft_max=k,
                n_draft=np.full(n_images, k, np.int32), cfg_scale=cfg_scale, temperature=temperature,
                mode=mode, nbr_k=nbr_k, delta=delta, row_ptr=None, col=None, n_forced=first_row + 1)
    if mode == MODE_RELAXED:
        case["row_ptr"], case["col"] = gen.neighbour_csr(gen.make_codebook(seed, v), nbr_k)
    case["block"] = np.concatenate([np.zeros((n_images, first_row + 1), np.int32), drafts], axis=1)
    return case


def _run_epilogue(case):
    import torch
    from paper_2511_13587_b200 import binding as vb
    c = case
    ms = c["ms"]
    b, k, v = c["n_images"], c["n_draft_max"], ms.vocab
    ctx = vb.vvs_create(vb.make_desc(ms, b * c["n_cfg"], c["rows"], max(1, c["nbr_k"])))
    wd = {"w_lm": H.to_dev(c["w"]["w_lm"]), "layers": []}
    vb.vvs_bind_weights(ctx, wd)
    if c["row_ptr"] is not None:
        rp, col = H.to_dev(c["row_ptr"]), H.to_dev(c["col"])
        vb.vvs_bind_neighbors(ctx, rp, col)
    o = dict(accept_len=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             next_token=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             accept_mask=torch.full((b, k), 9, dtype=torch.uint8, device="cuda"),
             margins=torch.zeros((b, k + 1), dtype=torch.float32, device="cuda"),
             target_probs=torch.zeros((b, c["rows"], v), dtype=torch.float32, device="cuda"))
    vb.vvs_epilogue(ctx, hidden_in=H.to_dev(c["hidden_in"]), n_rows_per_seq=c["rows"],
                    first_row=c["first_row"], drafts=H.to_dev(c["drafts"]), n_images=b,
                    n_cfg=c["n_cfg"], n_draft_max=k, n_draft=H.to_dev(c["n_draft"]),
                    draft_probs=H.to_dev(c["draft_probs"]), uniforms=H.to_dev(c["uniforms"]),
                    cfg_scale=c["cfg_scale"], temperature=c["temperature"], mode=c["mode"],
                    nbr_k=c["nbr_k"], delta=c["delta"], **o)
    res = {k_: H.to_host(t) for k_, t in o.items()}
    res["status"] = vb.vvs_device_status(ctx)
    res["launches"] = vb.vvs_last_launch_count(ctx)
    vb.vvs_destroy(ctx)
    return res


@pytest.mark.parametrize("d,v,n_images,n_cfg,k,bonus,mode,nbr_k,delta,tau", [
    (320, 4096, 1, 1, 4, True, MODE_STRICT, 1, float("inf"), 1.0),
    (320, 4096 + 136, 8, 2, 8, False, MODE_RELAXED, 64, float("inf"), 0.5),
    (512, 2048, 3, 2, 16, True, MODE_RELAXED, 1000, 0.2, 1.5),
    (512, 1000, 5, 1, 8, True, MODE_RELAXED, 1, float("inf"), 1.0),
    # points of the epilogue sweep at its own sizes (d in {1280, 4096}, V in {4096, 16384, 65536})
    (1280, 16384, 8, 2, 8, True, MODE_RELAXED, 64, float("inf"), 1.0),
    (1280, 16384, 1, 1, 4, True, MODE_RELAXED, 1000, 0.3, 0.5),
    (4096, 4096, 32, 2, 16, True, MODE_STRICT, 1, float("inf"), 1.5),
    (4096, 65536, 8, 2, 4, True, MODE_STRICT, 1, float("inf"), 1.0),
    (1280, 65536, 64, 1, 4, False, MODE_STRICT, 1, float("inf"), 0.7),
])
def test_epilogue_sweep_points(d, v, n_images, n_cfg, k, bonus, mode, nbr_k, delta, tau):
    rows = k + 1 if bonus else k
    case = _epilogue_case(d, v, n_images, n_cfg, k, rows, 0, mode, nbr_k, delta, seed=d + v + k, tau=tau)
    gpu = _run_epilogue(case)
    ora = O.epilogue(case["ms"], case["w"], case["hidden_in"], case["drafts"], case["n_draft"], 1,
                     case["draft_probs"], case["uniforms"], n_cfg, case["cfg_scale"],
                     case["temperature"], mode, case["row_ptr"], case["col"], nbr_k, delta)
    assert gpu["status"] == 0 and gpu["launches"] > 0
    dp = np.abs(gpu["target_probs"] - ora["target_probs"])
    assert dp.max() < 2e-3
    assert (dp / np.maximum(ora["target_probs"], 1e-12)).max() < 6e-2
    H.check_replay(case, gpu)
    if not bonus:                                        # no row after the last draft
        full = gpu["accept_len"] == k
        assert (gpu["next_token"][full] == -1).all()
        assert (gpu["next_token"][~full] >= 0).all()


def test_epilogue_fp32_matches_oracle_integers():
    case = _epilogue_case(256, 1024, 4, 2, 4, 5, 0, MODE_STRICT, 1, float("inf"), seed=9,
                          dtype=DTYPE_FP32, cfg_scale=1.7, temperature=0.9)
    gpu = _run_epilogue(case)
    ora = O.epilogue(case["ms"], case["w"], case["hidden_in"], case["drafts"], case["n_draft"], 1,
                     case["draft_probs"], case["uniforms"], 2, 1.7, 0.9)
    assert np.abs(gpu["target_probs"] - ora["target_probs"]).max() < 1e-5
    np.testing.assert_array_equal(gpu["accept_len"], ora["accept_len"])
    np.testing.assert_array_equal(gpu["next_token"], ora["next_token"])
    H.check_replay(case, gpu)


@pytest.mark.parametrize("dtype", [DTYPE_BF16, DTYPE_FP32])
def test_feature_cache_store_fetch(dtype):
    """Random store / fetch traffic with skip masks Bernoulli(0.5), gamma ~ U{1..5} and
    staleness 0..2 against the oracle ring: positions bit-exact, rows bit-exact copies."""
    import torch
    from paper_2511_13587_b200 import binding as vb
    d, n_images, n_cfg, cap, t_len, gmax = 1280, 16, 2, 13, 9, 5
    r = n_images * n_cfg
    ms = ModelShape("fc", 0, d, 0, 0, 0, 128, dtype=dtype)
    ctx = vb.vvs_create(vb.make_desc(ms, r, t_len))
    tdt = torch.bfloat16 if dtype == DTYPE_BF16 else torch.float32
    feat = torch.full((r, cap, d), 3.0, dtype=tdt, device="cuda")
    fpos = torch.full((r, cap), 123, dtype=torch.int32, device="cuda")
    newest = torch.full((r,), 55, dtype=torch.int32, device="cuda")
    fc = vb.make_fcache(feat, fpos, newest)
    vb.vvs_feature_cache_reset(ctx, fc)
    ofc = O.FeatureCache(r, cap, d)
    rng = gen.rng_for(77, f"fc.{dtype}")
    pos = rng.integers(0, 40, size=n_images).astype(np.int32)
    for step in range(12):
        hidden = gen.store(rng.standard_normal((r, t_len, d), dtype=np.float32), dtype)
        n_store_img = rng.integers(0, t_len + 1, size=n_images).astype(np.int32)
        base = np.tile(pos, n_cfg).astype(np.int32)
        if step % 4 == 3:                                # post verification: write back older positions
            base = np.maximum(base - 3, 0).astype(np.int32)
        n_store = np.tile(n_store_img, n_cfg).astype(np.int32)
        vb.vvs_feature_cache_store(ctx, fc, H.to_dev(hidden), t_len, H.to_dev(base), H.to_dev(n_store))
        ofc.store(O.widen(hidden), base, n_store)
        pos = np.maximum(pos, (base[:n_images] + n_store_img)).astype(np.int32)
        skip = (rng.random(n_images) < 0.5).astype(np.uint8)
        gamma = rng.integers(1, gmax + 1, size=r).astype(np.int32)
        stale = int(step % 3)
        out = torch.full((r, gmax, d), -5.0, dtype=tdt, device="cuda")
        out_pos = torch.full((r, gmax), -9, dtype=torch.int32, device="cuda")
        vb.vvs_feature_cache_fetch(ctx, fc, H.to_dev(skip), n_images, H.to_dev(gamma), gmax, stale,
                                   out, out_pos)
        want, want_pos = ofc.fetch(skip, gamma, stale, gmax)
        got, got_pos = H.to_host(out), H.to_host(out_pos)
        bits = vb.vvs_device_status(ctx)
        for row in range(r):
            if not skip[row % n_images]:
                assert (got_pos[row] == -9).all() and (got[row] == -5.0).all()
                continue
            g = gamma[row]
            np.testing.assert_array_equal(got_pos[row, :g], want_pos[row, :g])
            np.testing.assert_array_equal(got[row, :g], want[row, :g])
            assert (got_pos[row, g:] == -9).all()
        missed = any((want_pos[row, :gamma[row]] == -1).any() for row in range(r) if skip[row % n_images])
        assert bool(bits & vb.VVS_DEV_FCACHE_MISS) == missed
        np.testing.assert_array_equal(H.to_host(newest), ofc.newest)
        np.testing.assert_array_equal(H.to_host(fpos), ofc.fpos)
    vb.vvs_destroy(ctx)
