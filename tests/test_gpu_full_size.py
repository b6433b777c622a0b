"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

configs[1]: the whole LlamaGen-XL shape (36 layers, d = 1280, V = 16384), batch 1 with guidance,
K = 8: the oracle finishes one such step in seconds, so every output is compared.
configs[2] (16 images x guidance, relaxed acceptance, 36 layers) and configs[3] (the 7B shape, 32
layers, fill 1500): one full-depth trial each with a target-independent drafter (no teacher-forced
oracle passes; the oracle's single pass takes a minute or a few), every output compared, plus the
quick two-layer versions with the target-aware drafter."""
from dataclasses import replace

import numpy as np
import pytest

import helpers as H
from oracle import vvs_oracle as O
from vvs_synth import gen
from test_gpu_verify import _check_end_to_end
from vvs_synth.configs import B7, CONFIGS, MODE_RELAXED, XL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("chain_kernels", [False, True])
@pytest.mark.parametrize("deterministic", [True, False])
def test_config1_full_llamagen_xl_shape(deterministic, chain_kernels):
    """Fill 477: eight 64-key blocks per (sequence, head) in the per-projection path; four 128-key
    chunks per item, i.e. more attention work items than SMs, in the whole-chain kernels.  Fixed-order
    and arrival-order sums on both generations of kernels."""
    wl, fill = CONFIGS[1], 477
    case = H.build_case(wl.shape, wl.seed + fill, 1, 2, 1, 8, [fill], cfg_scale=wl.cfg_scale, q_noise=0.3)
    run = H.GpuRunner(wl.shape, case["w"], 2, 9, deterministic=deterministic, chain_kernels=chain_kernels)
    gpu = run.verify(case)
    assert (gpu["launches"] < 40) == chain_kernels      # one persistent kernel, or one kernel per projection
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    print("configs[1] full size: accept_len", gpu["accept_len"], "oracle", ora["accept_len"])
    # The configuration the benchmark times does not ask for probabilities.  With fixed-order sums
    # the step repeats bit for bit, so the sampled token is the one of the checked call.  With
    # arrival-order sums two runs differ in the last bits of the logits: the accepted prefix
    # (margins far above that) must repeat, the residual sample over 16384 almost equally likely
    # codes need not and is only checked for range.
    gpu2 = run.verify(case, want_probs=False)
    clear = np.ones(case["n_images"], bool)
    if not deterministic:       # a decision within the run-to-run distance of its threshold may flip
        clear = (H.replay_decisions(case, gpu["target_probs"])["margins"][:, :case["n_draft_max"]] > 2e-2).all(axis=1)
    np.testing.assert_array_equal(gpu2["accept_len"][clear], gpu["accept_len"][clear])
    ms = wl.shape
    assert ((gpu2["next_token"] >= ms.vocab_offset) & (gpu2["next_token"] < ms.vocab_offset + ms.vocab)).all()
    if deterministic:
        np.testing.assert_array_equal(gpu2["next_token"], gpu["next_token"])
        np.testing.assert_array_equal(gpu2["hidden"], gpu["hidden"])
    else:
        # the token of the call without probabilities, checked without them: on the residual row built
        # from the CHECKED call's probabilities, the CDF interval of the returned code must contain the
        # sample point u up to the distance two arrival-order runs can move a CDF: at this depth their
        # features differ by ~2 % of the row norm, single probabilities by a few per cent, and since those
        # differences are correlated over the codebook a CDF value moves by up to about 1e-2 (5.3e-3 seen)
        k, f = case["n_draft_max"], case["n_forced"]
        for b in range(case["n_images"]):
            if not clear[b]:
                continue
            n = int(gpu2["accept_len"][b])
            row = gpu["target_probs"][b][f - 1 + n].astype(np.float32)
            r = np.maximum(np.float32(0), row - case["draft_probs"][b][n]) if n < k else row
            cdf = np.cumsum(r.astype(np.float64)) / float(r.astype(np.float64).sum())
            t = int(gpu2["next_token"][b]) - ms.vocab_offset
            lo, hi, u = (cdf[t - 1] if t > 0 else 0.0), cdf[t], float(case["uniforms"][b][k])
            assert lo - 2e-2 <= u <= hi + 2e-2, (b, t, lo, u, hi)
    run.close()


def test_config3_7b_width_two_layers():
    """d = 4096, 32 heads of 128, MLP 11008, 8192 codes inside a 65536-row head, fill 1500."""
    ms = replace(B7, name="visual_ar_7b_2layers", n_layers=2)
    case = H.build_case(ms, 0x56565303, 1, 2, 1, 8, [1500])
    run = H.GpuRunner(ms, case["w"], 2, 9)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    assert ((gpu["next_token"] >= ms.vocab_offset) & (gpu["next_token"] < ms.vocab_offset + ms.vocab)).all()
    run.close()


def test_config2_batch16_relaxed_two_layers():
    """16 images x guidance = 32 sequences (288 block rows), fills drawn per image, relaxed
    acceptance with 64 neighbours: the per-projection tensor-core kernels, two token passes."""
    wl = CONFIGS[2]
    ms = replace(XL, name="llamagen_xl_2layers", n_layers=2)
    fills = [1, 575, 130, 288, 17, 400, 333, 128, 127, 129, 256, 500, 64, 9, 511, 200]
    case = H.build_case(ms, wl.seed, 16, 2, 1, 8, fills, mode=MODE_RELAXED, nbr_k=64, q_noise=1.5)
    run = H.GpuRunner(ms, case["w"], 32, 9, max_nbr_k=64)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    run.close()


def test_config1_full_shape_candidate_tree():
    """The configs[1] network at full depth on a candidate tree (two siblings below the root, a
    three-way split, chains): features, probabilities, walk and compacted cache rows."""
    from test_gpu_tree import TREE_A, _check_tree
    wl, fill = CONFIGS[1], 477
    case = H.build_tree_case(wl.shape, wl.seed + 1, 1, 2, 1, TREE_A, [fill], cfg_scale=wl.cfg_scale, q_noise=0.3)
    ora = H.run_tree_oracle(case)
    for deterministic, chain_kernels in ((False, False), (True, False), (False, True)):
        run = H.GpuRunner(wl.shape, case["w"], 2, 9, deterministic=deterministic, chain_kernels=chain_kernels)
        gpu = H.run_tree_gpu(run, case)
        assert (gpu["launches"] < 40) == chain_kernels
        _check_tree(case, gpu, ora)
        print("configs[1] tree: accept path", gpu["accept_path"][0][:gpu["accept_len"][0]], "oracle", ora["accept_path"])
        run.close()


@pytest.mark.parametrize("fill", [1, 583])
def test_config1_full_shape_cache_edges(fill):
    """Full depth with an almost empty cache (one 128-key chunk, 40 attention items) and with a
    cache that the block fills exactly (five chunks, 200 items: two per CTA for a third of them)."""
    wl = CONFIGS[1]
    assert fill + 9 <= wl.shape.s_max
    case = H.build_case(wl.shape, wl.seed + fill, 1, 2, 1, 8, [fill], cfg_scale=wl.cfg_scale, q_noise=0.3)
    ora = H.run_oracle(case)
    for deterministic, chain_kernels in ((False, False), (True, False), (True, True), (False, True)):
        run = H.GpuRunner(wl.shape, case["w"], 2, 9, deterministic=deterministic, chain_kernels=chain_kernels)
        gpu = run.verify(case)
        assert (gpu["launches"] < 40) == chain_kernels
        _check_end_to_end(case, gpu, ora)
        run.close()


def test_config2_full_depth_batch16_relaxed():
    """configs[2] as the benchmark runs it: 36 layers, 16 images x guidance = 288 block rows through
    the per-projection tensor-core kernels (two token passes, split-K sums, element-wise kernels),
    fills drawn per image, relaxed acceptance over 64 latent neighbours."""
    wl = CONFIGS[2]
    ms = wl.shape
    fills = [1, 575, 130, 288, 17, 400, 333, 128, 127, 129, 256, 500, 64, 9, 511, 200]
    case = H.build_case_independent(ms, wl.seed, 16, 2, 1, 8, fills, cfg_scale=wl.cfg_scale, mode=MODE_RELAXED,
                                    nbr_k=64, logit_std=1.0)
    ora = H.run_oracle(case)
    for deterministic in (False, True):    # arrival-order reductions (what the benchmark times), cluster reduction
        run = H.GpuRunner(ms, case["w"], 32, 9, max_nbr_k=64, deterministic=deterministic)
        gpu = run.verify(case)
        assert gpu["launches"] > 100       # one kernel per projection
        _check_end_to_end(case, gpu, ora)
        print("configs[2] full depth, fixed-order sums" if deterministic else "configs[2] full depth, arrival-order sums",
              "accept_len", gpu["accept_len"].tolist(), "oracle", ora["accept_len"].tolist())
        run.close()


def test_config3_full_depth_7b():
    """configs[3] as the benchmark runs it: 32 layers of the 7B shape (d = 4096, 32 heads of 128, MLP
    11008), 8192 codes inside a 65536-row head, fill 1500, one image with guidance, both whole-chain
    kernels.  The 13 GB of weights are drawn on the GPU (seeded) and copied to the host for the
    oracle, which widens one matrix at a time; the caches are cut to the slots the step can touch."""
    import torch
    wl = CONFIGS[3]
    ms = wl.shape
    fill, t_len = 1500, 9
    g = torch.Generator(device="cuda").manual_seed(wl.seed + 7)
    shp = gen.weight_shapes(ms)

    def draw(name):
        if name.startswith("norm"):
            return (1.0 + 0.1 * torch.randn(shp[name], generator=g, device="cuda")).to(torch.bfloat16)
        return (0.02 * torch.randn(shp[name], generator=g, device="cuda")).to(torch.bfloat16)

    def bits(t):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    wd = {n: draw(n) for n in ("tok_emb", "norm_f", "w_lm")}
    wd["layers"] = [{n: draw(n) for n in gen.LAYER_TENSORS} for _ in range(ms.n_layers)]
    w = {n: bits(wd[n]) for n in ("tok_emb", "norm_f", "w_lm")}
    w["layers"] = {l: {n: bits(t) for n, t in wd["layers"][l].items()} for l in range(ms.n_layers)}
    kv = [torch.randn((ms.n_layers, 2, ms.n_heads, ms.s_max, ms.head_dim), generator=g, device="cuda").to(torch.bfloat16)
          for _ in range(2)]
    case = H.build_case_independent(ms, wl.seed, 1, 2, 1, 8, [fill], cfg_scale=wl.cfg_scale, logit_std=1.0, w=w,
                                    kv=(bits(kv[0]), bits(kv[1])))
    import os
    from paper_2511_13587_b200 import binding as vb
    # the oracle only touches cache slots below fill + T: hand it that part (float64 copies of the
    # whole 2384-slot caches would be 10 GB)
    small = dict(case, kv_k=case["kv_k"][:, :, :, :fill + t_len], kv_v=case["kv_v"][:, :, :, :fill + t_len])
    ora = H.run_oracle(small)
    # per-projection kernels with arrival-order and with fixed-order sums (what the benchmark times), then
    # the two whole-chain kernels behind the library's debug switch
    for deterministic, chain_kernels in ((False, False), (True, False), (False, True), (True, True)):
        run = H.GpuRunner.__new__(H.GpuRunner)       # weights are on the device already: no second copy
        run.vb, run.ms, run.wd = vb, ms, wd
        if chain_kernels:
            os.environ["VVS_DEBUG_CHAIN_KERNELS"] = "1"
        try:
            run.ctx = vb.vvs_create(vb.make_desc(ms, 2, t_len, 1, deterministic))
        finally:
            os.environ.pop("VVS_DEBUG_CHAIN_KERNELS", None)
        vb.vvs_bind_weights(run.ctx, wd)
        gpu = run.verify(case, kv_keep=fill + t_len)
        assert (gpu["launches"] < 40) == chain_kernels
        assert gpu["kv_rest_untouched"]        # slots beyond the block, compared on the device
        _check_end_to_end(small, gpu, ora)
        print("configs[3] full depth", (deterministic, chain_kernels), "accept_len", gpu["accept_len"].tolist(),
              "oracle", ora["accept_len"].tolist())
        run.close()
