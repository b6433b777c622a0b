"""Parity of vvs_verify (through the C ABI) with the fp64 oracle on seeded inputs.

Two regimes.  Decision replay: the oracle's decision stage re-run on the float32 target
probabilities the GPU emitted must reproduce accept_len / accept_mask / next_token bit for bit
(decisions within 1e-4 of their threshold excluded and counted).  End to end: probabilities
within 2e-3 absolute (bf16) / 1e-5 (fp32), features within 1e-2 relative (bf16) / 1e-4 (fp32),
appended K/V within the same relative bound, integer outputs equal unless the uniform lies
between the oracle's acceptance ratio and the ratio of the GPU's own probabilities (counted and
printed per call)."""
from dataclasses import replace

import numpy as np
import pytest

import helpers as H
from vvs_synth.configs import (B7_SMALL, CONFIGS, DTYPE_BF16, MODE_RELAXED, TINY, XL_SMALL)

pytestmark = pytest.mark.gpu


def _tols(ms):
    """Probabilities: 2e-3 absolute at every depth.  Features (and what follows from them in
    relative terms): 1e-2 of the row norm up to 3 layers; every sublayer injects fresh bf16
    rounding of its GEMM inputs, which adds up like a random walk over depth, so the bound grows
    with sqrt(layers / 3).  At 36 layers the three bf16 implementations in this library (the
    whole-chain kernel, the per-projection tensor-core kernels, the plain generic kernels) measure
    2.0-3.1 % against the fp64 oracle and 3-4 % against one another on the random-init network."""
    if ms.dtype == DTYPE_BF16:
        depth = max(1.0, ms.n_layers / 3.0) ** 0.5
        h_rel = 1e-2 * depth
        # A feature error of h_rel of the row norm (~sqrt(d)) becomes a guided-logit error of
        # h_rel * sqrt(d) * 0.02 (weight std) * sqrt(2^2 + 1^2) (guidance 2.0); the largest of the
        # ~1e5 logits of a call sits near 5 sigma, and a logit error is a relative probability error.
        p_rel = max(6e-2 * depth, h_rel * ms.d_model ** 0.5 * 0.02 * 5.0 ** 0.5 * 5.0)
        return dict(p_abs=2e-3, p_rel=p_rel, h_rel=h_rel)
    return dict(p_abs=1e-5, p_rel=2e-4, h_rel=1e-4)


def _check_end_to_end(case, gpu, ora):
    ms = case["ms"]
    tol = _tols(ms)
    assert gpu["status"] == 0
    assert gpu["launches"] > 0
    # features: relative error of every row; the bound holds for the root mean square over the rows
    # of the call; the worst row is rounding noise further out in the tail: a quarter above the bound
    # for up to 32 rows, half above for up to 288
    h_err = H.rel_err_per_row(gpu["hidden"], ora["hidden"])
    assert np.sqrt(np.mean(h_err ** 2)) < tol["h_rel"]
    assert h_err.max() < (1.5 if h_err.size > 32 else 1.25) * tol["h_rel"]
    dp = np.abs(gpu["target_probs"] - ora["target_probs"])
    # 2e-3 absolute, except where a single probability is so large (the 7B-width head has logits
    # of std > 1) that its relative bound allows more
    assert (dp < np.maximum(tol["p_abs"], tol["p_rel"] * ora["target_probs"])).all()
    # guided-logit error of every probability that is not negligible (at least a tenth of the uniform
    # level 1 / V; the far tail of ~1e5 entries per call reaches any fixed sigma), measured where it is
    # exact, as |log(p / p_oracle)|, against the 5-sigma logit error of a row whose feature error is at
    # the worst-row allowance of the feature check above
    notable = ora["target_probs"] >= 0.1 / ms.vocab
    worst_row = 1.5 if h_err.size > 32 else 1.25
    with np.errstate(divide="ignore"):
        log_err = np.abs(np.log(gpu["target_probs"][notable] / ora["target_probs"][notable]))
    print(f"largest guided-logit error {log_err.max():.3f} (bound {worst_row * tol['p_rel']:.3f}); "
          f"feature error rms {np.sqrt(np.mean(h_err ** 2)):.4f}, worst row {h_err.max():.4f} (bound {tol['h_rel']:.4f})")
    assert log_err.max() < worst_row * tol["p_rel"]
    np.testing.assert_allclose(gpu["target_probs"].sum(-1), 1.0, atol=1e-4)
    # appended K/V are compared per (layer, head, slot) row of head_dim elements: in a deep network
    # the error of such a short row scatters around the feature error, hence twice the bound there
    H.check_new_cache_rows(case, gpu, ora, tol["h_rel"] * (2.0 if ms.n_layers > 3 else 1.0))
    # integer outputs against the oracle's own pipeline.  A differing accepted length is explained
    # only if, at the first differing draft, the uniform lies between the oracle's acceptance ratio and
    # the ratio the GPU's own probabilities give (both recomputed by the oracle's decision stage): the
    # float error of THAT ratio, not a blanket bound.  Explained ones are counted and reported.
    k = case["n_draft_max"]
    rep = H.replay_decisions(case, gpu["target_probs"])
    real, near = 0, 0
    for b in range(case["n_images"]):
        if gpu["accept_len"][b] != ora["accept_len"][b]:
            n = min(gpu["accept_len"][b], ora["accept_len"][b])
            r_ora, r_gpu = min(1.0, ora["ratios"][b][n]), min(1.0, rep["ratios"][b][n])
            if ora["margins"][b][n] <= abs(r_gpu - r_ora) + 1e-12:
                near += 1
            else:
                real += 1
    print(f"end-to-end integer check: {case['n_images']} images, {near} near-threshold accept_len "
          f"difference(s) explained by the ratio's float error, {real} unexplained; "
          f"feature error {H.rel_err_rows(gpu['hidden'], ora['hidden']):.4f} of the row norm "
          f"(bound {tol['h_rel']:.4f}), max |dp| {dp.max():.2e}")
    assert real == 0
    assert near <= max(1, case["n_images"] // 4)
    np.testing.assert_array_equal(
        gpu["new_len"], case["cache_len"] + case["n_forced"] +
        gpu["accept_len"][np.arange(len(gpu["new_len"])) % case["n_images"]])
    return H.check_replay(case, gpu)


def test_config0_tiny_fp32_strict():
    """The tiny float32 workload: 2 layers, d = 256, V = 1024, batch 1, no guidance, fill 64, K = 4."""
    w = CONFIGS[0]
    for trial in range(3):
        case = H.build_case(w.shape, w.seed + trial, 1, 1, 1, 4, [64], cfg_scale=1.0,
                            q_noise=0.7 if trial else 2.0, call_id=trial)
        run = H.GpuRunner(w.shape, case["w"], 1, 5)
        gpu = run.verify(case)
        ora = H.run_oracle(case)
        assert _check_end_to_end(case, gpu, ora) == 0
        np.testing.assert_array_equal(gpu["accept_len"], ora["accept_len"])
        np.testing.assert_array_equal(gpu["next_token"], ora["next_token"])
        run.close()


@pytest.mark.parametrize("chain_kernels", [False, True])
@pytest.mark.parametrize("deterministic", [True, False])
@pytest.mark.parametrize("n_images,fills", [(1, [288]), (3, [1, 575, 130])])
def test_xl_shape_small_bf16_cfg(n_images, fills, deterministic, chain_kernels):
    """LlamaGen-XL structure (2-D grid rope, 1 prefix token, guidance 2.0, K = 8) at reduced
    width/depth; an extra unused cache row must stay untouched.  18 and 54 tokens, fixed-order and
    arrival-order sums, per-projection kernels and the whole-chain / fused-epilogue kernels."""
    ms = XL_SMALL
    case = H.build_case(ms, 11 + n_images, n_images, 2, 1, 8, fills, kv_rows=2 * n_images + 1)
    run = H.GpuRunner(ms, case["w"], 2 * n_images, 9, deterministic=deterministic, chain_kernels=chain_kernels)
    gpu = run.verify(case)
    assert (gpu["launches"] < 20) == (chain_kernels and n_images == 1)    # one persistent kernel for all layers
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    # outputs not requested are not needed for the decisions
    gpu2 = run.verify(case, want_probs=False, want_hidden=False)
    if deterministic:
        np.testing.assert_array_equal(gpu2["accept_len"], gpu["accept_len"])
        np.testing.assert_array_equal(gpu2["next_token"], gpu["next_token"])
    else:
        # two arrival-order calls differ in the last bits: a decision may flip only where the uniform
        # sits within that distance of its ratio
        m = H.replay_decisions(case, gpu["target_probs"])["margins"][:, :8]
        clear = (m > 1e-2).all(axis=1)
        np.testing.assert_array_equal(gpu2["accept_len"][clear], gpu["accept_len"][clear])
    run.close()


@pytest.mark.parametrize("n_images,want_probs", [(4, True), (4, False), (12, False)])
def test_relaxed_acceptance_adjusted_residual_bf16(n_images, want_probs):
    """The adjusted-residual flag through vvs_verify on all three decision routes: probabilities
    written out, guided logits in scratch (at most 64 decision rows), and the second LM-head pass
    that recomputes the sampled row (more than 64 decision rows)."""
    ms = XL_SMALL
    fills = [10, 200, 333, 574, 55, 123, 400, 9, 77, 501, 268, 31][:n_images]
    case = H.build_case_independent(ms, 29, n_images, 2, 1, 8, fills, mode=MODE_RELAXED, nbr_k=16,
                                    logit_std=2.5)
    case["adjusted_residual"] = True
    run = H.GpuRunner(ms, case["w"], 2 * n_images, 9, max_nbr_k=16)
    gpu = run.verify(case, want_probs=True)
    if not want_probs:                                  # the route under test emits no probabilities:
        gpu2 = run.verify(case, want_probs=False)       # its integers must equal the checked route's
        m = H.replay_decisions(case, gpu["target_probs"])["margins"]   # (two runs differ in the last bits)
        clear = (m[:, :8] > 1e-2).all(axis=1)
        np.testing.assert_array_equal(gpu2["accept_len"][clear], gpu["accept_len"][clear])
        # the sampled code sits in a CDF bin about 1/V wide; run-to-run differences of the rows
        # may move a sample point across an edge now and then
        assert clear.sum() >= n_images // 2
        assert (gpu2["next_token"][clear] != gpu["next_token"][clear]).sum() <= max(1, n_images // 4)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    plain = run.verify(dict(case, adjusted_residual=False))
    m = H.replay_decisions(case, gpu["target_probs"])["margins"]
    clear = (m[:, :8] > 1e-2).all(axis=1)
    np.testing.assert_array_equal(plain["accept_len"][clear], gpu["accept_len"][clear])
    rejected = clear & (gpu["accept_len"] < 8)
    assert rejected.any() and (plain["next_token"][rejected] != gpu["next_token"][rejected]).any()
    run.close()


@pytest.mark.parametrize("delta", [float("inf"), 0.1, 0.0])
def test_relaxed_acceptance_bf16(delta):
    ms = XL_SMALL
    case = H.build_case(ms, 23, 4, 2, 1, 8, [10, 200, 333, 574], mode=MODE_RELAXED, nbr_k=16,
                        delta=delta, q_noise=1.5)
    run = H.GpuRunner(ms, case["w"], 8, 9, max_nbr_k=16)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    if delta == 0.0:                                    # relaxed with delta = 0 is strict
        strict = dict(case, mode=0, row_ptr=None, col=None)
        gpu_s = run.verify(strict)
        np.testing.assert_array_equal(gpu_s["accept_len"], gpu["accept_len"])
        np.testing.assert_array_equal(gpu_s["next_token"], gpu["next_token"])
    run.close()


@pytest.mark.parametrize("chain_kernels", [False, True])
@pytest.mark.parametrize("deterministic", [True, False])
def test_7b_shape_small_bf16(deterministic, chain_kernels):
    """7B structure: head_dim 128, 1-D rope, codebook inside a larger vocabulary."""
    ms = B7_SMALL
    case = H.build_case(ms, 31, 1, 2, 1, 8, [300])
    run = H.GpuRunner(ms, case["w"], 2, 9, deterministic=deterministic, chain_kernels=chain_kernels)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    assert ((gpu["next_token"] >= ms.vocab_offset) & (gpu["next_token"] < ms.vocab_offset + ms.vocab)).all()
    run.close()


@pytest.mark.parametrize("ms,n_images,n_forced,k,fills",
                         [(B7_SMALL, 3, 1, 8, [300, 7, 120]),          # head_dim 128, 54 block tokens
                          (XL_SMALL, 2, 3, 14, [100, 240]),            # 17 rows per sequence, 68 tokens
                          (B7_SMALL, 2, 2, 17, [377, 128])])           # head_dim 128, 19 rows, 76 tokens
def test_per_projection_kernels_head_dims_and_long_blocks(ms, n_images, n_forced, k, fills):
    """More than 32 block tokens: the per-projection tensor-core kernels, with both head
    dimensions and with more than 16 query rows per sequence; arrival-order sums (fused projection
    epilogues up to 64 tokens) and fixed-order sums (cluster reduction)."""
    case = H.build_case(ms, 61 + k, n_images, 2, n_forced, k, fills, q_noise=0.8)
    ora = H.run_oracle(case)
    for deterministic in (False, True):
        run = H.GpuRunner(ms, case["w"], 2 * n_images, n_forced + k, deterministic=deterministic)
        gpu = run.verify(case)
        assert gpu["launches"] > 20
        _check_end_to_end(case, gpu, ora)
        run.close()


@pytest.mark.parametrize("ms,n_forced,k,fills",
                         [(XL_SMALL, 1, 8, [0, 63, 64, 65, 128, 583]),    # empty cache, 64-key block edges, block fills the cache
                          (XL_SMALL, 2, 30, [129, 500]),                  # 32 rows per sequence: two full m-tiles
                          (B7_SMALL, 1, 8, [0, 64, 191, 391])])           # head_dim 128; 391 + 9 rows = capacity
def test_row_batched_attention_edges(ms, n_forced, k, fills):
    """More than 64 block tokens: rotation, cache append and attention run per (sequence, head) in one
    kernel that streams the cached keys in 64-key blocks."""
    n_images = len(fills)
    case = H.build_case_independent(ms, 83 + k, n_images, 2, n_forced, k, fills, logit_std=0.5)
    assert n_images * 2 * (n_forced + k) > 64
    ora = H.run_oracle(case)
    for deterministic in (False, True):
        run = H.GpuRunner(ms, case["w"], 2 * n_images, n_forced + k, deterministic=deterministic)
        gpu = run.verify(case)
        _check_end_to_end(case, gpu, ora)
        run.close()


@pytest.mark.parametrize("deterministic", [True, False])
def test_small_call_on_a_shape_the_streaming_kernel_does_not_take(deterministic):
    """d_ff = 880 is not a multiple of 32 or 128: ragged last weight tiles in the per-projection kernels,
    cluster reductions at 18 tokens in the fixed-order context (which must repeat bit for bit)."""
    ms = replace(XL_SMALL, name="llamagen_xl_small_ff880", d_ff=880)
    case = H.build_case(ms, 97, 1, 2, 1, 8, [211])
    run = H.GpuRunner(ms, case["w"], 2, 9, deterministic=deterministic)
    gpu = run.verify(case)
    _check_end_to_end(case, gpu, H.run_oracle(case))
    if deterministic:
        assert gpu["launches"] > 20
        again = run.verify(case)
        for key in ("accept_len", "next_token", "target_probs", "hidden", "kv_k", "kv_v"):
            np.testing.assert_array_equal(gpu[key], again[key], err_msg=key)
    run.close()


@pytest.mark.parametrize("chain_kernels", [False, True])
@pytest.mark.parametrize("deterministic", [True, False])
def test_ragged_drafts_forced_prefix_and_cache_edges(deterministic, chain_kernels):
    """n_draft below K (including 0), two forced rows, an empty cache and a cache that the block
    fills to capacity."""
    ms = replace(XL_SMALL, s_max=64)
    case = H.build_case(ms, 41, 4, 2, 2, 6, [0, 64 - 8, 5, 17], n_draft=[6, 3, 0, 1], q_noise=0.5)
    run = H.GpuRunner(ms, case["w"], 8, 8, deterministic=deterministic, chain_kernels=chain_kernels)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    assert (gpu["accept_len"] <= case["n_draft"]).all()
    assert gpu["accept_len"][2] == 0
    run.close()


def test_fp32_with_guidance_and_temperature():
    ms = replace(TINY, vocab=1000, lm_rows=1000, tok_rows=1000)
    case = H.build_case(ms, 51, 2, 2, 1, 4, [64, 9], cfg_scale=1.5, temperature=0.8, q_noise=0.6)
    run = H.GpuRunner(ms, case["w"], 4, 5)
    gpu = run.verify(case)
    ora = H.run_oracle(case)
    _check_end_to_end(case, gpu, ora)
    run.close()


def test_device_side_checks_report_instead_of_faulting():
    import torch
    ms = TINY
    case = H.build_case(ms, 61, 1, 1, 1, 4, [64])
    run = H.GpuRunner(ms, case["w"], 1, 5)
    vb = run.vb
    bad = dict(case, block=case["block"].copy())
    bad["block"][0, 0] = ms.tok_rows + 5                 # forced token outside the embedding
    assert run.verify(bad)["status"] & vb.VVS_DEV_BAD_TOKEN
    over = dict(case, cache_len=np.array([ms.s_max - 2], np.int32))
    res = run.verify(over)                               # block would overflow the cache
    assert res["status"] & vb.VVS_DEV_CACHE_OVERFLOW
    np.testing.assert_array_equal(res["kv_k"], H.O.widen(case["kv_k"]))   # nothing written
    ok = run.verify(case)
    assert ok["status"] == 0                             # context still usable
    # host-side capacity check
    a = dict(n_images=1, n_cfg=1, n_forced=1, n_draft_max=4, block=H.to_dev(case["block"]),
             kv_k=H.to_dev(case["kv_k"]), kv_v=H.to_dev(case["kv_v"]), kv_rows=1,
             cache_len=H.to_dev(over["cache_len"]), draft_probs=H.to_dev(case["draft_probs"]),
             uniforms=H.to_dev(case["uniforms"]),
             accept_len=torch.zeros(1, dtype=torch.int32, device="cuda"),
             next_token=torch.zeros(1, dtype=torch.int32, device="cuda"),
             new_len=torch.zeros(1, dtype=torch.int32, device="cuda"))
    host_len = over["cache_len"].copy()
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_verify(run.ctx, cache_len_host=host_len.ctypes.data, **a)
    assert e.value.status == -4
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_verify(run.ctx, **dict(a, n_draft_max=40))
    assert e.value.status == -2
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_verify(run.ctx, **dict(a, mode=1, nbr_k=4))
    assert e.value.status == -2                          # nbr_k above max_nbr_k
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_verify(run.ctx, **dict(a, temperature=0.0))
    assert e.value.status == -1
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_verify(run.ctx, **dict(a, draft_probs=H.to_dev(case["draft_probs"]).data_ptr() + 4))
    assert e.value.status == -3
    run.close()


def test_bounded_waits_give_up_and_leave_the_context_usable():
    """The failure path of the device-side waits, without hanging anything: a self-test kernel waits
    with a limit of a few hundred polls on barriers nobody arrives on; both wait helpers must return,
    VVS_DEV_TIMEOUT must show in the status word (reported once, then cleared), and a verify call on
    the same context must still work afterwards."""
    from paper_2511_13587_b200 import binding as vb
    ms = XL_SMALL
    case = H.build_case(ms, 5, 1, 2, 1, 8, [311])
    run = H.GpuRunner(ms, case["w"], 2, 9)
    assert vb.vvs_selftest_bounded_wait(run.ctx) == (1, 1)
    assert vb.vvs_device_status(run.ctx) & 8            # VVS_DEV_TIMEOUT
    with pytest.raises(vb.VvsError) as e:
        vb.vvs_selftest_bounded_wait(run.ctx)
        vb.vvs_device_status(run.ctx, raise_on_error=True)
    assert e.value.status == -7                          # VVS_ERR_DEVICE_TIMEOUT
    assert vb.vvs_device_status(run.ctx) == 0            # cleared by the read
    gpu = run.verify(case)
    assert gpu["status"] == 0
    H.check_replay(case, gpu)
    run.close()


def test_repeatable_across_calls():
    """Two calls on the same inputs.  A bf16 context created with deterministic = 1 (the default of
    the binding) takes every sum in a fixed order: all outputs and the appended K / V rows repeat bit
    for bit, with and without the probabilities being written out.  With deterministic = 0 split-K
    partial sums are added with float atomics, so the low bits (and, through bf16 rounding of
    activations, ~1e-2 of a probability) may move, but every decision must replay exactly on the
    probabilities of its own call.  The float32 context is bitwise repeatable."""
    ms = XL_SMALL
    case = H.build_case(ms, 71, 2, 2, 1, 8, [50, 400])
    for n_images, fills in ((1, [288]), (1, [50])):
        c1 = H.build_case(ms, 71 + fills[0], n_images, 2, 1, 8, fills)
        for chain_kernels in (False, True):
            run = H.GpuRunner(ms, c1["w"], 2 * n_images, 9, deterministic=True, chain_kernels=chain_kernels)
            a = run.verify(c1)
            b = run.verify(c1)
            assert (a["launches"] < 20) == chain_kernels     # the streaming whole-chain kernel / cluster reductions
            for key in ("accept_len", "next_token", "accept_mask", "new_len", "target_probs", "hidden", "kv_k", "kv_v"):
                np.testing.assert_array_equal(a[key], b[key], err_msg=key)
            c_ = run.verify(c1, want_probs=False)
            d_ = run.verify(c1, want_probs=False)
            for key in ("accept_len", "next_token", "new_len", "hidden"):
                np.testing.assert_array_equal(c_[key], d_[key], err_msg=key)
            np.testing.assert_array_equal(c_["accept_len"], a["accept_len"])
            run.close()
    # more than 32 block tokens in a fixed-order context: the K splits of every projection are a
    # cluster that adds its partial tiles in rank order (36, 72 and 288 tokens: one, one and two passes)
    for n_images, fills in ((2, [50, 400]), (4, [10, 200, 333, 574]), (16, list(range(5, 5 + 16 * 35, 35)))):
        c2 = H.build_case_independent(ms, 171 + n_images, n_images, 2, 1, 8, fills, logit_std=0.7)
        run = H.GpuRunner(ms, c2["w"], 2 * n_images, 9, deterministic=True)
        a = run.verify(c2)
        b = run.verify(c2)
        assert a["launches"] > 20
        for key in ("accept_len", "next_token", "accept_mask", "new_len", "target_probs", "hidden", "kv_k", "kv_v"):
            np.testing.assert_array_equal(a[key], b[key], err_msg=key)
        H.check_replay(c2, a)
        run.close()
    run = H.GpuRunner(ms, case["w"], 4, 9, deterministic=False)
    a = run.verify(case)
    b = run.verify(case)
    np.testing.assert_allclose(a["target_probs"], b["target_probs"], rtol=5e-2, atol=1e-7)
    assert H.rel_err_rows(a["hidden"], b["hidden"]) < 1e-2
    H.check_replay(case, a)
    H.check_replay(case, b)
    run.close()
    w = CONFIGS[0]
    case = H.build_case(w.shape, w.seed, 1, 1, 1, 4, [64], cfg_scale=1.0)
    run = H.GpuRunner(w.shape, case["w"], 1, 5)
    a = run.verify(case)
    b = run.verify(case)
    for key in ("accept_len", "next_token", "accept_mask", "new_len", "target_probs", "hidden"):
        np.testing.assert_array_equal(a[key], b[key])
    run.close()


def test_tensor_core_path_agrees_with_generic_kernels(monkeypatch):
    """The same bf16 step through the generic kernels (debug switch) and through the tensor-core
    GEMMs: both within tolerance of the oracle and of each other."""
    ms = XL_SMALL
    case = H.build_case(ms, 81, 2, 2, 1, 8, [7, 222])
    run = H.GpuRunner(ms, case["w"], 4, 9)
    fast = run.verify(case)
    run.close()
    monkeypatch.setenv("VVS_DEBUG_GENERIC", "1")
    run = H.GpuRunner(ms, case["w"], 4, 9)
    slow = run.verify(case)
    run.close()
    monkeypatch.delenv("VVS_DEBUG_GENERIC")
    assert slow["launches"] != fast["launches"]
    assert H.rel_err_rows(fast["hidden"], slow["hidden"]) < 1e-2
    np.testing.assert_allclose(fast["target_probs"], slow["target_probs"], rtol=6e-2, atol=1e-7)
    ora = H.run_oracle(case)
    _check_end_to_end(case, slow, ora)
    _check_end_to_end(case, fast, ora)
