"""The decoding loop (Supp. Alg. 2) of the package, a host-side driver over the C-ABI entry points,
against the oracle's loop.  On the float32 context the step is bitwise repeatable and its decisions
sit far from their thresholds, so the whole token sequence and the skip / verify log must agree with
the oracle; on the bf16 context the bookkeeping the algorithm fixes is checked on the device's own
outputs."""
import numpy as np
import pytest

import helpers as H
from oracle import vvs_oracle as O
from vvs_synth import gen, philox
from vvs_synth.configs import TINY, XL_SMALL
from vvs_synth.drafter import SyntheticDrafter

pytestmark = pytest.mark.gpu


def _gpu_loop(ms, seed, schedule, n_tokens, k, n_cfg, cfg_scale, fill0, n_paths, depth, ragged=False,
              deterministic=True):
    import torch
    from paper_2511_13587_b200 import binding as vb
    from paper_2511_13587_b200.loop import DecodeLoop
    w = gen.make_weights(ms, seed)
    kv_k, kv_v = gen.make_kv_cache(ms, seed, n_cfg)
    dr = SyntheticDrafter(seed, ms.vocab, k, n_paths=n_paths, depth=depth, ragged=ragged)
    codebook = gen.make_codebook(seed, ms.vocab, 8)
    ctx = vb.vvs_create(vb.make_desc(ms, n_cfg, 1 + 5 + k, 1, deterministic))
    wd = H.weights_to_dev(w)
    vb.vvs_bind_weights(ctx, wd)
    dk, dv = H.to_dev(kv_k), H.to_dev(kv_v)
    loop = DecodeLoop(ctx, ms, dk, dv, k, n_cfg, cfg_scale, n_paths, depth,
                      codebook=torch.from_numpy(codebook.astype(np.float32)).cuda())
    u_of = lambda it: philox.verify_uniforms(seed, it, 1, k)
    got = loop.run(dr.first_token(), dr.propose, u_of, n_tokens, schedule, fill0=fill0)
    status = vb.vvs_device_status(ctx)
    vb.vvs_destroy(ctx)
    want = O.decode_loop(ms, w, kv_k, kv_v, dr.first_token(), dr.propose, u_of, n_tokens, k, n_cfg, cfg_scale, schedule,
                         codebook=codebook, fill0=fill0)
    return got, want, status, (H.to_host(dk), H.to_host(dv))


@pytest.mark.parametrize("schedule,ragged", [(("never",), False), (("fixed", 2), False), (("fixed", 3), True),
                                             (("dynamic", 0.2, 0.8, 2), False)])
def test_loop_matches_oracle_token_for_token_fp32(schedule, ragged):
    ms = TINY
    got, want, status, (gk, gv) = _gpu_loop(ms, 77, schedule, 48, 4, 2, 1.5, 3, 6, 4, ragged)
    assert status == 0
    assert got["log"] == want["log"]
    assert got["tokens"] == want["tokens"]
    assert got["fill"] == want["fill"] and got["iterations"] == want["iterations"]
    assert got["last_token"] == want["last_token"] and got["pending"] == want["pending"]
    # the K/V the loop left behind (post verification restores the entries of unverified tokens)
    for r in range(2):
        np.testing.assert_allclose(gk[:, r, :, :got["fill"]], want["kc"][r][:, :, :got["fill"]], rtol=2e-4, atol=2e-5)
        np.testing.assert_allclose(gv[:, r, :, :got["fill"]], want["vc"][r][:, :, :got["fill"]], rtol=2e-4, atol=2e-5)
    if schedule[0] == "fixed":
        kinds = [e[0] for e in got["log"]]
        assert kinds == ["skip" if t % schedule[1] == schedule[1] - 1 else "verify" for t in range(len(kinds))]


@pytest.mark.parametrize("schedule", [("never",), ("fixed", 4), ("dynamic", 0.3, 0.8, 2)])
def test_loop_bookkeeping_bf16(schedule):
    """bf16 context (reduced LlamaGen-XL shape, guidance): what the algorithm fixes, on the device's
    own outputs; the skip / verify pattern does not depend on the target and must equal the oracle's."""
    ms = XL_SMALL
    got, want, status, _ = _gpu_loop(ms, 41, schedule, 100, 8, 2, 2.0, 1, 12, 5)
    assert status == 0
    assert [e[0] for e in got["log"]][:8] == [e[0] for e in want["log"]][:8]
    fill, tokens, prev_skip, pending = 1, 0, False, 0
    for entry in got["log"]:
        if entry[0] == "skip":
            assert not prev_skip                         # never two verification-free steps in a row (Sec. 4.1)
            gamma = entry[2]
            assert 0 <= gamma <= 5                       # Eq. 3 bound (paths of depth 5)
            pending, tokens, prev_skip = gamma, tokens + gamma, True
        else:
            _, f, n_acc, new_len = entry
            assert f == 1 + pending                      # post verification: the unverified tokens ride along
            assert 0 <= n_acc <= 8
            fill += f + n_acc
            assert new_len == fill                       # the device's fill level after the step
            pending, tokens, prev_skip = 0, tokens + n_acc + 1, False
    assert tokens == got["generated"] == len(got["tokens"]) >= 100 and fill == got["fill"]
    if schedule[0] != "never":
        assert got["skipped_steps"] > 0
