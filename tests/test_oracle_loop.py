"""Pins of the oracle's decoding loop (Supp. Alg. 2) and of the fixed-interval schedule (Sec. 4.4).

What the paper fixes and these tests check on the CPU: the fixed interval i skips exactly every i-th
step; no two verification-free steps follow each other; a step after a skip verifies the drafts
behind the unverified tokens in ONE pass and thereby restores their K/V entries and refreshes their
features (Sec. 4.1) -- so after any schedule the cache and the cached features must equal those of a
plain pass of the target over the tokens that were finally committed; never skipping is plain
speculative decoding (every iteration one verify call)."""
import numpy as np

from oracle import vvs_oracle as O
from vvs_synth import gen, philox
from vvs_synth.configs import TINY
from vvs_synth.drafter import SyntheticDrafter


def test_fixed_interval_schedule_pattern():
    for i in (2, 3, 4):
        s = [O.skip_schedule_fixed(t, i) for t in range(24)]
        assert sum(s) == 24 // i
        assert all(s[t] == (t % i == i - 1) for t in range(24))
        assert not any(a and b for a, b in zip(s, s[1:]))          # never two skips in a row
    assert not any(O.skip_schedule_fixed(t, 1) for t in range(8))  # "every step" would break that rule: never
    assert not any(O.skip_schedule_fixed(t, 0) for t in range(8))


def _loop(schedule, seed=77, n_tokens=40, k=4, n_cfg=1, ragged=False):
    ms = TINY
    w = gen.make_weights(ms, seed)
    kv_k, kv_v = gen.make_kv_cache(ms, seed, n_cfg)
    dr = SyntheticDrafter(seed, ms.vocab, k, n_paths=6, depth=4, ragged=ragged)
    codebook = gen.make_codebook(seed, ms.vocab, 8)
    res = O.decode_loop(ms, w, kv_k, kv_v, dr.first_token(), dr.propose, lambda it: philox.verify_uniforms(seed, it, 1, k),
                        n_tokens, k, n_cfg, 1.0 if n_cfg == 1 else 2.0, schedule, codebook=codebook, fill0=3)
    return ms, w, kv_k, kv_v, dr, res


def _check_against_plain_pass(ms, w, kv_k, kv_v, dr, res, n_cfg=1, fill0=3):
    """K/V of every committed position and the cached features equal a single teacher-forced pass of
    the target over the committed tokens."""
    committed = [ms.vocab_offset + dr.first_token()] + res["tokens"]
    n = res["fill"] - fill0                       # tokens whose K/V is in the cache
    assert 0 < n <= len(committed)
    assert committed[n] == res["last_token"] if not res["pending"] else True
    for r in range(n_cfg):
        kc, vc = O.widen(kv_k[:, r]), O.widen(kv_v[:, r])
        h = O.target_forward(ms, w, np.array(committed[:n]), kc, vc, fill0)
        np.testing.assert_allclose(res["kc"][r][:, :, :res["fill"]], kc[:, :, :res["fill"]], rtol=0, atol=1e-9)
        np.testing.assert_allclose(res["vc"][r][:, :, :res["fill"]], vc[:, :, :res["fill"]], rtol=0, atol=1e-9)
        fc = res["fcache"]
        newest = int(fc.newest[r])
        assert newest == res["fill"] - 1
        for pos in range(max(fill0, newest - fc.cap + 1), newest + 1):
            assert fc.fpos[r, pos % fc.cap] == pos
            np.testing.assert_allclose(fc.feat[r, pos % fc.cap], h[pos - fill0], rtol=0, atol=1e-9)


def test_never_skipping_is_plain_speculative_decoding():
    ms, w, kv_k, kv_v, dr, res = _loop(("never",))
    assert all(e[0] == "verify" and e[1] == 1 for e in res["log"])
    assert len(res["tokens"]) == sum(e[2] + 1 for e in res["log"]) >= 40
    _check_against_plain_pass(ms, w, kv_k, kv_v, dr, res)


def test_fixed_interval_loop_restores_cache_and_features():
    for interval in (2, 3):
        ms, w, kv_k, kv_v, dr, res = _loop(("fixed", interval), ragged=(interval == 3))
        kinds = [e[0] for e in res["log"]]
        assert kinds == ["skip" if t % interval == interval - 1 else "verify" for t in range(len(kinds))]
        pending = 0
        for e in res["log"]:
            if e[0] == "skip":
                assert 0 <= e[2] <= 4                    # truncation: at most the path's own length (Eq. 3)
                pending = e[2]
            else:
                assert e[1] == 1 + pending               # post verification: unverified tokens ride along
                pending = 0
        _check_against_plain_pass(ms, w, kv_k, kv_v, dr, res)


def test_dynamic_loop_with_guidance_never_skips_twice():
    ms, w, kv_k, kv_v, dr, res = _loop(("dynamic", 0.2, 0.8, 2), n_cfg=2, n_tokens=30)
    kinds = [e[0] for e in res["log"]]
    assert "skip" in kinds and "verify" in kinds
    assert not any(a == "skip" and b == "skip" for a, b in zip(kinds, kinds[1:]))
    assert kinds[0] == "verify"                          # V_last starts False: the first step is verified
    _check_against_plain_pass(ms, w, kv_k, kv_v, dr, res, n_cfg=2)
