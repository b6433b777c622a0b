"""Parity of vvs_skip_decide (dynamic verification skipping, paper Sec. 4.4, Eq. 2, Alg. 1) with the
oracle, through the C ABI: decisions bit-exact (a similarity within 1e-9 of the threshold is
excluded and counted), similarities within float32 rounding of the oracle's float64 value."""
import numpy as np
import pytest
import torch

from oracle import vvs_oracle as O
from paper_2511_13587_b200 import binding as vb
from vvs_synth import gen
from vvs_synth.configs import ModelShape

pytestmark = pytest.mark.gpu


def _ctx():
    return vb.vvs_create(vb.make_desc(ModelShape("skip", 0, 64, 0, 0, 0, 128), 1, 1, 1))


def _case(seed, b, n, l, v, dim, similar):
    """Candidate paths of a draft tree: every image has a stem shared by its paths up to a random
    depth (trees branch late when the drafter is confident); `similar` in [0, 1] biases the tokens
    after the branch point towards latent-space neighbours of the stem's token."""
    rng = gen.rng_for(seed, f"skip.{b}.{n}.{l}.{v}")
    cb = rng.standard_normal((v, dim)).astype(np.float32)
    paths = rng.integers(0, v, size=(b, n, l)).astype(np.int32)
    for i in range(b):
        branch = rng.integers(0, l + 1)
        paths[i, :, :branch] = paths[i, 0, :branch]
        if similar > 0:
            near = np.argsort(((cb[:, None, :] - cb[None, paths[i, 0], :]) ** 2).sum(-1), axis=0)[:4]   # [4, l]
            pick = rng.random((n, l)) < similar
            cand = near[rng.integers(0, 4, size=(n, l)), np.arange(l)[None, :]]
            paths[i] = np.where(pick & (np.arange(l)[None, :] >= branch), cand, paths[i])
    plen = rng.integers(max(1, l - 2), l + 1, size=(b, n)).astype(np.int32)
    last = (rng.random(b) < 0.8).astype(np.uint8)
    return cb, paths, plen, last


@pytest.mark.parametrize("b,n,l,v,dim,similar,alpha,thr,stride", [
    (1, 2, 1, 64, 8, 0.0, 0.5, 0.5, 1),
    (16, 12, 5, 16384, 8, 0.7, 0.8, 0.65, 2),      # LlamaGen-like: 8-dim latent codebook of 16384 codes
    (7, 33, 6, 8192, 256, 0.5, 0.6, 0.3, 2),
    (5, 60, 16, 1024, 32, 0.9, 1.0, 0.8, 1),        # the limits: 60 kept paths, depth 16
    (9, 9, 4, 300, 7, 0.3, 0.9, 0.0, 3),
])
def test_skip_decision_matches_oracle(b, n, l, v, dim, similar, alpha, thr, stride):
    cb, paths, plen, last = _case(17, b, n, l, v, dim, similar)
    ctx = _ctx()
    dec = torch.full((b,), 9, dtype=torch.uint8, device="cuda")
    sim = torch.full((b,), -7.0, dtype=torch.float32, device="cuda")
    for use_len, use_last in ((True, True), (False, False)):
        vb.vvs_skip_decide(ctx, torch.from_numpy(paths).cuda(), torch.from_numpy(plen).cuda() if use_len else None,
                           torch.from_numpy(cb).cuda(), torch.from_numpy(last).cuda() if use_last else None,
                           stride, alpha, thr, dec, sim)
        assert vb.vvs_device_status(ctx) == 0
        near = 0
        for i in range(b):
            want_d, want_s = O.skip_decision(paths[i], plen[i] if use_len else np.full(n, l), cb, alpha, thr,
                                             bool(last[i]) if use_last else True, stride)
            assert abs(float(sim[i]) - want_s) <= 2e-7 * max(1.0, abs(want_s)), (i, float(sim[i]), want_s)
            if abs(want_s - thr) < 1e-9 and (not use_last or last[i]):
                near += 1
                continue
            assert int(dec[i]) == int(want_d), (i, int(dec[i]), want_d, want_s)
        assert near <= 1
    vb.vvs_destroy(ctx)


def test_skip_decision_edge_cases_and_errors():
    ctx = _ctx()
    cb = torch.eye(8, device="cuda")
    dec = torch.zeros(2, dtype=torch.uint8, device="cuda")
    sim = torch.zeros(2, dtype=torch.float32, device="cuda")
    # image 0: identical kept paths (S = 1, skip); image 1: an out-of-range token is reported, not read
    paths = torch.tensor([[[1, 2], [5, 5], [1, 2]], [[1, 2], [0, 0], [99, 2]]], dtype=torch.int32, device="cuda")
    vb.vvs_skip_decide(ctx, paths, None, cb, None, 2, 0.5, 0.9, dec, sim)
    assert vb.vvs_device_status(ctx) == 1                                  # VVS_DEV_BAD_TOKEN
    assert dec.tolist() == [1, 0] and abs(float(sim[0]) - 1.0) < 1e-7
    assert abs(float(sim[1]) - (0.5 / 1.5)) < 1e-6                         # level 0 counts 0, level 1 is identical
    # a single kept path is similar to itself; beyond the limits the call is refused
    vb.vvs_skip_decide(ctx, paths[:, :1].contiguous(), None, cb, None, 2, 0.5, 0.9, dec, sim)
    assert dec.tolist() == [1, 1]
    big = torch.zeros((1, 200, 2), dtype=torch.int32, device="cuda")
    with pytest.raises(vb.VvsError):
        vb.vvs_skip_decide(ctx, big, None, cb, None, 2, 0.5, 0.9, dec, sim)
    vb.vvs_destroy(ctx)


def test_unverified_selection_is_bit_exact_with_oracle():
    """Sec. 4.2 / Eq. 3 through the C ABI: drawn path, gamma and kept tokens equal the oracle's."""
    ctx = _ctx()
    rng = gen.rng_for(23, "select")
    for b, n, l in ((1, 1, 1), (16, 24, 5), (9, 61, 16), (3, 7, 4)):
        paths = rng.integers(0, 16384, size=(b, n, l)).astype(np.int32)
        plen = rng.integers(0, l + 1, size=(b, n)).astype(np.int32)
        u = rng.random(b).astype(np.float32).clip(1e-6, 1 - 1e-6)
        u[0] = np.float32(1 - 1e-6)
        op = torch.full((b,), -9, dtype=torch.int32, device="cuda")
        og = torch.full((b,), -9, dtype=torch.int32, device="cuda")
        ot = torch.full((b, l), -9, dtype=torch.int32, device="cuda")
        for use_len in (True, False):
            vb.vvs_select_unverified(ctx, torch.from_numpy(paths).cuda(), torch.from_numpy(plen).cuda() if use_len else None,
                                     torch.from_numpy(u).cuda(), op, og, ot)
            assert vb.vvs_device_status(ctx) == 0
            for i in range(b):
                # both sides take floor(u * N) on the float32 product
                idx, g, toks = O.select_unverified(paths[i], plen[i] if use_len else np.full(n, l), np.float32(u[i]) * np.float32(n) / n)
                assert int(op[i]) == idx and int(og[i]) == g
                assert ot[i].tolist() == list(toks) + [-1] * (l - g)
    vb.vvs_destroy(ctx)
