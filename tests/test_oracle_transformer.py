"""Pins of the oracle's target-model forward (Alg. 2 line 9; Sec. 2: candidates are scored
"in parallel" in one pass; Sec. 4.1: post verification restores the missing KV entries) against
library routines, textbook identities and incremental decoding.  CPU only."""
from dataclasses import replace

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import vvs_oracle as O
from vvs_synth import gen
from vvs_synth.configs import DTYPE_FP32, ROPE_1D, ROPE_2D_GRID, ROPE_NONE, ModelShape

MS = ModelShape("pin", 2, 48, 3, 16, 80, 64, s_max=40, rope_mode=ROPE_1D, dtype=DTYPE_FP32)


def test_library_special_cases():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 48))
    g = rng.standard_normal(48)
    tx = torch.from_numpy(x)
    np.testing.assert_allclose(O.rmsnorm(x, g, 1e-5),
                               F.rms_norm(tx, (48,), torch.from_numpy(g), 1e-5).numpy(), rtol=1e-12)
    np.testing.assert_allclose(O.silu(x), F.silu(tx).numpy(), rtol=1e-12)
    np.testing.assert_allclose(O.softmax(x), torch.softmax(tx, -1).numpy(), rtol=1e-12)
    assert np.allclose(O.softmax(x + 1000.0), O.softmax(x))            # shift invariance


def test_attention_reduces_to_library_sdpa():
    """Block-vs-cache attention = scaled-dot-product attention with the mask 'cache slots
    plus causal inside the block'; a one-row block is plain decode attention."""
    rng = np.random.default_rng(1)
    h, hd, s, fill, t_len = 3, 16, 40, 21, 6
    kc = rng.standard_normal((h, s, hd))
    vc = rng.standard_normal((h, s, hd))
    q = rng.standard_normal((t_len, h, hd))
    got = O.attention_block_vs_cache(q, kc, vc, fill)
    n = fill + t_len
    mask = torch.zeros(t_len, n, dtype=torch.bool)
    for t in range(t_len):
        mask[t, :fill + t + 1] = True
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).transpose(0, 1),
                                         torch.from_numpy(kc[:, :n]), torch.from_numpy(vc[:, :n]),
                                         attn_mask=mask)
    np.testing.assert_allclose(got, ref.transpose(0, 1).numpy(), rtol=1e-10, atol=1e-12)
    one = O.attention_block_vs_cache(q[:1], kc, vc, fill)
    ref1 = F.scaled_dot_product_attention(torch.from_numpy(q[:1]).transpose(0, 1),
                                          torch.from_numpy(kc[:, :fill + 1]),
                                          torch.from_numpy(vc[:, :fill + 1]))
    np.testing.assert_allclose(one, ref1.transpose(0, 1).numpy(), rtol=1e-10, atol=1e-12)


def test_rope_is_a_position_rotation():
    """Pair i of the head is the complex number x[2i] + j x[2i+1] multiplied by
    exp(j * angle_i); dot products of 1-D rotated vectors depend on the position difference
    only; position 0 is the identity."""
    rng = np.random.default_rng(2)
    hd = 16
    x = rng.standard_normal(hd)
    y = rng.standard_normal(hd)
    for pos in (0, 1, 7, 300):
        ang = O.rope_angles(pos, hd, ROPE_1D, 10000.0)
        np.testing.assert_allclose(ang, [pos / 10000.0 ** (2 * i / hd) for i in range(hd // 2)],
                                   rtol=1e-12)
        z = (x[0::2] + 1j * x[1::2]) * np.exp(1j * ang)
        r = O.rope(x, ang)
        np.testing.assert_allclose(r[0::2], z.real, atol=1e-12)
        np.testing.assert_allclose(r[1::2], z.imag, atol=1e-12)
    np.testing.assert_array_equal(O.rope(x, O.rope_angles(0, hd, ROPE_1D, 10000.0)), x)

    def dot(pa, pb):
        return O.rope(x, O.rope_angles(pa, hd, ROPE_1D, 10000.0)) @ \
            O.rope(y, O.rope_angles(pb, hd, ROPE_1D, 10000.0))
    assert dot(5, 2) == pytest.approx(dot(105, 102), rel=1e-9)
    assert dot(5, 2) != pytest.approx(dot(5, 3), rel=1e-3)


def test_rope_2d_grid():
    """Grid rope: prefix positions are not rotated; the first half of the head depends on the
    grid row only, the second half on the grid column only; scores depend on (d_row, d_col)."""
    hd, w, npre = 16, 6, 1
    ang = lambda p: O.rope_angles(p, hd, ROPE_2D_GRID, 10000.0, w, npre)
    assert not ang(0).any()
    assert not ang(1).any()                                   # image token 0 = grid (0, 0)
    a = ang(1 + 2 * w + 3)                                    # grid (2, 3)
    b = ang(1 + 2 * w + 5)                                    # grid (2, 5)
    c = ang(1 + 4 * w + 3)                                    # grid (4, 3)
    np.testing.assert_array_equal(a[:hd // 4], b[:hd // 4])
    np.testing.assert_array_equal(a[hd // 4:], c[hd // 4:])
    assert (a[hd // 4:] != b[hd // 4:]).all() and (a[:hd // 4] != c[:hd // 4]).all()
    np.testing.assert_allclose(a[:hd // 4], [2 / 10000.0 ** (2 * j / (hd // 2)) for j in range(hd // 4)])
    np.testing.assert_allclose(a[hd // 4:], [3 / 10000.0 ** (2 * j / (hd // 2)) for j in range(hd // 4)])
    rng = np.random.default_rng(4)
    x, y = rng.standard_normal(hd), rng.standard_normal(hd)
    s1 = O.rope(x, ang(1 + 3 * w + 4)) @ O.rope(y, ang(1 + 1 * w + 1))
    s2 = O.rope(x, ang(1 + 4 * w + 5)) @ O.rope(y, ang(1 + 2 * w + 2))
    assert s1 == pytest.approx(s2, rel=1e-9)


class _TorchDecoder(torch.nn.Module):
    """Independent full-sequence causal decoder built from torch library routines."""

    def __init__(self, ms, w):
        super().__init__()
        self.ms, self.w = ms, w

    def forward(self, tokens, rot):
        ms = self.ms
        t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
        x = t(self.w["tok_emb"])[torch.as_tensor(tokens, dtype=torch.long)]
        n = x.shape[0]
        for l in range(ms.n_layers):
            w = self.w["layers"][l]
            a = F.rms_norm(x, (ms.d_model,), t(w["norm1"]), ms.rms_eps)
            q, k, v = F.linear(a, t(w["w_qkv"])).split(ms.d_model, dim=-1)
            shp = (n, ms.n_heads, ms.head_dim)
            q, k, v = (z.reshape(shp).transpose(0, 1) for z in (q, k, v))
            q, k = rot(q), rot(k)
            o = F.scaled_dot_product_attention(q, k, v, is_causal=True)
            x = x + F.linear(o.transpose(0, 1).reshape(n, ms.d_model), t(w["w_o"]))
            m = F.rms_norm(x, (ms.d_model,), t(w["norm2"]), ms.rms_eps)
            x = x + F.linear(F.silu(F.linear(m, t(w["w_gate"]))) * F.linear(m, t(w["w_up"])),
                             t(w["w_down"]))
        h = F.rms_norm(x, (ms.d_model,), t(self.w["norm_f"]), ms.rms_eps)
        lo = ms.vocab_offset
        return h, F.linear(h, t(self.w["w_lm"])[lo:lo + ms.vocab])


@pytest.mark.parametrize("rope_mode", [ROPE_NONE, ROPE_1D])
def test_forward_matches_torch_causal_decoder(rope_mode):
    """With an empty cache the block forward is an ordinary causal decoder: checked against a
    model assembled from torch's linear / rms_norm / silu / scaled_dot_product_attention."""
    ms = replace(MS, rope_mode=rope_mode, vocab=40, vocab_offset=8, lm_rows=64)
    w = gen.make_weights(ms, 5, w_std=0.2)
    tokens = gen.random_tokens(5, "tok", (11,), 0, ms.tok_rows)

    def rot(z):                                               # z [H, n, hd]
        if rope_mode == ROPE_NONE:
            return z
        half = ms.head_dim // 2
        pos = torch.arange(z.shape[1], dtype=torch.float64)[:, None]
        inv = ms.rope_base ** (-torch.arange(half, dtype=torch.float64) * 2 / ms.head_dim)
        zc = torch.view_as_complex(z.reshape(*z.shape[:-1], half, 2).contiguous())
        return torch.view_as_real(zc * torch.polar(torch.ones_like(pos * inv), pos * inv)).flatten(-2)

    kc = np.zeros((ms.n_layers, ms.n_heads, ms.s_max, ms.head_dim))
    vc = np.zeros_like(kc)
    h = O.target_forward(ms, w, tokens, kc, vc, 0)
    logits = O.lm_head_logits(ms, w, h)
    h_ref, l_ref = _TorchDecoder(ms, w)(tokens, rot)
    np.testing.assert_allclose(h, h_ref.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(logits, l_ref.numpy(), rtol=1e-9, atol=1e-11)
    assert logits.shape == (11, 40)


@pytest.mark.parametrize("rope_mode,grid_w,npre", [(ROPE_1D, 0, 0), (ROPE_2D_GRID, 5, 1)])
def test_block_verify_equals_token_by_token_decoding(rope_mode, grid_w, npre):
    """Parallel verification of a T-row block gives the same features and the same new cache
    entries as T single-token decode steps, and as one pass over prefix + block."""
    ms = replace(MS, rope_mode=rope_mode, rope_grid_w=grid_w, n_prefix=npre)
    w = gen.make_weights(ms, 9, w_std=0.2)
    seq = gen.random_tokens(9, "tok", (19,), 0, ms.tok_rows)
    fill, t_len = 13, 6
    shape = (ms.n_layers, ms.n_heads, ms.s_max, ms.head_dim)
    kc0, vc0 = np.zeros(shape), np.zeros(shape)
    h_all = O.target_forward(ms, w, seq, kc0, vc0, 0)          # one pass over everything
    kc1, vc1 = np.zeros(shape), np.zeros(shape)
    O.target_forward(ms, w, seq[:fill], kc1, vc1, 0)           # prefill
    kc_step, vc_step = kc1.copy(), vc1.copy()
    kc1[:, :, fill:] = 777.0                                   # garbage beyond the fill level
    vc1[:, :, fill:] = -777.0
    h_blk = O.target_forward(ms, w, seq[fill:], kc1, vc1, fill)
    np.testing.assert_allclose(h_blk, h_all[fill:], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(kc1[:, :, :fill + t_len], kc0[:, :, :fill + t_len], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(vc1[:, :, :fill + t_len], vc0[:, :, :fill + t_len], rtol=1e-9, atol=1e-11)
    assert (kc1[:, :, fill + t_len:] == 777.0).all()           # nothing written past the block
    for t in range(t_len):
        h_t = O.target_forward(ms, w, seq[fill + t:fill + t + 1], kc_step, vc_step, fill + t)
        np.testing.assert_allclose(h_t[0], h_all[fill + t], rtol=1e-9, atol=1e-11)


def test_guidance_special_cases():
    """l = l_u + s (l_c - l_u): s = 1 keeps the cond row, s = 0 the uncond row; identical rows
    make the scale irrelevant; no uncond row means no guidance."""
    rng = np.random.default_rng(6)
    lc, lu = rng.standard_normal((3, 9)), rng.standard_normal((3, 9))
    np.testing.assert_allclose(O.guided_probs(lc, lu, 1.0, 1.0), O.softmax(lc), rtol=1e-12)
    np.testing.assert_allclose(O.guided_probs(lc, lu, 0.0, 1.0), O.softmax(lu), rtol=1e-12)
    np.testing.assert_allclose(O.guided_probs(lc, lc, 3.7, 1.0), O.softmax(lc), rtol=1e-12)
    np.testing.assert_allclose(O.guided_probs(lc, None, 3.7, 1.0), O.softmax(lc), rtol=1e-12)
    np.testing.assert_allclose(O.guided_logits(lc, lu, 2.0), 2 * lc - lu, rtol=1e-12)
    np.testing.assert_allclose(O.guided_probs(lc, lu, 2.0, 0.5), O.softmax((2 * lc - lu) / 0.5), rtol=1e-12)


def test_verify_row_and_column_plumbing():
    """Whole-step wiring: cond/uncond rows of image b are rows b and B+b, the target row of
    draft i is block row n_forced-1+i, new_len = fill + n_forced + accept_len, and the step's
    target_probs equal softmax of guided logits of independently run sequences."""
    ms = replace(MS, vocab=32, lm_rows=64, vocab_offset=16, tok_rows=64)
    w = gen.make_weights(ms, 21, w_std=0.3)
    n_images, k, f = 2, 3, 2
    r = 2 * n_images
    kv_k, kv_v = gen.make_kv_cache(ms, 21, r)
    fills = np.array([5, 9, 7, 3], dtype=np.int32)
    block = gen.random_tokens(21, "blk", (n_images, f + k), 16, 48)
    q, _ = gen.independent_draft(21, 0, n_images, k, ms.vocab)
    u = np.array([[1e-6, 1e-6, 0.999999, 0.5], [0.999999, 0.5, 0.5, 0.25]], dtype=np.float32)
    n_draft = np.array([3, 3], dtype=np.int32)
    out = O.verify(ms, w, block, f, n_draft, kv_k, kv_v, fills, q, u, 2, 2.0)
    for b in range(n_images):
        rows = []
        for row in (b, n_images + b):
            kc, vc = O.widen(kv_k[:, row]), O.widen(kv_v[:, row])
            h = O.target_forward(ms, w, block[b], kc, vc, int(fills[row]))
            np.testing.assert_allclose(out["hidden"][row], h, rtol=1e-12)
            rows.append(O.lm_head_logits(ms, w, h))
        np.testing.assert_allclose(out["target_probs"][b], O.softmax(2 * rows[0] - rows[1]), rtol=1e-10)
    for b in range(n_images):                                  # stop at the first u >= ratio
        n = 0
        while n < 3 and u[b, n] < out["ratios"][b][n]:
            n += 1
        assert out["accept_len"][b] == n
    assert out["accept_len"][0] >= 2
    np.testing.assert_array_equal(out["new_len"], fills + f + out["accept_len"][[0, 1, 0, 1]])
    assert out["k_new"].shape == (ms.n_layers, r, ms.n_heads, f + k, ms.head_dim)
