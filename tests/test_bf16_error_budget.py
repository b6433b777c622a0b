"""Where does the 2-3 % feature error of the bf16 kernels at full depth come from?  CPU only.

The verify step's parity bound for features is 1e-2 of the row norm; the GPU tests scale it with
sqrt(layers / 3) (3.5e-2 at the 36 layers of the LlamaGen-XL shape) because every sublayer rounds
its GEMM inputs to bf16 again.  This file checks that claim WITHOUT the GPU: a float64 forward
built from the oracle's own pieces, in the oracle's order, in which only the operands the
workload declares bf16 ("bf16 weights/activations, fp32 softmax") are rounded to bf16 -- the
normalised GEMM inputs, q / k / v, the softmax weights before they multiply V, the attention
output, silu(gate) * up, and the features -- is compared with the unrounded oracle on the full
36-layer shape.  Its distance is the floor any bf16-activation implementation has on this random-init
network: if the kernels measured much more than this, they would have an error source of their own.
"""
import numpy as np

from oracle import vvs_oracle as O
from vvs_synth import gen
from vvs_synth.configs import CONFIGS


def _bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bfloat16 (ties to even), back to float64."""
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def _norm_in(x, scale, eps, defer):
    """The bf16 operand of a projection: bf16(rmsnorm(x) * scale), or -- what a kernel that applies
    1 / rms to the product does -- bf16(x * scale) / rms.  Both are legitimate placements of the one
    rounding; they differ in which bits are rounded away."""
    if not defer:
        return _bf16(O.rmsnorm(x, scale, eps))
    rms = np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return _bf16(x * scale) / rms


def _forward_with_rounded_activations(ms, w, tokens, kc, vc, fill, defer=False):
    """oracle.target_forward step by step, with bf16 rounding where an activation is stored or fed
    to a projection."""
    d, n_heads, hd = ms.d_model, ms.n_heads, ms.head_dim
    t_len = len(tokens)
    x = O.widen(w["tok_emb"][np.asarray(tokens)])
    ang = [O.rope_angles(fill + t, hd, ms.rope_mode, ms.rope_base, ms.rope_grid_w, ms.n_prefix) for t in range(t_len)]
    for l in range(ms.n_layers):
        lw = w["layers"][l]
        a = _norm_in(x, O.widen(lw["norm1"]), ms.rms_eps, defer)
        qkv = a @ O.widen(lw["w_qkv"]).T
        q = qkv[:, :d].reshape(t_len, n_heads, hd)
        k = qkv[:, d:2 * d].reshape(t_len, n_heads, hd)
        v = qkv[:, 2 * d:].reshape(t_len, n_heads, hd)
        for t in range(t_len):
            q[t] = _bf16(O.rope(q[t], ang[t]))
            kc[l, :, fill + t, :] = _bf16(O.rope(k[t], ang[t]))
            vc[l, :, fill + t, :] = _bf16(v[t])
        o = np.zeros((t_len, n_heads, hd))
        for h in range(n_heads):
            for t in range(t_len):
                n_keys = fill + t + 1
                s = kc[l, h, :n_keys] @ q[t, h] / np.sqrt(hd)
                e = np.exp(s - s.max())
                o[t, h] = (_bf16(e) @ vc[l, h, :n_keys]) / e.sum()   # P rounded, its sum kept exact
        x = x + _bf16(o.reshape(t_len, d)) @ O.widen(lw["w_o"]).T
        m = _norm_in(x, O.widen(lw["norm2"]), ms.rms_eps, defer)
        g = m @ O.widen(lw["w_gate"]).T
        u = m @ O.widen(lw["w_up"]).T
        x = x + _bf16(O.silu(g) * u) @ O.widen(lw["w_down"]).T
    return _bf16(O.rmsnorm(x, O.widen(w["norm_f"]), ms.rms_eps))


def test_bf16_rounding_helper_is_round_to_nearest_even():
    import torch
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000), [0.0, -0.0, 1.0, 1.00390625, 1.01171875]])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(_bf16(x), want)


def test_depth_scaled_feature_tolerance_is_the_floor_of_bf16_activations():
    wl = CONFIGS[1]
    ms = wl.shape
    fill, t_len = 288, 9
    w = gen.make_weights(ms, wl.seed)
    kv_k, kv_v = gen.make_kv_cache(ms, wl.seed, 1)
    tokens = gen.random_tokens(wl.seed, "budget", (t_len,), ms.vocab_offset, ms.vocab_offset + ms.vocab)
    kc, vc = O.widen(kv_k[:, 0]), O.widen(kv_v[:, 0])
    h_ref = O.target_forward(ms, w, tokens, kc.copy(), vc.copy(), fill)
    h_rnd = _forward_with_rounded_activations(ms, w, tokens, kc.copy(), vc.copy(), fill)
    rel = np.linalg.norm(h_rnd - h_ref, axis=1) / np.linalg.norm(h_ref, axis=1)
    print("bf16-activation emulation vs float64 oracle at %d layers: feature error per row %s (max %.4f)"
          % (ms.n_layers, np.round(rel, 4), rel.max()))
    # the rounding floor at full depth: above the plain 1e-2 (so a depth-independent bound cannot hold
    # for any bf16-activation path), inside the depth-scaled bound the GPU tests use, and of the size
    # the kernels measure (2.0-3.1 %): they add no error source of their own
    bound = 1e-2 * (ms.n_layers / 3.0) ** 0.5
    assert rel.max() > 1e-2
    assert rel.max() < bound
    assert 0.012 < np.median(rel) < 0.032
    # Two equally valid placements of the same roundings do not track each other: their rounding
    # noise is independent, so they sit as far from one another as each sits from the exact result
    # (times ~sqrt 2).  No bf16 path can therefore be held to 1e-2 of another bf16 path at this
    # depth; the exact float64 oracle with the depth-scaled bound is the meaningful reference.
    h_alt = _forward_with_rounded_activations(ms, w, tokens, kc.copy(), vc.copy(), fill, defer=True)
    rel_alt = np.linalg.norm(h_alt - h_ref, axis=1) / np.linalg.norm(h_ref, axis=1)
    rel_pair = np.linalg.norm(h_alt - h_rnd, axis=1) / np.linalg.norm(h_ref, axis=1)
    print("second placement vs oracle: max %.4f; the two placements vs each other: max %.4f" % (rel_alt.max(), rel_pair.max()))
    assert rel_alt.max() < bound
    assert rel_pair.max() > 1e-2
    # probabilities of one guided row pair (same features used for both rows: only the size matters)
    l_ref = O.lm_head_logits(ms, w, h_ref)
    l_rnd = O.lm_head_logits(ms, w, h_rnd)
    dp = np.abs(O.softmax(l_rnd) - O.softmax(l_ref)).max()
    print("max probability difference %.2e" % dp)
    assert dp < 2e-3
