"""Seeded synthetic inputs for the verify step: weights, KV caches, token blocks, draft
distributions, latent-neighbour tables, feature-cache traffic.

Every tensor has its own Philox stream keyed by (seed, tensor id), so any subset can be
generated independently and reproducibly.  bf16 tensors are carried as uint16 bit patterns
(numpy has no bf16); fp32 tensors as float32.  Nothing here implements a step of the
verification method: the generators only draw numbers, round them to the storage type and
arrange them in the layouts the library documents.
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from .configs import DTYPE_BF16, ModelShape

# ---------------------------------------------------------------------------------------
# storage-type helpers


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def store(x: np.ndarray, dtype: int) -> np.ndarray:
    """Round a float array to the storage type of `dtype` (uint16 bits for bf16, float32 else)."""
    x = np.asarray(x, dtype=np.float32)
    return f32_to_bf16_bits(x) if dtype == DTYPE_BF16 else x


def rng_for(seed: int, tensor_id: str) -> np.random.Generator:
    h = zlib.crc32(tensor_id.encode()) & 0xFFFFFFFF
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, h]))


def _normal(seed: int, tensor_id: str, shape, std: float, mean: float = 0.0) -> np.ndarray:
    g = rng_for(seed, tensor_id)
    a = g.standard_normal(shape, dtype=np.float32)
    a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return a


# ---------------------------------------------------------------------------------------
# model weights

LAYER_TENSORS = ("w_qkv", "w_o", "w_gate", "w_up", "w_down", "norm1", "norm2")


def weight_shapes(ms: ModelShape) -> dict:
    """Shapes of every weight tensor; projection matrices are [out_features, in_features]."""
    d, ff = ms.d_model, ms.d_ff
    return {
        "tok_emb": (ms.tok_rows, d), "norm_f": (d,), "w_lm": (ms.lm_rows, d),
        "w_qkv": (3 * d, d), "w_o": (d, d), "w_gate": (ff, d), "w_up": (ff, d),
        "w_down": (d, ff), "norm1": (d,), "norm2": (d,),
    }


def make_tensor(ms: ModelShape, seed: int, name: str, layer: int | None = None,
                w_std: float = 0.02, norm_jitter: float = 0.1, lm_std: float | None = None):
    shp = weight_shapes(ms)[name]
    tid = name if layer is None else f"layer{layer}.{name}"
    if name.startswith("norm"):
        a = _normal(seed, tid, shp, norm_jitter, 1.0)
    elif name == "w_lm" and lm_std is not None:
        a = _normal(seed, tid, shp, lm_std)
    else:
        a = _normal(seed, tid, shp, w_std)
    return store(a, ms.dtype)


def make_weights(ms: ModelShape, seed: int, layers=None, threads: int = 8, **kw) -> dict:
    """Returns {'tok_emb', 'norm_f', 'w_lm', 'layers': [ {w_qkv,..}, ... ]}.

    Weights ~ N(0, 0.02^2); RMSNorm scales ~ 1 + N(0, 0.1^2) (not exactly 1, so that a
    dropped scale is visible).  `layers` limits generation to a subset of layer indices.
    """
    layers = list(range(ms.n_layers)) if layers is None else list(layers)
    jobs = [("tok_emb", None), ("norm_f", None), ("w_lm", None)]
    jobs += [(n, l) for l in layers for n in LAYER_TENSORS]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        res = list(ex.map(lambda j: make_tensor(ms, seed, j[0], j[1], **kw), jobs))
    out = {"layers": {l: {} for l in layers}}
    for (n, l), a in zip(jobs, res):
        if l is None:
            out[n] = a
        else:
            out["layers"][l][n] = a
    return out


# ---------------------------------------------------------------------------------------
# KV cache, blocks, draft distributions


def make_kv_row(ms: ModelShape, seed: int, row: int, std: float = 1.0):
    """K and V of one sequence: [n_layers][n_heads][s_max][head_dim] each, own Philox streams."""
    shp = (ms.n_layers, ms.n_heads, ms.s_max, ms.head_dim)
    return (store(_normal(seed, f"kv.k.{row}", shp, std), ms.dtype),
            store(_normal(seed, f"kv.v.{row}", shp, std), ms.dtype))


def make_kv_cache(ms: ModelShape, seed: int, n_rows: int, std: float = 1.0, threads: int = 8):
    """K and V caches, layout [n_layers][n_rows][n_heads][s_max][head_dim], all slots ~N(0,1)
    (slots at and beyond a row's fill level are garbage the step must ignore or overwrite)."""
    with ThreadPoolExecutor(max_workers=threads) as ex:
        rows = list(ex.map(lambda r: make_kv_row(ms, seed, r, std), range(n_rows)))
    k = np.stack([r[0] for r in rows], axis=1)
    v = np.stack([r[1] for r in rows], axis=1)
    return k, v


def make_fills(seed: int, n_images: int, lo: int, hi: int, trial: int = 0) -> np.ndarray:
    g = rng_for(seed, f"fills.{trial}")
    return g.integers(lo, hi + 1, size=n_images, dtype=np.int64).astype(np.int32)


def random_tokens(seed: int, tid: str, shape, lo: int, hi: int) -> np.ndarray:
    """int32 tokens uniform in [lo, hi)."""
    return rng_for(seed, tid).integers(lo, hi, size=shape, dtype=np.int64).astype(np.int32)


def softmax_rows_f32(logits: np.ndarray) -> np.ndarray:
    """float32 probabilities of the drafter (an input of the step): exp-normalise each row in
    float64, then round to float32."""
    z = np.asarray(logits, dtype=np.float64)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return (e / e.sum(axis=-1, keepdims=True)).astype(np.float32)


def sample_rows(probs: np.ndarray, u: np.ndarray) -> np.ndarray:
    """Draw one index per row of `probs` from uniforms `u` (drafter-side sampling)."""
    cdf = np.cumsum(np.asarray(probs, dtype=np.float64), axis=-1)
    t = np.asarray(u, dtype=np.float64) * cdf[..., -1]
    idx = (cdf <= t[..., None]).sum(axis=-1)
    return np.minimum(idx, probs.shape[-1] - 1).astype(np.int32)


def independent_draft(seed: int, trial: int, n_images: int, n_draft: int, vocab: int,
                      logit_std: float = 2.0):
    """Target-independent drafter: q = softmax(N(0, std^2) logits), drafts sampled from q.
    Returns (draft_probs float32 [B,K,V], drafts int32 [B,K])."""
    g = rng_for(seed, f"draft.{trial}")
    logits = g.standard_normal((n_images, n_draft, vocab), dtype=np.float32) * np.float32(logit_std)
    q = softmax_rows_f32(logits)
    u = g.random((n_images, n_draft))
    return q, sample_rows(q, u)


def perturbed_draft_row(seed: int, tid: str, target_logits: np.ndarray, noise_std: float,
                        temperature: float = 1.0, gumbel: float = 0.0):
    """Drafter correlated with the target: logits = target/temperature + N(0, noise_std^2)
    + gumbel * Gumbel(0,1).  Returns (q float32 [V], token int32) with token ~ q."""
    g = rng_for(seed, tid)
    v = target_logits.shape[-1]
    z = np.asarray(target_logits, dtype=np.float64) / temperature
    z = z + g.standard_normal(v) * noise_std
    if gumbel:
        z = z - gumbel * np.log(-np.log(g.random(v)))
    q = softmax_rows_f32(z)
    tok = sample_rows(q[None, :], g.random(1))[0]
    return q, np.int32(tok)


# ---------------------------------------------------------------------------------------
# latent-space neighbour table (CSR)


def make_codebook(seed: int, vocab: int, latent_dim: int = 8) -> np.ndarray:
    return rng_for(seed, "codebook").standard_normal((vocab, latent_dim))


def neighbour_csr(codebook: np.ndarray, k: int, block: int = 1024):
    """Exact top-k Euclidean neighbours of every code (fp64 brute force), self first, ties
    broken by lower index.  Returns (row_ptr int32 [V+1], col int32 [V*k])."""
    e = np.asarray(codebook, dtype=np.float64)
    v = e.shape[0]
    k = min(k, v)
    sq = (e * e).sum(axis=1)
    col = np.empty((v, k), dtype=np.int32)
    for s in range(0, v, block):
        t = min(v, s + block)
        d2 = sq[s:t, None] + sq[None, :] - 2.0 * (e[s:t] @ e.T)
        d2[np.arange(t - s), np.arange(s, t)] = -1.0           # self is rank 0
        if k < v:
            part = np.argpartition(d2, k - 1, axis=1)[:, :k]
            kth = np.take_along_axis(d2, part, axis=1).max(axis=1)
            for r in range(t - s):
                cand = np.nonzero(d2[r] <= kth[r])[0]          # includes every tie at the k-th
                order = np.lexsort((cand, d2[r, cand]))
                col[s + r] = cand[order[:k]]
        else:
            for r in range(t - s):
                col[s + r] = np.lexsort((np.arange(v), d2[r]))
    row_ptr = (np.arange(v + 1, dtype=np.int64) * k).astype(np.int32)
    return row_ptr, col.reshape(-1)
