"""fp64 CPU oracle of the VVS target-model verification step.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module;
the CUDA library never does, and the two share no code.  Everything is written out plainly
in numpy float64 (a matmul / cumsum / exp from numpy may serve as a step), in the order the
paper states the method, with no blocking, fusion or reordering.

Naming.  The paper (Sec. 2, "Speculative Decoding") calls the draft distribution p and the
target distribution q.  This code uses the opposite, more common convention of the task
statement: **p = target, q = draft**.

What the paper fixes (Sec. 2; Sec. 4.1, 4.3; Algorithm 2 lines 9-11; Supp. "Memory
Overhead") and what it leaves open is listed per function.  Readings chosen where the paper
is silent or garbled:

* residual distribution: the paper prints max{0, p - q} in *its* naming (draft - target),
  un-normalised.  Used here: norm(max(0, target - draft)), the only sign for which strict
  verification is lossless, which the paper claims (Sec. 6 "lossless").
* relaxed acceptance (Sec. 2, LANTERN rule, garbled in print): the neighbourhood of a drafted
  token x is the first k entries of its CSR row, ordered by latent distance with x itself
  first; the accepted set A is {x} plus the longest distance-ordered prefix of the other
  entries whose cumulative target mass (not counting p(x)) stays <= delta; acceptance
  probability min(1, sum_{x' in A} p(x') / q(x)).  **parity unpinned** by the paper beyond
  "k = 1 or delta = 0 is strict" and the bounds p(x) <= P_A <= p(x) + delta.
* residual after a relaxed rejection: the plain norm(max(0, p - q)) by default.  Flag
  `adjusted_residual`: norm(max(0, p~ - q)) with p~ the adjusted target of the rejected draft x
  (the pooled mass of A sits on x, the other members of A carry none): the distribution under
  which the relaxed test of x is the plain speculative test.  **parity unpinned** by the paper
  for the choice; mass conservation, the hand example and k = 1 = strict are pinned.
* relaxed acceptance on a candidate tree (not printed): the chain's relaxed rule with the
  current residual p_res in the place of p at every sibling round.  **parity unpinned** by the
  paper; pinned here by k = 1 = the strict walk and by a chain-shaped tree = the chain rule.
* classifier-free guidance is not in the paper: l = l_u + s (l_c - l_u) on logits before the
  softmax; rows ordered [cond_0..cond_{B-1}, uncond_0..uncond_{B-1}].
* architecture (not in the paper): pre-norm RMSNorm (eps inside the square root, learned
  scale), SwiGLU MLP, no biases, untied LM head, attention scale 1/sqrt(head_dim).
* RoPE: consecutive-pair (even, odd) convention; 1-D on the absolute position, or 2-D over a
  w-wide token grid where prefix positions get no rotation, the first half of the head
  dimension rotates by grid row and the second half by grid column.  **parity unpinned**
  (convention only; its rotation properties are pinned).
* feature cache (Sec. 4.3): feature = final-norm output (LM-head input) of each committed
  block row, addressed by (row, absolute position) in a ring of `cap` slots; fetch(gamma, s)
  returns positions newest-s-gamma+1 .. newest-s.  **parity unpinned** for the choice of
  post-norm features and ring addressing; the index arithmetic itself is pinned.
* dynamic skip decision (Sec. 4.4, Eq. 2, Alg. 1): S^(l) = mean cosine over all unordered pairs
  of the paths kept by the stride-2 down-sampling, depth = shortest kept path, zero embedding =
  cosine 0.  **parity unpinned** for the pair-mean and the depth rule (the paper says only
  "cosine similarity of token representations at each position"); the depth weights, the
  no-two-skips guard, the threshold rule and the cosine itself are pinned.
* decisions are taken on the float32 target probabilities the step emits: ratios, pooled
  masses and the sampling CDF accumulate in float64 in ascending / distance order.
"""
from __future__ import annotations

import numpy as np

ROPE_NONE, ROPE_1D, ROPE_2D_GRID = 0, 1, 2
MODE_STRICT, MODE_RELAXED = 0, 1


# ---------------------------------------------------------------------------------------
# storage widening


def widen(a: np.ndarray) -> np.ndarray:
    """Exact widening of stored bits to float64: uint16 = bfloat16 bit patterns, else float."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


# ---------------------------------------------------------------------------------------
# transformer pieces (architecture per the workload description; the paper only says the
# target model M_T maps the candidate block to logits and hidden states, Alg. 2 line 9)


def rmsnorm(x: np.ndarray, scale: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * scale over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * scale


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def rope_angles(pos: int, head_dim: int, mode: int, base: float, grid_w: int = 0,
                n_prefix: int = 0) -> np.ndarray:
    """Rotation angle of each of the head_dim/2 consecutive pairs at absolute position pos."""
    half = head_dim // 2
    if mode == ROPE_NONE:
        return np.zeros(half)
    if mode == ROPE_1D:
        i = np.arange(half, dtype=np.float64)
        return pos * base ** (-2.0 * i / head_dim)
    if mode == ROPE_2D_GRID:
        if pos < n_prefix:
            return np.zeros(half)
        n = pos - n_prefix
        row, col = n // grid_w, n % grid_w
        quarter = half // 2
        j = np.arange(quarter, dtype=np.float64)
        freq = base ** (-2.0 * j / half)
        return np.concatenate([row * freq, col * freq])
    raise ValueError("rope mode")


def rope(x: np.ndarray, angles: np.ndarray) -> np.ndarray:
    """Rotate consecutive pairs (x[2i], x[2i+1]) of the last axis by angles[i]."""
    c, s = np.cos(angles), np.sin(angles)
    xe, xo = x[..., 0::2], x[..., 1::2]
    y = np.empty_like(x)
    y[..., 0::2] = xe * c - xo * s
    y[..., 1::2] = xe * s + xo * c
    return y


def softmax(z: np.ndarray) -> np.ndarray:
    e = np.exp(z - np.max(z, axis=-1, keepdims=True))
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_block_vs_cache(q: np.ndarray, kc: np.ndarray, vc: np.ndarray, fill: int) -> np.ndarray:
    """Parallel verification attention (Sec. 2: the candidates are appended to the input and
    scored in one pass): block row t sees cache slots [0, fill) and block rows 0..t, which
    already sit in slots fill..fill+t of kc/vc.

    q [T, H, hd]; kc, vc [H, S, hd].  Returns [T, H, hd]."""
    t_len, n_heads, hd = q.shape
    out = np.zeros_like(q)
    for h in range(n_heads):
        for t in range(t_len):
            n_keys = fill + t + 1
            s = kc[h, :n_keys] @ q[t, h] / np.sqrt(hd)
            w = softmax(s)
            out[t, h] = w @ vc[h, :n_keys]
    return out


def target_forward(ms, weights: dict, tokens: np.ndarray, kc: np.ndarray, vc: np.ndarray,
                   fill: int) -> np.ndarray:
    """M_T over one sequence's block (Alg. 2 line 9): returns the features h (final-norm
    output, i.e. the hidden state before the output head, Sec. 3 "Stale Feature Reusability")
    for every block row, and appends the block's keys/values to the float64 caches
    kc, vc [n_layers, H, S, hd] in slots fill..fill+T-1 (the KV entries a later step needs,
    Sec. 4.1)."""
    d, n_heads, hd = ms.d_model, ms.n_heads, ms.head_dim
    t_len = len(tokens)
    x = widen(weights["tok_emb"][np.asarray(tokens)])
    ang = [rope_angles(fill + t, hd, ms.rope_mode, ms.rope_base, ms.rope_grid_w, ms.n_prefix)
           for t in range(t_len)]
    for l in range(ms.n_layers):
        w = weights["layers"][l]
        a = rmsnorm(x, widen(w["norm1"]), ms.rms_eps)
        qkv = a @ widen(w["w_qkv"]).T
        q = qkv[:, 0 * d:1 * d].reshape(t_len, n_heads, hd)
        k = qkv[:, 1 * d:2 * d].reshape(t_len, n_heads, hd)
        v = qkv[:, 2 * d:3 * d].reshape(t_len, n_heads, hd)
        for t in range(t_len):
            q[t] = rope(q[t], ang[t])
            kc[l, :, fill + t, :] = rope(k[t], ang[t])
            vc[l, :, fill + t, :] = v[t]
        o = attention_block_vs_cache(q, kc[l], vc[l], fill).reshape(t_len, d)
        x = x + o @ widen(w["w_o"]).T
        m = rmsnorm(x, widen(w["norm2"]), ms.rms_eps)
        g = m @ widen(w["w_gate"]).T
        u = m @ widen(w["w_up"]).T
        x = x + (silu(g) * u) @ widen(w["w_down"]).T
    return rmsnorm(x, widen(weights["norm_f"]), ms.rms_eps)


def lm_head_logits(ms, weights: dict, hidden: np.ndarray) -> np.ndarray:
    """Logits over the image codebook only: rows vocab_offset .. vocab_offset+V-1 of the head."""
    w = widen(weights["w_lm"][ms.vocab_offset:ms.vocab_offset + ms.vocab])
    return hidden @ w.T


def guided_logits(l_cond: np.ndarray, l_uncond, cfg_scale: float) -> np.ndarray:
    """Classifier-free guidance on logits: l_u + s (l_c - l_u); without an uncond row, l_c."""
    return l_cond if l_uncond is None else l_uncond + cfg_scale * (l_cond - l_uncond)


def guided_probs(l_cond: np.ndarray, l_uncond, cfg_scale: float, temperature: float) -> np.ndarray:
    """Guided logits, then the temperature softmax (the paper samples at temperature 1)."""
    return softmax(guided_logits(l_cond, l_uncond, cfg_scale) / temperature)


# ---------------------------------------------------------------------------------------
# decision stage (Sec. 2): acceptance, accepted prefix, residual / bonus sample


def pooled_mass(p_row: np.ndarray, x: int, row_ptr: np.ndarray, col: np.ndarray, k: int,
                delta: float) -> float:
    """Relaxed (LANTERN) numerator: p(x) plus the target mass of the longest distance-ordered
    prefix of x's other neighbours whose running sum stays <= delta."""
    nb = col[row_ptr[x]:row_ptr[x + 1]][:k]
    assert len(nb) == 0 or nb[0] == x, "neighbour rows must list the token itself first"
    cum = 0.0
    for xn in nb[1:]:
        pn = float(p_row[xn])
        if cum + pn > delta:
            break
        cum += pn
    return float(p_row[x]) + cum


def pooled_neighbours(p_row: np.ndarray, x: int, row_ptr: np.ndarray, col: np.ndarray, k: int,
                      delta: float) -> list:
    """The neighbours of x (x itself excluded) whose mass pooled_mass adds to p(x): the same
    distance-ordered prefix, as a list of codebook indices."""
    nb = col[row_ptr[x]:row_ptr[x + 1]][:k]
    cum, taken = 0.0, []
    for xn in nb[1:]:
        pn = float(p_row[xn])
        if cum + pn > delta:
            break
        cum += pn
        taken.append(int(xn))
    return taken


def adjusted_target(p_row: np.ndarray, x: int, row_ptr: np.ndarray, col: np.ndarray, k: int,
                    delta: float) -> np.ndarray:
    """Target row under which the relaxed test of draft x is the plain speculative test (the
    adjusted distribution of the relaxed-acceptance construction the paper takes over in Sec. 2):
    the pooled neighbours' mass sits on x, the pooled neighbours carry none, every other code keeps
    its probability.  Same dtype as p_row (the moved mass is rounded to it)."""
    out = np.array(p_row, copy=True)
    mass = pooled_mass(p_row, x, row_ptr, col, k, delta)
    for xn in pooled_neighbours(p_row, x, row_ptr, col, k, delta):
        out[xn] = 0
    out[x] = mass
    return out


def acceptance_ratio(p_mass: float, q_x: float) -> float:
    """min(1, P / q(x)); a draft with q(x) = 0 is accepted iff P > 0."""
    if q_x > 0.0:
        return min(1.0, p_mass / q_x)
    return 1.0 if p_mass > 0.0 else 0.0


def inverse_cdf(r: np.ndarray, u: float):
    """Smallest index j with sum_{i<=j} r_i > u * sum(r), accumulating in float64 in ascending
    index; if rounding leaves none, the last index with r_j > 0.  Returns (j, margin) where
    margin is the distance of u*sum(r) to the nearest edge of bin j, as a fraction of sum(r)."""
    cdf = np.cumsum(r.astype(np.float64))
    total = cdf[-1]
    t = float(u) * total
    above = np.nonzero(cdf > t)[0]
    j = int(above[0]) if len(above) else int(np.nonzero(r > 0)[0][-1])
    lo = cdf[j - 1] if j > 0 else 0.0
    margin = min(abs(t - lo), abs(cdf[j] - t)) / total
    return j, margin


def decide(p32: np.ndarray, drafts: np.ndarray, n_draft: int, n_forced: int, q32: np.ndarray,
           u32: np.ndarray, mode: int = MODE_STRICT, row_ptr=None, col=None, k: int = 1,
           delta: float = float("inf"), adjusted_residual: bool = False) -> dict:
    """Sequential verification of one image's drafts against float32 target rows p32 [T, V].

    Draft i (token drafts[i], draft row q32[i]) is judged against p32[n_forced-1+i] with
    uniform u32[i]; verification stops at the first rejection.  The next token comes from
    norm(max(0, p - q)) of the rejecting position, or from the following target row if every
    draft was accepted (-1 if p32 has no such row); it uses the last uniform u32[-1].
    With `adjusted_residual` (relaxed mode only; off by default) the p of the residual is the
    adjusted target of the rejected draft instead of the plain row."""
    p32 = np.asarray(p32, dtype=np.float32)
    q32 = np.asarray(q32, dtype=np.float32)
    k_max = len(u32) - 1
    mask = np.zeros(k_max, dtype=np.uint8)
    margins = np.full(k_max + 1, np.inf)
    ratios = np.full(k_max, np.nan)
    n = 0
    for i in range(n_draft):
        x = int(drafts[i])
        row = p32[n_forced - 1 + i]
        if mode == MODE_RELAXED:
            mass = pooled_mass(row, x, row_ptr, col, k, delta)
        else:
            mass = float(row[x])
        ratio = acceptance_ratio(mass, float(q32[i, x]))
        ratios[i] = ratio
        margins[i] = abs(float(u32[i]) - ratio)
        if not float(u32[i]) < ratio:
            break
        mask[i] = 1
        n += 1
    src = n_forced - 1 + n
    if src >= p32.shape[0]:
        token = -1
    else:
        row = p32[src]
        if n < n_draft:
            if adjusted_residual and mode == MODE_RELAXED:
                row = adjusted_target(row, int(drafts[n]), row_ptr, col, k, delta)
            r = np.maximum(np.float32(0.0), row - q32[n])       # IEEE float32 subtraction
            if not np.any(r > 0):
                r = row                                          # p == q numerically
        else:
            r = row
        token, margins[k_max] = inverse_cdf(r, float(u32[k_max]))
    return {"accept_len": n, "accept_mask": mask, "next_token": int(token),
            "margins": margins, "ratios": ratios}


# ---------------------------------------------------------------------------------------
# the whole step (Alg. 2 lines 9-10)


def epilogue(ms, weights: dict, hidden: np.ndarray, drafts, n_draft, n_forced: int, draft_probs,
             uniforms, n_cfg: int, cfg_scale: float, temperature: float = 1.0, mode: int = MODE_STRICT,
             row_ptr=None, col=None, k: int = 1, delta: float = float("inf"),
             adjusted_residual: bool = False) -> dict:
    """LM head + guidance + softmax + decisions on given features.

    hidden [R, T, d] with R = n_cfg*B rows ordered cond images then uncond images (n_cfg = 2
    with guidance, else 1); drafts int [B, K]; draft_probs float32 [B, K, V]; uniforms
    [B, K+1]."""
    n_images = hidden.shape[0] // n_cfg
    t_len = hidden.shape[1]
    probs = np.zeros((n_images, t_len, ms.vocab))
    logits = np.zeros((n_images, t_len, ms.vocab))
    out = {"accept_len": np.zeros(n_images, np.int32), "next_token": np.zeros(n_images, np.int32),
           "accept_mask": np.zeros((n_images, uniforms.shape[1] - 1), np.uint8),
           "margins": np.zeros((n_images, uniforms.shape[1])),
           "ratios": np.zeros((n_images, uniforms.shape[1] - 1))}
    for b in range(n_images):
        l_c = lm_head_logits(ms, weights, widen(hidden[b]))
        l_u = lm_head_logits(ms, weights, widen(hidden[n_images + b])) if n_cfg == 2 else None
        logits[b] = guided_logits(l_c, l_u, cfg_scale)
        probs[b] = guided_probs(l_c, l_u, cfg_scale, temperature)
        dec = decide(probs[b].astype(np.float32), drafts[b], int(n_draft[b]), n_forced,
                     draft_probs[b], uniforms[b], mode, row_ptr, col, k, delta, adjusted_residual)
        for key in ("accept_len", "next_token", "accept_mask", "margins", "ratios"):
            out[key][b] = dec[key]
    out["target_probs"] = probs
    out["logits"] = logits
    return out


def verify(ms, weights: dict, block: np.ndarray, n_forced: int, n_draft: np.ndarray,
           kv_k: np.ndarray, kv_v: np.ndarray, cache_len: np.ndarray, draft_probs: np.ndarray,
           uniforms: np.ndarray, n_cfg: int, cfg_scale: float, temperature: float = 1.0,
           mode: int = MODE_STRICT, row_ptr=None, col=None, k: int = 1,
           delta: float = float("inf"), adjusted_residual: bool = False) -> dict:
    """One verification step for B images.

    block int [B, T] = n_forced committed tokens whose K/V is not yet cached, then K drafts,
    as embedding-table ids (a draft's codebook index is id - vocab_offset; next_token is
    returned as an embedding-table id as well).
    kv_k, kv_v stored caches [n_layers, R, H, S, hd] (read, not modified); cache_len int [R].
    Returns accept_len, next_token, new_len, accept_mask, target_probs [B,T,V] (float64),
    hidden [R,T,d] (float64), the new cache rows k_new/v_new [n_layers, R, H, T, hd] and the
    decision margins."""
    n_images, t_len = block.shape
    n_rows = n_images * n_cfg
    hidden = np.zeros((n_rows, t_len, ms.d_model))
    k_new = np.zeros((ms.n_layers, n_rows, ms.n_heads, t_len, ms.head_dim))
    v_new = np.zeros_like(k_new)
    for r in range(n_rows):
        b = r % n_images
        fill = int(cache_len[r])
        kc = widen(kv_k[:, r])
        vc = widen(kv_v[:, r])
        hidden[r] = target_forward(ms, weights, block[b], kc, vc, fill)
        k_new[:, r] = kc[:, :, fill:fill + t_len]
        v_new[:, r] = vc[:, :, fill:fill + t_len]
    drafts = block[:, n_forced:] - ms.vocab_offset            # embedding id -> codebook index
    out = epilogue(ms, weights, hidden, drafts, n_draft, n_forced, draft_probs, uniforms,
                   n_cfg, cfg_scale, temperature, mode, row_ptr, col, k, delta, adjusted_residual)
    out["next_token"] = np.where(out["next_token"] >= 0, out["next_token"] + ms.vocab_offset,
                                 -1).astype(np.int32)
    out["hidden"] = hidden
    out["k_new"], out["v_new"] = k_new, v_new
    out["new_len"] = np.array([int(cache_len[r]) + n_forced + int(out["accept_len"][r % n_images])
                               for r in range(n_rows)], dtype=np.int32)
    return out


# ---------------------------------------------------------------------------------------
# token-level feature cache (Sec. 4.3; Alg. 2 lines 5 and 11; Supp. "Memory Overhead")


class FeatureCache:
    """Per-row ring of the most recent token-level features, addressed by absolute position."""

    def __init__(self, n_rows: int, cap: int, d: int):
        self.cap = cap
        self.feat = np.zeros((n_rows, cap, d))
        self.fpos = np.full((n_rows, cap), -1, dtype=np.int32)
        self.newest = np.full(n_rows, -1, dtype=np.int32)

    def store(self, hidden: np.ndarray, base_pos: np.ndarray, n_store: np.ndarray) -> None:
        """UpdateCache(h_t): row r keeps hidden[r, t] for t < n_store[r] at absolute position
        base_pos[r] + t (slot = position mod cap; a re-stored position is overwritten, which
        is how post verification writes features back to their positions, Sec. 4.1)."""
        for r in range(hidden.shape[0]):
            for t in range(int(n_store[r])):
                pos = int(base_pos[r]) + t
                self.feat[r, pos % self.cap] = hidden[r, t]
                self.fpos[r, pos % self.cap] = pos
            if n_store[r] > 0:
                self.newest[r] = max(self.newest[r], int(base_pos[r]) + int(n_store[r]) - 1)

    def fetch(self, skip_mask: np.ndarray, gamma: np.ndarray, staleness: int, gamma_max: int):
        """Retrieve(C, a): for rows whose image is skip-masked, the gamma[r] most recent
        features ending `staleness` positions before the newest one, oldest first.  A position
        that was never stored or has been overwritten yields out_pos = -1 and a zero row.
        Rows not masked, and entries j >= gamma[r], are left zero / -1 here."""
        n_rows, _, d = self.feat.shape
        n_images = len(skip_mask)
        out = np.zeros((n_rows, gamma_max, d))
        out_pos = np.full((n_rows, gamma_max), -1, dtype=np.int32)
        for r in range(n_rows):
            if not skip_mask[r % n_images]:
                continue
            g = int(gamma[r])
            for j in range(g):
                pos = int(self.newest[r]) - staleness - g + 1 + j
                if pos >= 0 and self.newest[r] >= 0 and self.fpos[r, pos % self.cap] == pos:
                    out[r, j] = self.feat[r, pos % self.cap]
                    out_pos[r, j] = pos
        return out, out_pos


# ---------------------------------------------------------------------------------------
# Dynamic verification skipping (Sec. 4.4 "Fine-grained Skipped Step Scheduling", Eq. 2, Alg. 1)
#
# What the paper fixes: skip only if the last step was verified; the candidate paths are
# down-sampled with stride 2; S_bar = sum_l w_l S^(l), w_l = alpha^l / sum_k alpha^k, S^(l) the
# cosine similarity of the latent codebook embeddings of the tokens at depth l; skip iff
# S_bar >= T_sim.  Readings where it is silent (**parity unpinned** by the paper): S^(l) is the
# mean cosine over all unordered pairs of the kept paths; the depth L is the shortest kept path
# (deeper tokens are ignored); an embedding of norm 0 has cosine 0 with everything; fewer than
# two kept paths, or depth 0, give S_bar = 1 resp. 0.


def downsample_paths(n_paths: int, stride: int) -> list:
    """Alg. 1, Downsample(C, stride): every stride-th candidate path, starting with the first."""
    return list(range(0, n_paths, stride))


def path_similarity(paths: np.ndarray, path_len: np.ndarray, codebook: np.ndarray, alpha: float,
                    stride: int = 2) -> float:
    """Eq. 2 on the down-sampled paths.  paths int [N, Lmax] codebook indices, path_len int [N],
    codebook float [V, dim] (latent embeddings E)."""
    keep = downsample_paths(len(paths), stride)
    depth = int(min(path_len[i] for i in keep)) if keep else 0
    if depth <= 0:
        return 0.0
    if len(keep) < 2:
        return 1.0
    e = np.asarray(codebook, dtype=np.float64)
    w = np.array([alpha ** l for l in range(depth)], dtype=np.float64)
    w = w / w.sum()
    s_bar = 0.0
    for l in range(depth):
        total, pairs = 0.0, 0
        for a in range(len(keep)):
            for b in range(a + 1, len(keep)):
                x, y = e[paths[keep[a], l]], e[paths[keep[b], l]]
                nx, ny = np.sqrt(np.dot(x, x)), np.sqrt(np.dot(y, y))
                total += np.dot(x, y) / (nx * ny) if nx > 0.0 and ny > 0.0 else 0.0
                pairs += 1
        s_bar += w[l] * (total / pairs)
    return float(s_bar)


def skip_decision(paths, path_len, codebook, alpha: float, threshold: float, last_verified: bool,
                  stride: int = 2):
    """Alg. 1: (bypass verification?, S_bar).  Never two skipped steps in a row."""
    if not last_verified:
        return False, 0.0
    s_bar = path_similarity(np.asarray(paths), np.asarray(path_len), codebook, alpha, stride)
    return bool(s_bar >= threshold), s_bar


# ---------------------------------------------------------------------------------------
# Unverified token selection with truncation (Sec. 4.2, Eq. 3; Alg. 2 "UniformSample")
#
# The paper fixes: a verification-free step draws one candidate path uniformly at random and keeps
# its first gamma = min(L_s, floor(L_bar)) tokens, L_s the length of the drawn path, L_bar the mean
# length over all paths of the pruned tree.  Reading: path index = floor(u * N) for u in (0, 1).


def select_unverified(paths: np.ndarray, path_len: np.ndarray, u: float):
    """Returns (path index, gamma, the gamma kept tokens)."""
    n = len(paths)
    idx = min(n - 1, int(np.floor(float(u) * n)))
    gamma = min(int(path_len[idx]), int(np.floor(np.sum(path_len, dtype=np.int64) / n)))
    return idx, gamma, np.asarray(paths[idx][:gamma])


# ---------------------------------------------------------------------------------------
# Skipped-step scheduling and the decoding loop (Sec. 4.4 first paragraph; Sec. 4.1; Supp. Alg. 2)


def skip_schedule_fixed(step: int, interval: int) -> bool:
    """VVS-U (Sec. 4.4): with a fixed interval i, after i - 1 normally verified steps the i-th
    verification step is skipped.  Steps count from 0, so step t is skipped iff t mod i == i - 1;
    an interval below 2 never skips (two skipped steps in a row are not allowed, Sec. 4.1)."""
    return interval >= 2 and step % interval == interval - 1


def decode_loop(ms, weights: dict, kv_k: np.ndarray, kv_v: np.ndarray, first_token: int, propose, uniforms_of,
                n_tokens: int, k: int, n_cfg: int, cfg_scale: float, schedule, codebook=None, fill0: int = 1,
                fcache_cap: int = 16, gamma_cap: int = 5) -> dict:
    """Supp. Algorithm 2 for one image, with the drafter M_D replaced by the callable `propose`
    (iteration -> drafts [K] codebook indices, q [K, V], candidate paths, path_len, u_select) and the
    uniforms of iteration t given by uniforms_of(t) [1, K + 1].

    Per iteration: Decision (schedule = ("never",) | ("fixed", i) | ("dynamic", threshold, alpha,
    stride), the dynamic rule being Alg. 1 with its no-two-skips guard); if not skipped, ONE target
    pass over [last committed token, the still unverified tokens, the K drafts] (post verification,
    Sec. 4.1: n_forced = 1 + number of unverified tokens, their K/V restored, their features written
    back), Verify, UpdateCache; otherwise UniformSample with truncation (Sec. 4.2) and a Retrieve of
    the gamma most recent features for the drafter (Sec. 4.3).  V_last is read as "the last step was
    verified" and starts False.  The loop ends once n_tokens tokens were generated or the KV cache
    cannot take another block.

    kv_k, kv_v: stored caches [n_layers, n_cfg, H, S, hd], filled to fill0 (the prefilled prompt).
    Returns the generated tokens (embedding-table ids), the per-iteration log, the final fill, the
    float64 caches and the feature cache."""
    kc = [widen(kv_k[:, r]) for r in range(n_cfg)]
    vc = [widen(kv_v[:, r]) for r in range(n_cfg)]
    fc = FeatureCache(n_cfg, fcache_cap, ms.d_model)
    t_max = 1 + gamma_cap + k
    fill, generated, it, stored = fill0, 0, 0, 0
    last_tok, pending, v_last = ms.vocab_offset + int(first_token), [], False
    tokens, log = [], []
    while generated < n_tokens and fill + t_max <= ms.s_max:
        c = propose(it)
        if schedule[0] == "never":
            skip, sim = False, 0.0
        elif schedule[0] == "fixed":
            skip, sim = skip_schedule_fixed(it, int(schedule[1])), 0.0
        else:
            skip, sim = skip_decision(c["paths"], c["path_len"], codebook, schedule[2], schedule[1], v_last,
                                      schedule[3] if len(schedule) > 3 else 2)
        if skip and len(pending) + int(np.max(c["path_len"])) > gamma_cap:
            skip = False      # the next block could not hold more unverified tokens
        if not skip:
            f = 1 + len(pending)
            block = np.array([[last_tok] + pending + [ms.vocab_offset + int(x) for x in c["drafts"]]], dtype=np.int32)
            hidden = np.zeros((n_cfg, f + k, ms.d_model))
            for r in range(n_cfg):
                hidden[r] = target_forward(ms, weights, block[0], kc[r], vc[r], fill)
            out = epilogue(ms, weights, hidden, block[:, f:] - ms.vocab_offset, np.array([k]), f, c["q"][None],
                           uniforms_of(it), n_cfg, cfg_scale)
            n_acc = int(out["accept_len"][0])
            nxt = int(out["next_token"][0]) + ms.vocab_offset
            fc.store(hidden, np.full(n_cfg, fill), np.full(n_cfg, f + n_acc))
            tokens += [int(t) for t in block[0, f:f + n_acc]] + [nxt]
            log.append(("verify", f, n_acc, fill + f + n_acc))
            fill += f + n_acc
            stored += f + n_acc
            generated += n_acc + 1
            last_tok, pending, v_last = nxt, [], True
        else:
            idx, gamma, kept = select_unverified(c["paths"], c["path_len"], c["u_select"])
            g_fetch = min(gamma, gamma_cap, stored)
            feats = fc.fetch(np.ones(1, np.uint8), np.full(n_cfg, g_fetch), 0, gamma_cap) if g_fetch > 0 else None
            pending = pending + [ms.vocab_offset + int(t) for t in kept]
            tokens += [ms.vocab_offset + int(t) for t in kept]
            log.append(("skip", idx, gamma, g_fetch))
            generated += gamma
            v_last = False
            del feats
        it += 1
    return dict(tokens=tokens, log=log, fill=fill, last_token=last_tok, pending=pending, kc=kc, vc=vc, fcache=fc,
                iterations=it)


# ---------------------------------------------------------------------------------------
# Tree verification (Sec. 2 / Sec. 5: the drafter proposes a candidate TREE, EAGLE-2 style; the
# paper verifies it with the target in one pass and walks it with the sequential rule of Sec. 2)
#
# The paper does not print the tree rule.  Reading (**parity unpinned** by the paper; pinned here
# by the lossless identity and by "a tree that is a chain is the chain rule"): multi-round
# speculative sampling over the children of the current node, in index order, the children being
# independent draws from the drafter's distribution q at that node: child x is accepted iff
# u < min(1, p_res(x) / q(x)); after a rejection p_res <- norm(max(0, p_res - q)) and the next
# sibling is tried; when no child is left the next token is drawn from p_res (from the node's own
# target row if it has no children).  Block row t attends the cache and its ancestors only, and
# sits at position fill + depth(t).


def tree_ancestors(parent, t: int) -> list:
    """Block rows on the path root .. t (row 0 is the root; parent[0] = -1)."""
    path = []
    while t >= 0:
        path.append(t)
        t = int(parent[t])
    return path[::-1]


def tree_forward(ms, weights: dict, tokens: np.ndarray, parent: np.ndarray, kc: np.ndarray,
                 vc: np.ndarray, fill: int):
    """Features and keys/values of every node of the candidate tree: node t is the LAST row of
    the plain chain forward over its root path (cache untouched).  Returns h [T, d],
    k_node, v_node [n_layers, H, T, hd]."""
    t_len = len(tokens)
    h = np.zeros((t_len, ms.d_model))
    k_node = np.zeros((ms.n_layers, ms.n_heads, t_len, ms.head_dim))
    v_node = np.zeros_like(k_node)
    for t in range(t_len):
        path = tree_ancestors(parent, t)
        kc_t, vc_t = kc.copy(), vc.copy()
        ht = target_forward(ms, weights, np.asarray(tokens)[path], kc_t, vc_t, fill)
        h[t] = ht[-1]
        slot = fill + len(path) - 1
        k_node[:, :, t] = kc_t[:, :, slot]
        v_node[:, :, t] = vc_t[:, :, slot]
    return h, k_node, v_node


def tree_decide(p32: np.ndarray, draft_tokens: np.ndarray, parent: np.ndarray, n_forced: int,
                q32: np.ndarray, u32: np.ndarray, mode: int = MODE_STRICT, row_ptr=None, col=None,
                k: int = 1, delta: float = float("inf"), adjusted_residual: bool = False) -> dict:
    """Walk of one image's candidate tree.  p32 [T, V] float32 target rows (row t = distribution
    of the token after node t); draft node i = block row n_forced + i carries codebook token
    draft_tokens[i], was drawn from q32[i] (the drafter's distribution at its parent) and is judged
    with u32[i]; u32[K] drives the final sample.  The first residual is the float32 difference (as
    in the chain rule); later rounds work in float64.
    Relaxed mode: the numerator of a child's ratio is the pooled mass of the child and its
    neighbours in the CURRENT residual p_res (the chain's relaxed rule with p_res in the place
    of p); with `adjusted_residual` a rejection subtracts q from the adjusted p_res of the
    rejected child, otherwise from p_res itself."""
    relaxed = mode == MODE_RELAXED
    p32 = np.asarray(p32, dtype=np.float32)
    q32 = np.asarray(q32, dtype=np.float32)
    t_len, k_max = p32.shape[0], len(u32) - 1
    margins = np.full(k_max + 1, np.inf)
    cur, path = n_forced - 1, []
    while True:
        children = [c for c in range(n_forced, t_len) if int(parent[c]) == cur]
        if not children:
            r = p32[cur].astype(np.float64)                      # leaf: the bonus token
            break
        p_res, first_round, accepted = p32[cur].astype(np.float64), True, None
        sample_from = p_res                                      # un-normalised residual of the last rejection
        for c in children:
            i = c - n_forced
            x = int(draft_tokens[i])
            mass = pooled_mass(p_res, x, row_ptr, col, k, delta) if relaxed else float(p_res[x])
            ratio = acceptance_ratio(mass, float(q32[i, x]))
            margins[i] = abs(float(u32[i]) - ratio)
            if float(u32[i]) < ratio:
                accepted = c
                break
            adjust = relaxed and adjusted_residual
            if first_round:
                row = adjusted_target(p32[cur], x, row_ptr, col, k, delta) if adjust else p32[cur]
                r = np.maximum(np.float32(0.0), row - q32[i]).astype(np.float64)        # IEEE float32
            else:
                row = adjusted_target(p_res, x, row_ptr, col, k, delta) if adjust else p_res
                r = np.maximum(0.0, row - q32[i].astype(np.float64))
            z = float(np.sum(r))
            if z > 0.0:                                          # p_res == q numerically: keep p_res
                p_res, sample_from = r / z, r
                first_round = False
        if accepted is None:
            r = sample_from
            break
        path.append(accepted)
        cur = accepted
    token, margins[k_max] = inverse_cdf(r, float(u32[k_max]))
    return {"accept_len": len(path), "accept_path": path, "next_token": int(token), "margins": margins}


def tree_verify(ms, weights: dict, block: np.ndarray, parent: np.ndarray, n_forced: int,
                kv_k: np.ndarray, kv_v: np.ndarray, cache_len: np.ndarray, draft_probs: np.ndarray,
                uniforms: np.ndarray, n_cfg: int, cfg_scale: float, temperature: float = 1.0,
                mode: int = MODE_STRICT, row_ptr=None, col=None, k: int = 1, delta: float = float("inf"),
                adjusted_residual: bool = False) -> dict:
    """One verification step over candidate trees: tree_forward per sequence, guidance and
    softmax per image as in `epilogue`, then tree_decide.  block [B, T] embedding-table ids,
    parent [B, T].  Returns accept_len, accept_path (list per image, block rows), next_token
    (embedding-table id), new_len, target_probs [B, T, V], hidden [R, T, d] and the per-node
    keys/values k_node, v_node [n_layers, R, H, T, hd] (node order, not cache order)."""
    n_images, t_len = block.shape
    n_rows = n_images * n_cfg
    hidden = np.zeros((n_rows, t_len, ms.d_model))
    k_node = np.zeros((ms.n_layers, n_rows, ms.n_heads, t_len, ms.head_dim))
    v_node = np.zeros_like(k_node)
    for r in range(n_rows):
        b = r % n_images
        hidden[r], k_node[:, r], v_node[:, r] = tree_forward(
            ms, weights, block[b], parent[b], widen(kv_k[:, r]), widen(kv_v[:, r]), int(cache_len[r]))
    out = {"accept_len": np.zeros(n_images, np.int32), "next_token": np.zeros(n_images, np.int32),
           "accept_path": [], "margins": np.zeros((n_images, uniforms.shape[1])),
           "target_probs": np.zeros((n_images, t_len, ms.vocab))}
    for b in range(n_images):
        l_c = lm_head_logits(ms, weights, widen(hidden[b]))
        l_u = lm_head_logits(ms, weights, widen(hidden[n_images + b])) if n_cfg == 2 else None
        out["target_probs"][b] = guided_probs(l_c, l_u, cfg_scale, temperature)
        dec = tree_decide(out["target_probs"][b].astype(np.float32), block[b, n_forced:] - ms.vocab_offset,
                          parent[b], n_forced, draft_probs[b], uniforms[b], mode, row_ptr, col, k, delta,
                          adjusted_residual)
        out["accept_len"][b] = dec["accept_len"]
        out["accept_path"].append(dec["accept_path"])
        out["next_token"][b] = dec["next_token"] + ms.vocab_offset
        out["margins"][b] = dec["margins"]
    out["hidden"], out["k_node"], out["v_node"] = hidden, k_node, v_node
    out["new_len"] = np.array([int(cache_len[r]) + n_forced + int(out["accept_len"][r % n_images])
                               for r in range(n_rows)], dtype=np.int32)
    return out
