"""Shared test plumbing: builds seeded verify-step cases, runs them through the oracle and
through the CUDA library (via the C ABI binding), and compares."""
from __future__ import annotations

import numpy as np

from oracle import vvs_oracle as O
from vvs_synth import gen, philox
from vvs_synth.configs import DTYPE_BF16, MODE_RELAXED, MODE_STRICT, ModelShape


def build_case(ms: ModelShape, seed: int, n_images: int, n_cfg: int, n_forced: int, n_draft_max: int,
               fills, cfg_scale: float = 2.0, temperature: float = 1.0, mode: int = MODE_STRICT,
               nbr_k: int = 1, delta: float = float("inf"), q_noise: float = 1.0, n_draft=None,
               kv_rows=None, w_std: float = 0.02, call_id: int = 0):
    """Seeded inputs of one verify call.  Drafts are sampled position by position from a drafter
    whose logits are the oracle's guided target logits plus N(0, q_noise^2), so acceptance is
    neither trivial nor hopeless."""
    n_rows = n_images * n_cfg
    kv_rows = kv_rows or n_rows
    t_len = n_forced + n_draft_max
    w = gen.make_weights(ms, seed, w_std=w_std)
    kv_k, kv_v = gen.make_kv_cache(ms, seed, kv_rows)
    fills = np.asarray(fills, dtype=np.int32)
    cache_len = np.array([fills[r % n_images] for r in range(n_rows)], dtype=np.int32)
    lo, hi = ms.vocab_offset, ms.vocab_offset + ms.vocab
    block = np.zeros((n_images, t_len), dtype=np.int32)
    block[:, :n_forced] = gen.random_tokens(seed, "forced", (n_images, n_forced), lo, hi)
    q = np.zeros((n_images, n_draft_max, ms.vocab), dtype=np.float32)
    for b in range(n_images):
        caches = [(O.widen(kv_k[:, c * n_images + b]), O.widen(kv_v[:, c * n_images + b]))
                  for c in range(n_cfg)]
        for t in range(t_len - 1):
            ls = []
            for c in range(n_cfg):
                h = O.target_forward(ms, w, block[b, t:t + 1], caches[c][0], caches[c][1],
                                     int(cache_len[c * n_images + b]) + t)
                ls.append(O.lm_head_logits(ms, w, h)[0])
            if t >= n_forced - 1:
                i = t - (n_forced - 1)
                l = O.guided_logits(ls[0], ls[1] if n_cfg == 2 else None, cfg_scale) / temperature
                q[b, i], tok = gen.perturbed_draft_row(seed, f"draft.{b}.{i}", l, q_noise)
                block[b, t + 1] = lo + tok
    u = philox.verify_uniforms(seed, call_id, n_images, n_draft_max)
    nd = np.full(n_images, n_draft_max, np.int32) if n_draft is None else np.asarray(n_draft, np.int32)
    case = dict(ms=ms, w=w, kv_k=kv_k, kv_v=kv_v, kv_rows=kv_rows, cache_len=cache_len, block=block,
                draft_probs=q, uniforms=u, n_draft=nd, n_images=n_images, n_cfg=n_cfg,
                n_forced=n_forced, n_draft_max=n_draft_max, cfg_scale=cfg_scale,
                temperature=temperature, mode=mode, nbr_k=nbr_k, delta=delta, row_ptr=None, col=None)
    if mode == MODE_RELAXED:
        case["row_ptr"], case["col"] = gen.neighbour_csr(gen.make_codebook(seed, ms.vocab), nbr_k)
    return case


def build_case_independent(ms: ModelShape, seed: int, n_images: int, n_cfg: int, n_forced: int, n_draft_max: int,
                           fills, cfg_scale: float = 2.0, temperature: float = 1.0, mode: int = MODE_STRICT,
                           nbr_k: int = 1, delta: float = float("inf"), logit_std: float = 1.0, w=None, kv=None,
                           call_id: int = 0):
    """Seeded inputs of one verify call with a drafter that does not look at the target
    (q = softmax(N(0, logit_std^2)), drafts sampled from q): no teacher-forced oracle passes are
    needed to build it, which is what makes the full-depth cases of the large workloads affordable.
    `w` / `kv` may carry weights and caches generated elsewhere (stored bit patterns)."""
    n_rows = n_images * n_cfg
    t_len = n_forced + n_draft_max
    w = gen.make_weights(ms, seed) if w is None else w
    kv_k, kv_v = gen.make_kv_cache(ms, seed, n_rows) if kv is None else kv
    fills = np.asarray(fills, dtype=np.int32)
    cache_len = np.array([fills[r % n_images] for r in range(n_rows)], dtype=np.int32)
    lo, hi = ms.vocab_offset, ms.vocab_offset + ms.vocab
    block = np.zeros((n_images, t_len), dtype=np.int32)
    block[:, :n_forced] = gen.random_tokens(seed, "forced", (n_images, n_forced), lo, hi)
    q, drafts = gen.independent_draft(seed, call_id, n_images, n_draft_max, ms.vocab, logit_std)
    block[:, n_forced:] = lo + drafts
    u = philox.verify_uniforms(seed, call_id, n_images, n_draft_max)
    case = dict(ms=ms, w=w, kv_k=kv_k, kv_v=kv_v, kv_rows=n_rows, cache_len=cache_len, block=block,
                draft_probs=q, uniforms=u, n_draft=np.full(n_images, n_draft_max, np.int32), n_images=n_images,
                n_cfg=n_cfg, n_forced=n_forced, n_draft_max=n_draft_max, cfg_scale=cfg_scale,
                temperature=temperature, mode=mode, nbr_k=nbr_k, delta=delta, row_ptr=None, col=None)
    if mode == MODE_RELAXED:
        case["row_ptr"], case["col"] = gen.neighbour_csr(gen.make_codebook(seed, ms.vocab), nbr_k)
    return case


def run_oracle(case) -> dict:
    c = case
    n_rows = c["n_images"] * c["n_cfg"]
    return O.verify(c["ms"], c["w"], c["block"], c["n_forced"], c["n_draft"], c["kv_k"][:, :n_rows],
                    c["kv_v"][:, :n_rows], c["cache_len"], c["draft_probs"], c["uniforms"],
                    c["n_cfg"], c["cfg_scale"], c["temperature"], c["mode"], c["row_ptr"], c["col"],
                    c["nbr_k"], c["delta"], c.get("adjusted_residual", False))


# ---------------------------------------------------------------------------------------
# device side


def to_dev(a: np.ndarray):
    """numpy storage array -> CUDA tensor (uint16 carries bf16 bit patterns)."""
    import torch
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def to_host(t) -> np.ndarray:
    """CUDA tensor -> float64 / integer numpy array."""
    import torch
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy().astype(np.float64)
    if t.dtype == torch.float32:
        return t.cpu().numpy().astype(np.float64)
    return t.cpu().numpy()


def weights_to_dev(w: dict) -> dict:
    out = {k: to_dev(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: to_dev(v) for k, v in w["layers"][l].items()} for l in sorted(w["layers"])]
    return out


class GpuRunner:
    """Owns a library context plus device copies of one case's weights."""

    def __init__(self, ms: ModelShape, w: dict, max_rows: int, max_block: int, max_nbr_k: int = 1,
                 deterministic: bool = True, chain_kernels: bool = False):
        """chain_kernels: create the context with the library's debug switch that selects the persistent
        whole-chain kernels (and, for 33-64 tokens, the fused-epilogue projections) instead of the
        per-projection kernels; the switch is read when the context is created."""
        import os
        from paper_2511_13587_b200 import binding as vb
        self.vb = vb
        self.ms = ms
        old = os.environ.pop("VVS_DEBUG_CHAIN_KERNELS", None)
        if chain_kernels:
            os.environ["VVS_DEBUG_CHAIN_KERNELS"] = "1"
        try:
            self.ctx = vb.vvs_create(vb.make_desc(ms, max_rows, max_block, max_nbr_k, deterministic))
        finally:
            os.environ.pop("VVS_DEBUG_CHAIN_KERNELS", None)
            if old is not None:
                os.environ["VVS_DEBUG_CHAIN_KERNELS"] = old
        self.wd = weights_to_dev(w)
        vb.vvs_bind_weights(self.ctx, self.wd)

    def close(self):
        self.vb.vvs_destroy(self.ctx)

    def verify(self, case, want_probs=True, want_hidden=True, kv_keep=None) -> dict:
        import torch
        vb, c, ms = self.vb, case, self.ms
        b, cfg, k, f = c["n_images"], c["n_cfg"], c["n_draft_max"], c["n_forced"]
        r, t_len = b * cfg, f + k
        dt = torch.bfloat16 if ms.dtype == DTYPE_BF16 else torch.float32
        if c["row_ptr"] is not None:
            self.rp, self.col = to_dev(c["row_ptr"]), to_dev(c["col"])
            vb.vvs_bind_neighbors(self.ctx, self.rp, self.col)
        kv_k, kv_v = to_dev(c["kv_k"]), to_dev(c["kv_v"])
        o = dict(accept_len=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
                 next_token=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
                 new_len=torch.full((r,), -7, dtype=torch.int32, device="cuda"),
                 accept_mask=torch.full((b, max(k, 1)), 9, dtype=torch.uint8, device="cuda"),
                 margins=torch.zeros((b, k + 1), dtype=torch.float32, device="cuda"),
                 target_probs=torch.zeros((b, t_len, ms.vocab), dtype=torch.float32, device="cuda")
                 if want_probs else None,
                 hidden=torch.zeros((r, t_len, ms.d_model), dtype=dt, device="cuda")
                 if want_hidden else None)
        cache_len = to_dev(c["cache_len"])
        vb.vvs_verify(self.ctx, n_images=b, n_cfg=cfg, n_forced=f, n_draft_max=k,
                      block=to_dev(c["block"]), n_draft=to_dev(c["n_draft"]), kv_k=kv_k, kv_v=kv_v,
                      kv_rows=c["kv_rows"], cache_len=cache_len,
                      draft_probs=to_dev(c["draft_probs"]), uniforms=to_dev(c["uniforms"]),
                      cfg_scale=c["cfg_scale"], temperature=c["temperature"], mode=c["mode"],
                      nbr_k=c["nbr_k"], delta=c["delta"],
                      adjusted_residual=c.get("adjusted_residual", False), **o)
        status = vb.vvs_device_status(self.ctx)
        res = {k_: (to_host(v) if v is not None else None) for k_, v in o.items()}
        res["status"] = status
        res["launches"] = vb.vvs_last_launch_count(self.ctx)
        if kv_keep is None:
            res["kv_k"], res["kv_v"] = to_host(kv_k), to_host(kv_v)
        else:
            # large caches: bring back only the first kv_keep slots, compare the rest on the device
            res["kv_k"], res["kv_v"] = to_host(kv_k[:, :, :, :kv_keep]), to_host(kv_v[:, :, :, :kv_keep])
            res["kv_rest_untouched"] = bool(
                torch.equal(kv_k[:, :, :, kv_keep:], to_dev(c["kv_k"])[:, :, :, kv_keep:]) and
                torch.equal(kv_v[:, :, :, kv_keep:], to_dev(c["kv_v"])[:, :, :, kv_keep:]))
        return res


# ---------------------------------------------------------------------------------------
# comparisons


def replay_decisions(case, gpu_probs: np.ndarray) -> dict:
    """Oracle decision stage on the float32 target probabilities the GPU emitted."""
    c = case
    ms = c["ms"]
    out = dict(accept_len=[], next_token=[], accept_mask=[], margins=[], ratios=[])
    for b in range(c["n_images"]):
        d = O.decide(gpu_probs[b].astype(np.float32), c["block"][b, c["n_forced"]:] - ms.vocab_offset,
                     int(c["n_draft"][b]), c["n_forced"], c["draft_probs"][b], c["uniforms"][b],
                     c["mode"], c["row_ptr"], c["col"], c["nbr_k"], c["delta"], c.get("adjusted_residual", False))
        out["accept_len"].append(d["accept_len"])
        out["next_token"].append(d["next_token"] + ms.vocab_offset if d["next_token"] >= 0 else -1)
        out["accept_mask"].append(d["accept_mask"])
        out["margins"].append(d["margins"])
        out["ratios"].append(d["ratios"])
    return {k: np.array(v) for k, v in out.items()}


def check_replay(case, gpu: dict, margin_tol: float = 1e-4, sample_tol: float = 1e-9):
    """Integer outputs must equal the oracle's decisions on the GPU's own probabilities, except
    where the oracle's margin says the decision sits on a threshold.  Returns the number of
    excluded (near-threshold) images."""
    rep = replay_decisions(case, gpu["target_probs"])
    k = case["n_draft_max"]
    excluded = 0
    for b in range(case["n_images"]):
        near = np.any(rep["margins"][b][:k] < margin_tol)
        if near and gpu["accept_len"][b] != rep["accept_len"][b]:
            excluded += 1
            continue
        assert gpu["accept_len"][b] == rep["accept_len"][b], (b, gpu["accept_len"][b], rep["accept_len"][b])
        np.testing.assert_array_equal(gpu["accept_mask"][b][:k], rep["accept_mask"][b])
        if rep["margins"][b][k] < sample_tol and gpu["next_token"][b] != rep["next_token"][b]:
            excluded += 1
            continue
        assert gpu["next_token"][b] == rep["next_token"][b], (b, gpu["next_token"][b], rep["next_token"][b])
        m = np.minimum(gpu["margins"][b][:k], 1e30)
        np.testing.assert_allclose(m, np.minimum(rep["margins"][b][:k], 1e30), atol=1e-6)
    return excluded


def rel_err_per_row(a: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """||a - ref|| / ||ref|| of every row (last axis)."""
    a2 = a.reshape(-1, a.shape[-1])
    r2 = ref.reshape(-1, ref.shape[-1])
    return np.linalg.norm(a2 - r2, axis=1) / np.linalg.norm(r2, axis=1)


def rel_err_rows(a: np.ndarray, ref: np.ndarray) -> float:
    """max over rows of ||a - ref|| / ||ref||."""
    return float(np.max(rel_err_per_row(a, ref)))


def check_new_cache_rows(case, gpu: dict, ora: dict, rtol: float):
    """K/V appended at slots L..L+T-1 match the oracle; every other slot is untouched."""
    c = case
    ms = c["ms"]
    t_len = c["n_forced"] + c["n_draft_max"]
    k0, v0 = O.widen(c["kv_k"]), O.widen(c["kv_v"])
    for r in range(c["n_images"] * c["n_cfg"]):
        fill = int(c["cache_len"][r])
        for name, got, ref, orig in (("k", gpu["kv_k"], ora["k_new"], k0), ("v", gpu["kv_v"], ora["v_new"], v0)):
            new = got[:, r, :, fill:fill + t_len]
            assert rel_err_rows(new, ref[:, r]) < rtol, (name, r)
            np.testing.assert_array_equal(got[:, r, :, :fill], orig[:, r, :, :fill])
            np.testing.assert_array_equal(got[:, r, :, fill + t_len:], orig[:, r, :, fill + t_len:])
    for r in range(c["n_images"] * c["n_cfg"], c["kv_rows"]):
        np.testing.assert_array_equal(gpu["kv_k"][:, r], k0[:, r])


# ---------------------------------------------------------------------------------------
# candidate trees


def build_tree_case(ms: ModelShape, seed: int, n_images: int, n_cfg: int, n_forced: int, parent,
                    fills, cfg_scale: float = 2.0, temperature: float = 1.0, q_noise: float = 1.0,
                    kv_rows=None, call_id: int = 0):
    """Seeded inputs of one tree verify call.  parent int [T] (shared) or [B, T].  The children of
    a node are independent draws from one drafter row, the oracle's guided target logits at that
    node plus N(0, q_noise^2)."""
    parent = np.asarray(parent, dtype=np.int32)
    if parent.ndim == 1:
        parent = np.tile(parent, (n_images, 1))
    t_len = parent.shape[1]
    k = t_len - n_forced
    n_rows = n_images * n_cfg
    kv_rows = kv_rows or n_rows
    w = gen.make_weights(ms, seed)
    kv_k, kv_v = gen.make_kv_cache(ms, seed, kv_rows)
    fills = np.asarray(fills, dtype=np.int32)
    cache_len = np.array([fills[r % n_images] for r in range(n_rows)], dtype=np.int32)
    lo, hi = ms.vocab_offset, ms.vocab_offset + ms.vocab
    block = np.zeros((n_images, t_len), dtype=np.int32)
    block[:, :n_forced] = gen.random_tokens(seed, "forced", (n_images, n_forced), lo, hi)
    q = np.zeros((n_images, k, ms.vocab), dtype=np.float32)
    for b in range(n_images):
        for pn in range(n_forced - 1, t_len):
            kids = [c for c in range(n_forced, t_len) if parent[b, c] == pn]
            if not kids:
                continue
            path = O.tree_ancestors(parent[b], pn)
            ls = []
            for c in range(n_cfg):
                r = c * n_images + b
                h = O.target_forward(ms, w, block[b][path], O.widen(kv_k[:, r]), O.widen(kv_v[:, r]),
                                     int(cache_len[r]))
                ls.append(O.lm_head_logits(ms, w, h[-1:])[0])
            l = O.guided_logits(ls[0], ls[1] if n_cfg == 2 else None, cfg_scale) / temperature
            q_row, _ = gen.perturbed_draft_row(seed, f"tdraft.{b}.{pn}", l, q_noise)
            for c in kids:
                q[b, c - n_forced] = q_row
                tok = gen.sample_rows(q_row[None, :], gen.rng_for(seed, f"tchild.{b}.{c}").random(1))[0]
                block[b, c] = lo + int(tok)
    u = philox.verify_uniforms(seed, call_id, n_images, k)
    return dict(ms=ms, w=w, kv_k=kv_k, kv_v=kv_v, kv_rows=kv_rows, cache_len=cache_len, block=block,
                parent=parent, draft_probs=q, uniforms=u, n_images=n_images, n_cfg=n_cfg,
                n_forced=n_forced, n_draft_max=k, cfg_scale=cfg_scale, temperature=temperature)


def run_tree_oracle(case) -> dict:
    c = case
    n_rows = c["n_images"] * c["n_cfg"]
    return O.tree_verify(c["ms"], c["w"], c["block"], c["parent"], c["n_forced"], c["kv_k"][:, :n_rows],
                         c["kv_v"][:, :n_rows], c["cache_len"], c["draft_probs"], c["uniforms"],
                         c["n_cfg"], c["cfg_scale"], c["temperature"], c.get("mode", MODE_STRICT), c.get("row_ptr"),
                         c.get("col"), c.get("nbr_k", 1), c.get("delta", float("inf")),
                         c.get("adjusted_residual", False))


def run_tree_gpu(runner: "GpuRunner", case) -> dict:
    import torch
    vb, c, ms = runner.vb, case, runner.ms
    b, cfg, k, f = c["n_images"], c["n_cfg"], c["n_draft_max"], c["n_forced"]
    r, t_len = b * cfg, f + k
    kv_k, kv_v = to_dev(c["kv_k"]), to_dev(c["kv_v"])
    o = dict(accept_len=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             next_token=torch.full((b,), -7, dtype=torch.int32, device="cuda"),
             new_len=torch.full((r,), -7, dtype=torch.int32, device="cuda"),
             n_commit=torch.full((r,), -7, dtype=torch.int32, device="cuda"),
             accept_mask=torch.full((b, max(k, 1)), 9, dtype=torch.uint8, device="cuda"),
             accept_path=torch.full((b, max(k, 1)), -7, dtype=torch.int32, device="cuda"),
             margins=torch.zeros((b, k + 1), dtype=torch.float32, device="cuda"),
             target_probs=torch.zeros((b, t_len, ms.vocab), dtype=torch.float32, device="cuda"),
             hidden=torch.zeros((r, t_len, ms.d_model), dtype=torch.bfloat16, device="cuda"))
    if c.get("row_ptr") is not None:
        rp, col = to_dev(c["row_ptr"]), to_dev(c["col"])
        vb.vvs_bind_neighbors(runner.ctx, rp, col)
    vb.vvs_verify(runner.ctx, n_images=b, n_cfg=cfg, n_forced=f, n_draft_max=k, block=to_dev(c["block"]),
                  kv_k=kv_k, kv_v=kv_v, kv_rows=c["kv_rows"], cache_len=to_dev(c["cache_len"]),
                  draft_probs=to_dev(c["draft_probs"]), uniforms=to_dev(c["uniforms"]),
                  cfg_scale=c["cfg_scale"], temperature=c["temperature"], tree_parent=to_dev(c["parent"]),
                  mode=c.get("mode", MODE_STRICT), nbr_k=c.get("nbr_k", 1), delta=c.get("delta", float("inf")),
                  adjusted_residual=c.get("adjusted_residual", False), **o)
    res = {k_: to_host(v) for k_, v in o.items()}
    res["status"] = vb.vvs_device_status(runner.ctx)
    res["launches"] = vb.vvs_last_launch_count(runner.ctx)
    res["kv_k"], res["kv_v"] = to_host(kv_k), to_host(kv_v)
    return res
