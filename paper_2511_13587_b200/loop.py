"""The VVS decoding loop (the paper's Supp. Algorithm 2) as a host-side driver over the C-ABI entry
points, for one image.

Per iteration: the skip decision (never / the fixed-interval schedule VVS-U of Sec. 4.4 / the dynamic
rule of Alg. 1 through vvs_skip_decide); then either ONE target verification of the K drafts behind
the last committed token and the still unverified tokens (vvs_verify with n_forced = 1 + their
number: post verification, Sec. 4.1, restores their K/V and writes their features back through
vvs_feature_cache_store), or a verification-free step (vvs_select_unverified, Sec. 4.2, and a
vvs_feature_cache_fetch of the gamma most recent features for the drafter, Sec. 4.3).  The drafter is
a callable iteration -> proposal; every step of the method runs in the library's kernels, this file
only sequences calls and moves a few integers.

Device buffers are allocated once and reused, so that the library replays its captured graphs."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as vb


def fixed_interval_skips(step: int, interval: int) -> bool:
    """VVS-U: after interval - 1 verified steps the next one is skipped (steps count from 0)."""
    return interval >= 2 and step % interval == interval - 1


class DecodeLoop:
    def __init__(self, ctx: int, ms, kv_k: torch.Tensor, kv_v: torch.Tensor, k: int, n_cfg: int, cfg_scale: float,
                 n_paths: int, depth: int, codebook: torch.Tensor | None = None, fcache_cap: int = 16,
                 gamma_cap: int = 5):
        self.ctx, self.ms, self.kv_k, self.kv_v = ctx, ms, kv_k, kv_v
        self.k, self.n_cfg, self.cfg_scale, self.gamma_cap = k, n_cfg, cfg_scale, gamma_cap
        self.n_paths, self.depth, self.codebook = n_paths, depth, codebook
        self.t_max = 1 + gamma_cap + k
        dt = kv_k.dtype
        dev = kv_k.device
        z = lambda shape, dtype: torch.zeros(shape, dtype=dtype, device=dev)
        self.fc = vb.make_fcache(z((n_cfg, fcache_cap, ms.d_model), dt), z((n_cfg, fcache_cap), torch.int32),
                                 z((n_cfg,), torch.int32))
        self.out = dict(accept_len=z(1, torch.int32), next_token=z(1, torch.int32), new_len=z(n_cfg, torch.int32),
                        n_commit=z(n_cfg, torch.int32))
        self.hid = {t: z((n_cfg, t, ms.d_model), dt) for t in range(1 + k, self.t_max + 1)}
        self.block = z(self.t_max, torch.int32)
        self.cache_len = z(n_cfg, torch.int32)
        self.u = z((1, k + 1), torch.float32)
        self.q = z((1, k, ms.vocab), torch.float32)
        self.paths = z((1, n_paths, depth), torch.int32)
        self.path_len = z((1, n_paths), torch.int32)
        self.v_last = z(1, torch.uint8)
        self.u_sel = z(1, torch.float32)
        self.dec, self.sim = z(1, torch.uint8), z(1, torch.float32)
        self.sel_path, self.sel_gamma, self.sel_tok = z(1, torch.int32), z(1, torch.int32), z((1, depth), torch.int32)
        self.gam = z(n_cfg, torch.int32)
        self.fetch_out, self.fetch_pos = z((n_cfg, gamma_cap, ms.d_model), dt), z((n_cfg, gamma_cap), torch.int32)
        self.skip_all = torch.ones(1, dtype=torch.uint8, device=dev)

    def run(self, first_token: int, propose, uniforms_of, n_tokens: int, schedule, fill0: int = 1) -> dict:
        """schedule = ("never",) | ("fixed", interval) | ("dynamic", threshold, alpha[, stride]).
        Returns tokens (embedding-table ids), the per-iteration log, counters and the final fill."""
        ms, k, ctx = self.ms, self.k, self.ctx
        vb.vvs_feature_cache_reset(ctx, self.fc)
        fill, generated, it, stored, forwards, skips = fill0, 0, 0, 0, 0, 0
        last_tok, pending, v_last = ms.vocab_offset + int(first_token), [], False
        tokens, log = [], []
        while generated < n_tokens and fill + self.t_max <= ms.s_max:
            c = propose(it)
            self.paths.copy_(torch.from_numpy(np.ascontiguousarray(c["paths"][None])))
            self.path_len.copy_(torch.from_numpy(np.ascontiguousarray(c["path_len"][None])))
            if schedule[0] == "never":
                skip = False
            elif schedule[0] == "fixed":
                skip = fixed_interval_skips(it, int(schedule[1]))
            else:
                self.v_last.fill_(1 if v_last else 0)
                vb.vvs_skip_decide(ctx, self.paths, self.path_len, self.codebook, self.v_last,
                                   schedule[3] if len(schedule) > 3 else 2, schedule[2], schedule[1], self.dec, self.sim)
                skip = bool(self.dec.item())
            if skip and len(pending) + int(np.max(c["path_len"])) > self.gamma_cap:
                skip = False      # the next block could not hold more unverified tokens
            if not skip:
                f = 1 + len(pending)
                t_len = f + k
                self.block[:t_len].copy_(torch.tensor([last_tok] + pending + [ms.vocab_offset + int(x) for x in c["drafts"]],
                                                      dtype=torch.int32))
                self.cache_len.fill_(fill)
                self.u.copy_(torch.from_numpy(np.ascontiguousarray(uniforms_of(it), dtype=np.float32)))
                self.q.copy_(torch.from_numpy(np.ascontiguousarray(c["q"][None])))
                vb.vvs_verify(ctx, n_images=1, n_cfg=self.n_cfg, n_forced=f, n_draft_max=k, block=self.block, n_draft=None,
                              kv_k=self.kv_k, kv_v=self.kv_v, kv_rows=self.n_cfg, cache_len=self.cache_len,
                              draft_probs=self.q, uniforms=self.u, cfg_scale=self.cfg_scale, temperature=1.0, mode=0,
                              nbr_k=1, delta=float("inf"), hidden=self.hid[t_len], **self.out)
                vb.vvs_feature_cache_store(ctx, self.fc, self.hid[t_len], t_len, self.cache_len, self.out["n_commit"])
                n_acc, nxt = int(self.out["accept_len"].item()), int(self.out["next_token"].item())
                tokens += [ms.vocab_offset + int(x) for x in c["drafts"][:n_acc]] + [nxt]
                log.append(("verify", f, n_acc, fill + f + n_acc))
                fill += f + n_acc
                stored += f + n_acc
                generated += n_acc + 1
                last_tok, pending, v_last = nxt, [], True
                forwards += 1
            else:
                self.u_sel.fill_(float(c["u_select"]))
                vb.vvs_select_unverified(ctx, self.paths, self.path_len, self.u_sel, self.sel_path, self.sel_gamma,
                                         self.sel_tok)
                idx, gamma = int(self.sel_path.item()), int(self.sel_gamma.item())
                g_fetch = min(gamma, self.gamma_cap, stored)
                if g_fetch > 0:
                    self.gam.fill_(g_fetch)
                    vb.vvs_feature_cache_fetch(ctx, self.fc, self.skip_all, 1, self.gam, self.gamma_cap, 0, self.fetch_out,
                                               self.fetch_pos)
                kept = [ms.vocab_offset + int(t) for t in self.sel_tok[0, :gamma].tolist()]
                pending = pending + kept
                tokens += kept
                log.append(("skip", idx, gamma, g_fetch))
                generated += gamma
                v_last = False
                skips += 1
            it += 1
        torch.cuda.synchronize()
        return dict(tokens=tokens, log=log, fill=fill, last_token=last_tok, pending=pending, iterations=it,
                    target_forwards=forwards, skipped_steps=skips, generated=generated)
