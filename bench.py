"""Benchmark of the verify step: `python bench.py --gpus N --steps K --warmup W`.

One step = one pass of the whole hot path over one batch of synthetic input: vvs_verify
(embedding .. acceptance .. residual sample, KV append) followed by the feature-cache store of
the committed rows (and, for workload 2, the fetch for skip-masked images).  Prints ONE JSON
line.  `--impl reference` times the fp64 CPU oracle instead, on a bounded sample.

Multi-GPU: the step has no exchange between images, so N GPUs run N independent replicas
(weak scaling, no collective on the data path); torch.distributed is used only for the barrier
and the max-over-ranks of the device time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from vvs_synth import gen, philox  # noqa: E402
from vvs_synth.configs import CONFIGS, MODE_RELAXED  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum of ONE STEP (all launches of a verify call), summed over an
# ncu capture summarised under profiles/.  Keyed by (workload, fixed-order sums); each entry names the
# kernel sources the step runs and the first 16 hex digits of the SHA-256 over their concatenation when
# the counters were taken: the line reports null, and says why, once any of them has changed.
STEP_SOURCES = ("gemm_tc.cu", "attention_rows.cu", "kernels_generic.cu", "lmhead_tc.cu", "kernels_decide.cu")
NCU_CAPTURES = {
    (1, False): ("1748279beacd934c", 1.5709e+09, "profiles/verify_step_configs1_per_projection_launch_list_and_counters.txt"),
    (1, True): ("1748279beacd934c", 1.5459e+09, "profiles/verify_step_configs1_per_projection_launch_list_and_counters.txt"),
    (2, False): ("1748279beacd934c", 4.4629e+09, "profiles/verify_step_configs2_launch_list_and_counters.txt"),
    (2, True): ("1748279beacd934c", 4.0170e+09, "profiles/verify_step_configs2_launch_list_and_counters.txt"),
}
N_TRIALS = 32           # distinct (fill, block, draft) inputs cycled through the steps
DRAFT_LOGIT_STD = 1.0   # target-independent drafter: q = softmax(N(0, std^2))


def metric_name(wl) -> str:
    shape = {"llamagen": "LlamaGen-XL", "visual_a": "7B visual-AR"}.get(wl.shape.name[:8], wl.shape.name)
    return f"verified draft tokens/sec ({shape}-shaped verify step)"


def replica_seed(seed: int, rank: int) -> int:
    """Replicas draw their own inputs: rank r of a multi-GPU run uses its own seed."""
    return seed + 1000 * rank


def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum of `values` (floats) over all ranks; the identity for one rank."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_value(world: int, drafts_per_step: float, steps: int, ms_total: float) -> float:
    """Whole-job throughput: every replica verifies its own drafts in the (max over ranks) time."""
    return world * drafts_per_step * steps / (ms_total * 1e-3)


def sources_hash() -> str:
    h = hashlib.sha256()
    for name in STEP_SOURCES:
        with open(os.path.join(ROOT, "paper_2511_13587_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(index: int, deterministic: bool, chain_kernels: bool):
    """(DRAM bytes of one step, where they come from), or (None, reason)."""
    e = NCU_CAPTURES.get((index, deterministic))
    if chain_kernels or e is None:
        return None, "no ncu capture of this configuration under profiles/"
    sha, nbytes, summary = e
    if sources_hash() != sha:
        return None, f"{summary} is stale: a kernel source has changed since the capture"
    return nbytes, summary


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------
# synthetic inputs (host side, seeded)


def host_trial(wl, trial: int) -> dict:
    """Inputs of one verify call of workload `wl`: fills, block, draft distributions, uniforms."""
    ms = wl.shape
    b, k, f = wl.n_images, wl.n_draft_max, wl.n_forced
    fills = gen.make_fills(wl.seed, b, wl.fill_lo, wl.fill_hi, trial)
    q, drafts = gen.independent_draft(wl.seed, trial, b, k, ms.vocab, wl.q_noise_std)
    forced = gen.random_tokens(wl.seed, f"forced.{trial}", (b, f), ms.vocab_offset,
                               ms.vocab_offset + ms.vocab)
    block = np.concatenate([forced, drafts + ms.vocab_offset], axis=1).astype(np.int32)
    return dict(cache_len=np.tile(fills, wl.n_cfg).astype(np.int32), block=block, draft_probs=q,
                uniforms=philox.verify_uniforms(wl.seed, trial, b, k),
                n_draft=np.full(b, k, np.int32),
                skip_mask=(gen.rng_for(wl.seed, f"skip.{trial}").random(b) < 0.5).astype(np.uint8),
                # every step commits at least its forced row, so one stale feature is always cached
                gamma=np.ones(b * wl.n_cfg, np.int32))


def algorithmic_bytes(wl, trials) -> dict:
    """Bytes a step must move: every streamed weight once plus the K/V rows attention reads."""
    ms = wl.shape
    weights = ms.streamed_params * 2
    t_len = wl.block_len
    per_pos = ms.n_layers * 2 * ms.d_model * 2                 # K and V, all layers, bf16
    kv = float(np.mean([np.sum(t["cache_len"] + t_len) for t in trials])) * per_pos
    return {"weights": weights, "kv": kv, "total": weights + kv}


# ---------------------------------------------------------------------------------------------
# clocks


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *exc):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.proc.wait()
            self.thread.join(timeout=1)

    def summary(self) -> dict:
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = sorted({n for r in self.rows if len(r) >= 7 for n, v in zip(names, r[3:7])
                          if v.lower().startswith("active")})
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": reasons, "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# the CUDA arm


class VerifyBench:
    """One workload resident on this process's GPU: weights, caches, a library context, the
    seeded trials and the step function that the timed regions repeat."""

    def __init__(self, index: int, rank: int = 0, deterministic: bool = False, n_trials: int = N_TRIALS,
                 draft: str = "target", chain_kernels: bool = False):
        import torch
        from paper_2511_13587_b200 import binding as vb
        from vvs_synth.configs import DTYPE_BF16
        self.torch, self.vb, self.index = torch, vb, index
        self.wl = wl = CONFIGS[index]
        self.ms = ms = wl.shape
        self.b, self.cfg, self.k, self.f = wl.n_images, wl.n_cfg, wl.n_draft_max, wl.n_forced
        self.r, self.t_len = self.b * self.cfg, wl.block_len
        self.relaxed = wl.mode == MODE_RELAXED
        self.seed = seed = replica_seed(wl.seed, rank)
        self.tdt = torch.bfloat16 if ms.dtype == DTYPE_BF16 else torch.float32
        r, t_len, b = self.r, self.t_len, self.b
        dev = self.dev

        # resident state: weights, KV cache, neighbour table, feature cache
        if index == 3:
            # 13 GB of weights: drawn on the device (same distributions as the host generator; the
            # benchmark compares nothing with the oracle, the full-size parity tests do)
            g = torch.Generator(device="cuda").manual_seed(seed)
            shp = gen.weight_shapes(ms)

            def draw(name):
                if name.startswith("norm"):
                    return (1.0 + 0.1 * torch.randn(shp[name], generator=g, device="cuda")).to(torch.bfloat16)
                return (0.02 * torch.randn(shp[name], generator=g, device="cuda")).to(torch.bfloat16)

            wd = {n: draw(n) for n in ("tok_emb", "norm_f", "w_lm")}
            wd["layers"] = [{n: draw(n) for n in gen.LAYER_TENSORS} for _ in range(ms.n_layers)]
        else:
            hw = gen.make_weights(ms, seed)
            wd = {n: dev(v) for n, v in hw.items() if n != "layers"}
            wd["layers"] = [{n: dev(v) for n, v in hw["layers"][l].items()} for l in range(ms.n_layers)]
            del hw
        # cache K/V ~ N(0, 1), drawn on the device (the host generator's distribution)
        g = torch.Generator(device="cuda").manual_seed(seed + 1)
        self.kv_k = torch.empty((ms.n_layers, r, ms.n_heads, ms.s_max, ms.head_dim), dtype=self.tdt, device="cuda")
        self.kv_v = torch.empty_like(self.kv_k)
        for l in range(ms.n_layers):
            self.kv_k[l].copy_(torch.randn(self.kv_k[l].shape, generator=g, device="cuda"))
            self.kv_v[l].copy_(torch.randn(self.kv_v[l].shape, generator=g, device="cuda"))
        # the seeded cache, kept aside: set-up and statistics calls start from it, while the timed
        # calls leave their block rows behind in the live cache like a decoding loop does
        self.kv0_k = self.kv0_v = None
        if index != 0 and draft == "target":
            self.kv0_k, self.kv0_v = self.kv_k.clone(), self.kv_v.clone()
        self.wd = wd
        # chain_kernels: the library's debug switch (read at context creation) that selects the persistent
        # whole-chain kernels of the previous generation for calls of at most 32 tokens
        os.environ.pop("VVS_DEBUG_CHAIN_KERNELS", None)
        if chain_kernels:
            os.environ["VVS_DEBUG_CHAIN_KERNELS"] = "1"
        try:
            self.ctx = vb.vvs_create(vb.make_desc(ms, r, t_len, wl.nbr_k, deterministic=deterministic))
        finally:
            os.environ.pop("VVS_DEBUG_CHAIN_KERNELS", None)
        vb.vvs_bind_weights(self.ctx, wd)
        if self.relaxed:
            rp, col = gen.neighbour_csr(gen.make_codebook(seed, ms.vocab, wl.latent_dim), wl.nbr_k)
            self.rp_d, self.col_d = dev(rp), dev(col)
            vb.vvs_bind_neighbors(self.ctx, self.rp_d, self.col_d)
        cap = 5 + t_len
        self.fc = vb.make_fcache(torch.zeros((r, cap, ms.d_model), dtype=self.tdt, device="cuda"),
                                 torch.zeros((r, cap), dtype=torch.int32, device="cuda"),
                                 torch.zeros((r,), dtype=torch.int32, device="cuda"))
        vb.vvs_feature_cache_reset(self.ctx, self.fc)
        self.out = dict(accept_len=torch.zeros(b, dtype=torch.int32, device="cuda"),
                        next_token=torch.zeros(b, dtype=torch.int32, device="cuda"),
                        new_len=torch.zeros(r, dtype=torch.int32, device="cuda"),
                        n_commit=torch.zeros(r, dtype=torch.int32, device="cuda"),
                        hidden=torch.zeros((r, t_len, ms.d_model), dtype=self.tdt, device="cuda"))
        self.fetch_out = torch.zeros((r, 5, ms.d_model), dtype=self.tdt, device="cuda")
        self.fetch_pos = torch.zeros((r, 5), dtype=torch.int32, device="cuda")
        self.launches = 0
        self.keys = ("cache_len", "block", "draft_probs", "uniforms", "n_draft", "skip_mask", "gamma")
        self.trials = [host_trial(wl, t) for t in range(n_trials)]
        self.dtr = [{n: dev(t[n]) for n in self.keys} for t in self.trials]
        if index == 0 or draft == "independent":
            self.drafter = f"independent softmax(N(0,{wl.q_noise_std}^2))"
        else:
            self._draft_from_target()
            self.drafter = f"softmax(guided target logits + N(0,{wl.q_noise_std}^2)), position by position"

    def dev(self, a):
        torch = self.torch
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    def _verify(self, inp, out, **extra):
        wl = self.wl
        self.vb.vvs_verify(self.ctx, n_images=self.b, n_cfg=self.cfg, n_forced=self.f, n_draft_max=self.k,
                           block=inp["block"], n_draft=inp["n_draft"], kv_k=self.kv_k, kv_v=self.kv_v,
                           kv_rows=self.r, cache_len=inp["cache_len"], draft_probs=inp["draft_probs"],
                           uniforms=inp["uniforms"], cfg_scale=wl.cfg_scale, temperature=wl.temperature,
                           mode=wl.mode, nbr_k=wl.nbr_k, delta=wl.delta, **out, **extra)

    def _draft_from_target(self):
        """Replaces every trial's drafter rows and draft tokens: the row for draft j is the softmax of
        the library's own guided target logits for that position (given the forced tokens and
        drafts 0..j-1) plus N(0, q_noise_std^2) noise, and draft j is sampled from it - K set-up
        calls per trial, outside every timed region."""
        torch, ms, wl = self.torch, self.ms, self.wl
        b, k, f = self.b, self.k, self.f
        g = torch.Generator(device="cuda").manual_seed(self.seed + 2)
        probs = torch.zeros((b, self.t_len, ms.vocab), dtype=torch.float32, device="cuda")
        for inp in self.dtr:
            inp["block"][:, f:] = ms.vocab_offset
            for j in range(k):
                self.restore_cache()
                self._verify(inp, self.out, target_probs=probs)
                lg = torch.log(probs[:, f - 1 + j].clamp_min(1e-30))
                lg = lg + wl.q_noise_std * torch.randn(lg.shape, generator=g, device="cuda")
                qj = torch.softmax(lg, dim=-1)
                inp["draft_probs"][:, j] = qj
                tok = torch.multinomial(qj, 1, generator=g)[:, 0]
                inp["block"][:, f + j] = (ms.vocab_offset + tok).to(torch.int32)
        torch.cuda.synchronize()

    def restore_cache(self):
        if self.kv0_k is not None:
            self.kv_k.copy_(self.kv0_k)
            self.kv_v.copy_(self.kv0_v)

    def step(self, inp, out=None):
        vb, ctx = self.vb, self.ctx
        out = self.out if out is None else out
        self._verify(inp, out)
        if self.relaxed:   # the trials' fill levels are unrelated: start each from an empty feature cache
            vb.vvs_feature_cache_reset(ctx, self.fc)
            self.launches += 1
        vb.vvs_feature_cache_store(ctx, self.fc, out["hidden"], self.t_len, inp["cache_len"], out["n_commit"])
        self.launches += vb.vvs_last_launch_count(ctx) + 1
        if self.relaxed:   # workload 2: skip-masked images reuse cached features
            vb.vvs_feature_cache_fetch(ctx, self.fc, inp["skip_mask"], self.b, inp["gamma"], 5, 0,
                                       self.fetch_out, self.fetch_pos)
            self.launches += 1

    def region(self, steps: int, fn=None) -> float:
        """Device time (ms) of `steps` consecutive steps, events on the launching stream."""
        torch = self.torch
        fn = fn or (lambda i: self.step(self.dtr[i % len(self.dtr)]))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1)

    def acceptance(self, seeded_cache: bool = True) -> dict:
        """Untimed pass over the trials: accepted drafts, bonus-row samples and decisions whose
        uniform lies within 1e-4 of the acceptance ratio.  With `seeded_cache` every call starts
        from the seeded cache the drafter rows were made for; without it the calls see the cache
        as the timed region leaves it (block rows of other trials inside their prefix), where the
        drafter is further from the target."""
        torch = self.torch
        margins = torch.zeros((self.b, self.k + 1), dtype=torch.float32, device="cuda")
        acc = drafted = bonus = near = judged = 0
        for inp in self.dtr:
            if seeded_cache:
                self.restore_cache()
            self._verify(inp, self.out, margins=margins)
            a = self.out["accept_len"]
            acc += int(a.sum().item())
            drafted += int(inp["n_draft"].sum().item())
            bonus += int((a == inp["n_draft"]).sum().item())
            m = margins[:, :self.k]
            judged += int(torch.isfinite(m).sum().item())
            near += int((m < 1e-4).sum().item())
        return {"acceptance_rate": acc / max(drafted, 1), "per_decision_acceptance": acc / max(judged, 1),
                "mean_accept_len": acc / (len(self.dtr) * self.b),
                "bonus_row_samples": bonus, "calls": len(self.dtr) * self.b, "judged": judged,
                "near_threshold": near, "near_threshold_rule": "|u - ratio| < 1e-4"}

    def class_times(self, n_prof: int):
        vb = self.vb
        vb.vvs_profile_enable(self.ctx, True)
        for i in range(n_prof):
            self.step(self.dtr[i % len(self.dtr)])
        cls_ms, cls_n = vb.vvs_profile_read(self.ctx)
        vb.vvs_profile_enable(self.ctx, False)
        return cls_ms, cls_n

    def drafts_per_step(self, steps: int) -> float:
        return float(np.mean([self.trials[i % len(self.trials)]["n_draft"].sum() for i in range(steps)]))

    def roofline(self, cls_ms, cls_n, n_prof: int, pk: dict, ms_step: float) -> dict:
        """The roofline object of the kernel (or kernel set) that dominates the step."""
        ms = self.ms
        alg = algorithmic_bytes(self.wl, self.trials)
        per_step = {"gemm": cls_ms[0] / n_prof, "attention": cls_ms[1] / n_prof,
                    "other": cls_ms[2] / n_prof, "chain": cls_ms[3] / n_prof}
        if cls_n[3] > 0:
            # calls of at most 32 tokens: embedding + all decoder layers are ONE persistent kernel, which
            # streams every layer weight once and reads the K/V rows (the LM head is a separate launch)
            name = "whole-chain kernel (embedding + all decoder layers, one persistent launch)"
            dom_ms = cls_ms[3] / cls_n[3]
            dom_bytes = alg["total"] - ms.vocab * ms.d_model * 2
            dom_launches = cls_n[3] / n_prof
        else:
            # a launch per projection / attention / element-wise stage, each overlapping its programmatic
            # dependents: no single kernel dominates, so the object describes the whole step (all launches
            # of one verify call).  The class times below are taken with events BETWEEN the launches, which
            # removes that overlap: they add up to more than the step and only rank the classes.
            name = "whole step (per-projection GEMM, attention and element-wise launches together)"
            dom_ms, dom_bytes, dom_launches = ms_step, alg["total"], sum(cls_n) / n_prof
        achieved = dom_bytes / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
        return {"kernel": name, "bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / pk["hbm_gbs"], "peak_source": pk["source"],
                "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_ms,
                "launches_per_step": dom_launches, "class_ms_per_step": per_step}

    def close(self):
        self.vb.vvs_destroy(self.ctx)
        self.ctx = None
        self.wd = self.kv_k = self.kv_v = self.kv0_k = self.kv0_v = self.dtr = self.fc = self.out = None
        self.torch.cuda.empty_cache()


def timed_regions(fn_region, steps: int, world: int, barrier, min_ms: float = 500.0, max_repeats: int = 400,
                  device="cuda"):
    """Repeats a `steps`-long timed region (each one bracketed by barrier + synchronize, its device
    time taken as the maximum over ranks) until at least `min_ms` of device time has been
    measured.  Every rank sees the same (all-reduced) region times, so all ranks stop after the
    same region.  Returns the list of region times (ms)."""
    times = []
    while True:
        barrier()
        t = max_over_ranks([fn_region(steps)], world, device=device)[0]
        barrier()
        times.append(t)
        if sum(times) >= min_ms or len(times) >= max_repeats:
            return times


def run_ours(args) -> None:
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    S = VerifyBench(args.workload, rank, bool(args.deterministic), n_trials=args.trials, draft=args.draft,
                    chain_kernels=args.chain_kernels)
    wl, ms, vb = S.wl, S.ms, S.vb
    warm = max(args.warmup, 3)

    # ---- device-resident timing ---------------------------------------------------------------
    for i in range(warm):
        S.step(S.dtr[i % len(S.dtr)])
    barrier()
    S.launches = 0
    with ClockSampler(local) as clocks:
        regions = timed_regions(S.region, args.steps, world, barrier, min_ms=args.min_ms)
    gpu_launches = S.launches // len(regions)
    ms_region = float(np.median(regions))
    status = vb.vvs_device_status(S.ctx)
    drafts_per_step = S.drafts_per_step(args.steps)

    # ---- end to end: host buffers in, host results out, every step ------------------------------
    # The step's inputs sit in ONE pinned host buffer and its results come back in one: a call
    # costs one host->device and one device->host copy whatever the number of arguments.
    def packed(shapes, pinned):
        off, views = 0, {}
        for n, (shape, dtype) in shapes.items():
            views[n] = (off, int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size(), shape, dtype)
            off = (off + views[n][1] + 15) & ~15
        buf = torch.empty(off, dtype=torch.uint8).pin_memory() if pinned else torch.empty(off, dtype=torch.uint8, device="cuda")
        return buf, {n: buf[o:o + nb].view(dt).view(shape) for n, (o, nb, shape, dt) in views.items()}

    in_shapes = {n: (tuple(S.dtr[0][n].shape), S.dtr[0][n].dtype) for n in S.keys}
    res_names = ("accept_len", "next_token", "new_len")
    out_shapes = {n: (tuple(S.out[n].shape), S.out[n].dtype) for n in res_names}
    pin = []
    for t in S.dtr[:8]:
        buf, views = packed(in_shapes, True)
        for n in S.keys:
            views[n].copy_(t[n].cpu())
        pin.append(buf)
    stage_buf, stage = packed(in_shapes, False)
    res_dev_buf, res_dev = packed(out_shapes, False)
    res_host_buf, res_host = packed(out_shapes, True)
    out_e2e = dict(S.out, **res_dev)
    h2d = stage_buf.numel()
    d2h = res_host_buf.numel()

    def step_e2e(i):
        stage_buf.copy_(pin[i % len(pin)], non_blocking=True)
        S.step(stage, out_e2e)
        res_host_buf.copy_(res_dev_buf, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for i in range(3):
        step_e2e(i)
    regions_e2e = timed_regions(lambda n: S.region(n, step_e2e), args.steps, world, barrier, min_ms=args.min_ms)
    ms_e2e = float(np.median(regions_e2e))

    # ---- per-kernel-class timing for the roofline (separate pass, not the headline) -----------
    n_prof = min(args.steps, 8)
    cls_ms, cls_n = S.class_times(n_prof)
    accept_live = S.acceptance(seeded_cache=False)
    accept = S.acceptance()
    accept["live_cache"] = {n: accept_live[n] for n in ("acceptance_rate", "per_decision_acceptance", "mean_accept_len",
                                                        "bonus_row_samples", "near_threshold")}
    status |= vb.vvs_device_status(S.ctx)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    alg = algorithmic_bytes(wl, S.trials)
    ms_step = ms_region / args.steps
    roof = S.roofline(cls_ms, cls_n, n_prof, pk, ms_step)
    roof["traffic"], roof["traffic_source"] = ncu_traffic(args.workload, bool(args.deterministic), args.chain_kernels)
    b, cfg, k, t_len = S.b, S.cfg, S.k, S.t_len
    line = {
        "metric": metric_name(wl),
        "value": aggregate_value(world, drafts_per_step, args.steps, ms_region),
        "unit": "drafts/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
        "repeats": len(regions), "timed_ms": float(np.sum(regions)),
        "ms_per_step": ms_step, "ms_per_step_min": float(np.min(regions)) / args.steps,
        "ms_per_step_max": float(np.max(regions)) / args.steps, "verify_latency_us": ms_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if S.tdt == torch.bfloat16 else "f32",
        "data": "synthetic",
        "config": {"workload": f"configs[{args.workload}] {wl.name}", "n_images": b, "n_cfg": cfg,
                   "n_draft": k, "block_rows": t_len, "fill": f"U[{wl.fill_lo},{wl.fill_hi}] per trial",
                   "trials": len(S.trials), "draft": S.drafter,
                   "sums": "fixed order (bitwise repeatable)" if args.deterministic else "arrival order (split-K adds in L2)",
                   "kernels": "whole-chain kernels (previous generation, debug switch)" if args.chain_kernels
                              else "per-projection kernels",
                   "timing": "median over `repeats` regions of `steps` steps each, every region bracketed by barrier + synchronize",
                   "l2": f"weights streamed per step ({alg['weights'] / 1e9:.2f} GB) exceed the 126 MB L2; no flush needed"
                         if alg["weights"] > 126e6 else "weights fit in L2: a latency case, not a bandwidth case",
                   "parallelism": "replicas only (no collective)"},
        "acceptance": accept,
        "step_hbm": {"algorithmic_bytes": alg["total"], "achieved_gbs": alg["total"] / (ms_step * 1e-3) / 1e9,
                     "frac_of_measured": alg["total"] / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"],
                     "frac_of_8tbs": alg["total"] / (ms_step * 1e-3) / 1e9 / 8000.0},
        "roofline": roof,
        "e2e": {"value": aggregate_value(world, drafts_per_step, args.steps, ms_e2e), "unit": "drafts/s",
                "ms_per_step": ms_e2e / args.steps, "repeats": len(regions_e2e),
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": gpu_launches, "device_status": status, "clocks": clocks.summary(),
    }
    S.close()
    if world == 1 and not args.no_other and args.workload == 1:
        line["other_workloads"] = other_workloads(args, pk)
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, steps=args.cpu_steps)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def quick_measure(index: int, deterministic: bool, steps: int, pk: dict, min_ms: float = 300.0,
                  chain_kernels: bool = False) -> dict:
    """A short device-resident measurement of one workload (one GPU): median step time over
    repeated regions, the step's algorithmic bytes and roofline fraction, acceptance statistics."""
    import torch
    S = VerifyBench(index, 0, deterministic, n_trials=16, chain_kernels=chain_kernels)
    for i in range(3):
        S.step(S.dtr[i % len(S.dtr)])
    torch.cuda.synchronize()
    S.launches = 0
    regions = timed_regions(S.region, steps, 1, torch.cuda.synchronize, min_ms=min_ms)
    launches = S.launches // (len(regions) * steps)
    ms_step = float(np.median(regions)) / steps
    n_prof = min(steps, 8)
    cls_ms, cls_n = S.class_times(n_prof)
    roof = S.roofline(cls_ms, cls_n, n_prof, pk, ms_step)
    alg = algorithmic_bytes(S.wl, S.trials)
    res = {"workload": f"configs[{index}] {S.wl.name}", "ms_per_step": ms_step, "steps": steps, "repeats": len(regions),
           "drafts_per_s": S.drafts_per_step(steps) / (ms_step * 1e-3), "launches_per_step": launches,
           "sums": "fixed order" if deterministic else "arrival order",
           "kernels": "whole-chain (previous generation)" if chain_kernels else "per-projection",
           "algorithmic_bytes": alg["total"], "step_frac_of_measured_hbm": alg["total"] / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"],
           "roofline": {n: roof[n] for n in ("kernel", "achieved", "frac", "ms_per_launch", "class_ms_per_step")},
           "acceptance": S.acceptance(), "device_status": S.vb.vvs_device_status(S.ctx)}
    S.close()
    return res


def other_workloads(args, pk: dict) -> dict:
    """The workloads beside the headline one, each measured briefly on this GPU."""
    out = {"configs[1] fixed-order sums": quick_measure(1, True, 64, pk),
           "configs[1] whole-chain kernel, arrival-order sums": quick_measure(1, False, 64, pk, chain_kernels=True),
           "configs[1] whole-chain kernel, fixed-order sums": quick_measure(1, True, 64, pk, chain_kernels=True),
           "configs[0]": quick_measure(0, False, 256, pk, min_ms=100.0),
           "configs[2]": quick_measure(2, False, 16, pk),
           "configs[2] fixed-order sums": quick_measure(2, True, 16, pk),
           "configs[3]": quick_measure(3, False, 16, pk),
           "configs[3] fixed-order sums": quick_measure(3, True, 16, pk),
           "configs[4]": epilogue_sweep(steps=20, pk=pk)}
    return out


# ---------------------------------------------------------------------------------------------
# the oracle arm (CPU)


def cpu_baseline(wl, steps: int = 2) -> dict:
    """The fp64 numpy oracle, as it stands, on the host cores: `steps` verify steps of one image
    (its cond and uncond sequences) of the workload."""
    from oracle import vvs_oracle as O
    from threadpoolctl import threadpool_info
    ms = wl.shape
    w = gen.make_weights(ms, wl.seed)
    rows = [gen.make_kv_row(ms, wl.seed, c * wl.n_images) for c in range(wl.n_cfg)]
    kv_k = np.stack([x[0] for x in rows], axis=1)
    kv_v = np.stack([x[1] for x in rows], axis=1)
    row_ptr = col = None
    if wl.mode == MODE_RELAXED:
        row_ptr, col = gen.neighbour_csr(gen.make_codebook(wl.seed, ms.vocab, wl.latent_dim), wl.nbr_k)
    times, drafts = [], 0
    for s in range(steps):
        t = host_trial(wl, s)
        cl = np.array([t["cache_len"][c * wl.n_images] for c in range(wl.n_cfg)], np.int32)
        t0 = time.perf_counter()
        O.verify(ms, w, t["block"][:1], wl.n_forced, t["n_draft"][:1], kv_k, kv_v, cl,
                 t["draft_probs"][:1], t["uniforms"][:1], wl.n_cfg, wl.cfg_scale, wl.temperature,
                 wl.mode, row_ptr, col, wl.nbr_k, wl.delta)
        times.append(time.perf_counter() - t0)
        drafts += int(t["n_draft"][0])
    cores = max([i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"] or [1])
    return {"value": drafts / sum(times), "unit": "drafts/s", "cores": cores, "kind": "oracle",
            "sample": f"{steps} verify steps of 1 image ({wl.n_cfg} sequences) of configs[{wl_index(wl)}], "
                      f"numpy fp64, {sum(times):.1f} s", "s_per_step": sum(times) / steps}


def wl_index(wl) -> int:
    return [i for i, w in CONFIGS.items() if w is wl][0]


def run_reference(args) -> None:
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = CONFIGS[args.workload]
    n = max(1, min(args.steps, 3))
    base = cpu_baseline(wl, steps=n)
    line = {"impl": "reference", "metric": metric_name(wl),
            "value": base["value"], "unit": "drafts/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": n, "warmup": 0, "ms_per_step": base["s_per_step"] * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{args.workload}] {wl.name}",
                       "sample": base["sample"]},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": "drafts/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# configs[4]: the acceptance epilogue in isolation (LM head + guidance + softmax + decisions)

# (d, V, B, K, C, mode, neighbour k, drafter noise scale, temperature): every value of every axis
# of the sweep appears at least once; the noise scale skews the drafter against the target so that
# the measured acceptance rates run from a few per cent to above 90 %
SWEEP_POINTS = (
    (1280, 16384, 1, 8, 2, 0, 1, 1.0, 1.0), (1280, 16384, 1, 4, 1, 0, 1, 0.15, 0.5),
    (1280, 16384, 8, 8, 2, 1, 1, 0.5, 1.0), (1280, 16384, 16, 8, 2, 1, 64, 1.0, 1.0),
    (1280, 16384, 32, 8, 2, 0, 1, 2.0, 1.5), (1280, 16384, 8, 16, 2, 1, 1000, 1.5, 1.0),
    (1280, 4096, 64, 16, 2, 1, 64, 3.0, 1.0), (1280, 65536, 32, 4, 2, 0, 1, 0.3, 0.7),
    (4096, 4096, 8, 4, 2, 0, 1, 0.15, 1.0), (4096, 16384, 32, 8, 2, 0, 1, 1.0, 1.2),
    (4096, 65536, 8, 8, 2, 0, 1, 2.0, 1.0), (4096, 65536, 64, 16, 2, 0, 1, 0.5, 1.0),
    (4096, 65536, 64, 16, 1, 0, 1, 1.0, 1.0),
)


def epilogue_sweep(steps: int, pk: dict, only=None) -> dict:
    """Points of the acceptance-epilogue sweep through vvs_epilogue (LM head + guidance + softmax +
    decisions on given features), inputs drawn on the device.  Every point carries its time, the
    LM-head TFLOP/s (2 M d V over the whole call, which runs the LM head, the decision kernels and
    the one-row-per-image second pass), the bytes per second of the codebook stream, each as a
    fraction of the measured peak, and the measured acceptance rate.  The drafter row of a
    position is softmax(log p + scale * Gumbel noise), p the library's own target row.  `only`
    picks one point by its index (for a profiler capture of a single shape)."""
    import torch
    from paper_2511_13587_b200 import binding as vb
    from vvs_synth.configs import ModelShape
    points = []
    csr = {}
    chosen = SWEEP_POINTS if only is None else SWEEP_POINTS[only:only + 1]
    for d, v, b, k, c, mode, nbr_k, noise, temp in chosen:
        ms = ModelShape("epilogue", 0, d, 0, 0, 0, v)
        rows = k + 1
        ctx = vb.vvs_create(vb.make_desc(ms, b * c, rows, max(1, nbr_k)))
        g = torch.Generator(device="cuda").manual_seed(0x56565304)
        w_lm = (torch.randn((v, d), generator=g, device="cuda") * (2.0 / d ** 0.5)).to(torch.bfloat16)
        vb.vvs_bind_weights(ctx, {"w_lm": w_lm, "layers": []})
        if mode == MODE_RELAXED:
            if (v, nbr_k) not in csr:
                rp, col = gen.neighbour_csr(gen.make_codebook(0x56565304, v), nbr_k)
                csr[(v, nbr_k)] = (torch.from_numpy(rp).cuda(), torch.from_numpy(col).cuda())
            vb.vvs_bind_neighbors(ctx, *csr[(v, nbr_k)])
        hidden = torch.randn((b * c, rows, d), generator=g, device="cuda").to(torch.bfloat16)
        q = torch.full((b, k, v), 1.0 / v, dtype=torch.float32, device="cuda")
        drafts = torch.zeros((b, k), dtype=torch.int32, device="cuda")
        u = torch.rand((b, k + 1), generator=g, device="cuda").clamp_(1e-6, 1 - 1e-6)
        nd = torch.full((b,), k, dtype=torch.int32, device="cuda")
        o = dict(accept_len=torch.zeros(b, dtype=torch.int32, device="cuda"),
                 next_token=torch.zeros(b, dtype=torch.int32, device="cuda"))
        kw = dict(hidden_in=hidden, n_rows_per_seq=rows, first_row=0, drafts=drafts, n_images=b, n_cfg=c,
                  n_draft_max=k, n_draft=nd, draft_probs=q, cfg_scale=2.0, temperature=temp, mode=mode,
                  nbr_k=nbr_k, delta=float("inf"))
        # set-up: the target rows of this point, then the skewed drafter and its tokens
        probs = torch.zeros((b, rows, v), dtype=torch.float32, device="cuda")
        vb.vvs_epilogue(ctx, uniforms=u, target_probs=probs, **kw, **o)
        gum = -torch.log(-torch.log(torch.rand((b, k, v), generator=g, device="cuda").clamp_(1e-9, 1 - 1e-9)))
        q.copy_(torch.softmax(torch.log(probs[:, :k].clamp_min(1e-30)) + noise * gum, dim=-1))
        drafts.copy_(torch.multinomial(q.view(b * k, v), 1, generator=g).view(b, k).to(torch.int32))
        del probs, gum

        def call(uu=u):
            vb.vvs_epilogue(ctx, uniforms=uu, **kw, **o)

        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms_call = e0.elapsed_time(e1) / steps
        acc = first = calls = 0                      # acceptance statistics, untimed, fresh uniforms per call
        for _ in range(max(1, 256 // b)):
            uu = torch.rand((b, k + 1), generator=g, device="cuda").clamp_(1e-6, 1 - 1e-6)
            call(uu)
            acc += int(o["accept_len"].sum().item())
            first += int((o["accept_len"] >= 1).sum().item())
            calls += b
        m_rows = b * c * rows
        flops, byts = 2.0 * m_rows * d * v, d * v * 2 + m_rows * d * 2 + b * v * 4
        points.append({"d": d, "V": v, "B": b, "K": k, "C": c, "M": m_rows, "relaxed_k": nbr_k if mode else 0,
                       "temperature": temp, "drafter_noise": noise,
                       "us": ms_call * 1e3, "tflops": flops / ms_call / 1e9,
                       "frac_tensor": flops / ms_call / 1e9 / pk["bf16_tflops"],
                       "gbs": byts / ms_call / 1e6, "frac_hbm": byts / ms_call / 1e6 / pk["hbm_gbs"],
                       "first_draft_acceptance": first / calls, "acceptance_rate": acc / (calls * k),
                       "device_status": vb.vvs_device_status(ctx)})
        vb.vvs_destroy(ctx)
        del w_lm, hidden, q
        torch.cuda.empty_cache()
    # the dynamic skip decision (Alg. 1 / Eq. 2): 16 images, 24 candidate paths of depth 5 each,
    # the 8-dim latent codebook of 16384 codes; latency-bound (one CTA per image, a few hundred
    # dependent-load-limited cosine terms), reported as time per call
    ms = ModelShape("skip", 0, 64, 0, 0, 0, 128)
    ctx = vb.vvs_create(vb.make_desc(ms, 1, 1, 1))
    g = torch.Generator(device="cuda").manual_seed(7)
    cb = torch.randn((16384, 8), generator=g, device="cuda")
    paths = torch.randint(0, 16384, (16, 24, 5), generator=g, device="cuda", dtype=torch.int32)
    dec = torch.zeros(16, dtype=torch.uint8, device="cuda")
    sim = torch.zeros(16, dtype=torch.float32, device="cuda")
    for _ in range(3):
        vb.vvs_skip_decide(ctx, paths, None, cb, None, 2, 0.8, 0.65, dec, sim)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(100):
        vb.vvs_skip_decide(ctx, paths, None, cb, None, 2, 0.8, 0.65, dec, sim)
    e1.record()
    torch.cuda.synchronize()
    skip_us = e0.elapsed_time(e1) * 10.0
    vb.vvs_destroy(ctx)
    return {"metric": "acceptance epilogue in isolation (configs[4] sweep points)", "unit": "us per call",
            "skip_decide": {"images": 16, "paths": 24, "depth": 5, "codebook": [16384, 8], "stride": 2,
                            "us_per_call": skip_us, "bound": "latency (launch + one chain of L2 loads)"},
            "steps": steps, "dtype": "bf16", "data": "synthetic", "peak_source": pk["source"],
            "points": points}


def run_epilogue_sweep(args) -> None:
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    print(json.dumps(epilogue_sweep(args.steps, peaks(), only=args.sweep_point)))


# ---------------------------------------------------------------------------------------------
# Algorithm 2 of the paper as a loop over the library's entry points (one image)


def decoding_loops(ms, seed: int, runs, n_tokens: int = 576, k: int = 8, cfg_scale: float = 2.0,
                   latent_dim: int = 8, warm: bool = True):
    """Times the package's decoding loop (paper_2511_13587_b200.loop.DecodeLoop: Supp. Alg. 2 as a host
    loop over the C-ABI entry points) on model shape `ms` with the synthetic stand-in drafter.
    `runs` = [(name, schedule)], schedule = ("never",) | ("fixed", i) | ("dynamic", threshold, alpha).
    Returns (device status, {name: statistics}).  The drafter is synthetic (q = softmax(N(0,1)), a
    random candidate tree whose paths share a stem), so tokens per forward says nothing about image
    quality or real drafters."""
    import torch
    from paper_2511_13587_b200 import binding as vb
    from paper_2511_13587_b200.loop import DecodeLoop
    from vvs_synth.drafter import SyntheticDrafter
    n_paths, depth, t_max = 12, 5, 1 + 5 + k

    def dev(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    hw = gen.make_weights(ms, seed)
    wd = {n: dev(v) for n, v in hw.items() if n != "layers"}
    wd["layers"] = [{n: dev(v) for n, v in hw["layers"][l].items()} for l in range(ms.n_layers)]
    del hw
    kv_k = torch.randn((ms.n_layers, 2, ms.n_heads, ms.s_max, ms.head_dim), device="cuda").to(torch.bfloat16)
    kv_v = torch.randn_like(kv_k)
    ctx = vb.vvs_create(vb.make_desc(ms, 2, t_max, 1, deterministic=False))
    vb.vvs_bind_weights(ctx, wd)
    codebook = dev(gen.make_codebook(seed, ms.vocab, latent_dim).astype(np.float32))
    drafter = SyntheticDrafter(seed, ms.vocab, k, n_paths=n_paths, depth=depth, logit_std=DRAFT_LOGIT_STD)
    loop = DecodeLoop(ctx, ms, kv_k, kv_v, k, 2, cfg_scale, n_paths, depth, codebook=codebook)
    u_of = lambda it: philox.verify_uniforms(seed, it, 1, k)
    results = {}
    for name, schedule in runs:
        if warm:
            loop.run(drafter.first_token(), drafter.propose, u_of, n_tokens, schedule)   # captures the graphs
        t0 = time.perf_counter()
        r = loop.run(drafter.first_token(), drafter.propose, u_of, n_tokens, schedule)
        dt = time.perf_counter() - t0
        results[name] = {"tokens": r["generated"], "target_forwards": r["target_forwards"],
                         "skipped_steps": r["skipped_steps"], "iterations": r["iterations"],
                         "tokens_per_forward": r["generated"] / max(r["target_forwards"], 1),
                         "tokens_per_s": r["generated"] / dt, "seconds": dt, "final_fill": r["fill"]}
    status = vb.vvs_device_status(ctx)
    vb.vvs_destroy(ctx)
    return status, results


def run_generation_loop(args) -> None:
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = CONFIGS[1]
    runs = (("never skip (plain speculative decoding)", ("never",)),
            ("VVS-U, fixed interval 4", ("fixed", 4)), ("VVS-U, fixed interval 3", ("fixed", 3)),
            ("VVS-U, fixed interval 2", ("fixed", 2)), ("VVS-D, dynamic skip, threshold 0.65", ("dynamic", 0.65, 0.8)))
    status, results = decoding_loops(wl.shape, wl.seed, runs, k=wl.n_draft_max, cfg_scale=wl.cfg_scale,
                                     latent_dim=wl.latent_dim)
    print(json.dumps({"metric": "VVS decoding loop (Alg. 2), one 576-token image, LlamaGen-XL shape, synthetic drafter",
                      "unit": "generated tokens/s (host loop included)", "dtype": "bf16", "data": "synthetic",
                      "device_status": status, "runs": results}))


def run_tree_step(args) -> None:
    """Workload 6: tree calls of the verify step on the configs[1] network (one image with
    guidance, K = 8 nodes: a binary split at the root and below its first child, chains below),
    beside the chain call of the same size.  Drafter rows are target-independent (the cost does
    not depend on them); siblings are independent draws from one row."""
    import torch
    from paper_2511_13587_b200 import binding as vb
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if int(os.environ.get("RANK", "0")) != 0:
        return
    wl = CONFIGS[1]
    ms = wl.shape
    b, cfg, k, f = 1, 2, 8, 1
    r, t_len = b * cfg, f + k
    parent = np.array([[-1, 0, 0, 1, 1, 2, 3, 4, 6]], dtype=np.int32)

    def dev(a):
        a = np.ascontiguousarray(a)
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    hw = gen.make_weights(ms, wl.seed)
    wd = {n: dev(v) for n, v in hw.items() if n != "layers"}
    wd["layers"] = [{n: dev(v) for n, v in hw["layers"][l].items()} for l in range(ms.n_layers)]
    del hw
    g = torch.Generator(device="cuda").manual_seed(wl.seed)
    kv_k = torch.randn((ms.n_layers, r, ms.n_heads, ms.s_max, ms.head_dim), generator=g,
                       device="cuda").to(torch.bfloat16)
    kv_v = torch.randn_like(kv_k)
    ctx = vb.vvs_create(vb.make_desc(ms, r, t_len, 1, deterministic=bool(args.deterministic)))
    vb.vvs_bind_weights(ctx, wd)
    trials = []
    for t in range(N_TRIALS):
        h = host_trial(wl, t)
        q = h["draft_probs"]
        for c in range(f, t_len):                     # siblings share the drafter row of their parent
            first = min(x for x in range(f, t_len) if parent[0, x] == parent[0, c])
            q[:, c - f] = q[:, first - f]
            u = gen.rng_for(wl.seed, f"tree.{t}.{c}").random(1)
            h["block"][:, c] = ms.vocab_offset + gen.sample_rows(q[:, c - f], u)
        trials.append({n: dev(h[n]) for n in ("cache_len", "block", "draft_probs", "uniforms")})
    out = dict(accept_len=torch.zeros(b, dtype=torch.int32, device="cuda"),
               next_token=torch.zeros(b, dtype=torch.int32, device="cuda"),
               new_len=torch.zeros(r, dtype=torch.int32, device="cuda"),
               n_commit=torch.zeros(r, dtype=torch.int32, device="cuda"),
               target_probs=torch.zeros((b, t_len, ms.vocab), dtype=torch.float32, device="cuda"))
    path = torch.zeros((b, k), dtype=torch.int32, device="cuda")
    parent_d = dev(parent)

    def step(inp, tree):
        extra = dict(tree_parent=parent_d, accept_path=path) if tree else {}
        vb.vvs_verify(ctx, n_images=b, n_cfg=cfg, n_forced=f, n_draft_max=k, block=inp["block"], kv_k=kv_k,
                      kv_v=kv_v, kv_rows=r, cache_len=inp["cache_len"], draft_probs=inp["draft_probs"],
                      uniforms=inp["uniforms"], cfg_scale=wl.cfg_scale, temperature=wl.temperature, **out, **extra)

    res = {}
    for name, tree in (("chain", False), ("tree", True)):
        for i in range(max(args.warmup, 3)):
            step(trials[i % N_TRIALS], tree)
        torch.cuda.synchronize()
        acc = 0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.steps):
            step(trials[i % N_TRIALS], tree)
        e1.record()
        torch.cuda.synchronize()
        for i in range(min(args.steps, N_TRIALS)):     # acceptance statistics, untimed
            step(trials[i], tree)
            acc += int(out["accept_len"].sum().item())
        msps = e0.elapsed_time(e1) / args.steps
        res[name] = {"ms_per_step": round(msps, 4), "drafts_per_s": round(b * k / msps * 1e3, 1),
                     "mean_accept_len": round(acc / min(args.steps, N_TRIALS), 3),
                     "launches_per_step": vb.vvs_last_launch_count(ctx)}
    status = vb.vvs_device_status(ctx)
    print(json.dumps({"metric": "verify step on a candidate tree vs a chain, LlamaGen-XL shape, batch 1 with guidance, 8 drafted nodes",
                      "unit": "drafted tokens verified per second", "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "configs[1] network, tree parents " + str(parent[0].tolist()),
                                 "l2": "weights (1.48 GB) exceed L2", "probabilities_written": True},
                      "device_status": status, "runs": res}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)     # ~0.7 s timed region at configs[1]: several clock samples
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, choices=[0, 1, 2, 3, 4, 5, 6])
    ap.add_argument("--sweep-point", type=int, default=None, choices=range(len(SWEEP_POINTS)),
                    help="with --workload 4: run this one point of the sweep only")
    ap.add_argument("--deterministic", type=int, default=0, choices=[0, 1],
                    help="1: fixed-order sums (bitwise repeatable), 0: arrival-order split-K sums (faster)")
    ap.add_argument("--chain-kernels", action="store_true",
                    help="time the persistent whole-chain kernels of the previous generation (calls of at most 32 "
                         "tokens) instead of the per-projection kernels")
    ap.add_argument("--cpu-steps", type=int, default=2)   # 5-16 s of host time at configs[1], depending on the host
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-ms", type=float, default=500.0,
                    help="the --steps-long timed region is repeated until this much device time has been measured "
                         "(the line reports the median region); profiler runs pass a small value")
    ap.add_argument("--trials", type=int, default=N_TRIALS, help="distinct seeded inputs cycled through the steps")
    ap.add_argument("--draft", default="target", choices=["target", "independent"],
                    help="target: drafter rows from the library's own target logits plus noise (K set-up calls per "
                         "trial); independent: rows that ignore the target (no set-up calls: short profiler runs)")
    ap.add_argument("--no-other", action="store_true",
                    help="skip the short measurements of the other workloads that the default line carries")
    args = ap.parse_args()
    if args.workload == 4:
        run_epilogue_sweep(args)
    elif args.workload == 5:
        run_generation_loop(args)
    elif args.workload == 6:
        run_tree_step(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
