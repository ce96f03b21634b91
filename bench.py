#!/usr/bin/env python
"""Benchmark of the multi-agent PPO hot path: response tokens/s of one step = role-level advantage +
fused LM-head log-prob + PPO-clip/KL forward and backward (dHidden, dW), on synthetic data shaped like
the reflective code-generation workload (H=3584, V=152064, 2 separate models).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload code] [--impl unity|reference]

Prints ONE JSON line (rank 0).  With N > 1 (launched by torch.distributed.run) every rank processes
its own rollout groups (weak scaling); the only exchange is the all-reduce of the per-model valid-row
counts before the step and of dW after it.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "response tokens/s, fused LM-head logprob+PPO fwd+bwd; % of bf16 tensor peak"
UNIT = "tokens/s"


# DRAM traffic of each GEMM class from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum, one launch per
# class) on a cut of the code workload (profiles/k_gemm_code_cut90k.md), as bytes per logit the launch covers
# (valid rows x vocabulary columns).  Traffic grows in proportion to the logits covered (same chunk and group sizes),
# so a full-size launch is estimated as bytes_per_logit x its logits.  Valid only for the kernel source it was taken
# from: when the hash of gemm_tcgen05.cu differs, the benchmark reports null.
NCU_TRAFFIC = {"source_sha256_16": "29857bc22ec90b32",
               "bytes_per_logit": {"fwd_gemm": 1.754, "grad_gemm": 4.006, "dh_gemm": 6.530, "dw_gemm": 6.344}}


def ncu_traffic_per_launch(cls: str, logits_per_launch: float):
    import hashlib
    src = os.path.join(ROOT, "paper_2605_26646_b200", "csrc", "gemm_tcgen05.cu")
    try:
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    if sha != NCU_TRAFFIC["source_sha256_16"] or cls not in NCU_TRAFFIC["bytes_per_logit"]:
        return None
    return NCU_TRAFFIC["bytes_per_logit"][cls] * logits_per_launch


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample_run(w, n_rows, old, ref, adv):
    """Time the fp64 oracle (as it stands) on the first n_rows valid rows of the workload: advantage stage on the
    whole batch + log-prob / loss / backward on the sample.  Returns (seconds, rows)."""
    import numpy as np
    import torch
    from oracle import unity_oracle as orc
    import parity_harness as pu
    rows = torch.nonzero(w.tok_mask)[:n_rows, 0].numpy()
    hid_bits = pu.bf16_bits(w.hidden)
    W_bits = [pu.bf16_bits(x) for x in w.W]
    t0 = time.perf_counter()
    pu.oracle_advantage(w)
    orc.ppo_loss_fwd_bwd(hid_bits, W_bits, w.cu_seqlens.numpy(), w.inv_role.numpy(), w.role_model.numpy(),
                         w.target.numpy(), w.tok_mask.numpy(), np.asarray(old), np.asarray(ref), np.asarray(adv),
                         clip_lo=w.clip_lo, clip_hi=w.clip_hi, kl_coef=w.kl_coef, kl_mode=w.kl_mode,
                         ent_coef=w.ent_coef, inv_temperature=w.inv_temperature, n_roles=w.n_roles, rows=rows)
    return time.perf_counter() - t0, int(rows.size)


def oracle_tiny_run():
    """Time the fp64 oracle on the tiny configuration at full size: advantage, log-prob and loss forward + backward.
    Returns (seconds, valid rows)."""
    import numpy as np
    import torch
    import parity_harness as pu
    from paper_2605_26646_b200 import workloads as wl
    w = wl.make("tiny")
    t0 = time.perf_counter()
    oa = pu.oracle_advantage(w)
    ol = pu.oracle_logprob(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    pu.oracle_ppo(w, (cur + w.noise_old).numpy(), (cur + w.noise_ref).numpy(), oa["adv_tok"].astype(np.float32))
    return time.perf_counter() - t0, int((w.tok_mask != 0).sum().item())


def run_reference(args):
    """The reference arm: the oracle, unmodified, on the host cores, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2605_26646_b200 import workloads as wl
    # the same workload definition; hidden rows are only needed for the sampled rows, so a cut keeps host memory small
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"      # drawing the inputs is not part of the timed work
    w = wl.make(args.workload, device=gen_dev, cut_rows=max(args.ref_rows * 2, 256), cut_max_len=128)
    w.hidden = w.hidden.cpu()
    w.W = [x.cpu() for x in w.W]
    n = w.n_tok
    old = wl.normal(1, 901, n) * 0.05 - 11.0
    ref = wl.normal(1, 902, n) * 0.05 - 11.0
    adv = wl.normal(1, 903, n)
    times = []
    rows = 0
    for i in range(args.warmup + args.steps):
        dt, rows = oracle_sample_run(w, args.ref_rows, old, ref, adv)
        if i >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    val = rows / t
    cores = torch.get_num_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "H": w.H, "V": w.V, "K": w.K, "sample_rows": rows},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{rows} valid rows of the {args.workload} workload per step, fp64 numpy"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def measure_streaming():
    """Streaming stages at a size where they are HBM-bound rather than launch-bound, on 64 Mi tokens: role-level
    advantage (token broadcast), token-level GAE, clipped value loss, delayed-reward alignment and the ready-batch
    gather.  Prints one JSON line with achieved GB/s against the measured copy bandwidth.  Algorithmic bytes per token:
    advantage mask 1 + output 4; GAE rewards, values 8 + mask 1 + two outputs 8; value loss three inputs 12 + mask 1 +
    gradient 4; alignment mask 1 + output 4; gather 2 x row bytes.  Returns the table as a dict."""
    import torch
    from paper_2605_26646_b200 import binding as ub
    from paper_2605_26646_b200 import workloads as wl
    dev = torch.device("cuda", 0)
    n_inv, seq = 1 << 16, 1 << 10
    n = n_inv * seq
    R, G = 4, 2048
    inv_role = wl.randint(3, 1, n_inv, 0, R).to(torch.int32).to(dev)
    inv_group = (torch.arange(n_inv) // (n_inv // G)).to(torch.int32).to(dev)      # 32 consecutive invocations per group
    inv_traj = torch.arange(n_inv, dtype=torch.int32, device=dev)
    r_node = wl.normal(3, 3, n_inv).to(dev)
    cu = (torch.arange(n_inv + 1, dtype=torch.int64) * seq).to(dev)
    mask = (torch.rand(n, device=dev) < 0.8).to(torch.uint8)
    rewards, values = torch.randn(n, device=dev), torch.randn(n, device=dev)
    adv_inv, adv_tok = torch.empty(n_inv, device=dev), torch.empty(n, device=dev)
    a_out, r_out = torch.empty(n, device=dev), torch.empty(n, device=dev)
    ctx = ub.Context(0, 1 << 22)
    peaks = read_peaks()

    def timed(fn, reps=10):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    t_adv = timed(lambda: ctx.role_advantage(n_inv, R, G, inv_role, inv_group, inv_traj, r_node, None, None, None, 1e-6,
                                             0, cu, mask, adv_inv, adv_tok))
    # the same batch with its invocations in a seeded random order (rollout groups interleaved, as in a buffer that
    # fills in arrival order); token data is not moved: only the invocation-level arrays are permuted
    perm = torch.randperm(n_inv, generator=torch.Generator().manual_seed(5)).to(dev)
    role_s, group_s, r_s = inv_role[perm].contiguous(), inv_group[perm].contiguous(), r_node[perm].contiguous()
    t_adv_shuf = timed(lambda: ctx.role_advantage(n_inv, R, G, role_s, group_s, inv_traj, r_s, None, None, None, 1e-6,
                                                  0, cu, mask, adv_inv, adv_tok))
    # the statistics passes alone (same invocations, no tokens): what remains of the call is the token broadcast
    cu0 = torch.zeros(n_inv + 1, dtype=torch.int64, device=dev)
    none_tok = torch.empty(0, device=dev)
    t_adv_stats = timed(lambda: ctx.role_advantage(n_inv, R, G, inv_role, inv_group, inv_traj, r_node, None, None, None,
                                                   1e-6, 0, cu0, None, adv_inv, none_tok))
    # reference for the write-only streams: a plain device fill of the same output
    t_fill = timed(lambda: adv_tok.zero_())
    t_gae = timed(lambda: ctx.gae(cu, rewards, values, mask, 0.99, 0.95, a_out, r_out))
    vloss = torch.empty(R, device=dev)
    t_val = timed(lambda: ctx.value_loss_fwd_bwd(cu, inv_role, list(range(R)), R, mask, values, rewards, r_out, 0.2, None,
                                                 vloss, None, None, a_out))
    t_aln = timed(lambda: ctx.align_rewards(cu, mask, r_node, a_out))
    # ready batch: plan over all invocations (80 % of the trajectories complete), then gather a 4-byte token tensor
    done = (torch.rand(n_inv, device=dev) < 0.8).to(torch.uint8)
    order = torch.empty(n_inv, dtype=torch.int32, device=dev)
    out_cu = torch.empty(n_inv + 1, dtype=torch.int64, device=dev)
    m_off = torch.empty(R + 1, dtype=torch.int32, device=dev)
    p_off = torch.empty(R * 8 + 1, dtype=torch.int32, device=dev)
    totals = torch.empty(2, dtype=torch.int64, device=dev)
    t_plan = timed(lambda: ctx.ready_batch_plan(cu, inv_role, inv_traj, done, list(range(R)), R, 7, 8, 1, order, out_cu,
                                                m_off, p_off, totals))
    t_gat = timed(lambda: ctx.ready_batch_gather(order, cu, out_cu, totals, rewards, r_out, 0.0))
    kept_tok = int(totals[1].item())
    ctx.check_status()
    # Host side of unity_logprob_fwd on the smallest configuration: how long the call keeps the host (it returns once
    # everything is enqueued; nothing in it synchronises) and how long until the result is complete.
    wt = wl.make("tiny", device=dev)
    cxt = ub.Context(0, ub.unity_workspace_bytes(wt.n_tok, wt.H, wt.V, wt.K, wt.n_inv))
    t_cu, t_role, t_tgt, t_mask = wt.cu_seqlens.to(dev), wt.inv_role.to(dev), wt.target.to(dev), wt.tok_mask.to(dev)
    t_logp = torch.empty(wt.n_tok, device=dev)
    ret_us, done_us = [], []
    for i in range(23):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        cxt.logprob_fwd(wt.hidden, wt.W, t_cu, t_role, wt.role_model.tolist(), t_tgt, t_mask, 1.0, t_logp, None, None)
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        t2 = time.perf_counter()
        if i >= 3:
            ret_us.append((t1 - t0) * 1e6)
            done_us.append((t2 - t0) * 1e6)
    cxt.close()
    ret_us.sort()
    done_us.sort()
    out = {"mode": "micro", "tokens": n, "invocations": n_inv, "peak_hbm_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
           "role_advantage": {"ms": t_adv, "algorithmic_bytes": 5 * n + 28 * n_inv, "gbs": (5 * n + 28 * n_inv) / t_adv / 1e6,
                              "ms_shuffled_invocations": t_adv_shuf, "ms_statistics_passes_alone": t_adv_stats,
                              "broadcast_gbs": 5 * n / max(t_adv - t_adv_stats, 1e-6) / 1e6,
                              "broadcast_frac": 5 * n / max(t_adv - t_adv_stats, 1e-6) / 1e6 / peaks["hbm_gbs"]},
           "device_fill_f32": {"ms": t_fill, "algorithmic_bytes": 4 * n, "gbs": 4 * n / t_fill / 1e6,
                               "note": "torch fill of the 256 MiB token vector: what a write-only stream reaches here"},
           "gae": {"ms": t_gae, "algorithmic_bytes": 17 * n, "gbs": 17 * n / t_gae / 1e6},
           "value_loss": {"ms": t_val, "algorithmic_bytes": 17 * n, "gbs": 17 * n / t_val / 1e6},
           "align_rewards": {"ms": t_aln, "algorithmic_bytes": 5 * n, "gbs": 5 * n / t_aln / 1e6},
           "ready_batch_gather_f32": {"ms": t_gat, "algorithmic_bytes": 8 * kept_tok, "gbs": 8 * kept_tok / t_gat / 1e6},
           "ready_batch_plan": {"ms": t_plan, "note": "latency-bound: four small launches over the invocations"},
           "logprob_fwd_tiny_host": {"call_returns_after_us": ret_us[len(ret_us) // 2], "complete_after_us": done_us[len(done_us) // 2],
                                     "note": "median of 20 calls on the tiny configuration; the call is asynchronous (no stream "
                                             "synchronisation; UNITY_OPT_HOST_COUNTS = 0)"}}
    for k in ("role_advantage", "device_fill_f32", "gae", "value_loss", "align_rewards", "ready_batch_gather_f32"):
        out[k]["frac"] = out[k]["gbs"] / peaks["hbm_gbs"]
    ctx.close()
    return out


def run_micro(args):
    print(json.dumps(measure_streaming()), flush=True)


class Job:
    """One configuration set up for timing: seeded inputs resident on the device, a context with its workspace, output
    buffers, and `step()` = unity_role_advantage + unity_ppo_loss_fwd_bwd (+ the dW all-reduce when world > 1)."""

    def __init__(self, workload, dev, rank=0, world=1, stash_room=False, opts=(), ctas=(), cut_rows=0):
        import torch
        import torch.distributed as dist
        from paper_2605_26646_b200 import binding as ub
        from paper_2605_26646_b200 import sharding
        from paper_2605_26646_b200 import workloads as wl
        self.world, self.dev = world, dev
        kw = dict(seed_offset=1000 * rank)
        if cut_rows:
            kw.update(cut_rows=cut_rows)
        w = self.w = wl.make(workload, device=dev, **kw)
        n, H, V, K = w.n_tok, w.H, w.V, w.K
        self.d_inv_role, self.d_inv_group, self.d_inv_traj = w.inv_role.to(dev), w.inv_group.to(dev), w.inv_traj.to(dev)
        self.d_rn, self.d_rt, self.d_rj = w.r_node.to(dev), w.r_turn.to(dev), w.r_traj.to(dev)
        self.d_cu, self.d_mask, self.d_tgt = w.cu_seqlens.to(dev), w.tok_mask.to(dev), w.target.to(dev)
        self.role_model = w.role_model.tolist()
        self.lam = w.lam.tolist()
        ws_bytes = ub.unity_workspace_bytes(n, H, V, K, w.n_inv)
        if stash_room:      # room for the optional logit stash too (reported as an extra; the headline step never uses it)
            ws_bytes = max(ws_bytes, ub.unity_workspace_bytes_stash(n, H, V, K, w.n_inv))
        extra = 0
        mults = {6: 2, 7: 2}
        mults.update({o: v for o, v in opts if o in (6, 7)})
        if (mults[6], mults[7]) != (2, 2):         # non-default gradient chunks need their own G / dH scratch
            extra = 2 * mults[6] * 18944 * (mults[7] * 18944 + 2048) + 4 * mults[6] * 18944 * H
        ctx = self.ctx = ub.Context(dev.index, ws_bytes + extra)
        for o, v in opts:
            ctx.set_option(o, v)
        for option, value in enumerate(ctas):
            ctx.set_option(option, value)

        self.adv_inv = torch.empty(w.n_inv, device=dev)
        self.adv_tok = torch.empty(n, device=dev)
        self.logp = torch.empty(n, device=dev)
        self.ent = torch.empty(n, device=dev)
        self.loss = torch.empty(K, device=dev)
        self.metrics = torch.empty((K + w.n_roles) * ub.UNITY_N_METRICS, device=dev)
        self.dH = torch.empty(n, H, device=dev, dtype=torch.bfloat16)
        self.dW = [torch.empty(V, H, device=dev) for _ in range(K)]

        # current log-probs (stage 2) give the old / reference log-probs of the batch: logp + N(0, 0.05)
        self.lse0 = torch.empty(n, device=dev)
        ctx.logprob_fwd(w.hidden, w.W, self.d_cu, self.d_inv_role, self.role_model, self.d_tgt, self.d_mask,
                        w.inv_temperature, self.logp, self.ent, self.lse0)
        ctx.check_status()
        self.logp0, self.ent0 = self.logp.clone(), self.ent.clone()
        self.old = self.logp + w.noise_old.to(dev)
        self.ref = self.logp + w.noise_ref.to(dev)

        # per-model valid-row counts: the only quantity the ranks must agree on before the step
        tok_inv = torch.repeat_interleave(torch.arange(w.n_inv), w.cu_seqlens[1:] - w.cu_seqlens[:-1])
        tok_model = w.role_model[w.inv_role.long()[tok_inv]].long()
        counts = sharding.local_counts(tok_model, w.tok_mask, K)
        self.n_valid_local = int(counts.sum().item())
        self.norm = None
        self.n_valid_total = self.n_valid_local
        if world > 1:
            self.norm = sharding.global_norm(counts.to(dev))
            tot = torch.tensor([float(self.n_valid_local)], device=dev, dtype=torch.float64)
            dist.all_reduce(tot)
            self.n_valid_total = int(tot.item())

    def step(self, hid=None, tgt=None, msk=None, o=None, r=None):
        from paper_2605_26646_b200 import sharding
        w, ctx = self.w, self.ctx
        hid = w.hidden if hid is None else hid
        tgt = self.d_tgt if tgt is None else tgt
        msk = self.d_mask if msk is None else msk
        o = self.old if o is None else o
        r = self.ref if r is None else r
        ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, self.d_inv_role, self.d_inv_group, self.d_inv_traj,
                           self.d_rn, self.d_rt, self.d_rj, self.lam, w.adv_eps, w.adv_ddof, self.d_cu, msk,
                           self.adv_inv, self.adv_tok)
        ctx.ppo_loss_fwd_bwd(hid, w.W, self.d_cu, self.d_inv_role, self.role_model, tgt, msk, w.inv_temperature,
                             w.clip_lo, w.clip_hi, w.kl_coef, w.kl_mode, w.ent_coef, self.norm, False, o, r,
                             self.adv_tok, self.loss, self.metrics, self.logp, self.ent, None, self.dH, self.dW)
        if self.world > 1:
            sharding.allreduce_grads(self.dW)

    def sync_all(self):
        import torch
        import torch.distributed as dist
        torch.cuda.synchronize()
        if self.world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def measure(self, steps, warmup, sample_clocks=True):
        """`warmup` untimed steps, then `steps` steps between CUDA events (barrier + synchronize on both sides, maximum
        over ranks), SM clocks sampled meanwhile and every GEMM launch bracketed by the library's own event pairs."""
        import torch
        import torch.distributed as dist
        ctx = self.ctx
        for _ in range(warmup):
            self.step()
        ctx.check_status()
        sampler = ClockSampler(self.dev.index)
        if sample_clocks:
            sampler.start()
        ctx.set_profiling(True)
        launches0 = ctx.launch_count
        self.sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.step()
        e1.record()
        self.sync_all()
        ms_total = e0.elapsed_time(e1)
        launches = ctx.launch_count - launches0
        prof = ctx.get_profile()
        ctx.set_profiling(False)
        clocks = sampler.stop() if sample_clocks else None
        ctx.check_status()
        t = torch.tensor([ms_total], device=self.dev, dtype=torch.float64)
        if self.world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step = float(t.item()) / steps
        return dict(ms_total=ms_total, ms_step=ms_step, value=self.n_valid_total / (ms_step * 1e-3), launches=launches,
                    prof=prof, clocks=clocks)

    def kernel_table(self, prof, steps, ms_total, peak):
        """Per GEMM class: launches, summed device time, share of the timed region, TFLOP/s (2 H V flop per valid row
        and class) and its fraction of `peak`."""
        w = self.w
        kern = {}
        for name in ("fwd_gemm", "grad_gemm", "dh_gemm", "dw_gemm"):
            p = prof[name]
            if p["launches"] == 0:
                continue
            tf = 2.0 * w.H * w.V * self.n_valid_local * steps / (p["ms"] * 1e-3) / 1e12
            kern[name] = {"launches": p["launches"], "ms_total": p["ms"], "share_of_step": p["ms"] / ms_total,
                          "tflops": tf, "frac": tf / peak}
        return kern

    def close(self):
        self.ctx.close()


def measure_other_workload(name, dev, peaks, min_seconds=1.5, max_steps=60):
    """A short leg of another configuration with the headline's call sequence: 3 warm-ups, then at least 5 steps (more
    for a configuration whose step takes milliseconds, so that the clock sampler sees the leg)."""
    job = Job(name, dev)
    job.step()
    job.sync_all()
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    job.step()
    e1.record()
    job.sync_all()
    steps = int(min(max_steps, max(5, min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3))))
    m = job.measure(steps, 3)
    w = job.w
    alg = 6.0 * w.H * w.V * job.n_valid_local / (m["ms_step"] * 1e-3) / 1e12
    kern = job.kernel_table(m["prof"], steps, m["ms_total"], peaks["tflops_sustained"])
    out = {"value": m["value"], "unit": UNIT, "ms_per_step": m["ms_step"], "steps": steps, "warmup": 3 + 2,
           "H": w.H, "V": w.V, "K": w.K, "rows": w.n_tok, "valid_rows": job.n_valid_local, "invocations": w.n_inv,
           "tensor_frac_of_burst_peak_algorithmic_6HV": alg / peaks["tflops_burst"],
           "tensor_frac_of_peak_algorithmic_6HV": alg / peaks["tflops_sustained"],
           "tflops_per_class": {k: v["tflops"] for k, v in kern.items()}, "gpu_launches": int(m["launches"]),
           "clocks": m["clocks"]}
    job.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="code")
    ap.add_argument("--impl", default="unity", choices=["unity", "reference"])
    ap.add_argument("--ref-rows", type=int, default=256, help="valid rows per oracle step (reference arm / cpu baseline)")
    ap.add_argument("--micro", action="store_true", help="measure the streaming stages at an HBM-bound size instead")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ctas", default="", help="CTAs per tile for the fwd,grad,dH,dW GEMMs, e.g. 1,1,2,2 (default: library's)")
    ap.add_argument("--opt", default="", help="library tuning options as id=value,id=value (see UNITY_OPT_* in unity.h)")
    ap.add_argument("--cut-rows", type=int, default=0, help="profile-capture helper: run on a cut of the workload")
    args = ap.parse_args()
    if args.warmup < 3 and args.cut_rows == 0:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.micro:
        return run_micro(args)

    import torch
    import torch.distributed as dist
    from paper_2605_26646_b200 import binding as ub
    from paper_2605_26646_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---------------------------------------------------------------- inputs (each rank: its own rollout groups)
    opts = [tuple(int(x) for x in kv.split("=")) for kv in args.opt.split(",") if kv]
    ctas = [int(x) for x in args.ctas.split(",")] if args.ctas else []
    job = Job(args.workload, dev, rank, world, stash_room=True, opts=opts, ctas=ctas, cut_rows=args.cut_rows)
    w, ctx = job.w, job.ctx
    n, H, V, K = w.n_tok, w.H, w.V, w.K
    d_inv_role, d_inv_group, d_inv_traj = job.d_inv_role, job.d_inv_group, job.d_inv_traj
    d_rn, d_rt, d_rj = job.d_rn, job.d_rt, job.d_rj
    d_cu, d_mask, d_tgt = job.d_cu, job.d_mask, job.d_tgt
    role_model, lam, norm = job.role_model, job.lam, job.norm
    adv_inv, adv_tok, logp, ent, loss, metrics, dH, dW = (job.adv_inv, job.adv_tok, job.logp, job.ent, job.loss,
                                                          job.metrics, job.dH, job.dW)
    logp0, ent0, lse0, old, ref = job.logp0, job.ent0, job.lse0, job.old, job.ref
    n_valid_local, n_valid_total = job.n_valid_local, job.n_valid_total
    step, sync_all = job.step, job.sync_all

    # ---------------------------------------------------------------- timed region (device-resident inputs)
    m = job.measure(args.steps, args.warmup, sample_clocks=(rank == 0))
    ms_total, ms_step, value, launches, prof, clocks = (m["ms_total"], m["ms_step"], m["value"], m["launches"],
                                                         m["prof"], m["clocks"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---------------------------------------------------------------- extra (not the headline): on-policy shortcut
    # First PPO epoch: the current policy equals the old one, so the statistics of the log-prob pass are handed in
    # and the loss call skips its forward sweep (6*H*V instead of 8*H*V executed flop per token).
    shortcut = None
    if not args.no_e2e:
        def short_step():
            ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, d_inv_role, d_inv_group, d_inv_traj, d_rn, d_rt, d_rj,
                               lam, w.adv_eps, w.adv_ddof, d_cu, d_mask, adv_inv, adv_tok)
            ctx.ppo_loss_fwd_bwd(w.hidden, w.W, d_cu, d_inv_role, role_model, d_tgt, d_mask, w.inv_temperature,
                                 w.clip_lo, w.clip_hi, w.kl_coef, w.kl_mode, w.ent_coef, norm, False, old, ref, adv_tok,
                                 loss, metrics, logp, ent, None, dH, dW, logp_in=logp0, entropy_in=ent0, lse_in=lse0)
            if world > 1:
                sharding.allreduce_grads(dW)
        short_step()
        sync_all()
        e0.record()
        for _ in range(2):
            short_step()
        e1.record()
        sync_all()
        t3 = torch.tensor([e0.elapsed_time(e1)], device=dev, dtype=torch.float64)
        if world > 1:
            dist.all_reduce(t3, op=dist.ReduceOp.MAX)
        shortcut = {"value": n_valid_total / (float(t3.item()) / 2 * 1e-3), "unit": UNIT, "steps": 2,
                    "note": "loss call given logp/entropy/lse of unity_logprob_fwd (first PPO epoch): forward sweep skipped"}

    # ---------------------------------------------------------------- extras: the log-prob call alone, and one iteration
    # A PPO iteration of a worker group evaluates old and reference log-probs before the update: advantage +
    # 2 x unity_logprob_fwd + unity_ppo_loss_fwd_bwd.
    fwd_extra = iter_extra = None
    if not args.no_e2e:
        def fwd_call():
            ctx.logprob_fwd(w.hidden, w.W, d_cu, d_inv_role, role_model, d_tgt, d_mask, w.inv_temperature, logp, ent, lse0)
        fwd_call()
        sync_all()
        e0.record()
        for _ in range(2):
            fwd_call()
        e1.record()
        sync_all()
        t_f = e0.elapsed_time(e1) / 2
        e0.record()
        fwd_call()
        fwd_call()
        step(w.hidden, d_tgt, d_mask, old, ref)
        e1.record()
        sync_all()
        t_i = e0.elapsed_time(e1)
        ctx.check_status()
        fwd_extra = {"value": n_valid_local / (t_f * 1e-3), "unit": UNIT, "ms": t_f,
                     "tflops": 2.0 * H * V * n_valid_local / (t_f * 1e-3) / 1e12, "note": "unity_logprob_fwd alone (this rank)"}
        iter_extra = {"value": n_valid_local / (t_i * 1e-3), "unit": UNIT, "ms": t_i,
                      "note": "advantage + 2 x unity_logprob_fwd (old, reference) + unity_ppo_loss_fwd_bwd (this rank)"}

    # ---------------------------------------------------------------- extra (not the headline): logit stash
    # The loss call keeps the bf16 logits of one block of 18432 rows (about 6 GB) and turns them into dL/dz in place
    # instead of recomputing them: 6*H*V executed flop per token.  Same outputs within the parity tolerances.
    stash_extra = None
    if not args.no_e2e:
        ctx.set_option(ub.OPT_LOGIT_STASH, 1)
        step(w.hidden, d_tgt, d_mask, old, ref)
        sync_all()
        e0.record()
        for _ in range(2):
            step(w.hidden, d_tgt, d_mask, old, ref)
        e1.record()
        sync_all()
        ctx.set_option(ub.OPT_LOGIT_STASH, 0)
        ctx.check_status()
        t4 = torch.tensor([e0.elapsed_time(e1)], device=dev, dtype=torch.float64)
        if world > 1:
            dist.all_reduce(t4, op=dist.ReduceOp.MAX)
        stash_extra = {"value": n_valid_total / (float(t4.item()) / 2 * 1e-3), "unit": UNIT, "steps": 2,
                       "note": "UNITY_OPT_LOGIT_STASH: block-bounded bf16 logit stash instead of the recompute GEMM"}

    # ---------------------------------------------------------------- end to end: host buffers, copies timed
    e2e = None
    if not args.no_e2e:
        h_hid = torch.empty(w.hidden.shape, dtype=w.hidden.dtype, pin_memory=True)
        h_hid.copy_(w.hidden)
        h_tgt = w.target.pin_memory()
        h_msk = w.tok_mask.pin_memory()
        h_old = torch.empty(n, pin_memory=True)
        h_old.copy_(old)
        h_ref = torch.empty(n, pin_memory=True)
        h_ref.copy_(ref)
        h_loss = torch.empty(K + metrics.numel(), pin_memory=True)
        # Two sets of device buffers: the inputs of step i+1 are uploaded on a second stream while step i computes, as
        # a training loop that prefetches its next batch does.  Every step's upload and the read-back of its loss and
        # metrics lie inside the timed region; only the first upload cannot overlap anything.
        bufs = [(torch.empty_like(w.hidden), torch.empty_like(d_tgt), torch.empty_like(d_mask), torch.empty_like(old),
                 torch.empty_like(ref)) for _ in range(2)]
        h_in = (h_hid, h_tgt, h_msk, h_old, h_ref)
        h2d = sum(x.numel() * x.element_size() for x in h_in)
        d2h = h_loss.numel() * 4
        main_stream = torch.cuda.current_stream()
        copy_stream = torch.cuda.Stream()
        uploaded = [torch.cuda.Event(), torch.cuda.Event()]
        consumed = [torch.cuda.Event(), torch.cuda.Event()]

        def upload(i):
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(consumed[i % 2])          # the step that last used this set has finished
                for dst, src in zip(bufs[i % 2], h_in):
                    dst.copy_(src, non_blocking=True)
                uploaded[i % 2].record(copy_stream)

        def e2e_run(n_steps):
            upload(0)
            for i in range(n_steps):
                main_stream.wait_event(uploaded[i % 2])
                if i + 1 < n_steps:
                    upload(i + 1)
                step(*bufs[i % 2])
                consumed[i % 2].record(main_stream)
                h_loss[:K].copy_(loss, non_blocking=True)
                h_loss[K:].copy_(metrics, non_blocking=True)
                main_stream.synchronize()                        # the caller reads the loss of every step

        for ev in consumed:
            ev.record(main_stream)
        e2e_run(1)
        sync_all()
        n_e2e = max(1, min(args.steps, 3))
        e0.record()
        e2e_run(n_e2e)
        e1.record()
        sync_all()
        t2 = torch.tensor([e0.elapsed_time(e1)], device=dev, dtype=torch.float64)
        if world > 1:
            dist.all_reduce(t2, op=dist.ReduceOp.MAX)
        e2e = {"value": n_valid_total / (float(t2.item()) / n_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e}
        del h_hid, bufs

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---------------------------------------------------------------- roofline of the dominant kernel class
    peaks = read_peaks()
    peak = peaks["tflops_sustained"]           # kernels timed inside a long step: the sustained figure
    flops_per_tok = 2.0 * H * V                # algorithmic flops of ONE of the four contractions per valid row
    kern = job.kernel_table(prof, args.steps, ms_total, peak)
    dom = max(kern, key=lambda k: kern[k]["ms_total"])
    dp = kern[dom]
    roofline = {"bound": "tensor", "kernel": f"k_gemm<{dom}>", "achieved": dp["tflops"], "peak": peak,
                "unit": "TFLOP/s", "frac": dp["frac"],
                "traffic": ncu_traffic_per_launch(dom, float(V) * n_valid_local * args.steps / dp["launches"]),
                "peak_source": f"{peaks['source']} bf16 GEMM, sustained",
                "flops_per_launch": flops_per_tok * n_valid_local * args.steps / dp["launches"],
                "avg_launch_ms": dp["ms_total"] / dp["launches"],
                "launches_note": "per-launch figures average over every launch of the class, including those whose span "
                                 "of rows was empty and returned at once (the host does not know the row counts)"}
    step_tflops_alg = 6.0 * H * V * n_valid_local / (ms_step * 1e-3) / 1e12
    step_tflops_exe = 8.0 * H * V * n_valid_local / (ms_step * 1e-3) / 1e12

    cpu_baseline = None
    if not args.no_cpu_baseline:
        old_h, ref_h, adv_h = old.cpu().numpy(), ref.cpu().numpy(), adv_tok.cpu().numpy()
        w.hidden = w.hidden.cpu()
        w.W = [x.cpu() for x in w.W]
        # twice the reference arm's per-step sample: one pass of about 12 s on 16 host cores
        dt, rows = oracle_sample_run(w, 2 * args.ref_rows, old_h, ref_h, adv_h)
        cpu_baseline = {"value": rows / dt, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                        "sample": f"{rows} valid rows of the {args.workload} workload (one oracle pass, {dt:.1f} s), fp64 numpy"}
        # and the smallest configuration at full size: advantage, log-prob and loss forward + backward on every row
        dt_t, rows_t = oracle_tiny_run()
        cpu_baseline["tiny_full_size"] = {"value": rows_t / dt_t, "unit": UNIT, "seconds": dt_t,
                                          "sample": f"all {rows_t} valid rows of the tiny workload, all three calls"}

    # ---------------------------------------------------------------- the other configurations and the streaming stages
    # Short legs with the same call sequence (1 GPU only).
    other = streaming = None
    if world == 1 and not args.no_e2e and not args.cut_rows:
        job.close()                                   # releases the workspace; the other tensors are small beside 180 GB
        torch.cuda.empty_cache()
        other = {name: measure_other_workload(name, dev, peaks)
                 for name in ("rag_qa", "search", "stress", "code") if name != args.workload}
        torch.cuda.empty_cache()
        streaming = measure_streaming()

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": args.workload, "H": H, "V": V, "K": K, "n_roles": w.n_roles, "rows": n,
                       "valid_rows": n_valid_local, "invocations": w.n_inv,
                       "l2": "inputs larger than L2 (hidden %.1f GB, W %.1f GB per model)" % (n * H * 2 / 1e9, V * H * 2 / 1e9),
                       "step": "unity_role_advantage + unity_ppo_loss_fwd_bwd",
                       "exchange": "none" if world == 1 else "all-reduce of M_k (before) and dW (after)"},
            "tensor_frac_of_peak_algorithmic_6HV": step_tflops_alg / peak,
            "tensor_frac_of_peak_executed_8HV": step_tflops_exe / peak,
            "tensor_frac_of_burst_peak_algorithmic_6HV": step_tflops_alg / peaks["tflops_burst"],
            "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "kernels": kern,
            "on_policy_shortcut": shortcut, "logit_stash": stash_extra, "logprob_fwd": fwd_extra, "iteration": iter_extra,
            "other_workloads": other, "streaming": streaming, "cpu_baseline": cpu_baseline}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
