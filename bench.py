#!/usr/bin/env python
"""Benchmark of the token-level PPO path: response tokens/s and achieved HBM bandwidth.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|opt|...] [--impl ours|reference]

One step is one pass of the whole path over one synthetic batch that is resident in HBM:
log-probs of the actor logits and of the reference logits, the KL-penalised reward, GAE, and the
fused PPO loss forward/backward that writes bf16 dlogits.  The line printed at the end is JSON.

With --workload all (the default) the headline numbers (value, ms_per_step, e2e) are those of the
OPT-shaped workload, exactly K steps timed; the Llama-2-shaped, large-vocabulary and ragged
workloads are then timed the same way with step counts of their own, and every workload gets an
entry in "roofline_by_workload".  Per workload there are two timed passes: the headline pass (K
steps back to back, no events in between, so that each launch overlaps the tail of the one before
it) and a detail pass in which every experience call and every loss call is bracketed by CUDA
events on the launch stream, repeated until at least half a second has been timed.

--impl reference times the float64 CPU oracle (plain C, OpenMP over rows) on the host cores on
the same workload; it is a deliberately slow program, reported as a baseline, not a target.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused logprob+PPO fwd/bwd: logit GB/s vs HBM peak; response tokens/s"
UNIT = "response tokens/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0       # the "roughly 8 TB/s" of the hardware's data sheet, for the second fraction
DETAIL_MIN_MS = 500.0          # the detail pass repeats its K steps until this much has been timed
DETAIL_MIN_LAUNCHES = 20
ALL_WORKLOADS = ("opt", "llama2", "large_vocab", "ragged")
# steps per timed pass of the workloads other than the headline one (about 0.5 s each)
AUX_STEPS = {"llama2": 1000, "large_vocab": 100, "ragged": 120, "gpt2": 1500, "opt": 2000, "tiny": 2000}

# DRAM traffic per launch of the loss kernel (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures, keyed
# by workload; reported only while the kernel sources still hash to the value the captures were taken at, else null.
# The summaries and their commands are profiles/loss_creg_kernel_opt.md and profiles/loss_cring_kernel_large_vocab_8seq.md;
# the large-vocabulary figure is the 8-sequence capture (1050.897 MB + 996.266 MB) times 8, the bench's workload having
# 8 times the rows (rows are independent and streamed once each, so traffic grows in proportion).
NCU_TRAFFIC = {"sources_sha256": "1b545b70514a9280",
               "bytes_per_launch": {"opt": 302417920 + 357586944, "large_vocab": 8 * (1050897000 + 996265984)}}


def sources_digest() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2410_15651_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons of one GPU while a region runs (read-only queries):
    through NVML in a thread of this process every 10 ms, or, where the NVML module is missing, through an
    nvidia-smi child process every 100 ms."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    MASKS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.out = None
        self.thread = None
        self.rows = []          # (sm_mhz, sm_max_mhz, watts, set of active reasons)
        self.how = None

    def _nvml_loop(self, nvml, handle):
        import threading
        self._stop = threading.Event()

        def loop():
            mx = nvml.nvmlDeviceGetMaxClockInfo(handle, nvml.NVML_CLOCK_SM)
            while True:
                try:
                    try:
                        mask = nvml.nvmlDeviceGetCurrentClocksEventReasons(handle)
                    except AttributeError:
                        mask = nvml.nvmlDeviceGetCurrentClocksThrottleReasons(handle)
                    self.rows.append((float(nvml.nvmlDeviceGetClockInfo(handle, nvml.NVML_CLOCK_SM)), float(mx),
                                      nvml.nvmlDeviceGetPowerUsage(handle) / 1000.0,
                                      {n for n, m in self.MASKS.items() if mask & m}))
                except Exception:
                    pass
                if self._stop.wait(0.01):
                    return

        self.thread = threading.Thread(target=loop, daemon=True)
        self.thread.start()

    def start(self):
        try:
            import pynvml as nvml
            nvml.nvmlInit()
            self._nvml_loop(nvml, nvml.nvmlDeviceGetHandleByIndex(self.index))
            self.how = "nvml, 10 ms"
            return
        except Exception:
            self.thread = None
        try:
            self.out = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"], stdout=self.out, stderr=subprocess.DEVNULL)
            self.how = "nvidia-smi, 100 ms"
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.thread is not None:
            self._stop.set()
            self.thread.join(timeout=2)
        elif self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.out.flush()
            for l in open(self.out.name):
                r = l.strip().split(", ")
                try:
                    self.rows.append((float(r[0]), float(r[1]), float(r[2]),
                                      {n for n, v in zip(self.NAMES, r[3:7]) if v.strip().lower() == "active"}))
                except Exception:
                    continue
            os.unlink(self.out.name)
        else:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no NVML module and no nvidia-smi"]}
        sm = sorted(r[0] for r in self.rows)
        reasons = set().union(*[r[3] for r in self.rows]) if self.rows else set()
        bins = {}
        for v in sm:                                       # samples binned by SM clock, 100 MHz wide
            key = "%d-%d" % (int(v // 100) * 100, int(v // 100) * 100 + 99)
            bins[key] = bins.get(key, 0) + 1
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max((r[1] for r in self.rows), default=None),
                "sm_mhz_min": sm[0] if sm else None, "sm_mhz_bins": bins,
                "power_w_max": max((r[2] for r in self.rows), default=None), "samples": len(sm),
                "reasons": sorted(reasons), "sampled_by": self.how}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------ CUDA arm

class Path:
    """All buffers of one step, resident on the device, and the step itself (C-ABI calls only)."""

    def __init__(self, w, batch, dev, fused=True, in_place=False, global_mean=False):
        import torch
        from paper_2410_15651_b200 import binding, parallel
        self.b, self.w, self.binding, self.parallel = batch, w, binding, parallel
        B, T = w.B, w.T
        self.ws = binding.workspace(B, T, dev)
        f = lambda: torch.empty((B, T), dtype=torch.float32, device=dev)
        self.lp_act, self.lp_ref, self.rewards, self.adv, self.ret = f(), f(), f(), f(), f()
        self.exp = binding.Experience(B, T, dev)
        self.exp.lp_actor, self.exp.lp_ref, self.exp.rewards = self.lp_act, self.lp_ref, self.rewards
        self.exp.adv, self.exp.returns = self.adv, self.ret
        self.fused = fused
        self.global_mean = global_mean
        self.batch_loss = None
        # in place: the gradient overwrites the logits it was computed from.  The loss call then gets a copy of
        # the actor logits of its own, so that the experience phase of the next step still reads logits; after
        # the first step that copy holds gradients, which costs the same traffic to read.
        self.loss_logits = batch["actor"].clone() if in_place else batch["actor"]
        self.out = binding.PPOOutputs(self.loss_logits, in_place=in_place)
        self.N = int(batch["lengths"].sum().item())
        # old-policy log-probs = current + N(0, sigma^2) on valid tokens, prepared once outside the timed region
        cur = binding.gather_logprobs(batch["actor"], batch["ids"], batch["lengths"], self.ws)
        mask = torch.arange(T, device=dev)[None, :] < batch["lengths"][:, None]
        self.lp_old = (cur + batch["lp_old_noise"] * mask).contiguous()
        self.launches_per_step = 3 if fused else 5      # kernels of this library per step

    def experience(self):
        b, w, k = self.b, self.w, self.binding
        if self.fused:
            # experience phase in one call; the KL term uses the old-policy log-probs of the workload
            k.experience(b["actor"], b["ref"], b["ids"], b["lengths"], b["score"], b["values_old"], w.beta_kl,
                         w.reward_clip, w.gamma, w.lam, self.ws, self.exp, lp_old=self.lp_old)
        else:
            k.gather_logprobs(b["actor"], b["ids"], b["lengths"], self.ws, self.lp_act)
            k.gather_logprobs(b["ref"], b["ids"], b["lengths"], self.ws, self.lp_ref)
            k.kl_reward(self.lp_old, self.lp_ref, b["score"], b["lengths"], w.beta_kl, w.reward_clip, self.rewards)
            k.gae(self.rewards, b["values_old"], b["lengths"], w.gamma, w.lam, self.adv, self.ret)

    def loss(self):
        b, w, k = self.b, self.w, self.binding
        grad_scale = float(self.N)                       # gradients of the token sum: O(1) entries
        n_local = n_global = self.N
        if self.global_mean:
            # data parallel with one token mean over all ranks: all-reduce of the token counts before the loss call
            n_local, n_global = self.parallel.token_counts(b["lengths"])
            grad_scale = self.parallel.grad_scale_for_global_mean(n_local, n_global, upstream=float(n_global))
        k.ppo_loss_fwd_bwd(self.loss_logits, b["ids"], b["lengths"], self.lp_old, self.adv, b["values_new"],
                           b["values_old"], self.ret, w.clip_eps, w.value_clip, grad_scale, self.ws, self.out)
        if self.global_mean:
            self.batch_loss = self.parallel.combine_losses(self.out.loss, n_local, n_global)

    def step(self, ev=None):
        if ev is not None:
            ev[0].record()
        self.experience()
        if ev is not None:
            ev[1].record()
        self.loss()
        if ev is not None:
            ev[2].record()


def stats(xs):
    xs = sorted(xs)
    n = len(xs)
    return {"median": xs[n // 2], "best": xs[0], "mean": sum(xs) / n, "n": n}


def measure_workload(name, args, K, dev, rank, local_rank, world, with_e2e):
    """Times one workload; returns the pieces of the JSON line that belong to it."""
    import torch
    import torch.distributed as dist
    from paper_2410_15651_b200 import binding, inputs, parallel

    w = inputs.scaled(inputs.WORKLOADS[name], seed=inputs.WORKLOADS[name].seed + 1000 * rank)
    if args.sequences > 0:
        w = inputs.scaled(w, B=args.sequences)
    batch = inputs.make_batch(w, device=dev)
    if args.logits_dtype == "fp16":
        batch["actor"] = batch["actor"].to(torch.float16)
        batch["ref"] = batch["ref"].to(torch.float16)
    path = Path(w, batch, dev, fused=not args.separate_calls, in_place=args.in_place, global_mean=args.global_mean)
    B, T, V = w.B, w.T, w.V
    n_valid = path.N

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        path.step()
    assert binding.poll_status(path.ws) == 0

    # ---- headline pass: exactly K steps, one pair of CUDA events on the launching stream around all of them
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(visible_gpu_index(local_rank))
    sync_all()
    mem_before = (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev))
    sampler.start()
    t0.record()
    for i in range(K):
        path.step()
    t1.record()
    sync_all()
    mem_after = (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev))
    elapsed_ms = t0.elapsed_time(t1)
    assert binding.poll_status(path.ws) == 0

    # ---- detail pass: every experience call and every loss call between events; K steps, repeated until at
    # least DETAIL_MIN_MS have been timed (an event between two launches keeps the second from starting its
    # set-up under the tail of the first, so these steps are a little slower than the headline ones)
    exp_ms, loss_ms, detail_total = [], [], 0.0
    while detail_total < args.detail_ms or len(loss_ms) < min(DETAIL_MIN_LAUNCHES, K if args.detail_ms <= 0 else DETAIL_MIN_LAUNCHES):
        evs = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(3)) for _ in range(K)]
        for i in range(K):
            path.step(evs[i])
        torch.cuda.synchronize(dev)
        for a, b, c in evs:
            exp_ms.append(a.elapsed_time(b))
            loss_ms.append(b.elapsed_time(c))
        detail_total += evs[0][0].elapsed_time(evs[-1][2])
        if len(loss_ms) >= 20000:
            break
    sync_all()
    clocks = sampler.stop()
    assert binding.poll_status(path.ws) == 0
    exp_s, loss_s = stats(exp_ms), stats(loss_ms)

    # whole-job numbers: the slowest rank's time, the tokens of all ranks
    elapsed_ms = parallel.max_over_ranks(elapsed_ms, dev)
    loss_med = parallel.max_over_ranks(loss_s["median"], dev)
    exp_med = parallel.max_over_ranks(exp_s["median"], dev)
    total_tokens = parallel.sum_over_ranks(float(n_valid), dev)
    ms_per_step = elapsed_ms / K
    value = total_tokens / (ms_per_step * 1e-3)

    peak, peak_src = hbm_peak()
    loss_bytes = 2.0 * V * n_valid + 2.0 * V * B * T          # logits read on valid rows + dlogits written on all rows
    exp_bytes = 2 * (2.0 * V * n_valid)                       # actor and reference logits read on valid rows
    step_bytes = loss_bytes + exp_bytes
    achieved = loss_bytes / (loss_med * 1e-3) / 1e9
    exp_achieved = exp_bytes / (exp_med * 1e-3) / 1e9
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    traffic = None
    if NCU_TRAFFIC["sources_sha256"] == sources_digest():
        traffic = NCU_TRAFFIC["bytes_per_launch"].get(name)

    res = {
        "name": name, "value": value, "ms_per_step": ms_per_step, "n_valid": n_valid, "clocks": clocks,
        "launches": path.launches_per_step * K, "B": B, "T": T, "V": V,
        "workspace_bytes": int(path.ws.numel()), "mem": (mem_before, mem_after), "step_bytes": step_bytes,
        "roofline": {
            "bound": "hbm", "kernel": "rlhf_ppo_loss_fwd_bwd (one launch: row kernel with fused finalisation)",
            "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "frac_of_8000": achieved / NOMINAL_HBM_GBS, "peak_source": peak_src, "traffic": traffic,
            "ms_per_launch": loss_med, "ms_per_launch_best": loss_s["best"], "ms_per_launch_mean": loss_s["mean"],
            "launches_timed": loss_s["n"], "algorithmic_bytes_per_launch": loss_bytes,
            "step_gbs": step_gbs, "step_frac": step_gbs / peak,
            "note": ("frac is the loss call alone between two events; gradient lines that it leaves dirty in the "
                     "L2 are written back during the next kernel, so traffic can be below the algorithmic bytes and "
                     "step_frac (all three launches of a step, headline pass) is what a caller sees"),
        },
        "s1": {
            "bound": "hbm", "kernel": "rlhf_experience (dual log-prob kernel + reward/GAE kernel)",
            "achieved": exp_achieved, "peak": peak, "unit": "GB/s", "frac": exp_achieved / peak,
            "frac_of_8000": exp_achieved / NOMINAL_HBM_GBS, "ms_per_call": exp_med,
            "ms_per_call_best": exp_s["best"], "calls_timed": exp_s["n"], "algorithmic_bytes_per_call": exp_bytes,
        },
    }

    if with_e2e:
        # ---- end to end: inputs start in pinned host memory, losses are read back, every step
        host = {k: batch[k].cpu().pin_memory() for k in ("actor", "ref", "ids", "lengths", "values_old",
                                                          "values_new", "score")}
        host["lp_old"] = path.lp_old.cpu().pin_memory()
        loss_host = torch.empty(2, dtype=torch.float32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = loss_host.numel() * 4
        e_steps = max(3, min(20, K))

        def e2e_step():
            for k_ in ("actor", "ref", "ids", "lengths", "values_old", "values_new", "score"):
                batch[k_].copy_(host[k_], non_blocking=True)
            path.lp_old.copy_(host["lp_old"], non_blocking=True)
            path.step()
            loss_host.copy_(path.out.loss, non_blocking=True)

        for _ in range(2):
            e2e_step()
        sync_all()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e_steps):
            e2e_step()
        e1.record()
        sync_all()
        e2e_ms = parallel.max_over_ranks(e0.elapsed_time(e1), dev)
        res["e2e"] = {"value": total_tokens / (e2e_ms / e_steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "steps": e_steps,
                      "note": "bound by the host-to-device copy of the logits; a caller normally has them on the device"}
    del path, batch
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2410_15651_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torch.distributed.run for --gpus > 1")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    binding.lib()                                              # fail here, loudly, if not built
    names = list(ALL_WORKLOADS) if args.workload == "all" else [args.workload]
    results = {}
    for i, name in enumerate(names):
        K = args.steps if i == 0 else (args.aux_steps or AUX_STEPS[name])
        results[name] = measure_workload(name, args, K, dev, rank, local_rank, world, with_e2e=(i == 0))
    head = results[names[0]]

    # the top-level roofline: the workload whose loss launch is furthest below the peak (all have V >= 32000)
    worst = min((r for r in results.values() if r["V"] >= 32000), key=lambda r: r["roofline"]["frac"], default=head)
    roofline = dict(worst["roofline"])
    roofline["workload"] = worst["name"]
    by_workload = {}
    for n, r in results.items():
        by_workload[n] = {"shape": f"B={r['B']} T={r['T']} V={r['V']}", "response_tokens": r["n_valid"],
                          "ms_per_step": r["ms_per_step"], "tokens_per_s": r["value"],
                          "s4": {k: r["roofline"][k] for k in ("achieved", "frac", "frac_of_8000", "ms_per_launch",
                                                               "ms_per_launch_best", "launches_timed", "traffic",
                                                               "algorithmic_bytes_per_launch")},
                          "s1": {k: r["s1"][k] for k in ("achieved", "frac", "frac_of_8000", "ms_per_call",
                                                         "ms_per_call_best", "calls_timed")},
                          "step_gbs": r["roofline"]["step_gbs"], "step_frac": r["roofline"]["step_frac"],
                          "clocks": r["clocks"]}

    B, T, V = head["B"], head["T"], head["V"]
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{head['name']}: B={B} T={T} V={V} {args.logits_dtype} logits, {head['n_valid']} response tokens per GPU",
                   "also_timed": [n for n in names[1:]],
                   "l2": "inputs larger than L2 (%.2f GB touched per step)" % (head["step_bytes"] / 1e9),
                   "multi_gpu": ("one batch shard per rank; token counts all-reduced (NCCL) before the loss call, "
                                 "losses combined by a token-weighted all-reduce after it" if args.global_mean else
                                 "independent batch per rank, no data-path collective"),
                   "dlogits": "in place (over a copy of the logits)" if args.in_place else "separate bf16 [B,T,V] buffer",
                   "workspace_bytes": head["workspace_bytes"], "workspace_bound_16BT_plus_64K": 16 * B * T + 65536,
                   "torch_allocated_bytes_before_after": [head["mem"][0][0], head["mem"][1][0]],
                   "torch_reserved_bytes_before_after": [head["mem"][0][1], head["mem"][1][1]],
                   "calls_per_step": ("rlhf_gather_logprobs x2, rlhf_kl_reward, rlhf_gae, rlhf_ppo_loss_fwd_bwd"
                                      if args.separate_calls else "rlhf_experience, rlhf_ppo_loss_fwd_bwd")},
        "clocks": head["clocks"], "gpu_launches": head["launches"],
        "e2e": head["e2e"],
        "roofline": roofline,
        "roofline_s1": head["s1"],
        "roofline_by_workload": by_workload,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(names[0], budget_s=12.0)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ oracle arm

def oracle_pass(oracle, w, batch_np, seqs):
    """The whole path on the CPU oracle for the listed sequences; returns response tokens processed."""
    import numpy as np
    sl = np.asarray(seqs)
    actor, ref, ids = batch_np["actor"][sl], batch_np["ref"][sl], batch_np["ids"][sl]
    ln = batch_np["lengths"][sl]
    lp_act = oracle.gather_logprobs(actor, ids, ln)
    lp_ref = oracle.gather_logprobs(ref, ids, ln)
    valid = np.arange(w.T)[None, :] < ln[:, None]
    lp_old = np.where(valid, lp_act + batch_np["lp_old_noise"][sl], 0.0)
    r = oracle.kl_reward(lp_old, lp_ref, batch_np["score"][sl], ln, w.beta_kl, w.reward_clip)
    adv, ret = oracle.gae(r, batch_np["values_old"][sl], ln, w.gamma, w.lam)
    n = int(ln.sum())
    out = oracle.ppo_loss(actor, ids, ln, lp_old, adv, batch_np["values_new"][sl], batch_np["values_old"][sl],
                          ret, w.clip_eps, w.value_clip, float(max(n, 1)))
    for i in range(len(sl)):                                    # dlogits of every row, one sequence at a time
        rows = np.arange(i * w.T, (i + 1) * w.T)
        oracle.dlogits_rows(actor, ids, ln, out.g, rows)
    return n


def oracle_inputs(workload: str, n_seq: int):
    import numpy as np
    from paper_2410_15651_b200 import inputs
    w0 = inputs.WORKLOADS[workload]
    w = inputs.scaled(w0, B=min(w0.B, n_seq))
    b = inputs.make_batch(w, device="cpu")
    bn = {k: (inputs.bf16_bits(v) if v.dtype.is_floating_point and v.element_size() == 2 else v.numpy())
          for k, v in b.items()}
    bn["lengths"] = bn["lengths"].astype(np.int32)
    return w, bn


def cpu_baseline(workload: str, budget_s: float):
    """The oracle, as it stands, on a bounded sample of the workload: whole sequences, as many as fit in about
    `budget_s` seconds of wall time with all host threads, then about a third of that again with one thread."""
    import oracle
    oracle.build()
    w, bn = oracle_inputs(workload, n_seq=2)
    all_threads = oracle.num_threads()

    def timed(budget):
        t0 = time.perf_counter()
        oracle_pass(oracle, w, bn, [0])
        dt = time.perf_counter() - t0
        reps = max(1, int(budget / max(dt, 1e-3)))
        t0 = time.perf_counter()
        tokens = 0
        for i in range(reps):
            tokens += oracle_pass(oracle, w, bn, [i % w.B])
        return tokens, reps, time.perf_counter() - t0

    tokens, reps, dt = timed(budget_s)
    oracle.set_num_threads(1)
    tokens1, reps1, dt1 = timed(budget_s / 3)
    oracle.set_num_threads(all_threads)
    return {"value": tokens / dt, "unit": UNIT, "cores": all_threads, "nproc": os.cpu_count(), "kind": "oracle",
            "sample": f"{reps} sequence passes of the {workload} workload (T={w.T}, V={w.V}), "
                      f"{tokens} response tokens, {dt:.1f} s",
            "one_thread": {"value": tokens1 / dt1, "cores": 1,
                           "sample": f"{reps1} sequence passes, {tokens1} response tokens, {dt1:.1f} s"}}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    from paper_2410_15651_b200 import inputs
    name = "opt" if args.workload == "all" else args.workload
    w, bn = oracle_inputs(name, n_seq=2)
    full = inputs.WORKLOADS[name]
    for i in range(min(args.warmup, 2)):
        oracle_pass(oracle, w, bn, [0])
    t0 = time.perf_counter()
    tokens = 0
    steps = min(args.steps, 12)                               # each step: one sequence of the workload
    for i in range(steps):
        tokens += oracle_pass(oracle, w, bn, [i % w.B])
    dt = time.perf_counter() - t0
    value = tokens / dt
    sample = (f"each step = one sequence of the {name} workload (T={w.T}, V={w.V}); "
              f"{steps} steps timed, {tokens} response tokens")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{name}: B={full.B} T={full.T} V={full.V} bf16 logits (sampled by sequence)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "nproc": os.cpu_count(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="all",
                    choices=["all", "tiny", "opt", "llama2", "large_vocab", "ragged", "gpt2"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sequences", type=int, default=0,
                    help="override the number of sequences B of the workload (smaller cases for profiling)")
    ap.add_argument("--aux-steps", type=int, default=0,
                    help="steps per timed pass of the workloads after the first (default: about 0.5 s each)")
    ap.add_argument("--detail-ms", type=float, default=DETAIL_MIN_MS,
                    help="the event-timed pass repeats its steps until so many milliseconds have been timed "
                         "(0: one pass of --steps steps, for runs under a profiler)")
    ap.add_argument("--logits-dtype", default="bf16", choices=["bf16", "fp16"],
                    help="element type of the logits and of their gradient")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--in-place", action="store_true", help="dlogits overwrite the logits given to the loss call")
    ap.add_argument("--separate-calls", action="store_true",
                    help="experience phase as four calls (2 x gather_logprobs, kl_reward, gae) instead of rlhf_experience")
    ap.add_argument("--global-mean", action="store_true",
                    help="with --gpus N: one token mean over all ranks (token counts and losses all-reduced every step)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
