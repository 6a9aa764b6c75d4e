#!/usr/bin/env python
"""Benchmark of the A-3PO hot path: token log-probs fwd -> A-3PO loss fwd+bwd -> log-prob bwd.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 8b|1p5b|8b_packed]

One "step" is one pass of the whole path (a3po_train_step) over one synthetic batch.  The default
workload is the 8B-shaped batch of the paper's second set-up (H=4096, V=151,936, bf16, 64 sequences
x 2048 rows), the largest padded configuration that fits one GPU.  Prints ONE JSON line.

  value      whole-job valid (mask=1) tokens per second, inputs resident in HBM, per-kernel events off
  e2e        same metric through a3po_train_step_host: per-step inputs start in pinned host memory
  roofline   the dominant kernel's achieved TFLOP/s (algorithmic flops / CUDA-event duration of each
             launch, recorded by the library on its launch stream in a second, separately timed loop)
             against the measured bf16 peak
  configs    compact entries for the other named configurations: the 1.5B-shaped batch, the packed
             long-response 8B batch and the loss-only sweep at 2^24 and 2^26 tokens, each timed in
             its own window with its own clock samples
  cpu_baseline  the fp64 oracle timed on this machine's host cores on a bounded row sample

--impl reference times the oracle alone (the paper ships no runnable reference implementation).
With --gpus N > 1 the script starts one process per GPU itself (unless it already runs under
torchrun); every rank runs its own shard of sequences (weak scaling, no data-path collective); timing
is bracketed by barriers and the maximum over ranks is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "logprob+A-3PO loss fwd/bwd tokens/s; % of bf16 TC peak & HBM roofline"

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant GEMM kernel (the forward that keeps the softmax), from
# the one-pass ncu captures of the full-size launches summarised in profiles/step_8b_launch_list_and_dram.md: bytes
# per step over all its launches of the step (the row chunks); divided by the launches of a step for the per-launch
# figure.  Reset an entry to None when the kernel or its rasterisation changes.
NCU_TRAFFIC_PER_STEP = {
    "8b": {"gemm_tn<fwd_logsoftmax+keep>": 21.48e9 + 19.90e9 + 5.90e9 + 4.43e9},
    "1p5b": {"gemm_tn<fwd_logsoftmax+keep>": 0.70e9 + 2.72e9},
    # not captured (the step holds 60 GB and runs 2.6 s): the same kernel on the same 65,536-row chunks as the 8B-shaped
    # capture, whose traffic is per chunk launch; 16 full chunks plus one of 8,207 rows scaled by rows from the
    # 14,545-row launch
    "8b_packed": {"gemm_tn<fwd_logsoftmax+keep>": 16 * (21.48e9 + 19.90e9) + (5.90e9 + 4.43e9) * 8207 / 14545},
}
# Fused loss kernel (profiles/loss_kernel_16Mi_tokens_ncu_full.md): DRAM bytes per token at N = 2^24 (17 B read exactly;
# most of the 4 B of gradient written per token is still in L2 when the kernel ends).
NCU_TRAFFIC_PER_TOKEN_LOSS = {"loss_fwd_bwd": (285.257e6 + 21.87e6) / 16777216}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
LONG_REGION_S = 2.0      # a timed region longer than this runs under the power cap: the sustained peak applies


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi; windows are cut out by monotonic time."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []          # (arrival time, csv line)
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def window(self, t_begin, t_end):
        """Summary of the samples that arrived in [t_begin + 50 ms, t_end]."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sm, mx, power, reasons = [], [], [], set()
        for t, ln in list(self.lines):
            if t < t_begin + 0.05 or t > t_end:
                continue
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": max(mx),
                "power_w_max": max(power), "samples": len(sm), "reasons": sorted(reasons)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()


WORKLOAD_TEXT = {
    "1p5b": "1.5B-shaped: H=1536, V=151936, bf16 hidden/W, fp32 accumulate; 16 sequences (2 prompts x group 8) "
            "x 1024 rows, response lengths U[256,1024] right-padded and masked; staleness U{0..4}",
    "8b": "8B-shaped: H=4096, V=151936, bf16; 64 sequences (8 prompts x group 8) x 2048 rows, "
          "response lengths U[512,2048] right-padded and masked; staleness U{0..8}",
    "8b_packed": "8B-shaped long-response packed batch: H=4096, V=151936, bf16; 256 sequences (16 prompts x group 16) "
                 "packed (cu_seqlens), lengths U[512,8192]; staleness min(Geom(0.4)-1, 16); 5% of tokens masked out",
}


# ------------------------------------------------------------------------------------ oracle arm
def oracle_sample_step(sample):
    """fwd -> loss fwd/bwd -> bwd on a row sample, all in the fp64 oracle.  Returns seconds."""
    from oracle import a3po_oracle as orc
    t0 = time.perf_counter()
    logp, _ = orc.token_logprobs_fwd(sample["hidden"], sample["w"], sample["targets"])
    behav = sample["behav_from"](logp)
    args = (logp, behav, sample["versions"], sample["current_version"], sample["adv"], sample["mask"],
            sample["clip_eps"])
    orc.loss_fwd(*args)
    g = orc.loss_bwd(*args)
    orc.token_logprobs_bwd(sample["hidden"], sample["w"], sample["targets"], g)
    return time.perf_counter() - t0


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def make_oracle_sample(name, rows):
    """The first `rows` valid rows of the workload, operands widened for the oracle (host only)."""
    import numpy as np
    from paper_2512_06547_b200 import workloads
    wl = workloads.make_workload(name, "cpu", with_operands=False)
    idx = np.flatnonzero(wl.mask)[:rows]
    hidden, w = workloads.lm_head_operands(len(idx), wl.H, wl.V, wl.dtype, wl.meta["seed"], "cpu")
    noise = wl.behav_noise[idx]
    # widened to float64 once, here: the oracle would otherwise widen W (V x H) again on every call
    return dict(hidden=hidden.double().numpy(), w=w.double().numpy(), targets=wl.targets[idx],
                versions=wl.versions[idx], current_version=wl.current_version, adv=wl.adv[idx],
                mask=wl.mask[idx], clip_eps=wl.clip_eps, rows=len(idx),
                behav_from=lambda logp: workloads.behav_logp_from(logp, noise))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # size the row sample so that warm-up + K steps take about two minutes on this machine's cores
    probe = make_oracle_sample(args.workload, 16)
    per_row = oracle_sample_step(probe) / probe["rows"]
    total_steps = args.steps + args.warmup
    rows = int(max(8, min(args.oracle_rows, 120.0 / max(total_steps, 1) / per_row)))
    sample = make_oracle_sample(args.workload, rows)
    for _ in range(args.warmup):
        oracle_sample_step(sample)
    times = [oracle_sample_step(sample) for _ in range(args.steps)]
    mean_s = sum(times) / len(times)
    value = sample["rows"] / mean_s
    cores = oracle_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload],
                   "sample": f"each step = the first {sample['rows']} valid rows of the batch at full H and V"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": f"{sample['rows']} valid rows x {args.steps} steps, full H and V, fp64 numpy"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ our arm
def rank_seed(workload: str, rank: int) -> int:
    """Every rank draws its own shard of sequences (same shapes, different draws): weak scaling."""
    from paper_2512_06547_b200 import workloads
    return workloads.BASE_SEED + workloads._SEED_OFFSET[workload] + 1000 * rank


def reduce_over_ranks(times_ms, counts, device):
    """Whole-job figures: MAX over ranks of each time, SUM over ranks of each count.
    Works with any initialised process group (nccl on GPUs, gloo in the CPU test) or none."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.tolist()


def tensor_roofline(kernels, steps, h, v, region_s, peaks, workload=None, small=False):
    """Roofline object of the dominant GEMM kernel.  The peak is the measured cuBLAS bf16 figure that matches the
    timed region: the burst figure for a short region, the sustained one when the region is long enough for the
    board to sit at its power cap."""
    gemms = [k for k in kernels if k["kernel"].startswith("gemm_tn")]
    if not gemms:
        return {"bound": "tensor", "kernel": None, "achieved": None, "peak": None, "unit": "TFLOP/s", "frac": None,
                "traffic": None}
    dom = gemms[0]
    sustained = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    burst = peaks["bf16_tflops"]
    long_region = region_s > LONG_REGION_S
    peak = sustained if long_region else burst
    per_step = None if small else NCU_TRAFFIC_PER_STEP.get(workload, {}).get(dom["kernel"])
    launches_per_step = max(dom["launches"] // max(steps, 1), 1)
    all_flops = sum(2.0 * k["rows"] * v * h * steps for k in gemms)
    all_ms = sum(k["ms_total"] for k in gemms)
    return {"bound": "tensor", "kernel": dom["kernel"], "achieved": dom["tflops"], "peak": peak,
            "unit": "TFLOP/s", "frac": round(dom["tflops"] / peak, 4),
            "traffic": round(per_step / launches_per_step) if per_step else None,
            "algorithmic_flops_per_launch": 2.0 * dom["rows"] * v * h / launches_per_step,
            # the keeping forward: hidden rows in, 2 bytes per (row, vocabulary entry) out, W once per launch
            "algorithmic_bytes_per_launch": (round(dom["rows"] * (2.0 * h + 2.0 * ((v + 7) // 8 * 8))
                                                   / launches_per_step + 2.0 * v * h)
                                             if "keep" in dom["kernel"] else None),
            "launches_per_step": launches_per_step,
            "peak_source": "%s cuBLAS bf16, %s (timed region %.1f s)" % (
                peaks["_source"], "sustained" if long_region else "burst", region_s),
            "peak_burst": burst, "frac_of_burst": round(dom["tflops"] / burst, 4),
            "peak_sustained": sustained, "frac_of_sustained": round(dom["tflops"] / sustained, 4),
            "frac_of_nominal_2250": round(dom["tflops"] / 2250.0, 4),
            "all_gemm_tn_tflops": round(all_flops / (all_ms * 1e-3) / 1e12, 1)}


def time_step_workload(name, args, sampler, dev, rank, world, barrier, *, steps, warmup, with_e2e, small=False):
    """Builds the workload on `dev`, times `steps` passes of a3po_train_step with the per-kernel events off,
    then the same number again with them on (kernel table), then optionally the host-input entry."""
    import numpy as np
    import torch

    import paper_2512_06547_b200 as a3po
    from paper_2512_06547_b200 import workloads

    seed = rank_seed(name, rank)
    # --small: 4 sequences, for profiler captures; with a single group of 4 the Bernoulli rewards can all be
    # equal (zero advantages, nothing to back-propagate), so its advantages are drawn N(0,1) per sequence instead
    shrink = dict(n_prompts=1, group=4, reward_p=None) if small else {}
    wl = workloads.make_workload(name, dev, seed=seed, **shrink)
    n, h, v = wl.N, wl.H, wl.V
    dt = a3po.A3PO_BF16 if wl.dtype == "bf16" else a3po.A3PO_F32
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    targets, versions, adv, mask = (to_dev(x) for x in (wl.targets, wl.versions, wl.adv, wl.mask))
    n_valid = int(wl.mask.sum())

    ws_bytes = a3po.a3po_train_step_workspace_bytes(n, h, v, dt)
    ws = a3po.new_workspace(ws_bytes, dev)
    logp = torch.empty(n, device=dev)
    lse = torch.empty(n, device=dev)
    grad_logp = torch.empty(n, device=dev)
    loss = torch.zeros(1, device=dev)
    stats = a3po.new_stats(dev)
    grad_hidden = torch.empty_like(wl.hidden)
    grad_w = torch.zeros((v, h), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    # behaviour log-probs = current + noise (the recipe of the config); "current" comes from one untimed forward
    a3po.a3po_token_logprobs_fwd(wl.hidden, wl.w, targets, logp, lse, ws, row_mask=mask, status=status)
    torch.cuda.synchronize()
    behav_host = workloads.behav_logp_from(logp.cpu().numpy(), wl.behav_noise)
    behav = to_dev(behav_host)

    def step():
        if args.separate_calls:     # the three ABI calls one after the other: the backward recomputes the logits
            a3po.a3po_token_logprobs_fwd(wl.hidden, wl.w, targets, logp, lse, ws, row_mask=mask, status=status)
            a3po.a3po_loss_fwd_bwd(logp, behav, versions, wl.current_version, adv, mask, wl.clip_eps, loss,
                                   grad_logp, ws, stats=stats)
            a3po.a3po_token_logprobs_bwd(wl.hidden, wl.w, targets, lse, grad_logp, grad_hidden, grad_w, ws,
                                         status=status)
        else:                       # one call; the backward reuses what the forward kept in the workspace
            a3po.a3po_train_step(wl.hidden, wl.w, targets, behav, versions, wl.current_version, adv, mask,
                                 wl.clip_eps, logp, lse, grad_logp, loss, grad_hidden, grad_w, ws, stats=stats,
                                 status=status)

    def timed_loop(fn, k):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.monotonic()
        e0.record()
        for _ in range(k):
            fn()
        e1.record()
        barrier()
        t1 = time.monotonic()
        return e0.elapsed_time(e1), (t0, t1)

    for _ in range(warmup):
        step()
    barrier()

    # ---- timed region: device-resident inputs, per-kernel events off
    a3po.a3po_profile_enable(False)
    launches0 = a3po.a3po_kernel_launch_count()
    ms_total, win = timed_loop(step, steps)
    launches = a3po.a3po_kernel_launch_count() - launches0
    if int(status.item()) != 0:
        raise RuntimeError(f"device status word = {int(status.item())}")
    clocks = sampler.window(*win) if sampler else None

    # ---- the same loop again with one CUDA-event pair around every launch: the kernel table
    a3po.a3po_profile_enable(True)
    a3po.a3po_profile_read()
    ms_profiled, _ = timed_loop(step, steps)
    a3po.a3po_profile_enable(False)
    per_kernel = a3po.a3po_profile_read()

    out = dict(wl=wl, n=n, h=h, v=v, n_valid=n_valid, ms_total=ms_total, ms_profiled=ms_profiled, launches=launches,
               clocks=clocks, per_kernel=per_kernel, ws_bytes=ws_bytes, loss=float(loss.item()),
               bwd_rows=int((grad_logp != 0).sum().item()), e2e=None)

    # ---- e2e: host-resident per-step inputs through the C ABI's host entry
    if with_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_hidden = wl.hidden.cpu().pin_memory()
        h_targets, h_behav, h_versions, h_adv, h_mask = (pin(x) for x in (wl.targets, behav_host, wl.versions, wl.adv,
                                                                           wl.mask))
        h_loss = torch.zeros(1).pin_memory()
        h_stats = torch.zeros(24, dtype=torch.uint8).pin_memory()
        stage = a3po.new_workspace(a3po.a3po_train_step_stage_bytes(n, h, dt), dev)

        def host_step():
            a3po.a3po_train_step_host(h_hidden, h_targets, h_behav, h_versions, h_adv, h_mask, wl.current_version,
                                      wl.clip_eps, wl.w, grad_w, grad_hidden, stage, ws, h_loss, h_stats=h_stats,
                                      d_status=status)
            torch.cuda.current_stream().synchronize()   # the step's loss is read on the host
            return float(h_loss.item())

        for _ in range(min(warmup, 3)):
            host_step()
        copied = a3po.a3po_host_to_device_bytes()
        e2e_ms_total, _ = timed_loop(host_step, steps)
        copied = (a3po.a3po_host_to_device_bytes() - copied) // steps    # what the library really sent per step
        # where the difference to the device-resident loop goes: the host->device copies, timed on their own
        a3po.a3po_profile_enable(True)
        a3po.a3po_profile_read()
        for _ in range(3):
            host_step()
        a3po.a3po_profile_enable(False)
        h2d_ms = [ms for k, ms in a3po.a3po_profile_read() if k == "h2d_copies"]
        out["e2e"] = dict(ms_total=e2e_ms_total,
                          h2d=copied, h2d_of=h_hidden.numel() * h_hidden.element_size() + n * (4 + 4 + 4 + 4 + 1),
                          d2h=4 + 24,
                          h2d_ms=statistics.mean(h2d_ms) if h2d_ms else None)
        del h_hidden, stage
    del ws, grad_w, grad_hidden, wl.hidden, wl.w
    torch.cuda.empty_cache()
    return out


def kernel_table(per_kernel, steps, fwd_rows, bwd_rows, n, v, h):
    agg = {}
    for name, ms in per_kernel:
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += ms
    total = sum(x[1] for x in agg.values()) or 1.0
    # Algorithmic flops per launch = 2 * (rows that take part) * V * H: the forward processes the rows with
    # mask != 0, the backward contractions the rows whose upstream gradient is non-zero (padding and clipped
    # tokens contribute nothing, so they are not counted as work whether or not a kernel skips them).
    rows_of = {"gemm_tn<fwd_logsoftmax>": fwd_rows, "gemm_tn<fwd_logsoftmax+keep>": fwd_rows,
               "gemm_tn<dz>": bwd_rows, "gemm_tn<grad_hidden>": bwd_rows, "gemm_tn<grad_w>": bwd_rows}
    kernels = []
    for name, (cnt, ms) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        entry = {"kernel": name, "launches": cnt, "ms_total": round(ms, 4), "share": round(ms / total, 4)}
        if name.startswith("gemm_tn"):
            entry["rows"] = rows_of.get(name, n)
            # a step may split a contraction over several launches (row chunks): flops are per step
            entry["tflops"] = round(2.0 * entry["rows"] * v * h * steps / (ms * 1e-3) / 1e12, 1)
        kernels.append(entry)
    recomputes = any(k["kernel"] == "gemm_tn<dz>" for k in kernels)
    step_flops = 2.0 * v * h * (fwd_rows + (3 if recomputes else 2) * bwd_rows)
    return kernels, step_flops


def steps_for(seconds_per_step, min_seconds, lo, hi):
    k = int(min_seconds / max(seconds_per_step, 1e-6)) + 1
    return max(lo, min(hi, k))


def secondary_step_config(name, args, sampler, dev, barrier, peaks):
    """Compact entry for another named configuration: timed in its own window of >= 1.5 s."""
    import torch
    # one short probe to size the loop, then the timed run
    probe = time_step_workload(name, args, None, dev, 0, 1, barrier, steps=1, warmup=1, with_e2e=False)
    per_step = probe["ms_total"] * 1e-3
    steps = steps_for(per_step, 1.5, 2, 200)
    r = time_step_workload(name, args, sampler, dev, 0, 1, barrier, steps=steps, warmup=3 if per_step < 1 else 1,
                           with_e2e=False)
    kernels, step_flops = kernel_table(r["per_kernel"], steps, r["n_valid"], r["bwd_rows"], r["n"], r["v"], r["h"])
    ms_per_step = r["ms_total"] / steps
    roof = tensor_roofline(kernels, steps, r["h"], r["v"], r["ms_total"] * 1e-3, peaks, workload=name)
    torch.cuda.empty_cache()
    return {"workload": WORKLOAD_TEXT[name], "rows": r["n"], "valid_tokens": r["n_valid"], "steps": steps,
            "ms_per_step": round(ms_per_step, 4), "value": round(r["n_valid"] / (ms_per_step * 1e-3), 1),
            "unit": "tokens/s", "executed_tflops": round(step_flops / (ms_per_step * 1e-3) / 1e12, 1),
            "workspace_gib": round(r["ws_bytes"] / 2 ** 30, 2),
            "recompute_free": not any(k["kernel"] == "gemm_tn<dz>" for k in kernels),
            "roofline": {k: roof[k] for k in ("bound", "kernel", "achieved", "peak", "unit", "frac", "frac_of_burst",
                                              "frac_of_sustained", "peak_source", "traffic",
                                              "algorithmic_bytes_per_launch") if k in roof},
            "kernels": [{k: e[k] for k in ("kernel", "ms_total", "share", "tflops") if k in e} for e in kernels[:4]],
            "clocks": r["clocks"]}


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier(device_ids=[local_rank])
        torch.cuda.synchronize()

    peaks = load_peaks()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()          # started early: nvidia-smi needs a moment before its first sample
    r = time_step_workload(args.workload, args, sampler, dev, rank, world, barrier, steps=args.steps,
                           warmup=args.warmup, with_e2e=True, small=args.small)
    n, h, v, n_valid = r["n"], r["h"], r["v"], r["n_valid"]

    # ---- max over ranks
    (ms_total, e2e_ms_total), (total_valid, total_rows) = reduce_over_ranks(
        [r["ms_total"], r["e2e"]["ms_total"]], [float(n_valid), float(n)], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms_total / args.steps
    value = total_valid * args.steps / (ms_total * 1e-3)
    e2e_value = total_valid * args.steps / (e2e_ms_total * 1e-3)
    kernels, step_flops = kernel_table(r["per_kernel"], args.steps, n_valid, r["bwd_rows"], n, v, h)
    roofline = tensor_roofline(kernels, args.steps, h, v, ms_total * 1e-3, peaks, workload=args.workload,
                               small=args.small or args.separate_calls)

    # ---- the other named configurations, each in its own window (one GPU only)
    configs = None
    if world == 1 and not args.no_configs and not args.small:
        configs = {}
        for name in ("1p5b", "8b", "8b_packed"):
            if name != args.workload:
                configs[name] = secondary_step_config(name, args, sampler, dev, barrier, peaks)
        for tokens in (1 << 24, 1 << 26):
            configs["loss_sweep_2^%d" % (tokens.bit_length() - 1)] = loss_sweep_entry(
                tokens, sampler, dev, peaks, min_seconds=1.5)
    if sampler:
        sampler.stop()

    # ---- oracle beside it (rank 0, bounded sample)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sample = make_oracle_sample(args.workload, args.oracle_rows)
        secs = oracle_sample_step(sample)
        cpu_baseline = {"value": sample["rows"] / secs, "unit": "tokens/s", "cores": oracle_threads(),
                        "kind": "oracle", "seconds": round(secs, 2),
                        "sample": f"the first {sample['rows']} valid rows of the batch at full H and V, one step, "
                                  "fp64 numpy"}

    wl = r["wl"]
    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload] + (" [--small: 4 sequences only]" if args.small else ""),
                   "rows_per_gpu": n, "valid_tokens_per_gpu": n_valid,
                   "H": h, "V": v, "parallelism": f"dp{world} (independent shards)",
                   "workspace_gib": round(r["ws_bytes"] / 2 ** 30, 2),
                   "l2": "no flush: W (%.0f MB) and the kept-probabilities scratch are larger than the 126 MB L2"
                         % (v * h * 2 / 1e6),
                   **({"library": "tuning build: " + (" ".join(f"{k}={val}" for k, val in sorted(os.environ.items())
                                                               if k.startswith("A3PO_")) or "no switches set")}
                      if args.library == "tuning" else {})},
        "rows_per_s": total_rows * args.steps / (ms_total * 1e-3),
        "executed_tflops": round(step_flops * world / (ms_per_step * 1e-3) / 1e12, 1),
        "rows_processed": {"fwd": n_valid, "bwd": r["bwd_rows"], "of": n},
        "ms_per_step_with_kernel_events": r["ms_profiled"] / args.steps,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": r["e2e"]["h2d"],
                "d2h_bytes_per_step": r["e2e"]["d2h"], "ms_per_step": e2e_ms_total / args.steps,
                "h2d_ms_per_step": r["e2e"]["h2d_ms"], "host_bytes_per_step": r["e2e"]["h2d_of"],
                "note": "of hidden only the rows with mask != 0 cross the bus (the step reads no others)"},
        "gpu_launches": int(r["launches"]),
        "clocks": r["clocks"],
        "roofline": roofline,
        "kernels": kernels,
        "configs": configs,
        "cpu_baseline": cpu_baseline,
        "loss": r["loss"],
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ loss-only sweep
def loss_sweep_entry(n, sampler, dev, peaks, *, min_seconds=1.5, warmup=3):
    """Loss calls alone on the bandwidth-sweep workload at n tokens: fwd, bwd and fused fwd+bwd.  Each call is
    timed over a back-to-back loop of at least `min_seconds` (the per-token arrays, 21 n bytes, exceed L2 at
    both sizes the sweep is judged at; below 2 x L2 a 512 MB buffer is overwritten between iterations instead
    and every iteration gets its own event pair).  `call` figures cover every launch of the ABI call; `kernel`
    figures the streaming kernel alone, from the library's per-launch events in a second loop."""
    import numpy as np
    import torch

    import paper_2512_06547_b200 as a3po
    from paper_2512_06547_b200 import workloads

    inp = workloads.loss_sweep(n)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    logp, behav, versions, adv, mask = (to_dev(inp[k]) for k in ("logp", "behav_logp", "versions", "adv", "mask"))
    common = (logp, behav, versions, inp["current_version"], adv, mask, inp["clip_eps"])
    ws = a3po.new_workspace(a3po.a3po_loss_workspace_bytes(n), dev)
    loss = torch.zeros(1, device=dev)
    stats = a3po.new_stats(dev)
    grad = torch.empty(n, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if 21 * n < (256 << 20) else None
    calls = {
        "fwd": (lambda: a3po.a3po_loss_fwd(*common, loss, ws, stats=stats), 17),
        "bwd": (lambda: a3po.a3po_loss_bwd(*common, grad, ws, fwd_stats=stats), 21),
        "fwd_bwd": (lambda: a3po.a3po_loss_fwd_bwd(*common, loss, grad, ws, stats=stats), 22),
    }
    results = {}
    t_begin = time.monotonic()
    for name, (fn, bytes_per_token) in calls.items():
        a3po.a3po_profile_enable(False)
        for _ in range(max(warmup, 3)):
            fn()
        torch.cuda.synchronize()
        est = max(bytes_per_token * n / 5e12, 2e-5)
        iters = steps_for(est, min_seconds / len(calls), 20, 20000)
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                fn()
            e1.record()
            torch.cuda.synchronize()
            call_ms = e0.elapsed_time(e1) / iters
        else:
            iters = min(iters, 200)
            per = []
            for _ in range(iters):
                flush.fill_(1)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                per.append(e0.elapsed_time(e1))
            call_ms = statistics.mean(per)
        # the streaming kernel alone, and the launches of one call
        a3po.a3po_profile_enable(True)
        a3po.a3po_profile_read()
        reps = 20
        for _ in range(reps):
            if flush is not None:
                flush.fill_(1)
            fn()
        torch.cuda.synchronize()
        a3po.a3po_profile_enable(False)
        prof = a3po.a3po_profile_read()
        main_ms = [ms for k, ms in prof if k in ("loss_fwd", "loss_bwd", "loss_fwd_bwd")]
        kernel_ms = statistics.mean(main_ms)
        main_bytes = bytes_per_token - (1 if name == "fwd_bwd" else 0)     # the mask pre-count is its own kernel
        results[name] = {
            "call_ms": round(call_ms, 5), "kernel_ms": round(kernel_ms, 5), "launches_per_call": len(prof) // reps,
            "iterations": iters, "algorithmic_bytes_per_token": bytes_per_token,
            "call_gbs": round(bytes_per_token * n / (call_ms * 1e-3) / 1e9, 1),
            "kernel_gbs": round(main_bytes * n / (kernel_ms * 1e-3) / 1e9, 1),
        }
    t_end = time.monotonic()
    best = results["fwd_bwd"]
    hbm = peaks["hbm_gbs"]
    entry = {
        "workload": f"loss-only bandwidth sweep, N={n} tokens: fp32 logp / behaviour logp ~ -Exp(1), int32 per-token "
                    "versions (staleness U{0..8}), fp32 advantage, uint8 mask (90% kept), eps=0.2",
        "l2": "flushed between iterations" if flush is not None else "inputs exceed L2",
        "value": round(n / (best["call_ms"] * 1e-3), 1), "unit": "tokens/s", "ms_per_call": best["call_ms"],
        "roofline": {"bound": "hbm", "kernel": "a3po_loss_fwd_bwd (whole call, every launch)",
                     "achieved": best["call_gbs"], "peak": hbm, "unit": "GB/s",
                     "frac": round(best["call_gbs"] / hbm, 4),
                     "frac_of_nominal_8000": round(best["call_gbs"] / 8000.0, 4),
                     "kernel_only_achieved": best["kernel_gbs"], "kernel_only_frac": round(best["kernel_gbs"] / hbm, 4),
                     "traffic": round(NCU_TRAFFIC_PER_TOKEN_LOSS["loss_fwd_bwd"] * n),
                     "algorithmic_bytes_per_call": 22 * n,
                     "peak_source": f"{peaks['_source']} copy bandwidth"},
        "loss_calls": results,
        "clocks": sampler.window(t_begin, t_end) if sampler else None,
    }
    del logp, behav, versions, adv, mask, ws, grad, flush
    torch.cuda.empty_cache()
    return entry


def run_loss_sweep(args):
    import torch
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    entry = loss_sweep_entry(args.tokens, sampler, dev, peaks, min_seconds=args.min_seconds, warmup=args.warmup)
    sampler.stop()
    line = {
        "metric": METRIC, "value": entry["value"], "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": entry["ms_per_call"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": entry["workload"], "l2": entry["l2"]},
        "roofline": entry["roofline"], "loss_calls": entry["loss_calls"], "clocks": entry["clocks"],
        "gpu_launches": None, "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)


def respawn_under_torchrun(args):
    """`python bench.py --gpus N` with N > 1 outside torchrun: start one rank per GPU and hand over."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12)   # 8B-shaped: 12 x 0.2 s, a timed region above LONG_REGION_S
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b", choices=sorted(WORKLOAD_TEXT) + ["loss_sweep"])
    ap.add_argument("--tokens", type=int, default=1 << 26, help="token count of --workload loss_sweep")
    ap.add_argument("--min-seconds", type=float, default=1.5,
                    help="length of the timed window of --workload loss_sweep (short values for profiler captures)")
    ap.add_argument("--oracle-rows", type=int, default=1024,
                    help="valid rows of the batch the CPU oracle is timed on (about 12 s on 16 cores at the 8B shape)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the compact entries for the other named configurations")
    ap.add_argument("--small", action="store_true",
                    help="same shapes with 4 sequences only (a profiler-sized case; not a benchmark number)")
    ap.add_argument("--separate-calls", action="store_true",
                    help="time fwd / loss / bwd as three ABI calls (backward recomputes the logits) instead of "
                         "a3po_train_step")
    ap.add_argument("--library", default="product", choices=["product", "tuning"],
                    help="tuning: load lib/liba3po_tuning.so (same sources, -DA3PO_TUNING), whose scheduling constants "
                         "follow the A3PO_* environment variables; for A/B runs, not a benchmark number")
    args = ap.parse_args()
    if args.library == "tuning":
        from paper_2512_06547_b200 import binding, build as a3po_build
        binding.LIB_PATH = a3po_build.build(tuning=True)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(respawn_under_torchrun(args))
    if args.workload == "loss_sweep":
        run_loss_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_ours(args)


if __name__ == "__main__":
    main()
