#!/usr/bin/env python
"""Benchmark of the A-3PO hot path: token log-probs fwd -> A-3PO loss fwd+bwd -> log-prob bwd.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 1p5b|8b]

One "step" is one pass of the whole path over one synthetic batch shaped like the paper's
1.5B set-up (H=1536, V=151,936, bf16, 16 sequences x 1024 rows).  Prints ONE JSON line.

  value      whole-job valid (mask=1) tokens per second, inputs resident in HBM
  e2e        same metric through a3po_train_step_host: per-step inputs start in pinned host memory
  roofline   the dominant kernel's achieved TFLOP/s (algorithmic flops / CUDA-event duration of each
             launch, recorded by the library on its launch stream) against the measured bf16 peak
  cpu_baseline  the fp64 oracle timed on this machine's host cores on a bounded row sample

--impl reference times the oracle alone (the paper ships no runnable reference implementation).
With N > 1 (torchrun) every rank runs its own shard of sequences (weak scaling, no data-path
collective); timing is bracketed by barriers and the maximum over ranks is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "logprob+A-3PO loss fwd/bwd tokens/s; % of bf16 TC peak & HBM roofline"

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/.
# GEMM kernels (profiles/gemm_tn_small_case_ncu_full.md): bytes per row that takes part, taken on the --small case
# (2244 rows, H=1536, V=151936) and scaled by the rows of the launch (W re-reads and the kept logits / dz both grow
# with the rows).  Only valid for that H and V; reset an entry to None when its kernel changes.
NCU_TRAFFIC_PER_ROW_1P5B = {
    "gemm_tn<fwd_logsoftmax+keep_logits>": (880.164e6 + 682.214e6) / 2244,
    "gemm_tn<grad_hidden>": (1167.594e6 + 3.738e6) / 2244,
    "gemm_tn<fwd_logsoftmax>": (879.835e6 + 3.917e6) / 2244,
    "gemm_tn<dz>": (940.724e6 + 685.156e6) / 2244,
    "gemm_tn<grad_w>": None,     # its traffic (874 MB of fp32 output + operands) does not scale with the rows
}
# Loss kernels (profiles/loss_kernels_16Mi_tokens_ncu_full.md): bytes per token at N = 2^24.
NCU_TRAFFIC_PER_TOKEN_LOSS = {"loss_fwd_bwd": (285.231616e6 + 40.569600e6) / 16777216}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


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
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []          # (arrival time, csv line)
        self.thread = None
        self.t_begin = None
        self.t_end = None

    def mark_begin(self):
        self.t_begin = time.monotonic()

    def mark_end(self):
        self.t_end = time.monotonic()

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

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        window = [ln for t, ln in self.lines
                  if (self.t_begin is None or t >= self.t_begin + 0.05) and (self.t_end is None or t <= self.t_end)]
        for ln in (window or [ln for _, ln in self.lines]):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": max(mx),
                "power_w_max": max(power), "samples": len(sm), "reasons": sorted(reasons)}


WORKLOAD_TEXT = {
    "1p5b": "1.5B-shaped: H=1536, V=151936, bf16 hidden/W, fp32 accumulate; 16 sequences (2 prompts x group 8) "
            "x 1024 rows, response lengths U[256,1024] right-padded and masked; staleness U{0..4}",
    "8b": "8B-shaped: H=4096, V=151936, bf16; 64 sequences (8 prompts x group 8) x 2048 rows, "
          "response lengths U[512,2048]; staleness U{0..8}",
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
    probe = make_oracle_sample(args.workload, 32)
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


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2512_06547_b200 as a3po
    from paper_2512_06547_b200 import workloads

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

    # every rank draws its own shard of sequences (same shapes): weak scaling, no data-path collective
    seed = rank_seed(args.workload, rank)
    # --small: 4 sequences, for profiler captures; with a single group of 4 the Bernoulli rewards can all be
    # equal (zero advantages, nothing to back-propagate), so its advantages are drawn N(0,1) per sequence instead
    shrink = dict(n_prompts=1, group=4, reward_p=None) if args.small else {}
    wl = workloads.make_workload(args.workload, dev, seed=seed, **shrink)
    n, h, v = wl.N, wl.H, wl.V
    dt = a3po.A3PO_BF16 if wl.dtype == "bf16" else a3po.A3PO_F32
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    targets, versions, adv, mask = (to_dev(x) for x in (wl.targets, wl.versions, wl.adv, wl.mask))
    n_valid = int(wl.mask.sum())

    ws = a3po.new_workspace(a3po.a3po_train_step_workspace_bytes(n, h, v, dt), dev)
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
        else:                       # one call; the backward reuses the logits the forward kept in the workspace
            a3po.a3po_train_step(wl.hidden, wl.w, targets, behav, versions, wl.current_version, adv, mask,
                                 wl.clip_eps, logp, lse, grad_logp, loss, grad_hidden, grad_w, ws, stats=stats,
                                 status=status)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()          # started early: nvidia-smi needs a moment before its first sample
    for _ in range(args.warmup):
        step()
    barrier()

    # ---- timed region: device-resident inputs
    a3po.a3po_profile_enable(True)
    a3po.a3po_profile_read()
    launches0 = a3po.a3po_kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark_begin()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    sampler.mark_end()
    launches = a3po.a3po_kernel_launch_count() - launches0
    a3po.a3po_profile_enable(False)
    per_kernel = a3po.a3po_profile_read()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    if int(status.item()) != 0:
        raise RuntimeError(f"device status word = {int(status.item())}")

    # ---- e2e: host-resident per-step inputs through the C ABI's host entry
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

    for _ in range(min(args.warmup, 3)):
        host_step()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(args.steps):
        host_step()
    f1.record()
    barrier()
    e2e_ms_total = f0.elapsed_time(f1)
    h2d = h_hidden.numel() * h_hidden.element_size() + n * (4 + 4 + 4 + 4 + 1)
    d2h = 4 + 24

    # ---- max over ranks
    (ms_total, e2e_ms_total), (total_valid, total_rows) = reduce_over_ranks(
        [ms_total, e2e_ms_total], [float(n_valid), float(n)], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms_total / args.steps
    value = total_valid * args.steps / (ms_total * 1e-3)
    e2e_value = total_valid * args.steps / (e2e_ms_total * 1e-3)

    # ---- roofline of the dominant kernel, from the per-launch CUDA events of the timed region
    peaks = load_peaks()
    agg = {}
    for name, ms in per_kernel:
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += ms
    kernel_total = sum(x[1] for x in agg.values()) or 1.0
    # Algorithmic flops per launch = 2 * (rows that take part) * V * H: the forward processes the rows with
    # mask != 0, the three backward contractions the rows whose upstream gradient is non-zero (padding and
    # clipped tokens are skipped by the library, so they are not counted as work).
    fwd_rows = n_valid
    bwd_rows = int((grad_logp != 0).sum().item())
    rows_of = {"gemm_tn<fwd_logsoftmax>": fwd_rows, "gemm_tn<fwd_logsoftmax+keep_logits>": fwd_rows,
               "gemm_tn<dz>": bwd_rows, "gemm_tn<grad_hidden>": bwd_rows, "gemm_tn<grad_w>": bwd_rows}
    # contractions actually executed per step: forward + (dz recompute unless the logits were kept) + two gradients
    recomputes = any(name == "gemm_tn<dz>" for name in agg)
    step_flops = 2.0 * v * h * (fwd_rows + (3 if recomputes else 2) * bwd_rows)
    kernels = []
    for name, (cnt, ms) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        entry = {"kernel": name, "launches": cnt, "ms_total": round(ms, 4), "share": round(ms / kernel_total, 4)}
        if name.startswith("gemm_tn"):
            entry["rows"] = rows_of.get(name, n)
            # a step may split a contraction over several launches (row chunks): flops are per step
            entry["tflops"] = round(2.0 * entry["rows"] * v * h * args.steps / (ms * 1e-3) / 1e12, 1)
        kernels.append(entry)
    dom = kernels[0]
    sustained = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    if dom["kernel"].startswith("gemm_tn"):
        achieved = dom["tflops"]
        roofline = {"bound": "tensor", "kernel": dom["kernel"], "achieved": achieved, "peak": sustained,
                    "unit": "TFLOP/s", "frac": round(achieved / sustained, 4),
                    "traffic": (round(NCU_TRAFFIC_PER_ROW_1P5B[dom["kernel"]] * dom["rows"])
                                if (h, v) == (1536, 151936) and NCU_TRAFFIC_PER_ROW_1P5B.get(dom["kernel"]) else None),
                    "algorithmic_flops_per_launch": 2.0 * dom["rows"] * v * h,
                    "peak_source": f"{peaks['_source']} cuBLAS bf16, sustained (kernel timed inside a long step)",
                    "peak_burst": peaks["bf16_tflops"], "frac_of_burst": round(achieved / peaks["bf16_tflops"], 4),
                    "frac_of_nominal_2250": round(achieved / 2250.0, 4),
                    "all_gemm_tn_tflops": round(
                        sum(2.0 * k["rows"] * v * h * args.steps for k in kernels if k["kernel"].startswith("gemm_tn")) /
                        (sum(k["ms_total"] for k in kernels if k["kernel"].startswith("gemm_tn")) * 1e-3) / 1e12, 1)}
    else:
        roofline = {"bound": "hbm", "kernel": dom["kernel"], "achieved": None, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": None, "traffic": None}

    # ---- oracle beside it (rank 0, bounded sample)
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        sample = make_oracle_sample(args.workload, args.oracle_rows)
        secs = oracle_sample_step(sample)
        cpu_baseline = {"value": sample["rows"] / secs, "unit": "tokens/s", "cores": oracle_threads(),
                        "kind": "oracle", "seconds": round(secs, 2),
                        "sample": f"the first {sample['rows']} valid rows of the batch at full H and V, one step, "
                                  "fp64 numpy"}

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload] + (" [--small: 4 sequences only]" if args.small else ""),
                   "rows_per_gpu": n, "valid_tokens_per_gpu": n_valid,
                   "H": h, "V": v, "parallelism": f"dp{world} (independent shards)",
                   "l2": "no flush: W (%.0f MB) and the dz scratch are larger than the 126 MB L2"
                         % (v * h * 2 / 1e6)},
        "rows_per_s": total_rows * args.steps / (ms_total * 1e-3),
        "executed_tflops": round(step_flops * world / (ms_per_step * 1e-3) / 1e12, 1),
        "rows_processed": {"fwd": fwd_rows, "bwd": bwd_rows, "of": n},
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms_total / args.steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "kernels": kernels,
        "cpu_baseline": cpu_baseline,
        "loss": float(loss.item()),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------ loss-only sweep
def run_loss_sweep(args):
    """Loss kernels alone on the bandwidth-sweep workload: fwd, bwd and fused fwd+bwd at --tokens tokens.
    Every iteration is timed with its own CUDA-event pair; when the inputs are smaller than 2x L2 a 512 MB
    buffer is overwritten between iterations (untimed) to flush L2."""
    import numpy as np
    import torch

    import paper_2512_06547_b200 as a3po
    from paper_2512_06547_b200 import workloads

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n = args.tokens
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
    peaks = load_peaks()
    sampler = ClockSampler(0)
    sampler.start()
    results = {}
    a3po.a3po_profile_enable(True)
    sampler_marked = False
    for name, (fn, bytes_per_token) in calls.items():
        for _ in range(max(args.warmup, 3)):
            fn()
        torch.cuda.synchronize()
        a3po.a3po_profile_read()
        if not sampler_marked:
            sampler.mark_begin()
            sampler_marked = True
        call_ms = []
        for _ in range(args.steps):
            if flush is not None:
                flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            call_ms.append(e0.elapsed_time(e1))
        prof = a3po.a3po_profile_read()
        main_ms = [ms for k, ms in prof if k in ("loss_fwd", "loss_bwd", "loss_fwd_bwd")]
        kernel_ms = statistics.mean(main_ms)
        main_bytes = bytes_per_token - (1 if name == "fwd_bwd" else 0)     # the mask pre-count is its own kernel
        results[name] = {
            "call_ms": statistics.mean(call_ms), "kernel_ms": kernel_ms, "launches_per_call": len(prof) // args.steps,
            "algorithmic_bytes_per_token": bytes_per_token,
            "call_gbs": bytes_per_token * n / (statistics.mean(call_ms) * 1e-3) / 1e9,
            "kernel_gbs": main_bytes * n / (kernel_ms * 1e-3) / 1e9,
        }
    sampler.mark_end()
    a3po.a3po_profile_enable(False)
    clocks = sampler.stop()
    best = results["fwd_bwd"]
    line = {
        "metric": METRIC, "value": n / (best["call_ms"] * 1e-3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": best["call_ms"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"loss-only bandwidth sweep, N={n} tokens: fp32 logp / behaviour logp ~ -Exp(1), int32 "
                               "per-token versions (staleness U{0..8}), fp32 advantage, uint8 mask (90% kept), eps=0.2",
                   "l2": "flushed between iterations" if flush is not None else "inputs exceed L2"},
        "roofline": {"bound": "hbm", "kernel": "loss_fwd_bwd", "achieved": round(best["kernel_gbs"], 1),
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(best["kernel_gbs"] / peaks["hbm_gbs"], 4),
                     "frac_of_nominal_8000": round(best["kernel_gbs"] / 8000.0, 4),
                     "traffic": round(NCU_TRAFFIC_PER_TOKEN_LOSS["loss_fwd_bwd"] * n),
                     "algorithmic_bytes_per_launch": 21 * n,
                     "peak_source": f"{peaks['_source']} copy bandwidth"},
        "loss_kernels": results, "clocks": clocks, "gpu_launches": None, "e2e": None, "cpu_baseline": None,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="1p5b", choices=sorted(WORKLOAD_TEXT) + ["loss_sweep"])
    ap.add_argument("--tokens", type=int, default=1 << 26, help="token count of --workload loss_sweep")
    ap.add_argument("--oracle-rows", type=int, default=256)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--small", action="store_true",
                    help="same shapes with 4 sequences only (a profiler-sized case; not a benchmark number)")
    ap.add_argument("--separate-calls", action="store_true",
                    help="time fwd / loss / bwd as three ABI calls (backward recomputes the logits) instead of "
                         "a3po_train_step")
    args = ap.parse_args()
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
