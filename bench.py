#!/usr/bin/env python
"""Benchmark of the HB-SJD rollout path on B200.

A "step" is one whole rollout of one synthetic batch (state init, prefix pre-filling, every
verification round until all images are complete) through the C ABI.  One JSON line is printed:
committed image tokens/sec (device-resident inputs), the same through host buffers (`e2e`), the
roofline fraction of the dominant kernel, and the CPU oracle timed on a bounded sample.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload L|B|XL|stress|tiny] [--impl reference]

N > 1 (torchrun): independent replicas, one batch per rank, no data-path collective ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_18183_b200 import synth  # noqa: E402

METRIC = "committed image tokens/sec per B200 rollout; mean accepted tokens/forward"
UNIT = "tokens/s"
# DRAM bytes per GEMM launch (read + write) from an ncu capture of the rollout (dram__bytes_read.sum +
# dram__bytes_write.sum, summarised under profiles/): mean over the 97 GEMM launches of one Full round of workload L.
NCU_GEMM_TRAFFIC_BYTES_PER_LAUNCH = {"L": 54.9e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# nominal figures of the part, for context beside the measured denominators: dense bf16 tensor peak, HBM3e bandwidth
NOMINAL_PEAKS = {"bf16_tflops": 2250.0, "hbm_gbs": 7700.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 6 for i in range(4) if r[2 + i] == "Active"})
        busy = sorted(sm)[len(sm) // 2:] if sm else []  # upper half: samples under load
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def oracle_sample(w, weights, toks, k, lab, seed, ids, n_rounds):
    """The CPU oracle, as it stands, on the images `ids` of the batch: prefix pre-filling + n_rounds rounds
    (0 = to completion).  Returns (committed tokens, seconds, threads)."""
    from oracle import oracle as O
    model = O.Model(w.shape, weights)
    P = O.make_params(w.window, w.history_offset, cfg_scale=w.cfg_scale, temperature=w.temperature, top_k=w.top_k,
                      seed=seed)
    t0 = time.perf_counter()
    r = O.Rollout(model, toks[ids], k[ids], lab[ids], P, image_ids=ids)
    r.run(n_rounds)
    dt = time.perf_counter() - t0
    return r.stats()["committed"], dt, O.num_threads()


def sample_plan(w, k):
    """Bounded oracle sample per workload: (image ids, rounds, description), sized for roughly 10-15 s of CPU
    work per step.  The large models take the images with the shortest prefixes (cheapest pre-filling)."""
    order = [int(i) for i in np.argsort(k, kind="stable")]
    n_img, n_rounds = {"tiny": (w.batch, 0), "tiny_bf16": (w.batch, 0), "small_bf16": (w.batch, 0), "B": (8, 16),
                       "L": (2, 8), "XL": (1, 6), "stress": (2, 8)}.get(w.name, (1, 1))
    ids = list(range(n_img)) if n_img == w.batch else order[:n_img]
    what = (f"{n_img} image(s) of the batch with the shortest prefixes (ids {ids}, prefix lengths "
            f"{[int(k[i]) for i in ids]}): prefix pre-filling + {n_rounds or 'all'} rounds")
    return ids, n_rounds, what


def run_reference(args, w, weights, toks, k, lab):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    ids, n_rounds, what = sample_plan(w, k)
    times, toks_done = [], 0
    for it in range(args.warmup + args.steps):
        done, dt, threads = oracle_sample(w, weights, toks, k, lab, it, ids, n_rounds)
        if it >= args.warmup:
            times.append(dt)
            toks_done += done
    total = sum(times)
    val = toks_done / total
    sample = what + " per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": w.shape.dtype,
            "data": "synthetic", "config": workload_config(w),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def rank_inputs(w, rank):
    """Each rank rolls out its own batch (replicas, no exchange step): the input seed is offset by the rank."""
    return synth.make_inputs(w, seed=w.input_seed + 1000 * rank)


def max_over_ranks(ms_local, dist, device):
    """Step time of the job = the slowest rank's device time (an all-reduce MAX when there are several ranks)."""
    if dist is None:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(tokens_per_step_local, steps, dist, device, ms):
    """Whole-job throughput: tokens committed by all ranks in the timed steps / the max-over-ranks time."""
    total = float(tokens_per_step_local * steps)
    if dist is not None:
        import torch
        t = torch.tensor([total], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        total = float(t.item())
    return total / (ms * 1e-3), total


def l2_note(w):
    """How the timed steps relate to the 126 MB L2: bytes one round streams (weights once, logits once)."""
    s = w.shape
    es = 2 if s.dtype == "bf16" else 4
    weights = (s.n_layers * (4 * s.dim * s.dim + 3 * s.dim * s.ffn_hidden) + s.dim * s.vocab) * es
    rows = w.batch * (2 if w.cfg_scale != 1.0 else 1) * w.window
    per_round = weights + rows * s.vocab * 4
    if per_round > 126e6:
        return (f"inputs larger than L2: a round streams {per_round / 1e6:.0f} MB (weights once, logits once) "
                f"besides the KV pages")
    return (f"working set of {per_round / 1e6:.1f} MB per round fits the L2: a parity-sized configuration, "
            f"not a bandwidth measurement")


def workload_config(w):
    s = w.shape
    return {"workload": f"{w.name}: L{s.n_layers} D{s.dim} H{s.n_heads} F{s.ffn_hidden} V{s.vocab} "
                        f"T{s.T} batch {w.batch} window {w.window} cfg {w.cfg_scale} top_k {w.top_k} {s.dtype}",
            "batch": w.batch, "window": w.window, "cfg_scale": w.cfg_scale, "history_offset": w.history_offset,
            "prefix": list(w.prefix), "exec_mode": "hybrid", "verify": "probabilistic",
            "l2": l2_note(w)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="L", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--gamma-frac", type=float, default=1.0,
                    help="Eq. 6 threshold as a fraction of the batch (Full iff live > threshold); 1.0 = the measured "
                         "optimum on this implementation, always Compact; 0 = always Full")
    ap.add_argument("--exec-mode", default="hybrid", choices=["full", "compact", "hybrid", "sync"],
                    help="sync = Full execution with batch-synchronous progress (the ablation baseline of Table 2)")
    ap.add_argument("--window", type=int, default=0)
    ap.add_argument("--verify", default="prob", choices=["prob", "greedy"], help="Eq. 5 (default) or Eq. 4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    w = synth.WORKLOADS[args.workload]
    if args.window:
        w = synth.with_shape(w, window=args.window)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    weights = synth.make_weights(w.shape, w.weight_seed)
    toks, k, lab = rank_inputs(w, rank)

    if args.impl == "reference":
        run_reference(args, w, weights, toks, k, lab)
        return

    import torch
    from paper_2608_18183_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the rollout path has no CPU implementation")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    ctx = binding.Context(w.shape, weights, w.batch, w.window)
    mode = {"full": binding.EXEC_FULL, "compact": binding.EXEC_COMPACT, "hybrid": binding.EXEC_HYBRID,
            "sync": binding.EXEC_SYNC}[args.exec_mode]
    gamma = int(args.gamma_frac * w.batch)

    def params(seed):
        return binding.make_params(w.window, w.history_offset, w.cfg_scale, w.temperature, w.top_k,
                                   binding.VERIFY_GREEDY if args.verify == "greedy" else binding.VERIFY_PROB, mode,
                                   gamma, seed, -1)

    d_toks, d_k, d_lab = (torch.from_numpy(x).cuda() for x in (toks, k, lab))
    d_out = torch.empty((w.batch, w.shape.T), dtype=torch.int32, device="cuda")
    h_toks, h_k, h_lab = (torch.from_numpy(x).pin_memory() for x in (toks, k, lab))
    h_out = torch.empty((w.batch, w.shape.T), dtype=torch.int32).pin_memory()
    tokens_per_step = int((w.shape.T - k).sum())

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """K steps between two events on the library's stream (torch's current stream)."""
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        stats = [fn(args.warmup + i) for i in range(steps)]
        e1.record()
        torch.cuda.synchronize()
        ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        barrier()
        return ms, stats

    dev_step = lambda i: ctx.hbsjd_rollout(d_toks, d_k, d_lab, params(i), d_out)[1]
    host_step = lambda i: ctx.hbsjd_rollout_host(h_toks, h_k, h_lab, params(i), h_out)[1]

    for i in range(args.warmup):
        dev_step(i)
    sampler = ClockSampler(local)
    sampler.start()
    ms, stats = timed(dev_step, args.steps)
    clocks = sampler.stop()
    host_step(0)
    ms_e2e, _ = timed(host_step, args.steps)

    # kernel classes, timed with events on the library's stream over the same K steps
    ctx.hbsjd_profile(True)
    ms_prof, _ = timed(dev_step, args.steps)
    prof = ctx.hbsjd_profile_read()
    ctx.hbsjd_profile(False)
    # what an event pair adds to each timed launch (the launch latency that programmatic dependent launch hides
    # in the untimed pass): reported beside the raw figures, never subtracted from `achieved` / `frac`
    floor_us = ctx.hbsjd_profile_launch_floor(200)

    def net(c):
        """work rate with launches x floor taken out of the class's event time"""
        ms_net = c["ms"] - c["launches"] * floor_us * 1e-3
        return c["work"] / (ms_net * 1e-3) if ms_net > 0 else 0.0

    pk = peaks()
    g = prof["gemm"]
    gemm_tflops = g["work"] / (g["ms"] * 1e-3) / 1e12 if g["ms"] > 0 else 0.0
    roof = {"bound": "tensor", "kernel": "k_gemm_tcgen05 (all decoder GEMMs)", "achieved": gemm_tflops,
            "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
            "frac": gemm_tflops / pk["bf16_tflops_sustained"],
            "traffic": NCU_GEMM_TRAFFIC_BYTES_PER_LAUNCH.get(w.name) if not args.window else None,
            "peak_source": f"{pk['source']} sustained bf16 (kernel timed inside a long step)",
            "avg_launch_ms": g["ms"] / max(g["launches"], 1), "launches": g["launches"],
            "share_of_step": g["ms"] / ms_prof if ms_prof > 0 else None,
            "event_pair_launch_floor_us": floor_us,
            "frac_net_of_launch_floor": net(g) / 1e12 / pk["bf16_tflops_sustained"],
            "frac_of_measured_burst": gemm_tflops / pk["bf16_tflops"],
            "frac_of_nominal": gemm_tflops / NOMINAL_PEAKS["bf16_tflops"],
            "nominal_peak": NOMINAL_PEAKS["bf16_tflops"]}
    # the same class split by the activation rows of the launch: full rounds against the thinning tail of a rollout
    roof["by_rows"] = {
        name: {"launches": b["launches"], "ms_per_step": b["ms"] / args.steps,
               "achieved": b["work"] / (b["ms"] * 1e-3) / 1e12 if b["ms"] > 0 else 0.0,
               "frac": b["work"] / (b["ms"] * 1e-3) / 1e12 / pk["bf16_tflops_sustained"] if b["ms"] > 0 else 0.0,
               "frac_net_of_launch_floor": net(b) / 1e12 / pk["bf16_tflops_sustained"],
               # the same launches against the HBM roofline (operands read once, outputs written): the bound that
               # matters where the rows are few and a launch streams its weight matrix
               "hbm_frac": b["bytes"] / (b["ms"] * 1e-3) / 1e9 / pk["hbm_gbs"] if b["ms"] > 0 else 0.0}
        for name, b in prof["gemm_by_rows"].items()}
    if w.shape.dtype != "bf16":
        roof.update(bound="alu", peak=72.0, peak_source="fp32 CUDA-core FMA: 148 SMs x 128 lanes x 2 x 1.9 GHz")
        roof["frac"] = gemm_tflops / 72.0
        roof["frac_net_of_launch_floor"] = net(g) / 1e12 / 72.0
    other = {}
    for name in ("attention", "accept", "other"):
        c = prof[name]
        gbs = c["work"] / (c["ms"] * 1e-3) / 1e9 if c["ms"] > 0 else 0.0
        other[name] = {"bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                       "frac": gbs / pk["hbm_gbs"], "ms_per_step": c["ms"] / args.steps,
                       "share_of_step": c["ms"] / ms_prof if ms_prof > 0 else None,
                       "frac_net_of_launch_floor": net(c) / 1e9 / pk["hbm_gbs"],
                       "frac_of_nominal": gbs / NOMINAL_PEAKS["hbm_gbs"], "nominal_peak": NOMINAL_PEAKS["hbm_gbs"]}

    value, total_tokens = job_tokens_per_s(tokens_per_step, args.steps, dist, "cuda", ms)
    committed = sum(s["committed"] for s in stats)
    forwards = sum(s["image_forwards"] for s in stats)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.shape.dtype, "data": "synthetic",
            "config": workload_config(w) | {"exec_mode": args.exec_mode, "gamma": gamma,
                                            "verify": "greedy" if args.verify == "greedy" else "probabilistic"},
            "mean_accepted_tokens_per_forward": committed / max(forwards, 1),
            "rounds_per_step": sum(s["rounds"] for s in stats) / args.steps,
            "reject_rate": sum(s["rejects"] for s in stats) / max(forwards, 1),
            "ms_prefill_per_step": sum(s["ms_prefill"] for s in stats) / args.steps,
            "full_rounds": sum(s["full_rounds"] for s in stats), "compact_rounds": sum(s["compact_rounds"] for s in stats),
            "clocks": clocks,
            "e2e": {"value": total_tokens / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(toks.nbytes + k.nbytes + lab.nbytes),
                    "d2h_bytes_per_step": int(toks.nbytes)},
            "gpu_launches": int(sum(s["kernel_launches"] for s in stats)),
            "roofline": roof, "roofline_other": other, "profile_dropped": prof["dropped"]}

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ids, n_rounds, what = sample_plan(w, k)
        done, dt, threads = oracle_sample(w, weights, toks, k, lab, args.warmup, ids, n_rounds)
        line["cpu_baseline"] = {"value": done / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{what} ({done} tokens in {dt:.1f} s)"}
    if rank == 0:
        print(json.dumps(line))
    ctx.hbsjd_destroy()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
