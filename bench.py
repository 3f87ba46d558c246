#!/usr/bin/env python
"""Benchmark of the MuLoCo optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 0..4] [--impl reference]

One "step" is one full MuLoCo round of the workload: H inner steps of all K
workers (Muon prologue + Newton-Schulz + update, AdamW) followed by the outer
synchronisation of every fragment at its scheduled step -- every row of the hot
path runs in each timed step.  metric = optimizer-step parameter updates per
second, K * N_params * H per round.  Prints ONE JSON line on rank 0.

Default workload: benchmark configuration 2 (416M-shaped, K=16, H=30), the one
the target is quoted on.  With --gpus N > 1 every rank runs its own independent
K-worker problem on its own GPU (weak scaling, no data-path collective: the
method keeps its K workers on one GPU).
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

METRIC = "optimizer-step params/sec (inner Muon + outer sync) at K workers"
UNIT = "param-updates/s"

# Measured constants of the Newton-Schulz kernel (one launch = all 15 products of a chunk), quoted
# beside the live timings.  Source: one `ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,
# sm__pipe_tensor_cycles_active...` capture per shape mix of `bench.py --muon-only K 2 D F` (two
# layers, the configuration's K; both launches of an inner step).  Key: (d_model, ff).
#   bytes: DRAM bytes read + written per hidden-matrix parameter, worker and inner step.  Traffic
#          grows in proportion to the number of matrices, so a full launch is this figure times the
#          parameters it covers.
#   tensor_pct: sm__pipe_tensor_cycles_active, % of peak, of the two launches (square group, wide group).
NS_KERNEL_COUNTERS = {
    (768, 2048): {"bytes": 4.36606e9 / (14155776 * 8), "tensor_pct": (47.3, 56.8)},
    (1024, 2816): {"bytes": 17.98357e9 / (25690112 * 16), "tensor_pct": (64.8, 69.5)},
    (2048, 5632): {"bytes": 38.66371e9 / (102760448 * 8), "tensor_pct": (76.4, 78.7)},
    (3072, 8192): {"bytes": 48.34281e9 / (226492416 * 4), "tensor_pct": (79.6, 80.3)},
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx = float(f[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        med = sm[len(sm) // 2] if sm else None
        return {"sm_mhz": med, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(sm)}


def rank_seeds(base_seed: int, rank: int):
    """Seeds of rank `rank`'s independent K-worker problem: (initial weights, gradients)."""
    return base_seed + 1000 * rank, base_seed + 17 * rank


def max_over_ranks(ms: float, dist=None, device="cpu") -> float:
    """Device time of the slowest rank (every rank gets the same number back)."""
    if dist is None:
        return float(ms)
    import torch
    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(world: int, units_per_rank: float, ms_per_step: float) -> float:
    """Units all ranks processed per second: every rank runs its own full problem (weak scaling)."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def oracle_cores():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle_sample(w, seed=0, muon_reps=4):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload:
    one layer's hidden matrices for `muon_reps` (layer, worker) pairs (Muon; one pair
    when the matrices are very large), a 2^22-element AdamW slice, and the outer sync
    of three hidden matrices over all K replicas.  Returns the extrapolated parameter
    updates per second over a full round, a description of the sample and the seconds
    of oracle work."""
    import numpy as np
    from oracle import muloco_oracle as O
    from paper_2505_23725_b200 import configs

    rng = np.random.default_rng(seed)
    layer = [t for t in w.tensors if t.kind == configs.MUON and t.name.startswith("l0.")]
    reps_muon = muon_reps if layer and max(max(t.rows, t.cols) for t in layer) <= 4096 else 1   # (layer, worker) pairs sampled
    pm = sum(t.numel for t in layer) * reps_muon
    t_muon = 0.0
    for _ in range(reps_muon):
        Ws = [(0.02 * rng.standard_normal((t.rows, t.cols))).astype(np.float32) for t in layer]
        Ms = [np.zeros_like(x) for x in Ws]
        Gs = [rng.standard_normal((t.rows, t.cols)).astype(np.float32) for t in layer]
        t0 = time.perf_counter()
        for W, M, G in zip(Ws, Ms, Gs):
            O.muon_step(W, M, G, lr=w.muon_lr, beta=w.muon_beta, wd=w.muon_wd, nesterov=w.muon_nesterov)
        t_muon += time.perf_counter() - t0
    pa = 1 << 22
    th = rng.standard_normal(pa).astype(np.float32); m = np.zeros_like(th); v = np.zeros_like(th)
    g = rng.standard_normal(pa).astype(np.float32)
    t0 = time.perf_counter()
    O.adamw_step(th, m, v, g, t=1, lr=w.muon_lr, wd=w.muon_wd)
    t_adam = time.perf_counter() - t0
    t_sync, ps = 0.0, 0
    for t in layer[:2] + layer[-1:]:
        tg = (0.02 * rng.standard_normal((t.rows, t.cols))).astype(np.float32)
        u = np.zeros_like(tg)
        reps = [tg + (1e-3 * rng.standard_normal(tg.shape)).astype(np.float32) for _ in range(w.K)]
        t0 = time.perf_counter()
        if w.quant_bits:
            _, _, psi = O.quantize_blocks(O.pseudogradient_f32(tg, reps), w.quant_bits, w.quant_block)
        else:
            psi = O.pseudogradient(tg, reps)
        O.outer_nesterov(tg, u, psi, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
        for r in reps:
            r[...] = tg
        t_sync += time.perf_counter() - t0
        ps += t.numel
    n_muon = w.n_muon_params
    n_adam = w.n_params - n_muon
    t_round = w.H * w.K * (n_muon / pm * t_muon + n_adam / pa * t_adam) + w.n_params / ps * t_sync
    value = w.K * w.n_params * w.H / t_round
    sample = (f"{reps_muon} (layer, worker) Muon steps ({reps_muon * len(layer)} matrices, {pm} params, {t_muon:.2f} s), "
              f"AdamW on 2^22 elements ({t_adam:.3f} s), outer sync of {ps} params x K={w.K} replicas "
              f"({t_sync:.2f} s); extrapolated linearly to a full round of H={w.H} steps")
    return value, sample, t_muon + t_adam + t_sync


def run_reference(args, w):
    """--impl reference: the CPU oracle on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, tot = [], 0.0
    sample = ""
    for _ in range(args.warmup):
        time_oracle_sample(w)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v, sample, _ = time_oracle_sample(w)
        vals.append(v)
    tot = time.perf_counter() - t0
    value = sum(vals) / len(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(w, args):
    return {"workload": f"configs[{args.config}] {w.name}: K={w.K} H={w.H} J={w.J}, {w.n_params} params/replica "
                        f"({w.n_muon_params} on Muon), quant={w.quant_bits or 'none'}, NS {w.ns_mode}",
            "step": "one round = H inner steps (all K workers) + scheduled outer syncs",
            "l2": "inputs_larger_than_l2", "parallelism": "K replicas on one GPU; ranks independent"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--inner", default="muon", choices=["muon", "adamw"],
                    help="adamw: the DiLoCo baseline (AdamW on every tensor) instead of MuLoCo")
    ap.add_argument("--shard-workers", action="store_true",
                    help="with --gpus N: spread the workload's K workers over the N ranks (K/N each) and run the outer "
                         "sync as reduce-scatter + all-gather over NCCL (muloco_shard_*); total work is fixed "
                         "(strong scaling).  Default: every rank runs its own K-worker problem (weak scaling)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workspace-gb", type=float, default=0.0)
    ap.add_argument("--ns-only", type=int, nargs=3, metavar=("BATCH", "ROWS", "COLS"), default=None,
                    help="kernel study: time muloco_newton_schulz (bf16 engine) on a batch of one shape")
    ap.add_argument("--sync-only", type=int, nargs=3, metavar=("K", "MPARAMS", "QUANT"), default=None,
                    help="kernel study: time muloco_outer_sync on MPARAMS million parameters, K replicas, "
                         "QUANT in {0, 4, 8}")
    ap.add_argument("--quant-stages", type=int, default=1, help="with --sync-only: 2 = per-worker quantisation + "
                    "second quantisation of the mean (Algorithm 2)")
    ap.add_argument("--quant-block", type=int, default=128, help="with --sync-only: 32/64/128, or 0 = row-wise")
    ap.add_argument("--ef", action="store_true", help="with --sync-only --quant-stages 2 or --topk: error feedback")
    ap.add_argument("--topk", type=float, default=0.0, help="with --sync-only (QUANT 0): top-k sparsification of "
                    "every worker's delta, the fraction kept")
    ap.add_argument("--adamw-only", type=int, nargs=2, metavar=("K", "MPARAMS"), default=None,
                    help="kernel study: time the AdamW part of muloco_inner_step on MPARAMS million parameters")
    ap.add_argument("--grad-dtype", choices=["f32", "bf16"], default="f32", help="with --muon-only: gradient type")
    ap.add_argument("--muon-only", type=int, nargs=4, metavar=("K", "LAYERS", "D", "F"), default=None,
                    help="kernel study: muloco_inner_step on LAYERS layers of hidden matrices only "
                         "(prologue + Newton-Schulz with the fused parameter update), K workers")
    args = ap.parse_args()
    if args.muon_only:
        run_muon_only(args)
        return
    if args.ns_only:
        run_ns_only(args)
        return
    if args.sync_only or args.adamw_only:
        run_elementwise_only(args)
        return

    from paper_2505_23725_b200 import configs
    w = configs.workload(args.config)
    if args.inner == "adamw":
        w = configs.diloco_baseline(w)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2505_23725_b200 import binding, synth
    import __graft_entry__ as entry

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    if rank == 0:
        entry.build()
    distributed = world > 1
    if distributed:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
        dist.barrier()
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(dev)

    seed_init, seed_grad = rank_seeds(w.seed, rank)
    sharded = bool(args.shard_workers)
    K_total = w.K
    if sharded:
        import dataclasses
        if w.K % world != 0:
            raise SystemExit(f"--shard-workers: K={w.K} is not a multiple of {world} ranks")
        w = dataclasses.replace(w, K=w.K // world)       # this rank's share of the workers
        seed_init = rank_seeds(w.seed, 0)[0]             # every rank starts from the same global parameters
        if not distributed:                              # one rank: a communicator of its own
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1"); os.environ.setdefault("MASTER_PORT", "29533")
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(f"cuda:{local_rank}"))
    opt = binding.MuLoCo(w, dev, init_seed=seed_init, alloc_grads=True,
                         workspace_bytes=int(args.workspace_gb * (1 << 30)))
    synth.torch_fill_gradients(opt.grads, w.tensors, w.K, seed_grad, opt.device)
    torch.cuda.synchronize()

    def one_round(t0):
        """H inner steps with the streaming schedule; returns the step counter."""
        t = t0
        for _ in range(w.H):
            opt.inner_step(-1, None, 1.0)
            t += 1
            for f in opt.fragments_due(t):
                if sharded:
                    wire_bytes[0] += opt.sharded_outer_sync(f, dist)
                    sync_calls[0] += 3
                else:
                    opt.outer_sync(f)
                    sync_calls[0] += 1
        return t

    sync_calls = [0]
    wire_bytes = [0]

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    t = 0
    for _ in range(args.warmup):
        t = one_round(t)
    opt.sync_status()
    opt.set_timing(True)
    opt.get_timings()
    sync_calls[0] = 0
    wire_bytes[0] = 0
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    torch.cuda.cudart().cudaProfilerStart()      # lets `ncu --profile-from-start off` see the timed region only
    e0.record(opt.stream)
    for _ in range(args.steps):
        t = one_round(t)
    e1.record(opt.stream)
    barrier()
    torch.cuda.cudart().cudaProfilerStop()
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    phases, launches = opt.get_timings()
    opt.set_timing(False)
    opt.sync_status()
    ms_total = max_over_ranks(ms_total, dist if distributed else None, dev)
    ms_per_step = ms_total / args.steps
    units_per_round = w.K * w.n_params * w.H              # this rank's workers
    value = whole_job_value(world, units_per_round, ms_per_step)

    # ---- roofline of the dominant kernel (Newton-Schulz tensor-core GEMMs) ----------------
    peaks = load_peaks()
    inner_steps = args.steps * w.H
    n_adam = w.n_params - w.n_muon_params
    adam_bytes = n_adam * w.K * (28.0 if w.grad_dtype == "f32" else 26.0) * inner_steps
    if w.n_muon_params > 0:
        ns_ms_per_inner = phases["ns"] / inner_steps
        ns_tflops = w.ns_flops_credited() / (ns_ms_per_inner * 1e-3) / 1e12
        peak_tf = peaks["bf16_tflops_sustained"]
        ns_launches_per_inner = ns_launches_per_inner_step(launches, sync_calls[0], inner_steps, n_adam > 0)
        shape_key = None
        for tn in w.tensors:
            if tn.name.endswith(".w1"):
                shape_key = (tn.rows, tn.cols)
                break
        counters = NS_KERNEL_COUNTERS.get(shape_key)
        traffic = (counters["bytes"] * w.n_muon_params * w.K / ns_launches_per_inner) if counters else None
        executed = ns_tflops * w.ns_flops_executed() / w.ns_flops_credited()
        roofline = {"bound": "tensor", "kernel": "ns_tc_kernel (all Gram / polynomial / apply products of Newton-Schulz)",
                    "achieved": ns_tflops, "peak": peak_tf, "unit": "TFLOP/s", "frac": ns_tflops / peak_tf,
                    "peak_source": f"{peaks['source']} sustained bf16 matmul (kernel timed inside a long step)",
                    "frac_of_burst_peak": ns_tflops / peaks["bf16_tflops"],
                    "frac_of_nominal_2250": ns_tflops / 2250.0,
                    "executed_tflops": executed, "executed_frac": executed / peak_tf,
                    "launches_per_inner_step": ns_launches_per_inner,
                    "traffic": traffic,
                    "traffic_unit": "bytes per launch (average over the launches of an inner step)" if counters else
                                    "null: no counter capture exists for this shape mix",
                    "tensor_pipe_pct_ncu": list(counters["tensor_pct"]) if counters else None,
                    "tensor_pipe_source": "sm__pipe_tensor_cycles_active of the 2-layer case of this shape mix, "
                                          "launch alone (square group, wide group)",
                    "flops_convention": "credited 5*(4 s^2 l + 2 s^3) per matrix; symmetric products run upper-triangle tiles only",
                    "ms_per_inner_step": ns_ms_per_inner}
    else:
        # DiLoCo baseline: the inner step is the AdamW kernel alone (HBM-bound)
        ns_tflops = None
        gbs = adam_bytes / (phases["adamw"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "adamw_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": gbs / peaks["hbm_gbs"], "peak_source": f"{peaks['source']} copy bandwidth",
                    "traffic": adam_bytes / inner_steps,
                    "traffic_unit": "bytes per launch (ncu: DRAM traffic of this kernel equals its algorithmic bytes)"}
    n_sync_rounds = args.steps
    sync_gbs = w.sync_bytes() * n_sync_rounds / (phases["sync"] * 1e-3) / 1e9 if phases["sync"] > 0 else None
    adam_gbs = adam_bytes / (phases["adamw"] * 1e-3) / 1e9 if phases["adamw"] > 0 else None
    pro_bytes = w.n_muon_params * w.K * (14.0 if w.grad_dtype == "f32" else 12.0) * inner_steps
    pro_gbs = pro_bytes / (phases["prologue"] * 1e-3) / 1e9 if phases["prologue"] > 0 else None
    phase_report = {
        "ms_per_round": {k: v / args.steps for k, v in phases.items()},
        "ns_tflops_credited": ns_tflops,
        "ns_frac_of_burst_peak": (ns_tflops / peaks["bf16_tflops"]) if ns_tflops else None,
        "ns_frac_of_nominal_2250": (ns_tflops / 2250.0) if ns_tflops else None,
        "ns_tflops_executed": (ns_tflops * w.ns_flops_executed() / w.ns_flops_credited()) if ns_tflops else None,
        "sync_gbs": sync_gbs, "sync_frac_of_hbm": (sync_gbs / peaks["hbm_gbs"]) if sync_gbs else None,
        "adamw_gbs": adam_gbs, "adamw_frac_of_hbm": (adam_gbs / peaks["hbm_gbs"]) if adam_gbs else None,
        "prologue_gbs": pro_gbs, "hbm_peak_gbs": peaks["hbm_gbs"],
    }

    # ---- end to end through the host-buffer entry points ----------------------------------
    e2e = None
    if not args.no_e2e and not sharded:      # the host-buffer entry points drive the single-GPU sync
        e2e = run_e2e(opt, w, torch, dist if distributed else None, world)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, sample, _ = time_oracle_sample(w, muon_reps=12)      # 10-15 s of oracle work on 16 host cores
        cpu = {"value": v, "unit": UNIT, "cores": oracle_cores(), "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if sharded else "weak",
                "vs_baseline": None, "dtype": "bf16" if w.ns_mode == "bf16" else "f32", "data": "synthetic",
                "config": workload_config(w, args), "clocks": clocks, "e2e": e2e,
                "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu, "phases": phase_report}
        if sharded:
            line["config"]["parallelism"] = (f"K={K_total} workers spread over {world} ranks ({w.K} each); outer sync = "
                                             "local delta sums, NCCL reduce-scatter, Nesterov step on the shard, NCCL "
                                             "all-gather, broadcast into the local replicas")
            line["sharded_sync"] = {"wire_bytes_per_rank_per_round": wire_bytes[0] / args.steps}
        print(json.dumps(line))
    opt.close()
    if sharded and not distributed:
        dist.destroy_process_group()
    if distributed:
        dist.barrier()
        dist.destroy_process_group()


def ns_launches_per_inner_step(total_launches, sync_launches, inner_steps, has_adamw):
    """Newton-Schulz launches per inner step, from the library's own launch counter: an inner step
    launches, per workspace chunk, 2 staging kernels and 1 kernel that runs all 15 products, plus one
    AdamW kernel."""
    per_inner = (total_launches - sync_launches) / inner_steps - (1 if has_adamw else 0)
    return int(round(per_inner / 3.0))


def run_ns_only(args):
    """Small case for kernel studies and ncu captures: the standalone Newton-Schulz call
    (15 tensor-core launches per call) on BATCH matrices of ROWS x COLS."""
    import torch
    from paper_2505_23725_b200 import binding, configs
    import __graft_entry__ as entry
    entry.build()
    batch, rows, cols = args.ns_only
    w = configs.Workload("ns-only", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                         outer_lr=1.0, outer_momentum=0.0)
    opt = binding.MuLoCo(w, "cuda:0", init=[], workspace_bytes=int(args.workspace_gb * (1 << 30)))
    gen = torch.Generator(device="cuda"); gen.manual_seed(0)
    X = torch.randn(batch, rows, cols, device="cuda", generator=gen).to(torch.bfloat16)
    for _ in range(args.warmup):
        opt.newton_schulz(X, out_dtype=torch.bfloat16)
    opt.set_timing(True); opt.get_timings()
    torch.cuda.synchronize()
    torch.cuda.cudart().cudaProfilerStart()
    for _ in range(args.steps):
        opt.newton_schulz(X, out_dtype=torch.bfloat16)
    ph, launches = opt.get_timings()
    torch.cuda.cudart().cudaProfilerStop()
    opt.sync_status()
    s, l = min(rows, cols), max(rows, cols)
    flops = batch * 5.0 * (4.0 * s * s * l + 2.0 * s ** 3)
    ms = ph["ns"] / args.steps
    peaks = load_peaks()
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({"ns_only": [batch, rows, cols], "ms_per_call": ms, "tflops_credited": tf,
                      "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
                      "frac_of_burst_peak": tf / peaks["bf16_tflops"], "prologue_ms": ph["prologue"] / args.steps,
                      "launches": int(launches)}))
    opt.close()


def run_muon_only(args):
    """Small case of the real inner step for ncu captures: hidden matrices only, so the
    launches are exactly those of the benchmark's Muon path at a fraction of its depth."""
    import torch
    from paper_2505_23725_b200 import binding, configs, synth
    import __graft_entry__ as entry
    entry.build()
    K, L, d, F = args.muon_only
    w = configs.mini_workload(K=K, H=1, J=1, ns_mode="bf16", L=L, d=d, F=F, muon_lr=4.42e-2, muon_beta=0.9,
                              muon_wd=6.25e-4, grad_dtype=args.grad_dtype)
    opt = binding.MuLoCo(w, "cuda:0", init_seed=1, alloc_grads=True,
                         workspace_bytes=int(args.workspace_gb * (1 << 30)))
    synth.torch_fill_gradients(opt.grads, w.tensors, w.K, 3, opt.device)
    for _ in range(args.warmup):
        opt.inner_step(-1, None, 1.0)
    opt.set_timing(True); opt.get_timings()
    torch.cuda.synchronize()
    torch.cuda.cudart().cudaProfilerStart()
    for _ in range(args.steps):
        opt.inner_step(-1, None, 1.0)
    ph, launches = opt.get_timings()
    torch.cuda.cudart().cudaProfilerStop()
    opt.sync_status()
    peaks = load_peaks()
    tf = w.ns_flops_credited() / (ph["ns"] / args.steps * 1e-3) / 1e12
    print(json.dumps({"muon_only": [K, L, d, F], "params_per_replica": w.n_params, "ns_ms": ph["ns"] / args.steps,
                      "prologue_ms": ph["prologue"] / args.steps,
                      "prologue_gbs": w.n_params * K * (14.0 if args.grad_dtype == "f32" else 12.0)
                      / (ph["prologue"] / args.steps * 1e-3) / 1e9,
                      "ns_tflops_credited": tf,
                      "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"], "launches": int(launches)}))
    opt.close()


def run_elementwise_only(args):
    """Small cases for kernel studies and ncu captures of the two streaming kernels: the
    outer synchronisation (--sync-only) or AdamW (--adamw-only) over a few large tensors."""
    import torch
    from paper_2505_23725_b200 import binding, configs
    import __graft_entry__ as entry
    entry.build()
    sync = args.sync_only is not None
    K, mparams = (args.sync_only[0], args.sync_only[1]) if sync else args.adamw_only
    quant = args.sync_only[2] if sync else 0
    rows = max(1, mparams * 1000000 // (8 * 4096))
    ts = [configs.Tensor(f"t{i}", rows, 4096, configs.ADAMW, 0) for i in range(8)]
    w = configs.Workload("elementwise-only", K=K, H=1, J=1, tensors=ts, muon_lr=0.02, muon_beta=0.9, muon_wd=0.01,
                         outer_lr=0.7, outer_momentum=0.9, quant_bits=quant,
                         quant_stages=args.quant_stages if sync else 1, error_feedback=bool(args.ef and sync),
                         quant_block=args.quant_block, topk_fraction=args.topk if sync else 0.0)
    opt = binding.MuLoCo(w, "cuda:0", init_seed=1, alloc_grads=not sync)
    gen = torch.Generator(device="cuda"); gen.manual_seed(0)
    if sync:
        for k in range(K):
            opt.flat_theta_k[k].normal_(0.0, 0.02, generator=gen)
    else:
        for k in range(K):
            opt.flat_grads[k].normal_(0.0, 0.01, generator=gen)
    def sync_call():
        # a sync leaves theta_k = theta, so without new drift every later delta would be zero; the
        # radix select of top-k depends on the data, so the replicas drift again before every call
        # (outside the timed span: the phase timer brackets the library's own launches only)
        if args.topk > 0:
            for k in range(K):
                opt.flat_theta_k[k].add_(noise.normal_(0.0, 1e-3, generator=gen))
        opt.outer_sync(-1)
    noise = torch.empty_like(opt.flat_theta_g) if sync and args.topk > 0 else None
    call = sync_call if sync else (lambda: opt.inner_step(-1, None, 1.0))
    for _ in range(args.warmup):
        call()
    opt.set_timing(True); opt.get_timings()
    torch.cuda.synchronize()
    torch.cuda.cudart().cudaProfilerStart()
    for _ in range(args.steps):
        call()
    ph, launches = opt.get_timings()
    torch.cuda.cudart().cudaProfilerStop()
    opt.sync_status()
    peaks = load_peaks()
    n = w.n_params
    if sync:
        ms = ph["sync"] / args.steps
        nbytes = n * ((16.0 if args.ef else 8.0) * K + 16.0)      # error feedback: K more reads and writes
        if args.topk > 0:                                         # three histogram passes read theta and every delta
            nbytes += n * 3 * ((8.0 if args.ef else 4.0) * K + 4.0)
    else:
        ms = ph["adamw"] / args.steps
        nbytes = n * K * 28.0
    gbs = nbytes / (ms * 1e-3) / 1e9
    print(json.dumps({"sync_only" if sync else "adamw_only": [K, mparams, quant], "topk": args.topk, "params": n,
                      "ms_per_call": ms,
                      "gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"], "launches": int(launches)}))
    opt.close()


def run_e2e(opt, w, torch, dist, world):
    """The same round through muloco_inner_step_host / muloco_outer_sync_host: every inner
    step copies that step's gradients from pinned host memory, every sync reads the new
    global parameters back to the host.  One warm-up inner step, two timed rounds (both reported;
    the value is their mean)."""
    import psutil
    elt = 2 if w.grad_dtype == "bf16" else 4
    set_bytes = opt.flat_numel * elt
    avail = psutil.virtual_memory().available
    # every rank of the node pins its own sets: share the host memory that is free now
    n_sets = w.K if set_bytes * w.K * 1.5 < avail / max(world, 1) else 1
    # drop the device-resident gradients: in this mode they come from the host each step
    opt.grads = None; opt.flat_grads = None; opt._grad_table_all = None
    torch.cuda.empty_cache()
    host_flat = [torch.empty(opt.flat_numel, dtype=opt.gdtype).pin_memory() for _ in range(n_sets)]
    for hf in host_flat:
        hf.normal_(0.0, 0.01)
    host = [[host_flat[k % n_sets][o:o + t.numel].view(t.rows, t.cols) for o, t in zip(opt.offsets, w.tensors)]
            for k in range(w.K)]
    out_flat = torch.empty(opt.flat_numel, dtype=torch.float32).pin_memory()
    out = [out_flat[o:o + t.numel].view(t.rows, t.cols) for o, t in zip(opt.offsets, w.tensors)]
    opt.inner_step_host(-1, host, 1.0)
    torch.cuda.synchronize()
    rounds = 2
    per_round, d2h, t = [], 0, 0
    for _ in range(rounds):
        if dist:
            dist.barrier()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(opt.stream)
        d2h = 0
        for _ in range(w.H):
            opt.inner_step_host(-1, host, 1.0)
            t += 1
            for f in opt.fragments_due(t):
                opt.outer_sync_host(f, out)
                d2h += sum(tt.numel for tt in w.tensors if tt.fragment == f) * 4
        e1.record(opt.stream)
        torch.cuda.synchronize()
        per_round.append(max_over_ranks(e0.elapsed_time(e1), dist, opt.device))
    opt.sync_status()
    ms = sum(per_round) / len(per_round)
    h2d = w.n_params * elt * w.K * w.H
    return {"value": whole_job_value(world, w.K * w.n_params * w.H, ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "rounds_timed": rounds, "ms_per_round": per_round,
            "host_grad_sets": n_sets}


if __name__ == "__main__":
    main()
