"""The worker-sharded outer sync with two gloo ranks on CPU: the host-side choreography
(binding.sharded_outer_sync: layout, reduce-scatter, step on the shard, all-gather, broadcast) and
its byte accounting, with a numpy stand-in for the three CUDA passes that follows their
documented staging layout.  The result on both ranks must be the oracle's outer step over all
workers; the wire bytes must be 2 * 4 * stage_floats * (G - 1) / G."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import contextlib, json, sys
sys.path.insert(0, {root!r})
import numpy as np, torch
import torch.distributed as dist
from oracle import muloco_oracle as O
from paper_2505_23725_b200 import binding

rank, world = int(sys.argv[1]), 2
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
K_local, n, eta, mu = 3, 1000, 0.7, 0.9                     # 1000 elements = 8 units, the last one short

class CpuRank:
    # stand-in for the three CUDA passes: same staging layout (unit-major, 128 floats per unit)
    def __init__(self, theta, replicas):
        self.theta = theta.copy(); self.u = np.zeros_like(theta); self.rep = [r.copy() for r in replicas]
        self.n_units = -(-n // 128)
    def shard_layout(self, fragment, world, rank):
        us = -(-self.n_units // world)
        return us * world * 128, us * 128
    def new_buffer(self, k): return torch.zeros(k, dtype=torch.float32)
    def stream_context(self): return contextlib.nullcontext()
    def shard_delta(self, fragment, world, stage):
        acc = np.zeros(n, np.float32)
        for r in self.rep: acc = acc + (self.theta - r)
        stage.zero_(); stage[:n] = torch.from_numpy(acc)
    def shard_step(self, fragment, world, rank, reduced, out):
        lo = rank * reduced.numel(); hi = min(n, lo + reduced.numel())
        out.zero_()
        if hi > lo:
            psi = reduced.numpy()[:hi - lo].astype(np.float64) / (len(self.rep) * world)
            th, u = self.theta[lo:hi].copy(), self.u[lo:hi].copy()
            O.outer_nesterov(th, u, psi, outer_lr=eta, outer_momentum=mu)
            self.theta[lo:hi] = th; self.u[lo:hi] = u
            out[:hi - lo] = torch.from_numpy(th)
    def shard_broadcast(self, fragment, world, theta_all):
        self.theta[...] = theta_all.numpy()[:n]
        for r in self.rep: r[...] = self.theta

rng = np.random.default_rng(5)                               # the same stream on both ranks
theta = (0.02 * rng.standard_normal(n)).astype(np.float32)
reps = [theta + (1e-3 * rng.standard_normal(n)).astype(np.float32) for _ in range(K_local * world)]
me = CpuRank(theta, reps[rank * K_local:(rank + 1) * K_local])
wire = binding.sharded_outer_sync(me, -1, dist)
ref_t, ref_u = theta.copy(), np.zeros_like(theta)
O.outer_nesterov(ref_t, ref_u, O.pseudogradient(theta, reps), outer_lr=eta, outer_momentum=mu)
stage_floats, shard_floats = me.shard_layout(-1, world, rank)
lo, hi = rank * shard_floats, min(n, (rank + 1) * shard_floats)
print(json.dumps(dict(rank=rank, wire=wire, stage_floats=stage_floats, shard_floats=shard_floats,
      theta_err=float(np.max(np.abs(me.theta - ref_t) / (1e-6 * np.abs(ref_t) + 1e-6 * np.sqrt(np.mean(ref_t ** 2))))),
      u_err=float(np.max(np.abs(me.u[lo:hi] - ref_u[lo:hi]))),
      replicas_equal=bool(all(np.array_equal(r, me.theta) for r in me.rep)),
      theta_sum=float(me.theta.astype(np.float64).sum()))))
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_run_the_sharded_sync_and_count_its_bytes():
    code = WORKER.format(root=ROOT, port=_free_port())
    procs = [subprocess.Popen([sys.executable, "-c", code, str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True) for r in range(2)]
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=300)
        assert p.returncode == 0, e[-3000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    for d in outs:
        assert d["stage_floats"] == 8 * 128 and d["shard_floats"] == 4 * 128      # 8 units, 4 per rank
        assert d["wire"] == 2 * 4 * d["stage_floats"] * (2 - 1) // 2
        assert d["theta_err"] < 1.0 and d["u_err"] < 1e-9 and d["replicas_equal"]     # theta within 1e-6 (relative + rms floor)
    assert outs[0]["theta_sum"] == outs[1]["theta_sum"]                          # both ranks hold the same theta


def test_wire_bytes_formula():
    from paper_2505_23725_b200 import binding
    assert binding.shard_wire_bytes(1024, 1) == 0
    assert binding.shard_wire_bytes(1024, 2) == 4096
    assert binding.shard_wire_bytes(8 * 128 * 1000, 8) == 2 * 4 * 8 * 128 * 1000 * 7 // 8
