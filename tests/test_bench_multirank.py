"""The N > 1 path of bench.py on CPU: two gloo ranks.  The method keeps its K workers on
one GPU, so ranks run independent problems with no data-path collective; what the ranks
share is the timing protocol (barrier, max over ranks, whole-job aggregate) and the rule
that only rank 0 prints.  Those host-side pieces are exercised here without a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
dist.barrier()
ms = bench.max_over_ranks(100.0 + 50.0 * rank, dist, "cpu")      # rank 1 is the slow one
val = bench.whole_job_value(2, 1.0e9, ms)
print(json.dumps({{"rank": rank, "ms": ms, "value": val, "seeds": bench.rank_seeds(2, rank)}}))
dist.barrier()
dist.destroy_process_group()
"""


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_the_slowest_time_and_aggregate():
    code = WORKER.format(root=ROOT, port=_free_port())
    procs = [subprocess.Popen([sys.executable, "-c", code, str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True) for r in range(2)]
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == 150.0                 # max over ranks, same on both
    assert outs[0]["value"] == pytest.approx(2 * 1.0e9 / 0.150)     # units of BOTH ranks / slowest time
    assert outs[0]["seeds"] != outs[1]["seeds"]                    # ranks run different problems


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--config", "0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--config", "0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
