"""The library's stand-ins for a memory checker, on the GPU.

1. The debug build (libmuloco_debug.so, -DMULOCO_DEBUG) compiles index checks into the kernels
   (work-list cursors, matrix slots, tile coordinates, segment and unit indices); a failed check
   raises a status flag instead of touching memory.  A whole small round, ragged Newton-Schulz
   shapes, quantised and row-wise syncs and AdamW run against it, with the workspace canaries
   switched on: the status must stay clean, the canaries intact and the results equal to the
   oracle's.  It runs in a child process because the library path is fixed when the binding is
   first imported.
2. The canary check itself: the host overwrites one canary byte (a memset on the stream; no
   kernel misbehaves) and muloco_check_workspace names the region.
"""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs, synth
from helpers import gpu_for, relfro

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, {root!r}); sys.path.insert(0, {tests!r})
import numpy as np, torch
from oracle import muloco_oracle as O
from paper_2505_23725_b200 import binding, configs, synth
from helpers import oracle_for, gpu_for, to_dev, relfro, assert_close_1e6
assert binding.LIB_PATH.endswith("libmuloco_debug.so")

def watched(g):
    g.debug_set(binding.DEBUG_CANARIES, 1)
    return g

# a whole round of configuration 0 (fp32 engine), then the same shapes through the bf16 engine
for mode, tol in (("fp32", 1e-5), ("bf16", 2e-2)):
    w = configs.workload(0)
    rng = np.random.default_rng(w.seed)
    init = synth.init_weights(rng, w.tensors)
    gpu = watched(gpu_for(w, init, ns_mode=mode))
    orc = oracle_for(w, init)
    for _ in range(w.H):
        gs = [synth.host_gradients(rng, w.tensors) for _ in range(w.K)]
        gpu.inner_step(-1, to_dev(gs)); orc.inner_step_all(gs)
    gpu.outer_sync(-1); orc.outer_sync(-1)
    gpu.sync_status(); gpu.check_workspace()
    for i in range(len(w.tensors)):
        assert relfro(gpu.theta_g[i].cpu().numpy(), orc.theta_g[i]) < tol, (mode, i)
    gpu.close()

# ragged Newton-Schulz shapes, both engines, several tiles and a ragged tail, batches over a ring
ns = configs.Workload("ns-only", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                      outer_lr=1.0, outer_momentum=0.0)
ctx = watched(gpu_for(ns, []))
rng = np.random.default_rng(11)
for batch, m, n in [(2, 128, 352), (2, 352, 128), (1, 200, 300), (2, 257, 513), (1, 96, 1031), (3, 511, 129),
                    (40, 256, 256), (1, 8, 24), (70, 130, 64)]:
    X = np.stack([synth.lowrank_plus_noise(rng, m, n) for _ in range(batch)])
    for mode, tol in (("fp32", 1e-4), ("bf16", 2e-2)):
        out = ctx.newton_schulz(torch.from_numpy(X).cuda(), ns_mode=mode).cpu().numpy()
        ctx.sync_status(); ctx.check_workspace()
        for b in range(batch):
            assert relfro(out[b], O.newton_schulz(X[b])) < tol, (batch, m, n, mode)
ctx.close()

# AdamW tensors, a block-quantised sync in fragments, a row-wise two-stage sync with error feedback
for kw in (dict(quant_bits=4, J=2, H=2), dict(quant_bits=8, quant_block=0, quant_stages=2, error_feedback=True)):
    w = configs.mini_workload(K=3, L=2, d=64, F=96, vocab=300, norms=True, ns_mode="bf16", **kw)
    rng = np.random.default_rng(5)
    init = synth.init_weights(rng, w.tensors)
    gpu = watched(gpu_for(w, init))
    for _ in range(2):
        gpu.inner_step(-1, to_dev([synth.host_gradients(rng, w.tensors) for _ in range(w.K)]))
    for f in range(w.J):
        gpu.outer_sync(f)
    gpu.sync_status(); gpu.check_workspace()
    for k in range(w.K):
        for i in range(len(w.tensors)):
            assert torch.equal(gpu.theta_k[k][i], gpu.theta_g[i])
    gpu.close()
print("debug build: clean")
"""


def test_debug_build_runs_clean_with_canaries_intact():
    from paper_2505_23725_b200 import build
    lib = build.build_library(debug=True)
    env = dict(os.environ, MULOCO_LIBRARY=lib)
    code = CHILD.format(root=ROOT, tests=os.path.join(ROOT, "tests"))
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "debug build: clean" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


@pytest.mark.parametrize("mode,region,name", [("bf16", 1, "ring"), ("bf16", 0, "X0"), ("fp32", 3, "B")])
def test_an_overwritten_canary_is_reported(mode, region, name):
    import torch
    from paper_2505_23725_b200 import binding
    w = configs.Workload("ns-only", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                         outer_lr=1.0, outer_momentum=0.0)
    ctx = gpu_for(w, [])
    rng = np.random.default_rng(3)
    X = np.stack([synth.lowrank_plus_noise(rng, 256, 384) for _ in range(3)])
    Xd = torch.from_numpy(X).cuda()
    ctx.debug_set(binding.DEBUG_CANARIES, 1)
    ctx.newton_schulz(Xd, ns_mode=mode)
    ctx.sync_status(); ctx.check_workspace()            # nothing wrote outside its region
    ctx.debug_set(binding.DEBUG_CORRUPT_CANARY, region)
    out = ctx.newton_schulz(Xd, ns_mode=mode).cpu().numpy()
    ctx.sync_status()                                   # no kernel misbehaved ...
    with pytest.raises(binding.MulocoError) as e:       # ... but the canary after the region is gone
        ctx.check_workspace()
    assert e.value.status == binding.ESTATE and f"'{name}'" in str(e.value)
    ctx.check_workspace()                               # reported once
    for b in range(3):
        assert relfro(out[b], O.newton_schulz(X[b])) < (2e-2 if mode == "bf16" else 1e-4)
    ctx.newton_schulz(Xd, ns_mode=mode)
    ctx.sync_status(); ctx.check_workspace()            # the switch was one-shot
    ctx.close()
