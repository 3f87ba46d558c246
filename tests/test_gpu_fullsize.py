"""GPU parity at the benchmark's sizes, in the launch configuration bench.py times.

The CPU oracle needs seconds per matrix at these shapes, so the CUDA library
runs the whole workload and the oracle recomputes a SAMPLE of its outputs, one
tensor at a time, from the inputs the GPU had: for the inner step one hidden
matrix of every distinct shape in the first layer for worker 0 and in the
last layer for worker K-1, plus slices of the AdamW tensors; for the outer sync slices of
the same tensors over all K replicas.  Tolerances as everywhere: momentum,
AdamW and the outer step 1e-6 relative, bf16 Newton-Schulz update 2e-2
relative Frobenius, quantised pseudogradient bit-exact.

Every configuration runs at its full depth (configs[3]: 24 layers, 142 GB of state and
gradients; configs[4]: 28 layers, 162 GB), so the workspace chunking, the descriptor tables
and the launch shapes are the ones bench.py times; the oracle's cost is per sampled
matrix, not per layer.
"""

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs, synth
from helpers import assert_close_1e6, relfro

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().float().cpu().numpy()


def _sampled_tensors(w):
    """One tensor per distinct (kind, shape): its first occurrence (first layer) and its
    last occurrence (last layer), as two index lists."""
    first, last = {}, {}
    for i, t in enumerate(w.tensors):
        key = (t.kind, t.rows, t.cols)
        first.setdefault(key, i)
        last[key] = i
    return sorted(first.values()), sorted(last.values())


def _check_inner_and_sync(w, seed, slice_rows=64):
    import torch
    from paper_2505_23725_b200 import binding

    opt = binding.MuLoCo(w, "cuda:0", init_seed=seed, alloc_grads=True)
    synth.torch_fill_gradients(opt.grads, w.tensors, w.K, seed + 1, opt.device)
    K = w.K
    first, last = _sampled_tensors(w)
    sample = sorted(set(first) | set(last))
    workers = sorted({0, K - 1})
    pairs = [(0, i) for i in first] + [(K - 1, i) for i in last]      # worker 0 x first layer, worker K-1 x last
    adam_lr = w.muon_lr if w.adam_lr is None else w.adam_lr
    adam_wd = w.muon_wd if w.adam_wd is None else w.adam_wd

    opt.inner_step(-1, None, 1.0)                       # step 1: fills the momenta
    opt.sync_status()
    # fresh gradients for the compared step, so that momentum and gradient point in different
    # directions (with the same gradient twice, Nesterov's g + beta m is parallel to m)
    synth.torch_fill_gradients(opt.grads, w.tensors, w.K, seed + 2, opt.device)
    before = {}
    for k, i in dict.fromkeys(pairs):
        t = w.tensors[i]
        rows = slice(None) if t.kind == configs.MUON else slice(0, min(slice_rows, t.rows))
        before[(k, i)] = (rows, _np(opt.theta_k[k][i][rows]).copy(), _np(opt.state1[k][i][rows]).copy(),
                          _np(opt.state2[k][i][rows]).copy() if t.kind == configs.ADAMW else None,
                          _np(opt.grads[k][i][rows]).copy())
    opt.inner_step(-1, None, 1.0)                       # step 2: compared
    opt.sync_status()
    worst_ns = 0.0
    for (k, i), (rows, W0, M0, V0, G) in before.items():
        t = w.tensors[i]
        W1 = _np(opt.theta_k[k][i][rows])
        if t.kind == configs.MUON:
            W, M = W0.copy(), M0.copy()
            O.muon_step(W, M, G, lr=w.muon_lr, beta=w.muon_beta, wd=w.muon_wd, nesterov=w.muon_nesterov)
            assert_close_1e6(_np(opt.state1[k][i]), M, f"{w.name} momentum k={k} {t.name}")
            err = relfro(W1.astype(np.float64) - W0, W.astype(np.float64) - W0)
            worst_ns = max(worst_ns, err)
            assert err < 2e-2, f"{w.name} Muon update k={k} {t.name} ({t.rows}x{t.cols}): {err:.3e}"
        else:
            th, m, v = W0.copy(), M0.copy(), V0.copy()
            O.adamw_step(th, m, v, G, t=2, lr=adam_lr, beta1=w.adam_beta1, beta2=w.adam_beta2, eps=w.adam_eps,
                         wd=adam_wd, wd_mult=t.wd_mult)
            assert_close_1e6(_np(opt.state1[k][i][rows]), m, f"{w.name} Adam m k={k} {t.name}")
            assert_close_1e6(_np(opt.state2[k][i][rows]), v, f"{w.name} Adam v k={k} {t.name}")
            assert_close_1e6(W1, th, f"{w.name} AdamW theta k={k} {t.name}")

    # ---- outer sync of every fragment that is due over one period, sampled the same way ----
    for frag in range(w.J):
        ids = [i for i in sample if w.tensors[i].fragment == frag]
        snap = {}
        for i in ids:
            t = w.tensors[i]
            rows = slice(0, min(slice_rows, t.rows))
            snap[i] = (rows, _np(opt.theta_g[i][rows]).copy(), _np(opt.outer_u[i][rows]).copy(),
                       [_np(opt.theta_k[k][i][rows]).copy() for k in range(K)])
        untouched = [i for i in sample if w.tensors[i].fragment != frag]
        keep = {i: _np(opt.theta_k[0][i][:8]).copy() for i in untouched}
        opt.outer_sync(frag)
        opt.sync_status()
        for i, (rows, tg, u, reps) in snap.items():
            t = w.tensors[i]
            if w.quant_bits:
                psi32 = O.pseudogradient_f32(tg, reps)
                _, _, psi = O.quantize_blocks(psi32, w.quant_bits, w.quant_block)
                psi = psi.astype(np.float64)
            else:
                psi = O.pseudogradient(tg, reps)
            tg2, u2 = tg.copy(), u.copy()
            O.outer_nesterov(tg2, u2, psi, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
            got = _np(opt.theta_g[i][rows])
            assert_close_1e6(got, tg2, f"{w.name} theta_g {t.name}")
            assert_close_1e6(_np(opt.outer_u[i][rows]), u2, f"{w.name} u {t.name}")
            for k in workers:
                assert np.array_equal(_np(opt.theta_k[k][i][rows]), got), f"{w.name} broadcast k={k} {t.name}"
        for i, v in keep.items():
            assert np.array_equal(_np(opt.theta_k[0][i][:8]), v), f"{w.name}: fragment {frag} touched {w.tensors[i].name}"
    opt.close()
    del opt
    torch.cuda.empty_cache()
    return worst_ns


def test_config2_full_size_sampled_parity():
    w = configs.workload(2)
    assert w.K == 16 and w.n_params == 373867520
    worst = _check_inner_and_sync(w, seed=202)
    assert worst < 2e-2


def test_config1_full_size_sampled_parity():
    _check_inner_and_sync(configs.workload(1), seed=101)


def test_config3_full_size_int4_streaming_sampled_parity():
    w = configs.workload(3)
    assert w.J == 4 and w.quant_bits == 4 and {t.fragment for t in w.tensors} == {0, 1, 2, 3}
    assert w.K == 8 and sum(1 for t in w.tensors if t.name.endswith(".wq")) == 24
    _check_inner_and_sync(w, seed=303)


def test_config4_full_size_int8_bf16_grads_sampled_parity():
    w = configs.workload(4)
    assert w.quant_bits == 8 and w.grad_dtype == "bf16"
    assert w.K == 4 and sum(1 for t in w.tensors if t.name.endswith(".wq")) == 28
    _check_inner_and_sync(w, seed=404)
