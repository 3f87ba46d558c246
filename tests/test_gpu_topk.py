"""GPU parity for top-k sparsification (Section 2, "Compressed Communication"; Algorithm 2 with
top-k as the compressor): the CUDA library through its C ABI against the CPU oracle on the same
seeded inputs.  The kept set is decided by float32 comparisons that both sides take on the same
float32 values, so sparsified arrays, pseudogradients and error-feedback accumulators are compared
bit for bit; theta and u after the outer step within 1e-6."""
import dataclasses

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs
from helpers import assert_close_1e6, gpu_for, oracle_for

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().cpu().numpy()


@pytest.fixture(scope="module")
def ctx():
    w = configs.Workload("hooks", K=1, H=1, J=1, tensors=[], muon_lr=0.02, muon_beta=0.95, muon_wd=0.0,
                         outer_lr=1.0, outer_momentum=0.0)
    g = gpu_for(w, [])
    yield g
    g.close()


def _inputs(kind, n, rng):
    if kind == "normal":
        return rng.standard_normal(n).astype(np.float32)
    if kind == "wide":                       # magnitudes over 12 decades: many exponent bins
        return (rng.standard_normal(n) * 10.0 ** rng.uniform(-9, 3, n)).astype(np.float32)
    if kind == "ties":                       # few distinct magnitudes: the threshold is heavily tied
        return rng.integers(-4, 5, n).astype(np.float32)
    if kind == "sparse":                     # mostly exact zeros, as after an earlier sparsification
        x = rng.standard_normal(n).astype(np.float32)
        x[rng.random(n) < 0.9] = 0.0
        return x
    if kind == "denormal":
        return (rng.standard_normal(n) * 1e-41).astype(np.float32)
    if kind == "zeros":
        return np.zeros(n, np.float32)
    raise ValueError(kind)


@pytest.mark.parametrize("n", [1, 7, 128, 129, 4097, 8192 * 3 + 5, 1_000_003])
@pytest.mark.parametrize("kind", ["normal", "wide", "ties", "sparse", "denormal", "zeros"])
def test_topk_sparsify_vs_oracle(ctx, n, kind):
    import torch
    rng = np.random.default_rng(n * 7 + len(kind))
    x = _inputs(kind, n, rng)
    for frac in (0.005, 0.1, 0.5, 1.0):
        got = _np(ctx.topk_sparsify(torch.from_numpy(x).cuda(), frac))
        want = O.topk_sparsify(x, frac)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (n, kind, frac)
    ctx.sync_status()


def test_topk_sparsify_large_tensor_and_in_place(ctx):
    # an embedding-sized tensor (32000 x 1024), written over its input
    import torch
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(32000 * 1024) * 0.01).astype(np.float32)
    want = O.topk_sparsify(x, 0.01)
    xd = torch.from_numpy(x).cuda()
    ctx._check(ctx.lib.muloco_topk_sparsify(ctx.ctx, xd.data_ptr(), xd.numel(), 0.01, xd.data_ptr()))
    assert np.array_equal(_np(xd), want)
    assert np.count_nonzero(want) == O.topk_count(x.size, 0.01)
    ctx.sync_status()


def test_topk_sparsify_argument_errors_and_empty_input(ctx):
    import torch
    from paper_2505_23725_b200 import binding
    x = torch.zeros(16, device="cuda")
    for bad in (0.0, -0.5, 1.5, float("nan")):
        with pytest.raises(binding.MulocoError) as e:
            ctx.topk_sparsify(x, bad)
        assert e.value.status == binding.EINVAL
    assert ctx.topk_sparsify(torch.zeros(0, device="cuda"), 0.1).numel() == 0


SHAPES = [(128, 352), (352, 128), (5, 100), (3, 7), (1, 1000), (1, 129), (64, 128), (257, 131)]


def _workload(K, frac, ef, J=1, shapes=SHAPES, **kw):
    ts = [configs.Tensor(f"t{i}", r, c, configs.MUON if min(r, c) > 1 else configs.ADAMW, i % J)
          for i, (r, c) in enumerate(shapes)]
    base = dict(muon_lr=0.02, muon_beta=0.9, muon_wd=0.0, outer_lr=0.7, outer_momentum=0.9)
    base.update(kw)
    return configs.Workload("topk", K=K, H=J, J=J, tensors=ts, ns_mode="fp32", topk_fraction=frac,
                            error_feedback=ef, ef_beta=0.9, **base)


@pytest.mark.parametrize("K", [1, 2, 5, 16])
@pytest.mark.parametrize("frac,ef,J", [(0.01, False, 1), (0.25, False, 1), (0.05, True, 1), (0.5, True, 2), (1.0, False, 1)])
def test_topk_sync_vs_oracle(K, frac, ef, J):
    import torch
    w = _workload(K, frac, ef, J)
    rng = np.random.default_rng(900 + 10 * K + int(frac * 100) + ef)
    init = [rng.standard_normal((t.rows, t.cols)).astype(np.float32) * 0.02 for t in w.tensors]
    gpu = gpu_for(w, init)
    orc = oracle_for(w, init, topk_fraction=frac, error_feedback=ef, ef_beta=0.9)
    for rnd in range(3):                                   # three syncs: accumulators and momentum carry over
        for k in range(K):
            for i, t in enumerate(w.tensors):
                drift = (rng.standard_normal((t.rows, t.cols)) * 10.0 ** rng.uniform(-4, -1)).astype(np.float32)
                if rnd == 1 and i == 0:
                    drift = np.round(drift * 64).astype(np.float32) / 64     # a tied threshold in one tensor
                orc.theta_k[k][i][...] = orc.theta_g[i] + drift
                gpu.theta_k[k][i].copy_(torch.from_numpy(orc.theta_k[k][i]).cuda())
        frags = [-1] if J == 1 else list(range(J))
        for f in frags:
            gpu.outer_sync(f)
            orc.outer_sync(f)
        gpu.sync_status()
        for i in range(gpu.n):
            if ef:
                for k in range(K):
                    assert np.array_equal(_np(gpu.ef[k][i]), orc.ef[k][i]), f"E k={k} tensor {i} round {rnd}"
            assert_close_1e6(_np(gpu.theta_g[i]), orc.theta_g[i], f"theta_g {i} round {rnd}")
            assert_close_1e6(_np(gpu.outer_u[i]), orc.outer_u[i], f"u {i} round {rnd}")
            for k in range(K):
                assert np.array_equal(_np(gpu.theta_k[k][i]), _np(gpu.theta_g[i]))
            orc.theta_g[i][...] = _np(gpu.theta_g[i]); orc.outer_u[i][...] = _np(gpu.outer_u[i])
    gpu.close()


@pytest.mark.parametrize("ef", [False, True])
def test_topk_pseudogradient_is_bit_exact(ef):
    # eta_out = 1, mu = 0, u = 0: u_new = Psi exactly and theta_new = theta - Psi with theta = 0
    import torch
    K, frac, shape = 4, 0.03, (300, 1000)
    w = _workload(K, frac, ef, shapes=[shape], outer_lr=1.0, outer_momentum=0.0)
    rng = np.random.default_rng(19)
    init = [np.zeros(shape, dtype=np.float32)]
    gpu = gpu_for(w, init)
    efs = [np.zeros(shape, np.float32) for _ in range(K)] if ef else None
    tg = init[0].copy()
    for rnd in range(2):
        ths = [(tg + 0.05 * rng.standard_normal(shape)).astype(np.float32) for _ in range(K)]
        for k in range(K):
            gpu.theta_k[k][0].copy_(torch.from_numpy(ths[k]).cuda())
        gpu.outer_u[0].zero_()
        gpu.outer_sync(-1)
        gpu.sync_status()
        psi = O.sparsified_pseudogradient(tg, ths, frac, efs, 0.9)
        assert np.array_equal(_np(gpu.outer_u[0]), psi), rnd
        kept_by_someone = np.count_nonzero(psi)
        assert O.topk_count(psi.size, frac) <= kept_by_someone <= K * O.topk_count(psi.size, frac)
        if ef:
            for k in range(K):
                assert np.array_equal(_np(gpu.ef[k][0]), efs[k])
        tg = _np(gpu.theta_g[0]).copy()
    gpu.close()


def test_topk_configuration_errors_and_nonfinite_delta():
    from paper_2505_23725_b200 import binding
    z = [np.zeros((8, 128), np.float32)]
    for kw in (dict(quant_bits=8), dict(topk_fraction=1.5), dict(topk_fraction=-0.1)):
        w = dataclasses.replace(_workload(2, 0.1, False, shapes=[(8, 128)]), **kw)
        with pytest.raises(binding.MulocoError) as e:
            gpu_for(w, z)
        assert e.value.status == binding.EINVAL
    gpu = gpu_for(_workload(2, 0.1, False, shapes=[(8, 128)]), z)
    gpu.theta_k[1][0][2, 5] = float("inf")
    gpu.outer_sync(-1)
    with pytest.raises(binding.MulocoError) as e:
        gpu.sync_status()
    assert e.value.status == binding.ENONFINITE
    gpu.close()


def test_topk_sync_at_benchmark_shapes():
    """The 416M-shaped model's tensor shapes (embedding and head of 32000 x 1024, hidden matrices of
    1024 x 1024, 1024 x 2816 and 2816 x 1024, gain vectors) with two layers and K = 4: one sync with
    top-k and error feedback; the oracle recomputes one tensor of every distinct shape in full."""
    import torch
    from paper_2505_23725_b200 import binding
    K, frac = 4, 0.01
    ts = configs.llama_tensors(2, 1024, 2816, vocab=32000, norms=True)
    w = configs.Workload("topk-416M-shapes", K=K, H=1, J=1, tensors=ts, muon_lr=0.02, muon_beta=0.9, muon_wd=0.0,
                         outer_lr=0.7, outer_momentum=0.9, topk_fraction=frac, error_feedback=True, ef_beta=0.9)
    opt = binding.MuLoCo(w, "cuda:0", init_seed=11, alloc_grads=False)
    gen = torch.Generator(device="cuda"); gen.manual_seed(3)
    for k in range(K):
        opt.flat_theta_k[k].add_(torch.empty_like(opt.flat_theta_k[k]).normal_(0.0, 1e-3, generator=gen))
        opt.flat_ef[k].normal_(0.0, 1e-4, generator=gen)
    opt.flat_u.normal_(0.0, 1e-3, generator=gen)
    first = {}
    for i, t in enumerate(ts):
        first.setdefault((t.rows, t.cols), i)
    sample = sorted(first.values())
    snap = {i: (_np(opt.theta_g[i]).copy(), _np(opt.outer_u[i]).copy(), [_np(opt.theta_k[k][i]).copy() for k in range(K)],
                [_np(opt.ef[k][i]).copy() for k in range(K)]) for i in sample}
    opt.outer_sync(-1)
    opt.sync_status()
    for i, (tg, u, reps, efs) in snap.items():
        psi = O.sparsified_pseudogradient(tg, reps, frac, efs, 0.9)
        O.outer_nesterov(tg, u, psi, outer_lr=w.outer_lr, outer_momentum=w.outer_momentum)
        for k in range(K):
            assert np.array_equal(_np(opt.ef[k][i]), efs[k]), f"E k={k} {ts[i].name}"
        assert_close_1e6(_np(opt.theta_g[i]), tg, f"theta_g {ts[i].name}")
        assert_close_1e6(_np(opt.outer_u[i]), u, f"u {ts[i].name}")
        assert np.array_equal(_np(opt.theta_k[K - 1][i]), _np(opt.theta_g[i]))
    opt.close()
