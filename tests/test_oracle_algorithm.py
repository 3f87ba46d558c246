"""Pins for the oracle's Algorithm-1 driver: special cases with known answers
and the nuclear-norm identity of Proposition 4.2.  No GPU needed."""
import math

import numpy as np
import pytest

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import synth


def specs_small():
    return [O.TensorSpec("a", 8, 8), O.TensorSpec("b", 8, 20), O.TensorSpec("c", 20, 8),
            O.TensorSpec("e", 16, 6, kind="adamw"), O.TensorSpec("g", 1, 8, kind="adamw", wd_mult=0.0)]


def grads_for(rng, specs):
    return [rng.standard_normal((s.rows, s.cols)).astype(np.float32) for s in specs]


def ulp_diff(a, b):
    ai = a.view(np.int32).astype(np.int64); bi = b.view(np.int32).astype(np.int64)
    ai = np.where(ai < 0, -(ai & 0x7FFFFFFF), ai); bi = np.where(bi < 0, -(bi & 0x7FFFFFFF), bi)
    return np.abs(ai - bi)


# ---- P4: K=1, eta_out=1, mu=0 reproduces H plain inner steps ----------------
def test_k1_outer_identity_reproduces_plain_muon():
    rng = np.random.default_rng(0)
    specs = specs_small()
    init = synth.init_weights(rng, [type("T", (), dict(rows=s.rows, cols=s.cols, init="normal")) for s in specs])
    cfg = O.OracleConfig(K=1, H=3, muon_lr=0.05, muon_beta=0.9, muon_wd=0.01, adam_lr=0.01,
                         adam_wd=0.01, outer_lr=1.0, outer_momentum=0.0)
    orc = O.MuLoCoOracle(cfg, specs, init)
    # plain loop over the single-tensor step functions
    W = [w.copy() for w in init]; S1 = [np.zeros_like(w) for w in init]; S2 = [np.zeros_like(w) for w in init]
    for h in range(1, 4):
        g = grads_for(rng, specs)
        orc.inner_step(0, g)
        for i, s in enumerate(specs):
            if s.kind == "muon":
                O.muon_step(W[i], S1[i], g[i], lr=0.05, beta=0.9, wd=0.01)
            else:
                O.adamw_step(W[i], S1[i], S2[i], g[i], t=h, lr=0.01, wd=0.01, wd_mult=s.wd_mult)
    orc.outer_sync(-1)
    for i in range(len(specs)):
        # theta_g - (theta_g - theta_1) = theta_1 up to one rounding of the difference
        assert ulp_diff(orc.theta_g[i], W[i]).max() <= 1
        assert np.array_equal(orc.theta_k[0][i], orc.theta_g[i])
        assert np.allclose(orc.outer_u[i], (init[i].astype(np.float64) - W[i]), atol=1e-7)


# ---- P5: identical gradients: pseudogradient equals one worker's delta -------
def test_identical_gradients_give_single_worker_delta():
    rng = np.random.default_rng(1)
    specs = specs_small()
    init = [rng.standard_normal((s.rows, s.cols)).astype(np.float32) * 0.02 for s in specs]
    cfg = O.OracleConfig(K=4, H=2, muon_lr=0.05, adam_lr=0.01, outer_lr=0.7, outer_momentum=0.9)
    orc = O.MuLoCoOracle(cfg, specs, init)
    for h in range(2):
        g = grads_for(rng, specs)
        orc.inner_step_all([g] * 4)
    delta0 = [init[i].astype(np.float64) - orc.theta_k[0][i].astype(np.float64) for i in range(len(specs))]
    for k in range(1, 4):
        for i in range(len(specs)):
            assert np.array_equal(orc.theta_k[k][i], orc.theta_k[0][i])
    orc.outer_sync(-1)
    for i in range(len(specs)):
        assert np.array_equal(orc.last_psi[i], delta0[i])          # K = 4: exact
        # first sync from u = 0: theta = theta0 - eta (1 + mu) psi
        want = init[i].astype(np.float64) - 0.7 * 1.9 * delta0[i]
        assert np.allclose(orc.theta_g[i], want, rtol=0, atol=1e-7)
        for k in range(4):
            assert np.array_equal(orc.theta_k[k][i], orc.theta_g[i])


# ---- P6: Proposition 4.2 ------------------------------------------------------
@pytest.mark.parametrize("m,n", [(8, 12), (12, 8), (10, 10)])
def test_proposition_4_2_nuclear_norm_identity(m, n):
    """||Psi||_* = (sqrt(r)/K) sum_k sum_h rho alpha ||psi||_F, with psi the inner
    steps (weight decay off), alpha the effective step size and rho the cosine
    between each step and Psi* = U V^T of the pseudogradient."""
    rng = np.random.default_rng(m * 31 + n)
    K, H = 3, 4
    lr = 0.05
    specs = [O.TensorSpec("w", m, n)]
    init = [(0.02 * rng.standard_normal((m, n))).astype(np.float32)]
    cfg = O.OracleConfig(K=K, H=H, muon_lr=lr, muon_beta=0.9, muon_wd=0.0)
    orc = O.MuLoCoOracle(cfg, specs, init)
    steps = []                                   # the recorded optimizer steps psi^{(t+h,k)}
    for h in range(H):
        for k in range(K):
            before = orc.theta_k[k][0].astype(np.float64)
            orc.inner_step(k, [rng.standard_normal((m, n)).astype(np.float32)])
            steps.append((before - orc.theta_k[k][0].astype(np.float64)))
    psi = O.pseudogradient(orc.theta_g[0], [orc.theta_k[k][0] for k in range(K)])
    U, s, Vt = np.linalg.svd(psi, full_matrices=False)
    r = min(m, n)
    star = U @ Vt
    rhs = 0.0
    for st in steps:                             # alpha folded into st (alpha * psi)
        rho = np.sum(st * star) / (np.linalg.norm(st) * np.linalg.norm(star))
        rhs += rho * np.linalg.norm(st)
    rhs *= math.sqrt(r) / K
    assert s.sum() == pytest.approx(rhs, rel=1e-5)
    # each recorded step is eta' * O with ||O||_F in the Newton-Schulz band around sqrt(r)
    eta = lr * math.sqrt(n / m)
    for st in steps:
        assert 0.6 * math.sqrt(r) < np.linalg.norm(st) / eta < 1.25 * math.sqrt(r)


# ---- P10: streaming ------------------------------------------------------------
def test_streaming_touches_each_fragment_once_per_period():
    rng = np.random.default_rng(3)
    J, H, K = 2, 4, 2
    specs = [O.TensorSpec("a", 8, 8, fragment=0), O.TensorSpec("b", 8, 16, fragment=1),
             O.TensorSpec("e", 4, 8, kind="adamw", fragment=0), O.TensorSpec("h", 8, 4, kind="adamw", fragment=1)]
    init = [(0.02 * rng.standard_normal((s.rows, s.cols))).astype(np.float32) for s in specs]
    cfg = O.OracleConfig(K=K, H=H, J=J, muon_lr=0.05, adam_lr=0.01, outer_lr=0.7, outer_momentum=0.9)
    orc = O.MuLoCoOracle(cfg, specs, init)
    touched = {i: 0 for i in range(len(specs))}
    for t in range(1, H + 1):
        orc.inner_step_all([grads_for(rng, specs) for _ in range(K)])
        snap_g = [w.copy() for w in orc.theta_g]
        snap_k = [[w.copy() for w in orc.theta_k[k]] for k in range(K)]
        for f in O.fragments_due(t, H, J):
            orc.outer_sync(f)
            for i, s in enumerate(specs):
                if s.fragment == f:
                    touched[i] += 1
                    assert not np.array_equal(orc.theta_g[i], snap_g[i])
                    for k in range(K):
                        assert np.array_equal(orc.theta_k[k][i], orc.theta_g[i])
                else:                           # tensors of other fragments are untouched
                    assert np.array_equal(orc.theta_g[i], snap_g[i])
                    for k in range(K):
                        assert np.array_equal(orc.theta_k[k][i], snap_k[k][i])
    assert all(v == 1 for v in touched.values())


def test_j1_equals_non_streaming_and_state_is_kept_across_syncs():
    rng = np.random.default_rng(4)
    specs = specs_small()
    init = [(0.02 * rng.standard_normal((s.rows, s.cols))).astype(np.float32) for s in specs]
    cfg = O.OracleConfig(K=2, H=2, J=1, muon_lr=0.05, adam_lr=0.01, outer_lr=0.7, outer_momentum=0.9)
    a = O.MuLoCoOracle(cfg, specs, init); b = O.MuLoCoOracle(cfg, specs, init)
    gs = [[grads_for(rng, specs) for _ in range(2)] for _ in range(2)]
    for h in range(2):
        a.inner_step_all(gs[h]); b.inner_step_all(gs[h])
    a.outer_sync(-1); b.outer_sync(0)
    for i in range(len(specs)):
        assert np.array_equal(a.theta_g[i], b.theta_g[i])
    # inner optimizer state survives the sync
    assert any(np.any(m != 0) for m in a.state1[0])
    assert a.worker_step == [2, 2]


def test_quantised_sync_uses_dequantised_pseudogradient():
    rng = np.random.default_rng(6)
    specs = [O.TensorSpec("w", 4, 300)]
    init = [rng.standard_normal((4, 300)).astype(np.float32)]
    cfg = O.OracleConfig(K=2, H=1, muon_lr=0.05, outer_lr=0.5, outer_momentum=0.0, quant_bits=4)
    orc = O.MuLoCoOracle(cfg, specs, init)
    orc.inner_step_all([[rng.standard_normal((4, 300)).astype(np.float32)] for _ in range(2)])
    psi32 = O.pseudogradient_f32(orc.theta_g[0], [orc.theta_k[k][0] for k in range(2)])
    _, _, deq = O.quantize_blocks(psi32, 4, 128)
    orc.outer_sync(-1)
    assert np.array_equal(orc.last_psi[0], deq)
    assert len(np.unique(np.round(deq[0, :128] / np.abs(deq[0, :128]).max() * 7))) <= 15
    want = init[0].astype(np.float64) - 0.5 * deq
    assert np.allclose(orc.theta_g[0], want, atol=1e-7)


def test_config_validation():
    with pytest.raises(ValueError):
        O.MuLoCoOracle(O.OracleConfig(K=2, H=10, J=4), [], [])
    with pytest.raises(ValueError):
        O.MuLoCoOracle(O.OracleConfig(K=0, H=10), [], [])
