"""Shared helpers for the GPU parity tests: build the CUDA-side object and the
CPU oracle from one workload description and feed both the same bytes."""
import numpy as np

from oracle import muloco_oracle as O
from paper_2505_23725_b200 import configs, synth


def oracle_for(w, init, **over):
    specs = [O.TensorSpec(t.name, t.rows, t.cols, t.kind, t.fragment, t.wd_mult, t.lr_mult) for t in w.tensors]
    kw = dict(K=w.K, H=w.H, J=w.J, muon_lr=w.muon_lr, muon_beta=w.muon_beta, muon_wd=w.muon_wd,
              muon_nesterov=w.muon_nesterov,
              adam_lr=w.muon_lr if w.adam_lr is None else w.adam_lr,
              adam_wd=w.muon_wd if w.adam_wd is None else w.adam_wd,
              adam_beta1=w.adam_beta1, adam_beta2=w.adam_beta2, adam_eps=w.adam_eps,
              outer_lr=w.outer_lr, outer_momentum=w.outer_momentum,
              quant_bits=w.quant_bits, quant_block=w.quant_block)
    kw.update(over)
    return O.MuLoCoOracle(O.OracleConfig(**kw).f32(), specs, init)


def gpu_for(w, init, **kw):
    from paper_2505_23725_b200 import binding
    return binding.MuLoCo(w, "cuda:0", init=init, **kw)


def to_dev(grads_k):
    import torch
    return [[torch.from_numpy(np.ascontiguousarray(g)).cuda() for g in gk] for gk in grads_k]


def relfro(got, ref):
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    d = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / d) if d > 0 else float(np.linalg.norm(got))


def assert_close_1e6(got, ref, what=""):
    """fp32 elementwise steps: within 1e-6 relative, with an absolute floor of
    1e-6 of the tensor's RMS for entries that are themselves near zero."""
    got = np.asarray(got, dtype=np.float64); ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    err = np.abs(got - ref)
    tol = 1e-6 * np.abs(ref) + 1e-6 * rms + 1e-30
    bad = err > tol
    assert not bad.any(), f"{what}: {int(bad.sum())} of {ref.size} entries off; worst ratio {float((err / tol).max()):.2f}"
