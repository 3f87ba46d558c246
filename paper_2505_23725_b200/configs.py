"""Workload tables: tensor lists and hyper-parameters of the benchmark configurations.

Pure data (shapes, roles, fragment ids, hyper-parameters).  None of the
method's arithmetic lives here, so both the CUDA library's callers and the
tests of the CPU oracle may read it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

MUON, ADAMW = "muon", "adamw"


@dataclass
class Tensor:
    name: str
    rows: int
    cols: int
    kind: str = MUON
    fragment: int = 0
    wd_mult: float = 1.0
    lr_mult: Optional[float] = None     # None: sqrt(cols/rows) for Muon, 1 for AdamW
    init: str = "normal"                # "normal": N(0, 0.02^2); "ones": 1.0 (norm gains)

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass
class Workload:
    name: str
    K: int
    H: int
    J: int
    tensors: List[Tensor]
    muon_lr: float
    muon_beta: float
    muon_wd: float
    outer_lr: float
    outer_momentum: float
    muon_nesterov: bool = True
    ns_mode: str = "bf16"               # "bf16" | "fp32"
    quant_bits: int = 0                 # 0 (none), 8, 4 or 2
    quant_block: int = 128
    quant_stages: int = 1               # 2: per-worker quantisation, fp32 mean, second quantisation
    error_feedback: bool = False        # Algorithm 2's accumulators (needs quant_stages = 2 or top-k)
    ef_beta: float = 1.0
    topk_fraction: float = 0.0          # > 0: top-k sparsification of every worker's delta
    adam_lr: Optional[float] = None     # None: same as muon_lr
    adam_wd: Optional[float] = None     # None: same as muon_wd
    adam_beta1: float = 0.9
    adam_beta2: float = 0.99
    adam_eps: float = 1e-8
    seed: int = 0
    grad_dtype: str = "f32"
    notes: str = ""

    @property
    def n_params(self) -> int:
        return sum(t.numel for t in self.tensors)

    @property
    def n_muon_params(self) -> int:
        return sum(t.numel for t in self.tensors if t.kind == MUON)

    def ns_flops_credited(self) -> float:
        """5 * (4 s^2 l + 2 s^3) per hidden matrix, s = min dim, l = max dim, all K workers."""
        f = 0.0
        for t in self.tensors:
            if t.kind == MUON:
                s, l = min(t.rows, t.cols), max(t.rows, t.cols)
                f += 5.0 * (4.0 * s * s * l + 2.0 * s ** 3)
        return f * self.K

    def ns_flops_executed(self) -> float:
        """What the tensor-core engine multiplies: the two symmetric products of an iteration (Gram,
        polynomial) run only the tiles on and above the diagonal -- T(T+1)/2 of T^2 tiles of 256 rows
        (one tile for matrices of up to 128 rows) -- the third product runs in full."""
        f = 0.0
        for t in self.tensors:
            if t.kind == MUON:
                s, l = min(t.rows, t.cols), max(t.rows, t.cols)
                T = 1 if s <= 128 else -(-s // 256)
                tri = (T + 1) / (2.0 * T)
                f += 5.0 * (tri * 2.0 * s * s * l + tri * 2.0 * s ** 3 + 2.0 * s * s * l)
        return f * self.K

    def sync_bytes(self, fragment: int = -1) -> float:
        """(8K + 16) bytes per parameter of the fragment: K+2 fp32 reads and K+2 fp32 writes."""
        n = sum(t.numel for t in self.tensors if fragment < 0 or t.fragment == fragment)
        return n * (8.0 * self.K + 16.0)


def llama_tensors(L: int, d: int, F: int, J: int = 1, vocab: int = 0,
                  norms: bool = False) -> List[Tensor]:
    """Llama-style hidden matrices (Wq, Wk, Wv, Wo d x d; SwiGLU W1, W3 d x F; W2 F x d),
    optionally with embedding (vocab x d), head (d x vocab) and RMSNorm gains on AdamW.
    Layers are split into J contiguous fragments; the embedding goes with the
    first fragment, the final norm and the head with the last."""
    ts: List[Tensor] = []
    if vocab:
        ts.append(Tensor("embed", vocab, d, ADAMW, 0))
    for l in range(L):
        f = (l * J) // L
        for nm in ("wq", "wk", "wv", "wo"):
            ts.append(Tensor(f"l{l}.{nm}", d, d, MUON, f))
        ts.append(Tensor(f"l{l}.w1", d, F, MUON, f))
        ts.append(Tensor(f"l{l}.w3", d, F, MUON, f))
        ts.append(Tensor(f"l{l}.w2", F, d, MUON, f))
        if norms:
            ts.append(Tensor(f"l{l}.attn_norm", 1, d, ADAMW, f, wd_mult=0.0, init="ones"))
            ts.append(Tensor(f"l{l}.ffn_norm", 1, d, ADAMW, f, wd_mult=0.0, init="ones"))
    if norms:
        ts.append(Tensor("final_norm", 1, d, ADAMW, J - 1, wd_mult=0.0, init="ones"))
    if vocab:
        ts.append(Tensor("head", d, vocab, ADAMW, J - 1))
    return ts


def workload(idx: int) -> Workload:
    """The five benchmark configurations (index 0..4)."""
    if idx == 0:
        return Workload("cfg0-tiny", K=2, H=2, J=1, tensors=llama_tensors(2, 128, 352),
                        muon_lr=0.02, muon_beta=0.95, muon_wd=0.01, outer_lr=0.7,
                        outer_momentum=0.9, ns_mode="fp32", seed=0)
    if idx == 1:
        return Workload("cfg1-150M-shaped", K=8, H=30, J=1,
                        tensors=llama_tensors(12, 768, 2048, vocab=32000, norms=True),
                        muon_lr=1.25e-1, muon_beta=0.9, muon_wd=6.25e-4, outer_lr=0.9,
                        outer_momentum=0.8, seed=1)
    if idx == 2:
        return Workload("cfg2-416M-shaped", K=16, H=30, J=1,
                        tensors=llama_tensors(24, 1024, 2816, vocab=32000, norms=True),
                        muon_lr=4.42e-2, muon_beta=0.9, muon_wd=6.25e-4, outer_lr=1.0,
                        outer_momentum=0.9, seed=2)
    if idx == 3:
        return Workload("cfg3-1.76B-shaped-int4-streaming", K=8, H=100, J=4,
                        tensors=llama_tensors(24, 2048, 5632, J=4, vocab=32000, norms=True),
                        muon_lr=1.56e-2, muon_beta=0.9, muon_wd=1.25e-4, outer_lr=0.9,
                        outer_momentum=0.8, quant_bits=4, seed=3)
    if idx == 4:
        return Workload("cfg4-3.1B-shaped-int8", K=4, H=30, J=1,
                        tensors=llama_tensors(28, 3072, 8192, vocab=32000, norms=True),
                        muon_lr=1.56e-2, muon_beta=0.9, muon_wd=2.5e-4, outer_lr=0.9,
                        outer_momentum=0.8, quant_bits=8, seed=4, grad_dtype="bf16")
    raise ValueError("workload index must be 0..4")


def diloco_baseline(w: Workload) -> Workload:
    """The DiLoCo baseline of the paper's comparisons: the same workload with AdamW as the inner
    optimizer of EVERY tensor (Section 5, "DiLoCo"), outer step unchanged."""
    import dataclasses
    ts = [dataclasses.replace(t, kind=ADAMW) for t in w.tensors]
    return dataclasses.replace(w, tensors=ts, name=w.name + "-diloco")


def cosine_lr_scale(step: int, total_steps: int, warmup_steps: int = 0,
                    final_fraction: float = 0.1) -> float:
    """The learning-rate multiplier for inner step `step` (0-based) of `total_steps`: a linear
    warm-up over `warmup_steps`, then a half cosine from 1 down to `final_fraction` of the peak
    (Section 5: cosine decay to 0.1x the maximum).  The result is the `lr_scale` argument of the
    inner step; the library itself holds no schedule."""
    import math
    if total_steps <= 0 or not 0 <= step:
        raise ValueError("need total_steps > 0 and step >= 0")
    if not 0 <= warmup_steps < total_steps:
        raise ValueError("warmup_steps must lie in [0, total_steps)")
    if step < warmup_steps:
        return (step + 1) / warmup_steps
    span = max(1, total_steps - 1 - warmup_steps)
    t = min(1.0, (step - warmup_steps) / span)
    return final_fraction + (1.0 - final_fraction) * 0.5 * (1.0 + math.cos(math.pi * t))


def mini_workload(K=2, H=2, J=1, quant_bits=0, ns_mode="fp32", L=2, d=128, F=352,
                  vocab=0, norms=False, **kw) -> Workload:
    """A small custom workload for tests."""
    base = dict(muon_lr=0.02, muon_beta=0.95, muon_wd=0.01, outer_lr=0.7, outer_momentum=0.9)
    base.update(kw)
    return Workload("mini", K=K, H=H, J=J, tensors=llama_tensors(L, d, F, J, vocab, norms),
                    ns_mode=ns_mode, quant_bits=quant_bits, **base)
