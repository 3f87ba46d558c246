"""Seeded synthetic inputs (initial weights and gradients).

Input generation only: random matrices of the benchmark's recipe.  Nothing of
the optimizer's arithmetic lives here, so the CPU oracle's tests and the CUDA
library's callers can both draw their inputs from this module and see the
same bytes.

Recipe (benchmark configuration 0): a gradient of an m x n matrix is
U diag(s) V^T + 0.1 * mean(s) * N(0,1), with s_i = 1/i for i = 1..min(m,n) and
Haar-distributed U (m x r), V (n x r); initial weights are N(0, 0.02^2).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np


def haar(rng: np.random.Generator, n: int, r: int) -> np.ndarray:
    """n x r matrix with orthonormal columns, Haar-distributed: QR of a Gaussian
    matrix with the sign of R's diagonal folded into Q."""
    q, rr = np.linalg.qr(rng.standard_normal((n, r)))
    return q * np.sign(np.diag(rr))[None, :]


def spectrum(r: int) -> np.ndarray:
    return 1.0 / np.arange(1, r + 1, dtype=np.float64)


def lowrank_plus_noise(rng: np.random.Generator, m: int, n: int, noise: float = 0.1) -> np.ndarray:
    r = min(m, n)
    s = spectrum(r)
    g = (haar(rng, m, r) * s[None, :]) @ haar(rng, n, r).T
    g = g + noise * s.mean() * rng.standard_normal((m, n))
    return g.astype(np.float32)


def init_weights(rng: np.random.Generator, tensors: Sequence) -> List[np.ndarray]:
    out = []
    for t in tensors:
        if getattr(t, "init", "normal") == "ones":
            out.append(np.ones((t.rows, t.cols), dtype=np.float32))
        else:
            out.append((0.02 * rng.standard_normal((t.rows, t.cols))).astype(np.float32))
    return out


def host_gradients(rng: np.random.Generator, tensors: Sequence, shared=None,
                   adamw_std: float = 0.01) -> List[np.ndarray]:
    """One worker's gradients for one step.  Hidden matrices follow the
    low-rank-plus-noise recipe; AdamW tensors (embedding, head, gains) get plain
    Gaussian noise of standard deviation `adamw_std`.  If `shared` (a list of
    per-tensor low-rank parts) is given, only the noise is drawn afresh."""
    gs = []
    for i, t in enumerate(tensors):
        if t.kind == "muon":
            if shared is None:
                gs.append(lowrank_plus_noise(rng, t.rows, t.cols))
            else:
                r = min(t.rows, t.cols)
                e = 0.1 * spectrum(r).mean() * rng.standard_normal((t.rows, t.cols))
                gs.append((shared[i] + e).astype(np.float32))
        else:
            gs.append((adamw_std * rng.standard_normal((t.rows, t.cols))).astype(np.float32))
    return gs


def shared_lowrank(rng: np.random.Generator, tensors: Sequence) -> List:
    """Per-tensor low-rank component shared by all workers in one step."""
    out = []
    for t in tensors:
        if t.kind == "muon":
            r = min(t.rows, t.cols)
            out.append((haar(rng, t.rows, r) * spectrum(r)[None, :]) @ haar(rng, t.cols, r).T)
        else:
            out.append(None)
    return out


# ---------------------------------------------------------------------------
# Device-side generation for the large configurations (torch is used only to
# fill device memory with random numbers).
# ---------------------------------------------------------------------------
def torch_fill_gradients(grad_views, tensors: Sequence, K: int, seed: int, device,
                         adamw_std: float = 0.01) -> None:
    """Fill grad_views[k][i] (torch tensors on `device`, fp32 or bf16) in place.

    The Haar factors are drawn once per distinct shape and the low-rank part is
    shared by all layers and workers of that shape; every (worker, tensor) gets
    independent noise.  This differs from the small-configuration recipe only
    in reusing the low-rank part across layers, which does not change any cost.
    """
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    base = {}
    for t in tensors:
        if t.kind != "muon" or (t.rows, t.cols) in base:
            continue
        m, n = t.rows, t.cols
        r = min(m, n)
        s = 1.0 / torch.arange(1, r + 1, device=device, dtype=torch.float32)

        def _haar(nn):
            q, rr = torch.linalg.qr(torch.randn(nn, r, device=device, generator=gen))
            return q * torch.sign(torch.diagonal(rr))[None, :]

        base[(m, n)] = ((_haar(m) * s[None, :]) @ _haar(n).T, 0.1 * float(s.mean()))
    for k in range(K):
        for i, t in enumerate(tensors):
            dst = grad_views[k][i]
            if t.kind == "muon":
                b, std = base[(t.rows, t.cols)]
                noise = torch.randn(t.rows, t.cols, device=device, generator=gen)
                dst.copy_((b + std * noise).reshape(dst.shape))
            else:
                noise = torch.randn(t.rows, t.cols, device=device, generator=gen)
                dst.copy_((adamw_std * noise).reshape(dst.shape))
