"""CPU oracle for the MuLoCo optimizer step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step restatement of what the paper defines, in the
paper's order and notation.  It exists to check the CUDA library and to be
timed as the CPU baseline; nothing in the product path may import it, and it
imports nothing from the product (no shared kernels, tables or helpers).

Arithmetic: every state array is stored as float32 (as on the GPU).  Each
operation loads to float64, computes, and rounds ONCE to float32 on store.
The only exception is the compressors (block quantiser, top-k) and the
pseudogradient that feeds them, which are written in exact float32 operations
so that integer codes and kept sets are reproducible bit for bit.

Hyper-parameters cross the library boundary as float32; callers that want to
mirror the library pass values that are already float32-representable.

What each function follows:
  newton_schulz        Section 2 "Muon": X_j = p(X_{j-1} X_{j-1}^T) X_{j-1}
  muon_step            Section 2 "Muon" (momentum, update with decoupled decay),
                       Section 5 "MuLoCo" (learning-rate rescale sqrt(n/m))
  adamw_step           Section 4.3 (first/second moments, decoupled decay)
  pseudogradient       Eq. (2); Algorithm 1 (parameter delta, all-reduce of the outer delta)
  outer_nesterov       Eq. (3); Algorithm 1 (outer momentum, outer update)
  quantize_blocks      Section 2 "Compressed Communication" (linear quantisation)
                       in the per-block absmax form of the benchmark configs
  compressed_pseudogradient  Algorithm 2 (compression, error feedback) with the two
                       quantisations of Section 2 "Collectives for compressed communication"
  topk_sparsify        Section 2 "Compressed Communication" (top-k sparsification)
  sparsified_pseudogradient  Algorithm 2 with top-k as the compressor, sparsified once before
                       the all-gather (Appendix, "Assumptions around the collective used")
  fragments_due        Section 2 "Partitioned Communication in Streaming DiLoCo"
  MuLoCoOracle         Algorithm 1 (loop nest and initialisation)

Pins (tests/test_oracle_*.py, all run without a GPU): SVD closed form of the
Newton-Schulz map, exact rational iterates of the scalar quintic, rank-1 Muon
step, K=1 equivalence with plain Muon, identical-gradient pseudogradient,
Proposition 4.2's nuclear-norm identity, AdamW / outer-step closed forms,
quantiser error bound / ties / idempotence, streaming coverage, two-stage
compression (K=1 collapse, error bound, error-feedback conservation), top-k
(brute-force selection, best k-term approximation by enumeration, ties, counts).
Parity unpinned: none of the functions above; the bf16 production mode of the
GPU Newton-Schulz has no pin other than this oracle (tolerance 2e-2).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

# Section 2 "Muon": (a, b, c) of p(x) = a x + b x^3 + c x^5.
NS_COEFFS = (3.4445, -4.7750, 2.0315)


# --------------------------------------------------------------------------
# Newton-Schulz (Section 2, "Muon")
# --------------------------------------------------------------------------
def newton_schulz(U, steps: int = 5, coeffs=NS_COEFFS, eps: float = 1e-7):
    """Quintic Newton-Schulz orthogonalisation of one matrix, in float64.

    X_0 = U / (||U||_F + eps); each step maps X <- a X + b (X X^T) X +
    c (X X^T)^2 X, i.e. every singular value s -> a s + b s^3 + c s^5
    (Section 2 "Muon"; "quintic" in Section 5).  A matrix with more rows than
    columns is iterated on its transpose so the Gram matrix is min x min; the
    map is odd, so the result is the same matrix either way.
    """
    a, b, c = (float(x) for x in coeffs)
    X = np.asarray(U, dtype=np.float64)
    transposed = X.shape[0] > X.shape[1]
    if transposed:
        X = X.T
    X = X / (np.linalg.norm(X) + float(eps))
    for _ in range(steps):
        A = X @ X.T
        B = b * A + c * (A @ A)
        X = a * X + B @ X
    if transposed:
        X = X.T
    return X


# --------------------------------------------------------------------------
# Inner optimizers
# --------------------------------------------------------------------------
def muon_lr_mult(rows: int, cols: int) -> float:
    """Section 5 "MuLoCo": for W in R^{m x n} the learning rate is rescaled by
    sqrt(n / m), m = rows and n = cols of the tensor as stored."""
    return math.sqrt(cols / rows)


def muon_step(W, M, G, *, lr, beta, wd, nesterov=True, lr_mult=None, wd_mult=1.0,
              wd_uses_scaled_lr=True, ns_steps=5, coeffs=NS_COEFFS, eps=1e-7):
    """One Muon step on one hidden matrix; W and M (float32) are updated in place.

    m_t = beta m_{t-1} + g_t (no dampening);  U = g_t + beta m_t with Nesterov,
    else U = m_t;  O_t = NewtonSchulz(U);  W_t = W_{t-1} - eta O_t -
    eta lambda W_{t-1} with eta = lr * sqrt(n/m)  (Section 2 "Muon", Section 5).
    Returns O_t (float64) for diagnostics.
    """
    g = np.asarray(G, dtype=np.float64)
    m_new = float(beta) * M.astype(np.float64) + g
    M[...] = m_new.astype(np.float32)
    # the momentum that later steps see is the stored (float32) one
    m_st = M.astype(np.float64)
    Uin = g + float(beta) * m_st if nesterov else m_st
    O = newton_schulz(Uin, ns_steps, coeffs, eps)
    if lr_mult is None:
        lr_mult = muon_lr_mult(W.shape[0], W.shape[1])
    eta = float(lr) * float(lr_mult)
    eta_wd = eta if wd_uses_scaled_lr else float(lr)
    w = W.astype(np.float64)
    W[...] = (w - eta * O - eta_wd * float(wd) * float(wd_mult) * w).astype(np.float32)
    return O


def adamw_step(theta, m, v, g, *, t, lr, beta1=0.9, beta2=0.99, eps=1e-8, wd=0.0,
               wd_mult=1.0, bias_correction=True):
    """One AdamW step (Section 4.3); theta, m, v (float32) updated in place.

    m = b1 m + (1-b1) g;  v = b2 v + (1-b2) g*g;  theta <- theta -
    alpha ( m^ / (sqrt(v^) + eps) + lambda theta ), with m^ = m/(1-b1^t),
    v^ = v/(1-b2^t) when bias correction is on (t counts from 1).
    """
    g64 = np.asarray(g, dtype=np.float64)
    b1, b2 = float(beta1), float(beta2)
    m[...] = (b1 * m.astype(np.float64) + (1.0 - b1) * g64).astype(np.float32)
    v[...] = (b2 * v.astype(np.float64) + (1.0 - b2) * g64 * g64).astype(np.float32)
    mh = m.astype(np.float64)
    vh = v.astype(np.float64)
    if bias_correction:
        mh = mh / (1.0 - b1 ** t)
        vh = vh / (1.0 - b2 ** t)
    th = theta.astype(np.float64)
    step = mh / (np.sqrt(vh) + float(eps)) + float(wd) * float(wd_mult) * th
    theta[...] = (th - float(lr) * step).astype(np.float32)


# --------------------------------------------------------------------------
# Outer synchronisation
# --------------------------------------------------------------------------
def pseudogradient(theta_g, thetas: Sequence[np.ndarray]):
    """Eq. (2): Psi = (1/K) sum_k (theta_global - theta_k), in float64."""
    tg = theta_g.astype(np.float64)
    acc = np.zeros_like(tg)
    for th in thetas:
        acc += tg - th.astype(np.float64)
    return acc / len(thetas)


def pseudogradient_f32(theta_g, thetas: Sequence[np.ndarray]):
    """Eq. (2) in float32, workers in ascending order, then one multiply by
    float32(1/K).  This is the precision in which the quantiser takes its
    integer decisions, so both sides of a code comparison use it."""
    tg = theta_g.astype(np.float32)
    acc = np.zeros_like(tg)
    for th in thetas:
        acc = (acc + (tg - th.astype(np.float32))).astype(np.float32)
    return (acc * np.float32(1.0 / len(thetas))).astype(np.float32)


def quantize_blocks(psi, bits: int, block: int = 128):
    """Linear symmetric quantisation with one absmax scale per block.

    psi is a float32 matrix (a vector counts as one row).  Blocks are `block`
    consecutive elements of one row; the last block of a row may be short and
    no block spans two rows.  With qmax = 2^(bits-1) - 1, in float32:
        amax = max |x_i|;  inv = qmax / amax;  q_i = rint(x_i * inv)  (ties to
        even), clamped to [-qmax, qmax];  scale = amax / qmax;  x^_i = q_i * scale.
    An all-zero block gives codes 0 and scale 0.
    Returns (codes int8 [rows, cols], scales float32 [rows, nblk], dequant float32).
    """
    x = np.asarray(psi, dtype=np.float32)
    if x.ndim == 1:
        x = x.reshape(1, -1)
    rows, cols = x.shape
    nblk = (cols + block - 1) // block
    qmax = np.float32((1 << (bits - 1)) - 1)
    codes = np.zeros((rows, cols), dtype=np.int8)
    scales = np.zeros((rows, nblk), dtype=np.float32)
    deq = np.zeros((rows, cols), dtype=np.float32)
    for j in range(nblk):
        lo, hi = j * block, min(cols, (j + 1) * block)
        xb = x[:, lo:hi]
        amax = np.max(np.abs(xb), axis=1).astype(np.float32)          # [rows]
        nz = amax > 0
        inv = np.zeros_like(amax)
        sc = np.zeros_like(amax)
        with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
            inv[nz] = qmax / amax[nz]
            sc[nz] = amax[nz] / qmax
            q = np.rint((xb * inv[:, None]).astype(np.float32))
        q = np.clip(q, -qmax, qmax)
        q[~nz, :] = 0
        codes[:, lo:hi] = q.astype(np.int8)
        scales[:, j] = sc
        deq[:, lo:hi] = (q.astype(np.float32) * sc[:, None]).astype(np.float32)
    return codes, scales, deq


def compressed_pseudogradient(theta_g, thetas: Sequence[np.ndarray], bits: int, block: int = 128,
                              ef: Optional[Sequence[np.ndarray]] = None, ef_beta: float = 1.0):
    """Algorithm 2 with the two quantisations of Section 2 "Collectives for compressed
    communication" (Appendix, "Assumptions around the collective used"), in float32:

      per worker i:  Delta_i = theta - theta_i                       (parameter delta)
                     with EF:  E_i <- beta E_i + Delta_i;  Delta~_i = C(E_i);  E_i <- E_i - Delta~_i
                     else:     Delta~_i = C(Delta_i)                  (first quantisation, before
                                                                       the all-to-all reduce-scatter)
      Delta = (1/K) sum_i Delta~_i                                    (reduced in high precision)
      Psi   = C(Delta)                                                (second quantisation, before
                                                                       the all-gather)

    C is quantize_blocks followed by dequantisation.  Every operation is a single float32
    operation (no fused multiply-add), workers in ascending order, so that the integer
    codes of both quantisations are reproducible bit for bit.  `ef` (float32 arrays, one
    per worker) is updated in place.  Returns Psi (float32).
    """
    tg = np.asarray(theta_g, dtype=np.float32)
    K = len(thetas)
    acc = np.zeros_like(tg)
    beta = np.float32(ef_beta)
    for i, th in enumerate(thetas):
        delta = (tg - np.asarray(th, dtype=np.float32)).astype(np.float32)
        if ef is not None:
            e = ((beta * ef[i]).astype(np.float32) + delta).astype(np.float32)
            _, _, c = quantize_blocks(e, bits, block)
            ef[i][...] = (e - c.reshape(e.shape)).astype(np.float32)
        else:
            _, _, c = quantize_blocks(delta, bits, block)
        acc = (acc + c.reshape(tg.shape)).astype(np.float32)
    mean = (acc * np.float32(1.0 / K)).astype(np.float32)
    _, _, psi = quantize_blocks(mean, bits, block)
    return psi.reshape(tg.shape)


def topk_count(n: int, fraction: float) -> int:
    """How many entries of a tensor of n elements top-k keeps: floor(fraction * n), in double
    precision with `fraction` first rounded to float32 (how it crosses the library boundary),
    at least 1 and at most n."""
    return int(min(n, max(1, math.floor(float(np.float32(fraction)) * n))))


def topk_sparsify(x, fraction: float):
    """Top-k sparsification of one weight matrix (Section 2, "Compressed Communication"): the
    k% entries of largest magnitude are kept, every other entry becomes 0.

    The selection is over the whole tensor.  With kk = topk_count(n, fraction) and tau the
    kk-th largest magnitude, the entries with |x| >= tau are kept: entries tied with the
    kk-th one are all kept, so the result does not depend on an order among equals.
    Returns a float32 array of x's shape."""
    a = np.asarray(x, dtype=np.float32)
    flat = np.abs(a).reshape(-1)
    n = flat.size
    if n == 0:
        return a.copy()
    kk = topk_count(n, fraction)
    tau = np.sort(flat)[n - kk]
    return np.where(np.abs(a) >= tau, a, np.float32(0)).astype(np.float32)


def sparsified_pseudogradient(theta_g, thetas: Sequence[np.ndarray], fraction: float,
                              ef: Optional[Sequence[np.ndarray]] = None, ef_beta: float = 1.0):
    """Algorithm 2 with top-k as the compressor; the sparsified deltas are gathered from all
    workers, so each is sparsified once and nothing is compressed after the mean (Appendix,
    "Assumptions around the collective used").  In float32, workers in ascending order:

      per worker i:  Delta_i = theta - theta_i
                     with EF:  E_i <- beta E_i + Delta_i;  Delta~_i = topk(E_i);  E_i <- E_i - Delta~_i
                     else:     Delta~_i = topk(Delta_i)
      Psi = (1/K) sum_i Delta~_i

    `ef` (float32 arrays, one per worker) is updated in place.  Returns Psi (float32)."""
    tg = np.asarray(theta_g, dtype=np.float32)
    K = len(thetas)
    acc = np.zeros_like(tg)
    beta = np.float32(ef_beta)
    for i, th in enumerate(thetas):
        delta = (tg - np.asarray(th, dtype=np.float32)).astype(np.float32)
        if ef is not None:
            e = ((beta * ef[i]).astype(np.float32) + delta).astype(np.float32)
            c = topk_sparsify(e, fraction)
            ef[i][...] = (e - c).astype(np.float32)
        else:
            c = topk_sparsify(delta, fraction)
        acc = (acc + c).astype(np.float32)
    return (acc * np.float32(1.0 / K)).astype(np.float32)


def pack_int4(codes):
    """Two 4-bit two's-complement codes per byte along a row, element 2j in the
    low nibble; a row with an odd number of elements pads the last high nibble
    with 0."""
    c = np.asarray(codes, dtype=np.int8)
    if c.ndim == 1:
        c = c.reshape(1, -1)
    rows, cols = c.shape
    padded = np.zeros((rows, (cols + 1) // 2 * 2), dtype=np.int8)
    padded[:, :cols] = c
    lo = padded[:, 0::2].astype(np.uint8) & 0xF
    hi = padded[:, 1::2].astype(np.uint8) & 0xF
    return (lo | (hi << 4)).astype(np.uint8)


def outer_nesterov(theta_g, u, psi, *, outer_lr, outer_momentum):
    """Eq. (3): u <- mu u + eta_out Psi;  theta <- theta - mu u - eta_out Psi
    (the new u on the right-hand side).  theta_g and u (float32) in place."""
    mu, eta = float(outer_momentum), float(outer_lr)
    p = np.asarray(psi, dtype=np.float64)
    u_new = mu * u.astype(np.float64) + eta * p
    u[...] = u_new.astype(np.float32)
    theta_g[...] = (theta_g.astype(np.float64) - mu * u_new - eta * p).astype(np.float32)


def fragments_due(t: int, H: int, J: int) -> List[int]:
    """Streaming schedule (Section 2, "Partitioned Communication"): with J | H,
    subset j (1-based) is communicated at the multiples j*H/J of the interval;
    returns the 0-based fragment indices due after inner step t (t >= 1)."""
    if J <= 0 or H <= 0 or H % J != 0:
        raise ValueError("J must divide H")
    if t <= 0:
        return []
    return [j - 1 for j in range(1, J + 1) if t % H == (j * H // J) % H]


# --------------------------------------------------------------------------
# Algorithm 1
# --------------------------------------------------------------------------
@dataclass
class TensorSpec:
    name: str
    rows: int
    cols: int
    kind: str = "muon"          # "muon" | "adamw"
    fragment: int = 0
    wd_mult: float = 1.0
    lr_mult: Optional[float] = None   # None: sqrt(cols/rows) for muon, 1 for adamw


@dataclass
class OracleConfig:
    K: int
    H: int
    J: int = 1
    muon_lr: float = 0.02
    muon_beta: float = 0.9
    muon_wd: float = 0.0
    muon_nesterov: bool = True
    ns_steps: int = 5
    ns_coeffs: tuple = NS_COEFFS
    ns_eps: float = 1e-7
    wd_uses_scaled_lr: bool = True
    adam_lr: float = 1e-3
    adam_beta1: float = 0.9
    adam_beta2: float = 0.99
    adam_eps: float = 1e-8
    adam_wd: float = 0.0
    adam_bias_correction: bool = True
    outer_lr: float = 1.0
    outer_momentum: float = 0.0
    quant_bits: int = 0           # 0 = none, 8, 4, 2
    quant_block: int = 128        # 0 = one block per row (row-wise quantisation)
    quant_stages: int = 1         # 1: quantise the averaged pseudogradient once (benchmark form);
                                  # 2: per-worker quantisation, high-precision mean, second quantisation
    error_feedback: bool = False  # Algorithm 2 (needs quant_stages = 2 or topk_fraction > 0)
    ef_beta: float = 1.0
    topk_fraction: float = 0.0    # > 0: top-k sparsification of every worker's delta (no quantiser)

    def f32(self) -> "OracleConfig":
        """The same configuration with every real hyper-parameter rounded to
        float32, which is how it crosses the library boundary."""
        r = lambda x: float(np.float32(x))
        d = dict(self.__dict__)
        for k in ("muon_lr", "muon_beta", "muon_wd", "ns_eps", "adam_lr", "adam_beta1",
                  "adam_beta2", "adam_eps", "adam_wd", "outer_lr", "outer_momentum", "ef_beta", "topk_fraction"):
            d[k] = r(d[k])
        d["ns_coeffs"] = tuple(r(x) for x in self.ns_coeffs)
        return OracleConfig(**d)


class MuLoCoOracle:
    """Algorithm 1 with the gradients supplied by the caller.

    State (all float32): theta_k[k][i] replicas, theta_g[i], outer_u[i],
    state1[k][i] (Muon momentum or Adam m), state2[k][i] (Adam v or None).
    """

    def __init__(self, cfg: OracleConfig, specs: Sequence[TensorSpec],
                 init: Sequence[np.ndarray]):
        if cfg.K < 1 or cfg.H < 1 or cfg.J < 1 or cfg.H % cfg.J != 0:
            raise ValueError("need K,H,J >= 1 and J | H")
        self.cfg = cfg
        self.specs = list(specs)
        self.theta_g = [np.array(w, dtype=np.float32).reshape(s.rows, s.cols)
                        for w, s in zip(init, self.specs)]
        # Algorithm 1, initialisation: u <- 0, theta_i <- theta for all i
        self.outer_u = [np.zeros_like(w) for w in self.theta_g]
        self.theta_k = [[w.copy() for w in self.theta_g] for _ in range(cfg.K)]
        self.state1 = [[np.zeros_like(w) for w in self.theta_g] for _ in range(cfg.K)]
        self.state2 = [[np.zeros_like(w) if s.kind == "adamw" else None
                        for w, s in zip(self.theta_g, self.specs)] for _ in range(cfg.K)]
        if cfg.topk_fraction and cfg.quant_bits:
            raise ValueError("top-k sparsification and quantisation are not combined")
        if not 0.0 <= cfg.topk_fraction <= 1.0:
            raise ValueError("topk_fraction must lie in [0, 1]")
        if cfg.error_feedback and not cfg.topk_fraction and (cfg.quant_stages != 2 or not cfg.quant_bits):
            raise ValueError("error feedback needs the two-stage quantised sync or top-k")
        # Algorithm 2, initialisation: E_i <- 0
        self.ef = [[np.zeros_like(w) for w in self.theta_g] for _ in range(cfg.K)] if cfg.error_feedback else None
        self.worker_step = [0] * cfg.K
        self.last_psi: Dict[int, np.ndarray] = {}

    # Algorithm 1, inner loop body (Eq. 1) for one worker, gradients given
    def inner_step(self, worker: int, grads: Sequence[np.ndarray], lr_scale: float = 1.0):
        c = self.cfg
        self.worker_step[worker] += 1
        t = self.worker_step[worker]
        for i, s in enumerate(self.specs):
            if s.kind == "muon":
                muon_step(self.theta_k[worker][i], self.state1[worker][i], grads[i],
                          lr=c.muon_lr * lr_scale, beta=c.muon_beta, wd=c.muon_wd,
                          nesterov=c.muon_nesterov, lr_mult=s.lr_mult, wd_mult=s.wd_mult,
                          wd_uses_scaled_lr=c.wd_uses_scaled_lr, ns_steps=c.ns_steps,
                          coeffs=c.ns_coeffs, eps=c.ns_eps)
            else:
                lm = 1.0 if s.lr_mult is None else s.lr_mult
                adamw_step(self.theta_k[worker][i], self.state1[worker][i],
                           self.state2[worker][i], grads[i], t=t,
                           lr=c.adam_lr * lr_scale * lm, beta1=c.adam_beta1,
                           beta2=c.adam_beta2, eps=c.adam_eps, wd=c.adam_wd,
                           wd_mult=s.wd_mult, bias_correction=c.adam_bias_correction)

    def inner_step_all(self, grads_k: Sequence[Sequence[np.ndarray]], lr_scale: float = 1.0):
        for k in range(self.cfg.K):
            self.inner_step(k, grads_k[k], lr_scale)

    # Algorithm 1, outer step (Eqs. 2-3) for the tensors of one fragment (-1: all), then
    # the replicas of those tensors restart from the new global parameters.
    def outer_sync(self, fragment: int = -1):
        c = self.cfg
        for i, s in enumerate(self.specs):
            if fragment >= 0 and s.fragment != fragment:
                continue
            reps = [self.theta_k[k][i] for k in range(c.K)]
            blk = c.quant_block if c.quant_block > 0 else s.cols
            if c.topk_fraction:
                efs = [self.ef[k][i] for k in range(c.K)] if self.ef is not None else None
                psi = sparsified_pseudogradient(self.theta_g[i], reps, c.topk_fraction, efs, c.ef_beta)
            elif c.quant_bits and c.quant_stages == 2:
                efs = [self.ef[k][i] for k in range(c.K)] if self.ef is not None else None
                psi = compressed_pseudogradient(self.theta_g[i], reps, c.quant_bits, blk, efs, c.ef_beta)
            elif c.quant_bits:
                psi32 = pseudogradient_f32(self.theta_g[i], reps)
                _, _, psi = quantize_blocks(psi32, c.quant_bits, blk)
            else:
                psi = pseudogradient(self.theta_g[i], reps)
            self.last_psi[i] = np.array(psi)
            outer_nesterov(self.theta_g[i], self.outer_u[i], psi,
                           outer_lr=c.outer_lr, outer_momentum=c.outer_momentum)
            for k in range(c.K):
                self.theta_k[k][i][...] = self.theta_g[i]
