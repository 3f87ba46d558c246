"""ctypes binding of libmuloco (argument marshalling only).

Every optimizer step runs inside the CUDA library; this module only loads the
shared object, mirrors the C structs of include/muloco.h and turns torch
tensors into raw device pointers.  torch is used for device memory and streams.
There is no fallback: if the library cannot be loaded, or there is no CUDA
device, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import List, Optional, Sequence

import numpy as np

from . import configs as _cfg

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MULOCO_LIBRARY", os.path.join(_HERE, "libmuloco.so"))

OK, EINVAL, ESHAPE, ENOMEM, ECUDA, ENONFINITE, ETIMEOUT, ESTATE = range(8)
STATUS_NAMES = ["OK", "EINVAL", "ESHAPE", "ENOMEM", "ECUDA", "ENONFINITE", "ETIMEOUT", "ESTATE"]
MUON, ADAMW = 0, 1
NS_BF16, NS_FP32 = 0, 1
F32, BF16 = 0, 1
DEBUG_WAIT_LIMIT_NS, DEBUG_WITHHOLD_COPY, DEBUG_CANARIES, DEBUG_CORRUPT_CANARY = 1, 2, 3, 4
PHASES = ["prologue", "ns", "adamw", "sync", "copy"]

EXPORTS = [
    "muloco_create", "muloco_destroy", "muloco_inner_step", "muloco_inner_step_host",
    "muloco_outer_sync", "muloco_outer_sync_host", "muloco_fragments_due", "muloco_newton_schulz",
    "muloco_quantize", "muloco_topk_sparsify", "muloco_pseudogradient", "muloco_get_state", "muloco_set_state",
    "muloco_set_timing", "muloco_get_timings", "muloco_sync_status", "muloco_last_error",
    "muloco_newton_schulz_static", "muloco_debug_set", "muloco_check_workspace",
    "muloco_shard_layout", "muloco_shard_delta", "muloco_shard_step", "muloco_shard_broadcast",
]


class TensorDesc(C.Structure):
    _fields_ = [("rows", C.c_int64), ("cols", C.c_int64), ("kind", C.c_int32), ("fragment", C.c_int32),
                ("wd_mult", C.c_float), ("lr_mult", C.c_float)]


class Config(C.Structure):
    _fields_ = [("K", C.c_int32), ("H", C.c_int32), ("J", C.c_int32),
                ("muon_lr", C.c_float), ("muon_beta", C.c_float), ("muon_wd", C.c_float),
                ("muon_nesterov", C.c_int32), ("ns_steps", C.c_int32),
                ("ns_a", C.c_float), ("ns_b", C.c_float), ("ns_c", C.c_float), ("ns_eps", C.c_float),
                ("ns_mode", C.c_int32), ("wd_uses_scaled_lr", C.c_int32),
                ("adam_lr", C.c_float), ("adam_beta1", C.c_float), ("adam_beta2", C.c_float),
                ("adam_eps", C.c_float), ("adam_wd", C.c_float), ("adam_bias_correction", C.c_int32),
                ("outer_lr", C.c_float), ("outer_momentum", C.c_float),
                ("quant", C.c_int32), ("quant_block", C.c_int32), ("grad_dtype", C.c_int32),
                ("quant_stages", C.c_int32), ("workspace_bytes", C.c_uint64),
                ("error_feedback", C.c_int32), ("ef_beta", C.c_float),
                ("topk_fraction", C.c_float)]


class Buffers(C.Structure):
    _fields_ = [("theta_k", C.POINTER(C.c_void_p)), ("theta_g", C.POINTER(C.c_void_p)),
                ("outer_u", C.POINTER(C.c_void_p)), ("state1_k", C.POINTER(C.c_void_p)),
                ("state2_k", C.POINTER(C.c_void_p)), ("ef_k", C.POINTER(C.c_void_p))]


class MulocoError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"muloco status {STATUS_NAMES[status] if 0 <= status < 8 else status}: {msg}")
        self.status = status


_lib = None


def load_library():
    """Load libmuloco.so from the package directory; raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_23725_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.muloco_create.argtypes = [C.POINTER(Config), C.POINTER(TensorDesc), i32, C.POINTER(Buffers), vp,
                                  C.POINTER(vp)]
    lib.muloco_destroy.argtypes = [vp]
    lib.muloco_destroy.restype = None
    lib.muloco_inner_step.argtypes = [vp, i32, C.POINTER(vp), f32]
    lib.muloco_inner_step_host.argtypes = [vp, i32, C.POINTER(vp), f32]
    lib.muloco_outer_sync.argtypes = [vp, i32]
    lib.muloco_outer_sync_host.argtypes = [vp, i32, C.POINTER(vp)]
    lib.muloco_fragments_due.argtypes = [vp, i64, C.POINTER(i32)]
    lib.muloco_newton_schulz.argtypes = [vp, vp, i32, vp, i32, i32, i64, i64, i32]
    lib.muloco_quantize.argtypes = [vp, vp, i64, i64, i32, vp, vp, vp]
    lib.muloco_pseudogradient.argtypes = [vp, i32, vp]
    lib.muloco_topk_sparsify.argtypes = [vp, vp, i64, C.c_float, vp]
    lib.muloco_get_state.argtypes = [vp, vp, C.POINTER(C.c_size_t)]
    lib.muloco_set_state.argtypes = [vp, vp, C.c_size_t]
    lib.muloco_set_timing.argtypes = [vp, i32]
    lib.muloco_get_timings.argtypes = [vp, C.POINTER(f32), C.POINTER(i64)]
    lib.muloco_sync_status.argtypes = [vp]
    lib.muloco_last_error.argtypes = [vp]
    lib.muloco_last_error.restype = C.c_char_p
    lib.muloco_debug_set.argtypes = [vp, i32, i64]
    lib.muloco_check_workspace.argtypes = [vp]
    lib.muloco_shard_layout.argtypes = [vp, i32, i32, i32, C.POINTER(i64), C.POINTER(i64)]
    lib.muloco_shard_delta.argtypes = [vp, i32, i32, vp]
    lib.muloco_shard_step.argtypes = [vp, i32, i32, i32, vp, vp]
    lib.muloco_shard_broadcast.argtypes = [vp, i32, i32, vp]
    lib.muloco_newton_schulz_static.argtypes = [vp, vp, i32, i64, i64, vp, C.c_char_p, C.c_size_t]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("muloco_destroy", "muloco_last_error"):
            fn.restype = i32
    _lib = lib
    return lib


def newton_schulz_static(X, stream=None, out=None):
    """muloco_newton_schulz_static: fp32 Newton-Schulz of a small [batch, rows, cols]
    (or [rows, cols]) float32 CUDA tensor without any device allocation by the library.
    The result goes to `out` (same shape, float32, contiguous) when given; otherwise the
    output tensor is allocated here, by torch, before the call.  For callers that may
    not allocate; sizes beyond the library's fixed scratch raise MulocoError(ESHAPE)."""
    import torch
    lib = load_library()
    x = (X if X.dim() == 3 else X.unsqueeze(0)).contiguous()
    if x.dtype != torch.float32 or not x.is_cuda:
        raise ValueError("expects a float32 CUDA tensor")
    if out is None:
        o = torch.empty_like(x)
    else:
        o = out if out.dim() == 3 else out.unsqueeze(0)
        if o.shape != x.shape or o.dtype != torch.float32 or not o.is_contiguous() or o.device != x.device:
            raise ValueError("out must be a contiguous float32 tensor of X's shape on X's device")
    st = stream if stream is not None else torch.cuda.current_stream(x.device)
    err = C.create_string_buffer(256)
    with torch.cuda.device(x.device):
        rc = lib.muloco_newton_schulz_static(x.data_ptr(), o.data_ptr(), x.shape[0], x.shape[1], x.shape[2],
                                             C.c_void_p(st.cuda_stream), err, 256)
    if rc != OK:
        raise MulocoError(rc, err.value.decode())
    return o if X.dim() == 3 else o[0]


def shard_wire_bytes(stage_floats: int, world: int) -> int:
    """Bytes one rank moves per sharded sync: a reduce-scatter and an all-gather of stage_floats
    float32 values, (world - 1) / world of it each."""
    return 2 * 4 * stage_floats * (world - 1) // world


def _reduce_scatter_sum(dist, out, inp, group):
    """out <- this rank's shard of the element-wise sum of inp over the ranks."""
    if dist.get_backend(group) == "nccl":
        dist.reduce_scatter_tensor(out, inp, op=dist.ReduceOp.SUM, group=group)
    else:                                   # backends without reduce-scatter (gloo): all-reduce, keep the shard
        tmp = inp.clone()
        dist.all_reduce(tmp, op=dist.ReduceOp.SUM, group=group)
        r = dist.get_rank(group)
        out.copy_(tmp[r * out.numel():(r + 1) * out.numel()])


def sharded_outer_sync(opt, fragment: int, dist, group=None):
    """Drives the three shard calls of `opt` (a MuLoCo, or any object with shard_layout /
    shard_delta / shard_step / shard_broadcast and new_buffer) around the two collectives."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    stage_floats, shard_floats = opt.shard_layout(fragment, world, rank)
    if stage_floats == 0:
        return 0
    with opt.stream_context():
        stage = opt.new_buffer(stage_floats)
        reduced = opt.new_buffer(shard_floats)
        theta_shard = opt.new_buffer(shard_floats)
        opt.shard_delta(fragment, world, stage)
        if world > 1:
            _reduce_scatter_sum(dist, reduced, stage, group)
        else:
            reduced = stage
        opt.shard_step(fragment, world, rank, reduced, theta_shard)
        if world > 1:
            dist.all_gather_into_tensor(stage, theta_shard, group=group)
        else:
            stage = theta_shard
        opt.shard_broadcast(fragment, world, stage)
    return shard_wire_bytes(stage_floats, world)


def make_config(w: _cfg.Workload, workspace_bytes: int = 0, ns_mode: Optional[str] = None, **over) -> Config:
    c = Config()
    c.K, c.H, c.J = w.K, w.H, w.J
    c.muon_lr, c.muon_beta, c.muon_wd = w.muon_lr, w.muon_beta, w.muon_wd
    c.muon_nesterov = int(w.muon_nesterov)
    c.ns_steps = 5
    c.ns_a, c.ns_b, c.ns_c = 3.4445, -4.7750, 2.0315
    c.ns_eps = 1e-7
    mode = ns_mode or w.ns_mode
    c.ns_mode = NS_FP32 if mode == "fp32" else NS_BF16
    c.wd_uses_scaled_lr = 1
    c.adam_lr = w.muon_lr if w.adam_lr is None else w.adam_lr
    c.adam_wd = w.muon_wd if w.adam_wd is None else w.adam_wd
    c.adam_beta1, c.adam_beta2, c.adam_eps = w.adam_beta1, w.adam_beta2, w.adam_eps
    c.adam_bias_correction = 1
    c.outer_lr, c.outer_momentum = w.outer_lr, w.outer_momentum
    c.quant = w.quant_bits
    c.quant_block = w.quant_block
    c.quant_stages = w.quant_stages
    c.error_feedback = int(w.error_feedback)
    c.ef_beta = w.ef_beta
    c.topk_fraction = w.topk_fraction
    c.grad_dtype = BF16 if w.grad_dtype == "bf16" else F32
    c.workspace_bytes = workspace_bytes
    for k, v in over.items():
        setattr(c, k, v)
    return c


def _ptr_table(ptrs: Sequence[int]):
    arr = (C.c_void_p * max(1, len(ptrs)))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


class MuLoCo:
    """Owns the device state of one MuLoCo problem and forwards to the C ABI.

    State lives in flat torch buffers (one per replica / state kind) so that the
    tensors of a replica are contiguous; each tensor starts on a 256-byte
    boundary.  `self.theta_g[i]`, `self.theta_k[k][i]` ... are torch views.
    """

    ALIGN = 64  # elements

    def __init__(self, workload: _cfg.Workload, device="cuda:0", init: Optional[Sequence[np.ndarray]] = None,
                 workspace_bytes: int = 0, ns_mode: Optional[str] = None, stream=None, alloc_grads: bool = False,
                 init_seed: Optional[int] = None, **config_overrides):
        import torch

        self.torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: libmuloco has no CPU path")
        self.w = workload
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.K, self.n = workload.K, len(workload.tensors)
        self.cfg = make_config(workload, workspace_bytes, ns_mode, **config_overrides)
        self.offsets = []
        off = 0
        for t in workload.tensors:
            self.offsets.append(off)
            off += (t.numel + self.ALIGN - 1) // self.ALIGN * self.ALIGN
        self.flat_numel = off
        f32 = torch.float32
        dev = self.device
        self.flat_theta_g = torch.zeros(off, dtype=f32, device=dev)
        self.flat_u = torch.zeros(off, dtype=f32, device=dev)
        self.flat_theta_k = [torch.empty(off, dtype=f32, device=dev) for _ in range(self.K)]
        self.flat_s1 = [torch.empty(off, dtype=f32, device=dev) for _ in range(self.K)]
        # Adam's second moment exists for AdamW tensors only: its own compact buffer
        self.offsets2, off2 = [], 0
        for t in workload.tensors:
            self.offsets2.append(off2 if t.kind == _cfg.ADAMW else None)
            if t.kind == _cfg.ADAMW:
                off2 += (t.numel + self.ALIGN - 1) // self.ALIGN * self.ALIGN
        self.flat_s2 = [torch.empty(off2, dtype=f32, device=dev) if off2 else None for _ in range(self.K)]
        self.flat_ef = [torch.empty(off, dtype=f32, device=dev) for _ in range(self.K)] \
            if workload.error_feedback else None
        self.ef = [self._views(b) for b in self.flat_ef] if self.flat_ef else None
        self.theta_g = self._views(self.flat_theta_g)
        self.outer_u = self._views(self.flat_u)
        self.theta_k = [self._views(b) for b in self.flat_theta_k]
        self.state1 = [self._views(b) for b in self.flat_s1]
        self.state2 = [[b[o:o + t.numel].view(t.rows, t.cols) if (b is not None and o is not None) else None
                        for o, t in zip(self.offsets2, workload.tensors)] for b in self.flat_s2]
        if init is not None:
            for i, a in enumerate(init):
                self.theta_g[i].copy_(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev))
        elif init_seed is not None:
            # device-side initial weights for the large configurations: N(0, 0.02^2), gains = 1
            gen = torch.Generator(device=dev)
            gen.manual_seed(init_seed)
            self.flat_theta_g.normal_(0.0, 0.02, generator=gen)
            for i, t in enumerate(workload.tensors):
                if t.init == "ones":
                    self.theta_g[i].fill_(1.0)
        self.gdtype = torch.bfloat16 if workload.grad_dtype == "bf16" else torch.float32
        self.flat_grads = None
        self.grads = None
        self._grad_table_all = None
        if alloc_grads:
            self.alloc_grads()

        descs = (TensorDesc * max(1, self.n))()
        for i, t in enumerate(workload.tensors):
            descs[i].rows, descs[i].cols = t.rows, t.cols
            descs[i].kind = MUON if t.kind == _cfg.MUON else ADAMW
            descs[i].fragment = t.fragment
            descs[i].wd_mult = t.wd_mult
            descs[i].lr_mult = float("nan") if t.lr_mult is None else t.lr_mult
        bufs = Buffers()
        self._tables = [
            _ptr_table([self.theta_k[k][i].data_ptr() for k in range(self.K) for i in range(self.n)]),
            _ptr_table([v.data_ptr() for v in self.theta_g]),
            _ptr_table([v.data_ptr() for v in self.outer_u]),
            _ptr_table([self.state1[k][i].data_ptr() for k in range(self.K) for i in range(self.n)]),
            _ptr_table([(self.state2[k][i].data_ptr() if self.state2[k][i] is not None else 0)
                        for k in range(self.K) for i in range(self.n)]),
        ]
        bufs.theta_k, bufs.theta_g, bufs.outer_u, bufs.state1_k, bufs.state2_k = [
            C.cast(t, C.POINTER(C.c_void_p)) for t in self._tables]
        if self.ef is not None:
            self._tables.append(_ptr_table([self.ef[k][i].data_ptr() for k in range(self.K) for i in range(self.n)]))
            bufs.ef_k = C.cast(self._tables[-1], C.POINTER(C.c_void_p))
        self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self.ctx = C.c_void_p()
        st = self.lib.muloco_create(C.byref(self.cfg), descs, self.n, C.byref(bufs),
                                    C.c_void_p(self.stream.cuda_stream), C.byref(self.ctx))
        if st != OK:
            msg = self.lib.muloco_last_error(None).decode()
            self.ctx = None
            raise MulocoError(st, msg)

    # -- helpers --------------------------------------------------------------
    def _views(self, flat):
        return [flat[o:o + t.numel].view(t.rows, t.cols) for o, t in zip(self.offsets, self.w.tensors)]

    def alloc_grads(self):
        torch = self.torch
        self.flat_grads = [torch.zeros(self.flat_numel, dtype=self.gdtype, device=self.device)
                           for _ in range(self.K)]
        self.grads = [self._views(b) for b in self.flat_grads]
        self._grad_table_all = _ptr_table([self.grads[k][i].data_ptr() for k in range(self.K)
                                           for i in range(self.n)])

    def new_buffer(self, n: int):
        return self.torch.empty(n, dtype=self.torch.float32, device=self.device)

    def stream_context(self):
        return self.torch.cuda.stream(self.stream)

    def _check(self, st):
        if st != OK:
            raise MulocoError(st, self.lib.muloco_last_error(self.ctx).decode())

    def close(self):
        if getattr(self, "ctx", None):
            self.lib.muloco_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, one method per entry point ----------------------------------
    def inner_step(self, worker: int = -1, grads=None, lr_scale: float = 1.0):
        """muloco_inner_step.  grads: list (one worker) or list of lists (all) of torch
        tensors; None uses the buffers of alloc_grads()."""
        if grads is None:
            if worker < 0:
                table = self._grad_table_all
            else:
                table = _ptr_table([self.grads[worker][i].data_ptr() for i in range(self.n)])
        elif worker < 0:
            table = _ptr_table([grads[k][i].data_ptr() for k in range(self.K) for i in range(self.n)])
        else:
            table = _ptr_table([g.data_ptr() for g in grads])
        self._check(self.lib.muloco_inner_step(self.ctx, worker, C.cast(table, C.POINTER(C.c_void_p)), lr_scale))

    def inner_step_host(self, worker: int, host_grads, lr_scale: float = 1.0):
        """muloco_inner_step_host.  host_grads: like grads, but CPU (pinned) tensors."""
        if worker < 0:
            table = _ptr_table([host_grads[k][i].data_ptr() for k in range(self.K) for i in range(self.n)])
        else:
            table = _ptr_table([g.data_ptr() for g in host_grads])
        self._check(self.lib.muloco_inner_step_host(self.ctx, worker, C.cast(table, C.POINTER(C.c_void_p)),
                                                    lr_scale))

    def outer_sync(self, fragment: int = -1):
        self._check(self.lib.muloco_outer_sync(self.ctx, fragment))

    def outer_sync_host(self, fragment: int, host_theta_g):
        table = _ptr_table([(t.data_ptr() if t is not None else 0) for t in host_theta_g])
        self._check(self.lib.muloco_outer_sync_host(self.ctx, fragment, C.cast(table, C.POINTER(C.c_void_p))))

    def fragments_due(self, step: int) -> List[int]:
        out = (C.c_int32 * max(1, self.cfg.J))()
        n = self.lib.muloco_fragments_due(self.ctx, step, out)
        if n < 0:
            raise MulocoError(EINVAL, "muloco_fragments_due")
        return [out[i] for i in range(n)]

    def newton_schulz(self, X, out_dtype=None, ns_mode: str = "bf16"):
        """muloco_newton_schulz on a [batch, rows, cols] (or [rows, cols]) CUDA tensor."""
        torch = self.torch
        x = X if X.dim() == 3 else X.unsqueeze(0)
        x = x.contiguous()
        out_dtype = out_dtype or torch.float32
        o = torch.empty(x.shape, dtype=out_dtype, device=x.device)
        dt = {torch.float32: F32, torch.bfloat16: BF16}
        self._check(self.lib.muloco_newton_schulz(self.ctx, x.data_ptr(), dt[x.dtype], o.data_ptr(), dt[out_dtype],
                                                  x.shape[0], x.shape[1], x.shape[2],
                                                  NS_FP32 if ns_mode == "fp32" else NS_BF16))
        return o if X.dim() == 3 else o[0]

    def quantize(self, psi, bits: int):
        torch = self.torch
        p = psi.contiguous().view(-1, psi.shape[-1]) if psi.dim() > 1 else psi.contiguous().view(1, -1)
        rows, cols = p.shape
        blk = self.cfg.quant_block
        codes = torch.empty((rows, cols), dtype=torch.int8, device=p.device)
        scales = torch.empty((rows, (cols + blk - 1) // blk), dtype=torch.float32, device=p.device)
        deq = torch.empty((rows, cols), dtype=torch.float32, device=p.device)
        self._check(self.lib.muloco_quantize(self.ctx, p.data_ptr(), rows, cols, bits, codes.data_ptr(),
                                             scales.data_ptr(), deq.data_ptr()))
        return codes, scales, deq

    def topk_sparsify(self, x, fraction: float):
        torch = self.torch
        xc = x.contiguous()
        out = torch.empty_like(xc)
        self._check(self.lib.muloco_topk_sparsify(self.ctx, xc.data_ptr(), xc.numel(), fraction, out.data_ptr()))
        return out

    def pseudogradient(self, tensor: int):
        torch = self.torch
        t = self.w.tensors[tensor]
        out = torch.empty((t.rows, t.cols), dtype=torch.float32, device=self.device)
        self._check(self.lib.muloco_pseudogradient(self.ctx, tensor, out.data_ptr()))
        return out

    def get_state(self) -> bytes:
        n = C.c_size_t(0)
        self._check(self.lib.muloco_get_state(self.ctx, None, C.byref(n)))
        buf = C.create_string_buffer(n.value)
        self._check(self.lib.muloco_get_state(self.ctx, buf, C.byref(n)))
        return buf.raw[:n.value]

    def set_state(self, blob: bytes):
        self._check(self.lib.muloco_set_state(self.ctx, blob, len(blob)))

    def set_timing(self, on: bool):
        self._check(self.lib.muloco_set_timing(self.ctx, int(on)))

    def get_timings(self):
        ms = (C.c_float * len(PHASES))()
        launches = C.c_int64(0)
        self._check(self.lib.muloco_get_timings(self.ctx, ms, C.byref(launches)))
        return {p: ms[i] for i, p in enumerate(PHASES)}, launches.value

    def sync_status(self):
        self._check(self.lib.muloco_sync_status(self.ctx))

    # -- worker-sharded outer sync: three library calls around the caller's two collectives --------
    def shard_layout(self, fragment: int, world: int, rank: int):
        """muloco_shard_layout -> (stage_floats, shard_floats)."""
        a, b = C.c_int64(0), C.c_int64(0)
        self._check(self.lib.muloco_shard_layout(self.ctx, fragment, world, rank, C.byref(a), C.byref(b)))
        return a.value, b.value

    def shard_delta(self, fragment: int, world: int, stage):
        self._check(self.lib.muloco_shard_delta(self.ctx, fragment, world, stage.data_ptr()))

    def shard_step(self, fragment: int, world: int, rank: int, reduced, theta_shard):
        self._check(self.lib.muloco_shard_step(self.ctx, fragment, world, rank, reduced.data_ptr(),
                                               theta_shard.data_ptr()))

    def shard_broadcast(self, fragment: int, world: int, theta_all):
        self._check(self.lib.muloco_shard_broadcast(self.ctx, fragment, world, theta_all.data_ptr()))

    def sharded_outer_sync(self, fragment: int, dist, group=None):
        """The outer synchronisation with the workers spread over the ranks of `group`
        (torch.distributed): local delta sums -> reduce-scatter -> Nesterov step on the shard ->
        all-gather -> broadcast into the local replicas.  The collectives run on this context's
        stream.  Returns the bytes this rank sent and received over the wire (the ring
        algorithm's 2 * 4 * stage_floats * (world - 1) / world)."""
        return sharded_outer_sync(self, fragment, dist, group)

    def check_workspace(self):
        """muloco_check_workspace: raises MulocoError(ESTATE) if a workspace canary was overwritten."""
        self._check(self.lib.muloco_check_workspace(self.ctx))

    def debug_set(self, what: int, value: int):
        """muloco_debug_set (test hooks of the failure path)."""
        self._check(self.lib.muloco_debug_set(self.ctx, what, value))
