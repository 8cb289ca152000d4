"""Thin ctypes binding of libspeckv (argument marshalling only).

Every step of the path runs in the CUDA kernels behind the C ABI of ``include/speckv.h``;
this module only turns torch tensors into pointers, allocates outputs and scratch through
torch, and passes torch's current stream.  There is no CPU fallback: a missing library or a
non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass, field
from typing import Optional

import torch

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_STATIC_LIMIT = range(6)
F32, BF16 = 0, 1
ROW_OK, ROW_BAD_GAMMA, ROW_BAD_TOKEN, ROW_NONFINITE, ROW_BAD_TEMPERATURE, ROW_TIMEOUT = 0, 1, 2, 4, 8, 16

READ_ALL_TARGET_ROWS, SCHEDULE_SLICED = 1, 4   # speckv_batch.flags

STATIC_SCRATCH_BYTES = 4 << 20
EXPORTS = ("speckv_workspace_size", "speckv_signals", "speckv_signals_static", "speckv_select_gamma", "speckv_verify",
           "speckv_sample_workspace_size", "speckv_sample_draft",
           "speckv_step", "speckv_step_profiled", "speckv_status_string", "speckv_version")


class SpeckvError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} (status {code})")
        self.code = code


class _CBatch(C.Structure):
    _fields_ = [("B", C.c_int32), ("gamma_max", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
                ("draft_logits", C.c_void_p), ("draft_stride_b", C.c_int64), ("draft_stride_pos", C.c_int64),
                ("target_logits", C.c_void_p), ("target_stride_b", C.c_int64), ("target_stride_pos", C.c_int64),
                ("draft_tokens", C.c_void_p), ("gamma", C.c_void_p), ("temperature", C.c_void_p),
                ("temperature_scalar", C.c_float), ("uniforms", C.c_void_p), ("entropy_in_bits", C.c_int32),
                ("flags", C.c_int32)]


class _CMlp(C.Structure):
    _fields_ = [("n_in", C.c_int32), ("n_hidden", C.c_int32), ("n_out", C.c_int32),
                ("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p),
                ("gamma_choices", C.c_int32 * 8), ("feature_layout", C.c_int32),
                ("score_transform", C.c_int32)]


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """dlopen libspeckv.so (building it first if nvcc is available and it is stale)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _build.LIB_PATH
    if path is None:
        try:
            _build.build()
        except Exception as e:  # no nvcc on the box: use the shipped binary if there is one
            if not os.path.exists(p):
                raise RuntimeError(f"libspeckv.so is missing and could not be built: {e}") from e
    if not os.path.exists(p):
        raise RuntimeError(f"libspeckv.so not found at {p}; run `python -m paper_2605_02888_b200.build`")
    L = C.CDLL(p)
    vp, sz = C.c_void_p, C.c_size_t
    L.speckv_workspace_size.restype = C.c_int
    L.speckv_workspace_size.argtypes = [C.POINTER(_CBatch), C.POINTER(sz)]
    L.speckv_signals.restype = C.c_int
    L.speckv_signals.argtypes = [C.POINTER(_CBatch), vp, vp, vp, vp, vp, sz, vp]
    L.speckv_signals_static.restype = C.c_int
    L.speckv_signals_static.argtypes = [C.POINTER(_CBatch), vp, vp, vp, vp, vp]
    L.speckv_sample_workspace_size.restype = C.c_int
    L.speckv_sample_workspace_size.argtypes = [C.POINTER(_CBatch), C.POINTER(sz)]
    L.speckv_sample_draft.restype = C.c_int
    L.speckv_sample_draft.argtypes = [C.POINTER(_CBatch), vp, vp, vp, vp, sz, vp]
    L.speckv_select_gamma.restype = C.c_int
    L.speckv_select_gamma.argtypes = [C.c_int32, vp, vp, C.POINTER(_CMlp), vp, vp, vp]
    L.speckv_verify.restype = C.c_int
    L.speckv_verify.argtypes = [C.POINTER(_CBatch), vp, vp, vp, vp, sz, vp]
    L.speckv_step.restype = C.c_int
    L.speckv_step.argtypes = [C.POINTER(_CBatch), vp, C.POINTER(_CMlp)] + [vp] * 8 + [vp, sz, vp]
    # include/speckv_internal.h: the benchmark's timing aid and two test hooks
    L.speckv_step_profiled.restype = C.c_int
    L.speckv_step_profiled.argtypes = L.speckv_step.argtypes + [vp, vp, vp]
    L.speckv_internal_set_wait_limit.restype = C.c_int
    L.speckv_internal_set_wait_limit.argtypes = [C.c_int]
    L.speckv_internal_wait_probe.restype = C.c_int
    L.speckv_internal_wait_probe.argtypes = [C.c_int32, vp, vp, vp, sz, vp]
    L.speckv_internal_debug_report.restype = C.c_int
    L.speckv_internal_debug_report.argtypes = [C.POINTER(C.c_ulonglong), C.c_int, C.c_int]
    i32, i64 = C.c_int32, C.c_int64
    L.speckv_shard_workspace_size.restype = C.c_int
    L.speckv_shard_workspace_size.argtypes = [C.POINTER(_CBatch), C.POINTER(sz)]
    L.speckv_shard_sweep.restype = C.c_int
    L.speckv_shard_sweep.argtypes = [C.POINTER(_CBatch), i64, vp, vp, vp, sz, vp]
    L.speckv_shard_finish.restype = C.c_int
    L.speckv_shard_finish.argtypes = [C.POINTER(_CBatch), i32, i32, i32, vp, vp, vp, C.POINTER(_CMlp)] + [vp] * 8 + [vp, vp]
    L.speckv_shard_draw_sums.restype = C.c_int
    L.speckv_shard_draw_sums.argtypes = [C.POINTER(_CBatch), vp, vp, vp, sz, vp]
    L.speckv_shard_draw_pick.restype = C.c_int
    L.speckv_shard_draw_pick.argtypes = [C.POINTER(_CBatch), i64, i32, i32, vp, vp, vp, vp, sz, vp]
    L.speckv_status_string.restype = C.c_char_p
    L.speckv_status_string.argtypes = [C.c_int]
    L.speckv_version.restype = C.c_int
    L.speckv_version.argtypes = []
    if path is None:
        _lib = L
    return L


def status_string(code: int) -> str:
    return load_library().speckv_status_string(int(code)).decode()


def version() -> int:
    return load_library().speckv_version()


def _dev_ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _buf(t: Optional[torch.Tensor], dtype: torch.dtype, shape: tuple, dev: torch.device, name: str):
    """Pointer of a caller-provided buffer after checking what the library cannot: exact shape, dtype,
    contiguity and that it lives on the logits' device (a wrong one would be an out-of-bounds or
    foreign-address write on the GPU).  None passes through as NULL."""
    if t is None:
        return None
    if not t.is_cuda or t.device != dev:
        raise ValueError(f"{name} must be on {dev}, got {t.device}")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


@dataclass
class Batch:
    """One speculation step's inputs as CUDA tensors (see speckv_batch in speckv.h)."""
    draft_logits: torch.Tensor                      # [B, gamma_max, V] bf16 / fp32, V contiguous
    target_logits: Optional[torch.Tensor] = None    # [B, gamma_max+1, V]
    draft_tokens: Optional[torch.Tensor] = None     # [B, gamma_max] int32
    gamma: Optional[torch.Tensor] = None            # [B] int32
    temperature: Optional[torch.Tensor] = None      # [B] fp32
    temperature_scalar: float = 1.0
    uniforms: Optional[torch.Tensor] = None         # [B, gamma_max+1, 2] fp32
    entropy_in_bits: bool = False
    flags: int = 0                                  # READ_ALL_TARGET_ROWS | SCHEDULE_SLICED

    def shape(self):
        B, G, V = self.draft_logits.shape
        return B, G, V

    def _c(self) -> _CBatch:
        d = self.draft_logits
        if d.dim() != 3:
            raise ValueError("draft_logits must be [B, gamma_max, V]")
        if not d.is_cuda:
            raise ValueError("draft_logits must be a CUDA tensor (the library has no CPU path)")
        if d.dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("logits must be float32 or bfloat16")
        B, G, V = d.shape
        if V > 1 and d.stride(2) != 1:
            raise ValueError("the vocabulary dimension must be contiguous")
        c = _CBatch()
        c.B, c.gamma_max, c.V = B, G, V
        c.dtype = BF16 if d.dtype == torch.bfloat16 else F32
        c.draft_logits = d.data_ptr()
        c.draft_stride_b, c.draft_stride_pos = d.stride(0), d.stride(1)
        t = self.target_logits
        if t is not None:
            if tuple(t.shape) != (B, G + 1, V) or t.dtype != d.dtype or not t.is_cuda or t.device != d.device:
                raise ValueError("target_logits must be a CUDA tensor [B, gamma_max+1, V] of the draft's dtype")
            if V > 1 and t.stride(2) != 1:
                raise ValueError("the vocabulary dimension must be contiguous")
            c.target_logits = t.data_ptr()
            c.target_stride_b, c.target_stride_pos = t.stride(0), t.stride(1)
        for name, dt, shp in (("draft_tokens", torch.int32, (B, G)), ("gamma", torch.int32, (B,)),
                              ("temperature", torch.float32, (B,)), ("uniforms", torch.float32, (B, G + 1, 2))):
            a = getattr(self, name)
            setattr(c, name, _buf(a, dt, shp, d.device, name))
        c.temperature_scalar = float(self.temperature_scalar)
        c.entropy_in_bits = int(bool(self.entropy_in_bits))
        c.flags = int(self.flags)
        return c


@dataclass
class Mlp:
    """Controller parameters as CUDA fp32 tensors (see speckv_mlp in speckv.h)."""
    W1: torch.Tensor
    b1: torch.Tensor
    W2: torch.Tensor
    b2: torch.Tensor
    gamma_choices: tuple = (2, 4, 6, 8)
    feature_layout: int = 0
    score_transform: int = 0

    @property
    def n_in(self):
        return self.W1.shape[1]

    @property
    def n_out(self):
        # layout 2 (the paper's f(x, gamma)): one head, one score per candidate gamma
        return len(self.gamma_choices) if self.feature_layout == 2 else self.W2.shape[0]

    @property
    def n_comp(self):
        return self.n_in - (3, 4, 5)[self.feature_layout]

    def _c(self) -> _CMlp:
        m = _CMlp()
        m.n_hidden, m.n_in = self.W1.shape
        m.n_out = self.n_out
        if self.feature_layout == 2:
            if tuple(self.W2.shape) != (1, m.n_hidden if m.n_hidden else m.n_in) or tuple(self.b2.shape) != (1,) \
                    or tuple(self.b1.shape) != (m.n_hidden,):
                raise ValueError("inconsistent controller shapes for the paper-form predictor")
        elif self.W2.shape[1] != m.n_hidden or tuple(self.b1.shape) != (m.n_hidden,) or tuple(self.b2.shape) != (m.n_out,):
            raise ValueError("inconsistent controller shapes")
        if len(self.gamma_choices) < m.n_out or m.n_out > 8:
            raise ValueError("need one gamma choice per output (at most 8)")
        m.W1 = _dev_ptr(self.W1, torch.float32, "W1")
        m.b1 = _dev_ptr(self.b1, torch.float32, "b1")
        m.W2 = _dev_ptr(self.W2, torch.float32, "W2")
        m.b2 = _dev_ptr(self.b2, torch.float32, "b2")
        for j in range(m.n_out):
            m.gamma_choices[j] = int(self.gamma_choices[j])
        m.feature_layout, m.score_transform = int(self.feature_layout), int(self.score_transform)
        return m


def workspace_size(batch: Batch) -> int:
    n = C.c_size_t(0)
    c = batch._c()
    rc = load_library().speckv_workspace_size(C.byref(c), C.byref(n))
    if rc != OK:
        raise SpeckvError(rc, "speckv_workspace_size")
    return int(n.value)


def _workspace(batch: Batch, ws: Optional[torch.Tensor]) -> torch.Tensor:
    need = workspace_size(batch)
    if ws is None:
        ws = torch.empty(need, dtype=torch.uint8, device=batch.draft_logits.device)
    return ws


def _stream(dev) -> int:
    return torch.cuda.current_stream(dev).cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


@dataclass
class StepOutputs:
    """Caller-owned output buffers of one step; reusable across steps of the same shape."""
    H: torch.Tensor
    C: torch.Tensor
    feat: torch.Tensor
    scores: torch.Tensor
    gamma_next: torch.Tensor
    n_accepted: torch.Tensor
    out_tokens: torch.Tensor
    row_status: torch.Tensor
    workspace: torch.Tensor

    @staticmethod
    def allocate(batch: Batch, n_out: int = 4) -> "StepOutputs":
        B, G, V = batch.shape()
        dev = batch.draft_logits.device
        f = lambda *s: torch.empty(*s, dtype=torch.float32, device=dev)
        i = lambda *s: torch.empty(*s, dtype=torch.int32, device=dev)
        return StepOutputs(H=f(B, G), C=f(B, G), feat=f(B, 4), scores=f(B, n_out), gamma_next=i(B),
                           n_accepted=i(B), out_tokens=i(B, G + 1), row_status=i(B),
                           workspace=_workspace(batch, None))

    def as_dict(self):
        return {k: getattr(self, k) for k in ("H", "C", "feat", "scores", "gamma_next", "n_accepted",
                                              "out_tokens", "row_status")}

    def pointers(self, batch: "Batch", n_out: int) -> dict:
        """Device pointers of the buffers, each checked against the batch it is about to be used with."""
        B, G, V = batch.shape()
        dev = batch.draft_logits.device
        f32, i32 = torch.float32, torch.int32
        p = dict(H=_buf(self.H, f32, (B, G), dev, "H"), C=_buf(self.C, f32, (B, G), dev, "C"),
                 feat=_buf(self.feat, f32, (B, 4), dev, "feat"),
                 scores=_buf(self.scores, f32, (B, n_out), dev, "scores") if n_out else None,
                 gamma_next=_buf(self.gamma_next, i32, (B,), dev, "gamma_next"),
                 n_accepted=_buf(self.n_accepted, i32, (B,), dev, "n_accepted"),
                 out_tokens=_buf(self.out_tokens, i32, (B, G + 1), dev, "out_tokens"),
                 row_status=_buf(self.row_status, i32, (B,), dev, "row_status"))
        ws = self.workspace
        if ws is None or not ws.is_cuda or ws.device != dev or ws.dtype != torch.uint8 or not ws.is_contiguous():
            raise ValueError(f"workspace must be a contiguous uint8 tensor on {dev}")
        if ws.numel() < workspace_size(batch):
            raise ValueError(f"workspace holds {ws.numel()} bytes, this batch needs {workspace_size(batch)}")
        p["workspace"] = ws.data_ptr()
        return p


def speckv_signals(batch: Batch, out: Optional[StepOutputs] = None):
    """Draft signals (paper Sec. 4.2): H, C [B, gamma_max]; feat [B, 4]; row_status [B]."""
    L = load_library()
    c = batch._c()
    o = out or StepOutputs.allocate(batch)
    q = o.pointers(batch, 0)
    with torch.cuda.device(batch.draft_logits.device):
        rc = L.speckv_signals(C.byref(c), q["H"], q["C"], q["feat"], q["row_status"],
                              q["workspace"], o.workspace.numel(), _stream(batch.draft_logits.device))
    if rc != OK:
        raise SpeckvError(rc, "speckv_signals")
    return dict(H=o.H, C=o.C, feat=o.feat, row_status=o.row_status)


def speckv_signals_static(batch: Batch, H: torch.Tensor, Cc: torch.Tensor, feat: torch.Tensor,
                          row_status: torch.Tensor):
    """speckv_signals without a workspace argument, for callers that may not allocate device
    memory: the scratch is a fixed array inside the library (STATIC_SCRATCH_BYTES per device).
    All four outputs are caller-provided CUDA tensors; nothing is allocated here either.
    Raises SpeckvError(ERR_STATIC_LIMIT) when the batch needs more scratch than that."""
    L = load_library()
    c = batch._c()
    dev = batch.draft_logits.device
    B, G, _ = batch.shape()
    f32 = torch.float32
    ptrs = (_buf(H, f32, (B, G), dev, "H"), _buf(Cc, f32, (B, G), dev, "C"), _buf(feat, f32, (B, 4), dev, "feat"),
            _buf(row_status, torch.int32, (B,), dev, "row_status"))
    with torch.cuda.device(dev):
        rc = L.speckv_signals_static(C.byref(c), *ptrs, _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_signals_static")
    return dict(H=H, C=Cc, feat=feat, row_status=row_status)


def speckv_sample_draft(batch: Batch, uniforms: torch.Tensor, tokens: Optional[torch.Tensor] = None,
                        row_status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """Draft tokens (paper Sec. 3.1): tokens[b,i] ~ softmax(draft_logits[b,i] / T_b) by inverse CDF at
    uniforms[b,i] (argmax for T_b = 0); -1 beyond gamma_b.  uniforms: [B, gamma_max] fp32."""
    L = load_library()
    c = batch._c()
    B, G, V = batch.shape()
    dev = batch.draft_logits.device
    _buf(uniforms, torch.float32, (B, G), dev, "uniforms")
    if tokens is None:
        tokens = torch.empty(B, G, dtype=torch.int32, device=dev)
    if row_status is None:
        row_status = torch.empty(B, dtype=torch.int32, device=dev)
    if workspace is None:
        n = C.c_size_t(0)
        rc = L.speckv_sample_workspace_size(C.byref(c), C.byref(n))
        if rc != OK:
            raise SpeckvError(rc, "speckv_sample_workspace_size")
        workspace = torch.empty(int(n.value), dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        rc = L.speckv_sample_draft(C.byref(c), _buf(uniforms, torch.float32, (B, G), dev, "uniforms"),
                                   _buf(tokens, torch.int32, (B, G), dev, "tokens"),
                                   _buf(row_status, torch.int32, (B,), dev, "row_status"),
                                   _buf(workspace, torch.uint8, (workspace.numel(),), dev, "workspace"), workspace.numel(), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_sample_draft")
    return dict(tokens=tokens, row_status=row_status)


def speckv_select_gamma(feat: torch.Tensor, comp: Optional[torch.Tensor], mlp: Mlp,
                        scores: Optional[torch.Tensor] = None, gamma_next: Optional[torch.Tensor] = None):
    """Controller (paper Sec. 4.3, Eq. 1): scores [B, n_out], gamma_next [B]."""
    L = load_library()
    B = feat.shape[0]
    m = mlp._c()
    dev = feat.device
    if scores is None:
        scores = torch.empty(B, mlp.n_out, dtype=torch.float32, device=dev)
    if gamma_next is None:
        gamma_next = torch.empty(B, dtype=torch.int32, device=dev)
    if not feat.is_cuda:
        raise ValueError("feat must be a CUDA tensor (the library has no CPU path)")
    with torch.cuda.device(dev):
        rc = L.speckv_select_gamma(B, _buf(feat, torch.float32, (B, 4), dev, "feat"),
                                   _buf(comp, torch.float32, (B, mlp.n_comp), dev, "comp") if mlp.n_comp > 0 else None,
                                   C.byref(m), _buf(scores, torch.float32, (B, mlp.n_out), dev, "scores"),
                                   _buf(gamma_next, torch.int32, (B,), dev, "gamma_next"), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_select_gamma")
    return dict(scores=scores, gamma_next=gamma_next)


def speckv_verify(batch: Batch, out: Optional[StepOutputs] = None):
    """Verification (paper Sec. 3.1 / speculative sampling): n_accepted, out_tokens, row_status."""
    L = load_library()
    c = batch._c()
    o = out or StepOutputs.allocate(batch)
    dev = batch.draft_logits.device
    q = o.pointers(batch, 0)
    with torch.cuda.device(dev):
        rc = L.speckv_verify(C.byref(c), q["n_accepted"], q["out_tokens"], q["row_status"],
                             q["workspace"], o.workspace.numel(), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_verify")
    return dict(n_accepted=o.n_accepted, out_tokens=o.out_tokens, row_status=o.row_status)


def speckv_step(batch: Batch, comp: Optional[torch.Tensor], mlp: Mlp, out: Optional[StepOutputs] = None,
                events: Optional[tuple] = None):
    """Fused step: signals + controller + verification.  Returns the StepOutputs tensors.
    `events`: optional (before_sweep, after_sweep, after_resample) torch.cuda.Event objects
    (created with enable_timing=True); they are recorded before and after the sweep kernel and after
    the resample kernel (the last two coincide where the sweep kernel's grid draws the tokens itself)."""
    L = load_library()
    c = batch._c()
    m = mlp._c()
    o = out or StepOutputs.allocate(batch, mlp.n_out)
    dev = batch.draft_logits.device
    q = o.pointers(batch, mlp.n_out)
    B = batch.shape()[0]
    cptr = _buf(comp, torch.float32, (B, mlp.n_comp), dev, "comp") if (comp is not None and mlp.n_comp > 0) else None
    for name in ("W1", "b1", "W2", "b2"):
        if getattr(mlp, name).device != dev:
            raise ValueError(f"controller parameter {name} must be on {dev}")
    args = [C.byref(c), cptr, C.byref(m), q["H"], q["C"], q["feat"], q["scores"], q["gamma_next"], q["n_accepted"],
            q["out_tokens"], q["row_status"], q["workspace"], o.workspace.numel(), _stream(dev)]
    with torch.cuda.device(dev):
        if events is None:
            rc = L.speckv_step(*args)
        else:
            evs = []
            for e in events:
                if e is not None and not e.cuda_event:  # torch creates the event lazily on first record
                    e.record(torch.cuda.current_stream(dev))
                evs.append(None if e is None else e.cuda_event)
            rc = L.speckv_step_profiled(*args, *evs)
    if rc != OK:
        raise SpeckvError(rc, "speckv_step")
    return o.as_dict()


# ---- vocabulary-sharded step: the four calls of include/speckv.h, argument marshalling only ----
ROW_INFO_BYTES = 32


def shard_workspace(local: Batch) -> torch.Tensor:
    L = load_library()
    c = local._c()
    n = C.c_size_t(0)
    rc = L.speckv_shard_workspace_size(C.byref(c), C.byref(n))
    if rc != OK:
        raise SpeckvError(rc, "speckv_shard_workspace_size")
    return torch.empty(max(int(n.value), 256), dtype=torch.uint8, device=local.draft_logits.device)


def speckv_shard_sweep(local: Batch, v_begin: int, shard_state: torch.Tensor, shard_tokl: torch.Tensor,
                       workspace: torch.Tensor):
    """Local slice -> shard_state [B, 2G+1, 4] fp32, shard_tokl [B, G, 2] fp32 (both written)."""
    L = load_library()
    c = local._c()
    dev = local.draft_logits.device
    with torch.cuda.device(dev):
        rc = L.speckv_shard_sweep(C.byref(c), int(v_begin), _dev_ptr(shard_state, torch.float32, "shard_state"),
                                  _dev_ptr(shard_tokl, torch.float32, "shard_tokl"), _ptr(workspace),
                                  workspace.numel(), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_shard_sweep")


def speckv_shard_finish(local: Batch, n_shards: int, shard_width: int, V_total: int, all_state: torch.Tensor,
                        all_tokl: torch.Tensor, comp: Optional[torch.Tensor], mlp: Optional[Mlp], out: "StepOutputs",
                        row_info: torch.Tensor):
    """Gathered states -> every step output but the sampled rows' fresh token; row_info for the draw."""
    L = load_library()
    c = local._c()
    m = mlp._c() if mlp is not None else None
    dev = local.draft_logits.device
    with torch.cuda.device(dev):
        rc = L.speckv_shard_finish(C.byref(c), n_shards, shard_width, V_total,
                                   _dev_ptr(all_state, torch.float32, "all_state"),
                                   _dev_ptr(all_tokl, torch.float32, "all_tokl"),
                                   _dev_ptr(comp, torch.float32, "comp"), C.byref(m) if m is not None else None,
                                   _ptr(out.H), _ptr(out.C), _ptr(out.feat), _ptr(out.scores), _ptr(out.gamma_next),
                                   _ptr(out.n_accepted), _ptr(out.out_tokens), _ptr(out.row_status),
                                   _ptr(row_info), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_shard_finish")


def speckv_shard_draw_sums(local: Batch, row_info: torch.Tensor, shard_weight: torch.Tensor, workspace: torch.Tensor):
    """Local slice -> shard_weight [B, 2] fp64 (residual mass, target mass of the stop position)."""
    L = load_library()
    c = local._c()
    dev = local.draft_logits.device
    with torch.cuda.device(dev):
        rc = L.speckv_shard_draw_sums(C.byref(c), _ptr(row_info), _dev_ptr(shard_weight, torch.float64, "shard_weight"),
                                      _ptr(workspace), workspace.numel(), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_shard_draw_sums")


def speckv_shard_draw_pick(local: Batch, v_begin: int, rank: int, n_shards: int, row_info: torch.Tensor,
                           all_weight: torch.Tensor, out_tokens: torch.Tensor, workspace: torch.Tensor):
    """The shard holding the drawn token writes it into out_tokens[b, n_accepted[b]]."""
    L = load_library()
    c = local._c()
    dev = local.draft_logits.device
    with torch.cuda.device(dev):
        rc = L.speckv_shard_draw_pick(C.byref(c), int(v_begin), rank, n_shards, _ptr(row_info),
                                      _dev_ptr(all_weight, torch.float64, "all_weight"),
                                      _dev_ptr(out_tokens, torch.int32, "out_tokens"), _ptr(workspace),
                                      workspace.numel(), _stream(dev))
    if rc != OK:
        raise SpeckvError(rc, "speckv_shard_draw_pick")
