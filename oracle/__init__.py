"""ctypes loader for the SpecKV CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may
import this package.  It builds ``speckv_oracle.cpp`` with g++ on first use and
exposes the C entry points on numpy arrays.  bf16 logits are passed as uint16 bit
patterns.  The product package never imports it and it never imports the product.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "speckv_oracle.cpp")
_HDR = os.path.join(_HERE, "speckv_oracle.h")
_LIB = os.path.join(_HERE, "libspeckv_oracle.so")

DT_F32, DT_BF16 = 0, 1
ROW_OK, ROW_BAD_GAMMA, ROW_BAD_TOKEN, ROW_NONFINITE, ROW_BAD_TEMPERATURE = 0, 1, 2, 4, 8
NEAR_ACCEPT, NEAR_CDF, NEAR_GREEDY, NEAR_GAMMA, NEAR_SMALL_RESIDUAL, NEAR_CDF_ABS = 1, 2, 4, 8, 16, 32


def build(force: bool = False) -> str:
    """Compile the oracle shared library (g++, -O2, no fast-math) if it is stale."""
    stale = force or not os.path.exists(_LIB) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB) for s in (_SRC, _HDR))
    if stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread",
                               "-ffp-contract=off", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Batch(C.Structure):
    _fields_ = [("B", C.c_int32), ("gamma_max", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
                ("draft", C.c_void_p), ("draft_stride_row", C.c_int64), ("draft_stride_pos", C.c_int64),
                ("target", C.c_void_p), ("target_stride_row", C.c_int64), ("target_stride_pos", C.c_int64),
                ("draft_tokens", C.c_void_p), ("gamma", C.c_void_p), ("temperature", C.c_void_p),
                ("temperature_scalar", C.c_float), ("uniforms", C.c_void_p),
                ("entropy_in_bits", C.c_int32), ("n_threads", C.c_int32)]


class _Mlp(C.Structure):
    _fields_ = [("n_in", C.c_int32), ("n_hidden", C.c_int32), ("n_out", C.c_int32),
                ("W1", C.c_void_p), ("b1", C.c_void_p), ("W2", C.c_void_p), ("b2", C.c_void_p),
                ("gamma_choices", C.c_int32 * 8), ("feature_layout", C.c_int32),
                ("score_transform", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.oracle_signals.restype = C.c_int
        L.oracle_signals.argtypes = [C.POINTER(_Batch), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_select_gamma.restype = C.c_int
        L.oracle_select_gamma.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(_Mlp),
                                          C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_verify.restype = C.c_int
        L.oracle_verify.argtypes = [C.POINTER(_Batch), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_sample_draft.restype = C.c_int
        L.oracle_sample_draft.argtypes = [C.POINTER(_Batch)] + [C.c_void_p] * 4
        L.oracle_step.restype = C.c_int
        L.oracle_step.argtypes = [C.POINTER(_Batch), C.c_void_p, C.POINTER(_Mlp)] + [C.c_void_p] * 9
        L.oracle_softmax_row.restype = C.c_int
        L.oracle_softmax_row.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_double, C.c_void_p]
        L.oracle_entropy_nats.restype = C.c_double
        L.oracle_entropy_nats.argtypes = [C.c_void_p, C.c_int32]
        L.oracle_inverse_cdf.restype = C.c_int32
        L.oracle_inverse_cdf.argtypes = [C.c_void_p, C.c_int32, C.c_double, C.c_void_p]
        L.oracle_argmax_row.restype = C.c_int32
        L.oracle_argmax_row.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _logits(a: np.ndarray):
    """Accept float32 or uint16 (bf16 bit patterns) arrays of shape [..., V], V contiguous."""
    if a.dtype == np.float32:
        return DT_F32
    if a.dtype == np.uint16:
        return DT_BF16
    raise TypeError(f"logits must be float32 or uint16 (bf16 bits), got {a.dtype}")


@dataclass
class Batch:
    """Host-side description of one speculation step's inputs (numpy arrays)."""
    draft: np.ndarray                      # [B, gamma_max, V] float32 or uint16
    target: Optional[np.ndarray] = None    # [B, gamma_max+1, V]
    draft_tokens: Optional[np.ndarray] = None  # [B, gamma_max] int32
    gamma: Optional[np.ndarray] = None     # [B] int32
    temperature: Optional[np.ndarray] = None  # [B] float32
    temperature_scalar: float = 1.0
    uniforms: Optional[np.ndarray] = None  # [B, gamma_max+1, 2] float32
    entropy_in_bits: bool = False
    n_threads: int = 1

    def _c(self):
        d = self.draft
        assert d.ndim == 3 and d.strides[2] == d.itemsize
        dt = _logits(d)
        B, G, V = d.shape
        keep = [d]
        bt = _Batch()
        bt.B, bt.gamma_max, bt.V, bt.dtype = B, G, V, dt
        bt.draft = d.ctypes.data
        bt.draft_stride_row, bt.draft_stride_pos = d.strides[0] // d.itemsize, d.strides[1] // d.itemsize
        if self.target is not None:
            t = self.target
            assert t.shape == (B, G + 1, V) and t.dtype == d.dtype and t.strides[2] == t.itemsize
            bt.target = t.ctypes.data
            bt.target_stride_row, bt.target_stride_pos = t.strides[0] // t.itemsize, t.strides[1] // t.itemsize
            keep.append(t)
        for name, dtype, shape in (("draft_tokens", np.int32, (B, G)), ("gamma", np.int32, (B,)),
                                   ("temperature", np.float32, (B,)),
                                   ("uniforms", np.float32, (B, G + 1, 2))):
            a = getattr(self, name)
            if a is not None:
                a = np.ascontiguousarray(a, dtype=dtype)
                assert a.shape == shape, (name, a.shape, shape)
                keep.append(a)
                setattr(bt, name, a.ctypes.data)
        bt.temperature_scalar = float(self.temperature_scalar)
        bt.entropy_in_bits = int(bool(self.entropy_in_bits))
        bt.n_threads = int(self.n_threads)
        return bt, keep


@dataclass
class Mlp:
    """Controller parameters (float32 numpy arrays)."""
    W1: np.ndarray  # [n_hidden, n_in]
    b1: np.ndarray  # [n_hidden]
    W2: np.ndarray  # [n_out, n_hidden]
    b2: np.ndarray  # [n_out]
    gamma_choices: tuple = (2, 4, 6, 8)
    feature_layout: int = 0
    score_transform: int = 0

    def _c(self):
        W1 = np.ascontiguousarray(self.W1, np.float32)
        b1 = np.ascontiguousarray(self.b1, np.float32)
        W2 = np.ascontiguousarray(self.W2, np.float32)
        b2 = np.ascontiguousarray(self.b2, np.float32)
        m = _Mlp()
        if self.feature_layout == 2:
            # the paper's f(x, gamma): one output, evaluated per candidate; W1 [0, n_in] => linear
            m.n_hidden, m.n_in = W1.shape
            m.n_out = len(self.gamma_choices)
            assert W2.shape == (1, m.n_hidden if m.n_hidden else m.n_in) and b2.shape == (1,)
            assert b1.shape == (m.n_hidden,) and m.n_out <= 8
        else:
            m.n_hidden, m.n_in = W1.shape
            m.n_out = W2.shape[0]
            assert W2.shape[1] == m.n_hidden and b1.shape == (m.n_hidden,) and b2.shape == (m.n_out,)
        assert len(self.gamma_choices) >= m.n_out
        m.W1, m.b1, m.W2, m.b2 = W1.ctypes.data, b1.ctypes.data, W2.ctypes.data, b2.ctypes.data
        for j in range(m.n_out):
            m.gamma_choices[j] = int(self.gamma_choices[j])
        m.feature_layout, m.score_transform = int(self.feature_layout), int(self.score_transform)
        return m, [W1, b1, W2, b2]

    @property
    def n_comp(self) -> int:
        return self.W1.shape[1] - (3, 4, 5)[self.feature_layout]

    @property
    def n_out(self) -> int:
        return len(self.gamma_choices) if self.feature_layout == 2 else self.W2.shape[0]


def signals(bt: Batch):
    c, keep = bt._c()
    B, G = c.B, c.gamma_max
    H = np.zeros((B, G)); Cc = np.zeros((B, G)); feat = np.zeros((B, 4))
    st = np.zeros(B, np.int32)
    rc = lib().oracle_signals(C.byref(c), _ptr(H), _ptr(Cc), _ptr(feat), _ptr(st))
    if rc:
        raise ValueError("oracle_signals: invalid arguments")
    return dict(H=H, C=Cc, feat=feat, row_status=st)


def select_gamma(feat: np.ndarray, comp: Optional[np.ndarray], mlp: Mlp):
    m, keep = mlp._c()
    feat = np.ascontiguousarray(feat, np.float64)
    B = feat.shape[0]
    if comp is not None:
        comp = np.ascontiguousarray(comp, np.float32).reshape(B, mlp.n_comp)
    scores = np.zeros((B, m.n_out)); g = np.zeros(B, np.int32); near = np.zeros(B, np.int32)
    rc = lib().oracle_select_gamma(B, _ptr(feat), _ptr(comp), C.byref(m), _ptr(scores), _ptr(g), _ptr(near))
    if rc:
        raise ValueError("oracle_select_gamma: invalid arguments")
    return dict(scores=scores, gamma_next=g, near=near)


def verify(bt: Batch):
    c, keep = bt._c()
    B, G = c.B, c.gamma_max
    n = np.zeros(B, np.int32); out = np.zeros((B, G + 1), np.int32)
    st = np.zeros(B, np.int32); near = np.zeros(B, np.int32)
    rc = lib().oracle_verify(C.byref(c), _ptr(n), _ptr(out), _ptr(st), _ptr(near))
    if rc:
        raise ValueError("oracle_verify: invalid arguments")
    return dict(n_accepted=n, out_tokens=out, row_status=st, near=near)


def sample_draft(bt: Batch, uniforms: np.ndarray):
    """tokens[b,i] ~ softmax(draft[b,i] / T_b) by inverse CDF at uniforms[b,i]; argmax for T_b = 0."""
    c, keep = bt._c()
    B, G = c.B, c.gamma_max
    u = np.ascontiguousarray(uniforms, np.float32).reshape(B, G)
    tok = np.zeros((B, G), np.int32); st = np.zeros(B, np.int32); near = np.zeros(B, np.int32)
    rc = lib().oracle_sample_draft(C.byref(c), _ptr(u), _ptr(tok), _ptr(st), _ptr(near))
    if rc:
        raise ValueError("oracle_sample_draft: invalid arguments")
    return dict(tokens=tok, row_status=st, near=near)


def step(bt: Batch, comp: Optional[np.ndarray], mlp: Mlp):
    c, keep = bt._c()
    m, keep2 = mlp._c()
    B, G = c.B, c.gamma_max
    if comp is not None:
        comp = np.ascontiguousarray(comp, np.float32).reshape(B, mlp.n_comp)
    H = np.zeros((B, G)); Cc = np.zeros((B, G)); feat = np.zeros((B, 4))
    scores = np.zeros((B, m.n_out)); g = np.zeros(B, np.int32)
    n = np.zeros(B, np.int32); out = np.zeros((B, G + 1), np.int32)
    st = np.zeros(B, np.int32); near = np.zeros(B, np.int32)
    rc = lib().oracle_step(C.byref(c), _ptr(comp), C.byref(m), _ptr(H), _ptr(Cc), _ptr(feat),
                           _ptr(scores), _ptr(g), _ptr(n), _ptr(out), _ptr(st), _ptr(near))
    if rc:
        raise ValueError("oracle_step: invalid arguments")
    return dict(H=H, C=Cc, feat=feat, scores=scores, gamma_next=g, n_accepted=n, out_tokens=out,
                row_status=st, near=near)


def softmax_row(row: np.ndarray, T: float = 1.0):
    row = np.ascontiguousarray(row)
    p = np.zeros(row.shape[0])
    rc = lib().oracle_softmax_row(_ptr(row), _logits(row), row.shape[0], float(T), _ptr(p))
    return p, rc


def entropy_nats(p: np.ndarray) -> float:
    p = np.ascontiguousarray(p, np.float64)
    return lib().oracle_entropy_nats(_ptr(p), p.shape[0])


def inverse_cdf(w: np.ndarray, u: float):
    w = np.ascontiguousarray(w, np.float64)
    nb = C.c_int32(0)
    tok = lib().oracle_inverse_cdf(_ptr(w), w.shape[0], float(u), C.byref(nb))
    return tok, nb.value


def argmax_row(row: np.ndarray) -> int:
    row = np.ascontiguousarray(row)
    return lib().oracle_argmax_row(_ptr(row), _logits(row), row.shape[0])
