"""ctypes front end of the LASAD CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Compiles ``lasad_oracle.c`` (plain C, fp64, OpenMP over (batch, head)) with gcc into
``oracle/_build/`` and exposes its functions on numpy float64 arrays:

* :func:`recurrent` -- Algorithm 1's loop body (decay select, state update, readout);
* :func:`quadratic` -- the SAD recurrence of Section 3.4 unrolled into the explicit
  masked-decay sum over earlier tokens;
* :func:`layer_core` -- Algorithm 1's loop body with the operator's neighbours inside
  (SiLU on the query, Sigmoid on the gate, key tied to the gate, Norm on the output).

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s CPU-baseline leg import this
module.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lasad_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_OUT = os.path.join(_OUT_DIR, "liblasad_oracle.so")
_lock = threading.Lock()
_lib = None


class _Dims(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
        ("dk", ctypes.c_int32), ("dv", ctypes.c_int32),
        ("grid_w", ctypes.c_int32), ("prefix_len", ctypes.c_int32),
        ("t0", ctypes.c_int64), ("scale", ctypes.c_double),
        ("decay_stride", ctypes.c_int64 * 4),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle's C source with gcc if the shared object is missing or stale."""
    with _lock:
        fresh = os.path.exists(_OUT) and os.path.getmtime(_OUT) >= os.path.getmtime(_SRC)
        if fresh and not force:
            return _OUT
        os.makedirs(_OUT_DIR, exist_ok=True)
        tmp = _OUT + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _OUT)
        return _OUT


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        for name in ("lasad_oracle_recurrent", "lasad_oracle_quadratic"):
            fn = getattr(lib, name)
            fn.restype = ctypes.c_int
            fn.argtypes = [ctypes.POINTER(_Dims), dp, dp, dp, dp, dp, dp, dp]
        lib.lasad_oracle_layer_core.restype = ctypes.c_int
        lib.lasad_oracle_layer_core.argtypes = [ctypes.POINTER(_Dims), dp, dp, dp, dp, dp, ctypes.c_double, dp, dp]
        lib.lasad_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle's (batch, head) loop will use."""
    return int(_load().lasad_oracle_threads())


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def _run(name, q, k, v, decay, grid_w, prefix_len, t0, scale, state_in, want_state):
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    if q.ndim != 4 or k.shape != q.shape or v.ndim != 4 or v.shape[:3] != q.shape[:3]:
        raise ValueError("q,k must be [B,T,H,dk] and v [B,T,H,dv]")
    B, T, H, dk = q.shape
    dv = v.shape[3]
    # decay: anything that broadcasts to [B,T,H,dk]; a per-head constant is shape [H] -> [1,1,H,1]
    decay = np.asarray(decay, dtype=np.float64)
    if decay.ndim == 1 and decay.shape[0] == H:
        decay = decay.reshape(1, 1, H, 1)
    base = np.ascontiguousarray(decay)
    view = np.broadcast_to(base, (B, T, H, dk))
    strides = [s // 8 for s in view.strides]
    d = _Dims(B, T, H, dk, dv, int(grid_w), int(prefix_len), int(t0), float(scale),
              (ctypes.c_int64 * 4)(*strides))
    if state_in is not None:
        state_in = np.ascontiguousarray(state_in, dtype=np.float64)
        if state_in.shape != (B, H, dk, dv):
            raise ValueError("state_in must be [B,H,dk,dv]")
    o = np.empty((B, T, H, dv), dtype=np.float64)
    s_out = np.empty((B, H, dk, dv), dtype=np.float64) if want_state else None
    rc = getattr(_load(), name)(ctypes.byref(d), _ptr(q), _ptr(k), _ptr(v), _ptr(base),
                                _ptr(state_in), _ptr(o), _ptr(s_out))
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return o, s_out


def recurrent(q, k, v, decay, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None,
              want_state=True):
    """Algorithm 1 (decay select, state update, readout) in fp64.  Returns (o, state_out)."""
    return _run("lasad_oracle_recurrent", q, k, v, decay, grid_w, prefix_len, t0, scale,
                state_in, want_state)


def quadratic(q, k, v, decay, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None,
              want_state=True):
    """Explicit masked-decay sum (the SAD recurrence unrolled) in fp64.  Returns (o, state_out)."""
    return _run("lasad_oracle_quadratic", q, k, v, decay, grid_w, prefix_len, t0, scale,
                state_in, want_state)


def layer_core(q_pre, k, v, gate_pre, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None, eps=1e-6,
               want_state=True):
    """Algorithm 1's loop body with its neighbours: q = SiLU(q_pre), lambda = Sigmoid(gate_pre),
    k = 1 - lambda when ``k`` is None, the SAD recurrence, then a weight-free RMS norm of each
    head's output over its d_v channels.  Returns (normalised o, state_out), fp64."""
    q_pre = np.ascontiguousarray(q_pre, dtype=np.float64)
    gate_pre = np.ascontiguousarray(gate_pre, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    if k is not None:
        k = np.ascontiguousarray(k, dtype=np.float64)
    if q_pre.ndim != 4 or gate_pre.shape != q_pre.shape or (k is not None and k.shape != q_pre.shape) \
            or v.ndim != 4 or v.shape[:3] != q_pre.shape[:3]:
        raise ValueError("q_pre, gate_pre (and k) must be [B,T,H,dk] and v [B,T,H,dv]")
    B, T, H, dk = q_pre.shape
    dv = v.shape[3]
    d = _Dims(B, T, H, dk, dv, int(grid_w), int(prefix_len), int(t0), float(scale), (ctypes.c_int64 * 4)(0, 0, 0, 0))
    if state_in is not None:
        state_in = np.ascontiguousarray(state_in, dtype=np.float64)
        if state_in.shape != (B, H, dk, dv):
            raise ValueError("state_in must be [B,H,dk,dv]")
    o = np.empty((B, T, H, dv), dtype=np.float64)
    s_out = np.empty((B, H, dk, dv), dtype=np.float64) if want_state else None
    rc = _load().lasad_oracle_layer_core(ctypes.byref(d), _ptr(q_pre), _ptr(k), _ptr(v), _ptr(gate_pre),
                                         _ptr(state_in), float(eps), _ptr(o), _ptr(s_out))
    if rc != 0:
        raise MemoryError("oracle allocation failed")
    return o, s_out
