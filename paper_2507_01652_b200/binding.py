"""Thin Python binding of the LASAD C ABI (``include/lasad.h``): argument marshalling only.

Every step of the operator runs inside the CUDA library; this module turns torch CUDA tensors
into raw device pointers, element strides and a stream handle and calls ``lasad_forward`` /
``lasad_decode_step``.  There is no CPU path: if the library is missing or stale and cannot be
rebuilt, importing the handle raises.
"""
from __future__ import annotations

import ctypes
import threading

import torch

from . import build as _build

LASAD_OK = 0
LASAD_ERR_INVALID_ARG = -1
LASAD_ERR_UNSUPPORTED = -2
LASAD_ERR_CUDA = -3
LASAD_ERR_TIMEOUT = -4
LASAD_F32 = 0
LASAD_BF16 = 1
LASAD_OPT_PREFILL_IMPL = 0
LASAD_OPT_PREFILL_CHUNK = 1
LASAD_OPT_DECODE_TPU = 2
LASAD_OPT_WAIT_LIMIT = 3

EXPORTS = (
    "lasad_create", "lasad_destroy", "lasad_set_option", "lasad_reserve", "lasad_forward", "lasad_forward_host", "lasad_forward_static",
    "lasad_decode_step", "lasad_decode_step_pos", "lasad_forward_gated", "lasad_decode_step_gated",
    "lasad_forward_fused", "lasad_decode_step_fused",
    "lasad_last_device_status", "lasad_last_cuda_error", "lasad_launch_count", "lasad_strerror",
)


class LasadParams(ctypes.Structure):
    """Mirror of ``lasad_params``."""
    _fields_ = [
        ("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
        ("dk", ctypes.c_int32), ("dv", ctypes.c_int32),
        ("grid_w", ctypes.c_int32), ("prefix_len", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("t0", ctypes.c_int64), ("scale", ctypes.c_float), ("reserved", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
        ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
    ]


class LasadError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = load_library().lasad_strerror(code).decode()
        super().__init__(f"{where}: {msg} (code {code}){detail}")


_lib = None
_lib_lock = threading.Lock()


def load_library() -> ctypes.CDLL:
    """dlopen the in-tree library (building it first if the sources changed)."""
    global _lib
    with _lib_lock:
        if _lib is not None:
            return _lib
        path = _build.build()
        lib = ctypes.CDLL(path)
        vp, i32, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64
        pp = ctypes.POINTER(LasadParams)
        lib.lasad_create.restype = i32
        lib.lasad_create.argtypes = [ctypes.POINTER(vp), i32]
        lib.lasad_destroy.restype = i32
        lib.lasad_destroy.argtypes = [vp]
        lib.lasad_set_option.restype = i32
        lib.lasad_set_option.argtypes = [vp, i32, i32]
        lib.lasad_reserve.restype = i32
        lib.lasad_reserve.argtypes = [vp, ctypes.c_int64]
        lib.lasad_forward.restype = i32
        lib.lasad_forward.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_forward_host.restype = i32
        lib.lasad_forward_host.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_forward_static.restype = i32
        lib.lasad_forward_static.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_decode_step.restype = i32
        lib.lasad_decode_step.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_decode_step_pos.restype = i32
        lib.lasad_decode_step_pos.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_forward_gated.restype = i32
        lib.lasad_forward_gated.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_decode_step_gated.restype = i32
        lib.lasad_decode_step_gated.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp]
        lib.lasad_forward_fused.restype = i32
        lib.lasad_forward_fused.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp]
        lib.lasad_decode_step_fused.restype = i32
        lib.lasad_decode_step_fused.argtypes = [vp, pp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp]
        lib.lasad_last_device_status.restype = i32
        lib.lasad_last_device_status.argtypes = [vp, ctypes.POINTER(i32)]
        lib.lasad_last_cuda_error.restype = i32
        lib.lasad_last_cuda_error.argtypes = [vp]
        lib.lasad_launch_count.restype = u64
        lib.lasad_launch_count.argtypes = [vp]
        lib.lasad_strerror.restype = ctypes.c_char_p
        lib.lasad_strerror.argtypes = [i32]
        _lib = lib
        return lib


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LASAD_F32
    if t.dtype == torch.bfloat16:
        return LASAD_BF16
    raise TypeError(f"q, k, v, o must be float32 or bfloat16, got {t.dtype}")


def _ptr(t):
    # (an int is accepted where the prototype says c_void_p; None is a null pointer)
    return None if t is None else t.data_ptr()


try:
    _raw_stream = torch._C._cuda_getCurrentRawStream     # the current stream's handle without a Stream object
except AttributeError:       # pragma: no cover - older torch
    _raw_stream = None


def _stream(device, stream):
    if stream is not None:
        return stream
    if _raw_stream is not None:
        return _raw_stream(device.index if device.index is not None else torch.cuda.current_device())
    return torch.cuda.current_stream(device).cuda_stream


_params_cache = {}


def _params(kind, q, k, v, o, grid_w, prefix_len, t0, scale):
    """The call's ``lasad_params``.  The struct is cached per (shape, strides, dtype) -- building
    its ctypes arrays costs more than the rest of the marshalling -- and only its scalars are
    refreshed.  kind: "prefill" ([B,T,H,d] tensors) or "decode" ([B,H,d])."""
    key = (kind, q.shape, q.stride(), k.stride(), v.stride(), o.stride(), v.shape[-1], q.dtype)
    p = _params_cache.get(key)
    if p is None:
        if kind == "prefill":
            B, T, H, dk = q.shape
            p = LasadParams(B, T, H, dk, v.shape[3], 0, 0, _dtype_code(q), 0, 1.0, 0,
                            _strides3(q), _strides3(k), _strides3(v), _strides3(o))
        else:
            B, H, dk = q.shape
            p = LasadParams(B, 1, H, dk, v.shape[2], 0, 0, _dtype_code(q), 0, 1.0, 0,
                            _strides_decode(q), _strides_decode(k), _strides_decode(v), _strides_decode(o))
        if len(_params_cache) > 256:
            _params_cache.clear()
        _params_cache[key] = p
    p.grid_w = grid_w
    p.prefix_len = prefix_len
    p.t0 = t0
    p.scale = scale
    return p


def _check_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("all tensors must be CUDA tensors (there is no CPU path)")


def _strides3(t: torch.Tensor):
    """Element strides of (batch, token, head) for a [B,T,H,d] view with contiguous channels."""
    if t.dim() != 4 or (t.shape[3] > 1 and t.stride(3) != 1):
        raise ValueError("expected [B,T,H,d] with contiguous channels")
    return (ctypes.c_int64 * 3)(t.stride(0), t.stride(1), t.stride(2))


def _strides_decode(t: torch.Tensor):
    if t.dim() != 3 or (t.shape[2] > 1 and t.stride(2) != 1):
        raise ValueError("expected [B,H,d] with contiguous channels")
    return (ctypes.c_int64 * 3)(t.stride(0), 0, t.stride(1))


class Lasad:
    """A ``lasad_ctx`` bound to one CUDA device."""

    def __init__(self, device: int | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("LASAD needs a CUDA device: the operator has no CPU path")
        self._lib = load_library()
        self.device = torch.cuda.current_device() if device is None else int(device)
        h = ctypes.c_void_p()
        rc = self._lib.lasad_create(ctypes.byref(h), self.device)
        if rc != LASAD_OK:
            raise LasadError(rc, "lasad_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.lasad_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, option: int, value: int) -> None:
        rc = self._lib.lasad_set_option(self._h, option, value)
        if rc != LASAD_OK:
            raise LasadError(rc, "lasad_set_option")

    def reserve(self, units: int) -> None:
        """Pre-allocate the context's relay storage for prefill calls with B * H <= units."""
        rc = self._lib.lasad_reserve(self._h, int(units))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_reserve")

    @property
    def launch_count(self) -> int:
        return int(self._lib.lasad_launch_count(self._h))

    def device_status(self) -> int:
        out = ctypes.c_int(0)
        rc = self._lib.lasad_last_device_status(self._h, ctypes.byref(out))
        if rc != LASAD_OK:
            raise LasadError(rc, "lasad_last_device_status")
        return out.value

    def _raise(self, rc, where):
        detail = ""
        if rc == LASAD_ERR_CUDA:
            detail = f" [cudaError {self._lib.lasad_last_cuda_error(self._h)}]"
        raise LasadError(rc, where, detail)

    def lasad_forward(self, q, k, v, decay, grid_w, prefix_len=0, t0=0, scale=1.0,
                      state_in=None, o=None, state_out=None, want_state=True, stream=None):
        """Prefill over [B,T,H,d] tensors; returns (o, state_out).  Asynchronous on ``stream``."""
        _check_cuda(q, k, v, decay, state_in, o, state_out)
        B, T, H, dk = q.shape
        dv = v.shape[3]
        if o is None:
            o = torch.empty((B, T, H, dv), dtype=q.dtype, device=q.device)
        if state_out is None and want_state:
            state_out = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device)
        p = _params("prefill", q, k, v, o, grid_w, prefix_len, t0, scale)
        rc = self._lib.lasad_forward(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v),
                                     _ptr(decay), _ptr(state_in), _ptr(o), _ptr(state_out),
                                     _stream(q.device, stream))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_forward")
        return o, state_out

    def lasad_forward_host(self, q, k, v, decay, grid_w, o, prefix_len=0, t0=0, scale=1.0, state_in=None,
                           state_out=None, stream=None):
        """Prefill on HOST tensors (contiguous, ideally pinned): the library pipelines the copies
        with the kernels.  ``o`` (and ``state_out``) are host tensors that are complete once the
        stream has been synchronised.  Returns (o, state_out)."""
        for t in (q, k, v, decay, o, state_in, state_out):
            if t is not None and (t.is_cuda or not t.is_contiguous()):
                raise ValueError("lasad_forward_host takes contiguous host tensors")
        B, T, H, dk = q.shape
        dv = v.shape[3]
        p = LasadParams(B, T, H, dk, dv, grid_w, prefix_len, _dtype_code(q), t0, scale, 0,
                        _strides3(q), _strides3(k), _strides3(v), _strides3(o))
        dev = torch.device("cuda", self.device)
        st = torch.cuda.current_stream(dev).cuda_stream if stream is None else stream
        rc = self._lib.lasad_forward_host(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(decay),
                                          _ptr(state_in), _ptr(o), _ptr(state_out), ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_forward_host")
        return o, state_out

    def lasad_decode_step(self, q, k, v, decay, state, grid_w, prefix_len, t, scale=1.0, o=None,
                          stream=None):
        """One generation step for the token at absolute index ``t``; ``state`` is updated in
        place.  q, k, v are [B,H,d].  Returns o [B,H,dv]."""
        _check_cuda(q, k, v, decay, state, o)
        B, H, dk = q.shape
        dv = v.shape[2]
        if o is None:
            o = torch.empty((B, H, dv), dtype=q.dtype, device=q.device)
        if state.dtype != torch.float32 or not state.is_contiguous() or tuple(state.shape) != (B, H, dk, dv):
            raise ValueError("state must be contiguous float32 [B,H,dk,dv]")
        p = _params("decode", q, k, v, o, grid_w, prefix_len, t, scale)
        rc = self._lib.lasad_decode_step(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v),
                                         _ptr(decay), _ptr(state), _ptr(o), _stream(q.device, stream))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_decode_step")
        return o

    def lasad_forward_gated(self, q, k, v, gate, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None, o=None,
                            state_out=None, want_state=True, stream=None):
        """Prefill with a data-dependent gate [B,T,H,dk]; ``k=None`` ties the key to the gate
        (k = 1 - gate).  Returns (o, state_out)."""
        _check_cuda(q, k, v, gate, state_in, o, state_out)
        B, T, H, dk = q.shape
        dv = v.shape[3]
        if o is None:
            o = torch.empty((B, T, H, dv), dtype=q.dtype, device=q.device)
        if state_out is None and want_state:
            state_out = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q.device)
        if gate.dtype != q.dtype or tuple(gate.shape) != tuple(q.shape):
            raise ValueError("gate must have q's shape and dtype")
        if k is not None and tuple(k.stride()) != tuple(gate.stride()):
            raise ValueError("k and gate must share strides")
        p = LasadParams(B, T, H, dk, dv, grid_w, prefix_len, _dtype_code(q), t0, scale, 0,
                        _strides3(q), _strides3(gate), _strides3(v), _strides3(o))
        st = torch.cuda.current_stream(q.device).cuda_stream if stream is None else stream
        rc = self._lib.lasad_forward_gated(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate),
                                           _ptr(state_in), _ptr(o), _ptr(state_out), ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_forward_gated")
        return o, state_out

    def lasad_decode_step_gated(self, q, k, v, gate, state, grid_w, prefix_len, t, scale=1.0, o=None, stream=None):
        """One generation step with a data-dependent gate [B,H,dk]; ``state`` is updated in place."""
        _check_cuda(q, k, v, gate, state, o)
        B, H, dk = q.shape
        dv = v.shape[2]
        if o is None:
            o = torch.empty((B, H, dv), dtype=q.dtype, device=q.device)
        if state.dtype != torch.float32 or not state.is_contiguous() or tuple(state.shape) != (B, H, dk, dv):
            raise ValueError("state must be contiguous float32 [B,H,dk,dv]")
        if gate.dtype != q.dtype or tuple(gate.shape) != tuple(q.shape):
            raise ValueError("gate must have q's shape and dtype")
        if k is not None and tuple(k.stride()) != tuple(gate.stride()):
            raise ValueError("k and gate must share strides")
        p = LasadParams(B, 1, H, dk, dv, grid_w, prefix_len, _dtype_code(q), t, scale, 0,
                        _strides_decode(q), _strides_decode(gate), _strides_decode(v), _strides_decode(o))
        st = torch.cuda.current_stream(q.device).cuda_stream if stream is None else stream
        rc = self._lib.lasad_decode_step_gated(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(gate),
                                               _ptr(state), _ptr(o), ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_decode_step_gated")
        return o

    def lasad_decode_step_pos(self, q, k, v, decay, state, pos, prefix_len=0, grid_w=0, widths=None, scale=1.0,
                              o=None, stream=None):
        """One generation step with every sequence at its own position: ``pos`` int32 [B] on the
        device, ``widths`` int32 [B] or None (then ``grid_w`` for all).  Returns o [B,H,dv]."""
        _check_cuda(q, k, v, decay, state, o, pos, widths)
        B, H, dk = q.shape
        dv = v.shape[2]
        if o is None:
            o = torch.empty((B, H, dv), dtype=q.dtype, device=q.device)
        if state.dtype != torch.float32 or not state.is_contiguous() or tuple(state.shape) != (B, H, dk, dv):
            raise ValueError("state must be contiguous float32 [B,H,dk,dv]")
        for t in (pos, widths):
            if t is not None and (t.dtype != torch.int32 or not t.is_contiguous() or t.numel() != B):
                raise ValueError("pos / widths must be contiguous int32 [B]")
        p = LasadParams(B, 1, H, dk, dv, grid_w, prefix_len, _dtype_code(q), 0, scale, 0,
                        _strides_decode(q), _strides_decode(k), _strides_decode(v), _strides_decode(o))
        st = torch.cuda.current_stream(q.device).cuda_stream if stream is None else stream
        rc = self._lib.lasad_decode_step_pos(self._h, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(decay),
                                             _ptr(state), _ptr(o), _ptr(pos), _ptr(widths), ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_decode_step_pos")
        return o

    def lasad_forward_fused(self, q_pre, k, v, gate_pre, grid_w, prefix_len=0, t0=0, scale=1.0, state_in=None,
                            o=None, state_out=None, want_state=True, norm_eps=1e-6, stream=None):
        """Algorithm 1's loop body as one call: SiLU on ``q_pre``, Sigmoid on ``gate_pre``, ``k=None``
        ties the key to the gate, RMS norm on the output.  Returns (normalised o, state_out)."""
        _check_cuda(q_pre, k, v, gate_pre, state_in, o, state_out)
        B, T, H, dk = q_pre.shape
        dv = v.shape[3]
        if o is None:
            o = torch.empty((B, T, H, dv), dtype=q_pre.dtype, device=q_pre.device)
        if state_out is None and want_state:
            state_out = torch.empty((B, H, dk, dv), dtype=torch.float32, device=q_pre.device)
        if gate_pre.dtype != q_pre.dtype or tuple(gate_pre.shape) != tuple(q_pre.shape):
            raise ValueError("gate_pre must have q_pre's shape and dtype")
        if k is not None and tuple(k.stride()) != tuple(gate_pre.stride()):
            raise ValueError("k and gate_pre must share strides")
        p = LasadParams(B, T, H, dk, dv, grid_w, prefix_len, _dtype_code(q_pre), t0, scale, 0,
                        _strides3(q_pre), _strides3(gate_pre), _strides3(v), _strides3(o))
        st = torch.cuda.current_stream(q_pre.device).cuda_stream if stream is None else stream
        rc = self._lib.lasad_forward_fused(self._h, ctypes.byref(p), _ptr(q_pre), _ptr(k), _ptr(v), _ptr(gate_pre),
                                           _ptr(state_in), _ptr(o), _ptr(state_out), float(norm_eps),
                                           ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_forward_fused")
        return o, state_out

    def lasad_decode_step_fused(self, q_pre, k, v, gate_pre, state, grid_w, prefix_len, t, scale=1.0, o=None,
                                norm_eps=1e-6, stream=None):
        """One generation step of Algorithm 1's loop body (activations, state update, readout, norm);
        ``state`` is updated in place.  q_pre, gate_pre, v are [B,H,d]."""
        _check_cuda(q_pre, k, v, gate_pre, state, o)
        B, H, dk = q_pre.shape
        dv = v.shape[2]
        if o is None:
            o = torch.empty((B, H, dv), dtype=q_pre.dtype, device=q_pre.device)
        if state.dtype != torch.float32 or not state.is_contiguous() or tuple(state.shape) != (B, H, dk, dv):
            raise ValueError("state must be contiguous float32 [B,H,dk,dv]")
        if gate_pre.dtype != q_pre.dtype or tuple(gate_pre.shape) != tuple(q_pre.shape):
            raise ValueError("gate_pre must have q_pre's shape and dtype")
        if k is not None and tuple(k.stride()) != tuple(gate_pre.stride()):
            raise ValueError("k and gate_pre must share strides")
        p = LasadParams(B, 1, H, dk, dv, grid_w, prefix_len, _dtype_code(q_pre), t, scale, 0,
                        _strides_decode(q_pre), _strides_decode(gate_pre), _strides_decode(v), _strides_decode(o))
        st = torch.cuda.current_stream(q_pre.device).cuda_stream if stream is None else stream
        rc = self._lib.lasad_decode_step_fused(self._h, ctypes.byref(p), _ptr(q_pre), _ptr(k), _ptr(v),
                                               _ptr(gate_pre), _ptr(state), _ptr(o), float(norm_eps),
                                               ctypes.c_void_p(st))
        if rc != LASAD_OK:
            self._raise(rc, "lasad_decode_step_fused")
        return o


def lasad_forward_static(q, k, v, decay, grid_w, o, state_out=None, prefix_len=0, t0=0, scale=1.0,
                         state_in=None, device_status=None, stream=None):
    """``lasad_forward_static``: prefill on q's device with no context and no allocation.

    Every buffer, the output ``o`` included, is the caller's: this wrapper allocates nothing either.
    ``device_status`` is an optional int32 CUDA tensor of one element.  Raises on an error code."""
    _check_cuda(q, k, v, decay, state_in, o, state_out, device_status)
    B, T, H, dk = q.shape
    dv = v.shape[3]
    p = LasadParams(B, T, H, dk, dv, grid_w, prefix_len, _dtype_code(q), t0, scale, 0,
                    _strides3(q), _strides3(k), _strides3(v), _strides3(o))
    lib = load_library()
    with torch.cuda.device(q.device):
        st = torch.cuda.current_stream(q.device).cuda_stream if stream is None else stream
        rc = lib.lasad_forward_static(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(decay), _ptr(state_in),
                                      _ptr(o), _ptr(state_out), _ptr(device_status), ctypes.c_void_p(st))
    if rc != LASAD_OK:
        raise LasadError(rc, "lasad_forward_static")
    return o, state_out



_default = {}


def default_ctx(device: int | None = None) -> Lasad:
    dev = torch.cuda.current_device() if device is None else int(device)
    if dev not in _default:
        _default[dev] = Lasad(dev)
    return _default[dev]


def lasad_forward(q, k, v, decay, grid_w, **kw):
    """``lasad_forward`` on the default context of q's device."""
    return default_ctx(q.device.index).lasad_forward(q, k, v, decay, grid_w, **kw)


def lasad_decode_step(q, k, v, decay, state, grid_w, prefix_len, t, **kw):
    """``lasad_decode_step`` on the default context of q's device."""
    return default_ctx(q.device.index).lasad_decode_step(q, k, v, decay, state, grid_w, prefix_len, t, **kw)
