"""ctypes binding of librattn.so: argument marshalling only.

Every function has the name of the C entry point it calls (include/rattn.h) and does
nothing but turn torch tensors into device pointers, sizes and a stream handle.  There
is no fallback: if the library has not been built, loading it raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librattn.so")

RATTN_BF16, RATTN_F32 = 0, 1
MODE_RATTN, MODE_SWA_ONLY, MODE_FULL_CAUSAL = 0, 1, 2
FLAG_FORCE_GENERIC, FLAG_SAVE_RESIDUALS = 1, 2
PHI_SOFTMAX, PHI_RELU, PHI_IDENTITY = 0, 1, 2
LAYOUT_BHTD, LAYOUT_BTHD = 0, 1

EXPORTS = (
    "rattn_forward", "rattn_forward_ex", "rattn_backward", "rattn_backward_ex",
    "rattn_decode_step", "rattn_decode_step_ex", "rattn_workspace_bytes",
    "rattn_workspace_bytes_ex", "rattn_workspace_bytes_chunked",
    "rattn_read_status", "rattn_strerror", "rattn_last_cuda_error", "rattn_launch_count",
    "rattn_uses_tensor_path", "rattn_timing_enable", "rattn_timing_read",
    "rattn_forward_static", "rattn_static_status", "rattn_tune",
    "rattn_qk_prologue", "rattn_qk_prologue_backward", "rattn_qk_prologue_workspace_bytes", "rattn_qk_prologue_status", "rattn_decode_status", "rattn_forward_status",
)
TUNE_STATE_STRIDE, TUNE_OVERLAP, TUNE_UNIT_ORDER, TUNE_GRID, TUNE_DECODE_STAGES, TUNE_STATE_PROGRESS = 0, 1, 2, 3, 4, 5


class RattnParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("out", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("H_q", ctypes.c_int32), ("H_kv", ctypes.c_int32),
        ("T", ctypes.c_int32), ("d", ctypes.c_int32), ("w", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("mode", ctypes.c_int32),
        ("scale", ctypes.c_float), ("eps", ctypes.c_float),
        ("gamma_swa", ctypes.c_void_p), ("gamma_rla", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("state_out", ctypes.c_void_p), ("k_ring_out", ctypes.c_void_p),
        ("v_ring_out", ctypes.c_void_p),
        ("dout", ctypes.c_void_p), ("dq", ctypes.c_void_p), ("dk", ctypes.c_void_p),
        ("dv", ctypes.c_void_p), ("dgamma_swa", ctypes.c_void_p),
        ("dgamma_rla", ctypes.c_void_p),
        ("flags", ctypes.c_uint32), ("feature_map", ctypes.c_int32),
        ("state_in", ctypes.c_void_p), ("k_ring_in", ctypes.c_void_p), ("v_ring_in", ctypes.c_void_p),
        ("pos0", ctypes.c_int32), ("layout", ctypes.c_int32),
        ("seq_lens", ctypes.c_void_p), ("pos", ctypes.c_void_p),
    ]


class RattnQkParams(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("q_out", ctypes.c_void_p), ("k_out", ctypes.c_void_p),
        ("q_gain", ctypes.c_void_p), ("k_gain", ctypes.c_void_p),
        ("B", ctypes.c_int32), ("H_q", ctypes.c_int32), ("H_kv", ctypes.c_int32),
        ("T", ctypes.c_int32), ("d", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("eps", ctypes.c_float), ("theta", ctypes.c_float),
        ("pos0", ctypes.c_int32), ("layout", ctypes.c_int32), ("pos", ctypes.c_void_p),
    ]


class RattnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().rattn_strerror(code).decode()
        if code == -6:
            msg += f" [cudaError {lib().rattn_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2506_15545_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    L.rattn_forward.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
    L.rattn_forward.restype = ci
    L.rattn_forward_ex.argtypes = [ctypes.POINTER(RattnParams), vp]
    L.rattn_forward_ex.restype = ci
    L.rattn_backward.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, ci, ci, ci, ci, ci, ci,
                                 vp, vp, vp, vp]
    L.rattn_backward.restype = ci
    L.rattn_backward_ex.argtypes = [ctypes.POINTER(RattnParams), vp]
    L.rattn_backward_ex.restype = ci
    L.rattn_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, vp, vp]
    L.rattn_decode_step.restype = ci
    L.rattn_decode_step_ex.argtypes = [ctypes.POINTER(RattnParams), vp, vp, vp, ci, vp]
    L.rattn_decode_step_ex.restype = ci
    L.rattn_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci]
    L.rattn_workspace_bytes.restype = ctypes.c_size_t
    L.rattn_workspace_bytes_ex.argtypes = [ci, ci, ci, ci, ci, ci, ci, ci, ctypes.c_uint]
    L.rattn_workspace_bytes_ex.restype = ctypes.c_size_t
    L.rattn_workspace_bytes_chunked.argtypes = [ci, ci, ci, ci, ci, ci, ci, ctypes.c_uint]
    L.rattn_workspace_bytes_chunked.restype = ctypes.c_size_t
    L.rattn_read_status.argtypes = [vp, vp]
    L.rattn_read_status.restype = ci
    L.rattn_strerror.argtypes = [ci]
    L.rattn_strerror.restype = ctypes.c_char_p
    L.rattn_last_cuda_error.argtypes = []
    L.rattn_last_cuda_error.restype = ci
    L.rattn_launch_count.argtypes = []
    L.rattn_launch_count.restype = ctypes.c_uint64
    L.rattn_uses_tensor_path.argtypes = [ci, ci, ci, ci, ctypes.c_uint]
    L.rattn_uses_tensor_path.restype = ci
    L.rattn_forward_static.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci, ci, cf, vp, vp]
    L.rattn_forward_static.restype = ci
    L.rattn_static_status.argtypes = [vp]
    L.rattn_static_status.restype = ci
    L.rattn_tune.argtypes = [ci, ci]
    L.rattn_tune.restype = ci
    L.rattn_qk_prologue.argtypes = [ctypes.POINTER(RattnQkParams), vp]
    L.rattn_qk_prologue.restype = ci
    L.rattn_qk_prologue_backward.argtypes = [ctypes.POINTER(RattnQkParams), vp, vp, vp, vp, vp, vp, vp,
                                             ctypes.c_size_t, vp]
    L.rattn_qk_prologue_backward.restype = ci
    L.rattn_qk_prologue_workspace_bytes.argtypes = [ci, ci, ci, ci, ci]
    L.rattn_qk_prologue_workspace_bytes.restype = ctypes.c_size_t
    L.rattn_forward_status.argtypes = [vp]
    L.rattn_forward_status.restype = ci
    L.rattn_decode_status.argtypes = [vp]
    L.rattn_decode_status.restype = ci
    L.rattn_qk_prologue_status.argtypes = [vp]
    L.rattn_qk_prologue_status.restype = ci
    L.rattn_timing_enable.argtypes = [ci]
    L.rattn_timing_enable.restype = ci
    L.rattn_timing_read.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    L.rattn_timing_read.restype = ctypes.c_size_t
    _lib = L
    return L


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return RATTN_BF16
    if t.dtype == torch.float32:
        return RATTN_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _check(code: int, where: str):
    if code != 0:
        raise RattnError(code, where)


def _dense(*ts):
    for t in ts:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("tensors must be contiguous CUDA tensors")


def rattn_workspace_bytes(B, H_q, H_kv, T, d, w, dtype=RATTN_BF16) -> int:
    return int(lib().rattn_workspace_bytes(B, H_q, H_kv, T, d, w, dtype))


def rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, dtype=RATTN_BF16, mode=MODE_RATTN, flags=0) -> int:
    return int(lib().rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, dtype, mode, flags))


def rattn_workspace_bytes_chunked(B, H_q, H_kv, T, d, w, dtype=RATTN_BF16, flags=0) -> int:
    return int(lib().rattn_workspace_bytes_chunked(B, H_q, H_kv, T, d, w, dtype, flags))


def alloc_workspace_chunked(q, k, w, flags=0) -> torch.Tensor:
    """Workspace of a forward that resumes a sequence (pos0 > 0)."""
    B, H_q, T, d = q.shape
    n = rattn_workspace_bytes_chunked(B, H_q, k.shape[1], T, d, w, _dtype_code(q), flags)
    return torch.empty(n, dtype=torch.uint8, device=q.device)


def alloc_workspace(q, k, w, mode=None, flags=None, layout=LAYOUT_BHTD) -> torch.Tensor:
    """A uint8 device tensor for these shapes: exactly rattn_workspace_bytes_ex() bytes when
    mode and flags are given, else rattn_workspace_bytes() (enough for any mode and flags)."""
    if layout == LAYOUT_BTHD:
        B, T, H_q, d = q.shape
        H_kv = k.shape[2]
    else:
        B, H_q, T, d = q.shape
        H_kv = k.shape[1]
    if mode is None and flags is None:
        n = rattn_workspace_bytes(B, H_q, H_kv, T, d, w, _dtype_code(q))
    else:
        n = rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, _dtype_code(q), mode or 0, flags or 0)
    return torch.empty(n, dtype=torch.uint8, device=q.device)


def _params(q, k, v, out, w, scale, eps, gamma_swa, gamma_rla, mode, workspace, flags, phi=PHI_SOFTMAX,
            layout=LAYOUT_BHTD):
    p = RattnParams()
    p.feature_map = phi
    p.layout = layout
    p.q, p.k, p.v, p.out = q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr()
    if q.dim() == 4 and layout == LAYOUT_BTHD:
        p.B, p.T, p.H_q, p.d = q.shape
        p.H_kv = k.shape[2]
    elif q.dim() == 4:
        p.B, p.H_q, p.T, p.d = q.shape
        p.H_kv = k.shape[1]
    else:
        p.B, p.H_q, p.d = q.shape
        p.T = 1
        p.H_kv = k.shape[1]
    p.w = w
    p.dtype = _dtype_code(q)
    p.mode = mode
    p.scale, p.eps = scale, eps
    p.gamma_swa = None if gamma_swa is None else gamma_swa.data_ptr()
    p.gamma_rla = None if gamma_rla is None else gamma_rla.data_ptr()
    if workspace is not None:
        p.workspace = workspace.data_ptr()
        p.workspace_bytes = workspace.numel() * workspace.element_size()
    p.flags = flags
    return p


def rattn_forward(q, k, v, w, out=None, stream=None):
    """rattn_forward: bf16, scale 1, unit gains, eps 1e-6."""
    _dense(q, k, v, out)
    B, H_q, T, d = q.shape
    out = torch.empty_like(q) if out is None else out
    _check(lib().rattn_forward(_ptr(q), _ptr(k), _ptr(v), B, H_q, k.shape[1], T, d, w, _ptr(out),
                               _stream(stream)), "rattn_forward")
    return out


def rattn_forward_static(q, k, v, w, scale=1.0, out=None, stream=None):
    """rattn_forward_static: the forward that allocates nothing on the library side (its
    scratch is a fixed array inside the library).  `out` may be passed in so that the call
    allocates nothing on the Python side either."""
    _dense(q, k, v, out)
    B, H_q, T, d = q.shape
    out = torch.empty_like(q) if out is None else out
    _check(lib().rattn_forward_static(_ptr(q), _ptr(k), _ptr(v), B, H_q, k.shape[1], T, d, w, scale,
                                      _ptr(out), _stream(stream)), "rattn_forward_static")
    return out


def rattn_forward_ex(q, k, v, w, *, scale=1.0, eps=1e-6, gamma_swa=None, gamma_rla=None,
                     mode=MODE_RATTN, workspace=None, save_residuals=False, state_out=None,
                     k_ring_out=None, v_ring_out=None, out=None, flags=0, phi=PHI_SOFTMAX, state_in=None,
                     k_ring_in=None, v_ring_in=None, pos0=0, seq_lens=None, layout=LAYOUT_BHTD, stream=None):
    """layout=LAYOUT_BTHD: q, out are [B, T, H_q, d] and k, v [B, T, H_kv, d]."""
    _dense(q, k, v, out, gamma_swa, gamma_rla, workspace, state_out, k_ring_out, v_ring_out, state_in,
           k_ring_in, v_ring_in, seq_lens)
    out = torch.empty_like(q) if out is None else out
    if save_residuals:
        flags |= FLAG_SAVE_RESIDUALS
    p = _params(q, k, v, out, w, scale, eps, gamma_swa, gamma_rla, mode, workspace, flags, phi, layout)
    p.state_out = None if state_out is None else state_out.data_ptr()
    p.k_ring_out = None if k_ring_out is None else k_ring_out.data_ptr()
    p.v_ring_out = None if v_ring_out is None else v_ring_out.data_ptr()
    p.state_in = None if state_in is None else state_in.data_ptr()
    p.k_ring_in = None if k_ring_in is None else k_ring_in.data_ptr()
    p.v_ring_in = None if v_ring_in is None else v_ring_in.data_ptr()
    p.pos0 = pos0
    p.seq_lens = None if seq_lens is None else seq_lens.data_ptr()
    _check(lib().rattn_forward_ex(ctypes.byref(p), _stream(stream)), "rattn_forward_ex")
    return out


def rattn_backward(q, k, v, dout, workspace, w, dq=None, dk=None, dv=None, stream=None):
    """rattn_backward: bf16, scale 1, unit gains, eps 1e-6."""
    _dense(q, k, v, dout, workspace, dq, dk, dv)
    B, H_q, T, d = q.shape
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    _check(lib().rattn_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(workspace),
                                workspace.numel(), B, H_q, k.shape[1], T, d, w, _ptr(dq),
                                _ptr(dk), _ptr(dv), _stream(stream)), "rattn_backward")
    return dq, dk, dv


def rattn_backward_ex(q, k, v, dout, w, workspace, *, scale=1.0, eps=1e-6, gamma_swa=None,
                      gamma_rla=None, mode=MODE_RATTN, dq=None, dk=None, dv=None,
                      dgamma_swa=None, dgamma_rla=None, flags=0, phi=PHI_SOFTMAX, layout=LAYOUT_BHTD, stream=None):
    _dense(q, k, v, dout, workspace, gamma_swa, gamma_rla, dq, dk, dv, dgamma_swa, dgamma_rla)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    p = _params(q, k, v, dq, w, scale, eps, gamma_swa, gamma_rla, mode, workspace, flags, phi, layout)
    p.dout, p.dq, p.dk, p.dv = dout.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr()
    p.dgamma_swa = None if dgamma_swa is None else dgamma_swa.data_ptr()
    p.dgamma_rla = None if dgamma_rla is None else dgamma_rla.data_ptr()
    _check(lib().rattn_backward_ex(ctypes.byref(p), _stream(stream)), "rattn_backward_ex")
    return dq, dk, dv


def rattn_decode_step(q, k, v, k_ring, v_ring, state, pos, out=None, stream=None):
    """rattn_decode_step: bf16, scale 1, unit gains, eps 1e-6.  Ring and state in place."""
    _dense(q, k, v, k_ring, v_ring, state, out)
    B, H_q, d = q.shape
    out = torch.empty_like(q) if out is None else out
    _check(lib().rattn_decode_step(_ptr(q), _ptr(k), _ptr(v), _ptr(k_ring), _ptr(v_ring),
                                   _ptr(state), pos, B, H_q, k.shape[1], d, k_ring.shape[2],
                                   _ptr(out), _stream(stream)), "rattn_decode_step")
    return out


def rattn_decode_step_ex(q, k, v, k_ring, v_ring, state, pos, *, scale=1.0, eps=1e-6,
                         gamma_swa=None, gamma_rla=None, out=None, phi=PHI_SOFTMAX, pos_dev=None, flags=0,
                         stream=None):
    """pos_dev: optional int32 device tensor [B], one position per batch entry (then `pos` is ignored)."""
    _dense(q, k, v, k_ring, v_ring, state, out, gamma_swa, gamma_rla, pos_dev)
    out = torch.empty_like(q) if out is None else out
    p = _params(q, k, v, out, k_ring.shape[2], scale, eps, gamma_swa, gamma_rla, MODE_RATTN,
                None, flags, phi)
    p.pos = None if pos_dev is None else pos_dev.data_ptr()
    _check(lib().rattn_decode_step_ex(ctypes.byref(p), _ptr(k_ring), _ptr(v_ring), _ptr(state),
                                      pos, _stream(stream)), "rattn_decode_step_ex")
    return out


def rattn_read_status(workspace, stream=None) -> int:
    return int(lib().rattn_read_status(_ptr(workspace), _stream(stream)))


def rattn_static_status(stream=None) -> int:
    """Status word of rattn_forward_static's last call on the current device."""
    return int(lib().rattn_static_status(_stream(stream)))


def rattn_tune(knob: int, value: int) -> int:
    """Sets a tuning parameter of the tensor-core forward; returns the previous value."""
    r = int(lib().rattn_tune(knob, value))
    _check(r if r < 0 else 0, "rattn_tune")
    return r


def rattn_launch_count() -> int:
    return int(lib().rattn_launch_count())


def rattn_uses_tensor_path(d, w, dtype=RATTN_BF16, mode=MODE_RATTN, flags=0) -> bool:
    return bool(lib().rattn_uses_tensor_path(d, w, dtype, mode, flags))


def rattn_timing_enable(on: bool) -> None:
    lib().rattn_timing_enable(1 if on else 0)


def rattn_timing_read() -> dict:
    """{kernel name: (launches, total milliseconds)} since timing was enabled."""
    buf = ctypes.create_string_buffer(1 << 16)
    lib().rattn_timing_read(buf, len(buf))
    out = {}
    for line in buf.value.decode().splitlines():
        name, n, ms = line.rsplit(" ", 2)
        out[name] = (int(n), float(ms))
    return out


def _qk_params(q, k, q_out, k_out, q_gain, k_gain, theta, eps, pos0, pos, layout=LAYOUT_BHTD):
    p = RattnQkParams()
    _dense(q, k, q_out, k_out, q_gain, k_gain, pos)
    p.q, p.q_out = q.data_ptr(), None if q_out is None else q_out.data_ptr()
    hd = 2 if layout == LAYOUT_BTHD else 1              # which dimension counts the heads
    p.layout = layout
    p.B, p.d = q.shape[0], q.shape[3]
    p.H_q, p.T = q.shape[hd], q.shape[3 - hd]
    if k is not None:
        p.k, p.k_out = k.data_ptr(), None if k_out is None else k_out.data_ptr()
        p.H_kv = k.shape[hd]
    p.q_gain = None if q_gain is None else q_gain.data_ptr()
    p.k_gain = None if k_gain is None else k_gain.data_ptr()
    p.dtype = _dtype_code(q)
    p.eps, p.theta, p.pos0 = eps, 0.0 if theta is None else theta, pos0
    p.pos = None if pos is None else pos.data_ptr()
    return p


def rattn_qk_prologue_workspace_bytes(B, H_q, H_kv, T, d) -> int:
    return int(lib().rattn_qk_prologue_workspace_bytes(B, H_q, H_kv, T, d))


def rattn_forward_status(stream=None) -> int:
    """RATTN_ERR_TIMEOUT if a bounded wait expired in a rattn_forward call since the last query."""
    return int(lib().rattn_forward_status(_stream(stream)))


def rattn_decode_status(stream=None) -> int:
    return int(lib().rattn_decode_status(_stream(stream)))


def rattn_qk_prologue_status(stream=None) -> int:
    return int(lib().rattn_qk_prologue_status(_stream(stream)))


def rattn_qk_prologue(q, k, *, q_gain=None, k_gain=None, theta=5.0e5, eps=1e-6, pos0=0, pos=None,
                      inplace=False, layout=LAYOUT_BHTD, stream=None):
    """rattn_qk_prologue: qk-norm then rotary embedding of q [B,H_q,T,d] and k [B,H_kv,T,d] (k may be
    None).  theta None or <= 0: no rotation.  Returns (q_out, k_out); the inputs themselves if inplace."""
    q_out = q if inplace else torch.empty_like(q)
    k_out = None if k is None else (k if inplace else torch.empty_like(k))
    p = _qk_params(q, k, q_out, k_out, q_gain, k_gain, theta, eps, pos0, pos, layout)
    _check(lib().rattn_qk_prologue(ctypes.byref(p), _stream(stream)), "rattn_qk_prologue")
    return q_out, k_out


def rattn_qk_prologue_backward(q, k, dq_out, dk_out, *, q_gain=None, k_gain=None, theta=5.0e5, eps=1e-6,
                               pos0=0, pos=None, gain_grads=True, workspace=None, layout=LAYOUT_BHTD, stream=None):
    """rattn_qk_prologue_backward: gradients with respect to q, k (inputs as they were before the
    forward pass) and, with gain_grads, to the two gains.  Returns (dq, dk, dq_gain, dk_gain)."""
    _dense(dq_out, dk_out)
    dq = torch.empty_like(q)
    dk = None if k is None else torch.empty_like(k)
    dqg = dkg = None
    p = _qk_params(q, k, None, None, q_gain, k_gain, theta, eps, pos0, pos, layout)
    if gain_grads:
        dqg = torch.empty(q.shape[-1], dtype=torch.float32, device=q.device)
        dkg = None if k is None else torch.empty(q.shape[-1], dtype=torch.float32, device=q.device)
        if workspace is None:
            n = rattn_qk_prologue_workspace_bytes(p.B, p.H_q, p.H_kv, p.T, p.d)
            workspace = torch.empty(n, dtype=torch.uint8, device=q.device)
    nbytes = 0 if workspace is None else workspace.numel()
    _check(lib().rattn_qk_prologue_backward(ctypes.byref(p), _ptr(dq_out), _ptr(dk_out), _ptr(dq), _ptr(dk),
                                            _ptr(dqg), _ptr(dkg), _ptr(workspace), nbytes, _stream(stream)),
           "rattn_qk_prologue_backward")
    return dq, dk, dqg, dkg
