"""Thin ctypes binding of the C ABI in include/la.h.

Argument marshalling only: torch supplies device memory and the current
stream; every step of the computation runs in the CUDA library.  There is no
CPU fallback -- a missing or unloadable library raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libla.so")

LA_F32, LA_BF16 = 0, 1
LA_PHI_ELU1, LA_PHI_IDENTITY = 0, 1
LA_OP_LINEAR_FORWARD, LA_OP_LINEAR_BACKWARD, LA_OP_CAUSAL_FORWARD, LA_OP_CAUSAL_BACKWARD = 0, 1, 2, 3
LA_OP_CAUSAL_SAVED = 4
LA_OP_LINEAR_VARLEN_FORWARD, LA_OP_LINEAR_VARLEN_BACKWARD = 5, 6
LA_OP_LINEAR_SAVED = 7
LA_OP_DECODE_LAYER = 8
LA_OP_CAUSAL_VARLEN_FORWARD, LA_OP_CAUSAL_VARLEN_BACKWARD = 9, 10
_PHI = {"elu1": LA_PHI_ELU1, "identity": LA_PHI_IDENTITY}

EXPORTS = [
    "la_feature_map", "la_feature_map_poly2", "la_feature_map_poly2_backward", "la_feature_map_rff",
    "la_feature_map_rff_backward",
    "la_linear_attention", "la_linear_attention_noalloc", "la_linear_attention_backward",
    "la_linear_attention_varlen", "la_linear_attention_varlen_backward",
    "la_linear_attention_keep", "la_linear_attention_backward_kept",
    "la_causal_forward", "la_causal_forward_from", "la_causal_backward_from",
    "la_causal_backward", "la_recurrent_step", "la_recurrent_steps", "la_workspace_bytes", "la_status_string",
    "la_last_error", "la_last_device_status", "la_kernel_launches", "la_profile_enable", "la_profile_read",
    "la_profile_kernel_name", "la_version", "la_causal_plan", "la_plan_override",
    "la_decode_layer_step", "la_causal_forward_varlen", "la_causal_backward_varlen",
]


class la_problem(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int64), ("H", ctypes.c_int64), ("N", ctypes.c_int64),
                ("D", ctypes.c_int64), ("M", ctypes.c_int64), ("dtype", ctypes.c_int32),
                ("phi", ctypes.c_int32), ("eps", ctypes.c_float)]


class LaError(RuntimeError):
    def __init__(self, status: int, name: str, message: str):
        super().__init__(f"{name} ({status}): {message}")
        self.status, self.name = status, name


_lib = None


def lib() -> ctypes.CDLL:
    """Load libla.so (built in-tree by ``paper_2006_16236_b200.build``); raise if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2006_16236_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(la_problem)
        L.la_feature_map.argtypes = [vp, vp, i64, i32, i32, vp]
        L.la_feature_map_poly2.argtypes = [vp, vp, i64, i64, i64, i32, vp]
        L.la_feature_map_poly2_backward.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp]
        L.la_feature_map_rff.argtypes = [vp, vp, vp, i64, i64, i64, i32, vp]
        L.la_feature_map_rff_backward.argtypes = [vp, vp, vp, vp, i64, i64, i64, i32, vp]
        L.la_linear_attention.argtypes = [pp] + [vp] * 7 + [vp, sz, vp]
        L.la_linear_attention_noalloc.argtypes = [pp] + [vp] * 7 + [vp]
        L.la_linear_attention_backward.argtypes = [pp] + [vp] * 9 + [vp, sz, vp]
        L.la_linear_attention_varlen.argtypes = [pp] + [vp] * 8 + [vp, sz, vp]
        L.la_linear_attention_varlen_backward.argtypes = [pp] + [vp] * 10 + [vp, sz, vp]
        L.la_linear_attention_keep.argtypes = [pp] + [vp] * 8 + [vp, sz, vp, sz, vp]
        L.la_linear_attention_backward_kept.argtypes = [pp] + [vp] * 4 + [vp, sz] + [vp] * 6 + [vp, sz, vp]
        L.la_causal_forward.argtypes = [pp] + [vp] * 7 + [vp, sz] + [vp, sz, vp]
        L.la_causal_forward_from.argtypes = [pp] + [vp] * 9 + [vp, sz] + [vp, sz, vp]
        L.la_causal_backward_from.argtypes = [pp] + [vp] * 10 + [vp, sz] + [vp] * 5 + [vp, sz, vp]
        L.la_causal_backward.argtypes = [pp] + [vp] * 6 + [vp, sz] + [vp] * 3 + [vp, sz, vp]
        L.la_causal_forward_varlen.argtypes = [pp] + [vp] * 10 + [vp, sz, vp, sz, vp]
        L.la_causal_backward_varlen.argtypes = [pp] + [vp] * 11 + [vp, sz] + [vp] * 5 + [vp, sz, vp]
        L.la_recurrent_step.argtypes = [pp] + [vp] * 6 + [vp]
        L.la_recurrent_steps.argtypes = [pp] + [vp] * 6 + [vp]
        L.la_decode_layer_step.argtypes = [pp] + [vp] * 6 + [vp, sz, vp]
        L.la_workspace_bytes.argtypes = [pp, i32]
        L.la_workspace_bytes.restype = sz
        L.la_status_string.argtypes = [ctypes.c_int]
        L.la_status_string.restype = ctypes.c_char_p
        L.la_last_error.restype = ctypes.c_char_p
        L.la_last_device_status.argtypes = [vp]
        L.la_version.restype = ctypes.c_char_p
        L.la_kernel_launches.restype = ctypes.c_longlong
        L.la_causal_plan.argtypes = [pp, ctypes.POINTER(ctypes.c_int32), ctypes.c_int]
        L.la_profile_enable.argtypes = [ctypes.c_int]
        L.la_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int)]
        L.la_profile_kernel_name.argtypes = [ctypes.c_int]
        L.la_profile_kernel_name.restype = ctypes.c_char_p
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        L = lib()
        raise LaError(rc, L.la_status_string(rc).decode(), L.la_last_error().decode())


def _call(dev, fn, *args) -> None:
    """One library call with `dev` current: the library launches on, and keeps its per-device state for,
    the current device, which need not be the one the tensors live on."""
    if dev.index == torch.cuda.current_device():
        _check(fn(*args))
        return
    with torch.cuda.device(dev):
        _check(fn(*args))


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LA_F32
    if t.dtype == torch.bfloat16:
        return LA_BF16
    raise TypeError(f"unsupported dtype {t.dtype}: use float32 or bfloat16")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _dev(*ts):
    """All tensors given (None: not given) must be contiguous and live on one CUDA device; returns it."""
    dev = None
    for t in ts:
        if t is None:
            continue
        if not t.is_cuda:
            raise ValueError("tensors must live on a CUDA device")
        if not t.is_contiguous():
            raise ValueError("tensors must be contiguous")
        if dev is None:
            dev = t.device
        elif t.device != dev:
            raise ValueError(f"all tensors of a call must live on one device (got {dev} and {t.device})")
    return dev


_KINDS = {
    # kind -> (shape as a function of the problem, dtype: None = the I/O type of Q)
    "qk": (lambda p: (p.B, p.H, p.N, p.D), None),
    "v": (lambda p: (p.B, p.H, p.N, p.M), None),
    "row": (lambda p: (p.B, p.H, p.N), torch.float32),
    "S": (lambda p: (p.B, p.H, p.D, p.M), torch.float32),
    "Z": (lambda p: (p.B, p.H, p.D), torch.float32),
    "q1": (lambda p: (p.B, p.H, p.D), None),
    "v1": (lambda p: (p.B, p.H, p.M), None),
}


def _expect(p: la_problem, io_dtype, **named):
    """Shape and dtype of every tensor handed to the library, checked before any pointer is taken: the kernels
    trust the problem descriptor, so a short or mistyped tensor would be read or written past its end.
    named: name=(tensor or None, kind); see _KINDS."""
    for name, (t, kind) in named.items():
        if t is None:
            continue
        shape_of, dtype = _KINDS[kind]
        want_shape, want_dtype = tuple(shape_of(p)), (io_dtype if dtype is None else dtype)
        if tuple(t.shape) != want_shape or t.dtype != want_dtype:
            raise ValueError(f"{name} must have shape {list(want_shape)} and dtype {want_dtype} "
                             f"(got {list(t.shape)}, {t.dtype})")


def _buffer(name, t):
    if t is not None and (t.dtype != torch.uint8 or t.dim() != 1):
        raise ValueError(f"{name} must be a 1-D uint8 tensor (got {list(t.shape)}, {t.dtype})")


def make_problem(B, H, N, D, M, dtype_code, phi="elu1", eps=0.0) -> la_problem:
    return la_problem(B, H, N, D, M, dtype_code, _PHI[phi] if isinstance(phi, str) else int(phi), float(eps))


def _problem_of(Q, V, phi, eps) -> la_problem:
    if Q.dim() != 4 or V.dim() != 4:
        raise ValueError("expected Q,K [B,H,N,D] and V [B,H,N,M]")
    B, H, N, D = Q.shape
    return make_problem(B, H, N, D, V.shape[3], _dtype_code(Q), phi, eps)


_ws_cache = {}


def workspace(p: la_problem, op: int, device) -> torch.Tensor | None:
    """A cached scratch tensor of la_workspace_bytes(p, op) bytes on `device` (None if 0)."""
    need = lib().la_workspace_bytes(ctypes.byref(p), op)
    if need == 0:
        return None
    key = (str(device), op)
    buf = _ws_cache.get(key)
    if buf is None or buf.numel() < need:
        buf = torch.empty(need, dtype=torch.uint8, device=device)
        _ws_cache[key] = buf
    return buf


def la_workspace_bytes(p: la_problem, op: int) -> int:
    return lib().la_workspace_bytes(ctypes.byref(p), op)


def la_kernel_launches() -> int:
    return int(lib().la_kernel_launches())


def la_causal_plan(p: la_problem):
    """How the tensor-core causal kernels cut the sequences of p: a dict of plain lists, or None when p runs
    the general kernels.  Host only."""
    n = lib().la_causal_plan(ctypes.byref(p), None, 0)
    if n < 0:
        _check(n)
    if n == 0:
        return None
    buf = (ctypes.c_int32 * n)()
    got = lib().la_causal_plan(ctypes.byref(p), buf, n)
    if got != n:
        raise RuntimeError("la_causal_plan changed its size between two calls")
    v = list(buf)
    pieces, parts = v[0], v[1]
    o = 2
    out = {"pieces": pieces, "parts": parts}
    out["piece_begin"] = v[o:o + pieces + 1]; o += pieces + 1
    out["piece_first_part"] = v[o:o + pieces + 1]; o += pieces + 1
    out["part_begin"] = v[o:o + parts + 1]; o += parts + 1
    out["launch_order"] = v[o:o + pieces]
    return out


def la_plan_override(causal_pieces: int = -1, causal_short: int = -1, linear_splits: int = -1) -> None:
    """Process-wide overrides of the automatic piece / split plans (A/B checks and tests); no arguments: automatic."""
    _check(lib().la_plan_override(int(causal_pieces), int(causal_short), int(linear_splits)))


def la_profile_enable(on: bool) -> None:
    _check(lib().la_profile_enable(int(on)))


def la_profile_read() -> dict:
    """{kernel name: (mean ms per launch, launches)} for every kernel recorded since la_profile_enable(True)."""
    out = {}
    for k in range(8):
        ms, n = ctypes.c_double(), ctypes.c_int()
        _check(lib().la_profile_read(k, ctypes.byref(ms), ctypes.byref(n)))
        if n.value:
            out[lib().la_profile_kernel_name(k).decode()] = (ms.value, n.value)
    return out


def la_version() -> str:
    return lib().la_version().decode()


def la_last_device_status(device=None) -> None:
    """Synchronise the current stream; raise LaError if a kernel gave up on a bounded wait."""
    with torch.cuda.device(torch.cuda.current_device() if device is None else device):
        _check(lib().la_last_device_status(_stream(device)))


def la_feature_map(x: torch.Tensor, deriv: bool = False, out: torch.Tensor | None = None) -> torch.Tensor:
    if out is not None and (out.shape != x.shape or out.dtype != x.dtype):
        raise ValueError(f"out must have shape {list(x.shape)} and dtype {x.dtype}")
    dev = _dev(x, out)
    y = torch.empty_like(x) if out is None else out
    _call(dev, lib().la_feature_map, _ptr(x), _ptr(y), x.numel(), _dtype_code(x), int(deriv), _stream(dev))
    return y


def poly2_columns(D: int) -> int:
    """Feature columns the degree-2 polynomial map of a D-vector is padded to: D*D rounded up to a multiple of 8."""
    return (D * D + 7) // 8 * 8


def la_feature_map_poly2(x: torch.Tensor, C: int | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    """Degree-2 polynomial feature map along the last axis: [..., D] -> [..., C] (C defaults to poly2_columns(D));
    feed the result to the attention calls with phi="identity"."""
    D = x.shape[-1]
    C = poly2_columns(D) if C is None else C
    if out is not None and (tuple(out.shape) != tuple(x.shape[:-1]) + (C,) or out.dtype != x.dtype):
        raise ValueError(f"out must have shape {list(x.shape[:-1]) + [C]} and dtype {x.dtype}")
    dev = _dev(x, out)
    y = torch.empty(x.shape[:-1] + (C,), dtype=x.dtype, device=x.device) if out is None else out
    _call(dev, lib().la_feature_map_poly2, _ptr(x), _ptr(y), x.numel() // max(D, 1), D, C, _dtype_code(x), _stream(dev))
    return y


def la_feature_map_poly2_backward(x: torch.Tensor, dy: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """Gradient of la_feature_map_poly2 with respect to x for an upstream gradient dy [..., C]."""
    D, C = x.shape[-1], dy.shape[-1]
    if dy.shape[:-1] != x.shape[:-1] or dy.dtype != x.dtype:
        raise ValueError(f"dy must have shape {list(x.shape[:-1])} + [C] and dtype {x.dtype}")
    if out is not None and (out.shape != x.shape or out.dtype != x.dtype):
        raise ValueError(f"out must have shape {list(x.shape)} and dtype {x.dtype}")
    dev = _dev(x, dy, out)
    dx = torch.empty_like(x) if out is None else out
    _call(dev, lib().la_feature_map_poly2_backward, _ptr(x), _ptr(dy), _ptr(dx), x.numel() // max(D, 1), D, C,
                                               _dtype_code(x), _stream(dev))
    return dx


def la_feature_map_rff(x: torch.Tensor, W: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """Random Fourier features along the last axis: x [..., D], frequencies W [C/2, D] -> [..., C] =
    sqrt(2/C) [cos(x W^T), sin(x W^T)] (bf16); feed the result to the attention calls with phi="identity"."""
    D = x.shape[-1]
    if W.dim() != 2 or W.shape[1] != D or W.dtype != x.dtype:
        raise ValueError(f"W must have shape [C/2, {D}] and dtype {x.dtype} (got {list(W.shape)}, {W.dtype})")
    C = 2 * W.shape[0]
    if out is not None and (tuple(out.shape) != tuple(x.shape[:-1]) + (C,) or out.dtype != x.dtype):
        raise ValueError(f"out must have shape {list(x.shape[:-1]) + [C]} and dtype {x.dtype}")
    dev = _dev(x, W, out)
    y = torch.empty(x.shape[:-1] + (C,), dtype=x.dtype, device=x.device) if out is None else out
    _call(dev, lib().la_feature_map_rff, _ptr(x), _ptr(W), _ptr(y), x.numel() // max(D, 1), D, C, _dtype_code(x), _stream(dev))
    return y


def la_feature_map_rff_backward(x: torch.Tensor, W: torch.Tensor, dy: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """Gradient of la_feature_map_rff with respect to x for an upstream gradient dy [..., C] (W is a constant)."""
    D = x.shape[-1]
    if W.dim() != 2 or W.shape[1] != D or W.dtype != x.dtype:
        raise ValueError(f"W must have shape [C/2, {D}] and dtype {x.dtype} (got {list(W.shape)}, {W.dtype})")
    C = 2 * W.shape[0]
    if tuple(dy.shape) != tuple(x.shape[:-1]) + (C,) or dy.dtype != x.dtype:
        raise ValueError(f"dy must have shape {list(x.shape[:-1]) + [C]} and dtype {x.dtype}")
    if out is not None and (out.shape != x.shape or out.dtype != x.dtype):
        raise ValueError(f"out must have shape {list(x.shape)} and dtype {x.dtype}")
    dev = _dev(x, W, dy, out)
    dx = torch.empty_like(x) if out is None else out
    _call(dev, lib().la_feature_map_rff_backward, _ptr(x), _ptr(W), _ptr(dy), _ptr(dx), x.numel() // max(D, 1), D, C,
          _dtype_code(x), _stream(dev))
    return dx


def linear_saved_buffer(Q, V, phi="elu1", eps=0.0):
    """A buffer for what la_linear_attention() keeps for la_linear_attention_backward() (per-split sums over the keys)."""
    p = _problem_of(Q, V, phi, eps)
    need = lib().la_workspace_bytes(ctypes.byref(p), LA_OP_LINEAR_SAVED)
    return None if need == 0 else torch.empty(need, dtype=torch.uint8, device=Q.device)


def la_linear_attention(Q, K, V, phi="elu1", eps=0.0, O=None, den=None, KV=None, Zs=None, ws=None, saved=None,
                        lengths=None):
    """Non-causal form.  Returns O; pass preallocated den / KV / Zs tensors to receive them, and a
    linear_saved_buffer() to keep the sums over the keys for the backward pass (la_linear_attention_keep;
    lengths: optional [B] int32 device tensor of a right-padded ragged batch)."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), O=(O, "v"), den=(den, "row"), KV=(KV, "S"), Zs=(Zs, "Z"))
    _buffer("saved", saved), _buffer("ws", ws)
    if lengths is not None:
        _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, O, den, KV, Zs, saved, lengths, ws)
    O = torch.empty_like(V) if O is None else O
    if saved is not None:
        _call(dev, lib().la_linear_attention_keep, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(O), _ptr(den),
                                              _ptr(KV), _ptr(Zs), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws),
                                              _stream(dev))
        return O
    if lengths is not None:
        return la_linear_attention_varlen(Q, K, V, lengths, phi, eps, O, den, KV, Zs, ws)
    ws = workspace(p, LA_OP_LINEAR_FORWARD, dev) if ws is None else ws
    _call(dev, lib().la_linear_attention, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(den), _ptr(KV),
                                     _ptr(Zs), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                     _stream(dev))
    return O


def la_linear_attention_noalloc(Q, K, V, phi="elu1", eps=0.0, O=None, den=None, KV=None, Zs=None):
    """Non-causal forward through the entry point that uses the library's built-in scratch array.

    For callers that may not allocate device memory around the call; here only the output
    tensor is created when `O` is not passed in.  Raises LaError (LA_ERR_WORKSPACE) when the
    problem needs more scratch than the array holds."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), O=(O, "v"), den=(den, "row"), KV=(KV, "S"), Zs=(Zs, "Z"))
    dev = _dev(Q, K, V, O, den, KV, Zs)
    O = torch.empty_like(V) if O is None else O
    _call(dev, lib().la_linear_attention_noalloc, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(den),
                                             _ptr(KV), _ptr(Zs), _stream(dev))
    return O


def la_linear_attention_backward(Q, K, V, G, phi="elu1", eps=0.0, O=None, den=None,
                                 dQ=None, dK=None, dV=None, ws=None, saved=None, lengths=None):
    """Gradients of the non-causal form.  saved: what la_linear_attention(..., saved=...) kept for the same
    problem (la_linear_attention_backward_kept); lengths as there.  Returns (dQ, dK, dV)."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), G=(G, "v"), O=(O, "v"), den=(den, "row"),
            dQ=(dQ, "qk"), dK=(dK, "qk"), dV=(dV, "v"))
    _buffer("saved", saved), _buffer("ws", ws)
    if lengths is not None:
        _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, G, O, den, dQ, dK, dV, saved, lengths, ws)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    if saved is None and lengths is not None:
        return la_linear_attention_varlen_backward(Q, K, V, G, lengths, phi, eps, O, den, dQ, dK, dV, ws)
    ws = workspace(p, LA_OP_LINEAR_BACKWARD, dev) if ws is None else ws
    if saved is not None:
        _call(dev, lib().la_linear_attention_backward_kept, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(saved), _nbytes(saved), _ptr(O), _ptr(den),
            _ptr(G), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws), _nbytes(ws), _stream(dev))
        return dQ, dK, dV
    _call(dev, lib().la_linear_attention_backward, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(den), _ptr(G), _ptr(dQ), _ptr(dK), _ptr(dV),
        _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(), _stream(dev))
    return dQ, dK, dV


def _nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def saved_buffer(Q, V, phi="elu1", eps=0.0):
    """A buffer for what la_causal_forward() keeps for la_causal_backward() (None if the problem needs none)."""
    p = _problem_of(Q, V, phi, eps)
    need = lib().la_workspace_bytes(ctypes.byref(p), LA_OP_CAUSAL_SAVED)
    return None if need == 0 else torch.empty(need, dtype=torch.uint8, device=Q.device)


def la_causal_forward(Q, K, V, phi="elu1", eps=0.0, O=None, den=None, S_out=None, Z_out=None, saved=None, ws=None,
                      S_in=None, Z_in=None, lengths=None):
    """Causal form.  Returns O; pass preallocated den / S_out / Z_out tensors to receive them, and a
    saved_buffer() to keep phi(Q), phi(K) for the backward pass.  S_in / Z_in (fp32 [B,H,D,M] / [B,H,D]):
    the state the sequence continues from (la_causal_forward_from)."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), O=(O, "v"), den=(den, "row"), S_out=(S_out, "S"),
            Z_out=(Z_out, "Z"), S_in=(S_in, "S"), Z_in=(Z_in, "Z"))
    _buffer("saved", saved), _buffer("ws", ws)
    if lengths is not None:
        _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, O, den, S_out, Z_out, saved, S_in, Z_in, ws, lengths)
    O = torch.empty_like(V) if O is None else O
    if lengths is not None:             # la_causal_forward_varlen: right-padded ragged batch
        ws = workspace(p, LA_OP_CAUSAL_VARLEN_FORWARD, dev) if ws is None else ws
        _call(dev, lib().la_causal_forward_varlen, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(S_in),
              _ptr(Z_in), _ptr(O), _ptr(den), _ptr(S_out), _ptr(Z_out), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws),
              _stream(dev))
        return O
    ws = workspace(p, LA_OP_CAUSAL_FORWARD, dev) if ws is None else ws
    if S_in is None and Z_in is None:
        _call(dev, lib().la_causal_forward, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(den), _ptr(S_out),
                                       _ptr(Z_out), _ptr(saved), _nbytes(saved), _ptr(ws), _nbytes(ws), _stream(dev))
    else:
        _call(dev, lib().la_causal_forward_from, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(S_in), _ptr(Z_in), _ptr(O),
                                            _ptr(den), _ptr(S_out), _ptr(Z_out), _ptr(saved), _nbytes(saved), _ptr(ws),
                                            _nbytes(ws), _stream(dev))
    return O


def la_causal_backward(Q, K, V, G, phi="elu1", eps=0.0, O=None, den=None, saved=None, dQ=None, dK=None, dV=None,
                       ws=None, S_in=None, Z_in=None, dS_out=None, dZ_out=None, dS_in=None, dZ_in=None, lengths=None):
    """Gradients of the causal form; returns (dQ, dK, dV).  With any of the state arguments (fp32 [B,H,D,M] /
    [B,H,D]: the state the forward started from, the upstream gradient of its final state, and tensors that
    receive the gradient of the initial state) the call is la_causal_backward_from."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), G=(G, "v"), O=(O, "v"), den=(den, "row"),
            dQ=(dQ, "qk"), dK=(dK, "qk"), dV=(dV, "v"), S_in=(S_in, "S"), Z_in=(Z_in, "Z"), dS_out=(dS_out, "S"),
            dZ_out=(dZ_out, "Z"), dS_in=(dS_in, "S"), dZ_in=(dZ_in, "Z"))
    _buffer("saved", saved), _buffer("ws", ws)
    if lengths is not None:
        _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, G, O, den, dQ, dK, dV, saved, S_in, Z_in, dS_out, dZ_out, dS_in, dZ_in, ws, lengths)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    if lengths is not None:             # la_causal_backward_varlen
        ws = workspace(p, LA_OP_CAUSAL_VARLEN_BACKWARD, dev) if ws is None else ws
        _call(dev, lib().la_causal_backward_varlen, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(S_in),
              _ptr(Z_in), _ptr(O), _ptr(den), _ptr(G), _ptr(dS_out), _ptr(dZ_out), _ptr(saved), _nbytes(saved), _ptr(dQ), _ptr(dK),
              _ptr(dV), _ptr(dS_in), _ptr(dZ_in), _ptr(ws), _nbytes(ws), _stream(dev))
        return dQ, dK, dV
    ws = workspace(p, LA_OP_CAUSAL_BACKWARD, dev) if ws is None else ws
    state = (S_in, Z_in, dS_out, dZ_out, dS_in, dZ_in)
    if all(t is None for t in state):
        _call(dev, lib().la_causal_backward, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(den), _ptr(G), _ptr(saved), _nbytes(saved),
            _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws), _nbytes(ws), _stream(dev))
    else:
        _call(dev, lib().la_causal_backward_from, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(S_in), _ptr(Z_in), _ptr(O), _ptr(den), _ptr(G),
            _ptr(dS_out), _ptr(dZ_out), _ptr(saved), _nbytes(saved), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dS_in), _ptr(dZ_in),
            _ptr(ws), _nbytes(ws), _stream(dev))
    return dQ, dK, dV


def la_recurrent_step(q, k, v, S, Z, phi="elu1", eps=0.0, out=None):
    """One decode step: S, Z (fp32) are updated in place; returns out [B,H,M]."""
    if q.dim() != 3 or v.dim() != 3:
        raise ValueError("expected q,k [B,H,D], v [B,H,M], fp32 S [B,H,D,M] and Z [B,H,D]")
    B, H, D = q.shape
    M = v.shape[2]
    p = make_problem(B, H, 1, D, M, _dtype_code(q), phi, eps)
    _expect(p, q.dtype, q=(q, "q1"), k=(k, "q1"), v=(v, "v1"), S=(S, "S"), Z=(Z, "Z"), out=(out, "v1"))
    dev = _dev(q, k, v, S, Z, out)
    out = torch.empty_like(v) if out is None else out
    _call(dev, lib().la_recurrent_step, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(S), _ptr(Z), _ptr(out),
                                   _stream(dev))
    return out


class PreparedStep:
    """A decode call whose arguments were checked and marshalled once: calling it enqueues the same library call
    again on the stream it was prepared on (the tensors are updated in place, as in a generation loop whose
    buffers do not move).  Per call it costs one foreign-function call instead of the argument checks."""

    __slots__ = ("_fn", "_args", "_keep", "_dev", "out")

    def __init__(self, fn, args, keep, dev, out):
        self._fn, self._args, self._keep, self._dev, self.out = fn, args, keep, dev, out

    def __call__(self):
        rc = self._fn(*self._args)
        if rc != 0:
            _check(rc)
        return self.out


def prepare_recurrent_step(q, k, v, S, Z, phi="elu1", eps=0.0, out=None) -> PreparedStep:
    """la_recurrent_step with its checks done once: returns a callable that repeats the step on the same tensors
    (refill q, k, v in place between calls) on the stream that is current now, with the tensors' device current."""
    if q.dim() != 3 or v.dim() != 3:
        raise ValueError("expected q,k [B,H,D], v [B,H,M], fp32 S [B,H,D,M] and Z [B,H,D]")
    B, H, D = q.shape
    p = make_problem(B, H, 1, D, v.shape[2], _dtype_code(q), phi, eps)
    _expect(p, q.dtype, q=(q, "q1"), k=(k, "q1"), v=(v, "v1"), S=(S, "S"), Z=(Z, "Z"), out=(out, "v1"))
    dev = _dev(q, k, v, S, Z, out)
    if dev.index != torch.cuda.current_device():
        raise ValueError("make the tensors' device current before preparing a step")
    out = torch.empty_like(v) if out is None else out
    args = (ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(S), _ptr(Z), _ptr(out), _stream(dev))
    return PreparedStep(lib().la_recurrent_step, args, (p, q, k, v, S, Z, out), dev, out)


def la_decode_layer_step(x, Wqkv, Wo, S, Z, phi="elu1", eps=0.0, out=None, ws=None):
    """One decode step of a whole attention sublayer: x [B,F] -> y [B,F] with F = H*D (bf16, D = M = 64);
    Wqkv [3F,F] and Wo [F,F] are "outputs x inputs" like a linear layer's weight; S [B,H,D,M], Z [B,H,D] (fp32)
    are updated in place.  Returns y = attention(x) W_O + x."""
    if S.dim() != 4 or x.dim() != 2:
        raise ValueError("expected x [B,F], fp32 S [B,H,D,M] and Z [B,H,D]")
    B, H, D, M = S.shape
    F = H * D
    p = make_problem(B, H, 1, D, M, _dtype_code(x), phi, eps)
    _expect(p, x.dtype, S=(S, "S"), Z=(Z, "Z"))
    for name, t, shape in (("x", x, (B, F)), ("Wqkv", Wqkv, (3 * F, F)), ("Wo", Wo, (F, F)), ("out", out, (B, F))):
        if t is not None and (tuple(t.shape) != shape or t.dtype != x.dtype):
            raise ValueError(f"{name} must have shape {list(shape)} and dtype {x.dtype} (got {list(t.shape)}, {t.dtype})")
    _buffer("ws", ws)
    dev = _dev(x, Wqkv, Wo, S, Z, out, ws)
    out = torch.empty_like(x) if out is None else out
    ws = workspace(p, LA_OP_DECODE_LAYER, dev) if ws is None else ws
    _call(dev, lib().la_decode_layer_step, ctypes.byref(p), _ptr(x), _ptr(Wqkv), _ptr(Wo), _ptr(S), _ptr(Z), _ptr(out),
          _ptr(ws), _nbytes(ws), _stream(dev))
    return out


def la_recurrent_steps(q, k, v, S, Z, phi="elu1", eps=0.0, out=None):
    """N decode steps in one launch (all inputs known beforehand): q, k [B,H,N,D], v [B,H,N,M]; S, Z (fp32)
    are updated in place; returns out [B,H,N,M]."""
    p = _problem_of(q, v, phi, eps)
    _expect(p, q.dtype, q=(q, "qk"), k=(k, "qk"), v=(v, "v"), S=(S, "S"), Z=(Z, "Z"), out=(out, "v"))
    dev = _dev(q, k, v, S, Z, out)
    out = torch.empty_like(v) if out is None else out
    _call(dev, lib().la_recurrent_steps, ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(S), _ptr(Z), _ptr(out),
                                    _stream(dev))
    return out


def _lengths_arg(lengths, B, dev):
    if lengths.dtype != torch.int32 or tuple(lengths.shape) != (B,) or not lengths.is_contiguous():
        raise ValueError("lengths must be a contiguous int32 CUDA tensor of shape [B]")
    return lengths


def la_linear_attention_varlen(Q, K, V, lengths, phi="elu1", eps=0.0, O=None, den=None, KV=None, Zs=None, ws=None):
    """Non-causal form on a right-padded ragged batch: lengths[b] real positions per batch element; O and den
    are zero on the padding.  Returns O."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), O=(O, "v"), den=(den, "row"), KV=(KV, "S"), Zs=(Zs, "Z"))
    _buffer("ws", ws)
    _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, O, den, KV, Zs, lengths, ws)
    O = torch.empty_like(V) if O is None else O
    ws = workspace(p, LA_OP_LINEAR_VARLEN_FORWARD, dev) if ws is None else ws
    _call(dev, lib().la_linear_attention_varlen, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(O), _ptr(den),
                                            _ptr(KV), _ptr(Zs), _ptr(ws), _nbytes(ws), _stream(dev))
    return O


def la_linear_attention_varlen_backward(Q, K, V, G, lengths, phi="elu1", eps=0.0, O=None, den=None,
                                        dQ=None, dK=None, dV=None, ws=None):
    """Gradients of la_linear_attention_varlen; zero on the padding.  Returns (dQ, dK, dV)."""
    p = _problem_of(Q, V, phi, eps)
    _expect(p, Q.dtype, Q=(Q, "qk"), K=(K, "qk"), V=(V, "v"), G=(G, "v"), O=(O, "v"), den=(den, "row"),
            dQ=(dQ, "qk"), dK=(dK, "qk"), dV=(dV, "v"))
    _buffer("ws", ws)
    _lengths_arg(lengths, p.B, None)
    dev = _dev(Q, K, V, G, O, den, dQ, dK, dV, lengths, ws)
    dQ = torch.empty_like(Q) if dQ is None else dQ
    dK = torch.empty_like(K) if dK is None else dK
    dV = torch.empty_like(V) if dV is None else dV
    ws = workspace(p, LA_OP_LINEAR_VARLEN_BACKWARD, dev) if ws is None else ws
    _call(dev, lib().la_linear_attention_varlen_backward, ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths), _ptr(O), _ptr(den), _ptr(G), _ptr(dQ), _ptr(dK), _ptr(dV),
        _ptr(ws), _nbytes(ws), _stream(dev))
    return dQ, dK, dV
