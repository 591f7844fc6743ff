"""fp64 CPU oracle for linear attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy front end of ``la_oracle.c``.  It exists so that the tests,
the smoke check and the benchmark's CPU-baseline leg can ask "what should the
answer be?".  The CUDA library never imports or links it, and this package
never imports the CUDA binding.

All functions take array-likes shaped ``[B, H, N, D]`` / ``[B, H, N, M]`` (or
``[B, H, D]`` / ``[B, H, M]`` for the recurrent step), convert them to
contiguous float64 and return float64 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "la_oracle.c")
_LIB = os.path.join(_HERE, "libla_oracle.so")

PHI = {"elu1": 0, "identity": 1}


def build(force: bool = False) -> str:
    """Compile ``la_oracle.c`` into ``libla_oracle.so`` next to it (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None
_dp = ctypes.POINTER(ctypes.c_double)
_i64 = ctypes.c_int64


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.la_oracle_num_threads.restype = ctypes.c_int
        _lib.la_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib.la_oracle_feature_map.argtypes = [_dp, _dp, _i64, ctypes.c_int]
        _lib.la_oracle_attention_quadratic.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_int, ctypes.c_double] + [_dp] * 5)
        _lib.la_oracle_attention_quadratic_backward.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_int, ctypes.c_double] + [_dp] * 7)
        _lib.la_oracle_linear.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_int, ctypes.c_double] + [_dp] * 7)
        _lib.la_oracle_linear_backward.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_int, ctypes.c_double] + [_dp] * 7)
        _lib.la_oracle_causal_from_state.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_double] + [_dp] * 9)
        _lib.la_oracle_causal_backward_from_state.argtypes = (
            [_i64] * 5 + [ctypes.c_int, ctypes.c_double] + [_dp] * 13)
        _lib.la_oracle_recurrent_step.argtypes = (
            [_i64] * 4 + [ctypes.c_int, ctypes.c_double] + [_dp] * 6)
    return _lib


def _f64(a):
    if hasattr(a, "detach"):  # torch tensor (bf16 has no numpy dtype: widen first)
        a = a.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _shapes(Q, K, V):
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    if Q.ndim != 4 or K.shape != Q.shape or V.ndim != 4 or V.shape[:3] != Q.shape[:3]:
        raise ValueError("expected Q,K [B,H,N,D] and V [B,H,N,M]")
    B, H, N, D = Q.shape
    return Q, K, V, B, H, N, D, V.shape[3]


def num_threads() -> int:
    return _load().la_oracle_num_threads()


def set_threads(n: int) -> None:
    _load().la_oracle_set_threads(int(n))


def feature_map(x, deriv: bool = False):
    """Eq. 7: elu(x)+1 elementwise (or its slope when ``deriv``)."""
    x = _f64(x)
    y = np.empty_like(x)
    _load().la_oracle_feature_map(_p(x), _p(y), x.size, int(deriv))
    return y


def attention_quadratic(Q, K, V, causal: bool, phi: str = "elu1", eps: float = 0.0,
                        return_weights: bool = False):
    """Eq. 3 / Eq. 8 with sim(q,k)=phi(q).phi(k) on the explicit N x N matrix."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    O = np.empty((B, H, N, M))
    W = np.empty((B, H, N, N)) if return_weights else None
    _load().la_oracle_attention_quadratic(B, H, N, D, M, int(causal), PHI[phi], eps,
                                          _p(Q), _p(K), _p(V), _p(O), _p(W))
    return (O, W) if return_weights else O


def attention_quadratic_backward(Q, K, V, G, causal: bool, phi: str = "elu1", eps: float = 0.0):
    """Explicit chain rule through the N x N matrix; returns (dQ, dK, dV)."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    G = _f64(G)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(K), np.empty_like(V)
    _load().la_oracle_attention_quadratic_backward(
        B, H, N, D, M, int(causal), PHI[phi], eps,
        _p(Q), _p(K), _p(V), _p(G), _p(dQ), _p(dK), _p(dV))
    return dQ, dK, dV


def linear_attention(Q, K, V, causal: bool, phi: str = "elu1", eps: float = 0.0,
                     return_state: bool = False):
    """Eq. 5-6 (non-causal) or Eq. 9-12 / Algorithm 1 (causal); returns (O, den[, S, Z])."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    O = np.empty((B, H, N, M))
    den = np.empty((B, H, N))
    S = np.empty((B, H, D, M)) if return_state else None
    Z = np.empty((B, H, D)) if return_state else None
    _load().la_oracle_linear(B, H, N, D, M, int(causal), PHI[phi], eps,
                             _p(Q), _p(K), _p(V), _p(O), _p(den), _p(S), _p(Z))
    return (O, den, S, Z) if return_state else (O, den)


def causal_from_state(Q, K, V, S0, Z0, phi: str = "elu1", eps: float = 0.0):
    """Eq. 16-20 (attention part) run over N tokens from the state S0 [B,H,D,M], Z0 [B,H,D];
    returns (O, den, S_N, Z_N)."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    S0, Z0 = _f64(S0), _f64(Z0)
    if S0.shape != (B, H, D, M) or Z0.shape != (B, H, D):
        raise ValueError("state shape mismatch")
    O = np.empty((B, H, N, M))
    den = np.empty((B, H, N))
    S = np.empty((B, H, D, M))
    Z = np.empty((B, H, D))
    _load().la_oracle_causal_from_state(B, H, N, D, M, PHI[phi], eps, _p(Q), _p(K), _p(V), _p(S0), _p(Z0),
                                        _p(O), _p(den), _p(S), _p(Z))
    return O, den, S, Z


def causal_backward_from_state(Q, K, V, S0, Z0, G, dSN=None, dZN=None, phi: str = "elu1", eps: float = 0.0):
    """Gradient of sum(G * O) + <dSN, S_N> + <dZN, Z_N> for causal_from_state; returns (dQ, dK, dV, dS0, dZ0)."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    S0, Z0, G = _f64(S0), _f64(Z0), _f64(G)
    dSN = None if dSN is None else _f64(dSN)
    dZN = None if dZN is None else _f64(dZN)
    if S0.shape != (B, H, D, M) or Z0.shape != (B, H, D):
        raise ValueError("state shape mismatch")
    dQ, dK, dV = np.empty_like(Q), np.empty_like(K), np.empty_like(V)
    dS0, dZ0 = np.empty((B, H, D, M)), np.empty((B, H, D))
    _load().la_oracle_causal_backward_from_state(
        B, H, N, D, M, PHI[phi], eps, _p(Q), _p(K), _p(V), _p(S0), _p(Z0), _p(G), _p(dSN), _p(dZN),
        _p(dQ), _p(dK), _p(dV), _p(dS0), _p(dZ0))
    return dQ, dK, dV, dS0, dZ0


def linear_attention_backward(Q, K, V, G, causal: bool, phi: str = "elu1", eps: float = 0.0):
    """Eq. 13-15 on the ones-extended values, forward and reverse running sums."""
    Q, K, V, B, H, N, D, M = _shapes(Q, K, V)
    G = _f64(G)
    dQ, dK, dV = np.empty_like(Q), np.empty_like(K), np.empty_like(V)
    _load().la_oracle_linear_backward(
        B, H, N, D, M, int(causal), PHI[phi], eps,
        _p(Q), _p(K), _p(V), _p(G), _p(dQ), _p(dK), _p(dV))
    return dQ, dK, dV


def recurrent_step(q, k, v, S, Z, phi: str = "elu1", eps: float = 0.0):
    """Eq. 18-20: update S, Z (float64 arrays, IN PLACE), then read out; returns out [B,H,M]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    if not (isinstance(S, np.ndarray) and S.dtype == np.float64 and S.flags.c_contiguous
            and isinstance(Z, np.ndarray) and Z.dtype == np.float64 and Z.flags.c_contiguous):
        raise ValueError("S and Z must be contiguous float64 numpy arrays (updated in place)")
    B, H, D = q.shape
    M = v.shape[2]
    if S.shape != (B, H, D, M) or Z.shape != (B, H, D):
        raise ValueError("state shape mismatch")
    out = np.empty((B, H, M))
    _load().la_oracle_recurrent_step(B, H, D, M, PHI[phi], eps,
                                     _p(q), _p(k), _p(v), _p(S), _p(Z), _p(out))
    return out


# ---------------------------------------------------------------------------
# Degree-2 polynomial kernel (Section 3.2.1, "Feature Maps and Computational Cost"): the kernel
# sim(a, b) = (a . b)^2 has the exact finite feature map phi(a) = vec(a a^T) of dimension C = D^2.
# The paper names the kernel and its cost O(N D^2 M) without fixing its form; the homogeneous form is
# the one whose feature map has exactly D^2 components.  Plain numpy, written from the definitions.
# ---------------------------------------------------------------------------
def poly2_feature_map(x, C_pad: int | None = None):
    """phi(x)[..., i*D + j] = x_i x_j; columns D*D .. C_pad-1 (if asked for) are zero."""
    x = _f64(x)
    D = x.shape[-1]
    C = D * D
    C_pad = C if C_pad is None else int(C_pad)
    if C_pad < C:
        raise ValueError("C_pad is smaller than D*D")
    y = np.zeros(x.shape[:-1] + (C_pad,))
    for i in range(D):
        for j in range(D):
            y[..., i * D + j] = x[..., i] * x[..., j]
    return y


def poly2_feature_map_backward(x, dy):
    """Gradient of poly2_feature_map: dx_i = sum_j (dy[i*D + j] + dy[j*D + i]) x_j."""
    x, dy = _f64(x), _f64(dy)
    D = x.shape[-1]
    dx = np.zeros_like(x)
    for i in range(D):
        for j in range(D):
            dx[..., i] += (dy[..., i * D + j] + dy[..., j * D + i]) * x[..., j]
    return dx


def poly2_attention(Q, K, V, causal: bool, eps: float = 0.0):
    """Eq. 3 (Eq. 8 when causal) with sim(q, k) = (q . k)^2 on the explicit N x N matrix."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    B, H, N, _ = Q.shape
    O = np.empty(V.shape)
    for b in range(B):
        for h in range(H):
            A = (Q[b, h] @ K[b, h].T) ** 2
            if causal:
                A = np.tril(A)
            O[b, h] = (A @ V[b, h]) / (A.sum(axis=1, keepdims=True) + eps)
    return O


# ---------------------------------------------------------------------------
# Random Fourier features for the Gaussian (RBF) kernel, which the paper's conclusion names as a feature map
# to explore and does not write down.  Reading: the classical construction with the frequencies given by the
# caller, W [C/2, D], in its paired form
#     phi(x) = sqrt(2 / C) [cos(W x), sin(W x)]   in R^C,
# for which phi(x) . phi(y) = (2 / C) sum_c cos(w_c . (x - y)) exactly (a function of x - y alone, |phi(x)| = 1),
# and whose expectation over w_c ~ N(0, I) is exp(-|x - y|^2 / 2).  Plain numpy, written from the definition.
# ---------------------------------------------------------------------------
def rff_feature_map(x, W):
    """x [..., D], W [C/2, D] -> [..., C]: sqrt(2/C) cos(x W^T) in the first C/2 columns, sqrt(2/C) sin(x W^T) in the rest."""
    x, W = _f64(x), _f64(W)
    z = x @ W.T
    return np.concatenate([np.cos(z), np.sin(z)], axis=-1) * np.sqrt(1.0 / W.shape[0])


def rff_feature_map_backward(x, W, dy):
    """Gradient of rff_feature_map with respect to x: dx = sqrt(2/C) (-sin(z) * dy_cos + cos(z) * dy_sin) W, z = x W^T."""
    x, W, dy = _f64(x), _f64(W), _f64(dy)
    h = W.shape[0]
    z = x @ W.T
    t = (-np.sin(z) * dy[..., :h] + np.cos(z) * dy[..., h:]) * np.sqrt(1.0 / h)
    return t @ W


# ---------------------------------------------------------------------------
# One decode step of a whole attention sublayer, Eq. 16-20 with the projections written out:
#   q = x W_Q, k = x W_K, v = x W_V (split into H heads), s_i = s_{i-1} + phi(k) v^T, z_i = z_{i-1} + phi(k),
#   a = phi(q)^T s_i / (phi(q)^T z_i + eps) per head,  y = a W_O + x.
# The feed-forward part f_l of Eq. 20 stays with the caller (it acts on each position alone).  The
# projections are numpy matrix products; the state update and read-out are recurrent_step above.
# ---------------------------------------------------------------------------
def decode_layer_step(x, Wq, Wk, Wv, Wo, S, Z, phi: str = "elu1", eps: float = 0.0):
    """x [B,F]; Wq, Wk [F,H*D], Wv [F,H*M], Wo [H*M,F] (float64, applied as x @ W); S [B,H,D,M] and Z [B,H,D]
    (contiguous float64) are updated IN PLACE.  Returns y [B,F]."""
    x, Wq, Wk, Wv, Wo = (_f64(t) for t in (x, Wq, Wk, Wv, Wo))
    B, H, D, M = S.shape
    if x.ndim != 2 or x.shape[0] != B or Wq.shape != (x.shape[1], H * D) or Wk.shape != Wq.shape \
            or Wv.shape != (x.shape[1], H * M) or Wo.shape != (H * M, x.shape[1]):
        raise ValueError("shape mismatch between x, the projections and the state")
    q = (x @ Wq).reshape(B, H, D)
    k = (x @ Wk).reshape(B, H, D)
    v = (x @ Wv).reshape(B, H, M)
    a = recurrent_step(q, k, v, S, Z, phi, eps)
    return a.reshape(B, H * M) @ Wo + x
