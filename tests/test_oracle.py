"""Pins for the fp64 oracle (no GPU).

Every oracle routine is checked against something that is not the oracle:
closed forms, a hand-worked rational example, exact-rational brute force of the
definition, numpy/torch library one-liners, torch autograd through the
quadratic form, central finite differences and structural invariants.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ---------------------------------------------------------------- feature map
def test_phi_closed_forms():
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", "phi_values.txt")) as f:
        for line in f:
            line = line.split("#", 1)[0].split()
            if line:
                rows.append([float(t) for t in line])
    rows = np.array(rows)
    assert np.allclose(oracle.feature_map(rows[:, 0]), rows[:, 1], rtol=1e-15, atol=0)
    assert np.allclose(oracle.feature_map(rows[:, 0], deriv=True), rows[:, 2], rtol=1e-15, atol=0)


def test_phi_properties():
    x = np.linspace(-30, 30, 2001)
    y = oracle.feature_map(x)
    assert (y > 0).all()                                   # positive similarity
    assert (np.diff(y) > 0).all()                          # monotone
    neg = x <= 0
    assert np.array_equal(oracle.feature_map(x, True)[neg], y[neg])   # phi' = phi for x <= 0
    assert (oracle.feature_map(x, True)[~neg] == 1).all()
    # matches the library elu
    t = torch.nn.functional.elu(torch.from_numpy(x)) + 1
    # (elu(x) + 1 cancels for very negative x, hence the absolute tolerance)
    assert np.allclose(y, t.numpy(), rtol=1e-15, atol=3e-16)


# ------------------------------------------------------------ worked example
def _ex(worked_example, *names):
    return [worked_example[n][None, None] for n in names]


@pytest.mark.parametrize("routine", ["quadratic", "linear"])
def test_worked_example_forward(worked_example, routine):
    Q, K, V = _ex(worked_example, "Q", "K", "V")
    assert np.array_equal(oracle.feature_map(Q)[0, 0], worked_example["phiQ"])
    assert np.array_equal(oracle.feature_map(K)[0, 0], worked_example["phiK"])
    for causal, tag in ((True, "causal"), (False, "noncausal")):
        if routine == "quadratic":
            O = oracle.attention_quadratic(Q, K, V, causal)
        else:
            O, den = oracle.linear_attention(Q, K, V, causal)
            assert np.allclose(den[0, 0], worked_example[tag + "_den"][0], rtol=1e-15)
        assert np.allclose(O[0, 0], worked_example[tag + "_O"], rtol=1e-14, atol=1e-16)


def test_worked_example_states(worked_example):
    Q, K, V = _ex(worked_example, "Q", "K", "V")
    S = np.zeros((1, 1, 2, 2))
    Z = np.zeros((1, 1, 2))
    for i in range(3):
        out = oracle.recurrent_step(Q[:, :, i], K[:, :, i], V[:, :, i], S, Z)
        assert np.array_equal(S[0, 0], worked_example[f"S{i + 1}"])
        assert np.array_equal(Z[0, 0], worked_example[f"Z{i + 1}"][0])
        assert np.allclose(out[0, 0], worked_example["causal_O"][i], rtol=1e-14, atol=1e-16)
    _, _, S3, Z3 = oracle.linear_attention(Q, K, V, True, return_state=True)
    assert np.array_equal(S3[0, 0], worked_example["S3"])
    assert np.array_equal(Z3[0, 0], worked_example["Z3"][0])


@pytest.mark.parametrize("routine", ["quadratic", "linear"])
def test_worked_example_backward(worked_example, routine):
    Q, K, V, G = _ex(worked_example, "Q", "K", "V", "G")
    fn = (oracle.attention_quadratic_backward if routine == "quadratic"
          else oracle.linear_attention_backward)
    for causal, tag in ((True, "causal"), (False, "noncausal")):
        dQ, dK, dV = fn(Q, K, V, G, causal)
        assert np.allclose(dQ[0, 0], worked_example[tag + "_dQ"], rtol=1e-13, atol=1e-16)
        assert np.allclose(dK[0, 0], worked_example[tag + "_dK"], rtol=1e-13, atol=1e-16)
        assert np.allclose(dV[0, 0], worked_example[tag + "_dV"], rtol=1e-13, atol=1e-16)


# -------------------------------------------- exact brute force of definition
def _exact_attention(phiQ, phiK, V, causal):
    """Eq. 3 / Eq. 8 in exact rationals on already-mapped integer features."""
    N = len(phiQ)
    out = []
    for i in range(N):
        js = range(i + 1) if causal else range(N)
        w = [sum(Fraction(a) * Fraction(b) for a, b in zip(phiQ[i], phiK[j])) for j in js]
        den = sum(w)
        out.append([sum(wj * Fraction(V[j][e]) for wj, j in zip(w, js)) / den
                    for e in range(len(V[0]))])
    return out


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_exact_rational_bruteforce(causal, seed):
    rng = np.random.default_rng(seed)
    N, D, M = 7, 3, 4
    Qi = rng.integers(0, 6, (N, D))          # non-negative: phi(x) = x + 1 exactly
    Ki = rng.integers(0, 6, (N, D))
    Vi = rng.integers(-9, 10, (N, M))
    exact = _exact_attention((Qi + 1).tolist(), (Ki + 1).tolist(), Vi.tolist(), causal)
    exact = np.array([[float(x) for x in r] for r in exact])
    args = [a[None, None].astype(float) for a in (Qi, Ki, Vi)]
    assert np.allclose(oracle.attention_quadratic(*args, causal)[0, 0], exact, rtol=1e-14, atol=1e-15)
    assert np.allclose(oracle.linear_attention(*args, causal)[0][0, 0], exact, rtol=1e-13, atol=1e-14)
    # identity feature map on the mapped features gives the same thing
    argsI = [(Qi + 1)[None, None].astype(float), (Ki + 1)[None, None].astype(float), args[2]]
    assert np.allclose(oracle.attention_quadratic(*argsI, causal, phi="identity")[0, 0], exact,
                       rtol=1e-14, atol=1e-15)


# ----------------------------------------------------- library one-liner form
def _numpy_form(Q, K, V, causal, eps=0.0):
    fq = np.where(Q > 0, Q + 1, np.exp(np.minimum(Q, 0)))
    fk = np.where(K > 0, K + 1, np.exp(np.minimum(K, 0)))
    A = fq @ np.swapaxes(fk, -1, -2)
    if causal:
        A = np.tril(A)
    return (A @ V) / (A.sum(-1, keepdims=True) + eps), A


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape", [(2, 3, 17, 5, 7), (1, 2, 64, 8, 4), (1, 1, 1, 4, 4)])
def test_quadratic_and_linear_match_matrix_form(causal, shape):
    B, H, N, D, M = shape
    Q, K, V = rnd((B, H, N, D), 1), rnd((B, H, N, D), 2), rnd((B, H, N, M), 3)
    ref, A = _numpy_form(Q, K, V, causal)
    Oq, W = oracle.attention_quadratic(Q, K, V, causal, return_weights=True)
    Ol, den = oracle.linear_attention(Q, K, V, causal)
    assert np.allclose(Oq, ref, rtol=1e-12, atol=1e-13)
    assert np.allclose(Ol, ref, rtol=1e-11, atol=1e-12)
    assert np.allclose(den, A.sum(-1), rtol=1e-12)
    assert np.allclose(W, A / A.sum(-1, keepdims=True), rtol=1e-12, atol=0)
    # eps enters the denominator additively
    refe, _ = _numpy_form(Q, K, V, causal, eps=0.5)
    assert np.allclose(oracle.attention_quadratic(Q, K, V, causal, eps=0.5), refe, rtol=1e-12, atol=1e-13)
    assert np.allclose(oracle.linear_attention(Q, K, V, causal, eps=0.5)[0], refe, rtol=1e-11, atol=1e-12)


# ------------------------------------------------------------------ invariants
@pytest.mark.parametrize("causal", [True, False])
def test_weights_positive_rows_sum_to_one_constant_v(causal):
    B, H, N, D, M = 1, 2, 33, 6, 5
    Q, K = rnd((B, H, N, D), 4) * 3, rnd((B, H, N, D), 5) * 3
    V = np.broadcast_to(rnd((1, 1, 1, M), 6), (B, H, N, M)).copy()
    O, W = oracle.attention_quadratic(Q, K, V, causal, return_weights=True)
    allowed = np.tril(np.ones((N, N), bool)) if causal else np.ones((N, N), bool)
    assert (W[..., allowed] > 0).all() and (W[..., ~allowed] == 0).all()
    assert np.allclose(W.sum(-1), 1.0, rtol=1e-14)
    assert np.allclose(O, V, rtol=1e-13)                       # constant V is reproduced
    assert np.allclose(oracle.linear_attention(Q, K, V, causal)[0], V, rtol=1e-12)


def test_first_causal_output_is_first_value_and_uniform_keys_give_means():
    B, H, N, D, M = 2, 2, 19, 4, 3
    Q, K, V = rnd((B, H, N, D), 7), rnd((B, H, N, D), 8), rnd((B, H, N, M), 9)
    for fn in (lambda *a: oracle.attention_quadratic(*a), lambda *a: oracle.linear_attention(*a)[0]):
        assert np.allclose(fn(Q, K, V, True)[:, :, 0], V[:, :, 0], rtol=1e-13)
        Ku = np.broadcast_to(K[:, :, :1], K.shape).copy()     # all keys equal: uniform weights
        run_mean = np.cumsum(V, 2) / np.arange(1, N + 1)[None, None, :, None]
        assert np.allclose(fn(Q, Ku, V, True), run_mean, rtol=1e-12, atol=1e-13)
        full_mean = np.broadcast_to(V.mean(2, keepdims=True), V.shape)
        assert np.allclose(fn(Q, Ku, V, False), full_mean, rtol=1e-12, atol=1e-13)


def test_outputs_lie_in_value_range():
    Q, K, V = rnd((1, 1, 40, 8), 10), rnd((1, 1, 40, 8), 11), rnd((1, 1, 40, 3), 12)
    O = oracle.linear_attention(Q, K, V, True)[0]
    lo = np.minimum.accumulate(V, 2)
    hi = np.maximum.accumulate(V, 2)
    assert (O >= lo - 1e-12).all() and (O <= hi + 1e-12).all()


# ------------------------------------------------- recurrent == parallel form
@pytest.mark.parametrize("shape", [(2, 2, 23, 5, 3), (1, 3, 40, 8, 8)])
def test_recurrent_unrolled_equals_causal(shape):
    B, H, N, D, M = shape
    Q, K, V = rnd((B, H, N, D), 13), rnd((B, H, N, D), 14), rnd((B, H, N, M), 15)
    ref = oracle.attention_quadratic(Q, K, V, True)
    _, _, SN, ZN = oracle.linear_attention(Q, K, V, True, return_state=True)
    S, Z = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    for i in range(N):
        out = oracle.recurrent_step(Q[:, :, i], K[:, :, i], V[:, :, i], S, Z)
        assert np.allclose(out, ref[:, :, i], rtol=1e-11, atol=1e-12)
    assert np.allclose(S, SN, rtol=1e-13, atol=1e-13) and np.allclose(Z, ZN, rtol=1e-13)
    fk = oracle.feature_map(K)
    assert np.allclose(S, np.einsum("bhnd,bhnm->bhdm", fk, V), rtol=1e-12, atol=1e-12)   # Eq. 10
    assert np.allclose(Z, fk.sum(2), rtol=1e-13)                                          # Eq. 11


# ------------------------------------------------ continuation from a state
def test_causal_from_state_hand_example():
    # D = M = 1, identity features, q = k = 1, s_0 = 3, z_0 = 2, v = 1, 2, 3 (Eq. 18-20 by hand):
    # O_i = (3 + v_1 + .. + v_i) / (2 + i) = 4/3, 6/4, 9/5; final state s = 9, z = 5
    one = np.ones((1, 1, 3, 1))
    V = np.array([1.0, 2.0, 3.0]).reshape(1, 1, 3, 1)
    O, den, S, Z = oracle.causal_from_state(one, one, V, np.full((1, 1, 1, 1), 3.0), np.full((1, 1, 1), 2.0), phi="identity")
    assert np.allclose(O.ravel(), [4 / 3, 6 / 4, 9 / 5], rtol=1e-15)
    assert np.allclose(den.ravel(), [3.0, 4.0, 5.0]) and S.item() == 9.0 and Z.item() == 5.0


@pytest.mark.parametrize("shape", [(2, 2, 23, 5, 3), (1, 3, 40, 8, 8)])
def test_causal_from_state_equals_unrolled_recurrent_steps(shape):
    # Eq. 18-20 step by step from an arbitrary (positive-normaliser) state
    B, H, N, D, M = shape
    Q, K, V = rnd((B, H, N, D), 33), rnd((B, H, N, D), 34), rnd((B, H, N, M), 35)
    S0, Z0 = rnd((B, H, D, M), 36), np.abs(rnd((B, H, D), 37)) + 0.5
    O, den, SN, ZN = oracle.causal_from_state(Q, K, V, S0, Z0)
    S, Z = S0.copy(), Z0.copy()
    for i in range(N):
        out = oracle.recurrent_step(Q[:, :, i], K[:, :, i], V[:, :, i], S, Z)
        assert np.allclose(out, O[:, :, i], rtol=1e-11, atol=1e-12)
    assert np.allclose(S, SN, rtol=1e-13, atol=1e-13) and np.allclose(Z, ZN, rtol=1e-13)


@pytest.mark.parametrize("cut", [1, 17, 39])
def test_a_sequence_cut_in_two_calls_reproduces_the_definition(cut):
    # the definition (explicit N x N masked attention) on the whole sequence against: first part from zero,
    # second part continued from the first part's final state; zero state reduces to the causal form
    B, H, N, D, M = 2, 2, 40, 6, 5
    Q, K, V = rnd((B, H, N, D), 43), rnd((B, H, N, D), 44), rnd((B, H, N, M), 45)
    ref = oracle.attention_quadratic(Q, K, V, True)
    O1, _, S1, Z1 = oracle.linear_attention(Q[:, :, :cut], K[:, :, :cut], V[:, :, :cut], True, return_state=True)
    O2, den2, S2, Z2 = oracle.causal_from_state(Q[:, :, cut:], K[:, :, cut:], V[:, :, cut:], S1, Z1)
    assert np.allclose(np.concatenate([O1, O2], axis=2), ref, rtol=1e-11, atol=1e-12)
    _, denf, SN, ZN = oracle.linear_attention(Q, K, V, True, return_state=True)
    assert np.allclose(den2, denf[:, :, cut:], rtol=1e-12) and np.allclose(S2, SN, rtol=1e-12, atol=1e-13)
    assert np.allclose(Z2, ZN, rtol=1e-13)
    Oz, denz, Sz, Zz = oracle.causal_from_state(Q, K, V, np.zeros((B, H, D, M)), np.zeros((B, H, D)))
    assert np.allclose(Oz, ref, rtol=1e-11, atol=1e-12)


def test_backward_from_state_matches_finite_differences():
    # every argument, including the state the call starts from, with an upstream gradient on the final state
    B, H, N, D, M = 1, 2, 6, 3, 2
    Q, K, V, G = rnd((B, H, N, D), 51), rnd((B, H, N, D), 52), rnd((B, H, N, M), 53), rnd((B, H, N, M), 54)
    S0, Z0 = rnd((B, H, D, M), 55), np.abs(rnd((B, H, D), 56)) + 1.0
    dSN, dZN = rnd((B, H, D, M), 57), rnd((B, H, D), 58)

    def loss(Q, K, V, S0, Z0):
        O, _, SN, ZN = oracle.causal_from_state(Q, K, V, S0, Z0)
        return (G * O).sum() + (dSN * SN).sum() + (dZN * ZN).sum()

    grads = oracle.causal_backward_from_state(Q, K, V, S0, Z0, G, dSN, dZN)
    args = [Q, K, V, S0, Z0]
    h = 1e-6
    for a, g in zip(range(5), grads):
        x = args[a]
        for idx in np.ndindex(x.shape):
            up, dn = [t.copy() for t in args], [t.copy() for t in args]
            up[a][idx] += h
            dn[a][idx] -= h
            fd = (loss(*up) - loss(*dn)) / (2 * h)
            assert abs(fd - g[idx]) <= 1e-6 * max(1.0, abs(fd)), (a, idx, fd, g[idx])


@pytest.mark.parametrize("cut", [1, 9, 22])
def test_backward_chained_over_two_calls_equals_backward_of_the_whole(cut):
    # the gradient of the whole sequence (a routine pinned to autograd through the N x N definition above)
    # against two calls: the second part from the first part's final state, its state gradient fed to the first
    B, H, N, D, M = 2, 2, 23, 5, 4
    Q, K, V, G = rnd((B, H, N, D), 61), rnd((B, H, N, D), 62), rnd((B, H, N, M), 63), rnd((B, H, N, M), 64)
    rq, rk, rv = oracle.linear_attention_backward(Q, K, V, G, True)
    a, b = slice(0, cut), slice(cut, N)
    _, _, S1, Z1 = oracle.linear_attention(Q[:, :, a], K[:, :, a], V[:, :, a], True, return_state=True)
    q2, k2, v2, dS1, dZ1 = oracle.causal_backward_from_state(Q[:, :, b], K[:, :, b], V[:, :, b], S1, Z1, G[:, :, b])
    zS, zZ = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    q1, k1, v1, dS0, dZ0 = oracle.causal_backward_from_state(Q[:, :, a], K[:, :, a], V[:, :, a], zS, zZ, G[:, :, a], dS1, dZ1)
    for got, ref in ((np.concatenate([q1, q2], 2), rq), (np.concatenate([k1, k2], 2), rk), (np.concatenate([v1, v2], 2), rv)):
        assert np.allclose(got, ref, rtol=1e-10, atol=1e-12)
    # from a zero state and without a state gradient the routine is the causal backward itself
    q0, k0, v0, _, _ = oracle.causal_backward_from_state(Q, K, V, zS, zZ, G)
    assert np.allclose(q0, rq, rtol=1e-12, atol=1e-13) and np.allclose(k0, rk, rtol=1e-12, atol=1e-13)
    assert np.allclose(v0, rv, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------- gradients
def _torch_quadratic(Q, K, V, causal, eps=0.0, identity=False):
    phi = (lambda x: x) if identity else (lambda x: torch.nn.functional.elu(x) + 1)
    A = phi(Q) @ phi(K).transpose(-1, -2)
    if causal:
        A = torch.tril(A)
    return (A @ V) / (A.sum(-1, keepdim=True) + eps)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("shape", [(2, 2, 21, 5, 7), (1, 1, 48, 8, 4)])
@pytest.mark.parametrize("eps", [0.0, 0.25])
def test_backward_matches_autograd_through_quadratic_form(causal, shape, eps):
    B, H, N, D, M = shape
    Qn, Kn, Vn, Gn = rnd((B, H, N, D), 16), rnd((B, H, N, D), 17), rnd((B, H, N, M), 18), rnd((B, H, N, M), 19)
    Q, K, V = (torch.tensor(a, requires_grad=True) for a in (Qn, Kn, Vn))
    (_torch_quadratic(Q, K, V, causal, eps) * torch.tensor(Gn)).sum().backward()
    for fn in (oracle.attention_quadratic_backward, oracle.linear_attention_backward):
        dQ, dK, dV = fn(Qn, Kn, Vn, Gn, causal, eps=eps)
        assert np.allclose(dQ, Q.grad.numpy(), rtol=1e-9, atol=1e-11)
        assert np.allclose(dK, K.grad.numpy(), rtol=1e-9, atol=1e-11)
        assert np.allclose(dV, V.grad.numpy(), rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("causal", [True, False])
def test_backward_identity_feature_map(causal):
    B, H, N, D, M = 1, 2, 15, 4, 5
    Qn, Kn = np.abs(rnd((B, H, N, D), 20)) + 0.1, np.abs(rnd((B, H, N, D), 21)) + 0.1
    Vn, Gn = rnd((B, H, N, M), 22), rnd((B, H, N, M), 23)
    Q, K, V = (torch.tensor(a, requires_grad=True) for a in (Qn, Kn, Vn))
    (_torch_quadratic(Q, K, V, causal, identity=True) * torch.tensor(Gn)).sum().backward()
    for fn in (oracle.attention_quadratic_backward, oracle.linear_attention_backward):
        dQ, dK, dV = fn(Qn, Kn, Vn, Gn, causal, phi="identity")
        assert np.allclose(dQ, Q.grad.numpy(), rtol=1e-9, atol=1e-11)
        assert np.allclose(dK, K.grad.numpy(), rtol=1e-9, atol=1e-11)
        assert np.allclose(dV, V.grad.numpy(), rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("causal", [True, False])
def test_backward_matches_finite_differences(causal):
    B, H, N, D, M = 1, 1, 9, 3, 4
    Q, K, V, G = rnd((B, H, N, D), 24), rnd((B, H, N, D), 25), rnd((B, H, N, M), 26), rnd((B, H, N, M), 27)
    for a in (Q, K):                      # phi is only C^1 at 0: keep away from the kink
        a[np.abs(a) < 1e-3] = 0.5
    assert (Q < 0).any() and (K < 0).any() and (Q > 0).any() and (K > 0).any()
    loss = lambda q, k, v: float((oracle.attention_quadratic(q, k, v, causal) * G).sum())
    grads = oracle.linear_attention_backward(Q, K, V, G, causal)
    h = 1e-6
    for which, (arr, grad) in enumerate(zip((Q, K, V), grads)):
        fd = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            args_p, args_m = [Q.copy(), K.copy(), V.copy()], [Q.copy(), K.copy(), V.copy()]
            args_p[which][idx] += h
            args_m[which][idx] -= h
            fd[idx] = (loss(*args_p) - loss(*args_m)) / (2 * h)
        assert np.allclose(grad, fd, rtol=1e-6, atol=1e-8), which


@pytest.mark.parametrize("causal", [True, False])
def test_gradient_invariants(causal):
    B, H, N, D, M = 2, 2, 37, 6, 5
    Q, K, V, G = rnd((B, H, N, D), 28), rnd((B, H, N, D), 29), rnd((B, H, N, M), 30), rnd((B, H, N, M), 31)
    dQ, dK, dV = oracle.linear_attention_backward(Q, K, V, G, causal)
    # rows of the attention matrix sum to one  =>  sum_j dV_j = sum_i G_i
    assert np.allclose(dV.sum(2), G.sum(2), rtol=1e-11, atol=1e-12)
    # O is homogeneous of degree 0 in phi(Q_i)  =>  <phi(Q_i), grad phi(Q_i)> = 0
    ratio = lambda x: np.where(x > 0, x + 1.0, 1.0)           # phi / phi'
    assert np.abs((ratio(Q) * dQ).sum(-1)).max() < 1e-12
    # a global scale of phi(K) cancels  =>  sum_{j,d} phi(K_jd) grad phi(K_jd) = 0
    assert np.abs((ratio(K) * dK).sum((-1, -2))).max() < 1e-11


def test_linear_matches_quadratic_on_larger_case():
    B, H, N, D, M = 1, 2, 300, 16, 12
    Q, K, V, G = rnd((B, H, N, D), 32), rnd((B, H, N, D), 33), rnd((B, H, N, M), 34), rnd((B, H, N, M), 35)
    for causal in (True, False):
        assert np.allclose(oracle.linear_attention(Q, K, V, causal)[0],
                           oracle.attention_quadratic(Q, K, V, causal), rtol=1e-10, atol=1e-12)
        for a, b in zip(oracle.linear_attention_backward(Q, K, V, G, causal),
                        oracle.attention_quadratic_backward(Q, K, V, G, causal)):
            assert np.allclose(a, b, rtol=1e-9, atol=1e-11)


def test_threads_reported():
    assert oracle.num_threads() >= 1


# --------------------------------------------------------------------------
# Degree-2 polynomial kernel (Section 3.2.1): exact finite feature map.
# --------------------------------------------------------------------------
def test_poly2_feature_map_hand_example_and_kernel_identity():
    # a = (1, 2): a a^T = [[1, 2], [2, 4]], row-major; padding columns are zero
    assert oracle.poly2_feature_map([1.0, 2.0], 8).tolist() == [1.0, 2.0, 2.0, 4.0, 0.0, 0.0, 0.0, 0.0]
    # (3, -1).(1, 2) = 1, squared 1; by features: 9*1 + (-3)*2 + (-3)*2 + 1*4 = 1
    assert float(oracle.poly2_feature_map([3.0, -1.0]) @ oracle.poly2_feature_map([1.0, 2.0])) == 1.0
    rng = np.random.default_rng(3)
    for D in (1, 3, 8, 11):
        a, b = rng.standard_normal((50, D)), rng.standard_normal((50, D))
        lhs = (oracle.poly2_feature_map(a, 128) * oracle.poly2_feature_map(b, 128)).sum(-1)
        np.testing.assert_allclose(lhs, (a * b).sum(-1) ** 2, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("causal", [False, True])
def test_poly2_attention_equals_linear_attention_on_the_features(causal):
    """The similarity form on the N x N matrix of (q.k)^2 against the linear form (sums of phi(k) v^T)
    on the explicit features: two codes that share nothing."""
    rng = np.random.default_rng(5 + causal)
    B, H, N, D, M = 2, 2, 37, 4, 6
    Q, K, V = rng.standard_normal((B, H, N, D)), rng.standard_normal((B, H, N, D)), rng.standard_normal((B, H, N, M))
    ref = oracle.poly2_attention(Q, K, V, causal)
    fQ, fK = oracle.poly2_feature_map(Q, 24), oracle.poly2_feature_map(K, 24)
    np.testing.assert_allclose(oracle.linear_attention(fQ, fK, V, causal, "identity")[0], ref, rtol=1e-9, atol=1e-11)
    # hand case: one query, two keys: weights (q.k1)^2 : (q.k2)^2 = 4 : 1
    o = oracle.poly2_attention([[[[1.0, 0.0]] * 2]], [[[[2.0, 5.0], [1.0, -3.0]]]], [[[[10.0], [20.0]]]], False)
    np.testing.assert_allclose(o[0, 0, :, 0], [12.0, 12.0], rtol=1e-15)


def test_poly2_backward_matches_finite_differences():
    rng = np.random.default_rng(9)
    B, H, N, D, M = 1, 2, 9, 3, 4
    Q, K, V, G = (rng.standard_normal((B, H, N, d)) for d in (D, D, M, M))

    def loss(q, k):
        return float((oracle.poly2_attention(q, k, V, True) * G).sum())

    fQ, fK = oracle.poly2_feature_map(Q, 16), oracle.poly2_feature_map(K, 16)
    dfQ, dfK, _ = oracle.linear_attention_backward(fQ, fK, V, G, True, "identity")
    dQ, dK = oracle.poly2_feature_map_backward(Q, dfQ), oracle.poly2_feature_map_backward(K, dfK)
    h = 1e-6
    for X, dX, which in ((Q, dQ, 0), (K, dK, 1)):
        for idx in [(0, 0, 0, 0), (0, 1, 4, 2), (0, 0, 8, 1), (0, 1, 3, 0)]:
            Xp, Xm = X.copy(), X.copy()
            Xp[idx] += h
            Xm[idx] -= h
            fd = (loss(Xp, K) - loss(Xm, K)) / (2 * h) if which == 0 else (loss(Q, Xp) - loss(Q, Xm)) / (2 * h)
            assert abs(fd - dX[idx]) <= 1e-6 * max(1.0, abs(fd)), (which, idx, fd, dX[idx])


# ---------------------------------------------------------------------------
# Decode step of a whole attention sublayer (Eq. 16-20 with the projections)
# ---------------------------------------------------------------------------
def _layer_weights(F, H, D, M, seed):
    rng = np.random.default_rng(seed)
    s = 1.0 / np.sqrt(F)
    return (rng.standard_normal((F, H * D)) * s, rng.standard_normal((F, H * D)) * s,
            rng.standard_normal((F, H * M)) * s, rng.standard_normal((H * M, F)) * s)


def test_decode_layer_unrolled_equals_the_parallel_form_on_projected_inputs():
    """T steps of the layer, one position at a time, against Eq. 2's projections followed by the causal
    N x N definition (Eq. 8 with the feature-map kernel) and the output projection with its residual."""
    B, H, D, M, T = 3, 2, 4, 5, 9
    F = 6
    Wq, Wk, Wv, Wo = _layer_weights(F, H, D, M, 1)
    X = np.random.default_rng(2).standard_normal((B, T, F))
    S, Z = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    ys = np.stack([oracle.decode_layer_step(X[:, t], Wq, Wk, Wv, Wo, S, Z) for t in range(T)], 1)
    heads = lambda A, W, E: (A @ W).reshape(B, T, H, E).transpose(0, 2, 1, 3)
    O = oracle.attention_quadratic(heads(X, Wq, D), heads(X, Wk, D), heads(X, Wv, M), True)
    want = O.transpose(0, 2, 1, 3).reshape(B, T, H * M) @ Wo + X
    np.testing.assert_allclose(ys, want, rtol=1e-11, atol=1e-12)


def test_decode_layer_special_cases():
    B, H, D, M, F = 2, 2, 3, 3, 6
    Wq, Wk, Wv, Wo = _layer_weights(F, H, D, M, 3)
    x = np.random.default_rng(4).standard_normal((B, F))
    # a zero output projection leaves the residual alone, and the state still advances by phi(k) v^T
    S, Z = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    y = oracle.decode_layer_step(x, Wq, Wk, Wv, np.zeros_like(Wo), S, Z)
    np.testing.assert_array_equal(y, x)
    k, v = (x @ Wk).reshape(B, H, D), (x @ Wv).reshape(B, H, M)
    np.testing.assert_allclose(S, oracle.feature_map(k)[..., None] * v[:, :, None, :], rtol=1e-13)
    np.testing.assert_allclose(Z, oracle.feature_map(k), rtol=1e-13)
    # identity projections (F = H D = H M): the layer is the bare recurrent step plus the residual, and the
    # first step of a fresh sequence returns its own value (O_1 = V_1), so y = 2 x
    I = np.eye(F)
    S, Z = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    np.testing.assert_allclose(oracle.decode_layer_step(x, I, I, I, I, S, Z), 2 * x, rtol=1e-13)
    # by hand: one stream, one head, D = M = 1, all weights 1/2, x = (2): q = k = v = 1, phi = 2,
    # s = 2 * 1 = 2, z = 2, a = (2 * 2) / (2 * 2) = 1, y = 1 * 1/2 + 2 = 5/2; second step x = (-2): q = k = v = -1,
    # phi = e^-1, s = 2 - e^-1, z = 2 + e^-1, a = s / z, y = a / 2 - 2
    S, Z = np.zeros((1, 1, 1, 1)), np.zeros((1, 1, 1))
    h = np.full((1, 1), 0.5)
    assert oracle.decode_layer_step(np.array([[2.0]]), h, h, h, h, S, Z)[0, 0] == 2.5
    e = np.exp(-1.0)
    y2 = oracle.decode_layer_step(np.array([[-2.0]]), h, h, h, h, S, Z)[0, 0]
    np.testing.assert_allclose(y2, 0.5 * (2 - e) / (2 + e) - 2, rtol=1e-14)


# ---------------------------------------------------------------------------
# Random Fourier features (the conclusion's "approximating the RBF kernel with random Fourier features")
# ---------------------------------------------------------------------------
def test_rff_hand_example_norm_and_shift_invariance():
    # D = 1, one frequency pi/2, x = 1: z = pi/2, phi = sqrt(2/2) [cos z, sin z] = [0, 1]
    y = oracle.rff_feature_map([1.0], [[np.pi / 2]])
    assert abs(y[0]) < 1e-15 and y[1] == 1.0
    # two frequencies 0 and pi at x = 1: sqrt(1/2) [cos 0, cos pi, sin 0, sin pi] = [s, -s, 0, 0]
    y = oracle.rff_feature_map([1.0], [[0.0], [np.pi]])
    s = 0.5 ** 0.5
    assert np.allclose(y, [s, -s, 0.0, 0.0], atol=1e-15)
    rng = np.random.default_rng(5)
    W = rng.standard_normal((24, 6))
    x, yv, shift = rng.standard_normal((3, 7, 6))
    fx, fy = oracle.rff_feature_map(x, W), oracle.rff_feature_map(yv, W)
    # |phi(x)| = 1 whatever x and W are (cos^2 + sin^2 per frequency)
    assert np.allclose((fx ** 2).sum(-1), 1.0, atol=1e-14)
    # phi(x) . phi(y) = (2/C) sum_c cos(w_c . (x - y)): a function of the difference alone
    direct = np.cos((x - yv) @ W.T).mean(-1)
    assert np.allclose((fx * fy).sum(-1), direct, atol=1e-14)
    moved = (oracle.rff_feature_map(x + shift, W) * oracle.rff_feature_map(yv + shift, W)).sum(-1)
    assert np.allclose(moved, direct, atol=1e-13)


def test_rff_approximates_the_gaussian_kernel_within_its_sampling_error():
    """With w_c ~ N(0, I) the mean of cos(w . d) is exp(-|d|^2 / 2) and its variance is below 1/2 per frequency:
    20000 frequencies give a standard error below 0.005; five of them is the bound held here."""
    rng = np.random.default_rng(6)
    D, half = 4, 20000
    W = rng.standard_normal((half, D))
    x, y = rng.standard_normal((2, 16, D)) * 0.7
    approx = (oracle.rff_feature_map(x, W) * oracle.rff_feature_map(y, W)).sum(-1)
    exact = np.exp(-((x - y) ** 2).sum(-1) / 2)
    assert np.abs(approx - exact).max() < 5 * (0.5 / half) ** 0.5


def test_rff_backward_matches_finite_differences():
    rng = np.random.default_rng(7)
    W = rng.standard_normal((5, 3))
    x = rng.standard_normal((4, 3))
    dy = rng.standard_normal((4, 10))
    dx = oracle.rff_feature_map_backward(x, W, dy)
    h = 1e-6
    for i in range(4):
        for j in range(3):
            xp, xm = x.copy(), x.copy()
            xp[i, j] += h
            xm[i, j] -= h
            fd = ((oracle.rff_feature_map(xp, W) - oracle.rff_feature_map(xm, W)) * dy).sum() / (2 * h)
            assert abs(fd - dx[i, j]) < 1e-7 * max(1.0, abs(fd))
    # a frequency of zero contributes a constant feature: no gradient through it
    assert np.allclose(oracle.rff_feature_map_backward(x, np.zeros((5, 3)), dy), 0.0)
