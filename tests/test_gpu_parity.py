"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle, element by element."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2006_16236_b200 as la
from paper_2006_16236_b200.inputs import WORKLOADS, draw_qkvg, draw_workload
from parity import assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def gpu(*ts):
    return [None if t is None else t.to(DEV) for t in ts]


# shapes: (B, H, N, D, M); chosen to span several chunks and a ragged tail, N < chunk, D != M
SHAPES = [(1, 2, 256, 32, 32), (2, 3, 100, 16, 48), (1, 1, 1, 8, 8), (1, 2, 31, 64, 64),
          (2, 2, 33, 24, 40), (1, 2, 517, 128, 128), (1, 4, 384, 64, 64), (2, 2, 640, 32, 32)]
DTYPES = [torch.float32, torch.bfloat16]


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("n", [0, 1, 7, 8, 1000, 65536 + 3, 5 * 2 ** 20 + 13])
def test_feature_map(dtype, n):
    x = (torch.randn(n, generator=torch.Generator().manual_seed(n)) * 3).to(dtype)
    for deriv in (False, True):
        y = la.la_feature_map(x.to(DEV), deriv=deriv)
        assert_close(y, oracle.feature_map(x, deriv), dtype, "feature map")
    if n:
        xi = x.to(DEV)
        la.la_feature_map(xi, out=xi)                       # in place
        assert_close(xi, oracle.feature_map(x), dtype, "feature map in place")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES)
def test_causal_forward_backward(shape, dtype):
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=sum(shape), dtype=dtype)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    den = torch.empty((B, H, N), device=DEV)
    S = torch.empty((B, H, D, M), device=DEV)
    Z = torch.empty((B, H, D), device=DEV)
    O = la.la_causal_forward(Qd, Kd, Vd, den=den, S_out=S, Z_out=Z)
    Or, denr, Sr, Zr = oracle.linear_attention(Q, K, V, True, return_state=True)
    assert_close(O, Or, dtype, "O")
    assert_close(den, denr, dtype, "den")
    assert_close(S, Sr, dtype, "S_N")
    assert_close(Z, Zr, dtype, "Z_N")
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd)
    rq, rk, rv = oracle.linear_attention_backward(Q, K, V, G, True)
    assert_close(dQ, rq, dtype, "dQ", grad=True)
    assert_close(dK, rk, dtype, "dK", grad=True)
    assert_close(dV, rv, dtype, "dV", grad=True)
    la.la_last_device_status()


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES)
def test_noncausal_forward_backward(shape, dtype):
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=1 + sum(shape), dtype=dtype, scale=0.5)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    den = torch.empty((B, H, N), device=DEV)
    KV = torch.empty((B, H, D, M), device=DEV)
    Zs = torch.empty((B, H, D), device=DEV)
    O = la.la_linear_attention(Qd, Kd, Vd, den=den, KV=KV, Zs=Zs)
    Or, denr, Sr, Zr = oracle.linear_attention(Q, K, V, False, return_state=True)
    assert_close(O, Or, dtype, "O")
    assert_close(den, denr, dtype, "den")
    assert_close(KV, Sr, dtype, "KV")
    assert_close(Zs, Zr, dtype, "Zs")
    dQ, dK, dV = la.la_linear_attention_backward(Qd, Kd, Vd, Gd)
    rq, rk, rv = oracle.linear_attention_backward(Q, K, V, G, False)
    assert_close(dQ, rq, dtype, "dQ", grad=True)
    assert_close(dK, rk, dtype, "dK", grad=True)
    assert_close(dV, rv, dtype, "dV", grad=True)
    la.la_last_device_status()


@pytest.fixture
def plan_override():
    """la_plan_override() for one test; the automatic plans are restored afterwards."""
    yield la.la_plan_override
    la.la_plan_override()


@pytest.mark.parametrize("plan", [{"causal_pieces": 1}, {"causal_pieces": 3}, {"causal_pieces": 5}, {"causal_short": 0},
                                  {"causal_short": 4}, {"causal_short": 7}],
                         ids=lambda d: ",".join(f"{k[7:]}={v}" for k, v in d.items()))
@pytest.mark.parametrize("keep", [False, True], ids=["recompute", "saved"])
def test_causal_results_do_not_depend_on_the_piece_plan(plan_override, plan, keep):
    """The cut of a sequence into pieces and pre-pass parts (ragged lengths, a short middle piece, one piece)
    is an implementation choice: every plan has to give the oracle's result.  B*H = 64, 18 chunks."""
    plan_override(**plan)
    B, H, N, D = 4, 16, 18 * 128, 64
    p = la.make_problem(B, H, N, D, D, la.LA_BF16)
    pl = la.la_causal_plan(p)
    if "causal_pieces" in plan:
        assert pl["pieces"] == plan["causal_pieces"]
    else:
        short = plan["causal_short"]
        assert pl["pieces"] == (3 if short >= 4 else 2)
        if short >= 4:
            assert pl["piece_begin"][2] - pl["piece_begin"][1] == short
    Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=77, dtype=torch.bfloat16)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    saved = la.saved_buffer(Qd, Vd) if keep else None
    O = la.la_causal_forward(Qd, Kd, Vd, saved=saved)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, saved=saved)
    la.la_last_device_status()
    for b, h in ((0, 0), (1, 7), (3, 15)):
        sl = (slice(b, b + 1), slice(h, h + 1))
        q, k, v, g = Q[sl], K[sl], V[sl], G[sl]
        assert_close(O[sl], oracle.linear_attention(q, k, v, True)[0], torch.bfloat16, f"O[{b},{h}]")
        rq, rk, rv = oracle.linear_attention_backward(q, k, v, g, True)
        assert_close(dQ[sl], rq, torch.bfloat16, f"dQ[{b},{h}]", grad=True)
        assert_close(dK[sl], rk, torch.bfloat16, f"dK[{b},{h}]", grad=True)
        assert_close(dV[sl], rv, torch.bfloat16, f"dV[{b},{h}]", grad=True)


def test_backward_refuses_a_saved_buffer_of_another_plan(plan_override):
    """The saved buffer carries the plan of the forward pass that filled it.  A backward pass under another
    plan would look for the pre-pass records at other offsets: it reports the mismatch and computes nothing."""
    if os.environ.get("LA_DEBUG"):
        pytest.skip("in checked mode the call itself reads the status and raises; this test reads it afterwards")
    B, H, N, D = 4, 16, 18 * 128, 64
    Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=78, dtype=torch.bfloat16)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    p = la.make_problem(B, H, N, D, D, la.LA_BF16)
    need = []
    for pieces in (2, 3):
        plan_override(causal_pieces=pieces)
        need.append(la.la_workspace_bytes(p, la.LA_OP_CAUSAL_SAVED))
    saved = torch.empty(max(need), dtype=torch.uint8, device=DEV)       # large enough under either plan
    la.la_causal_forward(Qd, Kd, Vd, saved=saved)                       # ... filled under the plan of three pieces
    plan_override(causal_pieces=2)
    dQ = torch.full_like(Qd, 7.0)
    la.la_causal_backward(Qd, Kd, Vd, Gd, saved=saved, dQ=dQ)
    with pytest.raises(la.LaError) as e:
        la.la_last_device_status()
    assert e.value.status == -1 and "plan" in str(e.value)
    assert torch.all(dQ == 7.0)                 # the forward sweep wrote nothing
    la.la_last_device_status()                  # the flag is cleared, the context usable
    plan_override(causal_pieces=3)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, saved=saved)
    la.la_last_device_status()
    sl = (slice(1, 2), slice(5, 6))
    rq, rk, rv = oracle.linear_attention_backward(Q[sl], K[sl], V[sl], G[sl], True)
    assert_close(dQ[sl], rq, torch.bfloat16, "dQ", grad=True)
    assert_close(dK[sl], rk, torch.bfloat16, "dK", grad=True)
    assert_close(dV[sl], rv, torch.bfloat16, "dV", grad=True)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("dtype", DTYPES)
def test_eps_and_identity_feature_map(causal, dtype):
    B, H, N, D, M = 2, 2, 96, 32, 16
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=77, dtype=torch.float32)
    Q, K = (Q.abs() + 0.1).to(dtype), (K.abs() + 0.1).to(dtype)      # already "feature-mapped"
    V, G = V.to(dtype), G.to(dtype)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    fwd = la.la_causal_forward if causal else la.la_linear_attention
    bwd = la.la_causal_backward if causal else la.la_linear_attention_backward
    O = fwd(Qd, Kd, Vd, phi="identity", eps=0.75)
    assert_close(O, oracle.linear_attention(Q, K, V, causal, "identity", 0.75)[0], dtype, "O")
    grads = bwd(Qd, Kd, Vd, Gd, phi="identity", eps=0.75)
    for g, r, nm in zip(grads, oracle.linear_attention_backward(Q, K, V, G, causal, "identity", 0.75), "QKV"):
        assert_close(g, r, dtype, "d" + nm, grad=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(2, 3, 40, 64, 64), (1, 2, 24, 32, 32), (2, 2, 17, 16, 24), (1, 2, 9, 128, 64)])
def test_recurrent_steps_equal_causal_form(shape, dtype):
    B, H, N, D, M = shape
    Q, K, V, _ = draw_qkvg(B, H, N, D, M, seed=5 + sum(shape), dtype=dtype, with_grad=False)
    Qd, Kd, Vd = gpu(Q, K, V)
    ref = oracle.attention_quadratic(Q, K, V, True)
    S = torch.zeros((B, H, D, M), device=DEV)
    Z = torch.zeros((B, H, D), device=DEV)
    So, Zo = np.zeros((B, H, D, M)), np.zeros((B, H, D))
    outs = []
    for i in range(N):
        out = la.la_recurrent_step(Qd[:, :, i].contiguous(), Kd[:, :, i].contiguous(), Vd[:, :, i].contiguous(), S, Z)
        step_ref = oracle.recurrent_step(Q[:, :, i], K[:, :, i], V[:, :, i], So, Zo)
        assert_close(out, step_ref, dtype, f"step {i}")
        outs.append(out)
    assert_close(torch.stack(outs, 2), ref, dtype, "steps vs quadratic form")
    assert_close(S, So, dtype, "S")
    assert_close(Z, Zo, dtype, "Z")
    # the parallel form on the same sequence, and its final state, agree with the steps
    S2 = torch.empty_like(S)
    Z2 = torch.empty_like(Z)
    O = la.la_causal_forward(Qd, Kd, Vd, S_out=S2, Z_out=Z2)
    assert_close(O, torch.stack(outs, 2).double().cpu().numpy(), dtype, "parallel vs steps")
    assert_close(S2, So, dtype, "S_N of the parallel form")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(2, 3, 1, 64, 64), (2, 3, 40, 64, 64), (1, 2, 24, 32, 32), (2, 2, 17, 16, 24), (1, 2, 9, 128, 64),
                                   (3, 5, 130, 32, 64)])
def test_recurrent_steps_in_one_launch(shape, dtype):
    """N recurrent steps in one launch: bit-identical to N single-step launches, and equal to the oracle's
    recurrence from the same non-zero state."""
    B, H, N, D, M = shape
    Q, K, V, _ = draw_qkvg(B, H, N, D, M, seed=sum(shape) + 3, dtype=dtype, with_grad=False)
    g = torch.Generator().manual_seed(8)
    S0 = torch.randn((B, H, D, M), generator=g) * 2.0
    Z0 = torch.rand((B, H, D), generator=g) * 3.0 + 1.0
    Qd, Kd, Vd = gpu(Q, K, V)
    S, Z = S0.to(DEV), Z0.to(DEV)
    out = la.la_recurrent_steps(Qd, Kd, Vd, S, Z)
    S1, Z1 = S0.to(DEV), Z0.to(DEV)
    one = [la.la_recurrent_step(Qd[:, :, t].contiguous(), Kd[:, :, t].contiguous(), Vd[:, :, t].contiguous(), S1, Z1)
           for t in range(N)]
    la.la_last_device_status()
    assert torch.equal(out, torch.stack(one, dim=2)) and torch.equal(S, S1) and torch.equal(Z, Z1)
    Or, _, Sr, Zr = oracle.causal_from_state(Q, K, V, S0.double().numpy(), Z0.double().numpy())
    assert_close(out, Or, dtype, "out")
    assert_close(S, Sr, dtype, "S_N")
    assert_close(Z, Zr, dtype, "Z_N")


def test_prefill_then_decode_handoff():
    B, H, N, D, M = 2, 2, 64, 32, 32
    Q, K, V, _ = draw_qkvg(B, H, N + 1, D, M, seed=9, dtype=torch.float32, with_grad=False)
    Qd, Kd, Vd = gpu(Q, K, V)
    S = torch.empty((B, H, D, M), device=DEV)
    Z = torch.empty((B, H, D), device=DEV)
    la.la_causal_forward(Qd[:, :, :N].contiguous(), Kd[:, :, :N].contiguous(), Vd[:, :, :N].contiguous(),
                         S_out=S, Z_out=Z)
    out = la.la_recurrent_step(Qd[:, :, N].contiguous(), Kd[:, :, N].contiguous(), Vd[:, :, N].contiguous(), S, Z)
    ref = oracle.attention_quadratic(Q, K, V, True)[:, :, N]
    assert_close(out, ref, torch.float32, "decode after prefill")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(2, 3, 100, 16, 48), (1, 2, 31, 64, 64), (2, 2, 640, 32, 32), (1, 4, 384, 64, 64),
                                   (4, 16, 18 * 128, 64, 64), (2, 8, 1000, 64, 64)])
def test_causal_forward_from_a_state(shape, dtype):
    """The recurrence of Eq. 16-20 started from a given S_0, Z_0 (general kernels and, for bf16 D = M in
    {32, 64}, the tensor-core kernel, with several pieces per sequence at the larger shapes)."""
    B, H, N, D, M = shape
    Q, K, V, _ = draw_qkvg(B, H, N, D, M, seed=sum(shape) + 1, dtype=dtype, with_grad=False)
    g = torch.Generator().manual_seed(5)
    S0 = torch.randn((B, H, D, M), generator=g) * 3.0
    Z0 = torch.rand((B, H, D), generator=g) * 4.0 + 1.0
    Qd, Kd, Vd, S0d, Z0d = gpu(Q, K, V, S0, Z0)
    den = torch.empty((B, H, N), device=DEV)
    S = torch.empty((B, H, D, M), device=DEV)
    Z = torch.empty((B, H, D), device=DEV)
    O = la.la_causal_forward(Qd, Kd, Vd, den=den, S_out=S, Z_out=Z, S_in=S0d, Z_in=Z0d)
    la.la_last_device_status()
    sel = [(0, 0), (B - 1, H - 1)] if B * H > 8 else [(b, h) for b in range(B) for h in range(H)]
    for b, h in sel:
        sl = (slice(b, b + 1), slice(h, h + 1))
        Or, denr, Sr, Zr = oracle.causal_from_state(Q[sl], K[sl], V[sl], S0[sl].double().numpy(), Z0[sl].double().numpy())
        assert_close(O[sl], Or, dtype, f"O[{b},{h}]")
        assert_close(den[sl], denr, dtype, f"den[{b},{h}]")
        assert_close(S[sl], Sr, dtype, f"S_N[{b},{h}]")
        assert_close(Z[sl], Zr, dtype, f"Z_N[{b},{h}]")
    assert torch.equal(S0d.cpu(), S0) and torch.equal(Z0d.cpu(), Z0)        # the given state is only read


@pytest.mark.parametrize("dtype,D,chunks", [(torch.float32, 32, (100, 60, 96)), (torch.bfloat16, 64, (1024, 512, 2560))])
def test_chunked_prefill_then_decode(dtype, D, chunks):
    """A sequence processed in three calls, each continuing from the state the previous one returned, then one
    recurrent step: every output equals the definition on the whole sequence."""
    B, H = 2, 2
    N = sum(chunks)
    Q, K, V, _ = draw_qkvg(B, H, N + 1, D, D, seed=19, dtype=dtype, with_grad=False)
    Qd, Kd, Vd = gpu(Q, K, V)
    S = [torch.zeros((B, H, D, D), device=DEV), torch.empty((B, H, D, D), device=DEV)]
    Z = [torch.zeros((B, H, D), device=DEV), torch.empty((B, H, D), device=DEV)]
    outs, lo = [], 0
    for i, n in enumerate(chunks):
        sl = slice(lo, lo + n)
        outs.append(la.la_causal_forward(Qd[:, :, sl].contiguous(), Kd[:, :, sl].contiguous(), Vd[:, :, sl].contiguous(),
                                         S_in=S[i & 1], Z_in=Z[i & 1], S_out=S[(i + 1) & 1], Z_out=Z[(i + 1) & 1]))
        lo += n
    k = len(chunks) & 1
    last = la.la_recurrent_step(Qd[:, :, N].contiguous(), Kd[:, :, N].contiguous(), Vd[:, :, N].contiguous(), S[k], Z[k])
    la.la_last_device_status()
    ref = oracle.linear_attention(Q, K, V, True)[0]
    assert_close(torch.cat(outs, dim=2), ref[:, :, :N], dtype, "chunked prefill")
    assert_close(last, ref[:, :, N], dtype, "decode after chunked prefill")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("keep", [False, True], ids=["recompute", "saved"])
@pytest.mark.parametrize("shape", [(2, 3, 100, 16, 48), (1, 2, 31, 64, 64), (2, 2, 640, 32, 32), (4, 16, 18 * 128, 64, 64),
                                   (2, 8, 1000, 64, 64)])
def test_causal_backward_from_a_state(shape, keep, dtype):
    """Algorithm 1 (backward) with the forward sum started from [S_0 | Z_0] and the reverse sum from an upstream
    gradient of the final state; the gradient of the initial state is what the reverse sum ends with."""
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=sum(shape) + 2, dtype=dtype)
    g = torch.Generator().manual_seed(6)
    S0 = torch.randn((B, H, D, M), generator=g) * 3.0
    Z0 = torch.rand((B, H, D), generator=g) * 4.0 + 1.0
    dSN = torch.randn((B, H, D, M), generator=g) * 0.05
    dZN = torch.randn((B, H, D), generator=g) * 0.05
    Qd, Kd, Vd, Gd, S0d, Z0d, dSNd, dZNd = gpu(Q, K, V, G, S0, Z0, dSN, dZN)
    dS0 = torch.empty((B, H, D, M), device=DEV)
    dZ0 = torch.empty((B, H, D), device=DEV)
    saved = la.saved_buffer(Qd, Vd) if keep else None
    if keep and saved is None:
        pytest.skip("no saved buffer for problems on the general kernels")
    if keep:
        la.la_causal_forward(Qd, Kd, Vd, S_in=S0d, Z_in=Z0d, saved=saved)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, saved=saved, S_in=S0d, Z_in=Z0d, dS_out=dSNd, dZ_out=dZNd,
                                       dS_in=dS0, dZ_in=dZ0)
    la.la_last_device_status()
    sel = [(0, 0), (B - 1, H - 1)] if B * H > 8 else [(b, h) for b in range(B) for h in range(H)]
    for b, h in sel:
        sl = (slice(b, b + 1), slice(h, h + 1))
        rq, rk, rv, rS, rZ = oracle.causal_backward_from_state(
            Q[sl], K[sl], V[sl], S0[sl].double().numpy(), Z0[sl].double().numpy(), G[sl],
            dSN[sl].double().numpy(), dZN[sl].double().numpy())
        assert_close(dQ[sl], rq, dtype, f"dQ[{b},{h}]", grad=True)
        assert_close(dK[sl], rk, dtype, f"dK[{b},{h}]", grad=True)
        assert_close(dV[sl], rv, dtype, f"dV[{b},{h}]", grad=True)
        assert_close(dS0[sl], rS, dtype, f"dS_0[{b},{h}]", grad=True)
        assert_close(dZ0[sl], rZ, dtype, f"dZ_0[{b},{h}]", grad=True)


def test_backward_chained_over_two_calls():
    """A sequence processed and differentiated in two calls (the state and its gradient handed across) against
    the oracle's gradient of the whole sequence."""
    B, H, N, D, cut = 2, 4, 3072, 64, 1280
    Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=23, dtype=torch.bfloat16)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    a, b = slice(0, cut), slice(cut, N)
    part = lambda t, s: t[:, :, s].contiguous()
    S1 = torch.empty((B, H, D, D), device=DEV)
    Z1 = torch.empty((B, H, D), device=DEV)
    dS1, dZ1 = torch.empty_like(S1), torch.empty_like(Z1)
    la.la_causal_forward(part(Qd, a), part(Kd, a), part(Vd, a), S_out=S1, Z_out=Z1)
    q2, k2, v2 = la.la_causal_backward(part(Qd, b), part(Kd, b), part(Vd, b), part(Gd, b), S_in=S1, Z_in=Z1, dS_in=dS1, dZ_in=dZ1)
    q1, k1, v1 = la.la_causal_backward(part(Qd, a), part(Kd, a), part(Vd, a), part(Gd, a), dS_out=dS1, dZ_out=dZ1)
    la.la_last_device_status()
    rq, rk, rv = oracle.linear_attention_backward(Q, K, V, G, True)
    for got, ref, nm in ((torch.cat([q1, q2], 2), rq, "dQ"), (torch.cat([k1, k2], 2), rk, "dK"), (torch.cat([v1, v2], 2), rv, "dV")):
        assert_close(got, ref, torch.bfloat16, nm, grad=True)


@pytest.mark.parametrize("dtype,D,N", [(torch.float32, 32, 200), (torch.bfloat16, 64, 1024)])
def test_right_padded_causal_batches_need_no_mask(dtype, D, N):
    """Sequences of different lengths, padded on the right to one N (here with large junk): causality keeps
    the padding out of every real position's output, and an upstream gradient that is zero on the padding
    keeps it out of every real position's gradient and makes the padding's own gradients zero.  Each sequence
    is compared with the oracle run on its own length."""
    B, H = 3, 2
    lengths = [N, N - N // 3, 1 + N // 5]
    Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=29, dtype=dtype)
    for b, n in enumerate(lengths):
        Q[b, :, n:] = 7.0
        K[b, :, n:] = 9.0
        V[b, :, n:] = -50.0
        G[b, :, n:] = 0.0
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    O = la.la_causal_forward(Qd, Kd, Vd)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd)
    la.la_last_device_status()
    for b, n in enumerate(lengths):
        sl = (slice(b, b + 1), slice(None), slice(0, n))
        q, k, v, g = Q[sl], K[sl], V[sl], G[sl]
        assert_close(O[sl], oracle.linear_attention(q, k, v, True)[0], dtype, f"O, length {n}")
        rq, rk, rv = oracle.linear_attention_backward(q, k, v, g, True)
        assert_close(dQ[sl], rq, dtype, f"dQ, length {n}", grad=True)
        assert_close(dK[sl], rk, dtype, f"dK, length {n}", grad=True)
        assert_close(dV[sl], rv, dtype, f"dV, length {n}", grad=True)
        for t, nm in ((dQ, "dQ"), (dK, "dK"), (dV, "dV")):
            assert float(t[b, :, n:].float().abs().max()) == 0.0 if n < N else True, f"{nm} on the padding"


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape,lengths", [((3, 2, 100, 16, 48), [100, 37, 1]), ((4, 2, 517, 64, 64), [517, 0, 300, 129]),
                                           ((2, 4, 1024, 64, 64), [1024, 700]),
                                           ((5, 2, 2048, 64, 64), [2048, 0, 129, 1500, 1024]),
                                           ((3, 2, 512, 32, 32), [512, 130, 1])])
def test_noncausal_ragged_batches(shape, lengths, dtype):
    """Right-padded sequences of different lengths (key-padding mask): every sequence equals the oracle run on
    its own length, sums included, and everything is zero on the padding whatever the tensors hold there
    (not even numbers).  The bf16 cases with D = M in {32, 64} run the tensor-core
    kernels, whose splits end inside, at and before a sequence's end; the others the general kernels."""
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=sum(shape) + 4, dtype=dtype)
    for b, n in enumerate(lengths):
        Q[b, :, n:] = 5.0
        K[b, :, n:] = float("inf")
        V[b, :, n:] = -30.0
        G[b, :, n:] = float("nan")
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    ld = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    den = torch.empty((B, H, N), device=DEV)
    KV = torch.empty((B, H, D, M), device=DEV)
    Zs = torch.empty((B, H, D), device=DEV)
    O = la.la_linear_attention_varlen(Qd, Kd, Vd, ld, den=den, KV=KV, Zs=Zs)
    dQ, dK, dV = la.la_linear_attention_varlen_backward(Qd, Kd, Vd, Gd, ld)
    la.la_last_device_status()
    for b, n in enumerate(lengths):
        pad = (slice(b, b + 1), slice(None), slice(n, N))
        for t in (O, den, dQ, dK, dV):
            assert n == N or float(t[pad].float().abs().max()) == 0.0
        if n == 0:
            assert float(KV[b].abs().max()) == 0.0 and float(Zs[b].abs().max()) == 0.0
            continue
        sl = (slice(b, b + 1), slice(None), slice(0, n))
        q, k, v, g = Q[sl], K[sl], V[sl], G[sl]
        Or, denr, Sr, Zr = oracle.linear_attention(q, k, v, False, return_state=True)
        assert_close(O[sl], Or, dtype, f"O, length {n}")
        assert_close(den[sl], denr, dtype, f"den, length {n}")
        assert_close(KV[b:b + 1], Sr, dtype, f"KV, length {n}")
        assert_close(Zs[b:b + 1], Zr, dtype, f"Zs, length {n}")
        rq, rk, rv = oracle.linear_attention_backward(q, k, v, g, False)
        assert_close(dQ[sl], rq, dtype, f"dQ, length {n}", grad=True)
        assert_close(dK[sl], rk, dtype, f"dK, length {n}", grad=True)
        assert_close(dV[sl], rv, dtype, f"dV, length {n}", grad=True)


# --------------------------------------------------------------------------
# Degree-2 polynomial kernel (Section 3.2.1): explicit feature map + identity-mode attention.
# --------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("D,C", [(1, 8), (3, 16), (8, 64), (8, 72), (11, 128)])
def test_poly2_feature_map_and_its_gradient(D, C, dtype):
    rows = (3, 5, 67)                                   # 1005 rows: several blocks and a ragged tail
    g = torch.Generator().manual_seed(100 * D + C)
    x = torch.randn(rows + (D,), generator=g).to(dtype)
    dy = torch.randn(rows + (C,), generator=g).to(dtype)
    y = la.la_feature_map_poly2(x.to(DEV), C)
    dx = la.la_feature_map_poly2_backward(x.to(DEV), dy.to(DEV))
    ref = oracle.poly2_feature_map(x.double().numpy(), C)
    tol = 2.0 ** -23 if dtype == torch.float32 else 2.0 ** -8       # one rounding of an exact product
    got = y.double().cpu().numpy()
    assert got.shape == ref.shape
    assert np.all(np.abs(got - ref) <= tol * np.abs(ref)), np.abs(got - ref).max()
    assert np.all(got[..., D * D:] == 0.0)
    assert_close(dx, oracle.poly2_feature_map_backward(x.double().numpy(), dy.double().numpy()), dtype, "dx", grad=True)
    assert la.la_feature_map_poly2(torch.empty((0, D), dtype=dtype, device=DEV), C).shape == (0, C)


def test_poly2_feature_map_many_rows():
    """D = 8, C = 64 in bf16 has kernels of its own (several rows per thread in flight, the gradient rows staged
    through shared memory): enough rows for every block to loop, and a ragged end."""
    rows, D, C = 300001, 8, 64
    g = torch.Generator().manual_seed(77)
    x = torch.randn((rows, D), generator=g).to(torch.bfloat16)
    dy = torch.randn((rows, C), generator=g).to(torch.bfloat16)
    y = la.la_feature_map_poly2(x.to(DEV), C)
    dx = la.la_feature_map_poly2_backward(x.to(DEV), dy.to(DEV))
    ref = oracle.poly2_feature_map(x.double().numpy(), C)
    got = y.double().cpu().numpy()
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref)), np.abs(got - ref).max()
    assert_close(dx, oracle.poly2_feature_map_backward(x.double().numpy(), dy.double().numpy()), torch.bfloat16, "dx", grad=True)


@pytest.mark.parametrize("D,C,rows", [(64, 64, (3, 5, 67)), (64, 128, (2, 700)), (32, 64, (1000,)), (8, 128, (130,)), (64, 64, (40000,))],
                         ids=["D64_C64", "D64_C128", "D32_C64", "D8_C128", "D64_C64_many_tiles"])
def test_rff_feature_map_and_its_gradient(D, C, rows):
    """Random Fourier features on the tensor cores against the oracle: several row tiles per CTA, a ragged last
    tile, input widths below one K block (zero-filled by TMA) and both output widths."""
    g = torch.Generator().manual_seed(10 * D + C)
    x = torch.randn(rows + (D,), generator=g).to(torch.bfloat16)
    W = torch.randn((C // 2, D), generator=g).to(torch.bfloat16)
    dy = torch.randn(rows + (C,), generator=g).to(torch.bfloat16)
    y = la.la_feature_map_rff(x.to(DEV), W.to(DEV))
    dx = la.la_feature_map_rff_backward(x.to(DEV), W.to(DEV), dy.to(DEV))
    la.la_last_device_status()
    xr, Wr = x.double().numpy(), W.double().numpy()
    ref = oracle.rff_feature_map(xr, Wr)
    got = y.double().cpu().numpy()
    assert got.shape == ref.shape
    # every feature is below sqrt(2/C) in size: one bf16 rounding of that plus the fast sine's error
    assert np.abs(got - ref).max() <= (2.0 / C) ** 0.5 * 2.0 ** -8 * 1.5, np.abs(got - ref).max()
    assert_close(y, ref, torch.bfloat16, "rff y")
    assert_close(dx, oracle.rff_feature_map_backward(xr, Wr, dy.double().numpy()), torch.bfloat16, "rff dx", grad=True)
    # the same call again gives the same bits
    assert torch.equal(y, la.la_feature_map_rff(x.to(DEV), W.to(DEV)))
    assert la.la_feature_map_rff(torch.empty((0, D), dtype=torch.bfloat16, device=DEV), W.to(DEV)).shape == (0, C)


@pytest.mark.parametrize("causal", [False, True])
def test_rff_attention_end_to_end(causal):
    """Queries and keys -> random Fourier features on the device -> attention with the identity map (the general
    kernels: C = 128) and gradients back through both steps, against the oracle on the device's own features (a
    stored bf16 tensor, like every other input).  Small inputs and few positions per head keep the weights of
    Eq. 4, which are not guaranteed positive for signed features, away from zero."""
    B, H, N, D, C = 2, 2, 96, 64, 128
    Q, K, V, G = draw_qkvg(B, H, N, D, C, seed=77 + causal, dtype=torch.bfloat16)
    Q, K = (Q * 0.05).to(torch.bfloat16), (K * 0.05).to(torch.bfloat16)
    W = torch.randn((C // 2, D), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    Qd, Kd, Vd, Gd, Wd = gpu(Q, K, V, G, W)
    fQ, fK = la.la_feature_map_rff(Qd, Wd), la.la_feature_map_rff(Kd, Wd)
    fwd = la.la_causal_forward if causal else la.la_linear_attention
    bwd = la.la_causal_backward if causal else la.la_linear_attention_backward
    O = fwd(fQ, fK, Vd, phi="identity")
    dfQ, dfK, dV = bwd(fQ, fK, Vd, Gd, phi="identity")
    dQ, dK = la.la_feature_map_rff_backward(Qd, Wd, dfQ), la.la_feature_map_rff_backward(Kd, Wd, dfK)
    la.la_last_device_status()
    fq, fk = fQ.double().cpu().numpy(), fK.double().cpu().numpy()
    Vr, Gr, Wr = V.double().numpy(), G.double().numpy(), W.double().numpy()
    Oref = oracle.linear_attention(fq, fk, Vr, causal, phi="identity")[0]
    gq, gk, gv = oracle.linear_attention_backward(fq, fk, Vr, Gr, causal, phi="identity")
    assert_close(O, Oref, torch.bfloat16, "rff attention O")
    assert_close(dV, gv, torch.bfloat16, "rff attention dV", grad=True)
    # the map's gradient is judged on the upstream gradient the device handed it
    assert_close(dQ, oracle.rff_feature_map_backward(Q.double().numpy(), Wr, dfQ.double().cpu().numpy()), torch.bfloat16, "rff dQ", grad=True)
    assert_close(dK, oracle.rff_feature_map_backward(K.double().numpy(), Wr, dfK.double().cpu().numpy()), torch.bfloat16, "rff dK", grad=True)
    assert_close(dfQ, gq, torch.bfloat16, "rff attention dphi(Q)", grad=True)
    assert_close(dfK, gk, torch.bfloat16, "rff attention dphi(K)", grad=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape,signed", [((2, 2, 384, 8, 64), False), ((2, 2, 384, 8, 64), True),
                                          ((1, 3, 200, 5, 24), True)])
def test_poly2_attention_end_to_end(shape, signed, causal, dtype):
    """Queries and keys -> features on the device -> attention with the identity map; gradients through both
    steps.  D = 8 gives C = 64: in bf16 the tensor-core kernels; D = 5 (C = 25 padded to 32, M = 24) the
    general ones.  The features are a stored tensor of the I/O type: the device's must equal the oracle's,
    rounded once, bit for bit, and the attention step is judged on those, like every other input.  Against the
    exact kernel (q.k)^2 on the N x N matrix the fp32 path meets the fp32 gate; in bf16 the 2^-9 rounding
    of each stored feature is what remains (a weight (q.k)^2 is a sum of D^2 products that cancel), which
    no kernel downstream can remove: only a loose bound is asserted there.
    Signed queries and keys give signed features, and a weight that is small against the products it sums
    (the first causal rows above all).  The general kernels (fp32 arithmetic) hold the usual gates there; the
    tensor-core kernels round scores and state to bf16, an error relative to the products and not to their
    sum: for signed features in bf16 they are held to 0.15, and to the usual gates for features of one sign."""
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=sum(shape) + causal, dtype=dtype)
    if not signed:
        Q, K = Q.abs(), K.abs()
    loose = signed and dtype == torch.bfloat16 and D * D == 64 and M == 64           # tensor-core kernels

    def check(x, ref, what, grad=False):
        if loose:
            from parity import max_rel_err
            err = max_rel_err(x, ref)
            assert err < 0.15, f"{what}: {err:.3e}"
        else:
            assert_close(x, ref, dtype, what, grad=grad)

    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    fQ, fK = la.la_feature_map_poly2(Qd), la.la_feature_map_poly2(Kd)
    fwd = la.la_causal_forward if causal else la.la_linear_attention
    bwd = la.la_causal_backward if causal else la.la_linear_attention_backward
    O = fwd(fQ, fK, Vd, phi="identity")
    dfQ, dfK, dV = bwd(fQ, fK, Vd, Gd, phi="identity")
    dQ, dK = la.la_feature_map_poly2_backward(Qd, dfQ), la.la_feature_map_poly2_backward(Kd, dfK)
    la.la_last_device_status()
    q, k, v, g = (t.double().numpy() for t in (Q, K, V, G))
    C = fQ.shape[-1]
    rounded = lambda a: torch.from_numpy(a).to(dtype).double().numpy()
    rq, rk = rounded(oracle.poly2_feature_map(q, C)), rounded(oracle.poly2_feature_map(k, C))
    assert np.array_equal(fQ.double().cpu().numpy(), rq) and np.array_equal(fK.double().cpu().numpy(), rk)
    check(O, oracle.linear_attention(rq, rk, v, causal, "identity")[0], "O")
    exact = oracle.poly2_attention(q, k, v, causal)
    if dtype == torch.float32:
        assert_close(O, exact, dtype, "O against the exact kernel")
    else:
        from parity import max_rel_err
        assert max_rel_err(O, exact) < 0.2
    rfq, rfk, rv = oracle.linear_attention_backward(rq, rk, v, g, causal, "identity")
    check(dV, rv, "dV", grad=True)
    check(dQ, oracle.poly2_feature_map_backward(q, rounded(rfq)), "dQ", grad=True)
    check(dK, oracle.poly2_feature_map_backward(k, rounded(rfk)), "dK", grad=True)


def test_gradient_invariants_hold_on_gpu_results():
    B, H, N, D, M = 2, 4, 512, 64, 64
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=11, dtype=torch.float32)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    for bwd in (la.la_causal_backward, la.la_linear_attention_backward):
        dQ, dK, dV = bwd(Qd, Kd, Vd, Gd)
        assert torch.allclose(dV.sum(2), Gd.sum(2), rtol=1e-3, atol=1e-3)           # rows sum to one
        ratio = torch.where(Qd > 0, Qd + 1, torch.ones_like(Qd))                    # phi / phi'
        assert (ratio * dQ).sum(-1).abs().max() < 1e-3                              # degree-0 in phi(Q_i)


# --------------------------------------------------------------------------
# Full-size workloads, in the launch configuration the benchmark times; the
# oracle recomputes a sample of (batch, head) pairs, which are independent.
# --------------------------------------------------------------------------
def _sample_heads(B, H, k=3):
    pairs = [(0, 0), (B - 1, H - 1), (B // 2, H // 2)]
    return list(dict.fromkeys(pairs))[:k]


@pytest.mark.parametrize("name", ["causal_fp32_small", "causal_bf16_image", "causal_sweep_bf16_N4096",
                                  "causal_sweep_bf16_N8192", "causal_sweep_bf16_N16384",
                                  "causal_sweep_bf16_N32768", "causal_sweep_bf16_N65536", "causal_fp32_N4096"])
@pytest.mark.parametrize("keep", [False, True], ids=["recompute", "saved"])
def test_causal_workloads_full_size(name, keep):
    w = WORKLOADS[name]
    dtype = w.torch_dtype
    Q, K, V, G = draw_workload(w)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    den = torch.empty((w.B, w.H, w.N), device=DEV)
    saved = la.saved_buffer(Qd, Vd) if keep else None      # what a training step keeps for the backward pass
    if keep and saved is None:
        pytest.skip("this problem runs the general kernels, which keep nothing")
    O = la.la_causal_forward(Qd, Kd, Vd, den=den, saved=saved)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, O=O, den=den, saved=saved)
    la.la_last_device_status()
    for b, h in _sample_heads(w.B, w.H):
        sl = (slice(b, b + 1), slice(h, h + 1))
        q, k, v, g = Q[sl], K[sl], V[sl], G[sl]
        Or, denr = oracle.linear_attention(q, k, v, True)
        # unit-scale inputs: no row of any reference tensor is small by chance, so every row is also held to
        # the tolerance against itself alone (no neighbourhood floor)
        assert_close(O[sl], Or, dtype, f"{name} O[{b},{h}]", gate_row=True)
        assert_close(den[sl], denr, dtype, f"{name} den[{b},{h}]", gate_row=True)
        for got, ref, nm in zip((dQ, dK, dV), oracle.linear_attention_backward(q, k, v, g, True), "QKV"):
            assert_close(got[sl], ref, dtype, f"{name} d{nm}[{b},{h}]", grad=True, gate_row=True)
    # size-independent properties on the whole result
    assert torch.isfinite(O.float()).all() and torch.isfinite(dQ.float()).all()
    assert torch.allclose(O[:, :, 0].float(), Vd[:, :, 0].float(), rtol=1e-2, atol=1e-2)     # O_1 = V_1
    assert torch.allclose(dV.float().sum(2), Gd.float().sum(2), rtol=5e-2, atol=0.5 * (w.N ** 0.5) * 2e-2 + 0.5)


@pytest.mark.parametrize("name", ["causal_sweep_bf16_N8192", "causal_sweep_bf16_N32768", "noncausal_bf16_speech"])
def test_results_are_repeatable_bit_for_bit(name):
    """No atomics and a fixed summation order: repeated calls give identical bits.  A difference
    between repeats means one warp role read a buffer while another was still writing it."""
    w = WORKLOADS[name]
    Q, K, V, G = gpu(*draw_workload(w))
    fwd = la.la_causal_forward if w.kind == "causal" else la.la_linear_attention
    bwd = la.la_causal_backward if w.kind == "causal" else la.la_linear_attention_backward
    first = None
    for _ in range(6):
        cur = [fwd(Q, K, V)] + list(bwd(Q, K, V, G))
        la.la_last_device_status()
        if first is None:
            first = [t.clone() for t in cur]
        else:
            for a, b, nm in zip(first, cur, ("O", "dQ", "dK", "dV")):
                assert torch.equal(a, b), f"{name}: {nm} differs between repeats"


@pytest.mark.parametrize("shape", [(2, 2, 1024, 64), (1, 3, 384, 32), (3, 50, 2048, 64)])
def test_saved_buffer_matches_recomputation(shape):
    """The forward's saved phi(Q), phi(K) are the bf16 feature maps of Q and K, the forward's own result
    does not depend on saving them, dQ (whose operands are identical on both paths) is bit-identical, and
    dK, dV agree to rounding."""
    B, H, N, D = shape
    Q, K, V, G = gpu(*draw_qkvg(B, H, N, D, D, 91, torch.bfloat16, 1.0))
    saved = la.saved_buffer(Q, V)
    assert saved is not None and saved.numel() >= 2 * Q.numel() * 2
    saved.fill_(0xFF)
    O1 = la.la_causal_forward(Q, K, V, saved=saved)
    O0 = la.la_causal_forward(Q, K, V)
    assert torch.equal(O0, O1)
    rows = B * H * N
    stride = (rows * D * 2 + 1023) // 1024 * 1024
    phiq = saved[: rows * D * 2].view(torch.bfloat16).view(B, H, N, D)
    phik = saved[stride: stride + rows * D * 2].view(torch.bfloat16).view(B, H, N, D)
    for got, x in ((phiq, Q), (phik, K)):
        ref = oracle.feature_map(x.double().cpu().numpy())
        err = (got.double().cpu().numpy() - ref) / ref
        assert abs(err).max() <= 2.0 ** -8, abs(err).max()
    g0 = la.la_causal_backward(Q, K, V, G)
    g1 = la.la_causal_backward(Q, K, V, G, saved=saved)
    la.la_last_device_status()
    assert torch.equal(g0[0], g1[0]), "dQ differs"
    for a, b, nm in zip(g0[1:], g1[1:], "KV"):
        ref = a.double().cpu().numpy()
        assert_close(b, ref, torch.bfloat16, f"d{nm} saved vs recomputed", grad=True)


def test_noncausal_workload_full_size():
    w = WORKLOADS["noncausal_bf16_speech"]
    dtype = w.torch_dtype
    Q, K, V, G = draw_workload(w)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    O = la.la_linear_attention(Qd, Kd, Vd)
    dQ, dK, dV = la.la_linear_attention_backward(Qd, Kd, Vd, Gd)
    la.la_last_device_status()
    for b, h in _sample_heads(w.B, w.H):
        sl = (slice(b, b + 1), slice(h, h + 1))
        q, k, v, g = Q[sl], K[sl], V[sl], G[sl]
        assert_close(O[sl], oracle.linear_attention(q, k, v, False)[0], dtype, f"O[{b},{h}]")
        for got, ref, nm in zip((dQ, dK, dV), oracle.linear_attention_backward(q, k, v, g, False), "QKV"):
            assert_close(got[sl], ref, dtype, f"d{nm}[{b},{h}]", grad=True)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape,lengths", [((2, 3, 512, 64, 64), None), ((3, 2, 1024, 64, 64), [1024, 130, 700]),
                                           ((2, 2, 200, 16, 24), None), ((2, 2, 200, 16, 24), [200, 77])])
def test_noncausal_saved_sums_give_identical_results(shape, lengths, dtype):
    """What the non-causal forward keeps for the backward pass (the per-split sums over the keys) changes no bit
    of either call's results, on the tensor-core and on the general kernels, full-length and ragged; and the
    forward leaves its workspace alone when it is given a saved buffer."""
    B, H, N, D, M = shape
    Q, K, V, G = gpu(*draw_qkvg(B, H, N, D, M, seed=sum(shape) + 9, dtype=dtype))
    ld = None if lengths is None else torch.tensor(lengths, dtype=torch.int32, device=DEV)
    saved = la.linear_saved_buffer(Q, V)
    assert saved is not None and saved.numel() > 0
    O0 = la.la_linear_attention(Q, K, V, lengths=ld)
    g0 = la.la_linear_attention_backward(Q, K, V, G, lengths=ld)
    saved.fill_(0xFF)
    O1 = la.la_linear_attention(Q, K, V, lengths=ld, saved=saved)
    assert int((saved != 0xFF).sum()) > 0
    g1 = la.la_linear_attention_backward(Q, K, V, G, lengths=ld, saved=saved)
    la.la_last_device_status()
    assert torch.equal(O0, O1)
    for a, b, nm in zip(g0, g1, "QKV"):
        assert torch.equal(a, b), f"d{nm} differs with the saved sums"


def test_noncausal_ragged_workload_full_size():
    """The speech-shaped workload as a ragged batch (the paper's speech batches are: mean 800, max 2400
    frames): lengths between a third of N and N, one full and one of a single chunk plus one position."""
    w = WORKLOADS["noncausal_bf16_speech"]
    dtype = w.torch_dtype
    Q, K, V, G = draw_workload(w)
    g = torch.Generator().manual_seed(w.seed + 5)
    lengths = torch.randint(w.N // 3, w.N + 1, (w.B,), generator=g, dtype=torch.int32)
    lengths[0], lengths[w.B - 1] = w.N, 129
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    ld = lengths.to(DEV)
    O = la.la_linear_attention_varlen(Qd, Kd, Vd, ld)
    dQ, dK, dV = la.la_linear_attention_varlen_backward(Qd, Kd, Vd, Gd, ld)
    la.la_last_device_status()
    for b, h in _sample_heads(w.B, w.H):
        n = int(lengths[b])
        sl = (slice(b, b + 1), slice(h, h + 1), slice(0, n))
        q, k, v, gg = Q[sl], K[sl], V[sl], G[sl]
        assert_close(O[sl], oracle.linear_attention(q, k, v, False)[0], dtype, f"O[{b},{h}], length {n}")
        for got, ref, nm in zip((dQ, dK, dV), oracle.linear_attention_backward(q, k, v, gg, False), "QKV"):
            assert_close(got[sl], ref, dtype, f"d{nm}[{b},{h}], length {n}", grad=True)
    for b in range(w.B):
        n = int(lengths[b])
        for t in (O, dQ, dK, dV):
            assert n == w.N or float(t[b, :, n:].float().abs().max()) == 0.0


def test_decode_workload_full_size():
    w = WORKLOADS["decode_bf16_streams"]
    T = 3072
    Q, K, V, _ = draw_workload(w)
    # step-major copies, as a decoder would produce them: [T, B, H, D]
    q_t, k_t, v_t = (t.permute(2, 0, 1, 3).contiguous().to(DEV) for t in (Q, K, V))
    S = torch.zeros((w.B, w.H, w.D, w.M), device=DEV)
    Z = torch.zeros((w.B, w.H, w.D), device=DEV)
    outs = torch.empty((T, w.B, w.H, w.M), dtype=torch.bfloat16, device=DEV)
    for t in range(T):
        la.la_recurrent_step(q_t[t], k_t[t], v_t[t], S, Z, out=outs[t])
    la.la_last_device_status()
    outs = outs.permute(1, 2, 0, 3)                                   # [B, H, T, M]
    for b, h in _sample_heads(w.B, w.H):
        sl = (slice(b, b + 1), slice(h, h + 1))
        Or, _, Sr, Zr = oracle.linear_attention(Q[sl], K[sl], V[sl], True, return_state=True)
        assert_close(outs[sl], Or, torch.bfloat16, f"decode out[{b},{h}]")
        assert_close(S[sl], Sr, torch.bfloat16, f"decode S[{b},{h}]")
        assert_close(Z[sl], Zr, torch.bfloat16, f"decode Z[{b},{h}]")
    # the parallel causal form of the same sequences gives the same outputs
    bsub = slice(0, 8)
    O = la.la_causal_forward(*(t[bsub].contiguous().to(DEV) for t in (Q, K, V)))
    err = (O.float() - outs[bsub].float()).abs().max().item()
    assert err < 0.05, err


@pytest.mark.parametrize("B,H", [(256, 8), (3, 2), (130, 4), (37, 5), (20, 12)],
                         ids=["B256_H8", "B3_H2", "B130_H4", "B37_H5_odd_heads", "B20_H12"])
def test_decode_layer_steps_against_the_oracle(B, H):
    """A whole attention sublayer per token (projections, state update and read-out, output projection,
    residual), 12 tokens fed one at a time; the next token's input is made from the previous output, so the
    steps depend on each other as in generation.  The oracle walks the same steps in fp64 on the values the
    GPU actually saw as inputs (x is rounded to bf16 once per step on both sides)."""
    D = 64
    F = H * D
    g = torch.Generator().manual_seed(100 + B)
    s = 1.0 / F ** 0.5
    Wqkv = (torch.randn((3 * F, F), generator=g) * s).to(torch.bfloat16)
    Wo = (torch.randn((F, F), generator=g) * s).to(torch.bfloat16)
    x = torch.randn((B, F), generator=g).to(torch.bfloat16)
    S = torch.zeros((B, H, D, D), device=DEV)
    Z = torch.zeros((B, H, D), device=DEV)
    So, Zo = np.zeros((B, H, D, D)), np.zeros((B, H, D))
    Wd, Wod = Wqkv.to(DEV), Wo.to(DEV)
    W = Wqkv.double().numpy()
    Wq, Wk, Wv, Wout = W[:F].T, W[F:2 * F].T, W[2 * F:].T, Wo.double().numpy().T
    for t in range(12):
        y = la.la_decode_layer_step(x.to(DEV), Wd, Wod, S, Z)
        ref = oracle.decode_layer_step(x.double().numpy(), Wq, Wk, Wv, Wout, So, Zo)
        assert_close(y, ref, torch.bfloat16, f"layer step {t}")
        # the next input: a bounded function of this output (what the rest of a model would do), taken from the GPU
        x = torch.tanh(y.float().cpu()).to(torch.bfloat16) + (0.1 * torch.randn((B, F), generator=g)).to(torch.bfloat16)
    la.la_last_device_status()
    assert_close(S, So, torch.bfloat16, "layer S")
    assert_close(Z, Zo, torch.bfloat16, "layer Z")


def test_prepared_recurrent_step_repeats_the_regular_call():
    """The prepared form (checks and marshalling done once) enqueues exactly the regular call: same bits, state
    updated in place, inputs refilled in place between the steps."""
    B, H, D, M, T = 5, 3, 64, 64, 6
    Q, K, V, _ = draw_qkvg(B, H, T, D, M, seed=9, dtype=torch.bfloat16, with_grad=False)
    qs, ks, vs = (t.transpose(1, 2).transpose(0, 1).contiguous().to(DEV) for t in (Q, K, V))     # [T,B,H,.]
    S1, Z1 = torch.zeros((B, H, D, M), device=DEV), torch.zeros((B, H, D), device=DEV)
    S2, Z2 = torch.zeros_like(S1), torch.zeros_like(Z1)
    q, k, v = torch.empty_like(qs[0]), torch.empty_like(ks[0]), torch.empty_like(vs[0])
    step = la.prepare_recurrent_step(q, k, v, S2, Z2)
    for t in range(T):
        ref = la.la_recurrent_step(qs[t], ks[t], vs[t], S1, Z1)
        q.copy_(qs[t]); k.copy_(ks[t]); v.copy_(vs[t])
        out = step()
        assert torch.equal(out, ref), t
    assert torch.equal(S1, S2) and torch.equal(Z1, Z2)
    with pytest.raises(ValueError):
        la.prepare_recurrent_step(q, k, v, S2[:, :2], Z2)


def test_decode_layer_rejects_what_it_does_not_take():
    B, H, D = 4, 2, 32
    x = torch.zeros((B, H * D), dtype=torch.bfloat16, device=DEV)
    W3, W1 = torch.zeros((3 * H * D, H * D), dtype=torch.bfloat16, device=DEV), torch.zeros((H * D, H * D), dtype=torch.bfloat16, device=DEV)
    S, Z = torch.zeros((B, H, D, D), device=DEV), torch.zeros((B, H, D), device=DEV)
    with pytest.raises(la.LaError) as e:
        la.la_decode_layer_step(x, W3, W1, S, Z)
    assert e.value.status == -2


def _poison_padding(tensors, lengths):
    """Inf and NaN on everything behind each sequence's end: none of it may reach a result."""
    for i, t in enumerate(tensors):
        for b, n in enumerate(lengths):
            t[b, :, n:] = float("nan") if (i + b) % 2 else float("inf")


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape,lengths", [
    ((4, 2, 100, 16, 48), [100, 37, 1, 0]),                       # general kernels, ragged chunk tails
    ((3, 2, 384, 64, 64), [384, 129, 300]),                       # bf16: the tensor-core shapes
    ((6, 4, 1024, 64, 64), [1024, 0, 1, 128, 641, 900]),          # whole chunks, a chunk boundary, nothing at all
    ((2, 32, 2304, 64, 64), [2304, 1000]),                        # B*H = 64: sequences cut into pieces with a pre-pass
])
def test_causal_ragged_batches(shape, lengths, dtype):
    """la_causal_forward_varlen / _backward_varlen on a right-padded batch: every sequence against the oracle run
    on its own length; zeros on the padding, which holds Inf and NaN on the way in; the state handed back is the
    one at each sequence's own end, and a decode step continues from it (a ragged prefill followed by
    generation, checked against the N x N definition of the sequence one token longer)."""
    B, H, N, D, M = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, M, seed=300 + N + D, dtype=dtype)
    nxt = draw_qkvg(B, H, 1, D, M, seed=301 + N, dtype=dtype, with_grad=False)[:3]
    clean = [t.clone() for t in (Q, K, V, G)]
    _poison_padding((Q, K, V, G), lengths)
    Qd, Kd, Vd, Gd = gpu(Q, K, V, G)
    ln = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    den = torch.full((B, H, N), 7.0, device=DEV)
    S = torch.full((B, H, D, M), 7.0, device=DEV)
    Z = torch.full((B, H, D), 7.0, device=DEV)
    O = la.la_causal_forward(Qd, Kd, Vd, lengths=ln, den=den, S_out=S, Z_out=Z)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, lengths=ln)
    la.la_last_device_status()
    # the same with a saved buffer (poisoned beforehand: what lies behind a sequence's end in it is never read):
    # the forward's result does not depend on it, dQ is bit-identical, dK and dV agree to rounding
    saved = la.saved_buffer(Qd, Vd)
    if saved is not None:
        saved.fill_(0xFF)
        O2 = la.la_causal_forward(Qd, Kd, Vd, lengths=ln, saved=saved)
        g2 = la.la_causal_backward(Qd, Kd, Vd, Gd, lengths=ln, saved=saved)
        la.la_last_device_status()
        assert torch.equal(O2, O) and torch.equal(g2[0], dQ)
        for a, b2, nm in zip((dK, dV), g2[1:], "KV"):
            assert torch.all(b2.isfinite()), f"d{nm} with the saved buffer"
            assert_close(b2, a.double().cpu().numpy(), dtype, f"d{nm} saved vs recomputed", grad=True)
    # one decode step per stream from the state the ragged prefill handed back
    q1, k1, v1 = (t[:, :, 0].contiguous() for t in gpu(*nxt))
    out1 = la.la_recurrent_step(q1, k1, v1, S.clone(), Z.clone())
    for b, n in enumerate(lengths):
        sl = slice(b, b + 1)
        q, k, v, g = (t[sl, :, :n] for t in clean)
        for t, nm in ((O, "O"), (den, "den"), (dQ, "dQ"), (dK, "dK"), (dV, "dV")):
            assert torch.all(t[sl, :, n:] == 0), f"{nm}: padding of sequence {b} is not zero"
        Or, denr, Sr, Zr = oracle.linear_attention(q, k, v, True, return_state=True)
        assert_close(S[sl], Sr, dtype, f"S at the end, length {n}")
        assert_close(Z[sl], Zr, dtype, f"Z at the end, length {n}")
        if n:
            assert_close(O[sl, :, :n], Or, dtype, f"O, length {n}")
            assert_close(den[sl, :, :n], denr, dtype, f"den, length {n}")
            for got, ref, nm in zip((dQ, dK, dV), oracle.linear_attention_backward(q, k, v, g, True), "QKV"):
                assert_close(got[sl, :, :n], ref, dtype, f"d{nm}, length {n}", grad=True)
        longer = [torch.cat([a, c[sl]], 2) for a, c in zip((q, k, v), nxt)]
        assert_close(out1[sl], oracle.attention_quadratic(*longer, True)[:, :, n], dtype, f"decode after prefill, length {n}")


def test_causal_ragged_batch_from_a_state_with_state_gradients():
    """The ragged calls with every state argument: the sequences continue from S_0, Z_0, the upstream gradient
    of the state at each sequence's own end comes in, the gradient of the initial state goes out."""
    B, H, N, D = 3, 2, 512, 64
    lengths = [512, 200, 77]
    dtype = torch.bfloat16
    Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=410, dtype=dtype)
    g = torch.Generator().manual_seed(411)
    S0, Z0 = torch.randn((B, H, D, D), generator=g) * 3.0, torch.rand((B, H, D), generator=g) * 4.0 + 1.0
    dS, dZ = torch.randn((B, H, D, D), generator=g) * 0.05, torch.randn((B, H, D), generator=g) * 0.05
    Qd, Kd, Vd, Gd, S0d, Z0d, dSd, dZd = gpu(Q, K, V, G, S0, Z0, dS, dZ)
    ln = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    S1, Z1 = torch.empty_like(S0d), torch.empty_like(Z0d)
    O = la.la_causal_forward(Qd, Kd, Vd, lengths=ln, S_in=S0d, Z_in=Z0d, S_out=S1, Z_out=Z1)
    dS0, dZ0 = torch.empty_like(S0d), torch.empty_like(Z0d)
    dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd, lengths=ln, S_in=S0d, Z_in=Z0d, dS_out=dSd, dZ_out=dZd,
                                       dS_in=dS0, dZ_in=dZ0)
    la.la_last_device_status()
    for b, n in enumerate(lengths):
        sl = slice(b, b + 1)
        q, k, v, gg = (t[sl, :, :n] for t in (Q, K, V, G))
        Or, _, Sr, Zr = oracle.causal_from_state(q, k, v, S0[sl], Z0[sl])
        assert_close(O[sl, :, :n], Or, dtype, f"O from a state, length {n}")
        assert_close(S1[sl], Sr, dtype, f"S_N from a state, length {n}")
        assert_close(Z1[sl], Zr, dtype, f"Z_N from a state, length {n}")
        rq, rk, rv, rS, rZ = oracle.causal_backward_from_state(q, k, v, S0[sl], Z0[sl], gg, dS[sl], dZ[sl])
        assert_close(dQ[sl, :, :n], rq, dtype, f"dQ from a state, length {n}", grad=True)
        assert_close(dK[sl, :, :n], rk, dtype, f"dK from a state, length {n}", grad=True)
        assert_close(dV[sl, :, :n], rv, dtype, f"dV from a state, length {n}", grad=True)
        assert_close(dS0[sl], rS, dtype, f"dS_0, length {n}", grad=True)
        assert_close(dZ0[sl], rZ, dtype, f"dZ_0, length {n}", grad=True)
