"""Sequence lengths that are not a multiple of the 128-position chunk on the tensor-core kernels.

The last chunk of such a sequence is partly beyond its end, where memory holds the NEXT sequence
(or nothing): tile loads must read zeros there and nothing may be stored there.  Every tensor of
these tests sits at the front of a larger buffer filled with a marker, so that a store past a
tensor's end would be seen (and would be harmless); stores into the next sequence show up in the
comparison with the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2006_16236_b200 as la
from paper_2006_16236_b200.inputs import draw_qkvg
from parity import assert_close

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda")
SLACK = 32768           # elements behind every tensor
MARK = 1234.0


def _front(shape, dtype):
    n = int(np.prod(shape))
    flat = torch.full((n + SLACK,), MARK, dtype=dtype, device=DEV)
    return flat[:n].view(shape), flat[n:]


def _place(t):
    v, tail = _front(tuple(t.shape), t.dtype)
    v.copy_(t)
    return v, tail


def _untouched(tails):
    for nm, tail in tails.items():
        assert bool((tail == MARK).all()), f"{nm}: something was stored behind the tensor's end"


SHAPES = [(2, 3, 100, 64), (2, 3, 129, 64), (1, 5, 200, 32), (2, 8, 784, 32), (3, 2, 1000, 64), (1, 70, 700, 64),
          (2, 2, 1, 64), (1, 3, 127, 32), (1, 2, 2, 32)]


@pytest.mark.parametrize("keep", [False, True], ids=["recompute", "saved"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "B%d_H%d_N%d_D%d" % s)
def test_causal_any_length(shape, keep):
    B, H, N, D = shape
    p = la.make_problem(B, H, N, D, D, la.LA_BF16)
    assert la.la_causal_plan(p) is not None, "this shape is meant to run the tensor-core kernels"
    Q, K, V, G = draw_qkvg(B, H, N, D, D, 7 + N, torch.bfloat16, 1.0)
    tails = {}
    dev = {}
    for nm, t in zip("QKVG", (Q, K, V, G)):
        dev[nm], tails[nm] = _place(t.to(DEV))
    outs = {}
    for nm, like in (("O", V), ("dQ", Q), ("dK", K), ("dV", V)):
        outs[nm], tails[nm] = _front(tuple(like.shape), torch.bfloat16)
    den, tails["den"] = _front((B, H, N), torch.float32)
    S, tails["S"] = _front((B, H, D, D), torch.float32)
    Z, tails["Z"] = _front((B, H, D), torch.float32)
    saved = la.saved_buffer(dev["Q"], dev["V"]) if keep else None
    kw = {"saved": saved} if keep else {}
    la.la_causal_forward(dev["Q"], dev["K"], dev["V"], O=outs["O"], den=den, S_out=S, Z_out=Z, **kw)
    la.la_causal_backward(dev["Q"], dev["K"], dev["V"], dev["G"], dQ=outs["dQ"], dK=outs["dK"], dV=outs["dV"], **kw)
    la.la_last_device_status()
    _untouched(tails)
    q, k, v, g = (t.double().numpy() for t in (Q, K, V, G))
    O_ref, den_ref = oracle.linear_attention(q, k, v, causal=True)[:2]
    assert_close(outs["O"], O_ref, torch.bfloat16, "O")
    assert_close(den, den_ref, torch.bfloat16, "den")
    for nm, ref in zip(("dQ", "dK", "dV"), oracle.linear_attention_backward(q, k, v, g, causal=True)):
        assert_close(outs[nm], ref, torch.bfloat16, nm, grad=True)
    # the state at the sequence's end: what the unrolled recurrence holds after N steps
    fk = oracle.feature_map(k)
    assert_close(S, np.einsum("bhnd,bhnm->bhdm", fk, v), torch.bfloat16, "S_out")
    assert_close(Z, fk.sum(2), torch.bfloat16, "Z_out")


@pytest.mark.parametrize("shape", SHAPES[:5] + SHAPES[6:], ids=lambda s: "B%d_H%d_N%d_D%d" % s)
def test_noncausal_any_length(shape):
    B, H, N, D = shape
    Q, K, V, G = draw_qkvg(B, H, N, D, D, 11 + N, torch.bfloat16, 0.5)
    tails, dev, outs = {}, {}, {}
    for nm, t in zip("QKVG", (Q, K, V, G)):
        dev[nm], tails[nm] = _place(t.to(DEV))
    for nm, like in (("O", V), ("dQ", Q), ("dK", K), ("dV", V)):
        outs[nm], tails[nm] = _front(tuple(like.shape), torch.bfloat16)
    den, tails["den"] = _front((B, H, N), torch.float32)
    la.la_profile_enable(True)
    la.la_linear_attention(dev["Q"], dev["K"], dev["V"], O=outs["O"], den=den)
    la.la_linear_attention_backward(dev["Q"], dev["K"], dev["V"], dev["G"], dQ=outs["dQ"], dK=outs["dK"], dV=outs["dV"])
    la.la_last_device_status()
    names = set(la.la_profile_read())
    la.la_profile_enable(False)
    assert "linear_apply_kernel" in names, names
    _untouched(tails)
    q, k, v, g = (t.double().numpy() for t in (Q, K, V, G))
    O_ref, den_ref = oracle.linear_attention(q, k, v, causal=False)[:2]
    assert_close(outs["O"], O_ref, torch.bfloat16, "O")
    assert_close(den, den_ref, torch.bfloat16, "den")
    for nm, ref in zip(("dQ", "dK", "dV"), oracle.linear_attention_backward(q, k, v, g, causal=False)):
        assert_close(outs[nm], ref, torch.bfloat16, nm, grad=True)


@pytest.mark.parametrize("causal", [False, True])
def test_lengths_inside_a_batch_whose_own_length_is_odd(causal):
    """Both kinds of raggedness at once: N = 700 and per-sequence lengths below it (one of them 0, one of them N)."""
    B, H, N, D = 4, 2, 700, 64
    lengths = [700, 0, 333, 129]
    Q, K, V, G = draw_qkvg(B, H, N, D, D, 5, torch.bfloat16, 1.0)
    tails, dev, outs = {}, {}, {}
    for nm, t in zip("QKVG", (Q, K, V, G)):
        dev[nm], tails[nm] = _place(t.to(DEV))
    for nm, like in (("O", V), ("dQ", Q), ("dK", K), ("dV", V)):
        outs[nm], tails[nm] = _front(tuple(like.shape), torch.bfloat16)
    ln = torch.tensor(lengths, dtype=torch.int32, device=DEV)
    if causal:
        la.la_causal_forward(dev["Q"], dev["K"], dev["V"], lengths=ln, O=outs["O"])
        la.la_causal_backward(dev["Q"], dev["K"], dev["V"], dev["G"], lengths=ln, dQ=outs["dQ"], dK=outs["dK"], dV=outs["dV"])
    else:
        la.la_linear_attention_varlen(dev["Q"], dev["K"], dev["V"], ln, O=outs["O"])
        la.la_linear_attention_varlen_backward(dev["Q"], dev["K"], dev["V"], dev["G"], ln, dQ=outs["dQ"], dK=outs["dK"], dV=outs["dV"])
    la.la_last_device_status()
    _untouched(tails)
    for b, n in enumerate(lengths):
        for nm in ("O", "dQ", "dK", "dV"):
            assert not bool(outs[nm][b, :, n:].float().abs().max() > 0) if n < N else True, f"{nm}: padding of sequence {b} is not zero"
        if n == 0:
            continue
        q, k, v, g = (t[b:b + 1, :, :n].double().numpy() for t in (Q, K, V, G))
        O_ref = oracle.linear_attention(q, k, v, causal=causal)[0]
        assert_close(outs["O"][b:b + 1, :, :n], O_ref, torch.bfloat16, f"O of sequence {b}")
        for nm, ref in zip(("dQ", "dK", "dV"), oracle.linear_attention_backward(q, k, v, g, causal=causal)):
            assert_close(outs[nm][b:b + 1, :, :n], ref, torch.bfloat16, f"{nm} of sequence {b}", grad=True)


def test_prefill_in_odd_pieces_then_decode():
    """A prompt of 300 positions fed in calls of 77, 200 and 23 positions (none a multiple of the chunk), each
    continuing from the state the call before left, then two decode steps: the same outputs as the whole sequence."""
    B, H, D = 2, 3, 64
    cuts = [77, 200, 23]
    N = sum(cuts) + 2
    Q, K, V, _ = draw_qkvg(B, H, N, D, D, 3, torch.bfloat16, 1.0, with_grad=False)
    O_ref = oracle.linear_attention(*(t.double().numpy() for t in (Q, K, V)), causal=True)[0]
    S = torch.zeros((B, H, D, D), device=DEV)
    Z = torch.zeros((B, H, D), device=DEV)
    lo = 0
    for n in cuts:
        q, k, v = (t[:, :, lo:lo + n].contiguous().to(DEV) for t in (Q, K, V))
        S2, Z2 = torch.empty_like(S), torch.empty_like(Z)
        O = la.la_causal_forward(q, k, v, S_in=S, Z_in=Z, S_out=S2, Z_out=Z2)
        assert_close(O, O_ref[:, :, lo:lo + n], torch.bfloat16, f"positions {lo}..{lo + n}")
        S, Z, lo = S2, Z2, lo + n
    for i in range(lo, N):
        out = la.la_recurrent_step(Q[:, :, i].contiguous().to(DEV), K[:, :, i].contiguous().to(DEV), V[:, :, i].contiguous().to(DEV), S, Z)
        assert_close(out, O_ref[:, :, i], torch.bfloat16, f"decode step {i}")
    la.la_last_device_status()
