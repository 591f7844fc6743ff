"""The allocation-free non-causal forward, la_linear_attention_noalloc.

Some users of the library cannot allocate device memory at the point where they call
it (they are handed input and output buffers by a host framework, or run where a
cudaMalloc would stall the device), so this entry point keeps its scratch in a fixed
array inside the library.  The test drives it through the C ABI with preallocated
outputs, twice in a row on different data (the array keeps the first call's contents),
and compares each result with the regular entry point given a caller-owned workspace
(the same kernels on the same inputs: bit for bit) and with the fp64 oracle.
Collected last on purpose: a failure here cannot hide failures of the other tests.
"""
import ctypes

import pytest
import torch

import oracle
import paper_2006_16236_b200 as la
from paper_2006_16236_b200 import binding
from paper_2006_16236_b200.inputs import draw_qkvg
from parity import TOL, max_rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_noalloc_matches_regular_entry_point_on_two_calls(dtype):
    B, H, N, D, M = 2, 4, 1000, 64, 48
    outs = []
    O = torch.empty((B, H, N, M), dtype=dtype, device=DEV)
    den = torch.empty((B, H, N), device=DEV)
    KV = torch.empty((B, H, D, M), device=DEV)
    Zs = torch.empty((B, H, D), device=DEV)
    for call, seed in enumerate((21, 22)):
        Q, K, V, _ = draw_qkvg(B, H, N, D, M, seed=seed, dtype=dtype, scale=0.5, with_grad=False)
        Qd, Kd, Vd = Q.to(DEV), K.to(DEV), V.to(DEV)
        den_ref = torch.empty_like(den)
        KV_ref, Zs_ref = torch.empty_like(KV), torch.empty_like(Zs)
        O_ref = la.la_linear_attention(Qd, Kd, Vd, den=den_ref, KV=KV_ref, Zs=Zs_ref)
        p = la.make_problem(B, H, N, D, M, binding.LA_F32 if dtype == torch.float32 else binding.LA_BF16)
        rc = binding.lib().la_linear_attention_noalloc(
            ctypes.byref(p), ctypes.c_void_p(Qd.data_ptr()), ctypes.c_void_p(Kd.data_ptr()),
            ctypes.c_void_p(Vd.data_ptr()), ctypes.c_void_p(O.data_ptr()), ctypes.c_void_p(den.data_ptr()),
            ctypes.c_void_p(KV.data_ptr()), ctypes.c_void_p(Zs.data_ptr()),
            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0, binding.lib().la_last_error()
        torch.cuda.synchronize()
        # the regular entry point runs the same kernels on this shape (D != M keeps it off the tensor cores)
        assert torch.equal(O, O_ref) and torch.equal(den, den_ref), f"call {call}: not bit-identical"
        assert torch.equal(KV, KV_ref) and torch.equal(Zs, Zs_ref), f"call {call}: sums not bit-identical"
        assert max_rel_err(O, O_ref.double().cpu().numpy()) <= TOL[dtype], f"call {call}: O"
        assert max_rel_err(den, den_ref.double().cpu().numpy()) <= TOL[dtype], f"call {call}: den"
        # and against the oracle (Eq. 5-6 in fp64 on the same rounded inputs)
        o_ref, d_ref = oracle.linear_attention(Q, K, V, False)
        assert max_rel_err(O, o_ref) <= TOL[dtype], f"call {call}: O vs oracle"
        assert max_rel_err(den, d_ref) <= TOL[dtype], f"call {call}: den vs oracle"
        outs.append(O.clone())
    assert not torch.equal(outs[0], outs[1])          # the two calls really saw different data


def test_noalloc_rejects_problems_beyond_the_builtin_scratch():
    # 256 heads x 128 x 129 floats of partial sums (16.9 MB) exceed the 8 MiB array: refused, nothing
    # enqueued.  Every buffer has its full size (about 1 MB each), so that even a regression that let
    # the call through could not touch memory the test does not own.
    B, H, N, D, M = 32, 8, 8, 128, 128
    p = la.make_problem(B, H, N, D, M, binding.LA_F32)
    assert la.la_workspace_bytes(p, binding.LA_OP_LINEAR_FORWARD) > (8 << 20)
    Q, K, V, O = (torch.zeros((B, H, N, D), device=DEV) for _ in range(4))
    rc = binding.lib().la_linear_attention_noalloc(
        ctypes.byref(p), ctypes.c_void_p(Q.data_ptr()), ctypes.c_void_p(K.data_ptr()), ctypes.c_void_p(V.data_ptr()),
        ctypes.c_void_p(O.data_ptr()), None, None, None, None)
    assert rc == -3
    msg = binding.lib().la_last_error().decode()
    assert "scratch" in msg and str(8 << 20) in msg
    # the checks shared with la_linear_attention() apply here too
    too_long = la.make_problem(1, 1, 1 << 36, 128, 128, binding.LA_F32)
    assert binding.lib().la_linear_attention_noalloc(
        ctypes.byref(too_long), ctypes.c_void_p(Q.data_ptr()), ctypes.c_void_p(K.data_ptr()),
        ctypes.c_void_p(V.data_ptr()), ctypes.c_void_p(O.data_ptr()), None, None, None, None) == -2
