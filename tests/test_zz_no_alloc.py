"""The allocation-free non-causal forward, la_linear_attention_noalloc.

Some users of the library cannot allocate device memory at the point where they call
it (they are handed input and output buffers by a host framework, or run where a
cudaMalloc would stall the device), so this entry point keeps its scratch in a fixed
array inside the library.  The test drives it through the C ABI with preallocated
outputs, twice in a row on different data (the array keeps the first call's contents),
and compares each result with the regular entry point given a caller-owned workspace.
Collected last on purpose: a failure here cannot hide failures of the other tests.
"""
import ctypes

import pytest
import torch

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
        O_ref = la.la_linear_attention(Qd, Kd, Vd, den=den_ref)
        p = la.make_problem(B, H, N, D, M, binding.LA_F32 if dtype == torch.float32 else binding.LA_BF16)
        rc = binding.lib().la_linear_attention_noalloc(
            ctypes.byref(p), ctypes.c_void_p(Qd.data_ptr()), ctypes.c_void_p(Kd.data_ptr()),
            ctypes.c_void_p(Vd.data_ptr()), ctypes.c_void_p(O.data_ptr()), ctypes.c_void_p(den.data_ptr()),
            ctypes.c_void_p(KV.data_ptr()), ctypes.c_void_p(Zs.data_ptr()),
            ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert rc == 0, binding.lib().la_last_error()
        torch.cuda.synchronize()
        assert max_rel_err(O, O_ref.double().cpu().numpy()) <= TOL[dtype], f"call {call}: O"
        assert max_rel_err(den, den_ref.double().cpu().numpy()) <= TOL[dtype], f"call {call}: den"
        outs.append(O.clone())
    assert not torch.equal(outs[0], outs[1])          # the two calls really saw different data


def test_noalloc_rejects_problems_beyond_the_builtin_scratch():
    # 512 heads x 128 x 129 floats per split record exceeds the 8 MiB array: refused, nothing enqueued
    p = la.make_problem(64, 8, 4096, 128, 128, binding.LA_F32)
    buf = torch.empty(64, device=DEV)
    ptr = ctypes.c_void_p(buf.data_ptr())
    rc = binding.lib().la_linear_attention_noalloc(ctypes.byref(p), ptr, ptr, ptr, ptr, None, None, None, None)
    assert rc == -3
    msg = binding.lib().la_last_error().decode()
    assert "scratch" in msg and str(8 << 20) in msg
