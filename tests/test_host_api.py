"""Host-side checks that need no GPU: the library loads, exports the declared symbols,
sizes workspaces and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest
import torch

import paper_2006_16236_b200 as la
from paper_2006_16236_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "la.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(la_[a-z_]+)\s*\(", header))
    assert {"la_feature_map", "la_linear_attention", "la_linear_attention_backward", "la_causal_forward",
            "la_causal_backward", "la_recurrent_step", "la_workspace_bytes"} <= declared
    for name in declared:
        assert hasattr(L, name), name
    assert set(binding.EXPORTS) >= declared - {"la_problem"}


def test_version_and_status_strings(L):
    assert la.la_version() == "0.1"
    assert L.la_status_string(0) == b"LA_OK"
    assert L.la_status_string(-3) == b"LA_ERR_WORKSPACE"
    assert L.la_status_string(-99) == b"LA_ERR_UNKNOWN"


def test_workspace_sizes_are_independent_of_n_times_d_times_m(L):
    # constant-memory claim: scratch grows at most linearly in N with a per-token constant
    # that does not involve D*M (no per-position state is stored)
    for dt in (binding.LA_F32, binding.LA_BF16):
        for op in range(4):
            small = la.la_workspace_bytes(la.make_problem(2, 8, 4096, 64, 64, dt), op)
            big = la.la_workspace_bytes(la.make_problem(2, 8, 65536, 64, 64, dt), op)
            per_token_head = (big - small) / ((65536 - 4096) * 16)
            assert per_token_head <= 64 * 65 * 4 / 64 + 16, (dt, op, per_token_head)
    assert la.la_workspace_bytes(la.make_problem(1, 1, 0, 64, 64, 0), 3) == 0
    assert la.la_workspace_bytes(la.make_problem(1, 1, 128, 256, 64, 0), 3) == 0   # invalid -> 0


def _p(**kw):
    base = dict(B=1, H=1, N=128, D=64, M=64, dtype_code=binding.LA_F32)
    base.update(kw)
    return la.make_problem(**base)


@pytest.mark.parametrize("bh", [1, 2, 3, 5, 8, 16, 32, 48, 50, 64, 70, 74, 75, 100, 119, 120, 128, 148, 256])
@pytest.mark.parametrize("chunks", [1, 2, 3, 4, 8, 17, 64, 100, 128, 256, 1024])
def test_causal_plan_tiles_every_sequence(L, bh, chunks):
    """Pieces and pre-pass parts of the tensor-core causal kernels: both tile [0, N / 128) in order, a
    piece starts on a part boundary, every piece is launched exactly once, and the parts a pre-pass
    computes (all before the last piece, all after the first) are the ones a piece's start needs."""
    p = la.make_problem(bh, 1, chunks * 128, 64, 64, la.LA_BF16)
    plan = la.la_causal_plan(p)
    assert plan is not None
    n, q = plan["pieces"], plan["parts"]
    pb, fp, qb = plan["piece_begin"], plan["piece_first_part"], plan["part_begin"]
    assert n >= 1 and q >= n
    assert pb[0] == 0 and pb[n] == chunks and qb[0] == 0 and qb[q] == chunks
    assert all(pb[k] < pb[k + 1] for k in range(n)) and all(qb[j] < qb[j + 1] for j in range(q))
    assert fp[0] == 0 and fp[n] == q and all(fp[k] < fp[k + 1] for k in range(n))
    assert all(qb[fp[k]] == pb[k] for k in range(n + 1))
    if n > 1:
        assert min(pb[k + 1] - pb[k] for k in range(n)) >= 2          # a piece is at least two chunks
    assert sorted(plan["launch_order"]) == list(range(n))
    # long pieces are launched before a shorter one, so that the left-over SMs take the short pieces last
    lens = [pb[k + 1] - pb[k] for k in plan["launch_order"]]
    assert all(lens[i] + 1 >= lens[i + 1] for i in range(n - 1))
    # work per SM: no more CTAs of the long kind than SMs
    nlong = sum(1 for x in lens if x + 1 >= lens[0])
    assert bh * nlong <= 148 or n == 1 or nlong == 1


def test_causal_plan_of_the_bench_workload(L):
    # B*H = 64, 128 chunks: two long pieces around one short middle piece, 192 CTAs for 148 SMs
    plan = la.la_causal_plan(la.make_problem(8, 8, 16384, 64, 64, la.LA_BF16))
    assert plan["pieces"] == 3 and plan["launch_order"] == [0, 2, 1]
    pb = plan["piece_begin"]
    short = pb[2] - pb[1]
    assert 8 <= short <= 16 and abs((pb[1] - pb[0]) - (pb[3] - pb[2])) <= 1
    # problems that run the general kernels have no plan
    assert la.la_causal_plan(la.make_problem(1, 2, 256, 32, 32, la.LA_F32)) is None
    assert la.la_causal_plan(la.make_problem(1, 2, 256, 64, 48, la.LA_BF16)) is None
    # a length that is not a multiple of the chunk: the last chunk is partial
    ragged = la.la_causal_plan(la.make_problem(1, 2, 200, 64, 64, la.LA_BF16))
    assert ragged is not None and ragged["piece_begin"][-1] == 2


def test_bad_arguments_are_rejected_on_the_host(L):
    buf = ctypes.create_string_buffer(64)
    ok = ctypes.c_void_p((ctypes.addressof(buf) + 15) & ~15)
    odd = ctypes.c_void_p(ok.value + 4)
    null = ctypes.c_void_p(None)

    def causal(p, Q=ok, K=ok, V=ok, O=ok, ws=null, ws_bytes=0):
        return L.la_causal_forward(ctypes.byref(p) if p is not None else None, Q, K, V, O, null, null, null,
                                   null, 0, ws, ws_bytes, null)

    assert causal(None) == -1
    assert causal(_p(B=0)) == -1
    assert causal(_p(N=-1)) == -1
    assert causal(_p(dtype_code=7)) == -1
    assert causal(_p(D=12)) == -2
    assert causal(_p(D=256)) == -2
    assert causal(_p(eps=-1.0)) == -1
    assert causal(_p(), Q=null) == -1
    assert causal(_p(), V=odd) == -1
    assert b"16-byte" in L.la_last_error()
    assert causal(_p(N=0)) == 0                      # empty sequence: successful no-op
    # backward needs scratch: NULL or short workspace is refused
    p = _p()
    need = la.la_workspace_bytes(p, binding.LA_OP_CAUSAL_BACKWARD)
    assert need > 0
    args = [ctypes.byref(p), ok, ok, ok, null, null, ok, null, 0, ok, ok, ok]
    assert L.la_causal_backward(*args, null, 0, null) == -3
    assert L.la_causal_backward(*args, ok, need - 1, null) == -3
    # the optional saved buffer: a short or misaligned one is refused; problems on the general kernels need none
    pb = _p(dtype_code=binding.LA_BF16, N=256, D=64, M=64)
    keep = la.la_workspace_bytes(pb, binding.LA_OP_CAUSAL_SAVED)
    assert keep >= 2 * 256 * 64 * 2 * pb.B * pb.H
    big = ctypes.c_void_p(1 << 20)                   # never dereferenced: validation fails first
    args = [ctypes.byref(pb), big, big, big, null, null, big, big, keep - 1, big, big, big]
    assert L.la_causal_backward(*args, big, 1 << 40, null) == -3
    assert b"saved" in L.la_last_error()
    args[7] = ctypes.c_void_p((1 << 20) + 16)
    assert L.la_causal_backward(*args, big, 1 << 40, null) == -1
    assert la.la_workspace_bytes(_p(), binding.LA_OP_CAUSAL_SAVED) == 0
    assert L.la_recurrent_step(ctypes.byref(p), ok, ok, ok, null, ok, ok, null) == -1
    # continuation from a state: S_in and Z_in come together, must not overlap the outputs, exclude `saved`
    def cont(p, S_in, Z_in, S_out=null, Z_out=null, saved=null, saved_bytes=0):
        return L.la_causal_forward_from(ctypes.byref(p), ok, ok, ok, S_in, Z_in, ok, null, S_out, Z_out,
                                        saved, saved_bytes, null, 0, null)
    far = ctypes.c_void_p(1 << 30)
    assert cont(_p(), far, null) == -1
    assert cont(_p(), null, far) == -1
    assert cont(_p(), far, ctypes.c_void_p((1 << 30) + (1 << 20)), S_out=far) == -1
    assert b"overlap" in L.la_last_error()
    assert cont(_p(), odd, far) == -1
    assert cont(_p(N=0), null, null) == 0

    def back(p, S_in=null, Z_in=null, dS_out=null, dZ_out=null, dS_in=null, dZ_in=null):
        return L.la_causal_backward_from(ctypes.byref(p), ok, ok, ok, S_in, Z_in, null, null, ok, dS_out, dZ_out,
                                         null, 0, ok, ok, ok, dS_in, dZ_in, null, 0, null)
    assert back(_p(), S_in=far) == -1                                   # Z_in missing
    assert back(_p(), dS_out=far, dS_in=far) == -1                      # gradient in and out overlap
    assert b"overlap" in L.la_last_error()
    assert back(_p(), dZ_in=odd) == -1
    assert back(_p()) == -3                                             # plain backward: needs its workspace
    assert back(_p(N=0)) == 0
    # ragged batches: the lengths are required and 4-byte aligned
    pv = _p()
    need_v = la.la_workspace_bytes(pv, binding.LA_OP_LINEAR_VARLEN_FORWARD)
    assert need_v > 0 and la.la_workspace_bytes(pv, binding.LA_OP_LINEAR_VARLEN_BACKWARD) >= need_v
    assert L.la_linear_attention_varlen(ctypes.byref(pv), ok, ok, ok, null, ok, null, null, null, big, 1 << 40, null) == -1
    assert b"lengths" in L.la_last_error()
    assert L.la_linear_attention_varlen(ctypes.byref(pv), ok, ok, ok, ctypes.c_void_p(ok.value + 2), ok, null, null, null,
                                        big, 1 << 40, null) == -1
    assert L.la_linear_attention_varlen(ctypes.byref(pv), ok, ok, ok, ok, ok, null, null, null, null, 0, null) == -3
    assert L.la_linear_attention_varlen_backward(ctypes.byref(pv), ok, ok, ok, null, null, null, ok, ok, ok, ok,
                                                 big, 1 << 40, null) == -1
    # the non-causal saved buffer: optional, 16-byte aligned, large enough; with it the forward needs no workspace
    need_s = la.la_workspace_bytes(pv, binding.LA_OP_LINEAR_SAVED)
    assert need_s == la.la_workspace_bytes(pv, binding.LA_OP_LINEAR_FORWARD) > 0
    keep = lambda saved, nbytes, ws=null, wsb=0: L.la_linear_attention_keep(ctypes.byref(pv), ok, ok, ok, null, ok, null, null,
                                                                          null, saved, nbytes, ws, wsb, null)
    assert keep(odd, 1 << 40) == -1 and b"saved" in L.la_last_error()
    assert keep(ok, need_s - 1) == -3
    assert keep(null, 0) == -3                                          # no saved buffer: the workspace is required
    assert L.la_linear_attention_backward_kept(ctypes.byref(pv), ok, ok, ok, null, ok, need_s - 1, null, null, ok, ok, ok, ok,
                                               big, 1 << 40, null) == -3
    assert L.la_linear_attention_backward_kept(ctypes.byref(pv), ok, ok, ok, null, ok, need_s, null, null, ok, ok, ok, ok,
                                               null, 0, null) == -3     # the backward still needs its workspace
    assert L.la_feature_map(ok, ok, -5, 0, 0, null) == -1
    assert L.la_feature_map(ok, ok, 0, 0, 0, null) == 0
    assert L.la_feature_map(ok, ok, 4, 9, 0, null) == -1
    # degree-2 polynomial map: D*D <= C <= 128, C a multiple of 8; nothing to do for zero rows
    poly = lambda rows, D, C, dt=0, x=ok, y=ok: L.la_feature_map_poly2(x, y, rows, D, C, dt, null)
    assert poly(0, 8, 64) == 0
    assert poly(-1, 8, 64) == -1 and poly(4, 0, 8) == -1 and poly(4, 12, 144) == -1
    assert poly(4, 8, 56) == -1 and poly(4, 3, 12) == -1 and poly(4, 3, 136) == -1 and poly(4, 8, 64, dt=7) == -1
    assert poly(4, 8, 64, x=null) == -1 and poly(4, 8, 64, y=odd) == -1 and poly(4, 8, 64, x=odd) == -1
    assert L.la_feature_map_poly2_backward(ok, ok, ok, 4, 8, 64, 0, null) == -1          # dx aliases x
    assert b"alias" in L.la_last_error()
    assert L.la_feature_map_poly2_backward(ok, null, far, 4, 8, 64, 0, null) == -1
    assert L.la_feature_map_poly2_backward(ok, ok, far, 0, 8, 64, 0, null) == 0
    assert binding.poly2_columns(8) == 64 and binding.poly2_columns(5) == 32 and binding.poly2_columns(11) == 128
    # random Fourier features: bf16 (dtype 1), D a multiple of 8 in [8, 64], C = 64 or 128; all refusals come before any CUDA call
    rff = lambda rows, D, C, dt=1, x=ok, W=ok, y=ok: L.la_feature_map_rff(x, W, y, rows, D, C, dt, null)
    assert rff(0, 64, 64) == 0
    assert rff(-1, 64, 64) == -1 and rff(4, 0, 64) == -1 and rff(4, 64, 64, dt=5) == -1
    assert rff(4, 64, 64, dt=0) == -2 and rff(4, 72, 64) == -2 and rff(4, 12, 64) == -2 and rff(4, 64, 96) == -2
    assert rff(4, 64, 64, x=null) == -1 and rff(4, 64, 64, W=odd) == -1 and rff(4, 64, 64, y=null) == -1
    assert L.la_feature_map_rff_backward(ok, ok, ok, ok, 4, 64, 64, 1, null) == -1          # dx aliases x
    assert L.la_feature_map_rff_backward(ok, ok, null, far, 4, 64, 64, 1, null) == -1
    assert L.la_feature_map_rff_backward(ok, ok, ok, far, 0, 64, 64, 1, null) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()


def test_plan_override_is_an_explicit_call(L):
    p = la.make_problem(4, 16, 18 * 128, 64, 64, la.LA_BF16)
    auto = la.la_causal_plan(p)
    try:
        la.la_plan_override(causal_pieces=5)
        assert la.la_causal_plan(p)["pieces"] == 5
        la.la_plan_override(causal_short=0)
        assert la.la_causal_plan(p)["pieces"] == 2
        assert L.la_plan_override(0, -1, -1) == -1 and L.la_plan_override(-1, -2, -1) == -1
    finally:
        la.la_plan_override()
    assert la.la_causal_plan(p) == auto


def _cpu(shape, dtype=torch.float32):
    return torch.zeros(shape, dtype=dtype)


def test_binding_rejects_mismatched_tensors_before_any_pointer_is_taken():
    """The kernels trust the problem descriptor, which the binding derives from Q and V: every other tensor
    must agree with it.  CPU tensors throughout: a check that let one of these through would then stop at
    "must live on a CUDA device", never at a launch."""
    B, H, N, D, M = 2, 3, 16, 32, 16
    Q, K, V, G = _cpu((B, H, N, D)), _cpu((B, H, N, D)), _cpu((B, H, N, M)), _cpu((B, H, N, M))
    bad = [
        (la.la_causal_forward, (Q, _cpu((B, H, N - 1, D)), V), {}, "K"),
        (la.la_causal_forward, (Q, K.bfloat16(), V), {}, "K"),
        (la.la_causal_forward, (Q, K, _cpu((B, H, N + 1, M))), {}, "V"),
        (la.la_causal_forward, (Q, K, V), {"den": _cpu((B, H, N), torch.bfloat16)}, "den"),
        (la.la_causal_forward, (Q, K, V), {"den": _cpu((B, H, N - 1))}, "den"),
        (la.la_causal_forward, (Q, K, V), {"O": _cpu((B, H, N, D))}, "O"),
        (la.la_causal_forward, (Q, K, V), {"S_out": _cpu((B, H, M, D))}, "S_out"),
        (la.la_causal_forward, (Q, K, V), {"Z_in": _cpu((B, H, D), torch.float64), "S_in": _cpu((B, H, D, M))}, "Z_in"),
        (la.la_causal_forward, (Q, K, V), {"saved": _cpu((64,))}, "saved"),
        (la.la_causal_backward, (Q, K, V, _cpu((B, H, N, D))), {}, "G"),
        (la.la_causal_backward, (Q, K, V, G), {"dK": _cpu((B, H, N, D), torch.bfloat16)}, "dK"),
        (la.la_causal_backward, (Q, K, V, G), {"dS_in": _cpu((B, H, D))}, "dS_in"),
        (la.la_linear_attention, (Q, K, V), {"KV": _cpu((B, H, D, M), torch.bfloat16)}, "KV"),
        (la.la_linear_attention, (Q, K, V), {"Zs": _cpu((B, H, M))}, "Zs"),
        (la.la_linear_attention_backward, (Q, K, V, G), {"dV": _cpu((B, H, N, D))}, "dV"),
        (la.la_linear_attention_varlen, (Q, K, V, torch.zeros(B, dtype=torch.int64)), {}, "lengths"),
        (la.la_linear_attention_noalloc, (Q, K, V), {"den": _cpu((B, H, N + 3))}, "den"),
        (la.la_recurrent_step, (Q[:, :, 0], K[:, :, 0], V[:, :, 0], _cpu((B, H, D, M), torch.bfloat16), _cpu((B, H, D))), {}, "S"),
        (la.la_recurrent_step, (Q[:, :, 0], K[:, :, 1:3, 0], V[:, :, 0], _cpu((B, H, D, M)), _cpu((B, H, D))), {}, "k"),
        (la.la_recurrent_steps, (Q, K, V, _cpu((B, H, D, M)), _cpu((B, H, M))), {}, "Z"),
        (la.la_feature_map, (Q,), {"out": _cpu((B, H, N, D), torch.bfloat16)}, "out"),
        (la.la_feature_map_poly2, (_cpu((B, N, 4)),), {"out": _cpu((B, N, 8))}, "out"),
    ]
    for fn, args, kw, name in bad:
        with pytest.raises(ValueError, match=name):
            fn(*args, **kw)
    # well-formed arguments get as far as the device check and no further
    for fn, args in ((la.la_causal_forward, (Q, K, V)), (la.la_causal_backward, (Q, K, V, G)),
                     (la.la_linear_attention, (Q, K, V)), (la.la_feature_map, (Q,))):
        with pytest.raises(ValueError, match="CUDA device"):
            fn(*args)
