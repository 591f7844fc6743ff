"""Host-side checks that need no GPU: the library loads, exports the declared symbols,
sizes workspaces and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

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
    assert L.la_feature_map(ok, ok, -5, 0, 0, null) == -1
    assert L.la_feature_map(ok, ok, 0, 0, 0, null) == 0
    assert L.la_feature_map(ok, ok, 4, 9, 0, null) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
