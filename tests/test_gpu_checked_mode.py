"""Checked mode (LA_DEBUG=1): tensor arguments are looked up with the driver before a launch.

The variable is read once per process, so the checks run in a child process.  The failing case
is chosen so that it would be harmless even if the check did not fire: every tensor is really
there in full; only the workspace SIZE is overstated (a terabyte), which the span check refuses
while a launch would use no more of the workspace than exists.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import ctypes, sys
import numpy as np, torch
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
import oracle
import paper_2006_16236_b200 as la
from paper_2006_16236_b200 import binding
from paper_2006_16236_b200.inputs import draw_qkvg
from parity import assert_close

B, H, N, D = 2, 2, 512, 64
Q, K, V, G = draw_qkvg(B, H, N, D, D, seed=9, dtype=torch.bfloat16)
Qd, Kd, Vd, Gd = (t.cuda() for t in (Q, K, V, G))
# 1. checked mode computes what unchecked mode computes (the call synchronises and reads the status itself)
O = la.la_causal_forward(Qd, Kd, Vd)
dQ, dK, dV = la.la_causal_backward(Qd, Kd, Vd, Gd)
ref = oracle.linear_attention(*(t.double().numpy() for t in (Q, K, V)), causal=True)[0]
assert_close(O, ref, torch.bfloat16, "checked O")
S, Z = torch.zeros((B, H, D, D), device="cuda"), torch.zeros((B, H, D), device="cuda")
la.la_recurrent_step(Qd[:, :, 0].contiguous(), Kd[:, :, 0].contiguous(), Vd[:, :, 0].contiguous(), S, Z)
# 2. a workspace whose stated size reaches past its allocation is refused before anything is enqueued
p = la.make_problem(B, H, N, D, D, la.LA_BF16)
ws = la.workspace(p, la.LA_OP_CAUSAL_FORWARD, torch.device("cuda"))
assert ws.numel() > 0
Od = torch.empty_like(Vd)
n0 = la.la_kernel_launches()
vp = ctypes.c_void_p
rc = binding.lib().la_causal_forward(ctypes.byref(p), vp(Qd.data_ptr()), vp(Kd.data_ptr()), vp(Vd.data_ptr()), vp(Od.data_ptr()),
                                     None, None, None, None, 0, vp(ws.data_ptr()), ctypes.c_size_t(1 << 40),
                                     vp(torch.cuda.current_stream().cuda_stream))
msg = binding.lib().la_last_error().decode()
assert rc == -1, (rc, msg)
assert "checked mode" in msg and "ws" in msg, msg
assert la.la_kernel_launches() == n0, "nothing may be enqueued after a refused argument"
# 3. host memory where device memory is expected
host = torch.zeros(ws.numel(), dtype=torch.uint8).pin_memory()       # as large as the workspace: harmless whatever happens
rc = binding.lib().la_causal_forward(ctypes.byref(p), vp(Qd.data_ptr()), vp(Kd.data_ptr()), vp(Vd.data_ptr()), vp(Od.data_ptr()),
                                     None, None, None, None, 0, vp(host.data_ptr()), ctypes.c_size_t(ws.numel()),
                                     vp(torch.cuda.current_stream().cuda_stream))
msg = binding.lib().la_last_error().decode()
assert rc == -1 and "not device memory" in msg, (rc, msg)
assert la.la_kernel_launches() == n0
print("checked mode ok")
"""


def test_checked_mode_in_a_child_process():
    env = dict(os.environ, LA_DEBUG="1")
    r = subprocess.run([sys.executable, "-c", CHILD, ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "checked mode ok" in r.stdout
