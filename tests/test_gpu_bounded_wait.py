"""The give-up path of the kernels' bounded waits, exercised safely.

Every spin wait of the tensor-core kernels (on an mbarrier fed by TMA, by a tcgen05.commit or
by another warp role) goes through one routine with a poll limit; when the limit runs out the
routine ORs a code into the device status word and returns false, the role drains and the CTA
leaves normally.  A production launch never gets there, so this test builds a few lines of
CUDA around the very same header with the limit set to a thousand polls and waits on a barrier
that nobody arrives at: a few milliseconds, no trap, no fault, and the context stays usable.
"""
import ctypes
import os
import subprocess

import pytest
import torch

import paper_2006_16236_b200 as la

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_a_wait_that_runs_out_reports_and_returns(tmp_path):
    so = tmp_path / "libwait_timeout.so"
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
                    "-shared", "-DLA_WAIT_LIMIT=1000u", "-I", os.path.join(ROOT, "paper_2006_16236_b200", "csrc"),
                    "-o", str(so), os.path.join(ROOT, "tests", "cuda", "wait_timeout.cu")], check=True)
    lib = ctypes.CDLL(str(so))
    res = (ctypes.c_int * 4)()
    torch.zeros(1, device="cuda:0")                      # a context on the device the test uses
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    rc = lib.run_wait_timeout(res)
    t1.record()
    torch.cuda.synchronize()
    assert rc == 0, f"CUDA error {rc}: the context did not survive"
    status, silent, served, limit = list(res)
    assert limit == 1000
    assert served == 1                                   # a barrier that is arrived at completes the wait
    assert silent == 0                                   # the silent one makes it give up ...
    assert status == 4                                   # ... with exactly its own code (pipe timeout) in the status word
    assert t0.elapsed_time(t1) < 2000.0                  # milliseconds: bounded, and far below any watchdog
    # the context is intact: the library computes as before
    x = torch.linspace(-3, 3, 1000, device="cuda:0")
    y = la.la_feature_map(x)
    assert torch.allclose(y, torch.where(x > 0, x + 1, torch.exp(x)), rtol=1e-6, atol=1e-6)
    la.la_last_device_status()
