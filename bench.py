#!/usr/bin/env python
"""Benchmark of the linear-attention hot path on B200.

One step = la_causal_forward + la_causal_backward over one batch of synthetic
input (the feature map, the normalising division and the state recurrence are
fused inside those calls).  The default workload is the N=16384 point of the
sequence-length sweep (B=8, H=8, D=M=64, bf16); `--workload` selects any other
named workload, and, at one GPU, the remaining rows of the hot path (non-causal
forward+backward, the image-shaped causal case, the other sweep points and the
3072-step recurrent decode) are timed as well and reported under "rows".

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a
bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2006_16236_b200 import shard  # noqa: E402
from paper_2006_16236_b200.inputs import WORKLOADS, draw_qkvg, draw_workload  # noqa: E402

METRIC = "causal LA fwd+bwd tokens/s"
DEFAULT_WORKLOAD = "causal_sweep_bf16_N16384"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

def ncu_traffic():
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the library's kernels, by
    workload and kernel, as the last ncu capture of this source tree recorded them in a tracked JSON file
    (written by `python -m paper_2006_16236_b200.ncu_summary`); {} when there is none."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        with open(path) as f:
            return json.load(f)
    except (OSError, ValueError):
        return {}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    return dict(FALLBACK_PEAKS, source="fallback")


def elem_bytes(w):
    return 4 if w.dtype == "f32" else 2


def algorithmic_bytes(w, part):
    """Compulsory HBM bytes: every input read once, every output written once."""
    th = w.B * w.H * w.N
    e = elem_bytes(w)
    if w.kind == "decode":
        return w.B * w.H * (8 * w.D * w.M + 8 * w.D + (2 * w.D + 2 * w.M) * e)
    fwd = th * ((2 * w.D + 2 * w.M) * e + 4)                      # Q,K,V in; O, den out
    bwd = th * ((2 * w.D + 2 * w.M) * e + (2 * w.D + w.M) * e + 4)  # Q,K,V,G (+den) in; dQ,dK,dV out
    return {"fwd": fwd, "bwd": bwd, "both": fwd + bwd}[part]


def algorithmic_flops(w, part):
    th = w.B * w.H * w.N
    if w.kind == "decode":
        return w.B * w.H * 4 * w.D * w.M
    if w.kind == "noncausal":
        return {"fwd": 4, "bwd": 8, "both": 12}[part] * w.D * w.M * th
    return {"fwd": 4, "bwd": 10, "both": 14}[part] * w.D * w.M * th


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background; stop() keeps the samples that
    fall inside the given wall-clock windows (the timed region, extended by identical steps when it is
    shorter than a few sampling periods)."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self, windows):
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                clock, cmax = float(c[1]), float(c[2])
            except ValueError:
                continue
            if not any(lo <= ts <= hi for lo, hi in windows):
                continue
            sm.append(clock)
            mx.append(cmax)
            for nm, val in zip(names, c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus):
    return shard.init_process_group("nccl")


def barrier(world):
    shard.barrier(world)


def max_over_ranks(x, world, dev):
    return shard.max_over_ranks(x, world, dev)


# --------------------------------------------------------------------------- GPU arms
class CausalStep:
    def __init__(self, la, w, dev, from_state=False):
        self.la, self.w, self.dev = la, w, dev
        Q, K, V, G = draw_qkvg(w.B, w.H, w.N, w.D, w.M, w.seed, w.torch_dtype, w.scale)
        self.host = [t.pin_memory() for t in (Q, K, V, G)]
        self.d = [t.to(dev) for t in self.host]
        self.O = torch.empty_like(self.d[2])
        self.den = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
        self.grads = [torch.empty_like(self.d[0]), torch.empty_like(self.d[1]), torch.empty_like(self.d[2])]
        self.host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in [self.O] + self.grads]
        self.causal = w.kind == "causal"
        # a training step keeps phi(Q), phi(K) from the forward for the backward (None: nothing to keep)
        self.saved = la.saved_buffer(self.d[0], self.d[2]) if self.causal else la.linear_saved_buffer(self.d[0], self.d[2])
        # a step in the middle of a longer sequence: the forward continues from a given state and returns the
        # final one, the backward takes the final state's upstream gradient and returns the initial state's
        self.state = None
        if from_state:
            g = torch.Generator().manual_seed(w.seed + 1)
            sS, sZ = (w.B, w.H, w.D, w.M), (w.B, w.H, w.D)
            mk = lambda shape, scale, shift=0.0: (torch.rand(shape, generator=g) * scale + shift).to(dev)
            self.state = {"S_in": mk(sS, 2.0, -1.0), "Z_in": mk(sZ, 4.0, 1.0), "dS_out": mk(sS, 0.02, -0.01),
                          "dZ_out": mk(sZ, 0.02, -0.01), "S_out": torch.empty(sS, device=dev), "Z_out": torch.empty(sZ, device=dev),
                          "dS_in": torch.empty(sS, device=dev), "dZ_in": torch.empty(sZ, device=dev)}

    def fwd(self):
        Q, K, V, _ = self.d
        if self.causal and self.state:
            st = self.state
            self.la.la_causal_forward(Q, K, V, O=self.O, den=self.den, saved=self.saved, S_in=st["S_in"], Z_in=st["Z_in"],
                                      S_out=st["S_out"], Z_out=st["Z_out"])
        elif self.causal:
            self.la.la_causal_forward(Q, K, V, O=self.O, den=self.den, saved=self.saved)
        else:
            self.la.la_linear_attention(Q, K, V, O=self.O, den=self.den, saved=self.saved)

    def bwd(self):
        Q, K, V, G = self.d
        dQ, dK, dV = self.grads
        if self.causal and self.state:
            st = self.state
            self.la.la_causal_backward(Q, K, V, G, O=self.O, den=self.den, saved=self.saved, dQ=dQ, dK=dK, dV=dV,
                                       S_in=st["S_in"], Z_in=st["Z_in"], dS_out=st["dS_out"], dZ_out=st["dZ_out"],
                                       dS_in=st["dS_in"], dZ_in=st["dZ_in"])
        elif self.causal:
            self.la.la_causal_backward(Q, K, V, G, O=self.O, den=self.den, saved=self.saved, dQ=dQ, dK=dK, dV=dV)
        else:
            self.la.la_linear_attention_backward(Q, K, V, G, O=self.O, den=self.den, dQ=dQ, dK=dK, dV=dV, saved=self.saved)

    def step(self):
        self.fwd()
        self.bwd()

    def e2e_pipelined(self, n):
        """n end-to-end steps as a caller with a data pipeline runs them: every step copies its Q, K, V, G from
        pinned host memory, runs forward + backward through the binding and copies O, dQ, dK, dV back; the
        host-to-device copy of the next step and the device-to-host copy of the previous one run on their own
        streams next to the kernels (two sets of device buffers), so both directions of the link are busy."""
        main = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        if not hasattr(self, "sets"):
            second = ([torch.empty_like(t) for t in self.d], torch.empty_like(self.O),
                      torch.empty_like(self.den), [torch.empty_like(t) for t in self.grads])
            self.sets = [(self.d, self.O, self.den, self.grads), second]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_comp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        for i in range(n):
            b = i & 1
            d, O, den, grads = self.sets[b]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_comp[b])          # the kernels of step i - 2 have read this set
                for h, t in zip(self.host, d):
                    t.copy_(h, non_blocking=True)
                ev_in[b].record(s_in)
            main.wait_event(ev_in[b])
            if i >= 2:
                main.wait_event(ev_out[b])               # the results of step i - 2 have left this set
            Q, K, V, G = d
            if self.causal:
                self.la.la_causal_forward(Q, K, V, O=O, den=den, saved=self.saved)
                self.la.la_causal_backward(Q, K, V, G, O=O, den=den, saved=self.saved, dQ=grads[0], dK=grads[1], dV=grads[2])
            else:
                self.la.la_linear_attention(Q, K, V, O=O, den=den)
                self.la.la_linear_attention_backward(Q, K, V, G, O=O, den=den, dQ=grads[0], dK=grads[1], dV=grads[2])
            ev_comp[b].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[b])
                for h, t in zip(self.host_out, [O] + grads):
                    h.copy_(t, non_blocking=True)
                ev_out[b].record(s_out)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    def e2e_bytes(self):
        h2d = sum(t.numel() * t.element_size() for t in self.host)
        d2h = sum(t.numel() * t.element_size() for t in self.host_out)
        return h2d, d2h


def time_steps(run, steps, warmup, world, split=None):
    """Time `steps` calls of run() with CUDA events on the current stream; returns total ms and,
    when split=(fwd, bwd) is given instead of run, the mean ms of each part."""
    for _ in range(warmup):
        run() if split is None else (split[0](), split[1]())
    barrier(world)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(steps):
        if split is None:
            run()
        else:
            ev[i][0].record()
            split[0]()
            ev[i][1].record()
            split[1]()
            ev[i][2].record()
    t1.record()
    torch.cuda.synchronize()
    total = t0.elapsed_time(t1)
    barrier(world)
    if split is None:
        return total, None
    f = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    b = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    return total, (f, b)


# Compulsory HBM bytes of one launch of each main kernel, per token-head (D = M = dim, e = element bytes):
# the tensors that kernel has to read or write once (tile inputs, outputs, per-position scalars).
KERNEL_ALG_BYTES = {
    "causal_fwd_kernel": lambda d, e: 4 * d * e + 4,            # Q, K, V in; O, den out
    "causal_bwd_dq_kernel": lambda d, e: 5 * d * e + 8,         # Q, K, V, G in; dQ, dn, dl out
    "causal_bwd_dkv_kernel": lambda d, e: 6 * d * e + 8,        # Q, K, V, G, dn, dl in; dK, dV out
    "linear_apply_kernel": None,                                # three variants share the name: not ranked
}


def bench_attention(la, w, dev, steps, warmup, world, rank, pk, do_e2e=True, from_state=False):
    s = CausalStep(la, shard.rank_workload(w, world, rank), dev, from_state=from_state)
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    for _ in range(warmup):
        s.step()
    torch.cuda.synchronize()
    # Timed region: K plain steps.  The per-kernel durations (roofline, breakdown) come from a second pass
    # of K steps right after it with the library's event pairs around every kernel and an event between
    # forward and backward: those records cost about 7 % of a step, so they stay out of the timed region.
    launches0 = la.la_kernel_launches()
    t_lo = time.time()
    total_ms, _ = time_steps(s.step, steps, 0, world)
    launches = la.la_kernel_launches() - launches0
    la.la_profile_enable(True)
    _, (fwd_ms, bwd_ms) = time_steps(None, steps, 0, world, split=(s.fwd, s.bwd))
    t_hi = time.time()
    kernels = la.la_profile_read()
    la.la_profile_enable(False)
    windows = [(t_lo, t_hi)]
    if sampler:                 # the timed region may be shorter than a few sampling periods: keep the
        t2 = time.time()        # same load running for half a second so that the clocks are seen under it
        while time.time() - t2 < 0.5:
            s.step()
        torch.cuda.synchronize()
        windows.append((t2, time.time()))
    clocks = sampler.stop(windows) if sampler else None
    la.la_last_device_status()
    total_ms = max_over_ranks(total_ms, world, dev)
    ms = total_ms / steps
    tokens = w.tokens * world
    res = {
        "value": tokens / (ms * 1e-3), "ms_per_step": ms, "fwd_ms": fwd_ms, "bwd_ms": bwd_ms,
        "gpu_launches": int(launches), "clocks": clocks,
        "alg_gbs": algorithmic_bytes(w, "both") / ms * 1e-6,
        "alg_tflops": algorithmic_flops(w, "both") / ms * 1e-9,
        "kernels_ms": {k: {"ms_per_launch": v[0], "launches": v[1]} for k, v in kernels.items()},
    }
    res["hbm_frac"] = res["alg_gbs"] / pk["hbm_gbs"]
    res["tensor_frac_alg_flops"] = res["alg_tflops"] / pk["bf16_tflops_sustained"]
    # dominant kernel: the one with the largest total time among those with a defined byte count
    th = w.B * w.H * w.N
    # (kernels within 2 % of the largest total time count as tied: run-to-run noise would otherwise pick
    # between them; the tie goes to the one that moves the most algorithmic bytes)
    ranked = [(v[0] * v[1], k, v[0]) for k, v in kernels.items() if KERNEL_ALG_BYTES.get(k)]
    if ranked:
        top = max(r[0] for r in ranked)
        tied = [r for r in ranked if r[0] >= 0.98 * top]
        _, dom, dom_ms = max(tied, key=lambda r: KERNEL_ALG_BYTES[r[1]](w.D, elem_bytes(w)))
        dom_bytes = KERNEL_ALG_BYTES[dom](w.D, elem_bytes(w)) * th
    else:                       # general kernels: one kernel per call
        dom = ("la_causal_" if w.kind == "causal" else "la_linear_attention_") + ("backward" if bwd_ms >= fwd_ms else "forward")
        dom_ms = max(bwd_ms, fwd_ms)
        dom_bytes = algorithmic_bytes(w, "bwd" if bwd_ms >= fwd_ms else "fwd")
    ach = dom_bytes / dom_ms * 1e-6
    traffic = ncu_traffic()
    res["roofline"] = {
        "kernel": dom, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
        "peak_source": pk["source"] + " copy bandwidth (burst figure: the kernel is timed alone by its own event pair)",
        "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_ms,
        "traffic": traffic.get("bytes_per_launch", {}).get(w.name, {}).get(dom),
        "traffic_source": traffic.get("source"),
        # the whole step against the same peak: every input of forward + backward read once, every output written
        # once (4De+4 and 7De+4 bytes per token-head), over the time of the step.  `frac` above is the dominant
        # kernel on the bytes that kernel has to move; the second sweep's re-reads, the saved tiles and the
        # pre-passes only show here.
        "step_frac": res["hbm_frac"], "step_algorithmic_bytes": algorithmic_bytes(w, "both"), "step_ms": ms,
    }
    if do_e2e:
        e_steps = max(4, min(steps, 10))
        s.e2e_pipelined(3)
        e_ms, _ = time_steps(lambda: s.e2e_pipelined(e_steps), 1, 0, world)
        e_ms = max_over_ranks(e_ms, world, dev) / e_steps
        h2d, d2h = s.e2e_bytes()
        res["e2e"] = {"value": tokens / (e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e_ms,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e_steps,
                      "how": "every step copies its inputs from pinned host memory and its results back; copies of "
                             "neighbouring steps overlap the kernels on two extra streams (two sets of device buffers)"}
    del s
    torch.cuda.empty_cache()
    return res


def bench_decode(la, w, dev, pk, n_steps=None, batch=None):
    """3072 sequential la_recurrent_step launches, timed as a whole: once issued one by one
    from the host, once replayed from a CUDA graph that holds the same 3072 launches."""
    T = n_steps or w.N
    if batch:                   # same recipe, other batch size (a state that cannot stay in L2)
        import dataclasses
        w = dataclasses.replace(w, B=batch, N=T, name=f"{w.name}_B{batch}")
    Q, K, V, _ = draw_workload(w)
    q_t, k_t, v_t = (t[:, :, :T].permute(2, 0, 1, 3).contiguous().to(dev) for t in (Q, K, V))
    S = torch.zeros((w.B, w.H, w.D, w.M), device=dev)
    Z = torch.zeros((w.B, w.H, w.D), device=dev)
    out = torch.empty((T, w.B, w.H, w.M), dtype=w.torch_dtype, device=dev)

    def run_all():
        for t in range(T):
            la.la_recurrent_step(q_t[t], k_t[t], v_t[t], S, Z, out=out[t])

    def timed(fn):
        S.zero_()
        Z.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / T            # us per step

    for t in range(16):
        la.la_recurrent_step(q_t[t], k_t[t], v_t[t], S, Z, out=out[t])
    us_eager = timed(run_all)
    # the same loop as a C caller would issue it: the exported function with ready-made arguments, none of the
    # binding's per-call checks and allocations
    import ctypes
    from paper_2006_16236_b200 import binding
    fn = binding.lib().la_recurrent_step
    pr = ctypes.byref(binding.make_problem(w.B, w.H, 1, w.D, w.M, binding.LA_BF16 if w.dtype == "bf16" else binding.LA_F32))
    vp = ctypes.c_void_p
    argv = [(vp(q_t[t].data_ptr()), vp(k_t[t].data_ptr()), vp(v_t[t].data_ptr()), vp(out[t].data_ptr())) for t in range(T)]
    Sp, Zp, st = vp(S.data_ptr()), vp(Z.data_ptr()), vp(torch.cuda.current_stream().cuda_stream)

    def run_raw():
        for q, k, v, o in argv:
            fn(pr, q, k, v, Sp, Zp, o, st)

    us_raw = timed(run_raw)
    # the binding's prepared form: arguments checked and marshalled once per buffer set, then one foreign call per step
    steps = [la.prepare_recurrent_step(q_t[t], k_t[t], v_t[t], S, Z, out=out[t]) for t in range(T)]

    def run_prepared():
        for step in steps:
            step()

    us_prepared = timed(run_prepared)
    us_graph = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                run_all()
        torch.cuda.current_stream().wait_stream(side)
        timed(graph.replay)
        us_graph = timed(graph.replay)
    except Exception as exc:  # noqa: BLE001 - report, keep the eager number
        us_graph = None
        graph_error = repr(exc)
    la.la_last_device_status()
    us = min(us_eager, us_raw, us_graph) if us_graph else min(us_eager, us_raw)
    gbs = algorithmic_bytes(w, "both") / us * 1e-3
    res = {"workload": w.name, "steps_per_s": 1e6 / us, "us_per_step": us, "launches": T,
           "us_per_step_host_issued": us_eager, "us_per_step_host_issued_raw_c_abi": us_raw, "us_per_step_host_issued_prepared": us_prepared,
           "us_per_step_cuda_graph": us_graph,
           "alg_gbs": gbs, "hbm_frac": gbs / pk["hbm_gbs"], "state_bytes": S.numel() * 4,
           "note": ("state fits the 126 MB L2, so the fraction may exceed the DRAM roofline"
                    if S.numel() * 4 < 100e6 else "state exceeds L2: every step streams it from and to HBM")}
    if us_graph is None:
        res["graph_error"] = graph_error
    # the same steps sixteen at a time in one launch (inputs known beforehand): the state crosses HBM once per
    # sixteen steps instead of once per step
    G16 = 16
    T16 = min(T, 512) // G16 * G16
    if T16:
        chunks = [tuple(t[:, :, c:c + G16].contiguous().to(dev) for t in (Q, K, V)) for c in range(0, T16, G16)]
        o16 = torch.empty((w.B, w.H, G16, w.M), dtype=w.torch_dtype, device=dev)

        def run_fused():
            for qc, kc, vc in chunks:
                la.la_recurrent_steps(qc, kc, vc, S, Z, out=o16)

        run_fused()
        S.zero_()
        Z.zero_()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_fused()
        e1.record()
        torch.cuda.synchronize()
        res["us_per_step_16_steps_per_launch"] = e0.elapsed_time(e1) * 1e3 / T16
        la.la_last_device_status()
    return res


def bench_decode_layer(la, w, dev, pk, T=512):
    """T tokens through la_decode_layer_step (projections + recurrent step + output projection + residual per
    token), each token's input being the previous token's output (two buffers alternate), as in generation:
    issued call by call through the binding, through the raw C ABI, and replayed from a CUDA graph."""
    import ctypes
    from paper_2006_16236_b200 import binding
    B, H, D = w.B, w.H, w.D
    F = H * D
    g = torch.Generator().manual_seed(w.seed + 3)
    s = 1.0 / F ** 0.5
    Wqkv = (torch.randn((3 * F, F), generator=g) * s).to(torch.bfloat16).to(dev)
    Wo = (torch.randn((F, F), generator=g) * s * 0.1).to(torch.bfloat16).to(dev)
    x0 = torch.randn((B, F), generator=g).to(torch.bfloat16).to(dev)
    buf = [x0.clone(), torch.empty_like(x0)]
    S = torch.zeros((B, H, D, D), device=dev)
    Z = torch.zeros((B, H, D), device=dev)
    p = la.make_problem(B, H, 1, D, D, la.LA_BF16)
    ws = la.workspace(p, la.LA_OP_DECODE_LAYER, dev)

    def reset():
        buf[0].copy_(x0)
        S.zero_()
        Z.zero_()

    def run_binding():
        for t in range(T):
            la.la_decode_layer_step(buf[t & 1], Wqkv, Wo, S, Z, out=buf[(t + 1) & 1], ws=ws)

    fn = binding.lib().la_decode_layer_step
    vp = ctypes.c_void_p
    pr, st = ctypes.byref(p), vp(torch.cuda.current_stream().cuda_stream)
    args = [(vp(buf[t & 1].data_ptr()), vp(buf[(t + 1) & 1].data_ptr())) for t in range(2)]
    fixed = (vp(Wqkv.data_ptr()), vp(Wo.data_ptr()), vp(S.data_ptr()), vp(Z.data_ptr()))
    wsp, wsn = vp(ws.data_ptr()), ws.numel()

    def run_raw(stream=st):
        for t in range(T):
            x, y = args[t & 1]
            fn(pr, x, fixed[0], fixed[1], fixed[2], fixed[3], y, wsp, wsn, stream)

    def timed(fnc):
        reset()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fnc()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / T

    n0 = la.la_kernel_launches()
    run_raw()
    res = {"workload": f"decode_layer_B{B}_H{H}_D{D}", "tokens": T, "launches_per_token": (la.la_kernel_launches() - n0) // T,
           "us_per_token_host_issued": timed(run_binding), "us_per_token_host_issued_raw_c_abi": timed(run_raw)}
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                run_raw(vp(side.cuda_stream))
        torch.cuda.current_stream().wait_stream(side)
        timed(graph.replay)
        res["us_per_token_cuda_graph"] = timed(graph.replay)
    except Exception as exc:  # noqa: BLE001 - report, keep the eager numbers
        res["graph_error"] = repr(exc)
    la.la_profile_enable(True)
    reset()
    run_raw()
    torch.cuda.synchronize()
    res["kernels_us"] = {k: round(v[0] * 1e3, 2) for k, v in la.la_profile_read().items() if v[1]}
    la.la_profile_enable(False)
    la.la_last_device_status()
    best = min(v for k, v in res.items() if k.startswith("us_per_token"))
    res["tokens_per_s_per_stream"] = 1e6 / best
    # the bytes a token has to move: the fp32 state read and written once, the weights read once, x in, y out
    nbytes = B * H * (8 * D * D + 8 * D) + 4 * F * F * 2 + 2 * B * F * 2
    res["alg_gbs"] = nbytes / best * 1e-3
    res["hbm_frac"] = res["alg_gbs"] / pk["hbm_gbs"]
    res["note"] = "state (32 MiB) and weights (2 MiB) fit the L2: the fraction is against the HBM copy bandwidth for scale only"
    return res


# --------------------------------------------------------------------------- CPU oracle arm
def bench_poly2(la, w, dev, pk, iters=10):
    """Degree-2 polynomial feature map (Section 3.2.1) and its gradient on the headline workload's rows with
    D = 8 (C = 64 feature columns, what the tensor-core attention kernels take): two tensors alternate, so that
    each launch's 150 MB are not in L2 from the launch before."""
    rows, D, C = w.B * w.H * w.N, 8, 64
    g = torch.Generator(device="cpu").manual_seed(w.seed + 17)
    xs = [torch.randn((rows, D), generator=g).to(torch.bfloat16).to(dev) for _ in range(2)]
    ys = [torch.empty((rows, C), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    dxs = [torch.empty_like(x) for x in xs]
    out = {"rows": rows, "D": D, "C": C, "dtype": "bf16"}
    for name, fn, nbytes in (
            ("forward", lambda i: la.la_feature_map_poly2(xs[i], C, out=ys[i]), rows * (D + C) * 2),
            ("backward", lambda i: la.la_feature_map_poly2_backward(xs[i], ys[i], out=dxs[i]), rows * (2 * D + C) * 2)):
        for i in range(4):
            fn(i & 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record()
        for i in range(iters):
            fn(i & 1)
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / iters
        out[name] = {"ms": round(ms, 4), "alg_gbs": round(nbytes / ms / 1e6, 1),
                     "hbm_frac": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 3)}
    return out


def bench_ragged(la, w, dev, pk, iters=10):
    """The headline shape as a right-padded ragged batch (lengths uniform in [N/2, N], the mix of a speech batch):
    forward + backward through the calls that take `lengths`, against the same tensors processed at full length,
    both with the saved buffer."""
    Q, K, V, G = (t.to(dev) for t in draw_qkvg(w.B, w.H, w.N, w.D, w.M, w.seed, w.torch_dtype, w.scale))
    g = torch.Generator(device="cpu").manual_seed(w.seed + 23)
    lengths = torch.randint(w.N // 2, w.N + 1, (w.B,), generator=g, dtype=torch.int32)
    ln = lengths.to(dev)
    O, den = torch.empty_like(V), torch.empty((w.B, w.H, w.N), device=dev)
    dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)

    saved = la.saved_buffer(Q, V)

    def ragged():
        la.la_causal_forward(Q, K, V, lengths=ln, O=O, den=den, saved=saved)
        la.la_causal_backward(Q, K, V, G, lengths=ln, dQ=dQ, dK=dK, dV=dV, saved=saved)

    def full():
        la.la_causal_forward(Q, K, V, O=O, den=den, saved=saved)
        la.la_causal_backward(Q, K, V, G, dQ=dQ, dK=dK, dV=dV, saved=saved)

    out = {"lengths": lengths.tolist(), "real_fraction": round(float(lengths.sum()) / (w.B * w.N), 3)}
    for name, fn in (("ragged_ms", ragged), ("full_length_ms", full)):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        out[name] = round(e0.elapsed_time(e1) / iters, 4)
    out["real_tokens_per_s"] = round(float(lengths.sum()) / (out["ragged_ms"] * 1e-3), 1)
    la.la_last_device_status()
    return out


def bench_feature_map(la, w, dev, pk, iters=10):
    """The stand-alone feature map of Eq. 7 on the headline workload's Q (value and slope): two tensors alternate,
    so that a launch's 268 MB are not in L2 from the launch before."""
    rows, D = w.B * w.H * w.N, w.D
    g = torch.Generator(device="cpu").manual_seed(w.seed + 29)
    xs = [torch.randn((rows, D), generator=g).to(w.torch_dtype).to(dev) for _ in range(2)]
    ys = [torch.empty_like(x) for x in xs]
    nbytes = 2 * rows * D * xs[0].element_size()
    out = {"rows": rows, "D": D, "dtype": w.dtype}
    for name, deriv in (("value", False), ("slope", True)):
        for i in range(4):
            la.la_feature_map(xs[i & 1], deriv=deriv, out=ys[i & 1])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record()
        for i in range(iters):
            la.la_feature_map(xs[i & 1], deriv=deriv, out=ys[i & 1])
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / iters
        out[name] = {"ms": round(ms, 4), "alg_gbs": round(nbytes / ms / 1e6, 1),
                     "hbm_frac": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 3)}
    return out


def bench_rff(la, w, dev, pk, iters=10):
    """Random Fourier features (the map the paper's conclusion proposes) and their gradient on the headline
    workload's rows with D = 64 inputs and C = 64 features (what the tensor-core attention kernels take): two
    tensors alternate, so that a launch's 270 MB are not in L2 from the launch before."""
    rows, D, C = w.B * w.H * w.N, 64, 64
    g = torch.Generator(device="cpu").manual_seed(w.seed + 19)
    W = torch.randn((C // 2, D), generator=g).to(torch.bfloat16).to(dev)
    xs = [(torch.randn((rows, D), generator=g) * 0.5).to(torch.bfloat16).to(dev) for _ in range(2)]
    ys = [torch.empty((rows, C), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    dxs = [torch.empty_like(x) for x in xs]
    out = {"rows": rows, "D": D, "C": C, "dtype": "bf16"}
    for name, fn, nbytes in (
            ("forward", lambda i: la.la_feature_map_rff(xs[i], W, out=ys[i]), rows * (D + C) * 2),
            ("backward", lambda i: la.la_feature_map_rff_backward(xs[i], W, ys[i], out=dxs[i]), rows * (2 * D + C) * 2)):
        for i in range(4):
            fn(i & 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(dev)
        e0.record()
        for i in range(iters):
            fn(i & 1)
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / iters
        out[name] = {"ms": round(ms, 4), "alg_gbs": round(nbytes / ms / 1e6, 1),
                     "hbm_frac": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 3)}
    la.la_last_device_status()
    return out


def oracle_sample(w, pairs):
    """Inputs of the first `pairs` (batch, head) pairs of workload w, as [1, pairs, N, .]."""
    Q, K, V, G = draw_qkvg(1, pairs, w.N, w.D, w.M, w.seed, w.torch_dtype, w.scale)
    return [t.double().numpy() for t in (Q, K, V, G)]


def oracle_step(oracle, w, data):
    Q, K, V, G = data
    causal = w.kind == "causal"
    oracle.linear_attention(Q, K, V, causal)
    oracle.linear_attention_backward(Q, K, V, G, causal)


def cpu_baseline(w, budget_s=15.0):
    import oracle
    cores = oracle.num_threads()
    data = oracle_sample(w, cores)
    t0 = time.perf_counter()
    oracle_step(oracle, w, data)
    once = time.perf_counter() - t0
    reps = max(1, min(20, int(budget_s / max(once, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_step(oracle, w, data)
    dt = (time.perf_counter() - t0) / reps
    frac = cores / (w.B * w.H)
    # the same on one thread, on one (batch, head) pair
    one = [t[:, :1] for t in data]
    oracle.set_threads(1)
    try:
        t0 = time.perf_counter()
        oracle_step(oracle, w, one)
        dt1 = time.perf_counter() - t0
    finally:
        oracle.set_threads(cores)
    return {"value": w.tokens * frac / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"{cores} of {w.B * w.H} (batch, head) pairs of {w.name}, fwd+bwd, {reps} repetitions; "
                      "rate scaled to whole-workload tokens",
            "one_thread": {"value": w.tokens / (w.B * w.H) / dt1, "unit": "tokens/s", "cores": 1,
                           "sample": f"1 of {w.B * w.H} (batch, head) pairs, fwd+bwd, once; rate scaled to whole-workload tokens"}}


def run_reference(args):
    """The oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    w = WORKLOADS[args.workload]
    cores = oracle.num_threads()
    data = oracle_sample(w, cores)
    frac = cores / (w.B * w.H)
    for _ in range(args.warmup):
        oracle_step(oracle, w, data)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, w, data)
    ms = (time.perf_counter() - t0) / args.steps * 1e3
    value = w.tokens * frac / (ms * 1e-3)
    sample = f"{cores} of {w.B * w.H} (batch, head) pairs per step; rate scaled to whole-workload tokens"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(w, 1), timing="host wall clock around the oracle call on a bounded sample of the workload"),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "kind": "oracle", "cores": cores, "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_config(w, world):
    return {"workload": w.name, "mirrors": w.mirrors, "B_per_gpu": w.B, "H": w.H, "N": w.N, "D": w.D, "M": w.M,
            "io_dtype": w.dtype, "phi": "elu+1", "eps": 0.0, "seed": w.seed,
            "parallelism": f"{world} independent shard(s) of (batch, head) pairs, no collective",
            "l2": "per-step working set (inputs+outputs >= 1 GiB at the default workload) exceeds the 126 MB L2; no flush needed",
            "timing": "value: K plain steps between two CUDA events; roofline and breakdown: a second pass of K steps "
                      "with an event pair around every kernel (the records cost about 7 % of a step)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=[k for k, v in WORKLOADS.items() if v.kind != "decode"])
    ap.add_argument("--main-only", action="store_true", help="skip the other hot-path rows and the CPU baseline")
    ap.add_argument("--decode-only", type=int, default=0, metavar="T",
                    help="only the recurrent-decode rows, T steps each (a short run for a profiler capture)")
    ap.add_argument("--decode-batch", type=int, default=0, metavar="B",
                    help="with --decode-only: only the row with B streams per head (default: 256 and 2048)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    world, rank, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    import paper_2006_16236_b200 as la
    pk = peaks()
    w = WORKLOADS[args.workload]

    if args.decode_only:
        dw = next(v for v in WORKLOADS.values() if v.kind == "decode")
        batches = [args.decode_batch] if args.decode_batch else [dw.B, 2048]
        rows = {f"{dw.name}_B{b}": bench_decode(la, dw, dev, pk, n_steps=args.decode_only, batch=b) for b in batches}
        if not args.decode_batch:
            rows["decode_layer"] = bench_decode_layer(la, dw, dev, pk, T=args.decode_only)
        print(json.dumps({"rows": rows}))
        return
    main_res = bench_attention(la, w, dev, args.steps, args.warmup, world, rank, pk)

    rows = {}
    if world == 1 and not args.main_only:
        k, wu = max(3, min(args.steps, 10)), 3
        for name, ww in WORKLOADS.items():
            if name == w.name:
                continue
            if ww.kind == "decode":
                rows[name] = bench_decode(la, ww, dev, pk)
                rows[name + "_B2048"] = bench_decode(la, ww, dev, pk, n_steps=256, batch=2048)
                rows["decode_layer"] = bench_decode_layer(la, ww, dev, pk)
            else:
                r = bench_attention(la, ww, dev, k, wu, 1, 0, pk, do_e2e=False)
                rows[name] = {kk: r[kk] for kk in ("value", "ms_per_step", "fwd_ms", "bwd_ms", "alg_gbs", "hbm_frac",
                                                   "alg_tflops", "tensor_frac_alg_flops", "gpu_launches", "kernels_ms")}
                rows[name]["unit"] = "tokens/s"
        # the headline workload as a step in the middle of a longer sequence (state in and out, both passes)
        r = bench_attention(la, w, dev, k, wu, 1, 0, pk, do_e2e=False, from_state=True)
        rows[w.name + "_from_state"] = {kk: r[kk] for kk in ("value", "ms_per_step", "fwd_ms", "bwd_ms", "alg_gbs", "hbm_frac",
                                                              "gpu_launches", "kernels_ms")}
        rows[w.name + "_from_state"]["unit"] = "tokens/s"
        rows["feature_map_elu1"] = bench_feature_map(la, w, dev, pk)
        rows["feature_map_poly2"] = bench_poly2(la, w, dev, pk)
        rows["feature_map_rff"] = bench_rff(la, w, dev, pk)
        rows[w.name + "_ragged"] = bench_ragged(la, w, dev, pk)

    cpu = None
    if rank == 0 and world == 1 and not args.main_only:
        cpu = cpu_baseline(w)

    if rank == 0:
        line = {
            "metric": METRIC, "value": main_res["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": main_res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
            "data": "synthetic", "config": workload_config(w, world), "clocks": main_res["clocks"],
            "e2e": main_res.get("e2e"), "gpu_launches": main_res["gpu_launches"],
            "roofline": main_res["roofline"], "cpu_baseline": cpu,
            "breakdown": {kk: main_res[kk] for kk in ("fwd_ms", "bwd_ms", "alg_gbs", "hbm_frac", "alg_tflops",
                                                      "tensor_frac_alg_flops", "kernels_ms")},
            "peaks": {kk: pk.get(kk) for kk in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "source")},
            "rows": rows,
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
