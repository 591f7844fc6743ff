"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it only draws i.i.d. normal
tensors with the shapes of the paper's workloads (autoregressive pixel
sequences, a bidirectional speech encoder, the sequence-length sweep of the
synthetic benchmark, many-stream decoding) and rounds them to the I/O dtype.
Both the CUDA path and the CPU oracle consume exactly these values, so input
quantisation never counts as error.

Recipe: ``torch.Generator('cpu').manual_seed(seed)``; draw Q, K, V, G in that
order with ``torch.randn(shape, dtype=float32)``; multiply Q, K, V by ``scale``;
round once to the I/O dtype.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str          # "causal" | "noncausal" | "decode"
    B: int
    H: int
    N: int             # sequence length (number of decode steps for "decode")
    D: int
    M: int
    dtype: str         # "f32" | "bf16"
    seed: int
    scale: float = 1.0
    mirrors: str = ""

    @property
    def tokens(self) -> int:
        return self.B * self.N

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


def _sweep(n_log2: int) -> Workload:
    N = 1 << n_log2
    return Workload(f"causal_sweep_bf16_N{N}", "causal", 131072 // N, 8, N, 64, 64, "bf16",
                    4000 + n_log2, 1.0, "sequence-length scaling benchmark, batch ~ 1/N")


WORKLOADS = {
    w.name: w for w in [
        Workload("causal_fp32_small", "causal", 1, 2, 256, 32, 32, "f32", 0, 1.0,
                 "small fp32 reference case"),
        Workload("noncausal_bf16_speech", "noncausal", 8, 8, 4096, 64, 64, "bf16", 2, 0.125,
                 "bidirectional encoder shape (speech model)"),
        Workload("causal_bf16_image", "causal", 16, 8, 3072, 32, 32, "bf16", 3, 1.0,
                 "autoregressive pixel sequence, 32x32x3 image flattened"),
        _sweep(12), _sweep(13), _sweep(14), _sweep(15), _sweep(16),
        Workload("decode_bf16_streams", "decode", 256, 8, 3072, 64, 64, "bf16", 5, 1.0,
                 "many-stream autoregressive generation, one recurrent step per pixel"),
        Workload("causal_fp32_N4096", "causal", 32, 8, 4096, 64, 64, "f32", 6, 1.0,
                 "the N = 4096 point of the sequence-length benchmark in fp32 (general kernels)"),
    ]
}


def draw_qkvg(B: int, H: int, N: int, D: int, M: int, seed: int, dtype=torch.float32,
              scale: float = 1.0, with_grad: bool = True):
    """Return CPU tensors Q,K [B,H,N,D], V,G [B,H,N,M] (G is None without ``with_grad``)."""
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    Q = torch.randn((B, H, N, D), generator=g, dtype=torch.float32)
    K = torch.randn((B, H, N, D), generator=g, dtype=torch.float32)
    V = torch.randn((B, H, N, M), generator=g, dtype=torch.float32)
    G = torch.randn((B, H, N, M), generator=g, dtype=torch.float32) if with_grad else None
    if scale != 1.0:
        Q, K, V = Q * scale, K * scale, V * scale
    cast = lambda t: None if t is None else t.to(dtype).contiguous()
    return cast(Q), cast(K), cast(V), cast(G)


def draw_workload(w: Workload, with_grad: bool = True):
    """Tensors of a named workload.  For "decode", Q,K,V are [B,H,T,D]: step t uses slice t."""
    return draw_qkvg(w.B, w.H, w.N, w.D, w.M, w.seed, w.torch_dtype, w.scale,
                     with_grad and w.kind != "decode")
