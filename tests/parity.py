"""Error measure and tolerances shared by the GPU parity tests.

Measure: per element |x - r| / max(|r|, rms(r over the last axis at that
position)); the gate is the maximum over all elements.  The floor keeps the
measure meaningful where an output, being an average of zero-mean values,
passes through zero.  A row of the reference that is zero analytically (the
gradient of the first causal query: O_1 = V_1 whatever Q_1 is, so its gradient
is an exact cancellation) has no scale of its own; there the floor is the
largest magnitude in the tensor (1 if the whole tensor is zero, as for N = 1).  Gates: 1e-4 for fp32 I/O, 2e-2 for bf16 I/O (fp32
accumulation); inputs are rounded to the I/O type once and both sides consume
those rounded values.
"""
import numpy as np
import torch

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}


def max_rel_err(x, ref) -> float:
    x = x.detach().double().cpu().numpy() if hasattr(x, "detach") else np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    assert x.shape == ref.shape, (x.shape, ref.shape)
    if x.size == 0:
        return 0.0
    assert np.isfinite(x).all(), "non-finite values in the result"
    rms = np.sqrt((ref ** 2).mean(axis=-1, keepdims=True))
    biggest = np.abs(ref).max()
    if biggest < 1e-12:                                       # whole tensor analytically zero (N = 1)
        biggest = 1.0
    rms = np.where(rms > 1e-9 * biggest, rms, biggest)        # analytically-zero rows
    floor = np.maximum(np.abs(ref), rms)
    floor = np.where(floor > 0, floor, 1.0)
    return float((np.abs(x - ref) / floor).max())


def assert_close(x, ref, dtype, what=""):
    err = max_rel_err(x, ref)
    assert err <= TOL[dtype], f"{what}: max relative error {err:.3e} > {TOL[dtype]:.0e}"
    return err
