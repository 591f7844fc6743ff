"""Error measure and tolerances shared by the GPU parity tests.

Every output is a set of vectors, one per position (a row of O, dQ, dK, dV, a row of
the state, ...).  "Relative error" is taken per position in the max norm,

    err = max over positions i of  ||x_i - r_i||_inf / ||r_i||_inf ,

the largest deviation of any element, relative to the largest element of the vector
it belongs to.  Gates: 1e-4 for fp32 I/O, 2e-2 for bf16 I/O (fp32 accumulation);
inputs are rounded to the I/O type once and both sides consume those rounded values.

A row of the reference that is zero analytically has no scale of its own (the
gradient of the first causal query: O_1 = V_1 whatever Q_1 is, so its gradient is an
exact cancellation); there the floor is the largest magnitude in the tensor (1 if the
whole tensor is zero, as for N = 1).

A stricter element-wise variant, |x - r| / max(|r|, rms of r over the row), is also
computed (`max_rel_err_rms`).  fp32 results and the bf16 forward outputs meet the same
gates under it; bf16 gradients are allowed 5e-2 there: every gradient element is a
difference of terms about 2.4 times its own size (the gradient of a normalised
average is orthogonal to phi(Q_i)), each term carries the 2^-9 rounding of the bf16
tensor-core operands, and the maximum over 10^7..10^8 elements sits 5-6 standard
deviations out, which lands at 2-3e-2 of the row rms for any implementation that
feeds bf16 phi(Q), phi(K) tiles to the tensor cores.
"""
import numpy as np
import torch

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}
TOL_RMS_GRAD = {torch.float32: 1e-4, torch.bfloat16: 5e-2}


def _as_f64(x):
    return x.detach().double().cpu().numpy() if hasattr(x, "detach") else np.asarray(x, np.float64)


def _row_floor(ref, row_scale):
    biggest = np.abs(ref).max()
    if biggest < 1e-12:                                       # whole tensor analytically zero (N = 1)
        biggest = 1.0
    return np.where(row_scale > 1e-9 * biggest, row_scale, biggest)        # analytically-zero rows


def max_rel_err(x, ref) -> float:
    """Per-position relative error in the max norm (the gated measure)."""
    x, ref = _as_f64(x), np.asarray(ref, np.float64)
    assert x.shape == ref.shape, (x.shape, ref.shape)
    if x.size == 0:
        return 0.0
    assert np.isfinite(x).all(), "non-finite values in the result"
    floor = _row_floor(ref, np.abs(ref).max(axis=-1, keepdims=True))
    return float((np.abs(x - ref) / floor).max())


def max_rel_err_rms(x, ref) -> float:
    """Element-wise |x - r| / max(|r|, rms of r over the row)."""
    x, ref = _as_f64(x), np.asarray(ref, np.float64)
    if x.size == 0:
        return 0.0
    rms = _row_floor(ref, np.sqrt((ref ** 2).mean(axis=-1, keepdims=True)))
    return float((np.abs(x - ref) / np.maximum(np.abs(ref), rms)).max())


def assert_close(x, ref, dtype, what="", grad=False):
    err = max_rel_err(x, ref)
    assert err <= TOL[dtype], f"{what}: max relative error {err:.3e} > {TOL[dtype]:.0e}"
    strict = max_rel_err_rms(x, ref)
    gate = TOL_RMS_GRAD[dtype] if grad else TOL[dtype]
    assert strict <= gate, f"{what}: element-wise error over the row rms {strict:.3e} > {gate:.0e}"
    return err
