"""Error measure and tolerances shared by the GPU parity tests.

Every output is a set of vectors, one per position (a row of O, dQ, dK, dV, a row of
the state, ...; a [B,H,N] tensor such as den is a set of 1-vectors).  "Relative error" is
taken per position in the max norm,

    err = max over positions i of  ||x_i - r_i||_inf / scale_i ,
    scale_i = max(||r_i||_inf, median of ||r_j||_inf over the 33 positions around i),

the largest deviation of any element, relative to the largest element of the vector
it belongs to.  The median over the neighbouring positions only matters for a vector
that is much smaller than its neighbours: a row that vanishes analytically (the
gradient of the first causal query: O_1 = V_1 whatever Q_1 is) or by chance (with
nearly uniform attention a gradient row is close to c_i (1,...,1) with c_i of either
sign, and among thousands of rows some c_i fall arbitrarily close to 0); such a row
has no scale of its own and is judged against the rows next to it.  A tensor that is
zero altogether (N = 1) is compared absolutely.  Gates: 1e-4 for fp32 I/O, 2e-2 for
bf16 I/O (fp32 accumulation); inputs are rounded to the I/O type once and both sides
consume those rounded values.

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
    """row_scale: [..., N, 1] norm of each position's vector -> the scale it is judged against."""
    from scipy.ndimage import median_filter
    biggest = np.abs(ref).max()
    if biggest < 1e-12:                                       # whole tensor analytically zero (N = 1)
        return np.ones_like(row_scale)
    if row_scale.shape[-2] > 1:
        size = [1] * row_scale.ndim
        size[-2] = 33
        row_scale = np.maximum(row_scale, median_filter(row_scale, size=size, mode="mirror"))
    return np.where(row_scale > 1e-9 * biggest, row_scale, biggest)


def max_rel_err(x, ref) -> float:
    """Per-position relative error in the max norm (the gated measure)."""
    x, ref = _as_f64(x), np.asarray(ref, np.float64)
    assert x.shape == ref.shape, (x.shape, ref.shape)
    if x.size == 0:
        return 0.0
    assert np.isfinite(x).all(), "non-finite values in the result"
    if ref.ndim == 1:                                         # element-wise map: plain relative error
        return float((np.abs(x - ref) / np.maximum(np.abs(ref), 1e-30)).max())
    if ref.ndim == 3:                                         # [B,H,N]: one scalar per position
        x, ref = x[..., None], ref[..., None]
    floor = _row_floor(ref, np.abs(ref).max(axis=-1, keepdims=True))
    return float((np.abs(x - ref) / floor).max())


def max_rel_err_rms(x, ref) -> float:
    """Element-wise |x - r| / max(|r|, rms of r over the row)."""
    x, ref = _as_f64(x), np.asarray(ref, np.float64)
    if x.size == 0:
        return 0.0
    if ref.ndim == 1:
        return max_rel_err(x, ref)
    if ref.ndim == 3:
        x, ref = x[..., None], ref[..., None]
    rms = _row_floor(ref, np.sqrt((ref ** 2).mean(axis=-1, keepdims=True)))
    return float((np.abs(x - ref) / np.maximum(np.abs(ref), rms)).max())


def assert_close(x, ref, dtype, what="", grad=False):
    err = max_rel_err(x, ref)
    assert err <= TOL[dtype], f"{what}: max relative error {err:.3e} > {TOL[dtype]:.0e}"
    strict = max_rel_err_rms(x, ref)
    gate = TOL_RMS_GRAD[dtype] if grad else TOL[dtype]
    assert strict <= gate, f"{what}: element-wise error over the row rms {strict:.3e} > {gate:.0e}"
    return err
