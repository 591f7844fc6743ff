"""Where the gate on bf16 gradients comes from (no GPU needed).

The tensor-core kernels consume phi(Q) and phi(K) as bf16 tiles: that is the method's
prescribed data path, not a choice of these kernels.  This test measures what that one
rounding costs, with everything else exact: the fp64 oracle is run in its identity mode
on features rounded to bf16 (Algorithm 1's own convention: gradients with respect to
phi(Q), phi(K)), the chain rule through phi is applied in fp64, and the result is
compared with the oracle on the unrounded features under the measures of parity.py.
Nothing of the CUDA path is involved and nothing else is rounded: no bf16 scores, no
bf16 copy of the running state, no rounded outputs.

Finding (asserted below): under the element-wise measure with the row rms as floor, the
causal dQ already sits at 2e-2 and dK at 1.5e-2 on four heads of a 4096-position problem;
the maximum grows with the number of elements (6 to 7 sigma at benchmark size, 2.5e-2 on
sixteen heads of the N = 16384 benchmark problem).  A gate of 2e-2 under that measure
therefore cannot be met by any implementation that feeds bf16 feature tiles to the tensor
cores; TOL_RMS_GRAD = 5e-2 is this floor times two.  The gated row-norm measure stays
below 1e-2 for the same rounding, which is why it can be held to 2e-2.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_16236_b200.inputs import draw_qkvg
from parity import TOL, TOL_RMS_GRAD, max_rel_err, max_rel_err_rms


def _bf16(x):
    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).double().numpy()


def _gradients_with_rounded_features(Q, K, V, G, causal):
    fq, fk = oracle.feature_map(Q), oracle.feature_map(K)
    gq, gk, gv = oracle.linear_attention_backward(_bf16(fq), _bf16(fk), V, G, causal, phi="identity")
    return gq * oracle.feature_map(Q, True), gk * oracle.feature_map(K, True), gv


@pytest.mark.parametrize("shape", [(1, 4, 4096, 64), (1, 4, 3072, 32)], ids=["D64_N4096", "D32_N3072"])
def test_bf16_feature_tiles_alone_reach_the_strict_gate(shape):
    B, H, N, D = shape
    Q, K, V, G = (t.double().numpy() for t in draw_qkvg(B, H, N, D, D, seed=4, dtype=torch.bfloat16))
    ref = oracle.linear_attention_backward(Q, K, V, G, True)
    emu = _gradients_with_rounded_features(Q, K, V, G, True)
    gated = [max_rel_err(e, r) for e, r in zip(emu, ref)]
    rms = [max_rel_err_rms(e, r) for e, r in zip(emu, ref)]
    # the row-norm measure has room below its gate ...
    assert max(gated) <= 0.6 * TOL[torch.bfloat16], gated
    # ... the element-wise one has none: operand rounding alone is at the benchmark spec's 2e-2 for dQ
    assert rms[0] >= 0.9 * TOL[torch.bfloat16], rms
    assert rms[1] >= 0.6 * TOL[torch.bfloat16], rms
    # and the gate in force for gradients leaves about a factor of two for every other rounding of a kernel
    assert max(rms) <= 0.6 * TOL_RMS_GRAD[torch.bfloat16], rms
    # dV does not see the cancellation (it is linear in the features): an order of magnitude lower
    assert rms[2] <= 0.2 * TOL[torch.bfloat16], rms


def test_the_error_is_a_tail_of_many_small_ones():
    """The spread of the element-wise error is a third of a percent of the row rms; 2e-2 is its six-sigma tail."""
    B, H, N, D = 1, 2, 4096, 64
    Q, K, V, G = (t.double().numpy() for t in draw_qkvg(B, H, N, D, D, seed=5, dtype=torch.bfloat16))
    ref = oracle.linear_attention_backward(Q, K, V, G, True)[0][:, :, 64:]
    emu = _gradients_with_rounded_features(Q, K, V, G, True)[0][:, :, 64:]
    rel = (emu - ref) / np.sqrt((ref ** 2).mean(-1, keepdims=True))
    sigma = rel.std()
    assert 2e-3 <= sigma <= 5e-3, sigma
    assert np.abs(rel).max() >= 4.5 * sigma
