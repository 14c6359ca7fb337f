"""Where the comparison rule of the GPU parity tests comes from.

The kernels take bf16 inputs, accumulate in fp32, round the softmax weights to bf16 before the PV
product and round the output to bf16.  This file evaluates exactly that rounding scheme in fp64
numpy (no blocking, no online softmax: the max and the sum are exact) against the unrounded
result, on inputs drawn like the workloads' (i.i.d. N(0,1), head_dim 128, scale 1/sqrt(128)), and
checks that the scheme itself stays inside the three bounds of ``tests/_util.compare`` with room
to spare: the bounds measure the arithmetic the method prescribes, and a kernel that passes them
adds little on top."""
import numpy as np

import oracle
from tests._util import ABS_TOL, REL_TOL


def _bf16(x):
    return oracle.bits_to_f64(oracle.f64_to_bits(x))


def test_bf16_weight_and_output_rounding_stay_inside_the_comparison_rule():
    rng = np.random.default_rng(5)
    rows, keys, D = 2048, 4096, 128
    q, k, v = (_bf16(rng.standard_normal(s)) for s in [(rows, D), (keys, D), (keys, D)])
    s = (q @ k.T) / np.sqrt(D)
    p = np.exp(s - s.max(axis=1, keepdims=True))            # unnormalised weights in (0, 1]
    l = p.sum(axis=1, keepdims=True)
    exact = (p @ v) / l
    model = _bf16((_bf16(p) @ v) / l)                        # weights and output rounded to bf16
    err = np.abs(model - exact)
    rms = np.linalg.norm(exact, axis=1) / np.sqrt(D)
    row_rel = np.linalg.norm(model - exact, axis=1) / np.linalg.norm(exact, axis=1)
    el_rel = (err / (np.abs(exact) + rms[:, None])).max()
    # The scheme's own error: the absolute and the row-norm bounds hold with a wide margin; the elementwise
    # bound |err| <= REL_TOL * (|ref| + rms(row)) is the tight one -- the rounding scheme alone reaches 0.7-0.9
    # of it over a few hundred thousand elements (rounded weights add errors of about 1e-3 * rms(row) per
    # element, whose extremes reach 5-6 standard deviations), so the kernels must add almost nothing to it.
    assert err.max() <= 0.1 * ABS_TOL
    assert 5e-4 <= row_rel.max() <= 0.5 * REL_TOL
    assert 0.5 * REL_TOL <= el_rel <= REL_TOL
    # with the floor max(|ref|, rms) in place of the sum the same arithmetic sits right at the bound: that
    # form would test the noise of bf16 weights, not the kernels
    assert (err / np.maximum(np.abs(exact), rms[:, None])).max() > 0.85 * REL_TOL
    # output rounding alone (at most 2^-8 relative) is the smaller part
    out_only = np.abs(_bf16(exact) - exact) / (np.abs(exact) + rms[:, None])
    assert out_only.max() <= 2.0 ** -8 and el_rel > 2 * out_only.max()
