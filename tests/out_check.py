"""Element-level acceptance test for an output vector or matrix against the oracle's (numpy only).

Two numbers are formed: the relative L2 error, and the largest single-element error measured in
units of the reference's root mean square.  The first is the project's stated metric (1e-4 for
fp32 storage, 2e-2 for bf16 storage); the second is what notices ONE wrong element, or a short
wrong segment, which the L2 number of a wide vector averages away (one element of 4096 wholly
wrong moves the relative L2 error by only 1/64).  The bounds used by the tests are a small
multiple of the worst error measured on the GPU over the whole test suite (printed at the end of
a run with GRIFFIN_TEST_STATS=1), far inside the stated metric.
"""
import os

import numpy as np

STATED_L2 = {"f32": 1e-4, "bf16": 2e-2}      # the stated bounds on the relative L2 error
# bf16 storage: y is rounded to bf16 (half an ulp = 2^-9 of the element, elements reach 4-5 rms) and the
# activations between the two products are rounded to bf16 (2^-9 each, averaging out over k terms);
# measured worst case over the suite (1123 outputs): relative L2 3.0e-3, largest element error 0.019 rms.
# fp32 storage: fp32 accumulation over d and k terms in a fixed but different order from the oracle's;
# measured worst case (231 outputs): relative L2 1.3e-6, largest element error 1.2e-5 rms.
# The bounds are about 2.6 times (bf16) and 3-4 times (fp32) those worst cases.
TEST_L2 = {"f32": 5e-6, "bf16": 8e-3}
TEST_MAX_OVER_RMS = {"f32": 4e-5, "bf16": 0.05}

_stats = {}


def output_error(y, ref):
    """(relative L2 error, largest element error / rms of the reference)."""
    y, ref = np.asarray(y, np.float64), np.asarray(ref, np.float64)
    assert y.shape == ref.shape, (y.shape, ref.shape)
    assert np.all(np.isfinite(y)), "non-finite output"
    diff = y - ref
    norm = max(float(np.linalg.norm(ref)), 1e-300)
    rms = norm / np.sqrt(ref.size)
    return float(np.linalg.norm(diff)) / norm, float(np.max(np.abs(diff))) / rms


def assert_output(y, ref, dtype, what=None, scale=1.0):
    """Both bounds, for one output of storage type `dtype`.  scale = 2 when two rounded results are compared
    with each other instead of one with the exact reference."""
    l2, mx = output_error(y, ref)
    s = _stats.setdefault(dtype, [0.0, 0.0, 0])
    s[0], s[1], s[2] = max(s[0], l2 / scale), max(s[1], mx / scale), s[2] + 1
    assert l2 <= STATED_L2[dtype], ("relative L2 beyond the stated bound", what, l2)
    if os.environ.get("GRIFFIN_TEST_STATS") == "loose":     # collecting the worst case: only the stated bound applies
        return l2, mx
    assert l2 <= scale * TEST_L2[dtype], ("relative L2", what, l2)
    assert mx <= scale * TEST_MAX_OVER_RMS[dtype], ("largest element error / rms", what, mx)
    return l2, mx


def stats():
    return {k: {"worst_rel_l2": v[0], "worst_max_over_rms": v[1], "outputs": v[2]} for k, v in _stats.items()}
