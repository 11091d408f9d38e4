"""The tensor-core pair path evaluates GELU as u/2 (1 + tanh(u (c1 + c2 u^2))) with two fitted
coefficients instead of the erf form the layer is defined with.  This pins the coefficients that are
compiled into the kernels: read from the source, evaluated in fp64 on a dense grid, the formula must stay
within 2.8e-4 of u/2 (1 + erf(u / sqrt 2)) everywhere (the figure the header and the parity tolerance rely
on), and must be clearly better than the textbook tanh form's 4.7e-4."""
import math
import os
import re

import numpy as np

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                   "paper_2510_02345_b200", "csrc", "tc2_common.cuh")


def _coefficients():
    text = open(SRC).read()
    body = text[text.index("gelu_fast2("):]
    body = body[:body.index("return")]
    nums = [float(v) for v in re.findall(r"__float2half2_rn\(([0-9.eE+-]+)f\)", body)]
    assert len(nums) == 3 and nums[2] == 0.5, nums      # c2, c1, and the 1/2 of u/2
    return nums[1], nums[0]


def test_fitted_tanh_form_stays_within_its_stated_bound_of_the_erf_form():
    c1, c2 = _coefficients()
    u = np.linspace(-12.0, 12.0, 2_400_001)
    erf = np.vectorize(math.erf)
    exact = 0.5 * u * (1.0 + erf(u / math.sqrt(2.0)))
    fit = 0.5 * u * (1.0 + np.tanh(u * (c1 + c2 * u * u)))
    dev = np.abs(fit - exact)
    assert dev.max() <= 2.8e-4, dev.max()
    assert 1.0 < abs(u[np.argmax(dev)]) < 3.0          # the worst point sits on the shoulder, not in a tail
    textbook = 0.5 * u * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (u + 0.044715 * u ** 3)))
    assert np.abs(textbook - exact).max() > 4.0e-4      # what the refit improves on
    # odd symmetry of the correction and the limits: GELU(u) -> u for large u, -> 0 for large -u
    assert abs(fit[-1] - 12.0) < 1e-12 and abs(fit[0]) < 1e-12
