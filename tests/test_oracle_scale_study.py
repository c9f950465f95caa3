"""The oracle's E4M3 codec against closed forms on normal draws: what the scale study counts (elements that
underflow to zero, elements that land on the largest code) has a textbook value for N(0, sigma^2) inputs, so a
codec that rounds the wrong way near zero or near 448 fails here.

For y ~ N(0, sigma^2) encoded with round-to-nearest-even and saturation:
  * y becomes +-0 iff |y| <= 2^-10 (half the smallest subnormal 2^-9; the tie goes to the even code 0):
    probability erf(2^-10 / (sigma sqrt 2));
  * y becomes +-448 (code 0x7E) iff |y| >= 432 (the midpoint of 416 and 448; the tie goes to 448, whose mantissa
    field 110 is even; everything above 448 saturates): probability erfc(432 / (sigma sqrt 2)).
The draws are bf16 values (as the path's inputs are), which moves the two thresholds by less than 2^-8 relative.
"""
import math

import numpy as np
import pytest

import oracle
import synth


def _codes(sigma, n_tokens=2048):
    x = synth.draw_study_stream("gauss", sigma, 4, n_tokens)          # bf16 [4][n][8][64]: 4.2 M samples
    vals = x.float().numpy().astype(np.float32).reshape(-1)
    return vals, oracle.e4m3_encode_array(vals)


@pytest.mark.parametrize("log2_sigma", [-12, -10, -8, -6])
def test_underflow_fraction_of_a_normal_draw(log2_sigma):
    sigma = 2.0 ** log2_sigma
    vals, codes = _codes(sigma)
    p = math.erf(2.0 ** -10 / (sigma * math.sqrt(2)))
    got = float(((codes & 0x7F) == 0).mean())
    tol = 5 * math.sqrt(p * (1 - p) / vals.size) + 2.0 ** -8 * p + 1e-6      # sampling error + bf16 granularity
    assert abs(got - p) <= tol, (got, p, tol)


@pytest.mark.parametrize("log2_sigma", [7, 8, 9, 10])
def test_largest_code_fraction_of_a_normal_draw(log2_sigma):
    sigma = 2.0 ** log2_sigma
    vals, codes = _codes(sigma)
    p = math.erfc(432.0 / (sigma * math.sqrt(2)))
    got = float(((codes & 0x7F) == 0x7E).mean())
    tol = 5 * math.sqrt(p * (1 - p) / vals.size) + 2.0 ** -6 * p + 1e-6
    assert abs(got - p) <= tol, (got, p, tol)
    clipped = float((np.abs(vals) >= 464).mean())     # the study's "clipped" count: nearest would be a code above 448
    assert abs(clipped - math.erfc(464.0 / (sigma * math.sqrt(2)))) <= tol


def test_scaled_draw_never_clips_and_keeps_relative_error():
    """With scale = amax/448 nothing exceeds 448, and the relative RMS error of the codes that stay normal is the
    3-bit-mantissa figure: uniform rounding error over a binade gives about 2^-4 / sqrt(12) / E[m] ~ 0.026."""
    sigma = 2.0 ** -6
    x = synth.draw_study_stream("gauss", sigma, 4, 512).float().numpy().astype(np.float32).reshape(-1, 8, 64)
    scale = oracle.calibrate_scales(x, pow2=False)
    assert np.array_equal(scale, (np.abs(x).max(axis=(0, 2)) / np.float32(448)).astype(np.float32))
    y = (x / scale[None, :, None]).astype(np.float32)
    assert np.abs(y).max() < 448.0 * (1 + 2.0 ** -20)     # the float32 quotient of the largest element may round just above 448
    codes = oracle.e4m3_encode_array(y.reshape(-1))
    assert ((codes & 0x7F) == 0x7E).sum() >= 8              # every head's largest element lands on the largest code
    table = np.array([oracle.e4m3_decode(c) for c in range(256)])
    deq = table[codes].reshape(y.shape)
    big = np.abs(y) >= 2.0 ** -6                                            # normal codes only
    rel = np.sqrt(np.mean(((deq - y)[big] / y[big]) ** 2))
    assert 0.018 <= rel <= 0.032, rel
