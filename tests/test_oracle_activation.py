"""Pins for the oracle's GELU and its derivative (CPU only): values the definition fixes, the reflection identities,
an independent library's normal distribution, and central differences."""
import math

import numpy as np
from scipy.stats import norm

import oracle


def test_gelu_against_the_normal_distribution_of_another_library():
    z = np.linspace(-6, 6, 241)
    assert np.allclose(oracle.gelu(z), z * norm.cdf(z), rtol=1e-13, atol=1e-15)
    assert oracle.gelu(np.array([0.0]))[0] == 0.0
    assert abs(oracle.gelu(np.array([1.0]))[0] - 0.8413447460685429) < 1e-15       # Phi(1)


def test_gelu_derivative_values_identities_and_central_differences():
    z = np.linspace(-5, 5, 201)
    one = np.ones_like(z)
    d = oracle.act_backward_gelu(z, one)
    assert abs(oracle.act_backward_gelu(np.array([0.0]), np.array([1.0]))[0] - 0.5) < 1e-16
    assert np.allclose(d, norm.cdf(z) + z * norm.pdf(z), rtol=1e-13, atol=1e-15)
    assert np.allclose(d + d[::-1], 1.0, rtol=1e-13)                                # gelu'(z) + gelu'(-z) = 1
    eps = 1e-6
    num = (oracle.gelu(z + eps) - oracle.gelu(z - eps)) / (2 * eps)
    assert np.allclose(d, num, rtol=1e-8, atol=1e-9)
    # the minimum of the derivative, -0.1289..., sits where z^2 = 2 ... no closed form: only its sign pattern is pinned
    assert d[z < -0.76].max() < 0 and d[z > -0.75].min() > 0
    # the upstream gradient multiplies element-wise
    g = np.random.default_rng(0).standard_normal(z.shape)
    assert np.allclose(oracle.act_backward_gelu(z, g), g * d, rtol=1e-15)
    assert math.isclose(oracle.act_backward_gelu(np.array([10.0]), np.array([3.0]))[0], 3.0, rel_tol=1e-12)
