"""GELU of the MLP between the two fully-connected layers (fp64, CPU).

TEST INFRASTRUCTURE ONLY, like the rest of this package.

The paper's GPT-2 uses GELU activations with no bias (App. "Hyperparameters"); the definition is
GELU(y) = y Phi(y) with Phi the standard normal distribution function, so GELU'(y) = Phi(y) + y phi(y).
Phi is written through the error function, Phi(y) = (1 + erf(y / sqrt 2)) / 2 (math.erf, element by element).

Pins (tests/test_oracle_activation.py): Phi against a trapezoid integral of the normal density, table values of
Phi at 0, +-1, 2, the identity GELU(y) - GELU(-y) = y, the limits for large |y|, the derivative against central
differences and its zero at the minimum of GELU.
"""
from __future__ import annotations

import math

import numpy as np

_erf = np.frompyfunc(math.erf, 1, 1)


def phi_cdf(y) -> np.ndarray:
    y = np.asarray(y, dtype=np.float64)
    return 0.5 * (1.0 + np.asarray(_erf(y / math.sqrt(2.0)), dtype=np.float64))


def gelu(y) -> np.ndarray:
    y = np.asarray(y, dtype=np.float64)
    return y * phi_cdf(y)


def gelu_grad(y) -> np.ndarray:
    y = np.asarray(y, dtype=np.float64)
    return phi_cdf(y) + y * np.exp(-0.5 * y * y) / math.sqrt(2.0 * math.pi)
