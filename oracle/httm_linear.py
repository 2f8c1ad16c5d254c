"""CPU oracle of the projections around the path (Algorithm 1: Q, K, V = x W_qkv and out = Attn W_o): plain numpy
in float64.  TEST INFRASTRUCTURE ONLY: imported by tests/; the product path shares no code with it.

The operation has a plain definition, written out here: y[i][o] = sum_k x[i][k] * w[o][k] on the exact values of the
bf16 inputs (weights stored as [out_features][in_features]); no bias."""
from __future__ import annotations

import numpy as np

from . import httm_oracle as orc


def linear(x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """x [n][in], w [out][in] as bf16 bit patterns -> y [n][out] float64."""
    x = orc.bf16_to_double(x_bits)
    w = orc.bf16_to_double(w_bits)
    assert x.ndim == 2 and w.ndim == 2 and x.shape[1] == w.shape[1]
    return x @ w.T


def magnitude(x_bits: np.ndarray, w_bits: np.ndarray) -> np.ndarray:
    """sum_k |x[i][k]| |w[o][k]|: the scale of the rounding error of an fp32 accumulation of that sum."""
    return np.abs(orc.bf16_to_double(x_bits)) @ np.abs(orc.bf16_to_double(w_bits)).T
