"""Oracle for the quantization-error analysis (test infrastructure; never imported by the product path).

The paper's first experiment (Sec. 4.1 "Quantization-Error Evaluation", results in Sec. 4.2 / Table 1)
measures the reconstruction error of the K and V caches per head: with the dequantized cache A^,
MSE(A, A^) = ||A - A^||_F^2 / (number of entries) (App. B.4, Frobenius-norm perspective), next to the
norms of K and V themselves (Sec. 3: key norms exceed value norms).  This module restates, in fp64, the
four sums that all of these follow from, for token-wise groups:

    sum k^2,  sum (k - k^)^2,  sum v^2,  sum (v - v^)^2        per (batch, kv-head)

where k^ = fmaf(code, scale, zero) is the fp32 reconstruction of the group quantizer in quantizer.py.

`bit_balance` is the bit allocation that equalises the two error bounds of App. B.4,
||E_V||_F <~ sqrt(L d) / 2^b_V ||V||_F and likewise for K:  2^(b_K - b_V) ~ ||K||_F / ||V||_F.
(The paper prints the ratio inverted, ||V|| / ||K||, which contradicts its own conclusion b_K > b_V;
the algebra of its preceding line gives the form used here.)
"""
from __future__ import annotations

import math

import numpy as np

from . import quantizer


def side_sums(x_bits: np.ndarray, dtype: str, bits: int, g: int):
    """x_bits: uint16 (B, H, T, D).  Returns (sum x^2, sum (x - xhat)^2), each fp64 (B, H)."""
    x = quantizer.bits_to_f32(x_bits, dtype).astype(np.float64)
    if bits == 16:
        return (x * x).sum(axis=(2, 3)), np.zeros(x.shape[:2])
    codes, s16, z16 = quantizer.quantize_per_token(x_bits, dtype, bits, g)
    D = x_bits.shape[-1]
    xhat = quantizer.dequantize_groups(codes.reshape(x_bits.shape[:-1] + (D // g, g)), s16, z16)
    e = x - xhat.reshape(x.shape).astype(np.float64)
    return (x * x).sum(axis=(2, 3)), (e * e).sum(axis=(2, 3))


def quant_error_sums(k_bits, v_bits, dtype: str, kb: int, vb: int, gk: int, gv: int) -> np.ndarray:
    """fp64 (B, H, 4) = (sum k^2, sum (k - k^)^2, sum v^2, sum (v - v^)^2)."""
    k2, ke = side_sums(k_bits, dtype, kb, gk)
    v2, ve = side_sums(v_bits, dtype, vb, gv)
    return np.stack([k2, ke, v2, ve], axis=-1)


def bit_balance(sum_k2: float, sum_v2: float) -> float:
    """b_K - b_V that balances the Frobenius error bounds: log2(||K||_F / ||V||_F)."""
    return 0.5 * math.log2(sum_k2 / sum_v2)
