"""Oracle quantizer (test infrastructure; never imported by the product path).

Two quantizers live here:

* `quantize_groups` - the hot path's group-wise asymmetric round-to-nearest
  quantizer: the uniform scalar quantizer of App. B.1 (scale = range / number
  of steps, Q = round(A / scale), reconstruction = scale * Q) applied to each
  group after subtracting the group minimum, with the scale and the minimum
  stored as fp16.  Sec. 4.1 fixes the grouping (128-element groups, token-wise
  or channel-wise); the tie rule, the fp16 metadata and the order of the fp32
  operations are this build's fixed reading:

      mn, mx   = min, max of the group (each + 0.0f so that -0 becomes +0)
      scale32  = (mx - mn) / qmax            one fp32 subtraction, one fp32 division
      s16, z16 = fp16(scale32), fp16(mn)     round-to-nearest-even, saturating at +-65504
      s, z     = fp32(s16), fp32(z16)
      code     = 0                           if s == 0
               = clamp(rint((x - z) * (1.0f / s)), 0, qmax)   otherwise
      xhat     = fmaf(code, s, z)            one rounding to fp32, then RN to 16 bit

  Every operation is an individually rounded IEEE fp32 operation (NumPy
  float32 arithmetic), `rint` rounds half to even.

* `quantize_symmetric` - App. B.1 literally (per matrix, two's complement
  range, alpha = M / (2^(b-1) - 1)), in fp64; used only to check the error
  bounds of Theorems B.1/B.2.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
FP16_MAX = F32(65504.0)


# ----------------------------------------------------------------------------
# 16-bit <-> fp32 conversions on raw bit patterns
# ----------------------------------------------------------------------------
def bits_to_f32(bits: np.ndarray, dtype: str) -> np.ndarray:
    """Exact fp32 value of fp16 / bf16 bit patterns (uint16 array)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "fp16":
        return bits.view(np.float16).astype(np.float32)
    if dtype == "bf16":
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError(dtype)


def f32_to_fp16_bits(x: np.ndarray, saturate: bool = True) -> np.ndarray:
    """fp32 -> fp16 bit patterns, round-to-nearest-even; saturating to +-65504."""
    x = np.asarray(x, dtype=np.float32)
    if saturate:
        x = np.minimum(np.maximum(x, -FP16_MAX), FP16_MAX)
    with np.errstate(over="ignore"):
        return np.ascontiguousarray(x.astype(np.float16)).view(np.uint16)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def f32_to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "fp16":
        return f32_to_fp16_bits(x, saturate=False)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------
# Asymmetric group-wise quantizer (the hot path's definition)
# ----------------------------------------------------------------------------
def quantize_groups(x32: np.ndarray, bits: int):
    """Quantize along the last axis: every row of `x32` (..., g) is one group.

    Returns (codes uint8 (..., g), s16 uint16 (...), z16 uint16 (...)):
    the b-bit codes and the fp16 bit patterns of scale and zero-point.
    """
    assert bits in (1, 2, 3, 4, 6, 8)
    x = np.asarray(x32, dtype=np.float32)
    assert np.all(np.isfinite(x)), "precondition: finite inputs"
    qmax = F32(2 ** bits - 1)
    mn = x.min(axis=-1) + F32(0.0)
    mx = x.max(axis=-1) + F32(0.0)
    scale32 = (mx - mn) / qmax
    s16 = f32_to_fp16_bits(scale32)
    z16 = f32_to_fp16_bits(mn)
    s = bits_to_f32(s16, "fp16")
    z = bits_to_f32(z16, "fp16")
    nz = s != F32(0.0)
    inv = np.zeros_like(s)
    inv[nz] = F32(1.0) / s[nz]
    u = (x - z[..., None]) * inv[..., None]
    r = np.rint(u)
    r = np.minimum(np.maximum(r, F32(0.0)), qmax)
    codes = np.where(nz[..., None], r, F32(0.0)).astype(np.uint8)
    return codes, s16, z16


def dequantize_groups(codes: np.ndarray, s16: np.ndarray, z16: np.ndarray) -> np.ndarray:
    """xhat = fmaf(code, s, z) as fp32 (one rounding).  `codes` (..., g), metadata (...).

    code * s + z is exact in fp64 (8 + 11 significand bits, exponents within the
    fp16 range), so rounding the fp64 result to fp32 equals a fused multiply-add.
    """
    s = bits_to_f32(s16, "fp16").astype(np.float64)
    z = bits_to_f32(z16, "fp16").astype(np.float64)
    return (codes.astype(np.float64) * s[..., None] + z[..., None]).astype(np.float32)


def dequantize_groups_f64(codes, s16, z16) -> np.ndarray:
    """Exact reconstruction z + s * code in fp64 (what attention runs on)."""
    s = bits_to_f32(s16, "fp16").astype(np.float64)
    z = bits_to_f32(z16, "fp16").astype(np.float64)
    return z[..., None] + s[..., None] * codes.astype(np.float64)


def quantize_per_token(x_bits: np.ndarray, dtype: str, bits: int, g: int):
    """Token-wise (per-row) quantization with groups of g consecutive channels.

    x_bits: uint16 (..., D).  Returns codes (..., D), s16 (..., D/g), z16 (..., D/g).
    """
    D = x_bits.shape[-1]
    assert D % g == 0
    x = bits_to_f32(x_bits, dtype).reshape(x_bits.shape[:-1] + (D // g, g))
    codes, s16, z16 = quantize_groups(x, bits)
    return codes.reshape(x_bits.shape), s16, z16


def to_tail_fp16_bits(x_bits: np.ndarray, dtype: str) -> np.ndarray:
    """What the fp16 residual tail stores for an input element: fp16(x), saturating."""
    return f32_to_fp16_bits(bits_to_f32(x_bits, dtype), saturate=True)


def quantize_per_channel_block(tail_bits: np.ndarray, bits: int):
    """Channel-wise (per-column) quantization of one block of tokens.

    tail_bits: uint16 fp16 patterns (n_tokens, D) - the block as held in the fp16
    tail.  One group per channel, running down the tokens.
    Returns codes (n_tokens, D), s16 (D,), z16 (D,).
    """
    x = bits_to_f32(tail_bits, "fp16")
    codes_t, s16, z16 = quantize_groups(np.ascontiguousarray(x.T), bits)
    return np.ascontiguousarray(codes_t.T), s16, z16


# ----------------------------------------------------------------------------
# App. B.1 symmetric per-matrix quantizer (only for checking Thm B.1 / B.2)
# ----------------------------------------------------------------------------
def quantize_symmetric(A: np.ndarray, bits: int):
    """alpha = M / (2^(b-1) - 1), Q = round(A / alpha) in two's-complement range,
    Ahat = alpha * Q  (App. B.1).  Returns (Q int64, alpha float64, Ahat float64)."""
    A = np.asarray(A, dtype=np.float64)
    assert bits >= 2
    M = np.max(np.abs(A))
    top = 2 ** (bits - 1) - 1
    if M == 0.0:
        return np.zeros(A.shape, np.int64), 0.0, np.zeros_like(A)
    alpha = M / top
    Q = np.rint(A / alpha)
    Q = np.clip(Q, -(2 ** (bits - 1)), top).astype(np.int64)
    return Q, alpha, alpha * Q


def mse(A: np.ndarray, Ahat: np.ndarray) -> float:
    """MSE = ||A - Ahat||_F^2 / number of entries (App. B.4, Frobenius-norm perspective)."""
    d = np.asarray(A, np.float64) - np.asarray(Ahat, np.float64)
    return float(np.sum(d * d) / d.size)


# ----------------------------------------------------------------------------
# Randomized Hadamard rotation of keys (Sec. 4.4: rotate the keys before quantization)
# ----------------------------------------------------------------------------
def fwht_f32(x: np.ndarray) -> np.ndarray:
    """Unnormalised fast Walsh-Hadamard transform along the last axis in fp32, butterfly stages
    h = 1, 2, 4, ... in this order, (a, b) -> (a + b, a - b) with a the element whose index has bit h clear.
    Every addition is an individually rounded fp32 operation, so the result is reproducible bit for bit."""
    y = np.array(x, dtype=np.float32, copy=True)
    n = y.shape[-1]
    assert n & (n - 1) == 0
    h = 1
    while h < n:
        v = y.reshape(y.shape[:-1] + (n // (2 * h), 2, h))
        a = v[..., 0, :].copy()
        b = v[..., 1, :].copy()
        v[..., 0, :] = a + b
        v[..., 1, :] = a - b
        h *= 2
    return y


def rotate_f32(x32: np.ndarray, signs: np.ndarray) -> np.ndarray:
    """y = H (signs * x) / sqrt(D) in fp32: sign flip (exact), fwht_f32, one fp32 multiplication by
    float32(1/sqrt(D)).  `signs` is +-1 per channel.  The same map is its own inverse up to the signs:
    x = signs * H y / sqrt(D)."""
    D = x32.shape[-1]
    inv = np.float32(1.0 / np.sqrt(np.float64(D)))
    return fwht_f32(np.asarray(x32, np.float32) * signs.astype(np.float32)) * inv


def unrotate_f32(y32: np.ndarray, signs: np.ndarray) -> np.ndarray:
    D = y32.shape[-1]
    inv = np.float32(1.0 / np.sqrt(np.float64(D)))
    return (fwht_f32(np.asarray(y32, np.float32)) * inv) * signs.astype(np.float32)


def hadamard_rotate_f64(x: np.ndarray, signs: np.ndarray) -> np.ndarray:
    """The same rotation in exact-ish fp64 (used for queries in the fp64 attention)."""
    y = np.array(x, dtype=np.float64, copy=True) * signs.astype(np.float64)
    n = y.shape[-1]
    h = 1
    while h < n:
        v = y.reshape(y.shape[:-1] + (n // (2 * h), 2, h))
        a = v[..., 0, :].copy()
        b = v[..., 1, :].copy()
        v[..., 0, :] = a + b
        v[..., 1, :] = a - b
        h *= 2
    return y / np.sqrt(np.float64(n))
