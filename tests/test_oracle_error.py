"""Pins for the oracle's quantization-error sums (Sec. 4.1 experiment (i); MSE of App. B.4).  CPU only."""
import numpy as np
import torch

from oracle import error as oe
from oracle import quantizer as oq

RNG = np.random.default_rng(7)


def bf16_bits(x):
    return torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def fp16_bits(x):
    return np.asarray(x, np.float32).astype(np.float16).view(np.uint16)


def test_sums_against_an_explicit_loop_on_a_tiny_case():
    """Brute force: every element reconstructed one by one from its group's code, scale and zero."""
    x = fp16_bits(RNG.normal(size=(1, 2, 3, 64)))
    s = oe.side_sums(x, "fp16", 4, 32)
    xf = oq.bits_to_f32(x, "fp16").astype(np.float64)
    for h in range(2):
        tot2, tote = 0.0, 0.0
        for t in range(3):
            for gi in range(2):
                grp = xf[0, h, t, 32 * gi: 32 * gi + 32]
                c, s16, z16 = oq.quantize_groups(grp.astype(np.float32)[None], 4)
                sc = float(oq.bits_to_f32(s16, "fp16")[0]); z = float(oq.bits_to_f32(z16, "fp16")[0])
                for i in range(32):
                    xh = float(np.float32(float(c[0, i]) * sc + z))
                    tot2 += grp[i] ** 2
                    tote += (grp[i] - xh) ** 2
        assert abs(s[0][0, h] - tot2) <= 1e-12 * tot2
        assert abs(s[1][0, h] - tote) <= 1e-12 * tote


def test_error_sum_is_the_mse_times_the_number_of_entries():
    """App. B.4: MSE(A, A^) = ||A - A^||_F^2 / nnz; checked through the dequantizer and the library-style mean."""
    x = bf16_bits(RNG.normal(size=(2, 2, 40, 128)) * 3.0)
    x2, e2 = oe.side_sums(x, "bf16", 2, 128)
    codes, s16, z16 = oq.quantize_per_token(x, "bf16", 2, 128)
    xhat = oq.dequantize_groups(codes.reshape(2, 2, 40, 1, 128), s16, z16).reshape(2, 2, 40, 128)
    xf = oq.bits_to_f32(x, "bf16")
    for b in range(2):
        for h in range(2):
            assert np.isclose(e2[b, h] / (40 * 128), oq.mse(xf[b, h], xhat[b, h]), rtol=1e-12)
            assert np.isclose(x2[b, h], np.linalg.norm(xf[b, h].astype(np.float64)) ** 2, rtol=1e-12)


def test_uniform_data_has_mse_step_squared_over_twelve():
    """A uniform scalar quantizer on data uniform over its range has error variance step^2 / 12."""
    n = 4096
    x = RNG.uniform(-1.0, 1.0, size=(1, 1, n, 128)).astype(np.float32)
    x[..., 0] = -1.0
    x[..., 1] = 1.0                                   # every group spans exactly [-1, 1]
    xb = fp16_bits(x)
    for bits in (4, 8):
        step = 2.0 / (2 ** bits - 1)
        _, e2 = oe.side_sums(xb, "fp16", bits, 128)
        mse = e2[0, 0] / (n * 128)
        assert abs(mse / (step ** 2 / 12.0) - 1.0) < 0.03


def test_scaling_the_input_by_three_scales_both_sums_by_nine():
    """The quantizer is scale-equivariant (up to fp16 rounding of its metadata): error grows with the norm,
    which is the reason the paper gives keys more bits."""
    x = RNG.normal(size=(1, 2, 64, 128)).astype(np.float32)
    a = oe.side_sums(fp16_bits(x), "fp16", 4, 128)
    b = oe.side_sums(fp16_bits(4.0 * x), "fp16", 4, 128)       # a power of two: exactly equivariant
    assert np.allclose(b[0], 16.0 * a[0], rtol=1e-12) and np.allclose(b[1], 16.0 * a[1], rtol=1e-12)
    c = oe.side_sums(fp16_bits(3.0 * x), "fp16", 4, 128)
    assert np.allclose(c[0], 9.0 * a[0], rtol=2e-3) and np.allclose(c[1], 9.0 * a[1], rtol=5e-2)


def test_more_bits_less_error_and_keys_worse_than_values_at_equal_bits():
    """Table 1's qualitative content: error falls monotonically with the bit width (by about 4x per bit) and,
    at equal bits, the cache with the larger norm (keys) has the larger error."""
    k = bf16_bits(RNG.normal(size=(1, 2, 128, 128)) * 4.0)
    v = bf16_bits(RNG.normal(size=(1, 2, 128, 128)))
    e = {b: oe.quant_error_sums(k, v, "bf16", b, b, 128, 128).sum(axis=(0, 1)) for b in (2, 4, 8)}
    assert e[2][1] > e[4][1] > e[8][1] and e[2][3] > e[4][3] > e[8][3]
    assert 10 < e[2][1] / e[4][1] < 40                  # ((2^4-1)/(2^2-1))^2 = 25
    for b in (2, 4, 8):
        assert e[b][1] > 4 * e[b][3]
    # the allocation that balances the bounds gives the keys log2(4) = 2 more bits
    assert abs(oe.bit_balance(e[4][0], e[4][2]) - 2.0) < 0.05
    assert oe.bit_balance(1.0, 1.0) == 0.0 and oe.bit_balance(4.0, 1.0) == 1.0


def test_sixteen_bit_passthrough_has_no_error():
    x = bf16_bits(RNG.normal(size=(1, 1, 8, 64)))
    x2, e2 = oe.side_sums(x, "bf16", 16, 64)
    assert e2.sum() == 0.0 and x2.sum() > 0.0
