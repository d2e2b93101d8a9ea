"""Pins for the oracle quantizer: closed forms, invariants, brute force, library
conversions and the paper's printed error ratios.  CPU only."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import quantizer as oq

F32 = np.float32
RNG = np.random.default_rng(1234)


def fp16_values(x):
    """Round a float array to fp16 and return it as exact fp32 values."""
    return np.asarray(x, np.float32).astype(np.float16).astype(np.float32)


# ------------------------------------------------------------ conversions
def test_bf16_bits_match_torch():
    x = torch.randn(20000, dtype=torch.float32) * 37.0
    want = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = oq.f32_to_bf16_bits(x.numpy())
    assert np.array_equal(got, want)
    back = oq.bits_to_f32(got, "bf16")
    assert np.array_equal(back, x.to(torch.bfloat16).float().numpy())


def test_fp16_bits_match_torch_and_saturate():
    x = torch.randn(20000, dtype=torch.float32) * 300.0
    want = x.to(torch.float16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oq.f32_to_fp16_bits(x.numpy()), want)
    big = np.array([70000.0, -1e9, 65504.0, 65519.9, 65520.0], np.float32)
    got = oq.bits_to_f32(oq.f32_to_fp16_bits(big), "fp16")
    assert np.array_equal(got, np.array([65504.0, -65504.0, 65504.0, 65504.0, 65504.0], np.float32))


def test_bf16_ties_to_even():
    # 1 + 2^-8 is exactly between bf16 neighbours 1 and 1 + 2^-7 -> even (1.0)
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], np.float32)
    got = oq.bits_to_f32(oq.f32_to_bf16_bits(x), "bf16")
    assert np.array_equal(got, np.array([1.0, 1.0 + 2.0 ** -6], np.float32))


# ------------------------------------------------------------ closed forms
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_integer_ladder_is_exact(bits):
    """A group that holds exactly 0..qmax has scale 1, zero 0, codes = values."""
    qmax = 2 ** bits - 1
    g = 256
    vals = np.concatenate([np.arange(qmax + 1), RNG.integers(0, qmax + 1, g - qmax - 1)])
    RNG.shuffle(vals)
    x = vals.astype(np.float32)[None]
    codes, s16, z16 = oq.quantize_groups(x, bits)
    assert oq.bits_to_f32(s16, "fp16")[0] == 1.0 and oq.bits_to_f32(z16, "fp16")[0] == 0.0
    assert np.array_equal(codes[0], vals)
    assert np.array_equal(oq.dequantize_groups(codes, s16, z16)[0], x[0])


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("k,off", [(-3, 0.0), (2, -64.0), (-6, 0.5), (0, -7.0)])
def test_shifted_scaled_ladder(bits, k, off):
    """Power-of-two scaling and an fp16-exact offset keep the ladder exact."""
    qmax = 2 ** bits - 1
    vals = np.concatenate([np.arange(qmax + 1), RNG.integers(0, qmax + 1, 37)])
    x = (vals * 2.0 ** k + off).astype(np.float32)[None]
    assert np.array_equal(fp16_values(x), x)          # representable inputs
    codes, s16, z16 = oq.quantize_groups(x, bits)
    assert oq.bits_to_f32(s16, "fp16")[0] == 2.0 ** k
    assert oq.bits_to_f32(z16, "fp16")[0] == off
    assert np.array_equal(codes[0], vals)
    assert np.array_equal(oq.dequantize_groups(codes, s16, z16)[0], x[0])


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_constant_group(bits):
    for c in (0.0, -0.0, 3.25, -1e-3, 65504.0):
        x = np.full((1, 32), c, np.float32)
        x = fp16_values(x)
        codes, s16, z16 = oq.quantize_groups(x, bits)
        assert s16[0] == 0, "scale of a constant group is +0"
        assert np.all(codes == 0)
        xh = oq.dequantize_groups(codes, s16, z16)
        assert np.array_equal(xh, x + F32(0.0))
    # -0 is canonicalised: zero-point +0, never 0x8000
    x = np.array([[-0.0, 0.0, -0.0, 0.0]], np.float32)
    _, s16, z16 = oq.quantize_groups(x, bits)
    assert s16[0] == 0 and z16[0] == 0


def test_scale_formula_and_metadata_rounding():
    """scale = fp16((mx - mn)/qmax) with fp32 ops; zero = fp16(mn)."""
    x = np.array([[0.1, 0.7, -0.3, 0.25]], np.float32)
    x = fp16_values(x)
    for bits in (2, 4, 8):
        _, s16, z16 = oq.quantize_groups(x, bits)
        mn, mx = Fraction(float(x.min())), Fraction(float(x.max()))
        exact = (mx - mn) / (2 ** bits - 1)
        s = Fraction(float(oq.bits_to_f32(s16, "fp16")[0]))
        # within one fp32 rounding + one fp16 rounding of the exact quotient
        assert abs(s - exact) <= exact * Fraction(1, 2 ** 11) + exact * Fraction(1, 2 ** 23)
        assert Fraction(float(oq.bits_to_f32(z16, "fp16")[0])) == mn


# ------------------------------------------------------------ brute force
@pytest.mark.parametrize("g", [2, 3, 4])
def test_bruteforce_codes_are_nearest(g):
    """b = 2: among all 4^g code vectors the chosen one minimises the squared
    reconstruction error for the chosen (scale, zero), up to exact ties."""
    for trial in range(40):
        x = fp16_values(RNG.standard_normal((1, g)) * (1 + trial % 5))
        codes, s16, z16 = oq.quantize_groups(x, 2)
        s = float(oq.bits_to_f32(s16, "fp16")[0])
        z = float(oq.bits_to_f32(z16, "fp16")[0])
        xs = x[0].astype(np.float64)
        best = min(sum((xs[i] - (z + s * c[i])) ** 2 for i in range(g))
                   for c in itertools.product(range(4), repeat=g))
        mine = float(np.sum((xs - (z + s * codes[0].astype(np.float64))) ** 2))
        assert mine <= best * (1 + 1e-6) + 1e-12


# ------------------------------------------------------------ invariants
@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("g", [32, 64, 128])
def test_error_at_most_half_step(bits, g):
    """|x - xhat| <= scale/2 (entrywise bound in the proof of Thm B.1), for
    fp16-representable inputs (zero-point exact) and a normal fp16 scale."""
    x = fp16_values(RNG.standard_normal((500, g)) * RNG.lognormal(0, 1.5, (500, 1)))
    codes, s16, z16 = oq.quantize_groups(x, bits)
    s = oq.bits_to_f32(s16, "fp16").astype(np.float64)
    ok = (s16 & 0x7C00) != 0                      # normal scale
    assert ok.sum() > 400
    xh = oq.dequantize_groups_f64(codes, s16, z16)
    err = np.abs(x.astype(np.float64) - xh)
    assert np.all(err[ok] <= 0.5 * s[ok, None] * (1 + 1e-3))
    assert codes.max() == 2 ** bits - 1 and codes.min() == 0
    # each group's extreme values take the extreme codes
    assert np.all(np.take_along_axis(codes, x.argmin(-1)[:, None], -1) == 0)
    assert np.all(np.take_along_axis(codes[ok], x[ok].argmax(-1)[:, None], -1) == 2 ** bits - 1)


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_idempotent_on_reconstruction(bits):
    """Quantizing the reconstruction with the same (scale, zero) returns the same codes."""
    x = fp16_values(RNG.standard_normal((200, 64)))
    codes, s16, z16 = oq.quantize_groups(x, bits)
    s = oq.bits_to_f32(s16, "fp16")
    z = oq.bits_to_f32(z16, "fp16")
    xh = oq.dequantize_groups(codes, s16, z16)
    u = (xh - z[:, None]) * (F32(1.0) / s)[:, None]
    again = np.clip(np.rint(u), 0, 2 ** bits - 1).astype(np.uint8)
    assert np.array_equal(again, codes)


def test_round_half_to_even():
    # zero 0, scale 1 (values 0 and 15 present): 0.5 -> 0, 1.5 -> 2, 2.5 -> 2, 3.5 -> 4
    x = np.array([[0.0, 15.0, 0.5, 1.5, 2.5, 3.5, 6.5]], np.float32)
    codes, _, _ = oq.quantize_groups(x, 4)
    assert codes[0].tolist() == [0, 15, 0, 2, 2, 4, 6]


def test_dequantize_is_single_rounding_fma():
    """fmaf(c, s, z): compare with exact rational arithmetic rounded once to fp32."""
    c = RNG.integers(0, 256, 3000)
    s16 = RNG.integers(1, 0x7BFF, 3000).astype(np.uint16)
    z16 = RNG.integers(0, 0xFBFF, 3000).astype(np.uint16)
    z16 = z16[(z16 & 0x7C00) != 0x7C00][:2000]
    c, s16 = c[: len(z16)], s16[: len(z16)]
    got = oq.dequantize_groups(c[:, None].astype(np.uint8), s16, z16)[:, 0]
    s = oq.bits_to_f32(s16, "fp16")
    z = oq.bits_to_f32(z16, "fp16")
    for i in range(len(z16)):
        exact = Fraction(int(c[i])) * Fraction(float(s[i])) + Fraction(float(z[i]))
        r = Fraction(float(got[i]))
        lo = Fraction(float(np.nextafter(got[i], F32(-np.inf))))
        hi = Fraction(float(np.nextafter(got[i], F32(np.inf))))
        assert abs(exact - r) <= min(abs(exact - lo), abs(exact - hi))


def test_per_token_and_per_channel_wrappers():
    x = fp16_values(RNG.standard_normal((128, 64)))
    xb = x.astype(np.float16).view(np.uint16)
    codes, s16, z16 = oq.quantize_per_token(xb, "fp16", 4, 32)
    assert codes.shape == (128, 64) and s16.shape == (128, 2)
    for t in (0, 77):
        for j in (0, 1):
            c2, s2, z2 = oq.quantize_groups(x[t, 32 * j: 32 * j + 32][None], 4)
            assert np.array_equal(c2[0], codes[t, 32 * j: 32 * j + 32]) and s2[0] == s16[t, j] and z2[0] == z16[t, j]
    cc, sc, zc = oq.quantize_per_channel_block(xb, 4)
    assert cc.shape == (128, 64) and sc.shape == (64,)
    for d in (0, 13, 63):
        c2, s2, z2 = oq.quantize_groups(x[:, d][None], 4)
        assert np.array_equal(c2[0], cc[:, d]) and s2[0] == sc[d] and z2[0] == zc[d]
    # bf16 inputs: the tail keeps fp16(x); exact for bf16 values in the fp16 normal range
    xbf = oq.f32_to_bf16_bits(x)
    tail = oq.to_tail_fp16_bits(xbf, "bf16")
    assert np.array_equal(oq.bits_to_f32(tail, "fp16"), oq.bits_to_f32(xbf, "bf16"))


# ------------------------------------------------------------ MSE behaviour
def test_uniform_data_mse_is_step_squared_over_12():
    x = RNG.uniform(-1, 1, (4000, 128)).astype(np.float32)
    for bits in (2, 4, 8):
        codes, s16, z16 = oq.quantize_groups(x, bits)
        s = oq.bits_to_f32(s16, "fp16").astype(np.float64)
        xh = oq.dequantize_groups_f64(codes, s16, z16)
        ratio = np.mean((x - xh) ** 2) / np.mean(s ** 2 / 12.0)
        assert 0.93 < ratio < 1.07, (bits, ratio)


def _golden_rows():
    path = os.path.join(os.path.dirname(__file__), "golden", "table1_mse_c4.txt")
    rows = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows[f[0]] = [float(v) for v in f[1:]]
    return rows


def test_error_scaling_matches_paper_table1_ratios():
    """Error falls by ((2^b' - 1)/(2^b - 1))^2 between bit-widths; the paper's
    Table 1 key columns show the same ratios (K3/K4 ~ 4.6, K2/K4 ~ 21-25)."""
    x = RNG.standard_normal((3000, 128)).astype(np.float32)
    m = {}
    for bits in (2, 4, 8):
        codes, s16, z16 = oq.quantize_groups(x, bits)
        m[bits] = oq.mse(x, oq.dequantize_groups_f64(codes, s16, z16))
    assert m[2] > m[4] > m[8]
    assert abs(m[2] / m[4] / 25.0 - 1) < 0.08
    assert abs(m[4] / m[8] / 289.0 - 1) < 0.08
    ms = {b: oq.mse(x, oq.quantize_symmetric(x, b)[2]) for b in (2, 3, 4, 5, 6)}
    assert all(ms[b] > ms[b + 1] for b in (2, 3, 4, 5))
    assert abs(ms[3] / ms[4] / (7.0 / 3.0) ** 2 - 1) < 0.1     # symmetric: (2^(b-1)-1) steps
    for name, (k2, v2, k3, v3, k4, v4) in _golden_rows().items():
        assert 4.2 < k3 / k4 < 4.9, name                       # (15/7)^2 = 4.59
        assert 19.0 < k2 / k4 < 27.0, name                     # (15/3)^2 = 25
        assert k2 > v2 and k3 > v3 and k4 > v4, name           # keys dominate the error


def test_key_error_exceeds_value_error_when_key_norm_larger():
    """Sec. 3: with equal bits, the cache with the larger norm has the larger error."""
    k = (RNG.standard_normal((2000, 128)) * 3.0).astype(np.float32)
    v = RNG.standard_normal((2000, 128)).astype(np.float32)
    for bits in (2, 4):
        ek = oq.mse(k, oq.dequantize_groups_f64(*oq.quantize_groups(k, bits)))
        ev = oq.mse(v, oq.dequantize_groups_f64(*oq.quantize_groups(v, bits)))
        assert 7.0 < ek / ev < 11.0       # error scales with the squared norm (x9)


# ------------------------------------------------------------ App. B symmetric quantizer
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_symmetric_quantizer_bounds(bits):
    """Entrywise |A - Ahat| <= alpha/2 and Thm B.2: ||A - Ahat||_F <= sqrt(mn) M / (2 (2^(b-1) - 1))."""
    A = RNG.standard_normal((37, 53)) * 2.5
    Q, alpha, Ah = oq.quantize_symmetric(A, bits)
    M = np.abs(A).max()
    top = 2 ** (bits - 1) - 1
    assert alpha == M / top
    assert Q.min() >= -(2 ** (bits - 1)) and Q.max() <= top
    assert np.all(np.abs(A - Ah) <= alpha / 2 * (1 + 1e-12))
    bound = np.sqrt(A.size) * M / (2 * top)
    assert np.linalg.norm(A - Ah) <= bound
    assert bound <= np.sqrt(A.size) * np.linalg.norm(A) / (2 * top)
    # the entry of largest magnitude is reproduced exactly
    i = np.unravel_index(np.abs(A).argmax(), A.shape)
    assert abs(Ah[i] - A[i]) < 1e-12


@pytest.mark.parametrize("bits", [1, 3, 6])
def test_odd_widths_follow_the_same_formula(bits):
    """1, 3 and 6 bits (Table 1's 3-bit column, Sec. 4.1's 1- and 6-bit settings): an integer ladder 0..qmax is
    reproduced exactly, the error stays within half a step, and brute force over all code vectors of a tiny group
    finds nothing better."""
    qmax = 2 ** bits - 1
    ladder = np.arange(qmax + 1, dtype=np.float32)[None]
    c, s16, z16 = oq.quantize_groups(ladder, bits)
    assert np.array_equal(c[0], np.arange(qmax + 1)) and oq.bits_to_f32(s16, "fp16")[0] == 1.0
    rng = np.random.default_rng(bits)
    x = rng.normal(size=(50, 32)).astype(np.float16).astype(np.float32)
    c, s16, z16 = oq.quantize_groups(x, bits)
    s = oq.bits_to_f32(s16, "fp16").astype(np.float64)
    xh = oq.dequantize_groups_f64(c, s16, z16)
    z_exact = oq.bits_to_f32(z16, "fp16") == x.min(axis=1)
    assert c.max() <= qmax and np.all(np.abs(x - xh)[z_exact] <= (0.5 * s[:, None] * (1 + 1e-3) * np.ones_like(xh))[z_exact])
    if bits <= 3:
        import itertools
        g = x[0, :3][None]
        c3, s3, z3 = oq.quantize_groups(g, bits)
        sc = float(oq.bits_to_f32(s3, "fp16")[0]); z = float(oq.bits_to_f32(z3, "fp16")[0])
        best = min(sum((g[0, i] - (z + sc * cv[i])) ** 2 for i in range(3)) for cv in itertools.product(range(qmax + 1), repeat=3))
        mine = sum((g[0, i] - (z + sc * int(c3[0, i]))) ** 2 for i in range(3))
        assert mine <= best * (1 + 1e-9) + 1e-18
