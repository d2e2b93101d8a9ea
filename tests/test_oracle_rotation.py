"""Pins for the oracle's key rotation (randomized Hadamard transform before quantization, Sec. 4.4)."""
import numpy as np
import pytest
import scipy.linalg
import torch

from oracle import quantizer as oq
from oracle.cache import OracleCache
from paper_2502_15075_b200 import workloads as wl

RNG = np.random.default_rng(7)


def bits_of(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("D", [64, 128])
def test_fwht_is_the_sylvester_hadamard_matrix(D):
    x = RNG.standard_normal((9, D)).astype(np.float32)
    H = scipy.linalg.hadamard(D).astype(np.float64)
    assert np.allclose(oq.fwht_f32(x), x.astype(np.float64) @ H, rtol=0, atol=2e-5)
    e = np.zeros((1, D), np.float32)
    e[0, 5] = 1.0
    assert np.array_equal(oq.fwht_f32(e)[0], H[5].astype(np.float32))          # a unit vector picks a row exactly
    assert np.array_equal(oq.fwht_f32(np.ones((1, D), np.float32))[0], np.r_[D, np.zeros(D - 1)].astype(np.float32))


@pytest.mark.parametrize("D", [64, 128])
def test_rotation_is_orthogonal_and_its_own_inverse(D):
    x = RNG.standard_normal((50, D)).astype(np.float32) * 3
    s = RNG.choice([-1, 1], D).astype(np.int8)
    y = oq.rotate_f32(x, s)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-5)
    assert np.allclose(oq.unrotate_f32(y, s), x, atol=5e-6 * np.abs(x).max() * np.sqrt(D))
    # inner products are preserved: (H k) . (H q) = k . q
    q = RNG.standard_normal((50, D))
    k64 = oq.hadamard_rotate_f64(x, s)
    q64 = oq.hadamard_rotate_f64(q, s)
    assert np.allclose((k64 * q64).sum(-1), (x.astype(np.float64) * q).sum(-1), rtol=1e-10, atol=1e-10)
    assert np.allclose(oq.hadamard_rotate_f64(x, s), y, atol=1e-5)


def test_rotation_spreads_outlier_channels_and_lowers_key_error():
    """Sec. 4.4: rotating the keys disperses outliers; with 8 heavy channels the 4-bit reconstruction error drops."""
    w = wl.LLAMA_8B.with_(n_kv_heads=1, n_q_heads=4)
    k, _ = wl.make_kv(w, tokens=512, batch=1)
    x = k[0, 0].float().numpy()
    s = RNG.choice([-1, 1], 128).astype(np.int8)
    plain = oq.dequantize_groups_f64(*oq.quantize_groups(x, 4))
    y = oq.rotate_f32(x, s)
    rot = oq.unrotate_f32(oq.dequantize_groups(*oq.quantize_groups(y, 4)), s)
    assert np.abs(y).max() < 0.6 * np.abs(x).max()
    assert oq.mse(x, rot) < 0.5 * oq.mse(x, plain)


@pytest.mark.parametrize("k_axis", [0, 1])
def test_rotated_cache_roundtrip_and_attention(k_axis):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8, kb=8, vb=8, k_axis=k_axis)
    T = 300
    k, v = wl.make_kv(w, tokens=T, batch=1)
    q = wl.make_q(w, batch=1)
    s = RNG.choice([-1, 1], 128).astype(np.int8)

    def build(chunks):
        c = OracleCache(1, 2, 128, 8, 8, 128, 128, k_axis, "bf16", 384, k_signs=s)
        t = 0
        for n in chunks:
            c.append(bits_of(k)[:, :, t:t + n], bits_of(v)[:, :, t:t + n])
            t += n
        return c
    a, b = build([T]), build([1] * 130 + [170])
    assert np.array_equal(a.pages, b.pages)
    r = T % 128
    if k_axis:
        assert np.array_equal(a.k_tail[:, :, :r], b.k_tail[:, :, :r])
    # attention with rotated keys and rotated queries is close to exact attention on the unquantized inputs
    logits = torch.einsum("bhd,bhtd->bht", q.double(), k.double().repeat_interleave(4, 1)) / np.sqrt(128)
    exact = torch.einsum("bht,bhtd->bhd", torch.softmax(logits, -1), v.double().repeat_interleave(4, 1)).numpy()
    assert np.abs(a.decode(bits_of(q)) - exact).max() < 0.03
    # dequantize returns keys in the original space
    ko = np.zeros((1, 2, 384, 128), np.uint16)
    vo = np.zeros_like(ko)
    a.dequantize(ko, vo, 0, 384)
    got = oq.bits_to_f32(ko[:, :, :T], "bf16")
    assert np.abs(got - k.float().numpy()).max() < 0.25          # 8-bit codes of a rotated row + bf16 rounding
    assert not ko[:, :, T:].any()
