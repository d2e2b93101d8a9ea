"""Pins for the oracle's packed layout, fp64 attention and cache logic.  CPU only."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as oa
from oracle import layout as ol
from oracle import quantizer as oq
from oracle.cache import OracleCache
from paper_2502_15075_b200 import workloads as wl

RNG = np.random.default_rng(99)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


# ------------------------------------------------------------------ layout
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("fn", [ol.k_code_pos, ol.v_code_pos])
def test_code_positions_tile_the_region_exactly(D, b, fn):
    """Every (token, channel) owns a distinct b-bit field and together they cover
    the region with no gap: the index function is a bijection."""
    tt, dd = np.meshgrid(np.arange(128), np.arange(D), indexing="ij")
    byte, shift = fn(tt, dd, D, b)
    bitpos = (byte.astype(np.int64) * 8 + shift).ravel()
    assert bitpos.min() == 0 and np.all(bitpos % b == 0)
    assert len(np.unique(bitpos)) == 128 * D
    assert bitpos.max() == 128 * D * b - b


@pytest.mark.parametrize("D,kb,vb,gk,gv,k_axis", [
    (64, 4, 2, 32, 32, 0), (64, 4, 2, 64, 64, 0), (128, 4, 2, 128, 128, 0), (128, 2, 4, 128, 128, 0),
    (128, 8, 4, 128, 128, 0), (128, 4, 2, 128, 128, 1), (128, 8, 2, 128, 128, 1), (128, 16, 16, 128, 128, 0),
    (64, 16, 4, 64, 32, 0)])
def test_pack_unpack_roundtrip_and_sizes(D, kb, vb, gk, gv, k_axis):
    L = ol.Layout(D, kb, vb, gk, gv, k_axis)
    kmeta = 0 if kb == 16 else (4 * D if k_axis else 128 * D // gk * 4)
    vmeta = 0 if vb == 16 else 128 * D // gv * 4
    assert L.page_bytes == 128 * D * kb // 8 + 128 * D * vb // 8 + kmeta + vmeta
    assert L.page_bytes % 16 == 0 and L.v_codes_off % 16 == 0 and L.v_meta_off % 16 == 0
    page = RNG.integers(0, 256, L.page_bytes).astype(np.uint8)      # garbage: put must overwrite
    kc = RNG.integers(0, 2 ** kb, (128, D)).astype(np.uint16)
    vc = RNG.integers(0, 2 ** vb, (128, D)).astype(np.uint16)
    # write in two uneven pieces to exercise partial puts
    for sl in (slice(0, 37), slice(37, 128)):
        ol.put_k_codes(page, L, np.arange(128)[sl], kc[sl])
        ol.put_v_codes(page, L, np.arange(128)[sl], vc[sl])
    assert np.array_equal(ol.get_k_codes(page, L), kc)
    assert np.array_equal(ol.get_v_codes(page, L), vc)
    if vb != 16:
        s = RNG.integers(0, 65536, (128, D // gv)).astype(np.uint16)
        z = RNG.integers(0, 65536, (128, D // gv)).astype(np.uint16)
        ol.put_v_meta_tokens(page, L, np.arange(128), s, z)
        s2, z2 = ol.get_v_meta(page, L)
        assert np.array_equal(s, s2) and np.array_equal(z, z2)
        assert np.array_equal(ol.get_v_codes(page, L), vc)          # meta does not clobber codes
    if kb != 16 and k_axis == 1:
        s = RNG.integers(0, 65536, D).astype(np.uint16)
        z = RNG.integers(0, 65536, D).astype(np.uint16)
        ol.put_k_meta_channels(page, L, s, z)
        s2, z2 = ol.get_k_meta(page, L)
        assert np.array_equal(s, s2) and np.array_equal(z, z2)
    assert np.array_equal(ol.get_k_codes(page, L), kc)


def test_single_field_encoding_is_little_endian_words():
    """Spot values of the index function worked out by hand from its definition."""
    # K, D=128, 4-bit (2 fields per byte): d=0 -> chunk 0, r 0, word 0, byte 0 low nibble
    assert ol.k_code_pos(0, 0, 128, 4) == (0, 0)
    # d=1..3 are the next bytes of the same word; d=4 starts chunk 1 (16 bytes further)
    assert ol.k_code_pos(0, 1, 128, 4) == (1, 0)
    assert ol.k_code_pos(0, 3, 128, 4) == (3, 0)
    assert ol.k_code_pos(0, 4, 128, 4) == (16, 0)
    assert ol.k_code_pos(0, 8, 128, 4) == (32, 0)
    # d=16: r=1 -> same word, high nibble of byte 0 ; d=32: r=2 -> word 1 -> byte 4
    assert ol.k_code_pos(0, 16, 128, 4) == (0, 4)
    assert ol.k_code_pos(0, 17, 128, 4) == (1, 4)
    assert ol.k_code_pos(0, 32, 128, 4) == (4, 0)
    # token stride = 64 bytes
    assert ol.k_code_pos(3, 0, 128, 4) == (192, 0)
    # 2-bit: four fields per byte: d=16,32,48 share byte 0 at shifts 2,4,6; d=64 -> word 1
    assert ol.k_code_pos(0, 16, 128, 2) == (0, 2)
    assert ol.k_code_pos(0, 48, 128, 2) == (0, 6)
    assert ol.k_code_pos(0, 64, 128, 2) == (4, 0)
    assert ol.k_code_pos(0, 4, 128, 2) == (8, 0)
    # V, D=128, 2-bit (4 codes per byte, blocks of 32 tokens = 1024 bytes).  A word holds tokens
    # (2t, 2t+8, 2t+1, 2t+9) of one channel: token 0 -> byte 0, token 8 -> byte 1, token 1 -> byte 2, token 9 -> byte 3
    assert ol.v_code_pos(0, 0, 128, 2) == (0, 0)
    assert ol.v_code_pos(8, 0, 128, 2) == (1, 0)
    assert ol.v_code_pos(1, 0, 128, 2) == (2, 0)
    assert ol.v_code_pos(9, 0, 128, 2) == (3, 0)
    # tokens 2, 3 -> t = 1 -> the next 16-byte lane chunk; tokens 16..31 -> the word one further (kh = 1)
    assert ol.v_code_pos(2, 0, 128, 2) == (16, 0)
    assert ol.v_code_pos(16, 0, 128, 2) == (4, 0)
    # channel d+1 -> g = 1 -> four lane chunks further; d = 8 -> rh = 1 -> two words further
    assert ol.v_code_pos(0, 1, 128, 2) == (64, 0)
    assert ol.v_code_pos(0, 8, 128, 2) == (8, 0)
    # channels 16 apart share the byte: d = 16, 32, 48 at bits 2, 4, 6; d = 64 -> next group of 512 bytes
    assert ol.v_code_pos(0, 16, 128, 2) == (0, 2)
    assert ol.v_code_pos(0, 48, 128, 2) == (0, 6)
    assert ol.v_code_pos(0, 64, 128, 2) == (512, 0)
    # next block of 32 tokens: 4*128*2 = 1024 bytes further; the very last code of the page
    assert ol.v_code_pos(32, 0, 128, 2) == (1024, 0)
    assert ol.v_code_pos(127, 127, 128, 2) == (4095, 6)
    # head_dim 64: all four 16-channel slices share one group, a block is 512 bytes
    assert ol.v_code_pos(0, 48, 64, 2) == (0, 6)
    assert ol.v_code_pos(32, 0, 64, 2) == (512, 0)
    # quad-major word placement when a chunk has more than 4 words:
    # K, D=128, 8-bit (one field per byte, 8 words per chunk): d=2 -> byte 2; d=4 -> chunk 1 -> byte 16;
    # d=16 -> word 1 -> byte 4; d=64 -> word 4 -> second quad -> byte 4 chunks * 16 = 64; d=68 -> 64 + 16
    assert ol.k_code_pos(0, 2, 128, 8) == (2, 0)
    assert ol.k_code_pos(0, 4, 128, 8) == (16, 0)
    assert ol.k_code_pos(0, 16, 128, 8) == (4, 0)
    assert ol.k_code_pos(0, 64, 128, 8) == (64, 0)
    assert ol.k_code_pos(0, 68, 128, 8) == (80, 0)
    assert ol.k_code_pos(1, 0, 128, 8) == (128, 0)
    # V, D=128, 4-bit (2 codes per byte: d and d+16; a block is 2048 bytes): d = 32 -> next group of 512 bytes
    assert ol.v_code_pos(0, 16, 128, 4) == (0, 4)
    assert ol.v_code_pos(0, 32, 128, 4) == (512, 0)
    assert ol.v_code_pos(2, 64, 128, 4) == (1040, 0)
    assert ol.v_code_pos(32, 0, 128, 4) == (2048, 0)
    # 8-bit: one code per byte, every 16-channel slice has its own group of 512 bytes
    assert ol.v_code_pos(0, 0, 128, 8) == (0, 0)
    assert ol.v_code_pos(8, 0, 128, 8) == (1, 0)
    assert ol.v_code_pos(1, 0, 128, 8) == (2, 0)
    assert ol.v_code_pos(0, 16, 128, 8) == (512, 0)
    assert ol.v_code_pos(0, 9, 128, 8) == (72, 0)


def test_memory_ratio_k4v2_vs_k4v4():
    """Sec. 1: K4V2 needs 25 % less code memory than K4V4; with fp16 (scale, zero)
    per 128-group the page ratio is 104/136."""
    a = ol.Layout(128, 4, 2, 128, 128)
    b = ol.Layout(128, 4, 4, 128, 128)
    assert (a.k_codes_bytes + a.v_codes_bytes) / (b.k_codes_bytes + b.v_codes_bytes) == 0.75
    assert a.page_bytes == 128 * 104 and b.page_bytes == 128 * 136
    assert a.page_bytes == 13312


# ------------------------------------------------------------------ attention
def torch_reference_attention(q, K, V, seq_len):
    """Textbook softmax(q K^T / sqrt(D)) V through a library routine, fp64."""
    B, Hq, D = q.shape
    G = Hq // K.shape[1]
    out = np.zeros((B, Hq, D))
    for b in range(B):
        n = int(seq_len[b])
        if n == 0:
            continue
        kk = torch.from_numpy(K[b, :, :n]).repeat_interleave(G, dim=0)
        vv = torch.from_numpy(V[b, :, :n]).repeat_interleave(G, dim=0)
        qq = torch.from_numpy(q[b])[:, None, :]
        o = torch.nn.functional.scaled_dot_product_attention(qq[None], kk[None], vv[None])
        out[b] = o[0, :, 0].numpy()
    return out


def test_attention_matches_library_sdpa():
    B, Hq, Hkv, T, D = 2, 8, 2, 300, 64
    q = RNG.standard_normal((B, Hq, D))
    K = RNG.standard_normal((B, Hkv, T, D)) * 2
    V = RNG.standard_normal((B, Hkv, T, D))
    seq = np.array([300, 123])
    got = oa.decode_attention(q, K, V, seq)
    want = torch_reference_attention(q, K, V, seq)
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)


def test_attention_special_cases():
    D, T = 32, 50
    q = RNG.standard_normal(D)
    K = RNG.standard_normal((T, D))
    V = RNG.standard_normal((T, D))
    sc = 1 / math.sqrt(D)
    # T = 1: the output is the single value row
    assert np.allclose(oa.attend_one(q, K[:1], V[:1], sc), V[0], atol=1e-15)
    # T = 0
    assert np.array_equal(oa.attend_one(q, K[:0], V[:0], sc), np.zeros(D))
    # q = 0: uniform weights -> mean of V
    assert np.allclose(oa.attend_one(np.zeros(D), K, V, sc), V.mean(0), atol=1e-14)
    # convex combination: within the column-wise min/max of V
    o = oa.attend_one(q, K, V, sc)
    assert np.all(o <= V.max(0) + 1e-12) and np.all(o >= V.min(0) - 1e-12)
    # permutation of cached tokens leaves the output unchanged
    perm = RNG.permutation(T)
    assert np.allclose(oa.attend_one(q, K[perm], V[perm], sc), o, atol=1e-13)
    # scale matters and is applied to the logits: huge scale -> argmax token's value
    t = np.argmax(K @ q)
    assert np.allclose(oa.attend_one(q, K, V, 1e4), V[t], atol=1e-9)
    # two-token closed form: weights are a logistic of the logit difference
    l0, l1 = sc * K[0] @ q, sc * K[1] @ q
    w1 = 1 / (1 + math.exp(l0 - l1))
    assert np.allclose(oa.attend_one(q, K[:2], V[:2], sc), (1 - w1) * V[0] + w1 * V[1], atol=1e-14)


def test_lse_merge_any_partition():
    D, T = 16, 257
    q = RNG.standard_normal(D) * 3
    K = RNG.standard_normal((T, D))
    V = RNG.standard_normal((T, D))
    sc = 0.25
    whole = oa.attend_one(q, K, V, sc)
    for cuts in ([0, 257], [0, 1, 257], [0, 100, 100, 200, 257], [0, 128, 256, 257]):
        parts = [oa.partial_state(q, K[a:b], V[a:b], sc) for a, b in zip(cuts[:-1], cuts[1:])]
        assert np.allclose(oa.lse_merge(parts), whole, atol=1e-13)
    assert np.array_equal(oa.lse_merge([oa.partial_state(q, K[:0], V[:0], sc)]), np.zeros(D))


def test_gqa_mapping_and_identical_heads():
    B, Hq, Hkv, T, D = 1, 8, 2, 40, 16
    q = RNG.standard_normal((B, Hq, D))
    q[0, 1] = q[0, 0]                   # same KV group (G = 4): identical outputs
    q[0, 4] = q[0, 0]                   # other KV group: different output
    K = RNG.standard_normal((B, Hkv, T, D))
    V = RNG.standard_normal((B, Hkv, T, D))
    o = oa.decode_attention(q, K, V, np.array([T]))
    assert np.array_equal(o[0, 0], o[0, 1])
    assert not np.allclose(o[0, 0], o[0, 4])
    assert np.allclose(o[0, 4], oa.attend_one(q[0, 4], K[0, 1], V[0, 1], 1 / math.sqrt(D)))


# ------------------------------------------------------------------ cache
def test_cache_passthrough_reduces_to_exact_attention():
    """kb = vb = 16: the packed cache stores the inputs and decode equals textbook
    attention on them (library SDPA, fp64)."""
    w = wl.TINY.with_(kb=16, vb=16)
    k, v = wl.make_kv(w, tokens=200, batch=2)
    q = wl.make_q(w, batch=2)
    c = OracleCache(2, w.n_kv_heads, w.head_dim, 16, 16, 32, 32, 0, "fp16", 256)
    c.append(bits_of(k)[:, :, :150], bits_of(v)[:, :, :150])
    c.append(bits_of(k)[:, :, 150:], bits_of(v)[:, :, 150:])
    assert c.seq_len.tolist() == [200, 200]
    got = c.decode(bits_of(q))
    want = torch_reference_attention(q.double().numpy(), k.double().numpy(), v.double().numpy(), [200, 200])
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)
    ko = np.zeros((2, w.n_kv_heads, 256, w.head_dim), np.uint16)
    vo = np.zeros_like(ko)
    c.dequantize(ko, vo, 0, 256)
    assert np.array_equal(ko[:, :, :200], bits_of(k)) and np.array_equal(vo[:, :, :200], bits_of(v))
    assert not ko[:, :, 200:].any()


@pytest.mark.parametrize("k_axis", [0, 1])
def test_cache_append_is_chunking_invariant(k_axis):
    """Appending token by token, in ragged chunks or in bulk gives the same bytes."""
    w = wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=8, k_axis=k_axis)
    T = 300
    k, v = wl.make_kv(w, tokens=T, batch=1)
    kb_, vb_ = bits_of(k), bits_of(v)

    def build(chunks):
        c = OracleCache(1, 2, 128, 4, 2, 128, 128, k_axis, "bf16", 384)
        t = 0
        for n in chunks:
            c.append(kb_[:, :, t:t + n], vb_[:, :, t:t + n])
            t += n
        return c
    a = build([T])
    b = build([1] * 130 + [127, 43])
    c = build([100, 100, 100])
    for other in (b, c):
        assert np.array_equal(a.pages, other.pages)
        assert np.array_equal(a.seq_len, other.seq_len)
        if k_axis:
            r = T % 128
            assert np.array_equal(a.k_tail[:, :, :r], other.k_tail[:, :, :r])
    if k_axis:
        # tail holds the last T % 128 tokens as fp16; full blocks are channel-quantized
        r = T % 128
        assert np.array_equal(a.k_tail[0, 0, :r], oq.to_tail_fp16_bits(kb_[0, 0, 256:], "bf16"))
        L = a.L
        blk = oq.to_tail_fp16_bits(kb_[0, 1, 128:256], "bf16")
        codes, s16, z16 = oq.quantize_per_channel_block(blk, 4)
        assert np.array_equal(ol.get_k_codes(a.pages[0, 1, 1], L), codes)
        s2, z2 = ol.get_k_meta(a.pages[0, 1, 1], L)
        assert np.array_equal(s2, s16) and np.array_equal(z2, z16)
        assert not a.pages[0, 0, 2, : L.k_codes_bytes].any()      # partial page: K codes untouched


def test_cache_capacity_overflow_sets_status_and_writes_nothing():
    w = wl.TINY
    k, v = wl.make_kv(w, tokens=200, batch=1)
    c = OracleCache(1, 8, 64, 4, 2, 32, 32, 0, "fp16", 128)
    c.append(bits_of(k)[:, :, :100], bits_of(v)[:, :, :100])
    before = c.pages.copy()
    c.append(bits_of(k)[:, :, 100:], bits_of(v)[:, :, 100:])
    assert c.status == 1 and c.seq_len[0] == 100 and np.array_equal(before, c.pages)


def test_cache_dequantize_error_bound_and_decode_close_to_unquantized():
    w = wl.TINY.with_(kb=8, vb=8)
    T = 256
    k, v = wl.make_kv(w, tokens=T, batch=1)
    q = wl.make_q(w, batch=1)
    c = OracleCache(1, 8, 64, 8, 8, 32, 32, 0, "fp16", 256)
    c.append(bits_of(k), bits_of(v))
    Kh, Vh = c.values_f64()
    # 8-bit, range ~ 8 sigma over 32 values: step <= ~0.07 -> error <= 0.035
    assert np.abs(Kh - k.double().numpy()).max() < 0.04
    assert np.abs(Vh - v.double().numpy()).max() < 0.02
    exact = torch_reference_attention(q.double().numpy(), k.double().numpy(), v.double().numpy(), [T])
    assert np.abs(c.decode(bits_of(q)) - exact).max() < 0.02
    ko = np.zeros((1, 8, 256, 64), np.uint16)
    vo = np.zeros_like(ko)
    c.dequantize(ko, vo, 10, 200)
    assert not ko[:, :, :10].any() and not ko[:, :, 200:].any()
    got = oq.bits_to_f32(ko[:, :, 10:200], "fp16")
    assert np.abs(got - Kh[:, :, 10:200]).max() <= np.abs(Kh).max() * 2.0 ** -10
    s = c.decode_streams(bits_of(q), [(0, 3)])
    assert np.allclose(s[(0, 3)][0], c.decode(bits_of(q))[0, 3], atol=1e-14)


def test_k4v2_beats_k2v4_when_key_norm_exceeds_value_norm():
    """Thm 2 (key-prioritized quantization), in expectation: under an equal bit
    budget, giving the extra bits to the keys yields a smaller attention-output
    error on caches whose key norm exceeds the value norm.  8B- and 70B-shaped
    synthetic caches, 6 seeds each."""
    for base in (wl.LLAMA_8B, wl.LLAMA_70B):
        w = base.with_(n_kv_heads=2, n_q_heads=2 * (base.n_q_heads // base.n_kv_heads))
        e42, e24 = [], []
        for seed in range(6):
            k, v = wl.make_kv(w, layer=seed, tokens=512, batch=1)
            assert k.float().norm() > 1.5 * v.float().norm()
            q = wl.make_q(w, layer=seed, batch=1)
            exact = torch_reference_attention(q.double().numpy(), k.double().numpy(), v.double().numpy(), [512])
            for (kb, vb, acc) in ((4, 2, e42), (2, 4, e24)):
                c = OracleCache(1, 2, 128, kb, vb, 128, 128, 0, "bf16", 512)
                c.append(bits_of(k), bits_of(v))
                acc.append(np.linalg.norm(c.decode(bits_of(q)) - exact) / np.linalg.norm(exact))
        assert np.mean(e42) < np.mean(e24), (base.name, np.mean(e42), np.mean(e24))


def test_multi_row_attention_matches_library_causal_sdpa():
    """Several query rows with a decoder's causal mask against torch's scaled_dot_product_attention in fp64:
    the R rows are the last R positions of a T-token sequence."""
    B, Hq, Hkv, T, D, R = 2, 4, 2, 37, 16, 3
    q = RNG.normal(size=(B, R, Hq, D))
    K = RNG.normal(size=(B, Hkv, T, D))
    V = RNG.normal(size=(B, Hkv, T, D))
    got = oa.decode_attention_rows(q, K, V, [T, T])
    G = Hq // Hkv
    mask = torch.zeros((R, T), dtype=torch.bool)
    for r in range(R):
        mask[r, : T - (R - 1 - r)] = True
    qt = torch.from_numpy(q).permute(0, 2, 1, 3)                              # (B, Hq, R, D)
    kt = torch.from_numpy(K).repeat_interleave(G, 1)
    vt = torch.from_numpy(V).repeat_interleave(G, 1)
    want = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask).permute(0, 2, 1, 3).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)
    # one row is the plain decode step; the last row of several sees the whole cache
    one = oa.decode_attention_rows(q[:, -1:], K, V, [T, T])
    assert np.array_equal(one[:, 0], oa.decode_attention(q[:, -1], K, V, [T, T]))
    assert np.array_equal(got[:, -1], one[:, 0])
    # ragged: a sequence shorter than the number of rows leaves the rows without a token at zero
    short = oa.decode_attention_rows(q, K, V, [2, T])
    assert not short[0, 0].any() and short[0, 1].any() and short[0, 2].any()
    assert np.array_equal(short[0, 1, 0], V[0, 0, 0])                          # row 1 sees exactly token 0


@pytest.mark.parametrize("D,b", [(128, 1), (128, 3), (128, 6), (64, 6)])
def test_bit_plane_widths_tile_the_region_and_keep_their_planes_apart(D, b):
    """1-, 3- and 6-bit codes are stored as planes of 1, 2 or 4 bits (high plane first): every code bit of every
    (token, channel) owns one distinct bit of the region, the region is exactly 128*D*b/8 bytes, and the high
    plane of a code sits in the first part of the region."""
    L = ol.Layout(D, b, b, 64, 64, 0)
    assert L.k_codes_bytes == 128 * D * b // 8 and L.v_codes_bytes == 128 * D * b // 8
    for put, get, off in ((ol.put_k_codes, ol.get_k_codes, 0), (ol.put_v_codes, ol.get_v_codes, L.v_codes_off)):
        seen = np.zeros(L.page_bytes, np.uint16)
        for bit in range(b):                                   # one code bit at a time: count the region bits it sets
            page = np.zeros(L.page_bytes, np.uint8)
            put(page, L, np.arange(128), np.full((128, D), 1 << bit, np.uint16))
            ones = np.unpackbits(page[off: off + 128 * D * b // 8]).sum()
            assert ones == 128 * D and not page[:off].any() and not page[off + 128 * D * b // 8:].any()
            assert not (seen[: L.page_bytes] & page).any()     # no region bit serves two code bits
            seen |= page
            assert np.array_equal(get(page, L), np.full((128, D), 1 << bit, np.uint8))
        assert np.all(seen[off: off + 128 * D * b // 8] == 0xFF)
    # hand-computed: 3-bit key code 5 = (2-bit plane 2, 1-bit plane 1) of token 0, channel 0
    if b == 3:
        page = np.zeros(L.page_bytes, np.uint8)
        codes = np.zeros((1, D), np.uint16); codes[0, 0] = 5
        ol.put_k_codes(page, L, np.array([0]), codes)
        assert page[0] == 2 and page[128 * D * 2 // 8] == 1 and page.sum() == 3


def test_residual_window_keeps_recent_tokens_exact_and_flushes_whole_blocks():
    """Sec. 4.1's residual buffer: with R = 64 the newest seq_len mod 64 tokens of K and V are the 16-bit inputs
    themselves; the tokens behind them carry exactly the codes a cache without a window would have; any chunking
    of the appends gives the same state."""
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    T, R = 64 * 3 + 21, 64
    k, v = wl.make_kv(w, tokens=T, batch=2)
    kb_, vb_ = bits_of(k), bits_of(v)
    def build(chunks, residual):
        oc = OracleCache(2, 2, 128, 4, 2, 128, 128, 0, "bf16", 256, residual=residual)
        t = 0
        for n in chunks:
            oc.append(kb_[:, :, t:t + n], vb_[:, :, t:t + n]); t += n
        return oc
    a = build([T], R)
    for chunks in ([1] * T, [63, 1, 1, 64, 70, T - 199], [130, T - 130]):
        c = build(chunks, R)
        assert np.array_equal(a.pages, c.pages) and np.array_equal(a.seq_len, c.seq_len)
        n = T % R
        slots = np.arange(T - n, T) % R
        assert np.array_equal(a.kv_win[:, :, slots], c.kv_win[:, :, slots])
    plain = build([192], 0)                                     # the flushed part = a cache of the first 192 tokens
    assert np.array_equal(a.pages[:, :, :1], plain.pages[:, :, :1])
    assert np.array_equal(a.pages[:, :, 1, : ], plain.pages[:, :, 1])
    K, V = a.values_f64()
    assert np.array_equal(K[:, :, 192:T], oq.bits_to_f32(kb_[:, :, 192:T], "bf16").astype(np.float64))
    assert np.array_equal(V[:, :, 192:T], oq.bits_to_f32(vb_[:, :, 192:T], "bf16").astype(np.float64))
    Kp, _ = plain.values_f64()
    assert np.array_equal(K[:, :, :192], Kp[:, :, :192])
    # dequantize returns the window tokens bit for bit
    ko = np.zeros((2, 2, 256, 128), np.uint16); vo = np.zeros_like(ko)
    a.dequantize(ko, vo, 0, 256)
    assert np.array_equal(ko[:, :, 192:T], kb_[:, :, 192:T]) and np.array_equal(vo[:, :, 192:T], vb_[:, :, 192:T])
    # attention with a window is closer to exact attention than without (recent tokens carry no error)
    q = wl.make_q(w, batch=2)
    exact = oa.decode_attention(q.double().numpy(), k.double().numpy(), v.double().numpy(), [T, T])
    e_win = np.linalg.norm(a.decode(bits_of(q)) - exact)
    e_plain = np.linalg.norm(build([T], 0).decode(bits_of(q)) - exact)
    assert e_win < e_plain
