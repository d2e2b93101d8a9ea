"""Parity at the full sizes of the model-shaped configurations, one layer each, through the same C-ABI calls
and launch configuration the benchmark times.  The oracle checks sampled (batch, kv-head) streams one by one:
packed bytes of sampled pages bit for bit, attention outputs within rel-L2 2e-3 / max-abs 1e-2."""
import numpy as np
import pytest
import torch

from oracle import quantizer as oq
from oracle import layout as ol
from oracle.cache import OracleCache
from paper_2502_15075_b200 import workloads as wl

import kvq_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kvq():
    from paper_2502_15075_b200 import build
    build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


def _oracle_stream(gc, w, b, h, cap):
    """Oracle cache holding the GPU's bytes of one stream."""
    oc = OracleCache(1, 1, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis, w.dtype, cap)
    oc.pages = gc.pages_view()[b:b + 1, h:h + 1].cpu().numpy().copy()
    if oc.k_tail is not None:
        oc.k_tail = gc.tail_view()[b:b + 1, h:h + 1].cpu().view(torch.int16).numpy().view(np.uint16).copy()
    oc.seq_len[:] = int(gc.seq_len[b])
    return oc


def _check_pages_bit_exact(gc, w, k, v, b, h, pages, T):
    """Re-quantize sampled pages of one stream with the oracle from the original inputs."""
    L = ol.Layout(w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis)
    for p in pages:
        t0, t1 = p * 128, min(T, p * 128 + 128)
        oc = OracleCache(1, 1, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis, w.dtype, 128)
        oc.append(tl.bits_of(k[b:b + 1, h:h + 1, t0:t1]), tl.bits_of(v[b:b + 1, h:h + 1, t0:t1]))
        got = gc.pages_view()[b, h, p].cpu().numpy()
        n = t1 - t0
        if n == 128:
            assert np.array_equal(got, oc.pages[0, 0, 0]), f"page {p} of stream ({b},{h}) differs"
        else:   # partial page: compare the fields of the valid tokens
            assert np.array_equal(ol.get_v_codes(got, L)[:n], ol.get_v_codes(oc.pages[0, 0, 0], L)[:n])
            s1, z1 = ol.get_v_meta(got, L)
            s2, z2 = ol.get_v_meta(oc.pages[0, 0, 0], L)
            assert np.array_equal(s1[:n], s2[:n]) and np.array_equal(z1[:n], z2[:n])
            if w.k_axis == 0:
                assert np.array_equal(ol.get_k_codes(got, L)[:n], ol.get_k_codes(oc.pages[0, 0, 0], L)[:n])
            else:
                gt = gc.tail_view()[b, h].cpu().view(torch.int16).numpy().view(np.uint16)
                assert np.array_equal(gt[:n], oq.to_tail_fp16_bits(tl.bits_of(k[b, h, t0:t1]), w.dtype))


CASES = {
    "8b-k4v2": (wl.LLAMA_8B, None),
    "8b-k2v4": (wl.LLAMA_8B.with_(kb=2, vb=4), None),
    "8b-k4v4": (wl.LLAMA_8B.with_(kb=4, vb=4), None),
    "8b-k8v4": (wl.LLAMA_8B.with_(kb=8, vb=4), None),
    "14b-k4v2-tail127": (wl.SHAPED_14B, 16383),
    "14b-k8v2": (wl.SHAPED_14B.with_(kb=8), None),
    "70b": (wl.LLAMA_70B, None),
    "1b": (wl.LLAMA_1B, None),
}


@pytest.mark.parametrize("name", list(CASES))
def test_full_size_layer(kvq, name):
    w, T = CASES[name]
    T = w.context if T is None else T
    B, H = w.batch, w.n_kv_heads
    G = w.n_q_heads // H
    cap = ((T + 127) // 128) * 128
    k, v = wl.make_kv(w, layer=0, device="cuda", tokens=T)
    q = wl.make_q(w, layer=0, device="cuda")
    cfg = tl.gpu_config_for(kvq, w, B, cap)
    gc = kvq.Cache(cfg)
    # bulk build, then the last 129 tokens as a 128-token chunk and a single token (config 2: "append 128 then decode")
    cut = T - 129
    for lo, hi in ((0, cut), (cut, T - 1), (T - 1, T)):
        kvq.kvq_quantize_append(cfg, gc, k[:, :, lo:hi], v[:, :, lo:hi])
    assert kvq.kvq_check_status(gc) == 0
    assert gc.seq_len.tolist() == [T] * B
    out = tl.gpu_decode(kvq, cfg, gc, q)
    n_pages = cap // 128
    streams = [(0, 0), (B - 1, H - 1), (B // 2, H // 3)]
    for (b, h) in streams:
        _check_pages_bit_exact(gc, w, k, v, b, h, sorted({0, n_pages // 2, (cut // 128), n_pages - 1}), T)
        oc = _oracle_stream(gc, w, b, h, cap)
        want = oc.decode(tl.bits_of(q[b:b + 1, h * G:(h + 1) * G]))
        tl.assert_attention_close(out[b:b + 1, h * G:(h + 1) * G], want)
    # dequantize of the newest page is bit-exact against the oracle on the same bytes
    ko = torch.zeros((B, H, cap, w.head_dim), dtype=w.torch_dtype, device="cuda")
    vo = torch.zeros_like(ko)
    t_lo = ((T - 1) // 128) * 128
    kvq.kvq_dequantize(cfg, gc, ko, vo, t_lo, T)
    b, h = streams[1]
    oc = _oracle_stream(gc, w, b, h, cap)
    kr = np.zeros((1, 1, cap, w.head_dim), np.uint16)
    vr = np.zeros_like(kr)
    oc.dequantize(kr, vr, t_lo, T)
    assert np.array_equal(tl.bits_of(ko[b, h, t_lo:T]), kr[0, 0, t_lo:T])
    assert np.array_equal(tl.bits_of(vo[b, h, t_lo:T]), vr[0, 0, t_lo:T])


def test_full_size_ragged_lengths(kvq):
    """8B-shaped layer with seq_len ~ U(T/2, T): the flat split has to balance unequal streams."""
    w = wl.LLAMA_8B
    T, B, H, G = w.context, w.batch, w.n_kv_heads, 4
    k, v = wl.make_kv(w, layer=1, device="cuda")
    q = wl.make_q(w, layer=1, device="cuda")
    cfg = tl.gpu_config_for(kvq, w, B, T)
    gc = kvq.Cache(cfg)
    kvq.kvq_quantize_append(cfg, gc, k, v)
    lens = wl.ragged_seq_lens(w, T, B)
    lens[3] = 0
    lens[5] = 1
    gc.seq_len.copy_(lens)
    out = tl.gpu_decode(kvq, cfg, gc, q)
    assert not out[3].any()
    for (b, h) in [(0, 0), (5, 2), (B - 1, H - 1), (7, 4)]:
        oc = _oracle_stream(gc, w, b, h, T)
        want = oc.decode(tl.bits_of(q[b:b + 1, h * G:(h + 1) * G]))
        tl.assert_attention_close(out[b:b + 1, h * G:(h + 1) * G], want)
