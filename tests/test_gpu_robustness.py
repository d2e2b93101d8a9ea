"""Robustness of the CUDA path without faulting anything: the bounded device-side waits really expire and
leave the context usable; the two decode implementations agree with each other and with the oracle; no call
writes outside the buffers it was given (canary words behind every output)."""
import numpy as np
import pytest
import torch

from paper_2502_15075_b200 import workloads as wl

import kvq_testlib as tl

pytestmark = pytest.mark.gpu

CANARY = 0xA5


@pytest.fixture(scope="module")
def kvq():
    from paper_2502_15075_b200 import build
    build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


def padded(nbytes, pad=4096):
    """A uint8 CUDA buffer of nbytes with `pad` canary bytes behind it: (whole, view of the first nbytes)."""
    whole = torch.full((nbytes + pad,), CANARY, dtype=torch.uint8, device="cuda")
    return whole, whole[:nbytes]


def canary_intact(whole, nbytes):
    return bool((whole[nbytes:] == CANARY).all())


@pytest.mark.parametrize("name,w,B,T", [
    ("8b-k4v2", wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8), 2, 900),
    ("8b-k8v4", wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8, kb=8, vb=4), 1, 500),
    ("14b-chan", wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=8), 2, 128 * 4 + 70),
    ("70b-g8", wl.LLAMA_70B.with_(n_kv_heads=2, n_q_heads=16), 1, 1100),
])
def test_fast_and_generic_kernels_agree_with_the_oracle(kvq, name, w, B, T):
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cap = ((T + 127) // 128) * 128
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], cap)
    q = wl.make_q(w, batch=B).cuda()
    want = tl.oracle_on_gpu_codes(gc, w).decode(tl.bits_of(q))
    nws = max(16, kvq.kvq_workspace_bytes(cfg))
    outs = []
    for fn in (kvq.kvq_decode_attention, kvq.kvq_debug_decode_generic):
        ws_whole, ws = padded(nws)
        out_whole, out_b = padded(q.numel() * 4)
        out = out_b.view(torch.float32).view(q.shape)
        fn(cfg, gc, q, out, ws)
        torch.cuda.synchronize()
        assert kvq.kvq_check_status(gc) == 0
        assert canary_intact(ws_whole, nws) and canary_intact(out_whole, q.numel() * 4)
        got = out.double().cpu().numpy()
        tl.assert_attention_close(got, want)
        outs.append(got)
    tl.assert_attention_close(outs[0], outs[1], rel=2e-3)


def test_a_wait_that_runs_out_sets_the_status_and_leaves_the_context_usable(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B, T = 2, 128 * 40
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], T)
    q = wl.make_q(w, batch=B).cuda()
    ws = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device="cuda")
    out = torch.zeros(tuple(q.shape), dtype=torch.float32, device="cuda")
    good = tl.gpu_decode(kvq, cfg, gc, q)
    # page 57 of the 160 pages never arrives; every wait gives up after 2 ms
    kvq.kvq_debug_decode_stall(cfg, gc, q, out, ws, 57, 2000)
    torch.cuda.synchronize()                                   # returns: nothing hangs
    assert kvq.kvq_check_status(gc) == -7                      # KVQ_ERR_DEVICE_TIMEOUT
    gc.status.zero_()
    # the same cache and workspace work again, with and without the hook's short limit
    kvq.kvq_debug_decode_stall(cfg, gc, q, out, ws, -1, 50000)
    torch.cuda.synchronize()
    assert kvq.kvq_check_status(gc) == 0
    tl.assert_attention_close(out.double().cpu().numpy(), good, rel=1e-6, mabs=1e-6)
    again = tl.gpu_decode(kvq, cfg, gc, q)
    assert np.array_equal(again, good)


def test_append_and_dequantize_stay_inside_their_buffers(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B, cap, T = 2, 256, 200
    cfg = tl.gpu_config_for(kvq, w, B, cap)
    gc = kvq.Cache(cfg)
    n = gc.pages.numel()
    whole, view = padded(n)
    view.zero_()
    gc.pages = view
    gc.c.pages = view.data_ptr()
    k, v = wl.make_kv(w, tokens=T, batch=B)
    oc = tl.oracle_cache_for(w, B, cap)
    for lo, hi in ((0, 77), (77, 78), (78, T)):
        kvq.kvq_quantize_append(cfg, gc, k.cuda()[:, :, lo:hi], v.cuda()[:, :, lo:hi])
        oc.append(tl.bits_of(k)[:, :, lo:hi], tl.bits_of(v)[:, :, lo:hi])
    torch.cuda.synchronize()
    assert canary_intact(whole, n)
    tl.assert_caches_equal(gc, oc)
    nb = B * 2 * cap * 128 * 2
    kw, kb_ = padded(nb)
    vw, vb_ = padded(nb)
    kb_.zero_(); vb_.zero_()
    ko = kb_.view(torch.bfloat16).view(B, 2, cap, 128)
    vo = vb_.view(torch.bfloat16).view(B, 2, cap, 128)
    kvq.kvq_dequantize(cfg, gc, ko, vo, 0, cap)
    torch.cuda.synchronize()
    assert canary_intact(kw, nb) and canary_intact(vw, nb)
    assert not ko[:, :, T:].any() and not vo[:, :, T:].any()


def test_append_guard_rejects_lengths_near_int_max(kvq):
    """A corrupt seq_len close to INT_MAX must not pass the capacity check by wrapping around."""
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    cfg = tl.gpu_config_for(kvq, w, 2, 256)
    gc = kvq.Cache(cfg)
    k, v = wl.make_kv(w, tokens=8, batch=2)
    gc.seq_len.copy_(torch.tensor([2 ** 31 - 1, 2 ** 31 - 8], dtype=torch.int32))
    before = gc.pages.clone()
    kvq.kvq_quantize_append(cfg, gc, k.cuda(), v.cuda())
    assert kvq.kvq_check_status(gc) == -5
    assert gc.seq_len.tolist() == [2 ** 31 - 1, 2 ** 31 - 8] and torch.equal(gc.pages, before)
