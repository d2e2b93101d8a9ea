"""GPU parity of the tcgen05 / tensor-memory decode kernel: against the fp64 oracle on the same codes
(rel-L2 2e-3, max-abs 1e-2) and against the warp-level MMA kernel, on every configuration it serves."""
import numpy as np
import pytest
import torch

from paper_2502_15075_b200 import workloads as wl

import kvq_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kvq():
    from paper_2502_15075_b200 import build
    build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


def decode_impl(kvq, cfg, gc, q, impl, rows=1):
    n = kvq.kvq_workspace_bytes_rows(cfg, rows) if rows > 1 else kvq.kvq_workspace_bytes(cfg)
    ws = torch.empty(max(16, n), dtype=torch.uint8, device="cuda")
    out = torch.full(tuple(q.shape), float("nan"), dtype=torch.float32, device="cuda")
    kvq.kvq_debug_decode_impl(cfg, gc, q.cuda(), out, ws, impl)
    torch.cuda.synchronize()
    assert kvq.kvq_check_status(gc) == 0
    return out.double().cpu().numpy()


CASES = {
    # name: (workload, batch, tokens per sequence (ragged), kv heads)
    "k4v2": (wl.LLAMA_8B, 2, [700, 385], 2),
    "k4v2-one-token": (wl.LLAMA_8B, 2, [1, 129], 1),
    "k4v2-many-streams": (wl.LLAMA_8B, 5, [2000, 1500, 128, 0, 3000], 8),
    "k4v4": (wl.LLAMA_8B.with_(kb=4, vb=4), 2, [300, 1000], 2),
    "k8v4": (wl.LLAMA_8B.with_(kb=8, vb=4), 2, [300, 513], 2),
    "k8v2": (wl.LLAMA_8B.with_(kb=8, vb=2), 1, [640], 2),
    "k4v2-2heads": (wl.LLAMA_8B.with_(n_q_heads=16), 2, [700, 900], 2),       # two query heads per KV head
}


@pytest.mark.parametrize("name", list(CASES))
def test_tcgen05_decode_against_oracle_and_warp_kernel(kvq, name):
    w, B, lens, hk = CASES[name]
    w = w.with_(n_kv_heads=hk, n_q_heads=hk * (w.n_q_heads // w.n_kv_heads))
    T = max(lens)
    cap = ((T + 127) // 128) * 128 + 128
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg = tl.gpu_config_for(kvq, w, B, cap)
    gc = kvq.Cache(cfg)
    kd, vd = k.cuda(), v.cuda()
    # ragged lengths: append the longest length everywhere, then shorten (the codes beyond a length are unused)
    kvq.kvq_quantize_append(cfg, gc, kd, vd)
    gc.seq_len.copy_(torch.tensor(lens, dtype=torch.int32))
    torch.cuda.synchronize()
    oc = tl.oracle_on_gpu_codes(gc, w)
    for variant in ("normal", "large", "peaked"):
        q = wl.make_q(w, batch=B, variant=variant, k=k)
        want = oc.decode(tl.bits_of(q))
        got = decode_impl(kvq, cfg, gc, q, kvq.IMPL_TCGEN05)
        tl.assert_attention_close(got, want)
        other = decode_impl(kvq, cfg, gc, q, kvq.IMPL_WARP_MMA)
        tl.assert_attention_close(got, other, rel=2e-3, mabs=1e-2)


def test_tcgen05_decode_several_causal_rows(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=4)       # two heads per KV head x two rows = four virtual heads
    B, T, rows = 2, 900, 2
    cap = 1024
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], cap)
    oc = tl.oracle_on_gpu_codes(gc, w)
    q = torch.stack([wl.make_q(w, layer=r, batch=B) for r in range(rows)], dim=1).contiguous()
    want = oc.decode_rows(tl.bits_of(q))
    got = decode_impl(kvq, cfg, gc, q, kvq.IMPL_TCGEN05, rows=rows)
    tl.assert_attention_close(got, want)


def test_tcgen05_refuses_configurations_it_does_not_serve(kvq):
    w = wl.LLAMA_70B.with_(n_kv_heads=1, n_q_heads=8)      # eight query heads per KV head
    k, v = wl.make_kv(w, tokens=256, batch=1)
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [256], 256)
    q = wl.make_q(w, batch=1).cuda()
    ws = torch.empty(kvq.kvq_workspace_bytes(cfg), dtype=torch.uint8, device="cuda")
    out = torch.empty(tuple(q.shape), dtype=torch.float32, device="cuda")
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_debug_decode_impl(cfg, gc, q, out, ws, kvq.IMPL_TCGEN05)
    assert e.value.code == -2


def test_tcgen05_wait_that_runs_out_sets_the_status_and_frees_its_tensor_memory(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B, T = 2, 128 * 40
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], T)
    q = wl.make_q(w, batch=B).cuda()
    ws = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device="cuda")
    out = torch.zeros(tuple(q.shape), dtype=torch.float32, device="cuda")
    good = decode_impl(kvq, cfg, gc, q, kvq.IMPL_TCGEN05)
    # page 57 of the 160 pages never arrives; every wait gives up after 2 ms
    kvq.kvq_debug_decode_stall_impl(cfg, gc, q, out, ws, 57, 2000, kvq.IMPL_TCGEN05)
    torch.cuda.synchronize()                                   # returns: nothing hangs
    assert kvq.kvq_check_status(gc) == -7                      # KVQ_ERR_DEVICE_TIMEOUT
    gc.status.zero_()
    # the next launches find the SMs' tensor memory free again and give the same result as before
    for _ in range(3):
        again = decode_impl(kvq, cfg, gc, q, kvq.IMPL_TCGEN05)
        assert np.array_equal(again, good)


@pytest.mark.parametrize("R,T,chunks", [(64, 64 * 5 + 37, [64 * 5 + 37]), (128, 128 * 2 + 100, [300, 56]), (64, 40, [40])])
def test_tcgen05_decode_merges_the_residual_window(kvq, R, T, chunks):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B = 2
    cap = ((T + 127) // 128) * 128 + 128
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg, gc, _ = tl.build_both(kvq, w, k, v, chunks, cap, residual=R)
    q = wl.make_q(w, batch=B)
    want = tl.oracle_on_gpu_codes(gc, w).decode(tl.bits_of(q))
    tl.assert_attention_close(decode_impl(kvq, cfg, gc, q, kvq.IMPL_TCGEN05), want)
