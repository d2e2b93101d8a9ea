"""A decode step captured in a CUDA graph and replayed.

The library never synchronises, allocates or reads device memory on the host inside
kvq_quantize_append, kvq_decode_attention and kvq_dequantize, and every length the
kernels need is read from the cache on the device, so a step (append one token,
decode, dequantize the newest page) can be captured once and replayed while the cache
grows underneath it.  A replay reuses the launch id of the captured decode call; the
stream count words are cleared by the CTA that merges, so each replay starts clean.

Checked after every replay, through the C-ABI: the cache bit-exact against the oracle
that appended the same tokens, the attention output bit-exact against an eager call on
the same cache and close to the fp64 oracle on the same codes, and the dequantized
newest page bit-exact against an eager call.
"""
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


@pytest.mark.parametrize("name,w,T0", [
    ("token-wise K4V2, split streams", wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8), 5000),
    ("channel-wise K4V2 with a tail", wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=8), 1000),
])
def test_step_captured_once_replays_while_the_cache_grows(kvq, name, w, T0):
    B, n_replays = 2, 4
    cap = ((T0 + n_replays + 2 + 127) // 128) * 128
    k, v = wl.make_kv(w, layer=3, tokens=T0 + n_replays + 1, batch=B)
    cfg, gc, oc = tl.build_both(kvq, w, k[:, :, :T0].contiguous(), v[:, :, :T0].contiguous(), [T0], cap)
    kb, vb = tl.bits_of(k), tl.bits_of(v)
    kd, vd = k.cuda(), v.cuda()
    q_all = [wl.make_q(w, layer=10 + i, batch=B).cuda() for i in range(n_replays + 1)]

    # static buffers of the captured step
    k_in = torch.empty((B, w.n_kv_heads, 1, w.head_dim), dtype=w.torch_dtype, device="cuda")
    v_in = torch.empty_like(k_in)
    q_in = torch.empty_like(q_all[0])
    out = torch.empty(tuple(q_in.shape), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device="cuda")
    deq_k = torch.zeros((B, w.n_kv_heads, cap, w.head_dim), dtype=w.torch_dtype, device="cuda")
    deq_v = torch.zeros_like(deq_k)
    page0 = (T0 // 128) * 128          # the page that holds every appended token of this test
    assert (T0 + n_replays + 1) <= page0 + 128

    def step():
        kvq.kvq_quantize_append(cfg, gc, k_in, v_in)
        kvq.kvq_decode_attention(cfg, gc, q_in, out, ws)
        kvq.kvq_dequantize(cfg, gc, deq_k, deq_v, page0, page0 + 128)

    def feed(i):
        k_in.copy_(kd[:, :, T0 + i:T0 + i + 1]); v_in.copy_(vd[:, :, T0 + i:T0 + i + 1]); q_in.copy_(q_all[i])
        oc.append(kb[:, :, T0 + i:T0 + i + 1], vb[:, :, T0 + i:T0 + i + 1])

    # one eager step first (one-time set-up of the kernels happens outside the capture)
    feed(0)
    step()
    torch.cuda.synchronize()
    tl.assert_caches_equal(gc, oc)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    feed(1)                             # the capture itself launches nothing: the first replay runs this step
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    assert int(gc.seq_len.max().item()) == T0 + 1, name      # capturing did not run the step

    for i in range(1, n_replays + 1):
        if i > 1:
            feed(i)
        graph.replay()
        torch.cuda.synchronize()
        assert kvq.kvq_check_status(gc) == 0, name
        tl.assert_caches_equal(gc, oc)
        got = out.double().cpu().numpy()
        eager = tl.gpu_decode(kvq, cfg, gc, q_in)
        assert np.array_equal(got, eager), f"{name}: replay {i} differs from an eager call on the same cache"
        want = tl.oracle_on_gpu_codes(gc, w).decode(tl.bits_of(q_in))
        tl.assert_attention_close(got, want)
        ek, ev = torch.zeros_like(deq_k), torch.zeros_like(deq_v)
        kvq.kvq_dequantize(cfg, gc, ek, ev, page0, page0 + 128)
        torch.cuda.synchronize()
        n = T0 + 1 + i
        assert torch.equal(deq_k[:, :, page0:n].view(torch.int16), ek[:, :, page0:n].view(torch.int16)), name
        assert torch.equal(deq_v[:, :, page0:n].view(torch.int16), ev[:, :, page0:n].view(torch.int16)), name


def test_caches_can_share_one_tensor_of_sequence_lengths(kvq):
    """Caller-owned length storage: two layers' caches keep their lengths in the rows of one tensor, so that one
    operation sets both; the library reads and bumps them there."""
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B, T = 2, 300
    lens = torch.full((2, B), 77, dtype=torch.int32, device="cuda")      # stale contents: the constructor zeroes its row
    cfg = tl.gpu_config_for(kvq, w, B, 384)
    caches = [kvq.Cache(cfg, seq_len=lens[i]) for i in range(2)]
    assert int(lens.abs().sum().item()) == 0
    k, v = wl.make_kv(w, layer=5, tokens=T, batch=B)
    oc = tl.oracle_cache_for(w, B, 384)
    oc.append(tl.bits_of(k), tl.bits_of(v))
    kvq.kvq_quantize_append(cfg, caches[0], k.cuda(), v.cuda())
    kvq.kvq_quantize_append(cfg, caches[1], k.cuda()[:, :, :100], v.cuda()[:, :, :100])
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [[T] * B, [100] * B]
    tl.assert_caches_equal(caches[0], oc)
    lens[:, :] = torch.tensor([[200] * B, [100] * B], dtype=torch.int32)    # one operation sets both rows: layer 0 rewinds to 200 tokens
    q = wl.make_q(w, layer=5, batch=B).cuda()
    got = tl.gpu_decode(kvq, cfg, caches[0], q)
    want = tl.oracle_on_gpu_codes(caches[0], w).decode(tl.bits_of(q))
    tl.assert_attention_close(got, want)
