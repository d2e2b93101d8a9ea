"""Several causal query rows per head (kvq_decode_attention_rows) through the C-ABI against the fp64 oracle on the
same codes: the rows are the queries of the last R cached tokens, row r sees the tokens up to its own position."""
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


def make_q_rows(w, B, R, seed):
    g = torch.Generator().manual_seed(4242 + seed)
    return torch.randn((B, R, w.n_q_heads, w.head_dim), generator=g).to(w.torch_dtype)


def decode_rows(kvq, cfg, gc, q):
    R = q.shape[1]
    ws = torch.empty(max(16, kvq.kvq_workspace_bytes_rows(cfg, R)), dtype=torch.uint8, device="cuda")
    out = torch.full(tuple(q.shape), float("nan"), dtype=torch.float32, device="cuda")
    kvq.kvq_decode_attention_rows(cfg, gc, q.cuda(), out, ws)
    torch.cuda.synchronize()
    assert kvq.kvq_check_status(gc) == 0
    return out.double().cpu().numpy()


CASES = {
    "8b-g4-r2": (wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8), 2, 2, 128 * 5 + 3),
    "8b-g2-r4": (wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=4), 1, 4, 128 * 4),          # rows reach back over a page end
    "8b-g1-r8": (wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=2), 1, 8, 700),
    "8b-g2-r2-k8v4": (wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=4, kb=8, vb=4), 1, 2, 700),
    "8b-g4-r1": (wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8), 2, 1, 300),
    "14b-chan-g2-r2-tail": (wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=4), 2, 2, 128 * 3 + 50),
    "14b-chan-g2-r2-tail1": (wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=4), 1, 2, 128 * 2 + 1),
    "1b-d64-g2-r2": (wl.LLAMA_1B.with_(n_kv_heads=2, n_q_heads=4), 2, 2, 333),
    "70b-g8-r1": (wl.LLAMA_70B.with_(n_kv_heads=2, n_q_heads=16), 1, 1, 500),
}


@pytest.mark.parametrize("name", list(CASES))
def test_rows_match_the_oracle(kvq, name):
    w, B, R, T = CASES[name]
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cap = ((T + 127) // 128) * 128
    cfg, gc, _ = tl.build_both(kvq, w, k, v, [T], cap)
    q = make_q_rows(w, B, R, len(name))
    want = tl.oracle_on_gpu_codes(gc, w).decode_rows(tl.bits_of(q))
    got = decode_rows(kvq, cfg, gc, q)
    tl.assert_attention_close(got, want)
    if R == 1:      # one row is the plain decode step, bit for bit
        assert np.array_equal(got[:, 0], tl.gpu_decode(kvq, cfg, gc, q[:, 0].contiguous()))


def test_rows_with_ragged_and_too_short_sequences(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    B, R, cap = 4, 2, 512
    k, v = wl.make_kv(w, tokens=cap, batch=B)
    cfg, gc, oc = tl.build_both(kvq, w, k, v, [cap], cap)
    lens = [0, 1, 129, 400]                                 # no token, fewer tokens than rows, a page edge, ragged
    gc.seq_len.copy_(torch.tensor(lens, dtype=torch.int32))
    oc.seq_len[:] = lens
    q = make_q_rows(w, B, R, 9)
    got = decode_rows(kvq, cfg, gc, q)
    want = oc.decode_rows(tl.bits_of(q))
    tl.assert_attention_close(got, want)
    assert not got[0].any() and not got[1, 0].any() and got[1, 1].any()


def test_too_many_rows_are_rejected(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    cfg = tl.gpu_config_for(kvq, w, 1, 128)
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_workspace_bytes_rows(cfg, 3)                # 3 rows x 4 heads > 8 columns
    assert e.value.code == -2
    # K8V4 is served with up to 4 (row, head) pairs per KV head only
    w2 = w.with_(kb=8, vb=4)
    cfg2 = tl.gpu_config_for(kvq, w2, 1, 128)
    gc = kvq.Cache(cfg2)
    q = torch.zeros((1, 2, 8, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 2, 8, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(kvq.kvq_workspace_bytes_rows(cfg2, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_decode_attention_rows(cfg2, gc, q, out, ws)
    assert e.value.code == -2
