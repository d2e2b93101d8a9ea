"""kvq_quant_error through the C-ABI against the fp64 oracle: sum x^2 and sum (x - x^)^2 per (batch, kv-head)
for keys and values on the five model-shaped recipes (scaled-down token counts), within 1e-5 relative."""
import numpy as np
import pytest
import torch

from oracle import error as oe
from paper_2502_15075_b200 import workloads as wl

import kvq_testlib as tl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kvq():
    from paper_2502_15075_b200 import build
    build.build()
    from paper_2502_15075_b200 import kvq as mod
    return mod


CASES = {
    "tiny": (wl.TINY, 1, 512),
    "1b": (wl.LLAMA_1B, 2, 300),
    "8b-k4v2": (wl.LLAMA_8B, 2, 333),
    "8b-k2v4": (wl.LLAMA_8B.with_(kb=2, vb=4), 1, 200),
    "8b-k8v4-g32": (wl.LLAMA_8B.with_(kb=8, vb=4, gk=32, gv=64), 1, 200),
    "14b-tokenwise": (wl.SHAPED_14B.with_(k_axis=0), 1, 257),
    "70b": (wl.LLAMA_70B, 1, 400),
    "16bit-keys": (wl.LLAMA_8B.with_(kb=16), 1, 100),
    "8b-k3v3": (wl.LLAMA_8B.with_(kb=3, vb=3), 1, 200),        # Table 1's middle column
    "8b-k6v1": (wl.LLAMA_8B.with_(kb=6, vb=1), 1, 200),
}


@pytest.mark.parametrize("name", list(CASES))
def test_error_sums_match_the_oracle(kvq, name):
    w, B, T = CASES[name]
    w = w.with_(n_kv_heads=2, n_q_heads=2 * (w.n_q_heads // w.n_kv_heads)) if name != "tiny" else w
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg = tl.gpu_config_for(kvq, w, B, 128)
    sums = torch.zeros((B, w.n_kv_heads, 4), dtype=torch.float64, device="cuda")
    # in two chunks: the call accumulates
    cut = T // 3
    kd, vd = k.cuda(), v.cuda()
    kvq.kvq_quant_error(cfg, kd[:, :, :cut], vd[:, :, :cut], sums)
    kvq.kvq_quant_error(cfg, kd[:, :, cut:], vd[:, :, cut:], sums)
    torch.cuda.synchronize()
    want = oe.quant_error_sums(tl.bits_of(k), tl.bits_of(v), w.dtype, w.kb, w.vb, w.gk, w.gv)
    got = sums.cpu().numpy()
    assert np.allclose(got, want, rtol=1e-5, atol=0.0), np.abs(got / np.where(want == 0, 1, want) - 1).max()


def test_keys_err_more_than_values_and_balance_favours_keys(kvq):
    """Table-1-style ratio on the 8B-shaped recipe: at equal bits the key cache (outlier channels, larger
    norm) has the larger MSE, and the balanced allocation gives keys more bits (Theorem 2 / App. B.4)."""
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8, kb=4, vb=4)
    k, v = wl.make_kv(w, tokens=512, batch=2)
    cfg = tl.gpu_config_for(kvq, w, 2, 128)
    sums = torch.zeros((2, 2, 4), dtype=torch.float64, device="cuda")
    kvq.kvq_quant_error(cfg, k.cuda(), v.cuda(), sums)
    s = sums.sum(dim=(0, 1)).cpu().numpy()
    assert s[1] > 4 * s[3]
    delta = kvq.kvq_bit_balance(s[0], s[2])
    assert delta > 0.5 and abs(delta - oe.bit_balance(s[0], s[2])) < 1e-12


def test_channel_wise_keys_are_rejected(kvq):
    w = wl.SHAPED_14B.with_(n_kv_heads=2, n_q_heads=8)
    k, v = wl.make_kv(w, tokens=16, batch=1)
    cfg = tl.gpu_config_for(kvq, w, 1, 128)
    sums = torch.zeros((1, 2, 4), dtype=torch.float64, device="cuda")
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_quant_error(cfg, k.cuda(), v.cuda(), sums)
    assert e.value.code == -2
