"""Key-only randomized Hadamard rotation (Sec. 4.4) through the CUDA library: rotated keys are quantized bit for
bit like the oracle's, dequantize rotates back bit-exactly, decode rotates q and stays within tolerance."""
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


def signs_for(D, seed):
    return np.random.default_rng(seed).choice([-1, 1], D).astype(np.int8)


CASES = {
    "8b-k4v2": (wl.LLAMA_8B, 2, 700, [571, 128, 1]),
    "8b-k2v4": (wl.LLAMA_8B.with_(kb=2, vb=4), 1, 300, [300]),
    "8b-k8v4": (wl.LLAMA_8B.with_(kb=8, vb=4), 1, 300, [300]),
    "8b-g32": (wl.LLAMA_8B.with_(gk=32), 1, 260, [260]),
    "14b-k4v2": (wl.SHAPED_14B, 2, 128 * 2 + 63, [100, 219]),
    "14b-k8v2": (wl.SHAPED_14B.with_(kb=8), 1, 128 * 2 + 127, [383]),
    "1b": (wl.LLAMA_1B, 2, 333, [200, 133]),
    "tiny": (wl.TINY, 1, 512, [512]),
}


@pytest.mark.parametrize("name", list(CASES))
def test_rotated_keys_parity(kvq, name):
    w, B, T, chunks = CASES[name]
    hk = min(w.n_kv_heads, 2) if name != "tiny" else w.n_kv_heads
    w = w.with_(n_kv_heads=hk, n_q_heads=hk * (w.n_q_heads // w.n_kv_heads))
    cap = ((T + 127) // 128) * 128 + 128
    s = signs_for(w.head_dim, 11)
    k, v = wl.make_kv(w, tokens=T, batch=B)
    cfg, gc, oc = tl.build_both(kvq, w, k, v, chunks, cap, k_signs=s)
    assert kvq.kvq_check_status(gc) == 0
    tl.assert_caches_equal(gc, oc)
    ko = torch.zeros((B, w.n_kv_heads, cap, w.head_dim), dtype=w.torch_dtype, device="cuda")
    vo = torch.zeros_like(ko)
    kvq.kvq_dequantize(cfg, gc, ko, vo, 0, cap)
    kr = np.zeros((B, w.n_kv_heads, cap, w.head_dim), np.uint16)
    vr = np.zeros_like(kr)
    oc.dequantize(kr, vr, 0, cap)
    assert np.array_equal(tl.bits_of(ko), kr)
    assert np.array_equal(tl.bits_of(vo), vr)
    oc2 = tl.oracle_on_gpu_codes(gc, w)
    for variant in ("normal", "large", "peaked"):
        q = wl.make_q(w, batch=B, variant=variant, k=k)
        tl.assert_attention_close(tl.gpu_decode(kvq, cfg, gc, q), oc2.decode(tl.bits_of(q)))


def test_rotation_lowers_attention_error_on_outlier_keys(kvq):
    """Keys with 8 heavy channels per head: rotating them before 4-bit quantization lowers the error of the
    attention output against exact attention on the unquantized cache (Sec. 4.4, key-only rotation)."""
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8)
    e_rot, e_plain = [], []
    for seed in range(4):
        k, v = wl.make_kv(w, layer=seed, tokens=512, batch=1)
        q = wl.make_q(w, layer=seed, batch=1)
        logits = torch.einsum("bhd,bhtd->bht", q.double(), k.double().repeat_interleave(4, 1)) / np.sqrt(128)
        exact = torch.einsum("bht,bhtd->bhd", torch.softmax(logits, -1), v.double().repeat_interleave(4, 1)).numpy()
        for acc, sg in ((e_rot, signs_for(128, seed)), (e_plain, None)):
            cfg, gc, _ = tl.build_both(kvq, w, k, v, [512], 512, k_signs=sg)
            got = tl.gpu_decode(kvq, cfg, gc, q)
            acc.append(np.linalg.norm(got - exact) / np.linalg.norm(exact))
    assert np.mean(e_rot) < np.mean(e_plain)


def test_rotation_needs_quantized_keys(kvq):
    w = wl.LLAMA_8B.with_(n_kv_heads=2, n_q_heads=8, kb=16)
    cfg = tl.gpu_config_for(kvq, w, 1, 128)
    gc = kvq.Cache(cfg, k_signs=torch.ones(128, dtype=torch.int8))
    k, v = wl.make_kv(w, tokens=8, batch=1)
    with pytest.raises(kvq.KvqError) as e:
        kvq.kvq_quantize_append(cfg, gc, k.cuda(), v.cuda())
    assert e.value.code == -2
