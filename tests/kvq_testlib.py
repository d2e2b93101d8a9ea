"""Shared helpers for the parity tests: build the same cache through the CUDA
library and through the CPU oracle, and compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle.cache import OracleCache
from paper_2502_15075_b200 import workloads as wl

REL_L2_TOL = 2e-3     # attention output vs fp64 oracle on the same codes
MAX_ABS_TOL = 1e-2


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def oracle_cache_for(w: wl.Workload, batch: int, capacity: int, k_signs=None, residual=0) -> OracleCache:
    return OracleCache(batch, w.n_kv_heads, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis, w.dtype, capacity,
                       k_signs=k_signs, residual=residual)


def gpu_config_for(kvq, w: wl.Workload, batch: int, capacity: int, residual=0):
    return kvq.make_config(batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis,
                           w.torch_dtype, capacity, residual)


def build_both(kvq, w: wl.Workload, k: torch.Tensor, v: torch.Tensor, chunks, capacity: int, k_signs=None,
               residual=0):
    """Append k, v ([B,Hkv,T,D] CPU tensors) in the given chunk sizes through both paths.
    k_signs: optional +-1 per channel (numpy int8): rotate the keys on both sides."""
    B = k.shape[0]
    cfg = gpu_config_for(kvq, w, B, capacity, residual)
    gc = kvq.Cache(cfg, k_signs=None if k_signs is None else torch.from_numpy(k_signs))
    oc = oracle_cache_for(w, B, capacity, k_signs, residual)
    kd, vd = k.cuda(), v.cuda()
    kb_, vb_ = bits_of(k), bits_of(v)
    t = 0
    for n in chunks:
        kvq.kvq_quantize_append(cfg, gc, kd[:, :, t:t + n], vd[:, :, t:t + n])
        oc.append(kb_[:, :, t:t + n], vb_[:, :, t:t + n])
        t += n
    torch.cuda.synchronize()
    return cfg, gc, oc


def assert_caches_equal(gc, oc: OracleCache):
    """Bit-exact comparison of packed pages, metadata, tail and sequence lengths."""
    assert np.array_equal(gc.seq_len.cpu().numpy(), oc.seq_len)
    gp = gc.pages_view().cpu().numpy()
    if not np.array_equal(gp, oc.pages):
        bad = np.argwhere(gp != oc.pages)
        raise AssertionError(f"packed pages differ at {len(bad)} bytes, first (b,h,page,byte) = {bad[0].tolist()}: "
                             f"gpu {gp[tuple(bad[0])]} oracle {oc.pages[tuple(bad[0])]}")
    if oc.k_tail is not None:
        gt = gc.tail_view().cpu().view(torch.int16).numpy().view(np.uint16)
        for b in range(oc.B):
            r = int(oc.seq_len[b]) % 128
            assert np.array_equal(gt[b, :, :r], oc.k_tail[b, :, :r]), "fp16 tail differs"
    if oc.R:
        gw = gc.window_view().cpu().numpy().view(np.uint16)
        for b in range(oc.B):
            n = int(oc.seq_len[b])
            slots = np.arange(oc.flushed(b), n) % oc.R
            assert np.array_equal(gw[b][:, slots], oc.kv_win[b][:, slots]), "residual window differs"


def oracle_on_gpu_codes(gc, w: wl.Workload) -> OracleCache:
    """An oracle cache that holds exactly the bytes the GPU produced (attention parity is measured on the
    same codes)."""
    cfg = gc.cfg
    oc = oracle_cache_for(w, cfg.batch, cfg.capacity_tokens,
                          None if gc.k_signs is None else gc.k_signs.cpu().numpy(), cfg.residual_tokens)
    oc.pages = gc.pages_view().cpu().numpy().copy()
    if oc.R:
        oc.kv_win = gc.window_view().cpu().numpy().view(np.uint16).copy()
    if oc.k_tail is not None:
        oc.k_tail = gc.tail_view().cpu().view(torch.int16).numpy().view(np.uint16).copy()
    oc.seq_len = gc.seq_len.cpu().numpy().copy()
    return oc


def gpu_decode(kvq, cfg, gc, q: torch.Tensor, out_dtype=torch.float32, scale: float = 0.0) -> np.ndarray:
    ws = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device="cuda")
    out = torch.full(tuple(q.shape), float("nan"), dtype=out_dtype, device="cuda")
    kvq.kvq_decode_attention(cfg, gc, q.cuda(), out, ws, scale)
    torch.cuda.synchronize()
    assert kvq.kvq_check_status(gc) == 0
    return out.double().cpu().numpy()


def assert_attention_close(got: np.ndarray, want: np.ndarray, rel=REL_L2_TOL, mabs=MAX_ABS_TOL):
    assert np.all(np.isfinite(got))
    den = np.linalg.norm(want)
    rl2 = np.linalg.norm(got - want) / (den if den > 0 else 1.0)
    ma = np.abs(got - want).max()
    assert rl2 <= rel and ma <= mabs, f"attention mismatch: rel-L2 {rl2:.3e} (tol {rel}), max-abs {ma:.3e} (tol {mabs})"
    return rl2, ma
