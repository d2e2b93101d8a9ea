"""Seeded synthetic KV-cache workloads.

This module only draws random tensors with the shapes and value structure of
the model-shaped caches the quantization study looks at (keys with larger
norms / outlier channels than values).  It holds none of the method's
arithmetic (no quantizer, no packing, no attention): both the CPU oracle's
tests and the CUDA path's tests/bench feed from it, and it imports neither.

All tensors are produced by a seeded ``torch.Generator`` on the requested
device and returned in the workload's 16-bit dtype:

    K, V : [batch, n_kv_heads, T, head_dim]
    q    : [batch, n_q_heads, head_dim]
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Tuple

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    recipe: str            # which value recipe below
    layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context: int
    dtype: str             # "fp16" | "bf16"
    kb: int
    vb: int
    gk: int
    gv: int
    k_axis: int = 0        # 0 per-token groups along head_dim, 1 per-channel over 128-token blocks
    number: int = 0        # 1-based position in the config list (seed base)

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five model-shaped configurations (shapes only; values come from `recipe`).
TINY = Workload("tiny", "outlier4", 1, 1, 8, 8, 64, 512, "fp16", 4, 2, 32, 32, 0, 1)
LLAMA_1B = Workload("llama-3.2-1b-shaped", "lognormal", 16, 8, 32, 8, 64, 4096, "fp16", 4, 2, 64, 64, 0, 2)
LLAMA_8B = Workload("llama-3.1-8b-shaped", "outlier8x10", 32, 16, 32, 8, 128, 32768, "bf16", 4, 2, 128, 128, 0, 3)
SHAPED_14B = Workload("14b-shaped", "student_t3", 40, 32, 40, 10, 128, 16384, "bf16", 4, 2, 128, 128, 1, 4)
LLAMA_70B = Workload("llama-3.3-70b-shaped", "rotated", 80, 4, 64, 8, 128, 131072, "bf16", 4, 2, 128, 128, 0, 5)

CONFIGS = (TINY, LLAMA_1B, LLAMA_8B, SHAPED_14B, LLAMA_70B)


def layer_seed(w: Workload, layer: int) -> int:
    return 1000 * w.number + layer


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_kv(w: Workload, layer: int = 0, device="cpu", tokens: Optional[int] = None,
            batch: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Draw K and V for one layer.  `tokens` / `batch` override the workload's
    context / batch (used by scaled-down parity cases)."""
    T = w.context if tokens is None else tokens
    B = w.batch if batch is None else batch
    H, D = w.n_kv_heads, w.head_dim
    g = _gen(device, layer_seed(w, layer))
    shape = (B, H, T, D)
    k = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    v = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    r = w.recipe
    if r == "outlier4":
        # 4 random outlier channels (same set for every head), keys x4 there
        ch = torch.randperm(D, generator=g, device=device)[:4]
        k[..., ch] *= 4.0
    elif r == "lognormal":
        # per (head, channel) magnitude ~ lognormal(0, 1); values sigma 0.5
        mag = torch.exp(torch.randn((1, H, 1, D), generator=g, device=device))
        k *= mag
        v *= 0.5
    elif r == "outlier8x10":
        # 8 heavy channels per head, keys x10 there
        for h in range(H):
            ch = torch.randperm(D, generator=g, device=device)[:8]
            kh = k[:, h]
            kh[..., ch] = kh[..., ch] * 10.0
    elif r == "student_t3":
        # Student-t with 3 degrees of freedom: z / sqrt(chi2_3 / 3)
        c = torch.zeros(shape, device=device, dtype=torch.float32)
        for _ in range(3):
            c += torch.randn(shape, generator=g, device=device).square_()
        k /= torch.sqrt(c / 3.0)
        del c
    elif r == "rotated":
        # scaled Gaussian through a random orthogonal matrix; norm 2-4x the values'
        a = torch.randn((D, D), generator=g, device=device, dtype=torch.float32)
        qmat, _ = torch.linalg.qr(a)
        c = 2.0 + 2.0 * torch.rand((), generator=g, device=device)
        k = (k @ qmat) * c
    elif r == "gauss":
        pass
    else:
        raise ValueError(f"unknown recipe {r}")
    return k.to(w.torch_dtype).contiguous(), v.to(w.torch_dtype).contiguous()


def make_q(w: Workload, layer: int = 0, device="cpu", batch: Optional[int] = None,
           variant: str = "normal", k: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Decode queries, one row per query head.

    variant: "normal" N(0,1); "large" 8 x N(0,1) (large logits);
             "peaked" a cached key plus 0.1 x noise (sharply peaked softmax; needs `k`).
    """
    B = w.batch if batch is None else batch
    g = _gen(device, layer_seed(w, layer) + 500)
    q = torch.randn((B, w.n_q_heads, w.head_dim), generator=g, device=device, dtype=torch.float32)
    if variant == "large":
        q *= 8.0
    elif variant == "peaked":
        assert k is not None
        G = w.n_q_heads // w.n_kv_heads
        T = k.shape[2]
        pick = torch.randint(0, T, (B, w.n_q_heads), generator=g, device=device)
        kv = torch.arange(w.n_q_heads, device=device) // G
        base = k.float()[torch.arange(B, device=device)[:, None], kv[None, :], pick]
        q = base + 0.1 * q
    elif variant != "normal":
        raise ValueError(variant)
    return q.to(w.torch_dtype).contiguous()


def ragged_seq_lens(w: Workload, T: int, batch: int, seed: int = 0) -> torch.Tensor:
    """seq_len[b] ~ U(T/2, T), int32, on the CPU."""
    g = _gen("cpu", 77_000 + 1000 * w.number + seed)
    lo = max(1, T // 2)
    return torch.randint(lo, T + 1, (batch,), generator=g, dtype=torch.int32)


def packed_bytes_per_token(w: Workload) -> float:
    """Packed K + V code bytes plus fp16 (scale, zero) metadata per token per KV head."""
    D = w.head_dim
    kmeta = 4.0 * D / 128 if w.k_axis == 1 else 4.0 * D / w.gk
    if w.kb == 16:
        kmeta = 0.0
    vmeta = 0.0 if w.vb == 16 else 4.0 * D / w.gv
    return D * w.kb / 8 + D * w.vb / 8 + kmeta + vmeta
