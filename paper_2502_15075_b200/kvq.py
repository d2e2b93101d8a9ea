"""ctypes binding of libkvq.so: the same names as the C-ABI, argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in
the library's CUDA kernels.  Importing this module fails loudly when the
library has not been built (`python -m paper_2502_15075_b200.build`): there is
no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("KVQ_LIB_PATH") or os.path.join(_HERE, "libkvq.so")   # override: load another build

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_15075_b200.build` "
                      "(there is no fallback path)")
_lib = ctypes.CDLL(LIB_PATH)

KVQ_FP16, KVQ_BF16, KVQ_FP32 = 0, 1, 2
PAGE_TOKENS = 128
STATUS_CAPACITY, STATUS_DEVICE_TIMEOUT = 1, 2


class kvq_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "kb", "vb", "gk", "gv", "k_axis", "in_dtype",
        "capacity_tokens", "residual_tokens")]


class kvq_cache(ctypes.Structure):
    _fields_ = [("pages", ctypes.c_void_p), ("k_tail", ctypes.c_void_p),
                ("seq_len", ctypes.c_void_p), ("status", ctypes.c_void_p), ("k_signs", ctypes.c_void_p),
                ("kv_win", ctypes.c_void_p)]


_P = ctypes.POINTER
_lib.kvq_layout_version.restype = ctypes.c_int
_lib.kvq_page_bytes.argtypes = [_P(kvq_config), _P(ctypes.c_size_t)]
_lib.kvq_cache_bytes.argtypes = [_P(kvq_config), _P(ctypes.c_size_t), _P(ctypes.c_size_t)]
_lib.kvq_workspace_bytes.argtypes = [_P(kvq_config), _P(ctypes.c_size_t)]
_lib.kvq_window_bytes.argtypes = [_P(kvq_config), _P(ctypes.c_size_t)]
_lib.kvq_window_bytes.restype = ctypes.c_int
_lib.kvq_quantize_append.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p]
_lib.kvq_decode_attention.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                      ctypes.c_void_p]
_lib.kvq_decode_attention_static.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                             ctypes.c_int32, ctypes.c_float, ctypes.c_void_p]
_lib.kvq_dequantize.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p]
_lib.kvq_quant_error.argtypes = [_P(kvq_config), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                 ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
_lib.kvq_bit_balance.argtypes = [ctypes.c_double, ctypes.c_double, _P(ctypes.c_double)]
_lib.kvq_workspace_bytes_rows.argtypes = [_P(kvq_config), ctypes.c_int32, _P(ctypes.c_size_t)]
_lib.kvq_decode_attention_rows.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_int32,
                                           ctypes.c_void_p, ctypes.c_int32, ctypes.c_float, ctypes.c_void_p,
                                           ctypes.c_size_t, ctypes.c_void_p]
_lib.kvq_debug_decode_generic.argtypes = _lib.kvq_decode_attention.argtypes
_lib.kvq_debug_decode_stall.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                        ctypes.c_int64, ctypes.c_uint32, ctypes.c_void_p]
_lib.kvq_debug_decode_impl.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p,
                                       ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                       ctypes.c_int32, ctypes.c_void_p]
_lib.kvq_debug_decode_stall_impl.argtypes = [_P(kvq_config), _P(kvq_cache), ctypes.c_void_p, ctypes.c_void_p,
                                             ctypes.c_int32, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                             ctypes.c_int64, ctypes.c_uint32, ctypes.c_int32, ctypes.c_void_p]
_lib.kvq_check_status.argtypes = [_P(kvq_cache), ctypes.c_void_p]
_lib.kvq_strerror.argtypes = [ctypes.c_int]
_lib.kvq_strerror.restype = ctypes.c_char_p
for _f in ("kvq_page_bytes", "kvq_cache_bytes", "kvq_workspace_bytes", "kvq_quantize_append",
           "kvq_decode_attention", "kvq_decode_attention_static", "kvq_dequantize", "kvq_check_status",
           "kvq_quant_error", "kvq_bit_balance", "kvq_debug_decode_generic", "kvq_debug_decode_stall",
           "kvq_debug_decode_impl", "kvq_debug_decode_stall_impl", "kvq_workspace_bytes_rows", "kvq_decode_attention_rows"):
    getattr(_lib, _f).restype = ctypes.c_int

EXPORTS = ("kvq_layout_version", "kvq_page_bytes", "kvq_cache_bytes", "kvq_workspace_bytes",
           "kvq_quantize_append", "kvq_decode_attention", "kvq_decode_attention_static", "kvq_dequantize",
           "kvq_check_status", "kvq_strerror", "kvq_quant_error", "kvq_bit_balance", "kvq_workspace_bytes_rows",
           "kvq_decode_attention_rows", "kvq_window_bytes")
STATIC_SCRATCH_BYTES = 8 << 20


class KvqError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {_lib.kvq_strerror(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != 0:
        raise KvqError(code, where)


def _dtype_code(dt: torch.dtype) -> int:
    return {torch.float16: KVQ_FP16, torch.bfloat16: KVQ_BF16, torch.float32: KVQ_FP32}[dt]


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def kvq_strerror(code: int) -> str:
    return _lib.kvq_strerror(code).decode()


def kvq_layout_version() -> int:
    return _lib.kvq_layout_version()


def make_config(batch, n_q_heads, n_kv_heads, head_dim, kb, vb, gk, gv, k_axis, dtype, capacity_tokens,
                residual_tokens=0) -> kvq_config:
    code = _dtype_code(dtype) if isinstance(dtype, torch.dtype) else {"fp16": 0, "bf16": 1}[dtype]
    return kvq_config(batch, n_q_heads, n_kv_heads, head_dim, kb, vb, gk, gv, k_axis, code, capacity_tokens,
                      residual_tokens)


def kvq_window_bytes(cfg: kvq_config) -> int:
    out = ctypes.c_size_t()
    _check(_lib.kvq_window_bytes(ctypes.byref(cfg), ctypes.byref(out)), "kvq_window_bytes")
    return out.value


def kvq_page_bytes(cfg: kvq_config) -> int:
    out = ctypes.c_size_t()
    _check(_lib.kvq_page_bytes(ctypes.byref(cfg), ctypes.byref(out)), "kvq_page_bytes")
    return out.value


def kvq_cache_bytes(cfg: kvq_config):
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    _check(_lib.kvq_cache_bytes(ctypes.byref(cfg), ctypes.byref(a), ctypes.byref(b)), "kvq_cache_bytes")
    return a.value, b.value


def kvq_workspace_bytes(cfg: kvq_config) -> int:
    out = ctypes.c_size_t()
    _check(_lib.kvq_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)), "kvq_workspace_bytes")
    return out.value


class Cache:
    """Caller-owned buffers of one layer's packed cache (torch tensors) plus the POD handed to the library."""

    def __init__(self, cfg: kvq_config, device="cuda", k_signs: Optional[torch.Tensor] = None,
                 seq_len: Optional[torch.Tensor] = None):
        """k_signs: optional int8 tensor [head_dim] of +1 / -1: rotate the keys (randomized Hadamard).
        seq_len: optional caller-owned storage of the sequence lengths, a contiguous int32 CUDA tensor [batch]
        (e.g. a row of one [layers, batch] tensor, so that all layers' lengths can be set by one operation); it
        is zeroed here."""
        self.cfg = cfg
        self.k_signs = None if k_signs is None else k_signs.to(device=device, dtype=torch.int8).contiguous()
        assert self.k_signs is None or self.k_signs.numel() == cfg.head_dim
        pages_bytes, tail_bytes = kvq_cache_bytes(cfg)
        self.pages = torch.zeros(pages_bytes, dtype=torch.uint8, device=device)
        self.k_tail = torch.zeros(tail_bytes // 2, dtype=torch.float16, device=device) if tail_bytes else None
        if seq_len is None:
            self.seq_len = torch.zeros(cfg.batch, dtype=torch.int32, device=device)
        else:
            assert seq_len.is_cuda and seq_len.dtype == torch.int32 and seq_len.is_contiguous()
            assert tuple(seq_len.shape) == (cfg.batch,)
            self.seq_len = seq_len.zero_()
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        win_bytes = kvq_window_bytes(cfg)
        self.kv_win = torch.zeros(win_bytes // 2, dtype=torch.int16, device=device) if win_bytes else None
        self.c = kvq_cache(self.pages.data_ptr(), self.k_tail.data_ptr() if self.k_tail is not None else None,
                           self.seq_len.data_ptr(), self.status.data_ptr(),
                           self.k_signs.data_ptr() if self.k_signs is not None else None,
                           self.kv_win.data_ptr() if self.kv_win is not None else None)

    def pages_view(self) -> torch.Tensor:
        c = self.cfg
        return self.pages.view(c.batch, c.n_kv_heads, c.capacity_tokens // PAGE_TOKENS, -1)

    def window_view(self) -> Optional[torch.Tensor]:
        """int16 [B, Hkv, R, 2, D] bit patterns of the residual window, or None."""
        c = self.cfg
        return None if self.kv_win is None else self.kv_win.view(c.batch, c.n_kv_heads, c.residual_tokens, 2, c.head_dim)

    def tail_view(self) -> Optional[torch.Tensor]:
        c = self.cfg
        return None if self.k_tail is None else self.k_tail.view(c.batch, c.n_kv_heads, PAGE_TOKENS, c.head_dim)


def kvq_quantize_append(cfg: kvq_config, cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None):
    """k_new, v_new: CUDA tensors [B, Hkv, t_new, D] of the config's dtype, last dim contiguous,
    identical strides."""
    assert k_new.is_cuda and v_new.is_cuda and k_new.shape == v_new.shape and k_new.dim() == 4
    assert k_new.stride() == v_new.stride() and k_new.stride(3) == 1
    assert _dtype_code(k_new.dtype) == cfg.in_dtype and v_new.dtype == k_new.dtype
    assert k_new.shape[0] == cfg.batch and k_new.shape[1] == cfg.n_kv_heads and k_new.shape[3] == cfg.head_dim
    _check(_lib.kvq_quantize_append(ctypes.byref(cfg), ctypes.byref(cache.c), k_new.data_ptr(), v_new.data_ptr(),
                                    k_new.stride(0), k_new.stride(1), k_new.stride(2), k_new.shape[2],
                                    _stream_ptr(stream)), "kvq_quantize_append")


def kvq_decode_attention(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                         workspace: torch.Tensor, softmax_scale: float = 0.0,
                         stream: Optional[torch.cuda.Stream] = None):
    """q [B, Hq, D] (config dtype), out [B, Hq, D] (fp16/bf16/fp32), workspace: uint8 CUDA tensor of at
    least kvq_workspace_bytes(cfg)."""
    assert q.is_cuda and out.is_cuda and workspace.is_cuda and q.is_contiguous() and out.is_contiguous()
    assert tuple(q.shape) == (cfg.batch, cfg.n_q_heads, cfg.head_dim) and out.shape == q.shape
    assert _dtype_code(q.dtype) == cfg.in_dtype
    _check(_lib.kvq_decode_attention(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), out.data_ptr(),
                                     _dtype_code(out.dtype), float(softmax_scale), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "kvq_decode_attention")


def kvq_decode_attention_static(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                                softmax_scale: float = 0.0, stream: Optional[torch.cuda.Stream] = None):
    """kvq_decode_attention without a workspace argument, for callers that may not allocate device memory
    (an engine whose arena owns all of HBM, a plug-in that only receives input/output pointers): the split
    partials go to an 8 MiB buffer inside the library.  Raises KvqError(-8) when the configuration needs
    more than that.  Calls that can overlap on the GPU must not share a device: they would race on the
    buffer.  The first call on a device resolves the buffer's address; do it before any stream capture."""
    assert q.is_cuda and out.is_cuda and q.is_contiguous() and out.is_contiguous()
    assert tuple(q.shape) == (cfg.batch, cfg.n_q_heads, cfg.head_dim) and out.shape == q.shape
    assert _dtype_code(q.dtype) == cfg.in_dtype
    _check(_lib.kvq_decode_attention_static(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), out.data_ptr(),
                                            _dtype_code(out.dtype), float(softmax_scale), _stream_ptr(stream)),
           "kvq_decode_attention_static")


def kvq_dequantize(cfg: kvq_config, cache: Cache, k_out: Optional[torch.Tensor], v_out: Optional[torch.Tensor],
                   t_begin: int, t_end: int, stream: Optional[torch.cuda.Stream] = None):
    """k_out, v_out: [B, Hkv, capacity, D] contiguous CUDA tensors of the config dtype (or None)."""
    for t in (k_out, v_out):
        if t is not None:
            assert t.is_cuda and t.is_contiguous() and _dtype_code(t.dtype) == cfg.in_dtype
            assert tuple(t.shape) == (cfg.batch, cfg.n_kv_heads, cfg.capacity_tokens, cfg.head_dim)
    _check(_lib.kvq_dequantize(ctypes.byref(cfg), ctypes.byref(cache.c),
                               k_out.data_ptr() if k_out is not None else None,
                               v_out.data_ptr() if v_out is not None else None,
                               t_begin, t_end, _stream_ptr(stream)), "kvq_dequantize")


def kvq_quant_error(cfg: kvq_config, k: torch.Tensor, v: torch.Tensor, sums: torch.Tensor,
                    stream: Optional[torch.cuda.Stream] = None):
    """k, v: CUDA tensors [B, Hkv, T, D] of the config's dtype (last dim contiguous, identical strides);
    sums: CUDA float64 [B, Hkv, 4], added to: (sum k^2, sum (k - k^)^2, sum v^2, sum (v - v^)^2)."""
    assert k.is_cuda and v.is_cuda and k.shape == v.shape and k.dim() == 4 and k.stride() == v.stride()
    assert k.stride(3) == 1 and _dtype_code(k.dtype) == cfg.in_dtype and v.dtype == k.dtype
    assert sums.is_cuda and sums.dtype == torch.float64 and sums.is_contiguous()
    assert tuple(sums.shape) == (cfg.batch, cfg.n_kv_heads, 4) and k.shape[0] == cfg.batch and k.shape[1] == cfg.n_kv_heads
    _check(_lib.kvq_quant_error(ctypes.byref(cfg), k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2),
                                k.shape[2], sums.data_ptr(), _stream_ptr(stream)), "kvq_quant_error")


def kvq_bit_balance(sum_k2: float, sum_v2: float) -> float:
    out = ctypes.c_double()
    _check(_lib.kvq_bit_balance(float(sum_k2), float(sum_v2), ctypes.byref(out)), "kvq_bit_balance")
    return out.value


def kvq_workspace_bytes_rows(cfg: kvq_config, n_rows: int) -> int:
    out = ctypes.c_size_t()
    _check(_lib.kvq_workspace_bytes_rows(ctypes.byref(cfg), int(n_rows), ctypes.byref(out)), "kvq_workspace_bytes_rows")
    return out.value


def kvq_decode_attention_rows(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                              workspace: torch.Tensor, softmax_scale: float = 0.0,
                              stream: Optional[torch.cuda.Stream] = None):
    """q, out [B, R, Hq, D]: R causal query rows for the last R cached tokens of every sequence."""
    assert q.is_cuda and out.is_cuda and q.is_contiguous() and out.is_contiguous() and q.dim() == 4
    assert (q.shape[0], q.shape[2], q.shape[3]) == (cfg.batch, cfg.n_q_heads, cfg.head_dim) and out.shape == q.shape
    assert _dtype_code(q.dtype) == cfg.in_dtype
    _check(_lib.kvq_decode_attention_rows(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), q.shape[1],
                                          out.data_ptr(), _dtype_code(out.dtype), float(softmax_scale),
                                          workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                          _stream_ptr(stream)), "kvq_decode_attention_rows")


def kvq_debug_decode_generic(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                             workspace: torch.Tensor, softmax_scale: float = 0.0):
    """Test hook: kvq_decode_attention through the plain-ALU kernel whatever the configuration."""
    _check(_lib.kvq_debug_decode_generic(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), out.data_ptr(),
                                         _dtype_code(out.dtype), float(softmax_scale), workspace.data_ptr(),
                                         workspace.numel() * workspace.element_size(), _stream_ptr(None)),
           "kvq_debug_decode_generic")


IMPL_AUTO, IMPL_WARP_MMA, IMPL_TCGEN05 = 0, 1, 2


def kvq_debug_decode_impl(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                          workspace: torch.Tensor, impl: int, softmax_scale: float = 0.0,
                          stream: Optional[torch.cuda.Stream] = None):
    """Test / benchmark hook: decode through a chosen kernel of the fast path (IMPL_WARP_MMA, IMPL_TCGEN05).
    q, out [B, Hq, D] (one row) or [B, R, Hq, D]."""
    n_rows = q.shape[1] if q.dim() == 4 else 1
    _check(_lib.kvq_debug_decode_impl(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), int(n_rows),
                                      out.data_ptr(), _dtype_code(out.dtype), float(softmax_scale),
                                      workspace.data_ptr(), workspace.numel() * workspace.element_size(), int(impl),
                                      _stream_ptr(stream)), "kvq_debug_decode_impl")


def kvq_debug_decode_stall(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                           workspace: torch.Tensor, skip_page: int, wait_us: int):
    """Test hook: decode with one page copy withheld and every device-side wait limited to wait_us."""
    _check(_lib.kvq_debug_decode_stall(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), out.data_ptr(),
                                       _dtype_code(out.dtype), 0.0, workspace.data_ptr(),
                                       workspace.numel() * workspace.element_size(), int(skip_page), int(wait_us),
                                       _stream_ptr(None)), "kvq_debug_decode_stall")


def kvq_debug_decode_stall_impl(cfg: kvq_config, cache: Cache, q: torch.Tensor, out: torch.Tensor,
                                workspace: torch.Tensor, skip_page: int, wait_us: int, impl: int):
    """Test hook: kvq_debug_decode_stall through a chosen kernel of the fast path."""
    _check(_lib.kvq_debug_decode_stall_impl(ctypes.byref(cfg), ctypes.byref(cache.c), q.data_ptr(), out.data_ptr(),
                                            _dtype_code(out.dtype), 0.0, workspace.data_ptr(),
                                            workspace.numel() * workspace.element_size(), int(skip_page), int(wait_us),
                                            int(impl), _stream_ptr(None)), "kvq_debug_decode_stall_impl")


def kvq_check_status(cache: Cache, stream: Optional[torch.cuda.Stream] = None) -> int:
    """Synchronises the stream and returns the library's status code (0 = ok)."""
    return _lib.kvq_check_status(ctypes.byref(cache.c), _stream_ptr(stream))


# ----------------------------------------------------------------------------
# Host-buffer convenience calls: the same C-ABI entry points with the
# host<->device copies of the per-step tensors done around them.
# ----------------------------------------------------------------------------
def decode_attention_host(cfg: kvq_config, cache: Cache, q_host: torch.Tensor, out_host: torch.Tensor,
                          q_dev: torch.Tensor, out_dev: torch.Tensor, workspace: torch.Tensor,
                          softmax_scale: float = 0.0):
    """q_host (pinned) -> device, decode, out -> out_host (pinned).  Asynchronous on the current stream."""
    q_dev.copy_(q_host, non_blocking=True)
    kvq_decode_attention(cfg, cache, q_dev, out_dev, workspace, softmax_scale)
    out_host.copy_(out_dev, non_blocking=True)


def quantize_append_host(cfg: kvq_config, cache: Cache, k_host: torch.Tensor, v_host: torch.Tensor,
                         k_dev: torch.Tensor, v_dev: torch.Tensor):
    """Pinned host K/V -> device staging tensors -> quantize-append.  Asynchronous on the current stream."""
    k_dev.copy_(k_host, non_blocking=True)
    v_dev.copy_(v_host, non_blocking=True)
    kvq_quantize_append(cfg, cache, k_dev, v_dev)
