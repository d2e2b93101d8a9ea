"""Oracle packed KV cache: append, dequantize, decode (test infrastructure).

Mirrors the semantics of the library's three calls on NumPy arrays so that the
tests can compare bytes and values one by one:

* append: V is quantized token-wise at once.  K is quantized token-wise at once
  (k_axis 0), or channel-wise per 128-token block (k_axis 1): tokens first go to
  an fp16 residual tail (Sec. 4.1: recent tokens stay in full precision and are
  flushed periodically); when the block is complete it is quantized with one
  group per channel and written to its page.
* residual window (Sec. 4.1: "a 64-token residual buffer, which stores the most recent tokens in full precision
  before being periodically flushed"; token-wise keys only): with residual = R > 0 the newest seq_len mod R tokens
  of K and V stay as their 16-bit inputs in a ring of R slots (token t in slot t mod R); whenever R of them are
  complete they are quantized as a block and move to the pages.  Reading: the flush is block-aligned, so the
  window holds 0 .. R-1 tokens.
* dequantize: xhat = fmaf(code, scale, zero) rounded to the 16-bit input type.
* decode: fp64 attention (App. A.1) over z + s*code exactly, the tail as stored.
"""
from __future__ import annotations

import numpy as np

from . import attention, layout, quantizer
from .layout import PAGE_TOKENS, Layout

ERR_CAPACITY_BIT = 1


class OracleCache:
    def __init__(self, batch, n_kv_heads, head_dim, kb, vb, gk, gv, k_axis, dtype, capacity_tokens, k_signs=None,
                 residual=0):
        """k_signs: None, or +-1 per channel: keys are rotated by the randomized Hadamard transform
        y = H (signs * x) / sqrt(D) before quantization (Sec. 4.4, key-only rotation); queries get the same
        rotation at decode time and dequantize rotates back."""
        assert capacity_tokens % PAGE_TOKENS == 0
        assert not (k_axis == 1 and kb == 16)
        assert k_signs is None or kb != 16
        self.k_signs = None if k_signs is None else np.asarray(k_signs, np.int8)
        self.B, self.H, self.D = batch, n_kv_heads, head_dim
        self.dtype = dtype
        self.capacity = capacity_tokens
        self.L = Layout(head_dim, kb, vb, gk, gv, k_axis)
        self.pages = np.zeros((batch, n_kv_heads, capacity_tokens // PAGE_TOKENS, self.L.page_bytes), np.uint8)
        self.k_tail = np.zeros((batch, n_kv_heads, PAGE_TOKENS, head_dim), np.uint16) if k_axis == 1 else None
        self.seq_len = np.zeros(batch, np.int32)
        self.status = 0
        assert residual == 0 or (k_axis == 0 and residual > 0)
        self.R = residual
        # [B, H, R, 2, D]: 16-bit patterns of (key row, value row) of the tokens not yet quantized
        self.kv_win = np.zeros((batch, n_kv_heads, residual, 2, head_dim), np.uint16) if residual else None

    def flushed(self, b) -> int:
        """Tokens of sequence b that live in the pages (the rest is in the residual window)."""
        n = int(self.seq_len[b])
        return n if not self.R else (n // self.R) * self.R

    # ------------------------------------------------------------------ append
    def append(self, k_bits: np.ndarray, v_bits: np.ndarray):
        """k_bits, v_bits: uint16 [B, Hkv, t_new, D] patterns of the input dtype."""
        if self.R:
            return self._append_residual(k_bits, v_bits)
        return self._append_at(k_bits, v_bits, None)

    def _append_residual(self, k_bits, v_bits):
        R, t_new = self.R, k_bits.shape[2]
        for b in range(self.B):
            t0 = int(self.seq_len[b])
            if t0 + t_new > self.capacity:
                self.status |= ERR_CAPACITY_BIT
                continue
            f0, f1 = (t0 // R) * R, ((t0 + t_new) // R) * R
            if f1 > f0:
                # tokens f0 .. f1-1 are complete blocks: the old window's tokens followed by new ones
                kq = np.concatenate([self.kv_win[b, :, :t0 - f0, 0], k_bits[b, :, :f1 - t0]], axis=1)
                vq = np.concatenate([self.kv_win[b, :, :t0 - f0, 1], v_bits[b, :, :f1 - t0]], axis=1)
                self._append_at(kq[None], vq[None], (b, f0))
            for t in range(max(t0, f1), t0 + t_new):
                self.kv_win[b, :, t % R, 0] = k_bits[b, :, t - t0]
                self.kv_win[b, :, t % R, 1] = v_bits[b, :, t - t0]
            self.seq_len[b] = t0 + t_new

    def _append_at(self, k_bits, v_bits, where):
        """Quantize and store tokens; where = None: every sequence at its seq_len (which is advanced), or
        (b, position): one sequence's tokens at a given position (seq_len untouched)."""
        L = self.L
        t_new = k_bits.shape[2]
        for b in (range(self.B) if where is None else [where[0]]):
            t0 = int(self.seq_len[b]) if where is None else where[1]
            if where is not None:
                k_bits_b, v_bits_b = k_bits[0], v_bits[0]
            else:
                k_bits_b, v_bits_b = k_bits[b], v_bits[b]
            if where is None and t0 + t_new > self.capacity:
                self.status |= ERR_CAPACITY_BIT
                continue
            for h in range(self.H):
                done = 0
                while done < t_new:
                    t = t0 + done
                    p, slot = divmod(t, PAGE_TOKENS)
                    n = min(PAGE_TOKENS - slot, t_new - done)
                    slots = np.arange(slot, slot + n)
                    page = self.pages[b, h, p]
                    kx = k_bits_b[h, done:done + n]
                    vx = v_bits_b[h, done:done + n]
                    # values: always token-wise
                    if L.vb == 16:
                        layout.put_v_codes(page, L, slots, vx)
                    else:
                        c, s, z = quantizer.quantize_per_token(vx, self.dtype, L.vb, L.gv)
                        layout.put_v_codes(page, L, slots, c)
                        layout.put_v_meta_tokens(page, L, slots, s, z)
                    # keys
                    if self.k_signs is not None:
                        k32 = quantizer.rotate_f32(quantizer.bits_to_f32(kx, self.dtype), self.k_signs)
                    if L.k_axis == 0:
                        if L.kb == 16:
                            layout.put_k_codes(page, L, slots, kx)
                        else:
                            if self.k_signs is None:
                                c, s, z = quantizer.quantize_per_token(kx, self.dtype, L.kb, L.gk)
                            else:
                                c, s, z = quantizer.quantize_groups(k32.reshape(n, self.D // L.gk, L.gk), L.kb)
                                c = c.reshape(n, self.D)
                            layout.put_k_codes(page, L, slots, c)
                            layout.put_k_meta_tokens(page, L, slots, s, z)
                    else:
                        if self.k_signs is None:
                            self.k_tail[b, h, slot:slot + n] = quantizer.to_tail_fp16_bits(kx, self.dtype)
                        else:
                            self.k_tail[b, h, slot:slot + n] = quantizer.f32_to_fp16_bits(k32, saturate=True)
                        if slot + n == PAGE_TOKENS:      # block complete: flush the tail
                            c, s, z = quantizer.quantize_per_channel_block(self.k_tail[b, h], L.kb)
                            layout.put_k_codes(page, L, np.arange(PAGE_TOKENS), c)
                            layout.put_k_meta_channels(page, L, s, z)
                    done += n
            if where is None:
                self.seq_len[b] = t0 + t_new

    # ------------------------------------------------------- page -> values
    def _page_values(self, b, h, p, n_valid, exact: bool):
        """Reconstruction of the first n_valid tokens of page p.
        exact=True: fp64 z + s*c (for attention); False: fp32 fmaf (for dequantize).
        Returns (K (n,D), V (n,D))."""
        L, D = self.L, self.D
        page = self.pages[b, h, p]
        deq = quantizer.dequantize_groups_f64 if exact else quantizer.dequantize_groups
        # V
        if L.vb == 16:
            V = quantizer.bits_to_f32(layout.get_v_codes(page, L), self.dtype)
        else:
            c = layout.get_v_codes(page, L).reshape(PAGE_TOKENS, D // L.gv, L.gv)
            s, z = layout.get_v_meta(page, L)
            V = deq(c, s, z).reshape(PAGE_TOKENS, D)
        # K
        tail_tokens = L.k_axis == 1 and n_valid < PAGE_TOKENS
        if tail_tokens:
            K = quantizer.bits_to_f32(self.k_tail[b, h], "fp16")
        elif L.kb == 16:
            K = quantizer.bits_to_f32(layout.get_k_codes(page, L), self.dtype)
        elif L.k_axis == 0:
            c = layout.get_k_codes(page, L).reshape(PAGE_TOKENS, D // L.gk, L.gk)
            s, z = layout.get_k_meta(page, L)
            K = deq(c, s, z).reshape(PAGE_TOKENS, D)
        else:
            c = layout.get_k_codes(page, L)            # (128, D), one group per channel
            s, z = layout.get_k_meta(page, L)          # (D,)
            K = deq(np.ascontiguousarray(c.T), s, z).T
        if exact:
            K = K.astype(np.float64)
            V = V.astype(np.float64)
        return K[:n_valid], V[:n_valid]

    def _window_values(self, b, h, t_lo, t_hi):
        """Values (K, V) of the window tokens t_lo <= t < t_hi of stream (b, h) for attention: the 16-bit inputs,
        exactly.  With rotated keys the queries are rotated too, so the window's keys are given the same (exact,
        fp64) rotation: (H k) . (H q) = k . q."""
        slots = np.arange(t_lo, t_hi) % self.R
        kw = quantizer.bits_to_f32(self.kv_win[b, h, slots, 0], self.dtype).astype(np.float64)
        if self.k_signs is not None:
            kw = quantizer.hadamard_rotate_f64(kw, self.k_signs)
        return kw, quantizer.bits_to_f32(self.kv_win[b, h, slots, 1], self.dtype)

    def values_f64(self):
        """K-hat, V-hat as fp64 [B, Hkv, capacity, D]; zeros beyond seq_len."""
        K = np.zeros((self.B, self.H, self.capacity, self.D), np.float64)
        V = np.zeros_like(K)
        for b in range(self.B):
            n = int(self.seq_len[b])
            for h in range(self.H):
                for p in range((n + PAGE_TOKENS - 1) // PAGE_TOKENS):
                    nv = min(PAGE_TOKENS, n - p * PAGE_TOKENS)
                    k, v = self._page_values(b, h, p, nv, exact=True)
                    K[b, h, p * PAGE_TOKENS: p * PAGE_TOKENS + nv] = k
                    V[b, h, p * PAGE_TOKENS: p * PAGE_TOKENS + nv] = v
                if self.R and self.flushed(b) < n:
                    K[b, h, self.flushed(b):n], V[b, h, self.flushed(b):n] = self._window_values(b, h, self.flushed(b), n)
        return K, V

    # -------------------------------------------------------------- dequantize
    def dequantize(self, k_out: np.ndarray, v_out: np.ndarray, t_begin: int, t_end: int):
        """Writes 16-bit patterns of the input dtype into k_out, v_out
        [B, Hkv, capacity, D] for tokens t_begin <= t < min(t_end, seq_len[b])."""
        for b in range(self.B):
            hi = min(t_end, int(self.seq_len[b]))
            n = int(self.seq_len[b])
            for h in range(self.H):
                for p in range(t_begin // PAGE_TOKENS, (hi + PAGE_TOKENS - 1) // PAGE_TOKENS):
                    nv = min(PAGE_TOKENS, n - p * PAGE_TOKENS)
                    k, v = self._page_values(b, h, p, nv, exact=False)
                    lo_t = max(t_begin, p * PAGE_TOKENS)
                    hi_t = min(hi, p * PAGE_TOKENS + nv)
                    sl = slice(lo_t - p * PAGE_TOKENS, hi_t - p * PAGE_TOKENS)
                    ks = k[sl] if self.k_signs is None else quantizer.unrotate_f32(k[sl], self.k_signs)
                    k_out[b, h, lo_t:hi_t] = quantizer.f32_to_bits(ks, self.dtype)
                    v_out[b, h, lo_t:hi_t] = quantizer.f32_to_bits(v[sl], self.dtype)
                if self.R:                       # tokens still in the residual window come back as they went in
                    w_lo, w_hi = max(t_begin, self.flushed(b)), hi
                    if w_lo < w_hi:
                        slots = np.arange(w_lo, w_hi) % self.R
                        k_out[b, h, w_lo:w_hi] = self.kv_win[b, h, slots, 0]
                        v_out[b, h, w_lo:w_hi] = self.kv_win[b, h, slots, 1]

    # ------------------------------------------------------------------ decode
    def decode(self, q_bits: np.ndarray, scale=None) -> np.ndarray:
        """q_bits uint16 [B, Hq, D] of the input dtype -> fp64 [B, Hq, D]."""
        q = quantizer.bits_to_f32(q_bits, self.dtype).astype(np.float64)
        if self.k_signs is not None:
            q = quantizer.hadamard_rotate_f64(q, self.k_signs)      # (H k) . (H q) = k . q
        K, V = self.values_f64()
        return attention.decode_attention(q, K, V, self.seq_len, scale)

    def decode_rows(self, q_bits: np.ndarray, scale=None) -> np.ndarray:
        """q_bits uint16 [B, R, Hq, D]: R causal query rows for the last R cached tokens -> fp64 [B, R, Hq, D]."""
        q = quantizer.bits_to_f32(q_bits, self.dtype).astype(np.float64)
        if self.k_signs is not None:
            q = quantizer.hadamard_rotate_f64(q, self.k_signs)
        K, V = self.values_f64()
        return attention.decode_attention_rows(q, K, V, self.seq_len, scale)

    def decode_streams(self, q_bits: np.ndarray, streams, scale=None):
        """Same as decode but only for the listed (b, kv_head) streams; returns
        {(b, kv_head): fp64 (G, D)} (used to sample full-size workloads)."""
        import math
        q = quantizer.bits_to_f32(q_bits, self.dtype).astype(np.float64)
        if self.k_signs is not None:
            q = quantizer.hadamard_rotate_f64(q, self.k_signs)
        G = q.shape[1] // self.H
        sc = scale if scale and scale > 0 else 1.0 / math.sqrt(self.D)
        res = {}
        for (b, h) in streams:
            n = int(self.seq_len[b])
            Ks, Vs = [], []
            for p in range((n + PAGE_TOKENS - 1) // PAGE_TOKENS):
                nv = min(PAGE_TOKENS, n - p * PAGE_TOKENS)
                k, v = self._page_values(b, h, p, nv, exact=True)
                Ks.append(k)
                Vs.append(v)
            K = np.concatenate(Ks) if Ks else np.zeros((0, self.D))
            V = np.concatenate(Vs) if Vs else np.zeros((0, self.D))
            if self.R and self.flushed(b) < n:
                kw, vw = self._window_values(b, h, self.flushed(b), n)
                K[self.flushed(b):n], V[self.flushed(b):n] = kw, vw
            res[(b, h)] = np.stack([attention.attend_one(q[b, h * G + j], K, V, sc) for j in range(G)])
        return res
