"""Oracle decode attention in fp64 (test infrastructure).

App. A.1 notation: S = Q K^T / sqrt(d), A = softmax(S), output A V, here for a
single query row per head (one decode step) with d the head dimension, and
consecutive query heads sharing a KV head (grouped-query attention: query head
h reads KV head h // G, G = n_q_heads / n_kv_heads).
"""
from __future__ import annotations

import math

import numpy as np


def attend_one(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float) -> np.ndarray:
    """softmax(scale * K q) V for one query.  q (D,), K, V (T, D), all fp64.
    T == 0 gives zeros."""
    T = K.shape[0]
    if T == 0:
        return np.zeros(V.shape[1], np.float64)
    logits = scale * (K @ q)
    logits = logits - logits.max()
    p = np.exp(logits)
    p = p / p.sum()
    return p @ V


def decode_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, seq_len, scale=None) -> np.ndarray:
    """q (B, Hq, D); K, V (B, Hkv, T, D) fp64 (already dequantized);
    seq_len (B,) tokens to attend to.  Returns (B, Hq, D) fp64."""
    B, Hq, D = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(D)
    out = np.zeros((B, Hq, D), np.float64)
    for b in range(B):
        n = int(seq_len[b])
        for h in range(Hq):
            kv = h // G
            out[b, h] = attend_one(q[b, h].astype(np.float64), K[b, kv, :n], V[b, kv, :n], scale)
    return out


def partial_state(q, K, V, scale):
    """(m, l, o) of one token range: m = max logit, l = sum exp(logit - m),
    o = sum exp(logit - m) v  (unnormalised).  Empty range: (-inf, 0, 0)."""
    if K.shape[0] == 0:
        return -np.inf, 0.0, np.zeros(V.shape[1], np.float64)
    logits = scale * (K @ q)
    m = logits.max()
    p = np.exp(logits - m)
    return m, p.sum(), p @ V


def lse_merge(parts):
    """Merge split partial states by log-sum-exp: m* = max m_j,
    out = sum_j e^(m_j - m*) o_j / sum_j e^(m_j - m*) l_j."""
    ms = [m for m, _, _ in parts]
    mstar = max(ms)
    if not np.isfinite(mstar):
        return np.zeros_like(parts[0][2])
    num = sum(np.exp(m - mstar) * o for m, _, o in parts)
    den = sum(np.exp(m - mstar) * l for m, l, _ in parts)
    return num / den


def decode_attention_rows(q: np.ndarray, K: np.ndarray, V: np.ndarray, seq_len, scale=None) -> np.ndarray:
    """Several query rows per head (App. A.1: Q has one row per position, S = Q K^T / sqrt(d)), for the last R
    positions of each sequence, with the causal mask of a decoder (reading: the paper writes no mask; its models
    are causal language models): row r belongs to the token at position seq_len - R + r and attends to the
    tokens at positions <= its own, i.e. to the first seq_len - (R - 1 - r) tokens.

    q (B, R, Hq, D); K, V (B, Hkv, T, D) fp64; returns (B, R, Hq, D) fp64.  A row whose token does not exist
    (seq_len < R - r) gives zeros."""
    B, R, Hq, D = q.shape
    G = Hq // K.shape[1]
    if scale is None or scale <= 0:
        scale = 1.0 / math.sqrt(D)
    out = np.zeros((B, R, Hq, D), np.float64)
    for b in range(B):
        for r in range(R):
            n = max(0, int(seq_len[b]) - (R - 1 - r))
            for h in range(Hq):
                kv = h // G
                out[b, r, h] = attend_one(q[b, r, h].astype(np.float64), K[b, kv, :n], V[b, kv, :n], scale)
    return out
