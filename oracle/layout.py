"""Oracle packer / unpacker for the packed KV page (test infrastructure).

Written from the layout's published index function, independently of the CUDA
code.  The paper describes no packed layout; this one is the library's own
(layout version 2):

A page holds 128 consecutive tokens of one (batch, kv-head) stream as four
regions, in this order, each a multiple of 16 bytes:

    [K codes | K meta | V codes | V meta]

All multi-byte quantities are little-endian.  A b-bit code field number f of a
32-bit word occupies bits [f*b, f*b+b).

K codes (b = kb in {2,4,8}): token-major rows of D*b/8 bytes; a row holds 4
chunks of wpc = D*b/128 words.  With fpb = 8/b fields per byte, channel d of a
token lives in
    chunk  = (d % 16) // 4
    r      = d // 16                               register index inside the chunk
    word   = r // fpb,  bit = 8*(d % 4) + b*(r % fpb)
(byte j of a word holds channels 16r + 4*chunk + j for the fpb values of r that
share the word: masking one field out of every byte yields four consecutive
channels as four bytes).
V codes (b = vb in {2,4,8}): 4 blocks of 32 tokens, a block holds 4*D*b bytes.
A byte holds the codes of ONE token for the fpb = 8/b channels d, d+16, ...
that differ only in f below (field f at bit b*f).  With
    m  = d // 16,  f = m % fpb,  mw = m // fpb,  rh = (d % 16) // 8,  g = d % 8
    kh = tau // 16,  u = tau % 16,  t = (u % 8) // 2,  j = 2*(u % 2) + u // 8
channel d of token tau (0..31 inside its block) lives in
    byte = block*(4*D*b) + mw*512 + (4*g + t)*16 + 4*(2*rh + kh) + j,  bit = b*f
(the four bytes of a 32-bit word are tokens 2t, 2t+8, 2t+1, 2t+9 of one half
of the block for one channel; masking one field out of every byte yields four
tokens of one channel as four bytes, and a token's codes are whole bytes, so an
append never has to merge with bytes of other tokens).
Placement of (chunk, word) inside a K row of `nchunks` = 4 chunks: words are
kept in quads of qw = min(wpc, 4) words, quad-major:
    byte   = (word // 4)*(nchunks*4*qw) + chunk*(4*qw) + (word % 4)*4
(for wpc <= 4 this is simply chunk-major).
b = 16 (either side): plain rows [token][D] of the input's 16-bit patterns.
b in {1, 3, 6}: bit planes.  A 3-bit code is stored as a 2-bit plane (code >> 1) followed by a 1-bit plane
(code & 1), a 6-bit code as a 4-bit plane (code >> 2) followed by a 2-bit plane (code & 3), a 1-bit code as one
1-bit plane; every plane is a code region of its own width laid out as above (the high plane first), so the
region still holds 128*D*b/8 bytes.  1-bit planes need head_dim 128.

Meta: (scale fp16, zero fp16) pairs, 4 bytes each.  Per-token axis:
[128 tokens][D/g groups]; per-channel K: [D channels] (one group per channel
over the page's 128 tokens).  A 16-bit side has no meta.
"""
from __future__ import annotations

import dataclasses

import numpy as np

PAGE_TOKENS = 128


def planes(b: int):
    """Bit planes of a b-bit code, high plane first: [(plane bits, right shift of the code)]."""
    return {1: [(1, 0)], 2: [(2, 0)], 3: [(2, 1), (1, 0)], 4: [(4, 0)], 6: [(4, 2), (2, 0)], 8: [(8, 0)]}[b]


@dataclasses.dataclass(frozen=True)
class Layout:
    D: int
    kb: int
    vb: int
    gk: int
    gv: int
    k_axis: int = 0

    @property
    def k_codes_bytes(self):
        return PAGE_TOKENS * self.D * self.kb // 8

    @property
    def k_meta_bytes(self):
        if self.kb == 16:
            return 0
        return 4 * self.D if self.k_axis == 1 else PAGE_TOKENS * (self.D // self.gk) * 4

    @property
    def v_codes_bytes(self):
        return PAGE_TOKENS * self.D * self.vb // 8

    @property
    def v_meta_bytes(self):
        return 0 if self.vb == 16 else PAGE_TOKENS * (self.D // self.gv) * 4

    @property
    def k_meta_off(self):
        return self.k_codes_bytes

    @property
    def v_codes_off(self):
        return self.k_meta_off + self.k_meta_bytes

    @property
    def v_meta_off(self):
        return self.v_codes_off + self.v_codes_bytes

    @property
    def page_bytes(self):
        return self.v_meta_off + self.v_meta_bytes


# ----------------------------------------------------------------------------
# index functions: (token in page, channel) -> (byte offset in region, bit shift)
# ----------------------------------------------------------------------------
def _chunk_word_byte(chunk, word, wpc, nchunks):
    qw = min(wpc, 4)
    return (word // 4) * (nchunks * 4 * qw) + chunk * (4 * qw) + (word % 4) * 4


def k_code_pos(t, d, D, b):
    t = np.asarray(t)
    d = np.asarray(d)
    fpb = 8 // b                      # fields per byte
    chunk = (d % 16) // 4
    r = d // 16
    word = r // fpb
    bit = 8 * (d % 4) + b * (r % fpb)
    byte = t * (D * b // 8) + _chunk_word_byte(chunk, word, D * b // 128, 4) + bit // 8
    return byte, bit % 8


def v_code_pos(t, d, D, b):
    t = np.asarray(t)
    d = np.asarray(d)
    fpb = 8 // b                      # codes per byte (channels 16 apart)
    block = t // 32
    tau = t % 32
    kh = tau // 16
    u = tau % 16
    tq = (u % 8) // 2
    j = 2 * (u % 2) + u // 8
    m = d // 16
    f = m % fpb
    mw = m // fpb
    rh = (d % 16) // 8
    g = d % 8
    byte = block * (4 * D * b) + mw * 512 + (4 * g + tq) * 16 + 4 * (2 * rh + kh) + j
    return byte, b * f + 0 * byte


def _put_codes(region: np.ndarray, pos_fn, tokens: np.ndarray, codes: np.ndarray, D, b):
    """OR b-bit codes (n, D) of the given page-local tokens into a code region."""
    tt, dd = np.meshgrid(tokens, np.arange(D), indexing="ij")
    if b == 16:
        u = codes.astype(np.uint16)
        region[tt * 2 * D + 2 * dd] = (u & 0xFF).astype(np.uint8)
        region[tt * 2 * D + 2 * dd + 1] = (u >> 8).astype(np.uint8)
        return
    off = 0
    for pb, sh in planes(b):
        byte, shift = pos_fn(tt, dd, D, pb)
        byte = byte + off
        mask = (1 << pb) - 1
        part = (codes.astype(np.uint32).ravel() >> sh) & mask
        # clear, then set (fields never straddle bytes because the plane width divides 8)
        np.bitwise_and.at(region, byte.ravel(), (~(mask << shift.ravel()) & 0xFF).astype(np.uint8))
        np.bitwise_or.at(region, byte.ravel(), (part << shift.ravel()).astype(np.uint8))
        off += PAGE_TOKENS * D * pb // 8


def _get_codes(region: np.ndarray, pos_fn, D, b) -> np.ndarray:
    tt, dd = np.meshgrid(np.arange(PAGE_TOKENS), np.arange(D), indexing="ij")
    if b == 16:
        lo = region[tt * 2 * D + 2 * dd].astype(np.uint16)
        hi = region[tt * 2 * D + 2 * dd + 1].astype(np.uint16)
        return lo | (hi << 8)
    out = np.zeros(tt.shape, np.uint8)
    off = 0
    for pb, sh in planes(b):
        byte, shift = pos_fn(tt, dd, D, pb)
        out |= (((region[byte + off] >> shift.astype(np.uint8)) & ((1 << pb) - 1)) << sh).astype(np.uint8)
        off += PAGE_TOKENS * D * pb // 8
    return out


def put_k_codes(page: np.ndarray, L: Layout, tokens, codes):
    _put_codes(page[: L.k_codes_bytes], k_code_pos, np.asarray(tokens), codes, L.D, L.kb)


def put_v_codes(page: np.ndarray, L: Layout, tokens, codes):
    _put_codes(page[L.v_codes_off: L.v_codes_off + L.v_codes_bytes], v_code_pos,
               np.asarray(tokens), codes, L.D, L.vb)


def get_k_codes(page: np.ndarray, L: Layout) -> np.ndarray:
    return _get_codes(page[: L.k_codes_bytes], k_code_pos, L.D, L.kb)


def get_v_codes(page: np.ndarray, L: Layout) -> np.ndarray:
    return _get_codes(page[L.v_codes_off: L.v_codes_off + L.v_codes_bytes], v_code_pos, L.D, L.vb)


def _meta_view(page: np.ndarray, off: int, nbytes: int) -> np.ndarray:
    """uint16 view [n][2] = (scale bits, zero bits) of a meta region."""
    return page[off: off + nbytes].view(np.uint16).reshape(-1, 2)


def put_k_meta_tokens(page, L: Layout, tokens, s16, z16):
    """per-token axis: s16, z16 (n, D/gk)."""
    m = _meta_view(page, L.k_meta_off, L.k_meta_bytes).reshape(PAGE_TOKENS, L.D // L.gk, 2)
    m[np.asarray(tokens), :, 0] = s16
    m[np.asarray(tokens), :, 1] = z16


def put_k_meta_channels(page, L: Layout, s16, z16):
    """per-channel axis: s16, z16 (D,)."""
    m = _meta_view(page, L.k_meta_off, L.k_meta_bytes)
    m[:, 0] = s16
    m[:, 1] = z16


def put_v_meta_tokens(page, L: Layout, tokens, s16, z16):
    m = _meta_view(page, L.v_meta_off, L.v_meta_bytes).reshape(PAGE_TOKENS, L.D // L.gv, 2)
    m[np.asarray(tokens), :, 0] = s16
    m[np.asarray(tokens), :, 1] = z16


def get_k_meta(page, L: Layout):
    """(s16, z16): (128, D/gk) for the per-token axis, (D,) for per-channel."""
    m = _meta_view(page, L.k_meta_off, L.k_meta_bytes)
    if L.k_axis == 1:
        return m[:, 0].copy(), m[:, 1].copy()
    m = m.reshape(PAGE_TOKENS, L.D // L.gk, 2)
    return m[..., 0].copy(), m[..., 1].copy()


def get_v_meta(page, L: Layout):
    m = _meta_view(page, L.v_meta_off, L.v_meta_bytes).reshape(PAGE_TOKENS, L.D // L.gv, 2)
    return m[..., 0].copy(), m[..., 1].copy()
