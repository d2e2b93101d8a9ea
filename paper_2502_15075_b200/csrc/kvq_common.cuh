// Shared device/host definitions of libkvq: page geometry, the layout's index
// functions and the fixed-formula group quantizer (App. B.1 uniform scalar
// quantizer applied per group with a minimum offset).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvq.h"

namespace kvq {

constexpr int kPageTokens = KVQ_PAGE_TOKENS;
constexpr int kMaxGroupHeads = 8;  // query heads per KV head

// Everything a kernel needs to know about a cache, derived from kvq_config.
struct Geom {
  int B, Hq, Hkv, G, D;
  int kb, vb, gk, gv, k_axis, in_dtype;
  int capacity, n_pages;
  int k_codes_bytes, k_meta_off, k_meta_bytes;
  int v_codes_off, v_codes_bytes, v_meta_off, v_meta_bytes;
  int page_bytes;
  int rows;          // query rows per head of a decode call (1 = a plain decode step)
  int R;             // residual window: the newest seq_len % R tokens are not in the pages (0: no window)
};

// Pointers of one cache (device memory).
struct CachePtrs {
  uint8_t* pages;
  uint16_t* k_tail;
  int32_t* seq_len;
  uint32_t* status;
  const int8_t* k_signs;   // NULL: keys are not rotated
  uint16_t* kv_win;        // residual window [B][Hkv][R][2][D], or NULL
};

// Sequence length as the kernels use it: a corrupt value can never index outside the cache.
__device__ __forceinline__ int clamped_len(const int32_t* seq_len, int b, int capacity) {
  return min(max(seq_len[b], 0), capacity);
}

// Tokens of a sequence that live in the pages: all of them, or whole blocks of R when a residual window is kept.
__device__ __forceinline__ int paged_len(const int32_t* seq_len, int b, int capacity, int R) {
  const int n = clamped_len(seq_len, b, capacity);
  return R ? (n / R) * R : n;
}

// ---------------------------------------------------------------- conversions
__device__ __forceinline__ float bits16_to_f32(uint16_t u, int dtype) {
  if (dtype == KVQ_FP16) return __half2float(__ushort_as_half(u));
  return __uint_as_float(((uint32_t)u) << 16);
}

__device__ __forceinline__ uint16_t f32_to_fp16_sat_bits(float x) {
  x = fminf(fmaxf(x, -65504.0f), 65504.0f);
  return __half_as_ushort(__float2half_rn(x));
}

__device__ __forceinline__ uint16_t f32_to_bits16(float x, int dtype) {
  if (dtype == KVQ_FP16) return __half_as_ushort(__float2half_rn(x));
  return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}

// ---------------------------------------------------------------- quantizer
struct GroupParams {
  float s, z, inv;     // fp32 values of the stored fp16 scale / zero, and 1/s (0 when s == 0)
  uint32_t meta;       // s16 | z16 << 16
};

__device__ __forceinline__ GroupParams group_params(float mn, float mx, float qmax) {
  mn = __fadd_rn(mn, 0.0f);
  mx = __fadd_rn(mx, 0.0f);
  float scale32 = __fdiv_rn(__fsub_rn(mx, mn), qmax);
  uint16_t s16 = f32_to_fp16_sat_bits(scale32);
  uint16_t z16 = f32_to_fp16_sat_bits(mn);
  GroupParams p;
  p.s = __half2float(__ushort_as_half(s16));
  p.z = __half2float(__ushort_as_half(z16));
  p.inv = (p.s != 0.0f) ? __fdiv_rn(1.0f, p.s) : 0.0f;
  p.meta = (uint32_t)s16 | ((uint32_t)z16 << 16);
  return p;
}

__device__ __forceinline__ uint32_t code_of(float x, const GroupParams& p, float qmax) {
  float u = __fmul_rn(__fsub_rn(x, p.z), p.inv);
  float r = rintf(u);
  r = fminf(fmaxf(r, 0.0f), qmax);
  return (uint32_t)r;
}

// Same result as code_of without the round / convert instructions: after the clamp to [0, qmax], adding
// 1.5 * 2^23 rounds to nearest-even in the float adder and leaves the integer in the low mantissa bits
// (rounding and clamping to integer bounds commute).
__device__ __forceinline__ uint32_t code_of_fast(float x, const GroupParams& p, float qmax) {
  float u = __fmul_rn(__fsub_rn(x, p.z), p.inv);
  u = fminf(fmaxf(u, 0.0f), qmax);
  return __float_as_uint(__fadd_rn(u, 12582912.0f)) & 0xFFu;
}

// ---------------------------------------------------------------- key rotation (Sec. 4.4)
// A token row of D channels is spread over D/8 lanes, lane l holding channels 8l..8l+7.  Unnormalised
// Walsh-Hadamard transform with the butterfly stages in the order h = 1, 2, 4, ..., (a, b) -> (a + b, a - b)
// where a is the element whose index has bit h clear; every addition individually rounded.
template <int D>
__device__ __forceinline__ void fwht_row8(float (&x)[8], int l) {
#pragma unroll
  for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if ((i & h) == 0) {
        const float a = x[i], b = x[i + h];
        x[i] = __fadd_rn(a, b);
        x[i + h] = __fsub_rn(a, b);
      }
    }
  }
#pragma unroll
  for (int m = 1; m < D / 8; m <<= 1) {
    const bool upper = (l & m) != 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float o = __shfl_xor_sync(0xffffffffu, x[i], m);
      x[i] = upper ? __fsub_rn(o, x[i]) : __fadd_rn(x[i], o);
    }
  }
}

template <int D> __device__ __forceinline__ constexpr float inv_sqrt_dim() { return D == 128 ? 0.08838834764831845f : 0.125f; }

// y = H (signs * x) / sqrt(D)
template <int D>
__device__ __forceinline__ void rotate_row8(float (&x)[8], const int8_t* signs, int l) {
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __fmul_rn(x[i], (float)signs[8 * l + i]);
  fwht_row8<D>(x, l);
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __fmul_rn(x[i], inv_sqrt_dim<D>());
}

// x = signs * (H y / sqrt(D))
template <int D>
__device__ __forceinline__ void unrotate_row8(float (&x)[8], const int8_t* signs, int l) {
  fwht_row8<D>(x, l);
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = __fmul_rn(__fmul_rn(x[i], inv_sqrt_dim<D>()), (float)signs[8 * l + i]);
}

// ---------------------------------------------------------------- layout index functions
// Byte offset (inside the K-code region of a page) of the 32-bit word holding
// channel d of page-local token t, and the field's bit offset inside that word.
// Byte offset of (chunk, word) inside a K row (nchunks = 4): words are kept in quads of min(wpc, 4) words,
// quad-major, so that a lane's 16-byte load never conflicts with its neighbours'.
__host__ __device__ __forceinline__ int chunk_word_byte(int chunk, int word, int wpc, int nchunks) {
  int qw = wpc < 4 ? wpc : 4;
  return (word >> 2) * (nchunks * 4 * qw) + chunk * (4 * qw) + (word & 3) * 4;
}

__host__ __device__ __forceinline__ void k_code_pos(int t, int d, int D, int b, int& word_byte, int& bit) {
  int fpb = 8 / b;              // fields per byte
  int chunk = (d & 15) >> 2;
  int r = d >> 4;               // register index inside the chunk
  word_byte = t * (D * b / 8) + chunk_word_byte(chunk, r / fpb, D * b / 128, 4);
  bit = 8 * (d & 3) + b * (r % fpb);
}

// Value codes: 4 blocks of 32 tokens per page, 4*D*b bytes each.  A byte holds the codes of one token for the
// 8/b channels that lie 16 apart (field f at bit b*f); the four bytes of a word are tokens 2t, 2t+8, 2t+1, 2t+9
// of one 16-token half of the block.  Returns the word's byte offset and the field's bit offset inside the word.
__host__ __device__ __forceinline__ void v_code_pos(int t, int d, int D, int b, int& word_byte, int& bit) {
  const int fpb = 8 / b;
  const int blk = t >> 5, tau = t & 31, kh = tau >> 4, u = tau & 15;
  const int tq = (u & 7) >> 1, j = 2 * (u & 1) + (u >> 3);
  const int m = d >> 4, f = m % fpb, mw = m / fpb, rh = (d >> 3) & 1, gq = d & 7;
  word_byte = blk * (4 * D * b) + mw * 512 + (4 * gq + tq) * 16 + 4 * (2 * rh + kh);
  bit = 8 * j + b * f;
}

// Inverse maps: which channel (and tile-local token) sits in field f of a word.
__device__ __forceinline__ int k_field_channel(int chunk, int word, int f, int b) {
  int fpb = 8 / b;
  int r = word * fpb + (f % fpb);
  return 16 * r + 4 * chunk + (f / fpb);
}

// Word number w (0 .. D*b-1) of a value block: which block-local token and channel sit in byte j, field f.
__device__ __forceinline__ void v_field_pos(int w, int j, int f, int b, int& tau, int& d) {
  const int fpb = 8 / b;
  const int mw = w >> 7, lane = (w >> 2) & 31, sub = w & 3;
  const int gq = lane >> 2, tq = lane & 3, rh = sub >> 1, kh = sub & 1;
  tau = 16 * kh + 2 * tq + (j >> 1) + 8 * (j & 1);
  d = 16 * (fpb * mw + f) + 8 * rh + gq;
}

// Code widths 1, 3 and 6 are stored as bit planes: a high plane of 2 (4) bits followed by a low plane of 1 (2)
// bits, each a code region of its own width; 1-bit codes are one 1-bit plane.  planes_of: (high plane bits, low
// plane bits or 0).
__host__ __device__ __forceinline__ bool is_plane_width(int b) { return b == 1 || b == 3 || b == 6; }
__host__ __device__ __forceinline__ void planes_of(int b, int& hi, int& lo) {
  if (b == 3) { hi = 2; lo = 1; } else if (b == 6) { hi = 4; lo = 2; } else { hi = b; lo = 0; }
}

// Position of one plane's field of (token t, channel d) in a key (is_v = false) or value code region of a page:
// byte offset of the 32-bit word (from the region's start) and the field's bit offset.  plane 0 = high plane.
__device__ __forceinline__ void plane_pos(bool is_v, int t, int d, int D, int b, int plane, int& word_byte, int& bit,
                                          int& pbits) {
  int hi, lo;
  planes_of(b, hi, lo);
  pbits = plane == 0 ? hi : lo;
  if (is_v) v_code_pos(t, d, D, pbits, word_byte, bit); else k_code_pos(t, d, D, pbits, word_byte, bit);
  if (plane == 1) word_byte += kPageTokens * D * hi / 8;
}

// A code of any supported width from a code region.
__device__ __forceinline__ uint32_t load_code_any(const uint8_t* region, bool is_v, int t, int d, int D, int b) {
  int hi, lo, wb, bit, pb;
  planes_of(b, hi, lo);
  plane_pos(is_v, t, d, D, b, 0, wb, bit, pb);
  uint32_t c = (*reinterpret_cast<const uint32_t*>(region + wb) >> bit) & ((1u << hi) - 1u);
  if (lo) {
    plane_pos(is_v, t, d, D, b, 1, wb, bit, pb);
    c = (c << lo) | ((*reinterpret_cast<const uint32_t*>(region + wb) >> bit) & ((1u << lo) - 1u));
  }
  return c;
}

__device__ __forceinline__ uint32_t load_code(const uint8_t* region, int word_byte, int bit, int b) {
  uint32_t w = *reinterpret_cast<const uint32_t*>(region + word_byte);
  return (w >> bit) & ((1u << b) - 1u);
}

}  // namespace kvq
