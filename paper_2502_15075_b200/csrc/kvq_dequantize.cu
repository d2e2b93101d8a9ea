// kvq_dequantize kernel: x^ = fmaf(code, scale, zero) rounded to the 16-bit
// input type (App. B.1: A^ = scale * Q, here with the group minimum as offset).
//
// One CTA per (page, stream, side).  Fast path (head_dim 128, token-wise groups,
// 2 / 4 / 8 bits, keys not rotated): keys go straight from global to global
// memory (a thread owns a 16-byte chunk of a token row, whose bytes are four
// consecutive channels of every 16-channel slice), values through a padded
// [128][D + 8] shared tile; code bytes become floats by a byte permute and an
// exact subtraction.  General path (every other configuration): the packed page
// is copied to shared memory and expanded element by element into the tile.
// Both are bound by the 16-bit stores (they write 4-8x what they read).
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 256;
constexpr int kTilePad = 8;     // the shared [128][D + 8] tile: a row stride of D + 8 elements spreads the token rows
                                // over the banks (a stride of D would put every row on the same banks)

// All sizes that index arithmetic divides by are powers of two: use shifts.
__device__ __forceinline__ int ilog2(int x) { return 31 - __clz(x); }

__device__ __forceinline__ float meta_scale(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m & 0xFFFF))); }
__device__ __forceinline__ float meta_zero(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m >> 16))); }

// Expand the key codes of a page into tile[t][d] (16-bit patterns of dtype).
template <int B>
__device__ __forceinline__ void expand_keys(const uint8_t* spage, const Geom& g, uint16_t* tile, int tid) {
  const int D = g.D;
  constexpr int FPB = 8 / B;
  const int wpr = D * B / 32;          // words per token row
  const int wpc = wpr / 4;             // words per chunk
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + g.k_meta_off);
  const int lgk = ilog2(g.gk), ngk = D >> lgk;
  const int lwpr = ilog2(wpr), lwpc = ilog2(wpc);
  for (int idx = tid; idx < kPageTokens * wpr; idx += kThreads) {
    const int t = idx >> lwpr, wi = idx & (wpr - 1);
    const int chunk = wi >> lwpc, word = wi & (wpc - 1);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(spage + (size_t)t * (D * B / 8) +
                                                           chunk_word_byte(chunk, word, wpc, 4));
#pragma unroll
    for (int i = 0; i < FPB; ++i) {
      const int d0 = 16 * (word * FPB + i) + 4 * chunk;           // bytes j = 0..3 hold channels d0 + j
      uint16_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float code = (float)((w >> (8 * j + B * i)) & ((1u << B) - 1u));
        const uint32_t m = meta[g.k_axis == 1 ? d0 + j : t * ngk + ((d0 + j) >> lgk)];
        o[j] = f32_to_bits16(fmaf(code, meta_scale(m), meta_zero(m)), g.in_dtype);
      }
      *reinterpret_cast<uint2*>(tile + t * (D + kTilePad) + d0) =
          make_uint2((uint32_t)o[0] | ((uint32_t)o[1] << 16), (uint32_t)o[2] | ((uint32_t)o[3] << 16));
    }
  }
}

// Expand the value codes of a page into tile[t][d].
template <int B>
__device__ __forceinline__ void expand_values(const uint8_t* spage, const Geom& g, uint16_t* tile, int tid) {
  const int D = g.D;
  constexpr int FPB = 8 / B;
  const int wpb = D * B;               // words per 32-token block
  const uint32_t* codes = reinterpret_cast<const uint32_t*>(spage + g.v_codes_off);
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + g.v_meta_off);
  const int lgv = ilog2(g.gv), ngv = D >> lgv;
  const int lwpb = ilog2(wpb);
  for (int idx = tid; idx < 4 * wpb; idx += kThreads) {
    const int blk = idx >> lwpb, w = idx & (wpb - 1);
    const uint32_t word = codes[idx];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int f = 0; f < FPB; ++f) {
        int tau, d;
        v_field_pos(w, j, f, B, tau, d);
        const int t = blk * 32 + tau;
        const uint32_t m = meta[t * ngv + (d >> lgv)];
        const float code = (float)((word >> (8 * j + B * f)) & ((1u << B) - 1u));
        tile[t * (D + kTilePad) + d] = f32_to_bits16(fmaf(code, meta_scale(m), meta_zero(m)), g.in_dtype);
      }
    }
  }
}

// Expand a code region of a bit-plane width (1, 3, 6 bits) into tile[t][d], element by element.
__device__ __forceinline__ void expand_planes(const uint8_t* spage, const Geom& g, bool is_v, uint16_t* tile, int tid) {
  const int D = g.D, b = is_v ? g.vb : g.kb, gs = is_v ? g.gv : g.gk;
  const uint8_t* region = spage + (is_v ? g.v_codes_off : 0);
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + (is_v ? g.v_meta_off : g.k_meta_off));
  const int lD = ilog2(D), lgs = ilog2(gs), ng = D >> lgs;
  for (int idx = tid; idx < kPageTokens * D; idx += kThreads) {
    const int t = idx >> lD, d = idx & (D - 1);
    const uint32_t m = meta[t * ng + (d >> lgs)];
    const float code = (float)load_code_any(region, is_v, t, d, D, b);
    tile[t * (D + kTilePad) + d] = f32_to_bits16(fmaf(code, meta_scale(m), meta_zero(m)), g.in_dtype);
  }
}

// Rotated keys: reconstruct rows [lo, hi) in fp32, rotate back (x = signs * H y / sqrt(D)) and store 16-bit rows.
// A row is handled by D/8 consecutive lanes, lane l owning channels 8l..8l+7 (two code words of 4 channels each).
template <int B, int D>
__device__ __forceinline__ void dequant_keys_rotated(const uint8_t* spage, const Geom& g, const uint16_t* tail,
                                                     const int8_t* signs, uint16_t* out, int lo, int hi, int tid) {
  constexpr int FPB = 8 / B, LPR = D / 8, RPI = kThreads / LPR;     // rows per iteration of the CTA
  constexpr int wpc = D * B / 128;
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + g.k_meta_off);
  const int lgk = ilog2(g.gk), ngk = D >> lgk;
  const int l = tid % LPR;
  for (int t0 = lo; t0 < hi; t0 += RPI) {
    const int t = t0 + tid / LPR;
    const bool active = t < hi;
    float x[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) x[i] = 0.f;
    if (active) {
      if (tail) {
        const uint4 raw = *reinterpret_cast<const uint4*>(tail + (size_t)t * D + 8 * l);
        const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&rw[i]));
          x[2 * i] = f.x;
          x[2 * i + 1] = f.y;
        }
      } else {
        const int r = l >> 1, word = r / FPB, sh = B * (r % FPB);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int chunk = 2 * (l & 1) + hh;
          const uint32_t w = *reinterpret_cast<const uint32_t*>(spage + (size_t)t * (D * B / 8) +
                                                                 chunk_word_byte(chunk, word, wpc, 4));
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int d = 8 * l + 4 * hh + j;
            const uint32_t m = meta[g.k_axis == 1 ? d : t * ngk + (d >> lgk)];
            x[4 * hh + j] = fmaf((float)((w >> (8 * j + sh)) & ((1u << B) - 1u)), meta_scale(m), meta_zero(m));
          }
        }
      }
    }
    unrotate_row8<D>(x, signs, l);
    if (active) {
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        o[i] = (uint32_t)f32_to_bits16(x[2 * i], g.in_dtype) | ((uint32_t)f32_to_bits16(x[2 * i + 1], g.in_dtype) << 16);
      *reinterpret_cast<uint4*>(out + (size_t)t * D + 8 * l) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

template <int B>
__device__ __forceinline__ void dequant_keys_rotated_d(const uint8_t* spage, const Geom& g, const uint16_t* tail,
                                                       const int8_t* signs, uint16_t* out, int lo, int hi, int tid) {
  if (g.D == 128) dequant_keys_rotated<B, 128>(spage, g, tail, signs, out, lo, hi, tid);
  else dequant_keys_rotated<B, 64>(spage, g, tail, signs, out, lo, hi, tid);
}

// Copy token rows [lo, hi) of a tile with row stride `ts` elements to out rows (16-byte vectors).
__device__ __forceinline__ void store_rows(const uint16_t* tile, int ts, uint16_t* out, int D, int lo, int hi, int tid) {
  const int vpr = D / 8, lv = ilog2(vpr);
  for (int idx = tid; idx < (hi - lo) * vpr; idx += kThreads) {
    const int t = lo + (idx >> lv), v = idx & (vpr - 1);
    __stcs(reinterpret_cast<uint4*>(out + (size_t)t * D) + v, reinterpret_cast<const uint4*>(tile + t * ts)[v]);   // written once, not re-read here
  }
}

// ---------------------------------------------------------------------------------------------------------
// Fast path: head_dim 128, token-wise groups, widths 2 / 4 / 8, keys not rotated.  Everything a thread indexes
// is a compile-time offset from its own base; the four code bytes of a word become floats without a conversion
// instruction (byte -> 0x4B0000bb = 2^23 + code, minus 2^23: exact), so that an element costs one permute, one
// add, the fused multiply-add of the fixed formula and half a packing conversion.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float code_byte_f32(uint32_t bytes, int j) {
  // byte j of `bytes` as an exact float
  return __uint_as_float(__byte_perm(bytes, 0x4B000000u, 0x7540u + (uint32_t)j)) - 8388608.0f;
}
template <int DTYPE>
__device__ __forceinline__ uint32_t pack16(float a, float b) {
  if constexpr (DTYPE == KVQ_FP16) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
  } else {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
  }
}
template <int DTYPE>
__device__ __forceinline__ uint16_t one16(float a) {
  if constexpr (DTYPE == KVQ_FP16) return __half_as_ushort(__float2half_rn(a));
  else return __bfloat16_as_ushort(__float2bfloat16_rn(a));
}

// Keys of one page, straight from global memory to global memory: thread item = (token, 16-byte chunk of its
// row); the chunk's bytes are four consecutive channels of every 16-channel slice, so each slice gives one
// 8-byte store and the four threads of a token write 32 contiguous bytes.
template <int B, int DTYPE>
__device__ __forceinline__ void fast_keys(const Geom& g, const uint8_t* __restrict__ pg, uint16_t* __restrict__ out,
                                          int lo, int hi, int tid) {
  constexpr int D = 128, FPB = 8 / B, ROW = D * B / 8;
  constexpr int WPC = D * B / 128;                       // words per chunk: 1, 2 (one 8-byte load), 4, 8 (two quads)
  constexpr uint32_t MASK = ((1u << B) - 1u) * 0x01010101u;
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(pg + g.k_meta_off);
  const int lgk = ilog2(g.gk), ngk = D >> lgk;
  for (int item = tid; item < kPageTokens * 4; item += kThreads) {
    const int t = item >> 2, chunk = item & 3;
    if (t < lo || t >= hi) continue;
    uint32_t w[WPC];
    const uint8_t* row = pg + t * ROW;
    if constexpr (WPC == 2) {
      const uint2 v = __ldcs(reinterpret_cast<const uint2*>(row + chunk * 8));
      w[0] = v.x; w[1] = v.y;
    } else {
#pragma unroll
      for (int qd = 0; qd < WPC / 4; ++qd) {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(row + qd * 64 + chunk * 16));
        w[4 * qd + 0] = v.x; w[4 * qd + 1] = v.y; w[4 * qd + 2] = v.z; w[4 * qd + 3] = v.w;
      }
    }
    uint16_t* orow = out + (size_t)t * D + 4 * chunk;
#pragma unroll
    for (int r = 0; r < D / 16; ++r) {                   // slice r: channels 16 r + 4 chunk + {0..3}
      const uint32_t bytes = (w[r / FPB] >> (B * (r % FPB))) & MASK;
      const uint32_t m = __ldg(meta + t * ngk + ((16 * r) >> lgk));
      const float sc = meta_scale(m), ze = meta_zero(m);
      const float x0 = fmaf(code_byte_f32(bytes, 0), sc, ze), x1 = fmaf(code_byte_f32(bytes, 1), sc, ze);
      const float x2 = fmaf(code_byte_f32(bytes, 2), sc, ze), x3 = fmaf(code_byte_f32(bytes, 3), sc, ze);
      __stcs(reinterpret_cast<uint2*>(orow + 16 * r), make_uint2(pack16<DTYPE>(x0, x1), pack16<DTYPE>(x2, x3)));
    }
  }
}

// Values of one page: thread item = one 16-byte quad of code words = 8 tokens x 2 * (8 / B) channels that all
// share channel % 8; the elements go through the padded shared tile (conflict-free 2-byte stores) and the tile's
// rows leave with 16-byte stores.
template <int B, int DTYPE>
__device__ __forceinline__ void fast_values(const Geom& g, const uint8_t* __restrict__ pg, uint16_t* tile,
                                            uint16_t* __restrict__ out, int lo, int hi, int tid) {
  constexpr int D = 128, FPB = 8 / B, TS = D + kTilePad;
  constexpr int QPB = D * B / 4;                          // 16-byte quads per 32-token block
  constexpr uint32_t MASK = ((1u << B) - 1u) * 0x01010101u;
  const uint4* codes = reinterpret_cast<const uint4*>(pg + g.v_codes_off);
  const uint32_t* meta = reinterpret_cast<const uint32_t*>(pg + g.v_meta_off);
  const int lgv = ilog2(g.gv), ngv = D >> lgv;
  for (int item = tid; item < 4 * QPB; item += kThreads) {
    const int blk = item / QPB, qi = item % QPB, mw = qi >> 5, lane = qi & 31, gq = lane >> 2, tq = lane & 3;
    const uint4 v = __ldcs(codes + item);
    const uint32_t ww[4] = {v.x, v.y, v.z, v.w};           // sub = 2 rh + kh
#pragma unroll
    for (int kh = 0; kh < 2; ++kh) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int t = blk * 32 + 16 * kh + 2 * tq + (j >> 1) + 8 * (j & 1);
        uint16_t* trow = tile + t * TS + gq;
#pragma unroll
        for (int f = 0; f < FPB; ++f) {
          const int m16 = FPB * mw + f;                   // 16-channel slice
          const uint32_t m = __ldg(meta + t * ngv + ((16 * m16) >> lgv));
          const float sc = meta_scale(m), ze = meta_zero(m);
#pragma unroll
          for (int rh = 0; rh < 2; ++rh) {
            const uint32_t bytes = (ww[2 * rh + kh] >> (B * f)) & MASK;
            trow[16 * m16 + 8 * rh] = one16<DTYPE>(fmaf(code_byte_f32(bytes, j), sc, ze));
          }
        }
      }
    }
  }
  __syncthreads();
  store_rows(tile, TS, out, D, lo, hi, tid);
}

// grid (pages, streams, sides); blockIdx.z + side0: 0 values, 1 keys.
template <int KB, int VB, int DTYPE>
__global__ void __launch_bounds__(kThreads)
dequant_fast_kernel(Geom g, CachePtrs c, uint16_t* k_out, uint16_t* v_out, int t_begin, int t_end, int page0, int side0) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int tid = threadIdx.x;
  const int bh = blockIdx.y, b = bh / g.Hkv;
  const int n = paged_len(c.seq_len, b, g.capacity, g.R);
  const int hi = min(t_end, n);
  const int page = page0 + blockIdx.x;
  const int lo_t = max(t_begin, page * kPageTokens), hi_t = min(hi, page * kPageTokens + kPageTokens);
  if (lo_t >= hi_t) return;
  const uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
  const int lo = lo_t - page * kPageTokens, hi_l = hi_t - page * kPageTokens;
  const size_t out_base = ((size_t)bh * g.capacity + (size_t)page * kPageTokens) * 128;
  if (blockIdx.z + side0 == 0) {
    if constexpr (VB != 0) fast_values<VB, DTYPE>(g, pg, reinterpret_cast<uint16_t*>(smem), v_out + out_base, lo, hi_l, tid);
  } else {
    if constexpr (KB != 0) fast_keys<KB, DTYPE>(g, pg, k_out + out_base, lo, hi_l, tid);
  }
}

template <int KB, int VB>
int launch_fast(const Geom& g, const CachePtrs& c, uint16_t* k_out, uint16_t* v_out, int t_begin, int t_end, int page0,
                int n_pages, int side0, int n_sides, cudaStream_t stream) {
  const size_t smem = (size_t)kPageTokens * (128 + kTilePad) * 2;
  dim3 grid(n_pages, g.B * g.Hkv, n_sides);
  if (g.in_dtype == KVQ_FP16)
    dequant_fast_kernel<KB, VB, KVQ_FP16><<<grid, kThreads, smem, stream>>>(g, c, k_out, v_out, t_begin, t_end, page0, side0);
  else
    dequant_fast_kernel<KB, VB, KVQ_BF16><<<grid, kThreads, smem, stream>>>(g, c, k_out, v_out, t_begin, t_end, page0, side0);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

__global__ void __launch_bounds__(kThreads)
dequant_kernel(Geom g, CachePtrs c, uint16_t* k_out, uint16_t* v_out,
               int t_begin, int t_end, int page0, int side0) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int D = g.D, tid = threadIdx.x;
  uint8_t* spage = smem;
  uint16_t* tile = reinterpret_cast<uint16_t*>(smem + ((g.page_bytes + 15) & ~15));   // [128][D]
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv;
  const int n = paged_len(c.seq_len, b, g.capacity, g.R);      // tokens behind a residual window are in the pages
  const int hi = min(t_end, n);
  const int page = page0 + blockIdx.x;
  const int lo_t = max(t_begin, page * kPageTokens), hi_t = min(hi, page * kPageTokens + kPageTokens);
  if (lo_t >= hi_t) return;
  const int nv = min(kPageTokens, n - page * kPageTokens);
  const uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
  // only this CTA's side of the page: keys [0, v_codes_off), values [v_codes_off, page_bytes)
  const int side = blockIdx.z + side0;
  const int v16_lo = (side == 0 ? g.v_codes_off : 0) / 16;
  const int v16_hi = (side == 0 ? g.page_bytes : g.v_codes_off) / 16;
  for (int i = v16_lo + tid; i < v16_hi; i += kThreads)
    reinterpret_cast<uint4*>(spage)[i] = __ldcs(reinterpret_cast<const uint4*>(pg) + i);
  __syncthreads();
  const int lo = lo_t - page * kPageTokens, hi_l = hi_t - page * kPageTokens;
  const size_t out_base = ((size_t)bh * g.capacity + (size_t)page * kPageTokens) * D;

  // the side: 0 values, 1 keys (two CTAs share a page so that short ranges still fill the GPU)
  if (side == 0) k_out = nullptr; else v_out = nullptr;
  if (v_out) {
    if (g.vb == 16) {
      store_rows(reinterpret_cast<const uint16_t*>(spage + g.v_codes_off), D, v_out + out_base, D, lo, hi_l, tid);
    } else {
      if (is_plane_width(g.vb)) expand_planes(spage, g, true, tile, tid);
      else if (g.vb == 2) expand_values<2>(spage, g, tile, tid);
      else if (g.vb == 4) expand_values<4>(spage, g, tile, tid);
      else expand_values<8>(spage, g, tile, tid);
      __syncthreads();
      store_rows(tile, D + kTilePad, v_out + out_base, D, lo, hi_l, tid);
    }
  }
  if (k_out) {
    const bool tail_k = (g.k_axis == 1) && (nv < kPageTokens);
    if (c.k_signs) {
      const uint16_t* tail = tail_k ? c.k_tail + (size_t)bh * kPageTokens * D : nullptr;
      if (g.kb == 2) dequant_keys_rotated_d<2>(spage, g, tail, c.k_signs, k_out + out_base, lo, hi_l, tid);
      else if (g.kb == 4) dequant_keys_rotated_d<4>(spage, g, tail, c.k_signs, k_out + out_base, lo, hi_l, tid);
      else dequant_keys_rotated_d<8>(spage, g, tail, c.k_signs, k_out + out_base, lo, hi_l, tid);
    } else if (tail_k) {
      // keys of an incomplete channel-wise block live in the fp16 tail
      const uint16_t* tail = c.k_tail + (size_t)bh * kPageTokens * D;
      const int lD = ilog2(D);
      for (int idx = tid; idx < (hi_l - lo) * D; idx += kThreads) {
        const int t = lo + (idx >> lD), d = idx & (D - 1);
        const uint16_t hbits = tail[t * D + d];
        k_out[out_base + (size_t)t * D + d] =
            (g.in_dtype == KVQ_FP16) ? hbits : f32_to_bits16(bits16_to_f32(hbits, KVQ_FP16), KVQ_BF16);
      }
    } else if (g.kb == 16) {
      store_rows(reinterpret_cast<const uint16_t*>(spage), D, k_out + out_base, D, lo, hi_l, tid);
    } else {
      __syncthreads();          // the value tile has been copied out
      if (is_plane_width(g.kb)) expand_planes(spage, g, false, tile, tid);
      else if (g.kb == 2) expand_keys<2>(spage, g, tile, tid);
      else if (g.kb == 4) expand_keys<4>(spage, g, tile, tid);
      else expand_keys<8>(spage, g, tile, tid);
      __syncthreads();
      store_rows(tile, D + kTilePad, k_out + out_base, D, lo, hi_l, tid);
    }
  }
}

// Tokens still in the residual window are the 16-bit inputs themselves: copy their rows out.
__global__ void __launch_bounds__(kThreads)
window_dequant_kernel(Geom g, CachePtrs c, uint16_t* k_out, uint16_t* v_out, int t_begin, int t_end) {
  const int bh = blockIdx.x, b = bh / g.Hkv;
  const int D = g.D, R = g.R, vpr = D / 8;
  const int n = clamped_len(c.seq_len, b, g.capacity);
  const int lo = max(t_begin, (n / R) * R), hi = min(t_end, n);
  for (int idx = threadIdx.x; idx < (hi - lo) * 2 * vpr; idx += kThreads) {
    const int t = lo + idx / (2 * vpr), side = (idx / vpr) & 1, v = idx % vpr;
    uint16_t* dst = side ? v_out : k_out;
    if (!dst) continue;
    reinterpret_cast<uint4*>(dst + ((size_t)bh * g.capacity + t) * D)[v] =
        reinterpret_cast<const uint4*>(c.kv_win + (((size_t)bh * R + (t % R)) * 2 + side) * D)[v];
  }
}

}  // namespace

int launch_dequantize(const Geom& g, const CachePtrs& c, void* k_out, void* v_out, int t_begin, int t_end,
                      cudaStream_t stream) {
  if (t_end <= t_begin) return KVQ_OK;
  const int page0 = t_begin / kPageTokens;
  const int page1 = (t_end + kPageTokens - 1) / kPageTokens;
  const size_t smem = (size_t)((g.page_bytes + 15) & ~15) + (size_t)kPageTokens * (g.D + kTilePad) * 2;
  cudaFuncSetAttribute(dequant_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       128 * 128 * 4 + 128 * (128 + kTilePad) * 2);
  uint16_t* ko = static_cast<uint16_t*>(k_out);
  uint16_t* vo = static_cast<uint16_t*>(v_out);
  const int np = page1 - page0;
  // sides the fast kernel serves (head_dim 128, token-wise groups, 2 / 4 / 8 bits, keys not rotated)
  auto fast_bits = [](int b) { return b == 2 || b == 4 || b == 8; };
  const bool fast_v = vo && g.D == 128 && fast_bits(g.vb);
  const bool fast_k = ko && g.D == 128 && g.k_axis == 0 && !c.k_signs && fast_bits(g.kb);
  int rc = KVQ_OK;
  // A short range (the newest page of every stream in a decode step) is one launch for both sides; a long one
  // keeps a launch per side, where the key CTAs run without the value side's shared-memory tile.
  if (fast_v && fast_k && (long long)np * g.B * g.Hkv <= 148 * 8) {
#define KVQ_DQ_BOTH(KB_, VB_) \
    if (g.kb == KB_ && g.vb == VB_) rc = launch_fast<KB_, VB_>(g, c, ko, vo, t_begin, t_end, page0, np, 0, 2, stream);
    KVQ_DQ_BOTH(2, 2) KVQ_DQ_BOTH(2, 4) KVQ_DQ_BOTH(2, 8)
    KVQ_DQ_BOTH(4, 2) KVQ_DQ_BOTH(4, 4) KVQ_DQ_BOTH(4, 8)
    KVQ_DQ_BOTH(8, 2) KVQ_DQ_BOTH(8, 4) KVQ_DQ_BOTH(8, 8)
#undef KVQ_DQ_BOTH
    if (rc != KVQ_OK) return rc;
    if (g.R)
      window_dequant_kernel<<<g.B * g.Hkv, kThreads, 0, stream>>>(g, c, static_cast<uint16_t*>(k_out),
                                                                  static_cast<uint16_t*>(v_out), t_begin, t_end);
    return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
  }
  if (fast_v) {
    if (g.vb == 2) rc = launch_fast<0, 2>(g, c, ko, vo, t_begin, t_end, page0, np, 0, 1, stream);
    else if (g.vb == 4) rc = launch_fast<0, 4>(g, c, ko, vo, t_begin, t_end, page0, np, 0, 1, stream);
    else rc = launch_fast<0, 8>(g, c, ko, vo, t_begin, t_end, page0, np, 0, 1, stream);
    if (rc != KVQ_OK) return rc;
  }
  if (fast_k) {
    if (g.kb == 2) rc = launch_fast<2, 0>(g, c, ko, vo, t_begin, t_end, page0, np, 1, 1, stream);
    else if (g.kb == 4) rc = launch_fast<4, 0>(g, c, ko, vo, t_begin, t_end, page0, np, 1, 1, stream);
    else rc = launch_fast<8, 0>(g, c, ko, vo, t_begin, t_end, page0, np, 1, 1, stream);
    if (rc != KVQ_OK) return rc;
  }
  // whatever is left goes through the general kernel
  const bool gen_v = vo && !fast_v, gen_k = ko && !fast_k;
  if (gen_v || gen_k) {
    dim3 grid(np, g.B * g.Hkv, (gen_v && gen_k) ? 2 : 1);
    dequant_kernel<<<grid, kThreads, smem, stream>>>(g, c, ko, vo, t_begin, t_end, page0, gen_v ? 0 : 1);
  }
  if (g.R)
    window_dequant_kernel<<<g.B * g.Hkv, kThreads, 0, stream>>>(g, c, static_cast<uint16_t*>(k_out),
                                                                static_cast<uint16_t*>(v_out), t_begin, t_end);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
