// kvq_quantize_append kernels: group-wise asymmetric round-to-nearest
// quantization (App. B.1 quantizer per group; Sec. 4.1 grouping: token-wise
// groups along head_dim, or channel-wise groups over a 128-token block with an
// fp16 residual tail) and packing into the page layout.
//
// Token-wise kernel: one warp per 16-token tile of one stream.  Every lane loads
// 16 bytes (8 consecutive channels of one token), groups reduce min/max with
// shuffles, the 8 codes of a lane are merged into at most four partial words and
// OR-ed into an image of the packed tile in shared memory, and the finished image
// leaves with 16-byte coalesced stores.  The kernel is bound by reading the 16-bit
// inputs from HBM.
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t FULL = 0xffffffffu;

// Quantize one side (keys or values) of a 16-token tile held in global memory as rows of D 16-bit values.
// `img` is the warp's shared-memory image of the packed codes of the tile: for keys 16 token rows of
// D*BITS/8 bytes, for values the tile's D*BITS*2 bytes.  Tokens outside [lo, hi) are left alone.
template <int BITS, bool IS_V, int D, int DTYPE, bool ROT>
__device__ __forceinline__ void quantize_tile_side(const uint16_t* __restrict__ src, int64_t st, int gsz,
                                                   int lo, int hi, uint32_t* img,
                                                   uint32_t* __restrict__ meta_out, bool clear_first, int lane,
                                                   const int8_t* __restrict__ signs) {
  constexpr int lpr = D >> 3;                // lanes per token row (8 channels each)
  constexpr int rps = 32 / lpr;              // rows per step
  const int l = lane & (lpr - 1);
  const int d0 = l * 8;
  const int lpg = gsz >> 3;                  // lanes per group
  const int ng = D / gsz;
  const float qmax = (float)((1 << BITS) - 1);
#pragma unroll 4
  for (int step = 0; step < 16 / rps; ++step) {
    if (step * rps + rps <= lo || step * rps >= hi) continue;      // no new token in this step's rows (warp-uniform)
    const int tau = step * rps + lane / lpr;
    const bool valid = tau >= lo && tau < hi;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (valid) raw = *reinterpret_cast<const uint4*>(src + (int64_t)tau * st + d0);
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if constexpr (DTYPE == KVQ_BF16) {
        x[2 * i] = __uint_as_float(rw[i] << 16);
        x[2 * i + 1] = __uint_as_float(rw[i] & 0xFFFF0000u);
      } else {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&rw[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
      }
    }
    if constexpr (ROT) rotate_row8<D>(x, signs, l);      // keys only: y = H (signs * x) / sqrt(D)
    float mn = INFINITY, mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      mn = fminf(mn, x[i]);
      mx = fmaxf(mx, x[i]);
    }
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) {
      if (off < lpg) {
        mn = fminf(mn, __shfl_xor_sync(FULL, mn, off));
        mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, off));
      }
    }
    const GroupParams p = group_params(mn, mx, qmax);
    if (!valid) continue;
    if ((l & (lpg - 1)) == 0) meta_out[tau * ng + d0 / gsz] = p.meta;
    uint32_t code[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) code[i] = code_of_fast(x[i], p, qmax);

    if constexpr (!IS_V) {
      // keys: channels d0..d0+3 and d0+4..d0+7 are the four bytes of one word each (chunks 2(l%2), 2(l%2)+1),
      // register slot r = d0/16, field r % fpb of every byte
      constexpr int FPB = 8 / BITS;
      const int wpc = D * BITS / 128;
      const int r = l >> 1;
      const int sh = BITS * (r % FPB);
      const int word = r / FPB;
      const int row_words = D * BITS / 32;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const uint32_t w = (code[4 * hh] | (code[4 * hh + 1] << 8) | (code[4 * hh + 2] << 16) |
                            (code[4 * hh + 3] << 24)) << sh;
        const int chunk = 2 * (l & 1) + hh;
        atomicOr(&img[tau * row_words + chunk_word_byte(chunk, word, wpc, 4) / 4], w);
      }
    } else {
      // values: the lane's 8 channels d0 + kk belong to one lane-chunk group gidc = (d0/8) % 8, k = 8 (d0/64) + kk
      constexpr int PPW = 16 / BITS;
      const int wpc = D * BITS / 64;
      const int gidc = l & 7, h = l >> 3;            // d0 = 64 h + 8 gidc
      const int tidT = (tau & 7) >> 1, hiT = tau >> 3, oddT = tau & 1;
      const int chunk = 4 * gidc + tidT;
      constexpr int NWORD = BITS;                    // words this lane contributes to (8 codes, 8/BITS per word)
      uint32_t part[NWORD], mask[NWORD];
      int widx[NWORD];
#pragma unroll
      for (int i = 0; i < NWORD; ++i) { part[i] = 0; mask[i] = 0; widx[i] = 0; }
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        constexpr int NPOS = 8 / BITS;
        const int k = 8 * h + kk;
        const int word = k / NPOS;
        const int field = k % NPOS + NPOS * hiT + PPW * oddT;
        const int wo = kk / NPOS;
        widx[wo] = word;
        part[wo] |= code[kk] << (field * BITS);
        mask[wo] |= ((1u << BITS) - 1u) << (field * BITS);
      }
#pragma unroll
      for (int i = 0; i < NWORD; ++i) {
        uint32_t* dst = &img[chunk_word_byte(chunk, widx[i], wpc, 32) / 4];
        if (clear_first) atomicAnd(dst, ~mask[i]);
        atomicOr(dst, part[i]);
      }
    }
  }
}

// 16-bit passthrough of one side of a tile: rows [lo, hi) copied to the page as they are.
__device__ __forceinline__ void copy_tile_side(const uint16_t* __restrict__ src, int64_t st, int D, int lo, int hi,
                                               uint16_t* __restrict__ dst_rows, int lane) {
  const int lpr = D >> 3, rps = 32 / lpr, l = lane & (lpr - 1);
  for (int step = 0; step < 16 / rps; ++step) {
    if (step * rps + rps <= lo || step * rps >= hi) continue;
    const int tau = step * rps + lane / lpr;
    if (tau >= lo && tau < hi)
      *reinterpret_cast<uint4*>(dst_rows + (size_t)tau * D + l * 8) =
          *reinterpret_cast<const uint4*>(src + (int64_t)tau * st + l * 8);
  }
}

template <bool IS_V, int D, int DTYPE, bool ROT>
__device__ __forceinline__ void quantize_tile_side_bits(int bits, const uint16_t* src, int64_t st, int gsz,
                                                        int lo, int hi, uint32_t* img, uint32_t* meta_out,
                                                        bool clear_first, int lane, const int8_t* signs) {
  if (bits == 2)
    quantize_tile_side<2, IS_V, D, DTYPE, ROT>(src, st, gsz, lo, hi, img, meta_out, clear_first, lane, signs);
  else if (bits == 4)
    quantize_tile_side<4, IS_V, D, DTYPE, ROT>(src, st, gsz, lo, hi, img, meta_out, clear_first, lane, signs);
  else
    quantize_tile_side<8, IS_V, D, DTYPE, ROT>(src, st, gsz, lo, hi, img, meta_out, clear_first, lane, signs);
}

// Token-wise quantization of V (always) and of K (when do_k).  grid.y = stream, grid.x strides over the
// 16-token tiles touched by this append, one warp per tile.
template <int D, int DTYPE>
__global__ void __launch_bounds__(kThreads)
quant_token_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                   int64_t sb, int64_t sh, int64_t st, int t_new, int do_k) {
  __shared__ __align__(16) uint32_t sImg[kWarps][2][512];   // per warp: key image, value image (<= 2 KB each)
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (t0 < 0 || t0 + t_new > g.capacity) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int first_tile = t0 >> 4;
  const int n_tiles = ((t0 + t_new + 15) >> 4) - first_tile;
  uint32_t* kimg = sImg[warp][0];
  uint32_t* vimg = sImg[warp][1];
  const int k_row_words = D * g.kb / 32;          // words per key row (quantized)
  const int v_tile_words = D * g.vb / 2;          // words per value tile (quantized)

  for (int j = blockIdx.x * kWarps + warp; j < n_tiles; j += gridDim.x * kWarps) {
    const int tile = first_tile + j;
    const int tbeg = max(t0, tile * 16), tend = min(t0 + t_new, tile * 16 + 16);
    const int lo = tbeg & 15, hi = lo + (tend - tbeg);
    const bool full = (hi - lo) == 16;
    const int page = tile >> 3, tp0 = (tile & 7) * 16;        // page-local token of the tile's first row
    uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
    // row 0 of the tile in the input (may lie before the first new token; never dereferenced there)
    const int64_t off = (int64_t)b * sb + (int64_t)h * sh + (int64_t)(tile * 16 - t0) * st;

    // ---- values
    if (g.vb == 16) {
      copy_tile_side(v_new + off, st, D, lo, hi, reinterpret_cast<uint16_t*>(pg + g.v_codes_off) + (size_t)tp0 * D, lane);
    } else {
      uint4* gv = reinterpret_cast<uint4*>(pg + g.v_codes_off + (size_t)(tile & 7) * (v_tile_words * 4));
      for (int i = lane; i < v_tile_words / 4; i += 32)
        reinterpret_cast<uint4*>(vimg)[i] = full ? make_uint4(0u, 0u, 0u, 0u) : gv[i];
      __syncwarp();
      quantize_tile_side_bits<true, D, DTYPE, false>(g.vb, v_new + off, st, g.gv, lo, hi, vimg,
                                    reinterpret_cast<uint32_t*>(pg + g.v_meta_off) + tp0 * (D / g.gv), !full, lane,
                                    nullptr);
      __syncwarp();
      for (int i = lane; i < v_tile_words / 4; i += 32) gv[i] = reinterpret_cast<const uint4*>(vimg)[i];
    }
    // ---- keys
    if (do_k) {
      if (g.kb == 16) {
        copy_tile_side(k_new + off, st, D, lo, hi, reinterpret_cast<uint16_t*>(pg) + (size_t)tp0 * D, lane);
      } else {
        for (int i = lane; i < 16 * k_row_words / 4; i += 32) reinterpret_cast<uint4*>(kimg)[i] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
        uint32_t* kmeta = reinterpret_cast<uint32_t*>(pg + g.k_meta_off) + tp0 * (D / g.gk);
        if (c.k_signs)
          quantize_tile_side_bits<false, D, DTYPE, true>(g.kb, k_new + off, st, g.gk, lo, hi, kimg, kmeta, false,
                                                         lane, c.k_signs);
        else
          quantize_tile_side_bits<false, D, DTYPE, false>(g.kb, k_new + off, st, g.gk, lo, hi, kimg, kmeta, false,
                                                          lane, nullptr);
        __syncwarp();
        uint4* gk = reinterpret_cast<uint4*>(pg + (size_t)tp0 * (k_row_words * 4));
        const int v_lo = lo * k_row_words / 4, v_hi = hi * k_row_words / 4;   // 16-byte vectors of the new rows
        for (int i = v_lo + lane; i < v_hi; i += 32) gk[i] = reinterpret_cast<const uint4*>(kimg)[i];
      }
    }
    __syncwarp();
  }
}

// Pack K rows: `codes` holds bytes [ntok rows][D]; row r goes to page-local token slot0 + r.
__device__ __forceinline__ void pack_k_rows(const uint8_t* codes, int code_stride, int ntok, int slot0,
                                            uint8_t* kregion, int D, int b, int tid) {
  const int wpr = D * b / 32;    // words per row
  const int wpc = wpr / 4;       // words per chunk
  const int nf = 32 / b;
  for (int idx = tid; idx < ntok * wpr; idx += kThreads) {
    int r = idx / wpr, wi = idx % wpr;
    int chunk = wi / wpc, word = wi % wpc;
    uint32_t w = 0;
    for (int f = 0; f < nf; ++f) {
      int d = k_field_channel(chunk, word, f, b);
      w |= (uint32_t)codes[r * code_stride + d] << (f * b);
    }
    *reinterpret_cast<uint32_t*>(kregion + (size_t)(slot0 + r) * (D * b / 8) + chunk_word_byte(chunk, word, wpc, 4)) = w;
  }
}

// Channel-wise quantization of K over 128-token blocks with the fp16 tail.
// CTA j of a stream handles the j-th block touched by this append.  CTA 0 also
// handles the final block when that one is incomplete (it writes the tail, which
// CTA 0 must have finished reading first).
__global__ void __launch_bounds__(kThreads)
quant_kchan_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new,
                   int64_t sb, int64_t sh, int64_t st, int t_new) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int D = g.D;
  uint16_t* sX = reinterpret_cast<uint16_t*>(smem);          // [128][D] fp16 bits
  uint8_t* sC = smem + (size_t)kPageTokens * D * 2;           // [128][D] codes
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (t0 < 0 || t0 + t_new > g.capacity) return;
  const int end = t0 + t_new;
  const int first_page = t0 >> 7;
  const int nblk = ((end + 127) >> 7) - first_page;
  const bool last_partial = (end & 127) != 0;
  const int tid = threadIdx.x;
  uint16_t* tail = c.k_tail + (size_t)bh * kPageTokens * D;
  const float qmax = (float)((1 << g.kb) - 1);

  for (int pass = 0; pass < 2; ++pass) {
    int j;
    if (pass == 0) {
      j = blockIdx.x;
      if (j >= nblk) return;
      if (j == nblk - 1 && last_partial && j != 0) return;   // done by CTA 0 in its second pass
    } else {
      if (blockIdx.x != 0 || nblk <= 1 || !last_partial) return;
      j = nblk - 1;
      __syncthreads();
    }
    const int page = first_page + j;
    const int tb = page << 7;
    const int lo = max(t0, tb) - tb, hi = min(end, tb + 128) - tb;   // new tokens occupy slots [lo, hi)
    const bool complete = (hi == 128);
    // gather the block: slots [0, lo) from the tail, [lo, hi) from the input (as saturated fp16)
    // (a row is handled by D/8 consecutive lanes, which is what the rotation's shuffles expect; every lane of a
    // warp runs the loop body, rows past the end are inactive)
    const int vec_per_row = D / 8;   // 16-byte vectors
    for (int base = 0; base < hi * vec_per_row; base += kThreads) {
      const int idx = base + tid;
      const bool active = idx < hi * vec_per_row;
      const int slot = idx / vec_per_row, v = idx % vec_per_row;
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      const bool is_new = active && slot >= lo;
      if (active && !is_new) val = *reinterpret_cast<const uint4*>(tail + (size_t)slot * D + v * 8);
      if (is_new)
        val = *reinterpret_cast<const uint4*>(k_new + (int64_t)b * sb + (int64_t)h * sh +
                                              (int64_t)(tb + slot - t0) * st + v * 8);
      if (c.k_signs != nullptr || g.in_dtype == KVQ_BF16) {
        // new tokens: to fp32, rotate if asked, store as saturated fp16
        uint32_t* w = reinterpret_cast<uint32_t*>(&val);
        float x[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[2 * i] = bits16_to_f32((uint16_t)(w[i] & 0xFFFF), g.in_dtype);
          x[2 * i + 1] = bits16_to_f32((uint16_t)(w[i] >> 16), g.in_dtype);
        }
        if (c.k_signs != nullptr) {
          if (D == 128) rotate_row8<128>(x, c.k_signs, v); else rotate_row8<64>(x, c.k_signs, v);
        }
        if (is_new) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
            w[i] = (uint32_t)f32_to_fp16_sat_bits(x[2 * i]) | ((uint32_t)f32_to_fp16_sat_bits(x[2 * i + 1]) << 16);
        }
      }
      if (is_new && !complete) *reinterpret_cast<uint4*>(tail + (size_t)slot * D + v * 8) = val;
      if (active) *reinterpret_cast<uint4*>(sX + (size_t)slot * D + v * 8) = val;
    }
    if (!complete) continue;
    __syncthreads();
    uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
    for (int d = tid; d < D; d += kThreads) {
      float mn = INFINITY, mx = -INFINITY;
      for (int t = 0; t < kPageTokens; ++t) {
        float x = bits16_to_f32(sX[t * D + d], KVQ_FP16);
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
      GroupParams p = group_params(mn, mx, qmax);
      reinterpret_cast<uint32_t*>(pg + g.k_meta_off)[d] = p.meta;
      for (int t = 0; t < kPageTokens; ++t)
        sC[t * D + d] = (uint8_t)code_of(bits16_to_f32(sX[t * D + d], KVQ_FP16), p, qmax);
    }
    __syncthreads();
    pack_k_rows(sC, D, kPageTokens, 0, pg, D, g.kb, tid);
  }
}

__global__ void bump_seq_len_kernel(Geom g, CachePtrs c, int t_new) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= g.B) return;
  int t0 = c.seq_len[b];
  if (t0 < 0 || t0 + t_new > g.capacity) {
    atomicOr(c.status, KVQ_STATUS_CAPACITY);
  } else {
    c.seq_len[b] = t0 + t_new;
  }
}

}  // namespace

int launch_quantize_append(const Geom& g, const CachePtrs& c, const void* k_new, const void* v_new,
                           int64_t sb, int64_t sh, int64_t st, int t_new, cudaStream_t stream) {
  const uint16_t* k = static_cast<const uint16_t*>(k_new);
  const uint16_t* v = static_cast<const uint16_t*>(v_new);
  // tiles touched per stream: at most ceil(t_new / 16) + 1; one warp per tile, CTAs stride over them
  const int max_tiles = (t_new + 15) / 16 + 1;
  int gx = (max_tiles + kWarps - 1) / kWarps;
  const int streams = g.B * g.Hkv;
  const int want = (148 * 16 + streams - 1) / streams;       // enough CTAs to fill the GPU, not one per tile
  if (gx > want) gx = want;
  dim3 grid1(gx, streams);
  const int do_k = g.k_axis == 0 ? 1 : 0;
  if (g.D == 128 && g.in_dtype == KVQ_BF16)
    quant_token_kernel<128, KVQ_BF16><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new, do_k);
  else if (g.D == 128)
    quant_token_kernel<128, KVQ_FP16><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new, do_k);
  else if (g.in_dtype == KVQ_BF16)
    quant_token_kernel<64, KVQ_BF16><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new, do_k);
  else
    quant_token_kernel<64, KVQ_FP16><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new, do_k);
  if (g.k_axis == 1) {
    size_t smem = (size_t)kPageTokens * g.D * 3;
    cudaFuncSetAttribute(quant_kchan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 128 * 3);
    dim3 grid2((t_new + 127) / 128 + 1, streams);
    quant_kchan_kernel<<<grid2, kThreads, smem, stream>>>(g, c, k, sb, sh, st, t_new);
  }
  bump_seq_len_kernel<<<(g.B + 127) / 128, 128, 0, stream>>>(g, c, t_new);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
