// kvq_quantize_append kernels: group-wise asymmetric round-to-nearest
// quantization (App. B.1 quantizer per group; Sec. 4.1 grouping: token-wise
// groups along head_dim, or channel-wise groups over a 128-token block with an
// fp16 residual tail) and packing into the page layout.
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 128;

// One warp quantizes one token row of D elements (token-wise axis) and leaves
// the codes as bytes in `codes` (shared memory) and the (scale, zero) words in
// `meta` (global).  bits == 16: raw copy of the row to `raw_dst`.
__device__ __forceinline__ void quantize_row_warp(const uint16_t* __restrict__ row, int D, int bits, int gsz,
                                                  int dtype, uint8_t* codes, uint32_t* meta,
                                                  uint16_t* raw_dst, int lane) {
  const int epl = D >> 5;  // elements per lane: 2 (D=64) or 4 (D=128)
  uint16_t e[4];
  if (epl == 4) {
    uint2 v = *reinterpret_cast<const uint2*>(row + lane * 4);
    e[0] = v.x & 0xFFFF; e[1] = v.x >> 16; e[2] = v.y & 0xFFFF; e[3] = v.y >> 16;
  } else {
    uint32_t v = *reinterpret_cast<const uint32_t*>(row + lane * 2);
    e[0] = v & 0xFFFF; e[1] = v >> 16; e[2] = e[3] = 0;
  }
  if (bits == 16) {
    for (int i = 0; i < epl; ++i) raw_dst[lane * epl + i] = e[i];
    return;
  }
  float x[4];
  float mn = INFINITY, mx = -INFINITY;
  for (int i = 0; i < epl; ++i) {
    x[i] = bits16_to_f32(e[i], dtype);
    mn = fminf(mn, x[i]);
    mx = fmaxf(mx, x[i]);
  }
  const int lpg = gsz / epl;  // lanes per group
  for (int off = 1; off < lpg; off <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, off));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  }
  const float qmax = (float)((1 << bits) - 1);
  GroupParams p = group_params(mn, mx, qmax);
  if ((lane % lpg) == 0) meta[lane / lpg] = p.meta;
  for (int i = 0; i < epl; ++i) codes[lane * epl + i] = (uint8_t)code_of(x[i], p, qmax);
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

// Token-wise quantization of V (always) and of K (when do_k): one CTA per
// (16-token tile touched, stream).
__global__ void __launch_bounds__(kThreads)
quant_token_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                   int64_t sb, int64_t sh, int64_t st, int t_new, int do_k) {
  __shared__ __align__(16) uint8_t sK[16][128];
  __shared__ __align__(16) uint8_t sV[16][128];
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (t0 + t_new > g.capacity) return;
  const int tile = (t0 >> 4) + blockIdx.x;
  const int tbeg = max(t0, tile * 16), tend = min(t0 + t_new, tile * 16 + 16);
  if (tbeg >= tend) return;
  const int page = tile >> 3;
  uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int D = g.D;

  for (int t = tbeg + warp; t < tend; t += kThreads / 32) {
    const int tau = t & 15, tp = t & 127;
    const int64_t off = (int64_t)b * sb + (int64_t)h * sh + (int64_t)(t - t0) * st;
    quantize_row_warp(v_new + off, D, g.vb, g.gv, g.in_dtype, sV[tau],
                      reinterpret_cast<uint32_t*>(pg + g.v_meta_off) + tp * (D / g.gv),
                      reinterpret_cast<uint16_t*>(pg + g.v_codes_off) + tp * D, lane);
    if (do_k)
      quantize_row_warp(k_new + off, D, g.kb, g.gk, g.in_dtype, sK[tau],
                        reinterpret_cast<uint32_t*>(pg + g.k_meta_off) + tp * (D / g.gk),
                        reinterpret_cast<uint16_t*>(pg) + tp * D, lane);
  }
  __syncthreads();

  const int ntok = tend - tbeg;
  if (do_k && g.kb != 16) pack_k_rows(&sK[tbeg & 15][0], 128, ntok, tbeg & 127, pg, D, g.kb, tid);

  if (g.vb != 16) {
    const int b_ = g.vb;
    const int wpt = D * b_ / 2;     // words per tile
    const int wpc = D * b_ / 64;    // words per chunk
    const int nf = 32 / b_;
    const int lo = tbeg & 15, hi = lo + ntok;   // tile-local token range [lo, hi)
    const bool full = (ntok == 16);
    uint32_t* vt = reinterpret_cast<uint32_t*>(pg + g.v_codes_off + (size_t)(tile & 7) * (16 * D * b_ / 8));
    const uint32_t fm = (1u << b_) - 1u;
    for (int wi = tid; wi < wpt; wi += kThreads) {
      int chunk = wi / wpc, word = wi % wpc;
      uint32_t* wp = vt + chunk_word_byte(chunk, word, wpc, 32) / 4;
      uint32_t w = full ? 0u : *wp;
      for (int f = 0; f < nf; ++f) {
        int tau, d;
        v_field_pos(chunk, word, f, b_, tau, d);
        if (tau >= lo && tau < hi) w = (w & ~(fm << (f * b_))) | ((uint32_t)sV[tau][d] << (f * b_));
      }
      *wp = w;
    }
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
  if (t0 + t_new > g.capacity) return;
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
    const int vec_per_row = D / 8;   // 16-byte vectors
    for (int idx = tid; idx < hi * vec_per_row; idx += kThreads) {
      int slot = idx / vec_per_row, v = idx % vec_per_row;
      uint4 val;
      if (slot < lo) {
        val = *reinterpret_cast<const uint4*>(tail + (size_t)slot * D + v * 8);
      } else {
        const uint16_t* src = k_new + (int64_t)b * sb + (int64_t)h * sh + (int64_t)(tb + slot - t0) * st + v * 8;
        val = *reinterpret_cast<const uint4*>(src);
        if (g.in_dtype == KVQ_BF16) {
          uint32_t* w = reinterpret_cast<uint32_t*>(&val);
          for (int i = 0; i < 4; ++i) {
            uint16_t a = f32_to_fp16_sat_bits(bits16_to_f32(w[i] & 0xFFFF, KVQ_BF16));
            uint16_t bb = f32_to_fp16_sat_bits(bits16_to_f32(w[i] >> 16, KVQ_BF16));
            w[i] = (uint32_t)a | ((uint32_t)bb << 16);
          }
        }
        if (!complete) *reinterpret_cast<uint4*>(tail + (size_t)slot * D + v * 8) = val;
      }
      *reinterpret_cast<uint4*>(sX + (size_t)slot * D + v * 8) = val;
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
  if (t0 + t_new > g.capacity) {
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
  dim3 grid1((t_new + 15) / 16 + 1, g.B * g.Hkv);
  quant_token_kernel<<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new, g.k_axis == 0 ? 1 : 0);
  if (g.k_axis == 1) {
    size_t smem = (size_t)kPageTokens * g.D * 3;
    cudaFuncSetAttribute(quant_kchan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 128 * 3);
    dim3 grid2((t_new + 127) / 128 + 1, g.B * g.Hkv);
    quant_kchan_kernel<<<grid2, kThreads, smem, stream>>>(g, c, k, sb, sh, st, t_new);
  }
  bump_seq_len_kernel<<<(g.B + 127) / 128, 128, 0, stream>>>(g, c, t_new);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
