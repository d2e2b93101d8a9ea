// Generic decode-attention kernel (plain ALU arithmetic, every supported
// configuration) and the split-merge pass.  softmax(q K^T / sqrt(d)) V
// (App. A.1) over the reconstructed cache, one query row per head; the G query
// heads of a KV head share each page read.  The sequence is split over CTAs;
// each writes an unnormalised partial (m, l, o) that the merge pass combines by
// log-sum-exp.
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 128;

// Loop over the G query heads of the group with a compile-time trip count, so
// that per-head arrays stay in registers.
#define KVQ_FOR_HEADS(gh) _Pragma("unroll") for (int gh = 0; gh < kMaxGroupHeads; ++gh) if (gh < G)

__device__ __forceinline__ float meta_scale(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m & 0xFFFF))); }
__device__ __forceinline__ float meta_zero(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m >> 16))); }

// Workspace: float [B*Hq][n_split][D + 2] = (m, l, o[0..D)).
__global__ void __launch_bounds__(kThreads)
decode_generic_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ q, float scale_log2e,
                      float* __restrict__ ws, int n_split) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int D = g.D, G = g.G;
  uint8_t* spage = smem;
  float* sq = reinterpret_cast<float*>(smem + g.page_bytes);   // [G][D], prescaled
  float* sp = sq + G * D;                                      // [G][128] logits, then probabilities
  float* sred = sp + G * kPageTokens;                          // [G] page max
  const int bh = blockIdx.y, split = blockIdx.x;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = clamped_len(c.seq_len, b, g.capacity);
  const int n_pages = (n + kPageTokens - 1) / kPageTokens;
  const int chunk = (n_pages + n_split - 1) / n_split;
  const int p0 = split * chunk, p1 = min(n_pages, p0 + chunk);

  for (int i = tid; i < G * D; i += kThreads) {
    int gh = i / D, d = i % D;
    float v = bits16_to_f32(q[((size_t)b * g.Hq + h * G + gh) * D + d], g.in_dtype) * scale_log2e;
    if (c.k_signs) v *= (float)c.k_signs[d];
    sq[i] = v;
  }
  if (c.k_signs) {
    // rotated keys: q' = H (signs * q) / sqrt(D), butterflies in shared memory
    for (int hh = 1; hh < D; hh <<= 1) {
      __syncthreads();
      for (int i = tid; i < G * D / 2; i += kThreads) {
        const int gh = i / (D / 2), p = i % (D / 2);
        const int d0 = (p / hh) * 2 * hh + (p % hh);
        const float a = sq[gh * D + d0], bq = sq[gh * D + d0 + hh];
        sq[gh * D + d0] = a + bq;
        sq[gh * D + d0 + hh] = a - bq;
      }
    }
    __syncthreads();
    const float inv = rsqrtf((float)D);
    for (int i = tid; i < G * D; i += kThreads) sq[i] *= inv;
  }
  float m[kMaxGroupHeads], l[kMaxGroupHeads], o[kMaxGroupHeads];
  for (int gh = 0; gh < kMaxGroupHeads; ++gh) { m[gh] = -INFINITY; l[gh] = 0.f; o[gh] = 0.f; }
  const int nsub = kThreads / D;           // token subsets in the PV phase (1 or 2)
  const int my_d = tid % D, my_sub = tid / D;
  const uint16_t* tail = g.k_axis == 1 ? c.k_tail + (size_t)bh * kPageTokens * D : nullptr;

  for (int p = p0; p < p1; ++p) {
    const int nv = min(kPageTokens, n - p * kPageTokens);
    const uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + p) * g.page_bytes;
    __syncthreads();
    for (int i = tid; i < g.page_bytes / 16; i += kThreads)
      reinterpret_cast<uint4*>(spage)[i] = reinterpret_cast<const uint4*>(pg)[i];
    __syncthreads();

    // ---- logits: thread = token
    {
      const int tp = tid;
      float acc[kMaxGroupHeads];
      for (int gh = 0; gh < kMaxGroupHeads; ++gh) acc[gh] = 0.f;
      if (tp < nv) {
        const bool tail_k = (g.k_axis == 1) && (nv < kPageTokens);
        if (tail_k || g.kb == 16) {
          const uint16_t* row = tail_k ? tail + tp * D : reinterpret_cast<const uint16_t*>(spage) + tp * D;
          const int dt = tail_k ? KVQ_FP16 : g.in_dtype;
          for (int d = 0; d < D; ++d) {
            float kv = bits16_to_f32(row[d], dt);
            KVQ_FOR_HEADS(gh) acc[gh] = fmaf(sq[gh * D + d], kv, acc[gh]);
          }
        } else if (is_plane_width(g.kb)) {
          const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + g.k_meta_off);
          for (int d = 0; d < D; ++d) {
            uint32_t mm = meta[tp * (D / g.gk) + d / g.gk];
            float kv = fmaf((float)load_code_any(spage, false, tp, d, D, g.kb), meta_scale(mm), meta_zero(mm));
            KVQ_FOR_HEADS(gh) acc[gh] = fmaf(sq[gh * D + d], kv, acc[gh]);
          }
        } else {
          const int bk = g.kb, nf = 32 / bk, wpr = D * bk / 32, wpc = wpr / 4;
          const uint32_t* roww = reinterpret_cast<const uint32_t*>(spage + (size_t)tp * (D * bk / 8));
          const uint32_t* meta = reinterpret_cast<const uint32_t*>(spage + g.k_meta_off);
          for (int wi = 0; wi < wpr; ++wi) {
            int chunkk = wi / wpc, word = wi % wpc;
            uint32_t w = roww[chunk_word_byte(chunkk, word, wpc, 4) / 4];
            for (int f = 0; f < nf; ++f) {
              int d = k_field_channel(chunkk, word, f, bk);
              uint32_t mm = meta[g.k_axis == 1 ? d : tp * (D / g.gk) + d / g.gk];
              float kv = fmaf((float)((w >> (f * bk)) & ((1u << bk) - 1u)), meta_scale(mm), meta_zero(mm));
              KVQ_FOR_HEADS(gh) acc[gh] = fmaf(sq[gh * D + d], kv, acc[gh]);
            }
          }
        }
      }
      KVQ_FOR_HEADS(gh) sp[gh * kPageTokens + tp] = (tp < nv) ? acc[gh] : -INFINITY;
    }
    __syncthreads();
    // ---- page max per head
    for (int gh = warp; gh < G; gh += kThreads / 32) {
      float v = -INFINITY;
      for (int i = lane; i < kPageTokens; i += 32) v = fmaxf(v, sp[gh * kPageTokens + i]);
      for (int off = 16; off; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
      if (lane == 0) sred[gh] = v;
    }
    __syncthreads();
    float alpha[kMaxGroupHeads];
    KVQ_FOR_HEADS(gh) {
      float mn = fmaxf(m[gh], sred[gh]);
      alpha[gh] = exp2f(m[gh] - mn);     // m = -inf at the first page: alpha = 0
      m[gh] = mn;
      sp[gh * kPageTokens + tid] = exp2f(sp[gh * kPageTokens + tid] - mn);   // own element; -inf -> 0
    }
    __syncthreads();
    // ---- PV: thread = (channel, token subset)
    KVQ_FOR_HEADS(gh) { o[gh] *= alpha[gh]; l[gh] *= alpha[gh]; }
    {
      const uint32_t* vmeta = reinterpret_cast<const uint32_t*>(spage + g.v_meta_off);
      for (int tp = my_sub; tp < nv; tp += nsub) {
        float vv;
        if (g.vb == 16) {
          vv = bits16_to_f32(reinterpret_cast<const uint16_t*>(spage + g.v_codes_off)[tp * D + my_d], g.in_dtype);
        } else {
          uint32_t mm = vmeta[tp * (D / g.gv) + my_d / g.gv];
          vv = fmaf((float)load_code_any(spage + g.v_codes_off, true, tp, my_d, D, g.vb), meta_scale(mm), meta_zero(mm));
        }
        KVQ_FOR_HEADS(gh) {
          float pr = sp[gh * kPageTokens + tp];
          o[gh] = fmaf(pr, vv, o[gh]);
          l[gh] += pr;
        }
      }
    }
  }
  // ---- combine token subsets (head_dim 64: two subsets) and write the partial
  __syncthreads();
  float* sx = sp;   // reuse: [G][D] o, then [G] l
  if (nsub == 2) {
    if (my_sub == 1) {
      KVQ_FOR_HEADS(gh) sx[gh * D + my_d] = o[gh];
      if (my_d == 0) { KVQ_FOR_HEADS(gh) sx[G * D + gh] = l[gh]; }
    }
    __syncthreads();
    if (my_sub == 0) {
      KVQ_FOR_HEADS(gh) { o[gh] += sx[gh * D + my_d]; l[gh] += sx[G * D + gh]; }
    }
  }
  if (my_sub == 0) {
    KVQ_FOR_HEADS(gh) {
      float* dst = ws + (((size_t)b * g.Hq + h * G + gh) * n_split + split) * (D + 2);
      if (my_d == 0) { dst[0] = m[gh]; dst[1] = l[gh]; }
      dst[2 + my_d] = o[gh];
    }
  }
}

// out[b,h,:] = sum_j e^(m_j - m*) o_j / sum_j e^(m_j - m*) l_j  (base-2 exponents).
__global__ void merge_kernel(const float* __restrict__ ws, void* __restrict__ out, int out_dtype, int D, int n_split) {
  const int bh = blockIdx.x, d = threadIdx.x;
  const float* base = ws + (size_t)bh * n_split * (D + 2);
  float mstar = -INFINITY;
  for (int j = 0; j < n_split; ++j) mstar = fmaxf(mstar, base[j * (D + 2)]);
  float num = 0.f, den = 0.f;
  if (mstar != -INFINITY) {
    for (int j = 0; j < n_split; ++j) {
      const float* pj = base + j * (D + 2);
      float mj = pj[0];
      if (mj == -INFINITY) continue;
      float w = exp2f(mj - mstar);
      num = fmaf(w, pj[2 + d], num);
      den = fmaf(w, pj[1], den);
    }
  }
  float r = (den > 0.f) ? num / den : 0.f;
  size_t oi = (size_t)bh * D + d;
  if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = r;
  else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(r, out_dtype);
}

}  // namespace

int launch_decode_generic(const Geom& g, const CachePtrs& c, const void* q, float scale_log2e, float* ws,
                          int n_split, cudaStream_t stream) {
  size_t smem = (size_t)g.page_bytes + (size_t)g.G * g.D * 4 + (size_t)g.G * kPageTokens * 4 + 64;
  cudaFuncSetAttribute(decode_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
  dim3 grid(n_split, g.B * g.Hkv);
  decode_generic_kernel<<<grid, kThreads, smem, stream>>>(g, c, static_cast<const uint16_t*>(q), scale_log2e, ws,
                                                          n_split);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

int launch_merge(const Geom& g, const float* ws, void* out, int out_dtype, int n_split, cudaStream_t stream) {
  merge_kernel<<<g.B * g.Hq, g.D, 0, stream>>>(ws, out, out_dtype, g.D, n_split);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
