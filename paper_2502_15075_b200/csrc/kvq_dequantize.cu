// kvq_dequantize kernel: x^ = fmaf(code, scale, zero) rounded to the 16-bit
// input type (App. B.1: A^ = scale * Q, here with the group minimum as offset).
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
dequant_kernel(Geom g, CachePtrs c, uint16_t* __restrict__ k_out, uint16_t* __restrict__ v_out,
               int t_begin, int t_end, int page0) {
  extern __shared__ __align__(16) uint8_t spage[];
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv;
  const int n = c.seq_len[b];
  const int hi = min(t_end, n);
  const int page = page0 + blockIdx.x;
  const int lo_t = max(t_begin, page * kPageTokens), hi_t = min(hi, page * kPageTokens + kPageTokens);
  if (lo_t >= hi_t) return;
  const int nv = min(kPageTokens, n - page * kPageTokens);
  const int D = g.D, tid = threadIdx.x;
  const uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
  for (int i = tid; i < g.page_bytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(spage)[i] = reinterpret_cast<const uint4*>(pg)[i];
  __syncthreads();
  const bool tail_k = (g.k_axis == 1) && (nv < kPageTokens);
  const uint16_t* tail = tail_k ? c.k_tail + (size_t)bh * kPageTokens * D : nullptr;
  const size_t out_base = (size_t)bh * g.capacity * D;

  for (int idx = tid; idx < (hi_t - lo_t) * D; idx += kThreads) {
    const int t = lo_t + idx / D, d = idx % D;
    const int tp = t - page * kPageTokens;
    if (v_out) {
      uint16_t r;
      if (g.vb == 16) {
        r = reinterpret_cast<const uint16_t*>(spage + g.v_codes_off)[tp * D + d];
      } else {
        int wb, bit;
        v_code_pos(tp, d, D, g.vb, wb, bit);
        float code = (float)load_code(spage + g.v_codes_off, wb, bit, g.vb);
        uint32_t m = reinterpret_cast<const uint32_t*>(spage + g.v_meta_off)[tp * (D / g.gv) + d / g.gv];
        float s = __half2float(__ushort_as_half((uint16_t)(m & 0xFFFF)));
        float z = __half2float(__ushort_as_half((uint16_t)(m >> 16)));
        r = f32_to_bits16(fmaf(code, s, z), g.in_dtype);
      }
      v_out[out_base + (size_t)t * D + d] = r;
    }
    if (k_out) {
      uint16_t r;
      if (tail_k) {
        uint16_t hbits = tail[tp * D + d];
        r = (g.in_dtype == KVQ_FP16) ? hbits : f32_to_bits16(bits16_to_f32(hbits, KVQ_FP16), KVQ_BF16);
      } else if (g.kb == 16) {
        r = reinterpret_cast<const uint16_t*>(spage)[tp * D + d];
      } else {
        int wb, bit;
        k_code_pos(tp, d, D, g.kb, wb, bit);
        float code = (float)load_code(spage, wb, bit, g.kb);
        int mi = (g.k_axis == 1) ? d : tp * (D / g.gk) + d / g.gk;
        uint32_t m = reinterpret_cast<const uint32_t*>(spage + g.k_meta_off)[mi];
        float s = __half2float(__ushort_as_half((uint16_t)(m & 0xFFFF)));
        float z = __half2float(__ushort_as_half((uint16_t)(m >> 16)));
        r = f32_to_bits16(fmaf(code, s, z), g.in_dtype);
      }
      k_out[out_base + (size_t)t * D + d] = r;
    }
  }
}

}  // namespace

int launch_dequantize(const Geom& g, const CachePtrs& c, void* k_out, void* v_out, int t_begin, int t_end,
                      cudaStream_t stream) {
  if (t_end <= t_begin) return KVQ_OK;
  const int page0 = t_begin / kPageTokens;
  const int page1 = (t_end + kPageTokens - 1) / kPageTokens;
  cudaFuncSetAttribute(dequant_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 128 * 4);
  dim3 grid(page1 - page0, g.B * g.Hkv);
  dequant_kernel<<<grid, kThreads, g.page_bytes, stream>>>(g, c, static_cast<uint16_t*>(k_out),
                                                           static_cast<uint16_t*>(v_out), t_begin, t_end, page0);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
