// kvq_quant_error: the reconstruction-error analysis of the cache quantizer in one pass over new K and V
// (Sec. 4.1 experiment (i); MSE(A, A^) = ||A - A^||_F^2 / entries, App. B.4).  Every token row is quantized in
// registers exactly as kvq_quantize_append would (same group parameters, same codes), reconstructed as
// x^ = fmaf(code, scale, zero) and compared with the input; nothing packed is written.  Per (batch, kv-head)
// the kernel adds sum x^2 and sum (x - x^)^2 of keys and of values to four doubles.
#include <math.h>

#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 256;
constexpr uint32_t FULL = 0xffffffffu;

// One side (keys: blockIdx.z = 0, values: 1).  A row of D channels is spread over D/8 lanes, 8 channels each.
template <int D, int DTYPE>
__global__ void __launch_bounds__(kThreads)
quant_error_kernel(Geom g, const uint16_t* __restrict__ k, const uint16_t* __restrict__ v, int64_t sb, int64_t sh,
                   int64_t st, int n_tokens, double* __restrict__ sums) {
  constexpr int LPR = D / 8, RPW = 32 / LPR;            // lanes per row, rows per warp step
  const int side = blockIdx.z;
  const int bh = blockIdx.y, b = bh / g.Hkv, h = bh % g.Hkv;
  const int bits = side ? g.vb : g.kb, gsz = side ? g.gv : g.gk;
  const uint16_t* in = (side ? v : k) + (int64_t)b * sb + (int64_t)h * sh;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int l = lane % LPR, r0 = lane / LPR;
  const int lpg = gsz >> 3;                              // lanes per group
  const float qmax = (float)((1 << (bits & 15)) - 1);
  double acc2 = 0.0, acce = 0.0;
  const int rows_per_cta_step = (kThreads / 32) * RPW;
  for (int base = blockIdx.x * rows_per_cta_step; base < n_tokens; base += gridDim.x * rows_per_cta_step) {
    const int t = base + warp * RPW + r0;
    const bool valid = t < n_tokens;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (valid) raw = *reinterpret_cast<const uint4*>(in + (int64_t)t * st + 8 * l);
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = bits16_to_f32((uint16_t)(rw[i] & 0xFFFF), DTYPE);
      x[2 * i + 1] = bits16_to_f32((uint16_t)(rw[i] >> 16), DTYPE);
    }
    float s2 = 0.f, se = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s2 = fmaf(x[i], x[i], s2);
    if (bits != 16) {
      float mn = x[0], mx = x[0];
#pragma unroll
      for (int i = 1; i < 8; ++i) { mn = fminf(mn, x[i]); mx = fmaxf(mx, x[i]); }
#pragma unroll
      for (int off = 1; off < 16; off <<= 1) {
        if (off < lpg) {
          mn = fminf(mn, __shfl_xor_sync(FULL, mn, off));
          mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, off));
        }
      }
      const GroupParams p = group_params(mn, mx, qmax);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float xh = __fmaf_rn((float)code_of(x[i], p, qmax), p.s, p.z);
        const float e = __fsub_rn(x[i], xh);
        se = fmaf(e, e, se);
      }
    }
    if (valid) { acc2 += (double)s2; acce += (double)se; }
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    acc2 += __shfl_xor_sync(FULL, acc2, off);
    acce += __shfl_xor_sync(FULL, acce, off);
  }
  if (lane == 0) {
    atomicAdd(sums + (size_t)bh * 4 + 2 * side, acc2);
    atomicAdd(sums + (size_t)bh * 4 + 2 * side + 1, acce);
  }
}

}  // namespace

int launch_quant_error(const Geom& g, const void* k, const void* v, int64_t sb, int64_t sh, int64_t st, int n_tokens,
                       double* sums, cudaStream_t stream) {
  const int streams = g.B * g.Hkv;
  const int rows_per_cta = (kThreads / 32) * (32 / (g.D / 8));
  int gx = (n_tokens + rows_per_cta - 1) / rows_per_cta;
  const int want = (148 * 8 + 2 * streams - 1) / (2 * streams);
  if (gx > want) gx = want;
  if (gx < 1) gx = 1;
  dim3 grid(gx, streams, 2);
  const uint16_t* kk = static_cast<const uint16_t*>(k);
  const uint16_t* vv = static_cast<const uint16_t*>(v);
  if (g.D == 128 && g.in_dtype == KVQ_BF16) quant_error_kernel<128, KVQ_BF16><<<grid, kThreads, 0, stream>>>(g, kk, vv, sb, sh, st, n_tokens, sums);
  else if (g.D == 128) quant_error_kernel<128, KVQ_FP16><<<grid, kThreads, 0, stream>>>(g, kk, vv, sb, sh, st, n_tokens, sums);
  else if (g.in_dtype == KVQ_BF16) quant_error_kernel<64, KVQ_BF16><<<grid, kThreads, 0, stream>>>(g, kk, vv, sb, sh, st, n_tokens, sums);
  else quant_error_kernel<64, KVQ_FP16><<<grid, kThreads, 0, stream>>>(g, kk, vv, sb, sh, st, n_tokens, sums);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
