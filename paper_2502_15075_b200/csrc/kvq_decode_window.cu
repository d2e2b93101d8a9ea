// Decode attention over the residual window (Sec. 4.1's buffer of recent full-precision tokens): the newest
// seq_len % R tokens of a stream are 16-bit rows in a ring, not pages.  One CTA per (batch, kv-head) stream computes
// softmax-attention partials (m, l, o) of all (row, head) pairs over those at most R - 1 tokens in fp32 and leaves
// them in the stream's last partial slot, where the main kernel's merge picks them up; a stream without pages gets
// its output written here.  The work is tiny (R - 1 tokens), plain ALU code is enough.
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 128;
constexpr int kMaxVH = kMaxGroupHeads;      // (row, head) pairs per KV head

__global__ void __launch_bounds__(kThreads)
decode_window_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ q, float c1, float* __restrict__ ws, int s_cap,
                     void* __restrict__ out, int out_dtype) {
  __shared__ float sq[kMaxVH][128];          // queries, prescaled (softmax scale * log2 e)
  __shared__ float sp[kMaxVH][128];          // logits, then weights
  __shared__ float sm[kMaxVH], sl[kMaxVH];
  const int stream = blockIdx.x, b = stream / g.Hkv, h = stream % g.Hkv;
  const int D = g.D, R = g.R, Gq = g.G, VH = g.G * g.rows;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = clamped_len(c.seq_len, b, g.capacity);
  const int f = (n / R) * R, nw = n - f;     // tokens f .. n-1 are in the window
  auto out_index = [&](int vh, int d) {
    return (((size_t)b * g.rows + vh / Gq) * g.Hq + (size_t)h * Gq + vh % Gq) * D + d;
  };
  auto store_out = [&](size_t oi, float r) {
    if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = r;
    else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(r, out_dtype);
  };
  if (nw == 0) {
    if (n == 0) {                            // an empty sequence: zeros
      for (int idx = tid; idx < VH * D; idx += kThreads) store_out(out_index(idx / D, idx % D), 0.f);
    }
    return;
  }
  for (int idx = tid; idx < VH * D; idx += kThreads) {
    const int vh = idx / D, d = idx % D;
    const uint16_t* qrow = q + (((size_t)b * g.rows + vh / Gq) * g.Hq + (size_t)h * Gq + vh % Gq) * D;
    sq[vh][d] = bits16_to_f32(qrow[d], g.in_dtype) * c1;
  }
  __syncthreads();
  const uint16_t* win = c.kv_win + (size_t)stream * R * 2 * D;
  for (int idx = tid; idx < VH * nw; idx += kThreads) {
    const int vh = idx / nw, i = idx % nw, t = f + i;
    const int limit = n - (g.rows - 1 - vh / Gq);          // causal limit of the pair's query row
    float acc = -INFINITY;
    if (t < limit) {
      const uint16_t* krow = win + (size_t)(t % R) * 2 * D;
      acc = 0.f;
      for (int d = 0; d < D; ++d) acc = fmaf(sq[vh][d], bits16_to_f32(krow[d], g.in_dtype), acc);
    }
    sp[vh][i] = acc;
  }
  __syncthreads();
  for (int vh = warp; vh < VH; vh += kThreads / 32) {
    float m = -INFINITY;
    for (int i = lane; i < nw; i += 32) m = fmaxf(m, sp[vh][i]);
    for (int off = 16; off; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    float l = 0.f;
    for (int i = lane; i < nw; i += 32) {
      const float p = (m == -INFINITY) ? 0.f : exp2f(sp[vh][i] - m);
      sp[vh][i] = p;
      l += p;
    }
    for (int off = 16; off; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
    if (lane == 0) { sm[vh] = m; sl[vh] = l; }
  }
  __syncthreads();
  for (int idx = tid; idx < VH * D; idx += kThreads) {
    const int vh = idx / D, d = idx % D;
    float o = 0.f;
    for (int i = 0; i < nw; ++i)
      o = fmaf(sp[vh][i], bits16_to_f32(win[((size_t)((f + i) % R) * 2 + 1) * D + d], g.in_dtype), o);
    if (f == 0) {                            // no pages at all: this is the whole attention
      store_out(out_index(vh, d), sl[vh] > 0.f ? o / sl[vh] : 0.f);
    } else {
      float* dst = ws + (((size_t)stream * s_cap + (s_cap - 1)) * VH + vh) * (D + 2);
      if (d == 0) { dst[0] = sm[vh]; dst[1] = sl[vh]; }
      dst[2 + d] = o;
    }
  }
}

}  // namespace

int launch_decode_window(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype, float c1,
                         float* ws, int s_cap, cudaStream_t stream) {
  decode_window_kernel<<<g.B * g.Hkv, kThreads, 0, stream>>>(g, c, static_cast<const uint16_t*>(q), c1, ws, s_cap, out,
                                                             out_dtype);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
