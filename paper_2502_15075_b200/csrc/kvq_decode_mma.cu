// Dispatch of the fast decode path and its merge pass.
#include "kvq_decode_mma_kernel.cuh"

namespace kvq {
namespace mma {

// Instantiation units (kvq_decode_mma_inst_*.cu).
#define KVQ_MMA_DECL(D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB)                                                  \
  extern template int launch_mma_inst<D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB>(const Geom&, const CachePtrs&,     \
                                                                                 const void*, float, float*, int, \
                                                                                 cudaStream_t);
#include "kvq_decode_mma_list.inc"
#undef KVQ_MMA_DECL

// out[b,h,:] = sum_j 2^(m_j - m*) o_j / sum_j 2^(m_j - m*) l_j over the slots the flat split gave this stream.
__global__ void merge_flat_kernel(Geom g, const int32_t* __restrict__ seq_len, const float* __restrict__ ws,
                                  void* __restrict__ out, int out_dtype, int grid, int s_cap) {
  const int bh = blockIdx.x, d = threadIdx.x;
  const int b = bh / g.Hq, hq = bh % g.Hq;
  const int h = hq / g.G, gh = hq % g.G;
  const int D = g.D;
  long long N = 0, before = 0;
  int pages_max = 0, pages_b = 0;
  for (int i = 0; i < g.B; ++i) {
    int p = (clamped_len(seq_len, i, g.capacity) + kPageTokens - 1) >> 7;
    if (i < b) before += p;
    if (i == b) pages_b = p;
    N += p;
    pages_max = max(pages_max, p);
  }
  N *= g.Hkv;
  before *= g.Hkv;
  float r = 0.f;
  if (pages_b > 0) {
    const FlatPlan plan = make_plan(N, pages_max, grid, s_cap);
    const long long xs = before + (long long)h * pages_b;
    const int c_first = plan.cta_of(xs), c_last = plan.cta_of(xs + pages_b - 1);
    const int n = min(c_last - c_first + 1, s_cap);
    const float* base = ws + (((size_t)(b * g.Hkv + h) * s_cap) * g.G + gh) * (D + 2);
    const size_t slot_stride = (size_t)g.G * (D + 2);
    // slots are few: issue all loads of a batch of 8 before using any (the merge is latency-bound)
    float mstar = -INFINITY, num = 0.f, den = 0.f;
    for (int j0 = 0; j0 < n; j0 += 8) {
      float mj[8], lj[8], oj[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const bool on = j0 + u < n;
        const float* pj = base + (size_t)(on ? j0 + u : 0) * slot_stride;
        mj[u] = on ? pj[0] : -INFINITY;
        lj[u] = on ? pj[1] : 0.f;
        oj[u] = on ? pj[2 + d] : 0.f;
      }
      float mb = mstar;
#pragma unroll
      for (int u = 0; u < 8; ++u) mb = fmaxf(mb, mj[u]);
      if (mb == -INFINITY) continue;
      const float keep = (mstar == -INFINITY) ? 0.f : exp2f(mstar - mb);
      num *= keep;
      den *= keep;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float w = (mj[u] == -INFINITY) ? 0.f : exp2f(mj[u] - mb);
        num = fmaf(w, oj[u], num);
        den = fmaf(w, lj[u], den);
      }
      mstar = mb;
    }
    r = den > 0.f ? num / den : 0.f;
  }
  const size_t oi = (size_t)bh * D + d;
  if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = r;
  else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(r, out_dtype);
}

}  // namespace mma

constexpr int kFlatGrid = 2 * 148;   // slot capacity is sized for grids up to twice this

int flat_slot_cap(const Geom& g) {
  const int streams = g.B * g.Hkv;
  int s = (2 * kFlatGrid + streams - 1) / streams + 2;
  if (s > g.n_pages + 1) s = g.n_pages + 1;
  return s;
}

size_t flat_workspace_bytes(const Geom& g) {
  return (size_t)g.B * g.Hkv * flat_slot_cap(g) * g.G * (g.D + 2) * sizeof(float);
}

// Finds the instantiation for this geometry; launches it unless `probe`.  *grid = CTAs of the launch.
static int pick(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap,
                cudaStream_t stream, bool probe, int* grid) {
  const int ngk = (g.k_axis == 1 || g.kb == 16) ? 1 : g.D / g.gk;
  const int ngv = (g.vb == 16) ? 1 : g.D / g.gv;
  const int nh = g.G <= 4 ? 1 : 2;                                         // query heads per lane
#define KVQ_MMA_DECL(D_, KB_, VB_, KAXIS_, NGK_, NGV_, NH_, NW_, MINB_)                                      \
  if (g.D == D_ && g.kb == KB_ && g.vb == VB_ && g.k_axis == KAXIS_ && ngk == NGK_ && ngv == NGV_ &&          \
      NH_ == nh) {                                                                                            \
    *grid = 148 * MINB_;                                                                                      \
    if (probe) return KVQ_OK;                                                                                 \
    return mma::launch_mma_inst<D_, KB_, VB_, KAXIS_, NGK_, NGV_, NH_, NW_, MINB_>(g, c, q, c1, ws, s_cap,    \
                                                                                   stream);                  \
  }
#include "kvq_decode_mma_list.inc"
#undef KVQ_MMA_DECL
  return KVQ_ERR_UNSUPPORTED;
}

bool decode_mma_supported(const Geom& g) {
  if (g.B > mma::kMaxBatchFlat) return false;
  CachePtrs none{};
  int grid = 0;
  return pick(g, none, nullptr, 0.f, nullptr, 0, nullptr, true, &grid) == KVQ_OK;
}

int launch_decode_mma(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype, float c1,
                      float* ws, cudaStream_t stream) {
  const int s_cap = flat_slot_cap(g);
  int grid = 0;
  int rc = pick(g, c, q, c1, ws, s_cap, stream, false, &grid);
  if (rc != KVQ_OK) return rc;
  mma::merge_flat_kernel<<<g.B * g.Hq, g.D, 0, stream>>>(g, c.seq_len, ws, out, out_dtype, grid, s_cap);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
