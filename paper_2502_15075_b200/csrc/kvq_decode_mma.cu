// Dispatch of the fast decode path (the merge of the split partials is part of the kernel).
#include <atomic>
#include <chrono>

#include "kvq_decode_mma_kernel.cuh"

namespace kvq {
namespace mma {

// Instantiation units (kvq_decode_mma_inst_*.cu).
#define KVQ_MMA_DECL(D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB)                                                  \
  extern template int launch_mma_inst<D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB>(                                   \
      const Geom&, const CachePtrs&, const void*, float, float*, int, void*, int, unsigned long long,              \
      unsigned long long, long long, cudaStream_t);
#include "kvq_decode_mma_list.inc"
#undef KVQ_MMA_DECL

}  // namespace mma

constexpr int kFlatGrid = 2 * 148;   // slot capacity is sized for grids up to twice this

int flat_slot_cap(const Geom& g) {
  const int streams = g.B * g.Hkv;
  int s = (2 * kFlatGrid + streams - 1) / streams + 2;
  if (s > g.n_pages + 1) s = g.n_pages + 1;
  if (g.R) s += 1;                           // one more slot per stream: the partial of the residual window
  return s;
}

// Partials [streams][slots][G][D + 2] floats, then one 64-bit count word per stream.
size_t flat_workspace_bytes(const Geom& g) {
  const int s_cap = flat_slot_cap(g);
  return mma::tag_offset_floats(g.B * g.Hkv, s_cap, g.G * g.rows, g.D) * sizeof(float) + (size_t)g.B * g.Hkv * 8;
}

// Id of a launch: the words that count a stream's finished partials carry it, so that neither stale workspace
// contents nor an earlier call's counts are ever taken for this call's.  Starts at a clock value, never 0.
static unsigned long long next_call_id() {
  static std::atomic<unsigned long long> counter{
      ((unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() << 20) | 1ull};
  unsigned long long v = counter.fetch_add(1, std::memory_order_relaxed);
  return v ? v : counter.fetch_add(1, std::memory_order_relaxed);
}

// Finds the instantiation for this geometry; launches it unless `probe`.  *grid = CTAs of the launch.
static int pick(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap, void* out,
                int out_dtype, const DecodeDebug& dbg, cudaStream_t stream, bool probe, int* grid) {
  const int ngk = (g.k_axis == 1 || g.kb == 16) ? 1 : g.D / g.gk;
  const int ngv = (g.vb == 16) ? 1 : g.D / g.gv;
  const int nh = g.G * g.rows <= 4 ? 1 : 2;                                // (virtual) query heads per lane
#define KVQ_MMA_DECL(D_, KB_, VB_, KAXIS_, NGK_, NGV_, NH_, NW_, MINB_)                                      \
  if (g.D == D_ && g.kb == KB_ && g.vb == VB_ && g.k_axis == KAXIS_ && ngk == NGK_ && ngv == NGV_ &&          \
      NH_ == nh) {                                                                                            \
    *grid = 148 * MINB_;                                                                                      \
    if (probe) return KVQ_OK;                                                                                 \
    return mma::launch_mma_inst<D_, KB_, VB_, KAXIS_, NGK_, NGV_, NH_, NW_, MINB_>(                          \
        g, c, q, c1, ws, s_cap, out, out_dtype, next_call_id(),                                               \
        dbg.wait_us ? 1000ull * dbg.wait_us : mma::kWaitTimeoutNs, dbg.skip_page, stream);                    \
  }
#include "kvq_decode_mma_list.inc"
#undef KVQ_MMA_DECL
  return KVQ_ERR_UNSUPPORTED;
}

bool decode_mma_supported(const Geom& g) {
  if (g.B > mma::kMaxBatchFlat) return false;
  CachePtrs none{};
  int grid = 0;
  return pick(g, none, nullptr, 0.f, nullptr, 0, nullptr, 0, DecodeDebug{}, nullptr, true, &grid) == KVQ_OK;
}

int launch_decode_mma(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype, float c1,
                      float* ws, const DecodeDebug& dbg, cudaStream_t stream) {
  const int s_cap = flat_slot_cap(g);
  int grid = 0;
  if (g.R) {      // the residual window first: its partial (or, for sequences without pages, the output) is ready
                  // when the main kernel's last finisher merges
    int rc = launch_decode_window(g, c, q, out, out_dtype, c1, ws, s_cap, stream);
    if (rc != KVQ_OK) return rc;
  }
  const bool tc_ok = decode_tc_supported(g, c);
  if (dbg.fast_impl == 2 && !tc_ok) return KVQ_ERR_UNSUPPORTED;
  if (tc_ok && dbg.fast_impl == 2)
    return launch_decode_tc(g, c, q, c1, ws, s_cap, out, out_dtype, next_call_id(),
                            dbg.wait_us ? 1000ull * dbg.wait_us : mma::kWaitTimeoutNs, dbg.skip_page, stream);
  return pick(g, c, q, c1, ws, s_cap, out, out_dtype, dbg, stream, false, &grid);
}

}  // namespace kvq
