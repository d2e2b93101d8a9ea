// Explicit instantiations of the fast decode kernel (split over several files to compile in parallel).
#include "kvq_decode_mma_kernel.cuh"

namespace kvq {
namespace mma {
#define KVQ_MMA_DECL(D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB)                                          \
  template int launch_mma_inst<D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB>(                                          \
      const Geom&, const CachePtrs&, const void*, float, float*, int, void*, int, unsigned long long,              \
      unsigned long long, long long, cudaStream_t);
KVQ_MMA_DECL(128, 4, 2, 0, 4, 1, 2, 4, 2)
KVQ_MMA_DECL(128, 4, 2, 0, 2, 2, 2, 4, 2)
KVQ_MMA_DECL(64, 4, 2, 0, 2, 2, 1, 4, 3)
#undef KVQ_MMA_DECL
}  // namespace mma
}  // namespace kvq
