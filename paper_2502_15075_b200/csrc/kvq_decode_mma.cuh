// Fused low-bit decode attention, fast path: softmax(q K^T / sqrt(d)) V
// (App. A.1) over the packed cache, with K^ = z + s*code and V^ likewise
// reconstructed inside the contraction.
//
// Structure (one CTA = 4 consumer warps + 1 producer warp, several CTAs per SM):
//  * the producer streams whole 128-token pages into a four-stage shared-memory ring
//    with cp.async.bulk (one bulk copy per page with an L2 evict-first policy,
//    completion on an mbarrier);
//  * each consumer warp owns one 32-token block of every page and loads its operand
//    fragments with 16-byte shared loads (the page layout already is fragment order);
//  * both contractions are integer tensor-core MMAs on the raw code bytes
//    (mma.m16n8k32, int32 accumulate; one mask per operand register): q enters as 16-bit
//    fixed point in two signed bytes (channel-wise keys: q*s per page in three), the softmax
//    weight times the value scale as 31-bit fixed point in four unsigned bytes (24 bits in
//    three for 8 heads); the 8 MMA columns carry (head, limb) pairs;
//  * scale and zero-point never touch the codes:  q.K^_t = s_t (q.c_t) + z_t sum(q)
//    and  o = sum_t (p_t s_t) c_t + sum_t p_t z_t ;
//  * the sequence is split flat over the grid: CTA i takes the i-th share of all pages
//    of all streams (shares balanced by time where the arithmetic limits the kernel: a
//    stream boundary counts as ten pages, the launch waves of an SM are weighted) and
//    writes one unnormalised partial (m, l, o) per stream it touches; the CTA that
//    publishes the last partial of a stream merges them by log-sum-exp and writes the
//    output (no second kernel, nobody waits).
// Every wait on an mbarrier is bounded in time; on expiry the kernel sets
// KVQ_STATUS_DEVICE_TIMEOUT, keeps arriving at its barriers without computing, and returns.
#pragma once

#include "kvq_internal.h"

namespace kvq {
namespace mma {

constexpr unsigned long long kWaitTimeoutNs = 2000000000ull;   // default limit of a device-side wait: 2 s

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Same, letting the hardware park the thread for up to `hint_ns` while the phase is pending.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Slow path of a wait: poll with a parking hint, give up after limit_ns.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  const unsigned long long t0 = globaltimer_ns();
  while (true) {
    if (mbar_try_wait_hint(bar, parity, 4000u)) return true;
    if (globaltimer_ns() - t0 > limit_ns) return false;
  }
}
// Wait for the phase with the given parity; bounded in time (false = gave up).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, limit_ns);
}
// L2 policy for data that is read once: the streamed pages leave the cache first (a layer's packed cache is
// larger than the L2, and keeping its lines only delays the lines that are about to be fetched).
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// One bulk copy global -> this CTA's shared memory, completion counted in bytes on `bar`.
// dst, src and bytes are multiples of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// D += A(16x16, row) * B(16x8, col), fp16 operands, fp32 accumulate.
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D += A(16x32, row, unsigned bytes) * B(32x8, col, signed bytes), int32 accumulate.
__device__ __forceinline__ void mma16832_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Transpose an 8x8 matrix of 16-bit elements held one row-pair per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ------------------------------------------------------------------ half2 helpers on raw registers
__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }

// (a, b) in fp32 -> fp16 pairs hi and lo with hi + lo = (a, b) to 22 bits: hi = fp16(x), lo = fp16(x - hi).
__device__ __forceinline__ void split_h2(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(a, b);
  const float2 hf = __half22float2(h);
  hi = as_u32(h);
  lo = as_u32(__floats2half2_rn(a - hf.x, b - hf.y));
}

// ------------------------------------------------------------------ operand registers from packed words
// Key codes as unsigned-byte MMA operands: masking one field out of every byte of a packed word yields the
// codes of four consecutive channels as four bytes, ready for an integer MMA (8-bit codes need nothing at all).
// key_slot(kw, r): the four code bytes of register slot r (channels 16 r + 4 chunk + {0..3}) of a lane's KW
// packed words; r is a constant after unrolling.
template <int B, int KW>
__device__ __forceinline__ uint32_t key_slot(const uint32_t (&kw)[KW], int r) {
  if constexpr (B == 8) {
    return kw[r];
  } else {
    constexpr int FPB = 8 / B;
    constexpr uint32_t MASK = ((1u << B) - 1u) * 0x01010101u;
    return (kw[r / FPB] >> (B * (r % FPB))) & MASK;
  }
}

// Load a lane's NWORDS packed words from a pointer that addresses the lane's chunk; quads of words lie
// `quad_stride` bytes apart.
template <int NWORDS>
__device__ __forceinline__ void load_words(const uint8_t* p, int quad_stride, uint32_t (&w)[NWORDS]) {
  if constexpr (NWORDS >= 4) {
#pragma unroll
    for (int qd = 0; qd < NWORDS / 4; ++qd) {
      uint4 v = *reinterpret_cast<const uint4*>(p + qd * quad_stride);
      w[4 * qd + 0] = v.x; w[4 * qd + 1] = v.y; w[4 * qd + 2] = v.z; w[4 * qd + 3] = v.w;
    }
  } else if constexpr (NWORDS == 2) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    w[0] = v.x; w[1] = v.y;
  } else {
    w[0] = *reinterpret_cast<const uint32_t*>(p);
  }
}

__device__ __forceinline__ float meta_s(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m & 0xFFFF))); }
__device__ __forceinline__ float meta_z(uint32_t m) { return __half2float(__ushort_as_half((uint16_t)(m >> 16))); }

// ------------------------------------------------------------------ flat split and merge bookkeeping
constexpr int kMaxBatchFlat = 1024;   // the flat partition keeps a per-batch prefix in shared memory

// Flat split of all pages over the grid.
struct FlatPlan {
  long long N;       // total pages over all streams
  int c_eff;         // CTAs that take part
  __device__ __forceinline__ int cta_of(long long x) const { return (int)(((x + 1) * c_eff - 1) / N); }
  __device__ __forceinline__ long long lo(int c) const { return (long long)c * N / c_eff; }
};

__device__ __forceinline__ FlatPlan make_plan(long long N, int pages_max, int grid, int s_cap) {
  FlatPlan p;
  p.N = N;
  long long cap = pages_max > 0 ? (long long)(s_cap - 1) * N / pages_max : 0;
  long long ce = grid;
  if (ce > N) ce = N;
  if (ce > cap) ce = cap;
  p.c_eff = (int)ce;
  return p;
}

// Split partials of a stream are merged by whichever CTA publishes the last of them: after storing its partial a
// CTA counts itself in the stream's word, which holds (launch id << 24 | count).  A word that carries another id
// (stale contents, an earlier launch) restarts at 1, so the workspace needs no initialisation; the CTA that
// reaches the expected count merges and clears the word, so that a replayed launch with the same id starts clean.
__device__ __forceinline__ unsigned tagged_count(unsigned long long* p, unsigned long long id40) {
  // the usual case in one round trip: the word already carries this launch's id
  unsigned long long old = atomicAdd(p, 1ull);
  if ((old >> 24) == id40) return (unsigned)((old + 1ull) & 0xFFFFFFull);
  // otherwise the addition went into a word of another launch (or a cleared one): start it, or count into it once
  // somebody else has started it (whatever the stray additions left is overwritten by the start)
  old += 1ull;
  while (true) {
    const unsigned long long nw = ((old >> 24) == id40) ? old + 1ull : ((id40 << 24) | 1ull);
    const unsigned long long r = atomicCAS(p, old, nw);
    if (r == old) return (unsigned)(nw & 0xFFFFFFull);
    old = r;
  }
}
// Offset (in floats) of the count words behind the partials: [streams] 64-bit words.
__host__ __device__ inline size_t tag_offset_floats(int streams, int s_cap, int G, int D) {
  return ((size_t)streams * s_cap * G * (D + 2) + 3) & ~(size_t)3;
}

}  // namespace mma
}  // namespace kvq
