// Fused low-bit decode attention, fast path: softmax(q K^T / sqrt(d)) V
// (App. A.1) over the packed cache, with K^ = z + s*code and V^ likewise
// reconstructed inside the contraction.
//
// Structure (one CTA = NW consumer warps + 1 producer warp, several CTAs per SM):
//  * the producer streams whole 128-token pages into a shared-memory ring with
//    cp.async.bulk (one bulk copy per page, completion on an mbarrier);
//  * each consumer warp owns 16-token tiles of every page: it loads its operand
//    fragments with 16-byte shared loads (the page layout already is fragment order);
//  * token-wise keys: the code bytes go straight into integer tensor-core MMAs
//    (mma.m16n8k32 u8 x s8 -> s32; one mask or shift+mask per register), with q held as
//    22-bit fixed point split into three signed bytes per head, so q.c_t is exact;
//    channel-wise keys: fp16 MMAs on codes converted with LOP3 + HFMA2, channel scales
//    folded into q once per page;
//  * values: codes become integer-valued fp16 with one LOP3 + one HFMA2 per pair and
//    PV runs on fp16 MMAs (mma.m16n8k16, fp32 accumulate) for the <= 8 query heads
//    that share the KV head;
//  * scale and zero-point never touch the codes:  q.K^_t = s_t (q.c_t) + z_t sum(q)
//    and  o = sum_t (p_t s_t) c_t + sum_t p_t z_t ;
//  * the sequence is split flat over the grid: CTA i takes the i-th equal share of
//    all pages of all streams, writes one unnormalised partial (m, l, o) per stream
//    it touches, and a merge pass combines them by log-sum-exp.
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
// One bulk copy global -> this CTA's shared memory, completion counted in bytes on `bar`.
// dst, src and bytes are multiples of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
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
__device__ __forceinline__ uint32_t h2fma(uint32_t a, uint32_t b, uint32_t c) {
  return as_u32(__hfma2(as_h2(a), as_h2(b), as_h2(c)));
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) { return as_u32(__floats2half2_rn(lo, hi)); }

// (a, b) in fp32 -> fp16 pairs hi and lo with hi + lo = (a, b) to 22 bits: hi = fp16(x), lo = fp16(x - hi).
__device__ __forceinline__ void split_h2(float a, float b, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(a, b);
  const float2 hf = __half22float2(h);
  hi = as_u32(h);
  lo = as_u32(__floats2half2_rn(a - hf.x, b - hf.y));
}

// Four values times `scale` rounded to integers |Q| < 2^22 and split into three balanced signed bytes,
// Q = b0 * 65536 + b1 * 256 + b2; byte j of w0 / w1 / w2 is b0 / b1 / b2 of t[j] (an s8 MMA operand each).
__device__ __forceinline__ void fixed_point_limbs(const float (&t)[4], float scale, uint32_t& w0, uint32_t& w1,
                                                  uint32_t& w2) {
  w0 = w1 = w2 = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int Q = __float2int_rn(t[j] * scale);
    const int b2 = (int)(int8_t)(Q & 0xFF);
    const int Q1 = (Q - b2) >> 8;
    const int b1 = (int)(int8_t)(Q1 & 0xFF);
    const int b0 = (Q1 - b1) >> 8;
    w0 |= (uint32_t)(b0 & 0xFF) << (8 * j);
    w1 |= (uint32_t)(b1 & 0xFF) << (8 * j);
    w2 |= (uint32_t)(b2 & 0xFF) << (8 * j);
  }
}

// ------------------------------------------------------------------ code -> fp16 conversion
// A word holds 32/B fields; pair i = (field i, field i + 16/B) becomes one half2 register holding the two
// codes as exact fp16 integers: the field bits are OR-ed into the mantissa of 1024.0 (0x6400), which yields
// 1024 + code * 2^shift, and one HFMA2 with (2^-shift, -1024 * 2^-shift) brings that back to `code` exactly.
constexpr uint32_t kMagic = 0x64006400u;   // (1024.0, 1024.0)

// (x & MASK) | 0x64006400 as one LOP3 (truth table 0xEA = (a & b) | c).
template <uint32_t MASK>
__device__ __forceinline__ uint32_t field_to_magic(uint32_t x) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "n"(MASK), "r"(kMagic));
  return d;
}

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

// Value codes as fp16 MMA operands without arithmetic: (x & mask) | 0x64006400 puts the B-bit field at
// position `pos` of the low byte of each 16-bit half into the mantissa of 1024.0, giving the two halves the
// values 1024 + code * 2^(B * pos) of two consecutive tokens.
template <int B>
__device__ __forceinline__ uint32_t biased_pair(uint32_t x, int pos) {
  const uint32_t mask = (((1u << B) - 1u) << (B * pos)) * 0x00010001u;
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "r"(mask), "r"(kMagic));
  return d;
}

// Codes are centred on the middle of their range before the PV contraction.
template <int B> constexpr float kCodeMid = (float)(1 << (B - 1));

// biased_pair, then one HFMA2: (1024 + code * 2^(B pos)) * 2^-(B pos) - (1024 * 2^-(B pos) + MID) = code - MID,
// exact in fp16 (all constants and the result are representable).
template <int B>
__device__ __forceinline__ uint32_t centered_pair(uint32_t x, int pos) {
  const float inv = 1.f / (float)(1 << (B * pos));
  const __half2 scale = __float2half2_rn(inv);
  const __half2 off = __float2half2_rn(-(1024.f * inv + kCodeMid<B>));
  return as_u32(__hfma2(as_h2(biased_pair<B>(x, pos)), scale, off));
}

template <int B> struct Unpack;

template <> struct Unpack<4> {
  static constexpr int PPW = 4;
  __device__ static __forceinline__ void run(uint32_t x, uint32_t (&o)[4]) {
    const uint32_t y = x >> 8;
    o[0] = h2fma(field_to_magic<0x000f000fu>(x), 0x3c003c00u, 0xe400e400u);   // * 1     - 1024
    o[1] = h2fma(field_to_magic<0x00f000f0u>(x), 0x2c002c00u, 0xd400d400u);   // * 1/16  - 64
    o[2] = h2fma(field_to_magic<0x000f000fu>(y), 0x3c003c00u, 0xe400e400u);
    o[3] = h2fma(field_to_magic<0x00f000f0u>(y), 0x2c002c00u, 0xd400d400u);
  }
};

template <> struct Unpack<2> {
  static constexpr int PPW = 8;
  __device__ static __forceinline__ void run(uint32_t x, uint32_t (&o)[8]) {
    const uint32_t y = x >> 10;
    o[0] = h2fma(field_to_magic<0x00030003u>(x), 0x3c003c00u, 0xe400e400u);   // * 1     - 1024
    o[1] = h2fma(field_to_magic<0x000c000cu>(x), 0x34003400u, 0xdc00dc00u);   // * 1/4   - 256
    o[2] = h2fma(field_to_magic<0x00300030u>(x), 0x2c002c00u, 0xd400d400u);   // * 1/16  - 64
    o[3] = h2fma(field_to_magic<0x00c000c0u>(x), 0x24002400u, 0xcc00cc00u);   // * 1/64  - 16
    o[4] = h2fma(field_to_magic<0x03000300u>(x), 0x1c001c00u, 0xc400c400u);   // * 1/256 - 4
    o[5] = h2fma(field_to_magic<0x00030003u>(y), 0x3c003c00u, 0xe400e400u);
    o[6] = h2fma(field_to_magic<0x000c000cu>(y), 0x34003400u, 0xdc00dc00u);
    o[7] = h2fma(field_to_magic<0x00300030u>(y), 0x2c002c00u, 0xd400d400u);
  }
};

template <> struct Unpack<8> {
  static constexpr int PPW = 2;
  __device__ static __forceinline__ void run(uint32_t x, uint32_t (&o)[2]) {
    // bytes (b0, 0x64, b2, 0x64) and (b1, 0x64, b3, 0x64): 1024 + code in each half
    o[0] = h2fma(__byte_perm(x, 0x64646464u, 0x4240), 0x3c003c00u, 0xe400e400u);
    o[1] = h2fma(__byte_perm(x, 0x64646464u, 0x4341), 0x3c003c00u, 0xe400e400u);
  }
};

// Load a lane's NWORDS words of chunk `chunk` from a row / tile that holds `nchunks` chunks (quad-major).
template <int NWORDS>
__device__ __forceinline__ void load_chunk(const uint8_t* base, int chunk, int nchunks, uint32_t (&w)[NWORDS]) {
  if constexpr (NWORDS >= 4) {
#pragma unroll
    for (int qd = 0; qd < NWORDS / 4; ++qd) {
      uint4 v = *reinterpret_cast<const uint4*>(base + qd * (nchunks * 16) + chunk * 16);
      w[4 * qd + 0] = v.x; w[4 * qd + 1] = v.y; w[4 * qd + 2] = v.z; w[4 * qd + 3] = v.w;
    }
  } else if constexpr (NWORDS == 2) {
    uint2 v = *reinterpret_cast<const uint2*>(base + chunk * 8);
    w[0] = v.x; w[1] = v.y;
  } else {
    w[0] = *reinterpret_cast<const uint32_t*>(base + chunk * 4);
  }
}

// Same, from a pointer that already addresses the lane's chunk; quads of words lie `quad_stride` bytes apart.
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

}  // namespace mma
}  // namespace kvq
