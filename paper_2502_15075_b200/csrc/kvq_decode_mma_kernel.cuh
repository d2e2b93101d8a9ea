// The templated fast decode kernel (see kvq_decode_mma.cuh for the design).
#pragma once

#include <type_traits>

#include "kvq_decode_mma.cuh"

namespace kvq {
namespace mma {

// Shared-memory carve-up (dynamic): ring | barriers | prefix | misc | per-warp fp32 masters | (m, l) | channel-wise scratch
struct SmemLayout {
  int page_stride, ring_bytes, bar_off, pref_off, misc_off, master_off, ml_off, chan_off, total;
};
// master: per consumer warp, 4 NH heads x (D + 8) floats (the row padding keeps a warp's accesses conflict-free).
// chan: channel-wise keys keep, per ring stage, the page's q operands made by the preparation warp
// (NH x 2 x D/16 x 32 words) followed by 8 zero-point sums and 8 fixed-point scales (one per head).
__host__ __device__ inline int chan_stage_bytes(int D, int nh) { return nh * 2 * (D / 16) * 32 * 4 + 64; }
__host__ __device__ inline SmemLayout smem_layout(int page_bytes, int stages, int nw, int batch, int D, int nh,
                                                  bool chan) {
  SmemLayout s;
  s.page_stride = (page_bytes + 127) & ~127;
  s.ring_bytes = s.page_stride * stages;
  s.bar_off = s.ring_bytes;
  s.pref_off = s.bar_off + 16 * 8 * 2;                      // up to 32 barriers: (full, empty[, ready]) per stage
  s.misc_off = (s.pref_off + 2 * (batch + 1) * 4 + 15) & ~15;      // two prefixes: pages, and pages + stream gaps
  s.master_off = s.misc_off + 64;
  s.ml_off = s.master_off + nw * 4 * nh * (D + 8) * 4;
  s.chan_off = s.ml_off + nw * 4 * nh * 2 * 4;
  s.total = s.chan_off + (chan ? stages * chan_stage_bytes(D, nh) : 0);
  return s;
}

// prmt.b32 with the full selector semantics (a selector nibble with bit 3 set replicates the sign of the byte).
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}
// D += A(16x32, row, unsigned bytes) * B(32x8, col, unsigned bytes), int32 accumulate.
__device__ __forceinline__ void mma16832_u8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Four values times `scale` rounded to integers |Q| <= 32512 and split into two balanced signed bytes,
// Q = hi * 256 + lo; returns the four hi bytes (lo_limb = 0) or the four lo bytes (lo_limb = 1) as one word
// and adds the four Q to `qsum`.
__device__ __forceinline__ uint32_t fixed_point_limb(const float (&t)[4], float scale, int lo_limb, int& qsum) {
  uint32_t w = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int Q = __float2int_rn(t[j] * scale);
    const int lo = (int)(int8_t)(Q & 0xFF);
    const int hi = (Q - lo) >> 8;
    w |= (uint32_t)((lo_limb ? lo : hi) & 0xFF) << (8 * j);
    qsum += Q;
  }
  return w;
}

// The split balances time, not pages.  Ending one stream and starting the next (fold and combine the warps'
// state, store and publish the partial, perhaps merge; load and convert the next queries) costs a CTA as much as
// ~9 pages (8.4 us on the 8B-shaped layer: CTAs whose share crosses a stream boundary ended at 81.2 us, the others
// at 72.8 us), and of the three CTAs that share an SM the hardware favours the older ones (launch waves ended at
// 68.9 / 72.7 / 76.8 us with equal work).  So every stream is given kGapPages virtual pages in front of its real
// ones and the shares of the launch waves are weighted; the split is taken on that virtual axis.
#ifndef KVQ_GAP_PAGES
#define KVQ_GAP_PAGES 10
#endif
#ifndef KVQ_WAVE_W0
#define KVQ_WAVE_W0 1040
#endif
constexpr int kGapPages = KVQ_GAP_PAGES;
constexpr int kWaveWeight0 = KVQ_WAVE_W0;  // share of a first-wave CTA in thousandths of the mean (third wave: 2000 - this)
constexpr float kQFix = 32512.0f;          // largest |Q| of the 16-bit fixed-point q (hi limb stays within +-127)
constexpr float kQFix3 = 8300000.0f;       // ... of the 24-bit fixed-point q * s of channel-wise keys (three limbs)

// Four values times `scale` rounded to integers |Q| <= kQFix3 and taken apart as two's-complement bytes,
// Q = b2 * 65536 + b1 * 256 + b0 with b2 signed and b1, b0 unsigned.  Operand words of a lane: even operand
// columns (odd = 0) carry b2 in n-tile 0 (signed bytes) and b1 in n-tile 1 (unsigned bytes), odd columns nothing in
// n-tile 0 and b0 in n-tile 1.  Byte j of a word belongs to t[j].
__device__ __forceinline__ void fixed_point_bytes3(const float (&t)[4], float scale, int odd, uint32_t& w_nt0,
                                                   uint32_t& w_nt1) {
  const uint32_t q0 = (uint32_t)__float2int_rn(t[0] * scale), q1 = (uint32_t)__float2int_rn(t[1] * scale);
  const uint32_t q2 = (uint32_t)__float2int_rn(t[2] * scale), q3 = (uint32_t)__float2int_rn(t[3] * scale);
  // byte k of each of the four integers -> one word: selectors pick byte k of (q0, q1) and of (q2, q3)
  const uint32_t sel = odd ? 0x0040u : 0x0051u;                  // odd: byte 0; even: byte 1
  const uint32_t lo01 = prmt(q0, q1, sel), lo23 = prmt(q2, q3, sel);
  w_nt1 = prmt(lo01, lo23, 0x5410u);
  const uint32_t hi01 = prmt(q0, q1, 0x0062u), hi23 = prmt(q2, q3, 0x0062u);   // byte 2 of each
  w_nt0 = odd ? 0u : prmt(hi01, hi23, 0x5410u);
}
// The softmax weights enter PV as fixed point P = rint(p * s_V * 2^PBITS / s_lim), p = 2^(logit - reference) with the
// reference kHeadroom bits above the largest logit seen so far, so that a larger logit rarely forces a rescale.
// Tokens whose P falls below one unit vanish, so the width matters over long contexts: four byte limbs (31 bits)
// where one lane serves one head, three (24 bits, less headroom) where it serves two.
template <int NH> constexpr int kPBits = NH == 1 ? 31 : 24;
template <int NH> constexpr float kHeadroom = NH == 1 ? 6.0f : 1.0f;
constexpr int kFlushBlocks = 512;          // fold the int32 value accumulators at least this often (no overflow)

// The query values a lane needs as MMA operand: head hb (a (row, head) pair when several rows are served), channels
// 16 r + 4 tid + {0..3} for every slot r, in fp32, rotated like the keys if the cache rotates them; heads >= G are
// zero.  Returns max |q| over the lane's values (the caller reduces over the quad).
template <int D>
__device__ __forceinline__ float load_q_lane(const Geom& g, const CachePtrs& c, const uint16_t* __restrict__ q, int b,
                                             int h, int hb, int tid, float (&qv)[D / 16][4]) {
  constexpr int NR = D / 16;
  constexpr uint32_t FULL = 0xffffffffu;
  const int Gq = g.G, G = g.G * g.rows;
        const uint16_t* qrow = q + (((size_t)b * g.rows + hb / Gq) * g.Hq + (size_t)h * Gq + hb % Gq) * D;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          uint2 raw = make_uint2(0u, 0u);
          if (hb < G) raw = *reinterpret_cast<const uint2*>(qrow + 16 * r + 4 * tid);
          qv[r][0] = bits16_to_f32((uint16_t)(raw.x & 0xFFFF), g.in_dtype);
          qv[r][1] = bits16_to_f32((uint16_t)(raw.x >> 16), g.in_dtype);
          qv[r][2] = bits16_to_f32((uint16_t)(raw.y & 0xFFFF), g.in_dtype);
          qv[r][3] = bits16_to_f32((uint16_t)(raw.y >> 16), g.in_dtype);
        }
        if (c.k_signs != nullptr) {
          // rotated keys: give q the same rotation, q' = H (signs * q) / sqrt(D); channel 16 r + 4 tid + j,
          // so the butterflies run over j inside the lane, over tid across lanes, over r inside the lane
#pragma unroll
          for (int r = 0; r < NR; ++r) {
#pragma unroll
            for (int j = 0; j < 4; ++j) qv[r][j] *= (float)c.k_signs[16 * r + 4 * tid + j];
            float a = qv[r][0], bq = qv[r][1], cq = qv[r][2], dq = qv[r][3];
            qv[r][0] = (a + bq) + (cq + dq); qv[r][1] = (a - bq) + (cq - dq);
            qv[r][2] = (a + bq) - (cq + dq); qv[r][3] = (a - bq) - (cq - dq);
#pragma unroll
            for (int m = 1; m < 4; m <<= 1) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float o = __shfl_xor_sync(FULL, qv[r][j], m);
                qv[r][j] = (tid & m) ? o - qv[r][j] : qv[r][j] + o;
              }
            }
          }
#pragma unroll
          for (int hh = 1; hh < NR; hh <<= 1) {
#pragma unroll
            for (int r = 0; r < NR; ++r) {
              if ((r & hh) == 0) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const float a = qv[r][j], bq = qv[r + hh][j];
                  qv[r][j] = a + bq;
                  qv[r + hh][j] = a - bq;
                }
              }
            }
          }
#pragma unroll
          for (int r = 0; r < NR; ++r) {
#pragma unroll
            for (int j = 0; j < 4; ++j) qv[r][j] *= inv_sqrt_dim<D>();
          }
        }
        float amax = 0.f;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
#pragma unroll
          for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fabsf(qv[r][j]));
        }
  return amax;
}

// Weighted position of a CTA on the virtual axis in units of 1 / (148 * 1000 * waves) of the whole: two or three launch
// waves of 148 CTAs (one per CTA that an SM holds) with weights W0, [1000,] 2000 - W0.
#ifndef KVQ_WAVE2_W0
#define KVQ_WAVE2_W0 1000   /* two CTAs per SM: weighting the waves did not pay (70B-shaped layer: 147.8 us equal, 149.9 us at 1040, 154.1 us at 1080) */
#endif
template <int WAVES> struct WaveWeights;
template <> struct WaveWeights<3> { static constexpr int w[3] = {kWaveWeight0, 1000, 2000 - kWaveWeight0}; };
template <> struct WaveWeights<2> { static constexpr int w[3] = {KVQ_WAVE2_W0, 2000 - KVQ_WAVE2_W0, 0}; };
template <int WAVES>
__device__ __forceinline__ long long wave_prefix(int cta) {
  constexpr int W0 = WaveWeights<WAVES>::w[0], W1 = WaveWeights<WAVES>::w[1], W2 = WaveWeights<WAVES>::w[2];
  const int k = cta / 148, r = cta % 148;
  return (k == 0 ? 0 : k == 1 ? W0 : k == 2 ? W0 + W1 : W0 + W1 + W2) * 148ll + (long long)r * (k == 0 ? W0 : k == 1 ? W1 : W2);
}
// First virtual page of a CTA's share: equal shares, or shares weighted by launch wave.
template <int WAVES>
static __device__ __forceinline__ long long share_start_virtual(const FlatPlan& plan, bool waves, int cta) {
  if (!waves) return plan.lo(cta);
  return plan.N * wave_prefix<WAVES>(cta) / (148ll * 1000 * WAVES);
}
// The CTA whose share holds virtual page v: the largest c with N prefix(c) < (v + 1) U, found wave by wave (the
// prefix is linear inside a wave), one division.
template <int WAVES>
static __device__ __forceinline__ int cta_of_virtual(const FlatPlan& plan, bool waves, long long v) {
  if (!waves) return plan.cta_of(v);
  constexpr int W0 = WaveWeights<WAVES>::w[0], W1 = WaveWeights<WAVES>::w[1], W2 = WaveWeights<WAVES>::w[2];
  const long long a = (v + 1) * (148ll * 1000 * WAVES) - 1;      // N prefix(c) <= a
  const long long b1 = plan.N * (148ll * W0), b2 = plan.N * (148ll * (W0 + W1));
  const int k = (WAVES == 3 && a >= b2) ? 2 : a >= b1 ? 1 : 0;
  const long long base = k == 2 ? b2 : k == 1 ? b1 : 0;
  const long long r = (a - base) / (plan.N * (k == 2 ? W2 : k == 1 ? W1 : W0));
  return 148 * k + (int)(r < 147 ? r : 147);
}
// Flat index of the first real page at or after the start of a CTA's share (sPref: pages, sVPref: pages + gaps).
template <int WAVES>
static __device__ __forceinline__ long long share_start(const FlatPlan& plan, bool waves, int cta, const int* sPref,
                                                     const int* sVPref, int B, int Hkv, int gap) {
  const long long v = share_start_virtual<WAVES>(plan, waves, cta);
  if (v >= plan.N) return sPref[B];
  int lo_ = 0, hi_ = B - 1;                        // last batch entry with sVPref <= v
  while (lo_ < hi_) {
    const int mid = (lo_ + hi_ + 1) >> 1;
    if (sVPref[mid] <= v) lo_ = mid; else hi_ = mid - 1;
  }
  const int pb = (sPref[lo_ + 1] - sPref[lo_]) / Hkv, len = pb + gap;
  const int vs = (int)(v - sVPref[lo_]), hh = vs / len, off = vs % len;
  return (long long)sPref[lo_] + (long long)hh * pb + max(0, off - gap);
}

// Template parameters: head_dim, key bits, value bits, key axis (0 token-wise, 1 channel-wise), key / value groups
// per row, NH = query heads per lane (1: up to 4 heads per KV head, 2: up to 8), consumer warps (4: one per
// 32-token block of a page), resident CTAs per SM.
//
// Both contractions run on integer tensor-core MMAs over the raw code bytes (m16n8k32, int32 accumulate).
// The 8 columns of an MMA carry (head, limb) pairs: q as 16-bit fixed point in two signed bytes for QK^T, the
// softmax weight times the value scale as 31-bit (NH = 2: 24-bit) fixed point in unsigned bytes for PV.  Lane (g, t) of a
// warp (g = lane / 4, t = lane % 4) owns query heads t (and t + 4 when NH = 2): its accumulator columns 2t, 2t+1
// are the limbs of that head, so logits, softmax and the fixed-point weights need no exchange between lanes.
template <int D, int KB, int VB, int KAXIS, int NGK, int NGV, int NH, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1 + (KAXIS == 1 ? 1 : 0)) * 32, MINB)
decode_mma_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ q, float c1, float* __restrict__ ws,
                  int s_cap, int stages, void* __restrict__ out, int out_dtype, unsigned long long call_id,
                  unsigned long long wait_ns, long long skip_x) {
  constexpr int NR = D / 16;                // 16-channel register slots per key row
  constexpr int KS32 = D / 32;              // k-steps of an 8-bit MMA over the channels
  constexpr int MT = D / 16;                // m-tiles of PV (16 channels each)
  constexpr int KW = D * KB / 128;          // key words per lane per token row
  constexpr int FPBV = 8 / VB;              // value codes per byte (channels 16 apart)
  constexpr int VQ = MT / FPBV;             // quads of value words per lane per 32-token block
  constexpr int NTV = NH == 1 ? 2 : 3;      // n-tiles of PV: (head, limb) columns
  constexpr int NTK = KAXIS == 1 ? 2 : 1;   // n-tiles of QK^T per head set: two byte limbs of q, or three of q * s
  constexpr int NHEADS = 4 * NH;
  constexpr int MSTRIDE = D + 8;
  constexpr int K_ROW_BYTES = D * KB / 8;
  constexpr int V_BLOCK_BYTES = 4 * D * VB;
  // page geometry (the same numbers the host put into Geom)
  constexpr int K_META_OFF = kPageTokens * K_ROW_BYTES;
  constexpr int V_CODES_OFF = K_META_OFF + (KAXIS == 1 ? 4 * D : kPageTokens * NGK * 4);
  constexpr int V_META_OFF = V_CODES_OFF + 4 * V_BLOCK_BYTES;
  constexpr int NCONS = NW * 32;
  constexpr int NG = NW / 4;                // groups of four consumer warps; a group takes every NG-th page
  constexpr uint32_t FULL = 0xffffffffu;
  // The time-balanced split (stream gaps, wave weights) pays where the arithmetic per page limits the kernel
  // (token-wise and channel-wise keys alike: 14B-shaped channel-wise K4V2 188 -> 184 us); pages of 10 bits per
  // element pair and more lose with it (channel-wise K8V2 193 -> 197 us) and keep the plain split by pages.
  constexpr int GAP = (KB + VB <= 8) ? kGapPages : 0;
  constexpr int WAVES = MINB == 2 ? 2 : 3;          // CTAs per SM = launch waves (the weights apply to a grid of 148 * WAVES)
  static_assert(NW % 4 == 0, "four consumer warps per page, one per 32-token block");
  static_assert(KAXIS == 0 || KB != 2, "channel-wise 2-bit keys are not instantiated");
  static_assert(MT % FPBV == 0, "value m-tiles come in groups that share a byte");

  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout sl = smem_layout(g.page_bytes, stages, NW, g.B, D, NH, KAXIS == 1);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sl.bar_off);   // full[0..stages), empty[0..stages)
  int* sPref = reinterpret_cast<int*>(smem + sl.pref_off);
  int* sVPref = sPref + (g.B + 1);                                   // the same prefix with kGapPages more per stream
  int* sMisc = reinterpret_cast<int*>(smem + sl.misc_off);           // [0] pages_max, [1] abort flag, [2] published count, [4..7] share ends, [8..9] segment slot / partials, [10..13] CTAs taking part, cursor
  float* sMaster = reinterpret_cast<float*>(smem + sl.master_off);   // [NW][NHEADS][MSTRIDE]
  float* sML = reinterpret_cast<float*>(smem + sl.ml_off);           // [NW][NHEADS][2] = (reference, l)

  const int tid_ = threadIdx.x, lane = tid_ & 31, warp = tid_ >> 5;
  const int gid = lane >> 2, tid = lane & 3;
  // Several query rows per head (g.rows > 1) are served as virtual heads: row r of head j is virtual head
  // r * Gq + j, with its own causal limit on the tokens it may see.
  const int B = g.B, Hkv = g.Hkv, Gq = g.G, G = g.G * g.rows;

  // ---- plan, all of it on warp 0 (the others wait at one barrier): pages per sequence, prefix over the batch,
  // this CTA's share of the pages and the stream its first page lies in
  const int s_plan = s_cap - (g.R ? 1 : 0);       // the last partial slot of a stream belongs to its residual window
  if (warp == 0) {
    int carry = 0, vcarry = 0, pmax = 0;
    for (int base = 0; base < B; base += 32) {
      const int i = base + lane;
      const int pages = (i < B) ? (paged_len(c.seq_len, i, g.capacity, g.R) + kPageTokens - 1) >> 7 : 0;
      pmax = max(pmax, pages);
      int v = pages * Hkv;
      int vv = v > 0 ? v + GAP * Hkv : 0;
      for (int off = 1; off < 32; off <<= 1) {
        int u = __shfl_up_sync(FULL, v, off), uu = __shfl_up_sync(FULL, vv, off);
        if (lane >= off) { v += u; vv += uu; }
      }
      if (i < B) { sPref[i + 1] = v + carry; sVPref[i + 1] = vv + vcarry; }
      carry += __shfl_sync(FULL, v, 31);
      vcarry += __shfl_sync(FULL, vv, 31);
    }
    for (int off = 16; off; off >>= 1) pmax = max(pmax, __shfl_xor_sync(FULL, pmax, off));
    if (lane == 0) {
      sPref[0] = 0; sVPref[0] = 0; sMisc[0] = pmax; sMisc[1] = 0;
      for (int s = 0; s < stages; ++s) {
        mbar_init(smem_u32(&bars[s]), 1);
        mbar_init(smem_u32(&bars[stages + s]), 4);
        if constexpr (KAXIS == 1) mbar_init(smem_u32(&bars[2 * stages + s]), 1);     // ready: operands of the page made
      }
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (lane < 2) {
      // lane 0: the share's first page, the CTAs that take part and the cursor; lane 1: the share's end
      const FlatPlan p0 = make_plan(vcarry, pmax + GAP, gridDim.x, s_plan);
      long long x0 = 0;
      if (p0.N != 0 && (int)blockIdx.x < p0.c_eff) {
        if constexpr (GAP == 0) {
          x0 = p0.lo(blockIdx.x + lane);
        } else {
          const bool w0 = gridDim.x == WAVES * 148 && p0.c_eff == (int)gridDim.x && p0.N >= 8ll * gridDim.x;
          x0 = share_start<WAVES>(p0, w0, (int)blockIdx.x + lane, sPref, sVPref, B, Hkv, GAP);
        }
      }
      *reinterpret_cast<long long*>(sMisc + 4 + 2 * lane) = x0;
      if (lane == 0) {
        int cb = 0, ch = 0, cp = 0;
        if (x0 < carry) {                      // a real page: (sequence, kv head, page) of the share's first page
          int lo_ = 0, hi_ = B - 1;            // last sequence with sPref <= x0
          while (lo_ < hi_) {
            int mid = (lo_ + hi_ + 1) >> 1;
            if (sPref[mid] <= x0) lo_ = mid; else hi_ = mid - 1;
          }
          cb = lo_;
          const int pb = (sPref[cb + 1] - sPref[cb]) / Hkv, r = (int)x0 - sPref[cb];
          if (pb > 0) { ch = r / pb; cp = r % pb; }
        }
        sMisc[10] = p0.c_eff; sMisc[11] = cb; sMisc[12] = ch; sMisc[13] = cp;
      }
    }
  }
  __syncthreads();
  // an empty sequence has no page and therefore no CTA of its own: its output rows are zero (with a residual
  // window the window kernel, which runs first, has written the rows of sequences without pages)
  for (int bb = blockIdx.x; bb < B && g.R == 0; bb += gridDim.x) {
    if (sPref[bb + 1] == sPref[bb]) {
      for (int i = tid_; i < g.rows * g.Hq * D; i += blockDim.x) {
        const size_t oi = (size_t)bb * g.rows * g.Hq * D + i;
        if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = 0.f;
        else static_cast<uint16_t*>(out)[oi] = 0;
      }
    }
  }
  // the plan lives on the virtual axis (pages + a gap in front of every stream)
  FlatPlan plan;
  plan.N = sVPref[B];
  plan.c_eff = sMisc[10];
  if (plan.N == 0 || (int)blockIdx.x >= plan.c_eff) return;
  unsigned long long* counts = reinterpret_cast<unsigned long long*>(ws + tag_offset_floats(B * Hkv, s_cap, G, D));
  const bool waves = GAP != 0 && gridDim.x == WAVES * 148 && plan.c_eff == (int)gridDim.x && plan.N >= 8ll * gridDim.x;
  const long long x_lo = *reinterpret_cast<const long long*>(sMisc + 4), x_hi = *reinterpret_cast<const long long*>(sMisc + 6);
  if (x_lo >= x_hi) return;                          // a share that lies inside a gap (tiny problems only)

  // ---- cursor: first page of this CTA -> (b, h, page)
  int b = sMisc[11], h = sMisc[12], page = sMisc[13];
  int pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
  const uint32_t ring = smem_u32(smem);
  const uint32_t bar0 = smem_u32(bars);
  volatile int* abort_flag = sMisc + 1;
  volatile int* n_published = sMisc + 2;      // count returned for the partial just published
  const unsigned long long id40 = (call_id & 0xFFFFFFFFFFull) ? (call_id & 0xFFFFFFFFFFull) : 1ull;

  // =========================================================== producer warp
  if (warp == NW) {
    if (lane == 0) {
      int it = 0, stage = 0;
      uint32_t phase = 1;                // parity of the previous round of `empty`
      bool ok = true;
      const uint64_t policy = l2_evict_first_policy();
      for (long long x = x_lo; x < x_hi; ++x, ++it) {
        if (it >= stages) {
          ok = mbar_wait(bar0 + 8 * (stages + stage), phase, wait_ns);
          if (!ok || *abort_flag) { ok = false; break; }
        }
        const uint8_t* src = c.pages + ((size_t)(b * Hkv + h) * g.n_pages + page) * (size_t)g.page_bytes;
        const uint32_t fb = bar0 + 8 * stage;
        if (x != skip_x) {          // (skip_x: test hook - a page that never arrives makes the consumers' bounded wait expire)
          mbar_expect_tx(fb, (uint32_t)g.page_bytes);
          bulk_load(ring + stage * sl.page_stride, src, (uint32_t)g.page_bytes, fb, policy);
        }
        if (++stage == stages) { stage = 0; phase ^= 1; }
        if (++page == pages_b) {
          page = 0;
          if (++h == Hkv) {
            h = 0;
            do { ++b; } while (b < B && sPref[b + 1] == sPref[b]);
            if (b < B) pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
      }
      // Never leave while a copy may still be writing this CTA's shared memory: wait (bounded) for the
      // last copies issued, whether or not a consumer is still going to.
      for (int k = 1; k <= stages && k <= it; ++k) {
        const int j = it - k;
        mbar_wait(bar0 + 8 * (j % stages), (j / stages) & 1, wait_ns);
      }
    }
    return;
  }

  // =========================================================== preparation warp (channel-wise keys)
  // Per page, the operand of the integer QK^T MMAs is q_d * s_d in 24-bit fixed point (scale from max|q| of the head
  // times the page's largest channel scale), and sum_d q_d z_d is one fp32 scalar per head.  One warp makes both for
  // every page, in the lane arrangement the consumers' B fragments have, leaves them in the stage's operand buffer
  // and signals the stage's `ready` barrier; for the incomplete last block it leaves q split into fp16 high and
  // low parts instead (operands of the fp16 MMAs on the tail keys).
  if constexpr (KAXIS == 1) {
    if (warp == NW + 1) {
      constexpr int CSB = NH * 2 * NR * 32 * 4 + 64;
      int stage = 0;
      uint32_t phase = 0;
      float qv[NH][NR][4];
      float amaxB[NH];
      int cur_b = -1, cur_h = -1;
      for (long long x = x_lo; x < x_hi; ++x) {
        if (b != cur_b || h != cur_h) {          // a new stream: its queries
          cur_b = b; cur_h = h;
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
            float am = load_q_lane<D>(g, c, q, b, h, (gid >> 1) + 4 * nh, tid, qv[nh]);
            am = fmaxf(am, __shfl_xor_sync(FULL, am, 1));
            amaxB[nh] = fmaxf(am, __shfl_xor_sync(FULL, am, 2));
          }
        }
        const int n_tok = paged_len(c.seq_len, b, g.capacity, g.R);
        const bool tail_pg = n_tok - page * kPageTokens < kPageTokens;
        const bool got = mbar_wait(bar0 + 8 * stage, phase, wait_ns);
        if (!__all_sync(FULL, got) || *abort_flag) {
          *abort_flag = 1;
          if (lane == 0) atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
          return;
        }
        const uint8_t* sp = smem + stage * sl.page_stride;
        uint32_t* ops = reinterpret_cast<uint32_t*>(smem + sl.chan_off + stage * CSB);     // [NH][2][NR][32]
        float* opf = reinterpret_cast<float*>(ops + NH * 2 * NR * 32);                      // zq[8], hs[8]
        if (tail_pg) {
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
            for (int r = 0; r < NR; ++r) {
              uint32_t h0, l0_, h1, l1_;
              split_h2(qv[nh][r][0], qv[nh][r][2], h0, l0_);
              split_h2(qv[nh][r][1], qv[nh][r][3], h1, l1_);
              ops[((nh * 2 + 0) * NR + r) * 32 + lane] = (gid & 1) ? l0_ : h0;
              ops[((nh * 2 + 1) * NR + r) * 32 + lane] = (gid & 1) ? l1_ : h1;
            }
          }
        } else {
          const uint32_t* km = reinterpret_cast<const uint32_t*>(sp + K_META_OFF);
          float smax = 0.f;
          if (4 * lane < D) {
            const uint4 mm = *reinterpret_cast<const uint4*>(km + 4 * lane);
            smax = fmaxf(fmaxf(meta_s(mm.x), meta_s(mm.y)), fmaxf(meta_s(mm.z), meta_s(mm.w)));
          }
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) smax = fmaxf(smax, __shfl_xor_sync(FULL, smax, off));
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
            const int hb = (gid >> 1) + 4 * nh;
            const float am = amaxB[nh] * smax;
            const float scale = am > 0.f ? kQFix3 / am : 0.f;
            float zsum = 0.f;
#pragma unroll
            for (int r = 0; r < NR; ++r) {
              const uint4 mm = *reinterpret_cast<const uint4*>(km + 16 * r + 4 * tid);     // (s, z) of 4 channels
              const uint32_t mw[4] = {mm.x, mm.y, mm.z, mm.w};
              float t[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 sz = __half22float2(as_h2(mw[j]));
                t[j] = qv[nh][r][j] * sz.x;
                zsum = fmaf(qv[nh][r][j], sz.y, zsum);
              }
              uint32_t w0, w1;
              fixed_point_bytes3(t, scale, gid & 1, w0, w1);
              ops[((nh * 2 + 0) * NR + r) * 32 + lane] = w0;
              ops[((nh * 2 + 1) * NR + r) * 32 + lane] = w1;
            }
            zsum += __shfl_xor_sync(FULL, zsum, 1);
            zsum += __shfl_xor_sync(FULL, zsum, 2);
            if (tid == 0 && (gid & 1) == 0) {
              opf[hb] = c1 * zsum;
              opf[8 + hb] = am > 0.f ? c1 / scale : 0.f;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar0 + 8 * (2 * stages + stage));
        if (++stage == stages) { stage = 0; phase ^= 1; }
        if (++page == pages_b) {
          page = 0;
          if (++h == Hkv) {
            h = 0;
            do { ++b; } while (b < B && sPref[b + 1] == sPref[b]);
            if (b < B) pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
          }
        }
      }
      return;
    }
  }

  // =========================================================== consumer warps
  uint32_t qB[NH][NTK][NR];    // QK^T B operands: column gid = (head gid/2 + 4 nh, limb gid%2), channels 16 r + 4 tid + {0..3};
                               // channel-wise keys: n-tile 0 carries (byte 2 signed, none), n-tile 1 (byte 1, byte 0) unsigned
  float hs[NH];                // c1 / fixed-point scale of q, own heads (tid + 4 nh)
  float qsum[NH][NGK];         // c1 * sum of q over each key group, own heads
  float zq[NH];                // channel-wise keys: c1 * sum_d q_d z_d of the current page, own heads
  float m_ref[NH], l[NH], zacc[NH][NGV];
  int Oi[NTV][MT][4];          // PV accumulators: NH = 1: n-tiles (limb 3, 2 | limb 1, 0) of head tid; NH = 2: (head tid:
                               // limb 2, 1 | head tid + 4: limb 2, 1 | limb 0 of both)
  constexpr float PONE = (float)(1u << (kPBits<NH> - 1)) * 2.0f;     // 2^PBITS
  // sscale = 2^PBITS / s_lim, s_lim a power of two above every value scale folded into the weights so far (2^-40 at first)
  float sscale = PONE / 9.094947e-13f;
  float* myM = sMaster + warp * NHEADS * MSTRIDE;
  const int grp = warp >> 2, wq = warp & 3;       // page group of this warp, and its 32-token block inside a page
  int page_no = 0;
  int stage = grp;             // ring slot and parity of this group's next page (pages go to the groups in turn)
  uint32_t phase = 0;
  int turn = 0;                // CTA-wide page counter modulo NG
  bool aborted = false;
  constexpr int KCB = (KW < 4 ? KW : 4) * 4;     // bytes of a lane chunk's first quad of key words
  const int lane_k = (wq * 32 + gid) * K_ROW_BYTES + tid * KCB;
  const int lane_km = K_META_OFF + (wq * 32 + gid) * 4 * NGK;
  const int lane_v = V_CODES_OFF + wq * V_BLOCK_BYTES + lane * 16;
  const int lane_vm = V_META_OFF + (wq * 32 + gid) * 4 * NGV;

  // Fold the int32 accumulators into the warp's fp32 master (each (head, channel) belongs to one lane) and clear them.
  auto flush_acc = [&]() {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const float fw = (1.0f / sscale) / (float)(1 << (VB * (mt % FPBV)));      // sscale is a power of two
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int d = 16 * mt + 8 * r + gid;
        if constexpr (NH == 1) {
          const float v = fmaf((float)Oi[0][mt][2 * r], 16777216.f,
                               fmaf((float)Oi[0][mt][2 * r + 1], 65536.f,
                                    fmaf((float)Oi[1][mt][2 * r], 256.f, (float)Oi[1][mt][2 * r + 1])));
          myM[tid * MSTRIDE + d] += v * fw;
        } else {
          const float v0 = fmaf((float)Oi[0][mt][2 * r], 65536.f, fmaf((float)Oi[0][mt][2 * r + 1], 256.f,
                                                                        (float)Oi[2][mt][2 * r]));
          const float v1 = fmaf((float)Oi[1][mt][2 * r], 65536.f, fmaf((float)Oi[1][mt][2 * r + 1], 256.f,
                                                                        (float)Oi[2][mt][2 * r + 1]));
          myM[tid * MSTRIDE + d] += v0 * fw;
          myM[(tid + 4) * MSTRIDE + d] += v1 * fw;
        }
      }
#pragma unroll
      for (int nt = 0; nt < NTV; ++nt) { Oi[nt][mt][0] = Oi[nt][mt][1] = Oi[nt][mt][2] = Oi[nt][mt][3] = 0; }
    }
  };

  for (long long x = x_lo; x < x_hi;) {
    const int seg_pages = (int)min((long long)(pages_b - page), x_hi - x);
    const int n_tok = paged_len(c.seq_len, b, g.capacity, g.R);   // tokens of the sequence that are in the pages
    // a block is unmasked when all of its 32 tokens exist and every query row may see them (several causal rows:
    // row r sees the first n - (rows - 1 - r) tokens of the n the sequence holds, window included)
    const int n_unmasked = min(n_tok, clamped_len(c.seq_len, b, g.capacity) - (g.rows - 1));
    const int stream = b * Hkv + h;
    // which of the stream's partials this CTA writes, and how many there are: one thread works it out now, everybody
    // reads it after the barrier at the segment's end (the barrier that closed the last segment keeps its readers apart)
    if (tid_ == 0) {
      const long long xs = (long long)sVPref[b] + (long long)h * (pages_b + GAP) + GAP;   // first real page of this stream, virtual axis
      const int c_first = cta_of_virtual<WAVES>(plan, waves, xs);
      sMisc[8] = (int)blockIdx.x - c_first;
      sMisc[9] = cta_of_virtual<WAVES>(plan, waves, xs + pages_b - 1) - c_first + 1;
    }

    // ---- segment start: q operands, group sums and a clean state for this stream's heads
    {
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        const int hb = (gid >> 1) + 4 * nh;                          // head of this lane's operand column
        float qv[NR][4];
        float amax = 0.f;
        if constexpr (KAXIS == 0) amax = load_q_lane<D>(g, c, q, b, h, hb, tid, qv);
        amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 2));
        if constexpr (KAXIS == 1) {
          // channel-wise keys: the operands depend on the page's scales; the preparation warp makes them per page
          hs[nh] = 0.f;
        } else {
          // 16-bit fixed point relative to the head's largest entry: Q = rint(q * scale), |Q| <= 32512
          const float scale = amax > 0.f ? kQFix / amax : 0.f;
          const float hsb = amax > 0.f ? c1 / scale : 0.f;
          int qs[NGK];
#pragma unroll
          for (int j = 0; j < NGK; ++j) qs[j] = 0;
#pragma unroll
          for (int r = 0; r < NR; ++r) qB[nh][0][r] = fixed_point_limb(qv[r], scale, gid & 1, qs[r / (NR / NGK)]);
          hs[nh] = __shfl_sync(FULL, hsb, 8 * tid);
          // the zero-point term uses the sum of the same fixed-point q the MMAs see: the two large terms
          // s (q . c) and z sum(q) of a logit then cancel exactly as they do for the exact q
#pragma unroll
          for (int j = 0; j < NGK; ++j) {
            int v = qs[j];
            v += __shfl_xor_sync(FULL, v, 1);
            v += __shfl_xor_sync(FULL, v, 2);
            qsum[nh][j] = hs[nh] * (float)__shfl_sync(FULL, v, 8 * tid);
          }
        }
        m_ref[nh] = -INFINITY;
        l[nh] = 0.f;
        zq[nh] = 0.f;
#pragma unroll
        for (int j = 0; j < NGV; ++j) zacc[nh][j] = 0.f;
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
        for (int nt = 0; nt < NTV; ++nt) { Oi[nt][mt][0] = Oi[nt][mt][1] = Oi[nt][mt][2] = Oi[nt][mt][3] = 0; }
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + gid] = 0.f;
          myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + 8 + gid] = 0.f;
        }
      }
    }

    for (int pp = 0; pp < seg_pages; ++pp) {
      const bool mine = turn == grp;
      if (++turn == NG) turn = 0;
      if (!mine) continue;
      const int nv = min(kPageTokens, n_tok - (page + pp) * kPageTokens);
      const bool tail_k = (KAXIS == 1) && (nv < kPageTokens);
      if (!aborted) {
        const bool got = mbar_wait(bar0 + 8 * stage, phase, wait_ns);
        if (!__all_sync(FULL, got)) {
          aborted = true;
          *abort_flag = 1;
          if (lane == 0) atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
        }
      }
      const uint8_t* sp = smem + stage * sl.page_stride;

      // ---- channel-wise keys: the page's operands come from the preparation warp (stage buffer, `ready` barrier)
      if constexpr (KAXIS == 1) {
        if (!aborted) {
          const bool got = mbar_wait(bar0 + 8 * (2 * stages + stage), phase, wait_ns);
          if (!__all_sync(FULL, got)) {
            aborted = true;
            *abort_flag = 1;
            if (lane == 0) atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
          }
        }
        if (!aborted) {
          constexpr int CSB = NH * 2 * NR * 32 * 4 + 64;
          const uint32_t* ops = reinterpret_cast<const uint32_t*>(smem + sl.chan_off + stage * CSB);
          const float* opf = reinterpret_cast<const float*>(ops + NH * 2 * NR * 32);
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
            for (int nt = 0; nt < NTK; ++nt) {
#pragma unroll
              for (int r = 0; r < NR; ++r) qB[nh][nt][r] = ops[((nh * 2 + nt) * NR + r) * 32 + lane];
            }
            zq[nh] = opf[tid + 4 * nh];
            hs[nh] = opf[8 + tid + 4 * nh];
          }
        }
      }

      if (!aborted && wq * 32 < nv) {
        const uint8_t* sp_k = sp + lane_k;
        const uint8_t* sp_km = sp + lane_km;
        const uint8_t* sp_v = sp + lane_v;
        const uint8_t* sp_vm = sp + lane_vm;

        auto do_block = [&](auto masked_tag) {
          constexpr bool MASKED = decltype(masked_tag)::value;
          float L[2][2][NH];                 // [tile][row gid / gid + 8][head]
          bool vld[2][2];
          // ------------------------------------------------------------ logits of the block's two 16-token tiles
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const int tok0 = wq * 32 + 16 * u + gid;        // page-local tokens of this lane's two rows: tok0, tok0 + 8
            vld[u][0] = !MASKED || tok0 < nv;
            vld[u][1] = !MASKED || tok0 + 8 < nv;
            if (KAXIS == 1 && tail_k) {
              // tokens of the incomplete block: fp16 keys from the tail against q as fp16 high + low parts (operand
              // column gid = (head gid/2 + 4 nh, part gid%2), so lane columns 2 tid, 2 tid + 1 are the two parts of
              // head tid + 4 nh)
              const uint16_t* tl = c.k_tail + ((size_t)stream * kPageTokens + tok0) * D;
#pragma unroll
              for (int nh = 0; nh < NH; ++nh) {
                float S[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int r = 0; r < NR; ++r) {
                  uint2 ra = make_uint2(0u, 0u), rb = make_uint2(0u, 0u);
                  if (vld[u][0]) ra = *reinterpret_cast<const uint2*>(tl + 16 * r + 4 * tid);
                  if (vld[u][1]) rb = *reinterpret_cast<const uint2*>(tl + 8 * D + 16 * r + 4 * tid);
                  const uint32_t a0 = __byte_perm(ra.x, ra.y, 0x5410), a1 = __byte_perm(rb.x, rb.y, 0x5410);
                  const uint32_t a2 = __byte_perm(ra.x, ra.y, 0x7632), a3 = __byte_perm(rb.x, rb.y, 0x7632);
                  mma16816(S, a0, a1, a2, a3, qB[nh][0][r], qB[nh][NTK - 1][r]);    // q's fp16 parts, made by the preparation warp
                }
                L[u][0][nh] = c1 * (S[0] + S[1]);
                L[u][1][nh] = c1 * (S[2] + S[3]);
              }
            } else {
              uint32_t ka[KW], kb2[KW];
              const uint8_t* krow = sp_k + u * (16 * K_ROW_BYTES);           // this lane's chunk of row tok0
              load_words<KW>(krow, 64, ka);
              load_words<KW>(krow + 8 * K_ROW_BYTES, 64, kb2);
              int S[NGK][NH][NTK][4];
#pragma unroll
              for (int j = 0; j < NGK; ++j) {
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
                  for (int nt = 0; nt < NTK; ++nt) { S[j][nh][nt][0] = S[j][nh][nt][1] = S[j][nh][nt][2] = S[j][nh][nt][3] = 0; }
                }
              }
#pragma unroll
              for (int s = 0; s < KS32; ++s) {
                const int j = s / (KS32 / NGK);
                const uint32_t a0 = key_slot<KB, KW>(ka, 2 * s), a1 = key_slot<KB, KW>(kb2, 2 * s);
                const uint32_t a2 = key_slot<KB, KW>(ka, 2 * s + 1), a3 = key_slot<KB, KW>(kb2, 2 * s + 1);
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
                  for (int nt = 0; nt < NTK; ++nt) {
                    if (nt == 0) mma16832_u8s8(S[j][nh][nt], a0, a1, a2, a3, qB[nh][nt][2 * s], qB[nh][nt][2 * s + 1]);
                    else mma16832_u8u8(S[j][nh][nt], a0, a1, a2, a3, qB[nh][nt][2 * s], qB[nh][nt][2 * s + 1]);
                  }
                }
              }
              // accumulator columns 2 tid, 2 tid + 1 = (hi, lo) limbs of head tid + 4 nh: sum_d code_d Q_d = 256 hi + lo
              // (channel-wise keys: the signed top byte in n-tile 0, the two unsigned lower bytes in n-tile 1, combined in fp32)
              if constexpr (KAXIS == 1) {
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) {
                  const float t0 = fmaf((float)S[0][nh][0][0], 65536.f, fmaf((float)S[0][nh][NTK - 1][0], 256.f, (float)S[0][nh][NTK - 1][1]));
                  const float t1 = fmaf((float)S[0][nh][0][2], 65536.f, fmaf((float)S[0][nh][NTK - 1][2], 256.f, (float)S[0][nh][NTK - 1][3]));
                  L[u][0][nh] = fmaf(t0, hs[nh], zq[nh]);
                  L[u][1][nh] = fmaf(t1, hs[nh], zq[nh]);
                }
              } else {
                const uint32_t* km = reinterpret_cast<const uint32_t*>(sp_km + u * (16 * 4 * NGK));   // row tok0
#pragma unroll
                for (int nh = 0; nh < NH; ++nh) { L[u][0][nh] = 0.f; L[u][1][nh] = 0.f; }
#pragma unroll
                for (int j = 0; j < NGK; ++j) {
                  const float2 ma = __half22float2(as_h2(km[j]));                       // (scale, zero) of row tok0
                  const float2 mb = __half22float2(as_h2(km[8 * NGK + j]));             // ... of row tok0 + 8
#pragma unroll
                  for (int nh = 0; nh < NH; ++nh) {
                    const float t0 = (float)(S[j][nh][0][0] * 256 + S[j][nh][0][1]);
                    const float t1 = (float)(S[j][nh][0][2] * 256 + S[j][nh][0][3]);
                    L[u][0][nh] += fmaf(ma.x * hs[nh], t0, ma.y * qsum[nh][j]);
                    L[u][1][nh] += fmaf(mb.x * hs[nh], t1, mb.y * qsum[nh][j]);
                  }
                }
              }
            }
            if (MASKED) {
              const int tokg = (page + pp) * kPageTokens + tok0;        // position of row tok0 in the sequence
              const int n_all = clamped_len(c.seq_len, b, g.capacity);
#pragma unroll
              for (int nh = 0; nh < NH; ++nh) {
                // tokens the lane's head may attend to: the causal limit of its query row
                const int lim = n_all - (g.rows - 1 - min((tid + 4 * nh) / Gq, g.rows - 1));
                if (!vld[u][0] || tokg >= lim) L[u][0][nh] = -INFINITY;
                if (!vld[u][1] || tokg + 8 >= lim) L[u][1][nh] = -INFINITY;
              }
            }
          }

          // ------------------------------------------------------------ value scales and zero-points of the four rows
          float sv[2][2][NGV], zv[2][2][NGV];
          float smax = 0.f;
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            const uint32_t* vm = reinterpret_cast<const uint32_t*>(sp_vm + u * (16 * 4 * NGV));
#pragma unroll
            for (int j = 0; j < NGV; ++j) {
              const uint32_t ma = vld[u][0] ? vm[j] : 0u;
              const uint32_t mb = vld[u][1] ? vm[8 * NGV + j] : 0u;
              const float2 fa = __half22float2(as_h2(ma)), fb = __half22float2(as_h2(mb));
              sv[u][0][j] = fa.x; zv[u][0][j] = fa.y;
              sv[u][1][j] = fb.x; zv[u][1][j] = fb.y;
              smax = fmaxf(smax, fmaxf(fa.x, fb.x));
            }
          }

          // ------------------------------------------------------------ softmax reference / scale check (rarely taken)
          float bmax[NH];
          // (the int32 accumulators are also folded every kFlushBlocks pages, long before they can overflow)
          bool trig = (smax * sscale >= PONE) | ((page_no & (kFlushBlocks - 1)) == kFlushBlocks - 1);
#pragma unroll
          for (int nh = 0; nh < NH; ++nh) {
            bmax[nh] = fmaxf(fmaxf(L[0][0][nh], L[0][1][nh]), fmaxf(L[1][0][nh], L[1][1][nh]));
            trig |= bmax[nh] > m_ref[nh];
          }
          if (__any_sync(FULL, trig)) {
            flush_acc();                                   // with the scale the accumulated weights were made with
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) smax = fmaxf(smax, __shfl_xor_sync(FULL, smax, off));
            if (smax * sscale >= PONE) {
              // next power of two above the largest value scale: p * s * sscale < 2^PBITS for every p <= 1
              sscale = PONE / __uint_as_float((__float_as_uint(smax) & 0x7F800000u) + 0x00800000u);
            }
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) {
              float bm = bmax[nh];
#pragma unroll
              for (int off = 4; off < 32; off <<= 1) bm = fmaxf(bm, __shfl_xor_sync(FULL, bm, off));
              if (bm > m_ref[nh]) {
                const float nref = bm + kHeadroom<NH>;
                const float a = (m_ref[nh] == -INFINITY) ? 0.f : ex2(m_ref[nh] - nref);
                m_ref[nh] = nref;
                l[nh] *= a;
#pragma unroll
                for (int j = 0; j < NGV; ++j) zacc[nh][j] *= a;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                  myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + gid] *= a;
                  myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + 8 + gid] *= a;
                }
              }
            }
          }

          // ------------------------------------------------------------ weights: p = 2^(logit - reference) <= 2^-headroom,
          // P = rint(p * s_V * sscale) < 2^PBITS
          uint32_t bV[NGV][NTV][2];
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            float p[2][NH];
#pragma unroll
            for (int nh = 0; nh < NH; ++nh) {
              p[0][nh] = ex2(L[u][0][nh] - m_ref[nh]);
              p[1][nh] = ex2(L[u][1][nh] - m_ref[nh]);
              if (MASKED) {       // a head that has seen no token yet has no reference: its weights are zero
                if (L[u][0][nh] == -INFINITY) p[0][nh] = 0.f;
                if (L[u][1][nh] == -INFINITY) p[1][nh] = 0.f;
              }
              l[nh] += p[0][nh] + p[1][nh];
            }
#pragma unroll
            for (int j = 0; j < NGV; ++j) {
              const float sa = sv[u][0][j] * sscale, sb = sv[u][1][j] * sscale;
              uint32_t Pa[NH], Pb[NH];
#pragma unroll
              for (int nh = 0; nh < NH; ++nh) {
                zacc[nh][j] = fmaf(p[0][nh], zv[u][0][j], fmaf(p[1][nh], zv[u][1][j], zacc[nh][j]));
                Pa[nh] = __float2uint_rn(p[0][nh] * sa);      // token tok0
                Pb[nh] = __float2uint_rn(p[1][nh] * sb);      // token tok0 + 8
              }
              // one 16-bit element per (column, lane row) = that column's limb of tokens (tok0, tok0 + 8); the 8x8
              // transpose turns lane columns into the B operand (column = lane/4, tokens 2t, 2t+8, 2t+1, 2t+9)
              if constexpr (NH == 1) {
                bV[j][0][u] = movmatrix_trans(prmt(Pa[0], Pb[0], 0x6273));       // limbs (3, 2): bytes a3 b3 a2 b2
                bV[j][1][u] = movmatrix_trans(prmt(Pa[0], Pb[0], 0x4051));       // limbs (1, 0): bytes a1 b1 a0 b0
              } else {
                bV[j][0][u] = movmatrix_trans(prmt(Pa[0], Pb[0], 0x5162));       // head tid: (hi, mid)
                bV[j][1][u] = movmatrix_trans(prmt(Pa[1], Pb[1], 0x5162));       // head tid + 4: (hi, mid)
                bV[j][2][u] = movmatrix_trans(prmt(prmt(Pa[0], Pb[0], 0x0040), prmt(Pa[1], Pb[1], 0x0040), 0x5410));
              }
            }
          }

          // ------------------------------------------------------------ PV on the raw code bytes: one mask per register.
          // Field f of every byte belongs to m-tile FPBV q + f, whose accumulators carry the factor 2^(VB f).
#pragma unroll
          for (int qd = 0; qd < VQ; ++qd) {
            const uint4 vw = *reinterpret_cast<const uint4*>(sp_v + qd * 512);
#pragma unroll
            for (int f = 0; f < FPBV; ++f) {
              const int mt = FPBV * qd + f;
              const int j = mt / (MT / NGV);
              uint32_t a0 = vw.x, a2 = vw.y, a1 = vw.z, a3 = vw.w;     // words (rh, kh) = (0,0), (0,1), (1,0), (1,1)
              if constexpr (VB != 8) {
                constexpr uint32_t M0 = ((1u << VB) - 1u) * 0x01010101u;
                const uint32_t mask = M0 << (VB * f);
                a0 &= mask; a1 &= mask; a2 &= mask; a3 &= mask;
              }
#pragma unroll
              for (int nt = 0; nt < NTV; ++nt) mma16832_u8u8(Oi[nt][mt], a0, a1, a2, a3, bV[j][nt][0], bV[j][nt][1]);
            }
          }
        };

        // the masked variant also serves the last tokens when several causal query rows see different prefixes
        if ((page + pp) * kPageTokens + wq * 32 + 32 <= n_unmasked) do_block(std::false_type{});
        else do_block(std::true_type{});
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar0 + 8 * (stages + stage));
      stage += NG;
      if (stage >= stages) { stage -= stages; phase ^= 1; }
      ++page_no;
    }

    // ---- segment end: finish this warp's state, combine the NW warps, write the partial
    {
      flush_acc();
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          l[nh] += __shfl_xor_sync(FULL, l[nh], off);
#pragma unroll
          for (int j = 0; j < NGV; ++j) zacc[nh][j] += __shfl_xor_sync(FULL, zacc[nh][j], off);
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int j = mt / (MT / NGV);
          myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + gid] += zacc[nh][j];
          myM[(tid + 4 * nh) * MSTRIDE + 16 * mt + 8 + gid] += zacc[nh][j];
        }
        if (gid == 0) {
          sML[(warp * NHEADS + tid + 4 * nh) * 2 + 0] = m_ref[nh];
          sML[(warp * NHEADS + tid + 4 * nh) * 2 + 1] = l[nh];
        }
      }
      named_bar_sync(1, NCONS);
      // The flat split gives a stream to a run of consecutive CTAs, one partial slot each.  A CTA that holds the
      // whole stream writes the output at once; otherwise it stores its partial, counts itself in, and the CTA
      // that completes the count merges all partials of the stream by log-sum-exp and stores the output.
      const int slot = sMisc[8], n_part = sMisc[9];
      const bool has_win = clamped_len(c.seq_len, b, g.capacity) > n_tok;    // the window kernel left a partial in slot s_cap - 1
      if (slot >= 0 && slot < s_plan) {
        for (int idx = tid_; idx < G * D; idx += NCONS) {
          const int head = idx / D, d = idx % D;
          float mstar = -INFINITY;
#pragma unroll
          for (int w = 0; w < NW; ++w) mstar = fmaxf(mstar, sML[(w * NHEADS + head) * 2]);
          float o = 0.f, lsum = 0.f;
#pragma unroll
          for (int w = 0; w < NW; ++w) {
            const float mw = sML[(w * NHEADS + head) * 2];
            const float f = (mw == -INFINITY) ? 0.f : ex2(mw - mstar);
            o = fmaf(f, sMaster[(w * NHEADS + head) * MSTRIDE + d], o);
            lsum = fmaf(f, sML[(w * NHEADS + head) * 2 + 1], lsum);
          }
          if (n_part == 1 && !has_win) {
            const float r = lsum > 0.f ? o / lsum : 0.f;
            const size_t oi = (((size_t)b * g.rows + head / Gq) * g.Hq + (size_t)h * Gq + head % Gq) * D + d;
            if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = r;
            else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(r, out_dtype);
          } else {
            float* dst = ws + (((size_t)stream * s_cap + slot) * G + head) * (D + 2);
            if (d == 0) { dst[0] = mstar; dst[1] = lsum; }
            dst[2 + d] = o;
          }
        }
        if (n_part > 1 || has_win) {
          __threadfence();
          named_bar_sync(1, NCONS);
          if (tid_ == 0) *n_published = (int)tagged_count(counts + stream, id40);
          named_bar_sync(1, NCONS);
          if (*n_published == n_part) {
            __threadfence();
            for (int idx = tid_; idx < G * D; idx += NCONS) {
              const int head = idx / D, d = idx % D;
              const float* base = ws + (((size_t)stream * s_cap) * G + head) * (D + 2);
              const size_t slot_stride = (size_t)G * (D + 2);
              float mstar = -INFINITY, num = 0.f, den = 0.f;
              const int n_merge = n_part + (has_win ? 1 : 0);
              for (int j0 = 0; j0 < n_merge; j0 += 4) {
                float mj[4], lj[4], oj[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {                   // issue the loads of a batch before using any
                  const bool on = j0 + u < n_merge;
                  const int sj = (j0 + u < n_part) ? j0 + u : s_cap - 1;      // the window's partial comes last
                  const float* pj = base + (size_t)(on ? sj : 0) * slot_stride;
                  mj[u] = on ? __ldcg(pj) : -INFINITY;
                  lj[u] = on ? __ldcg(pj + 1) : 0.f;
                  oj[u] = on ? __ldcg(pj + 2 + d) : 0.f;
                }
                float mb = mstar;
#pragma unroll
                for (int u = 0; u < 4; ++u) mb = fmaxf(mb, mj[u]);
                if (mb == -INFINITY) continue;
                const float keep = (mstar == -INFINITY) ? 0.f : ex2(mstar - mb);
                num *= keep;
                den *= keep;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float wgt = (mj[u] == -INFINITY) ? 0.f : ex2(mj[u] - mb);
                  num = fmaf(wgt, oj[u], num);
                  den = fmaf(wgt, lj[u], den);
                }
                mstar = mb;
              }
              const float r = den > 0.f ? num / den : 0.f;
              const size_t oi = (((size_t)b * g.rows + head / Gq) * g.Hq + (size_t)h * Gq + head % Gq) * D + d;
              if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = r;
              else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(r, out_dtype);
            }
            if (tid_ == 0) counts[stream] = 0ull;
          }
        }
      }
      named_bar_sync(1, NCONS);
    }

    // ---- advance the cursor past this segment
    x += seg_pages;
    page += seg_pages;
    if (page == pages_b) {
      page = 0;
      if (++h == Hkv) {
        h = 0;
        do { ++b; } while (b < B && sPref[b + 1] == sPref[b]);
        if (b < B) pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
      }
    }
  }
}

// Launches one instantiation; defined per instantiation unit.
template <int D, int KB, int VB, int KAXIS, int NGK, int NGV, int NH, int NW, int MINB>
int launch_mma_inst(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap,
                    void* out, int out_dtype, unsigned long long call_id, unsigned long long wait_ns, long long skip_x,
                    cudaStream_t stream) {
  const int budget = (227 * 1024) / MINB - 1024;            // shared memory per CTA for MINB resident CTAs per SM
  int stages = (budget - smem_layout(0, 0, NW, g.B, D, NH, KAXIS == 1).total) /
               (((g.page_bytes + 127) & ~127) + (KAXIS == 1 ? chan_stage_bytes(D, NH) : 0));
  // Deeper rings do not help: the kernel is bound by its arithmetic, not by copy latency, and more bytes in
  // flight cost DRAM efficiency (8B shape, K4V2: 5 stages 95 us, 3-4 stages 91-92 us, 2 stages 97 us).
  if (stages > 4) stages = 4;
  if (stages < 2 || stages < NW / 4) return KVQ_ERR_UNSUPPORTED;
  const SmemLayout sl = smem_layout(g.page_bytes, stages, NW, g.B, D, NH, KAXIS == 1);
  auto kern = decode_mma_kernel<D, KB, VB, KAXIS, NGK, NGV, NH, NW, MINB>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sl.total) != cudaSuccess)
    return KVQ_ERR_CUDA_LAUNCH;
  kern<<<148 * MINB, (NW + 1 + (KAXIS == 1 ? 1 : 0)) * 32, sl.total, stream>>>(g, c, static_cast<const uint16_t*>(q), c1, ws, s_cap,
                                                         stages, out, out_dtype, call_id, wait_ns, skip_x);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace mma
}  // namespace kvq
