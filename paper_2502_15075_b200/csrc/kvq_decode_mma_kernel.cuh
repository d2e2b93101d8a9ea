// The templated fast decode kernel (see kvq_decode_mma.cuh for the design).
#pragma once

#include <type_traits>

#include "kvq_decode_mma.cuh"

namespace kvq {
namespace mma {

constexpr int kMaxBatchFlat = 1024;   // the flat partition keeps a per-batch prefix in shared memory

// Flat split of all pages over the grid, identical in the decode and the merge kernel.
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

// Shared-memory carve-up (dynamic): ring | barriers | prefix | combine buffer
struct SmemLayout {
  int page_stride, ring_bytes, bar_off, pref_off, misc_off, comb_off, chan_off, total;
};
// chan: channel-wise keys need, per CTA, two buffers of per-page q limbs (3 x D/16 x 32 words), the partial
// zero-point sums (64 floats) and the stream's q in fp32 (D/16 x 32 x 4 floats).
__host__ __device__ inline SmemLayout smem_layout(int page_bytes, int stages, int nw, int D, bool chan) {
  SmemLayout s;
  s.page_stride = (page_bytes + 127) & ~127;
  s.ring_bytes = s.page_stride * stages;
  s.bar_off = s.ring_bytes;
  s.pref_off = s.bar_off + 16 * 8 * 2;                      // up to 16 stages x (full, empty)
  s.misc_off = s.pref_off + (kMaxBatchFlat + 1) * 4;
  s.comb_off = (s.misc_off + 64 + 127) & ~127;
  int per_warp = (D / 16 * 4 + 4) * 32 * 4;                 // O fragments + m, l per lane
  s.chan_off = s.comb_off + (nw / 2 > 0 ? nw / 2 : 1) * per_warp;
  s.total = s.chan_off + (chan ? (2 * 3 * (D / 16) * 32 * 4 + 2 * 64 * 4 + (D / 16) * 32 * 16) : 0);
  return s;
}

// Template parameters: head_dim, key bits, value bits, key axis (0 token-wise: keys go through integer MMAs
// on the raw code bytes with q in 22-bit fixed point split into NL = 3 signed bytes; 1 channel-wise: fp16 MMAs
// with the channel scales folded into q per page), key / value groups per row, q limbs, consumer warps,
// resident CTAs per SM.
template <int D, int KB, int VB, int KAXIS, int NGK, int NGV, int NL, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1) * 32, MINB)
decode_mma_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ q, float c1, float* __restrict__ ws,
                  int s_cap, int stages) {
  constexpr int NR = D / 16;                // 16-channel register slots per row (r index of the key layout)
  constexpr int KS32 = D / 32;              // k-steps of an 8-bit MMA
  constexpr int MT = D / 16;                // m-tiles of PV (channels)
  constexpr int KW = D * KB / 128;          // K words per lane per token row
  constexpr int VW = D * VB / 64;           // V words per lane per 16-token tile
  constexpr int FPB = 8 / KB;               // key fields per byte
  constexpr int NPOS = 8 / VB;              // value code positions inside a byte
  constexpr int K_ROW_BYTES = D * KB / 8;
  constexpr int V_TILE_BYTES = 16 * D * VB / 8;
  constexpr int NCONS = NW * 32;
  constexpr int TPW = (kPageTokens / 16) / NW;   // tiles per warp per page
  constexpr uint32_t FULL = 0xffffffffu;
  static_assert(KAXIS == 0 || KB != 2, "channel-wise 2-bit keys are not instantiated");

  extern __shared__ __align__(128) uint8_t smem[];
  const SmemLayout sl = smem_layout(g.page_bytes, stages, NW, D, KAXIS == 1);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sl.bar_off);   // full[0..stages), empty[0..stages)
  int* sPref = reinterpret_cast<int*>(smem + sl.pref_off);
  int* sMisc = reinterpret_cast<int*>(smem + sl.misc_off);           // [0] pages_max, [1] abort flag
  float* sComb = reinterpret_cast<float*>(smem + sl.comb_off);

  const int tid_ = threadIdx.x, lane = tid_ & 31, warp = tid_ >> 5;
  const int gid = lane >> 2, tid = lane & 3;
  const int B = g.B, Hkv = g.Hkv, G = g.G;

  // ---- plan: pages per sequence, prefix over the batch
  if (tid_ == 0) { sPref[0] = 0; sMisc[0] = 0; sMisc[1] = 0; }
  __syncthreads();
  for (int b = tid_; b < B; b += blockDim.x) {
    int pages = (clamped_len(c.seq_len, b, g.capacity) + kPageTokens - 1) >> 7;
    sPref[b + 1] = pages * Hkv;
    atomicMax(&sMisc[0], pages);
  }
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int base = 0; base < B; base += 32) {
      int i = base + lane;
      int v = (i < B) ? sPref[i + 1] : 0;
      for (int off = 1; off < 32; off <<= 1) {
        int u = __shfl_up_sync(FULL, v, off);
        if (lane >= off) v += u;
      }
      if (i < B) sPref[i + 1] = v + carry;
      carry += __shfl_sync(FULL, v, 31);
    }
  }
  if (tid_ == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[stages + s]), NW);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const FlatPlan plan = make_plan(sPref[B], sMisc[0], gridDim.x, s_cap);
  if (plan.N == 0 || (int)blockIdx.x >= plan.c_eff) return;
  const long long x_lo = plan.lo(blockIdx.x), x_hi = plan.lo(blockIdx.x + 1);

  // ---- cursor: first page of this CTA -> (b, h, page)
  int b = 0;
  {
    int lo_ = 0, hi_ = B - 1;            // last b with sPref[b] <= x_lo
    while (lo_ < hi_) {
      int mid = (lo_ + hi_ + 1) >> 1;
      if (sPref[mid] <= x_lo) lo_ = mid; else hi_ = mid - 1;
    }
    b = lo_;
  }
  int pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
  int h = (int)((x_lo - sPref[b]) / pages_b);
  int page = (int)((x_lo - sPref[b]) % pages_b);
  const uint32_t ring = smem_u32(smem);
  const uint32_t bar0 = smem_u32(bars);
  volatile int* abort_flag = sMisc + 1;

  // =========================================================== producer warp
  if (warp == NW) {
    if (lane == 0) {
      int it = 0, stage = 0;
      uint32_t phase = 1;                // parity of the previous round of `empty`
      bool ok = true;
      for (long long x = x_lo; x < x_hi; ++x, ++it) {
        if (it >= stages) {
          ok = mbar_wait(bar0 + 8 * (stages + stage), phase);
          if (!ok || *abort_flag) { ok = false; break; }
        }
        const uint8_t* src = c.pages + ((size_t)(b * Hkv + h) * g.n_pages + page) * (size_t)g.page_bytes;
        const uint32_t fb = bar0 + 8 * stage;
        mbar_expect_tx(fb, (uint32_t)g.page_bytes);
        bulk_load(ring + stage * sl.page_stride, src, (uint32_t)g.page_bytes, fb);
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
        // gave up: flag it, then let the copies already in flight land before the CTA exits
        *abort_flag = 1;
        atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
        for (int k = 1; k <= stages && k <= it; ++k) {
          const int j = it - k;
          mbar_wait(bar0 + 8 * (j % stages), (j / stages) & 1);
        }
      }
    }
    return;
  }

  // =========================================================== consumer warps
  // q operands: signed-byte limbs (token-wise keys) or fp16 pairs (channel-wise keys), heads >= G are zero.
  // Slot r holds channels 16 r + 4 tid + {0..3} of head gid.
  uint32_t ql[NL][NR];
  constexpr int OWN = (NR / NW > 0) ? NR / NW : 1;     // channel-wise keys: slots whose per-page limbs this warp makes
  float qk[(KAXIS == 1) ? OWN : 1][4];       // ... and the stream's q (rotated if asked) on those slots, fp32
  float amax_h = 0.f;                        // ... and max |q| of head gid
  uint32_t* sB = reinterpret_cast<uint32_t*>(smem + sl.chan_off);          // [2][NL][NR][32] per-page q limbs
  float* sZ = reinterpret_cast<float*>(smem + sl.chan_off + 2 * NL * NR * 32 * 4);   // [2][8 heads][8] partial sums
  float4* sQ = reinterpret_cast<float4*>(smem + sl.chan_off + 2 * NL * NR * 32 * 4 + 2 * 64 * 4);   // [NR][32]
  int page_no = 0;
  float qsum[2][NGK];                        // c1 * sum of q over each key group, heads (2 tid, 2 tid + 1)
  float hs0 = 0.f, hs1 = 0.f;                // c1 / fixed-point scale of heads (2 tid, 2 tid + 1)
  float O[MT][4];
  float zacc[2][NGV];
  float m0, m1, l0, l1;
  int stage = 0;
  uint32_t phase = 0;
  bool aborted = false;
  // byte offsets inside a page of this lane's operands for the warp's first tile (rows warp*16 + gid, +8)
  constexpr int KCB = (KW < 4 ? KW : 4) * 4, VCB = (VW < 4 ? VW : 4) * 4;     // bytes of a lane chunk's first quad
  const int lane_k = (warp * 16 + gid) * K_ROW_BYTES + tid * KCB;
  const int lane_km = g.k_meta_off + (warp * 16 + gid) * 4 * NGK;
  const int lane_v = g.v_codes_off + warp * V_TILE_BYTES + lane * VCB;
  const int lane_vm = g.v_meta_off + (warp * 16 + gid) * 4 * NGV;

  for (long long x = x_lo; x < x_hi;) {
    const int seg_pages = (int)min((long long)(pages_b - page), x_hi - x);
    const int n_tok = clamped_len(c.seq_len, b, g.capacity);
    const int stream = b * Hkv + h;

    // ---- segment start: q operands and group sums for this stream's heads
    {
      float part[NGK];
#pragma unroll
      for (int j = 0; j < NGK; ++j) part[j] = 0.f;
      float qv[NR][4];
      float amax = 0.f;
      const uint16_t* qrow = q + ((size_t)b * g.Hq + (size_t)h * G + gid) * D;
#pragma unroll
      for (int r = 0; r < NR; ++r) {
        uint2 raw = make_uint2(0u, 0u);
        if (gid < G) raw = *reinterpret_cast<const uint2*>(qrow + 16 * r + 4 * tid);
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
#pragma unroll
      for (int r = 0; r < NR; ++r) {
        float f[4] = {qv[r][0], qv[r][1], qv[r][2], qv[r][3]};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          amax = fmaxf(amax, fabsf(f[j]));
          part[r / (NR / NGK)] += f[j];
        }
      }
      static_assert(NL == 3, "three signed 8-bit limbs");
      amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 1));
      amax = fmaxf(amax, __shfl_xor_sync(FULL, amax, 2));
      if constexpr (KAXIS == 1) {
        // channel-wise keys: the limbs depend on the page's scales and are made per page; keep what that needs
        amax_h = amax;
#pragma unroll
        for (int i = 0; i < OWN; ++i) {
#pragma unroll
          for (int r = 0; r < NR; ++r) {       // (compile-time indices keep qv in registers)
            if (r == warp * OWN + i) {
#pragma unroll
              for (int j = 0; j < 4; ++j) qk[i][j] = qv[r][j];
            }
          }
        }
        named_bar_sync(2, NCONS);                       // nobody still reads the previous stream's copy
        if (warp == 0) {
#pragma unroll
          for (int r = 0; r < NR; ++r) sQ[r * 32 + lane] = make_float4(qv[r][0], qv[r][1], qv[r][2], qv[r][3]);
        }
        named_bar_sync(2, NCONS);
      }
      if constexpr (KAXIS == 0) {
        // per head: 22-bit fixed point relative to the head's largest entry, Q = rint(q * 2^k) with
        // |Q| < 2^22, split into three balanced signed bytes  Q = l0 * 65536 + l1 * 256 + l2
        int e = (int)((__float_as_uint(amax) >> 23) & 0xFF) - 127;
        e = max(e, -60);
        const int k = 21 - e;
        const float scale = __uint_as_float((uint32_t)(127 + k) << 23);
        const float hs = c1 * __uint_as_float((uint32_t)(127 - k) << 23);
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          fixed_point_limbs(qv[r], scale, ql[0][r], ql[1][r], ql[2][r]);
        }
        hs0 = __shfl_sync(FULL, hs, (2 * tid) * 4);
        hs1 = __shfl_sync(FULL, hs, (2 * tid + 1) * 4);
      }
#pragma unroll
      for (int j = 0; j < NGK; ++j) {
        float v = part[j];
        v += __shfl_xor_sync(FULL, v, 1);
        v += __shfl_xor_sync(FULL, v, 2);
        qsum[0][j] = c1 * __shfl_sync(FULL, v, (2 * tid) * 4);
        qsum[1][j] = c1 * __shfl_sync(FULL, v, (2 * tid + 1) * 4);
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) { O[mt][0] = O[mt][1] = O[mt][2] = O[mt][3] = 0.f; }
#pragma unroll
      for (int j = 0; j < NGV; ++j) { zacc[0][j] = zacc[1][j] = 0.f; }
      m0 = m1 = -INFINITY;
      l0 = l1 = 0.f;
    }

    for (int pp = 0; pp < seg_pages; ++pp) {
      const int nv = min(kPageTokens, n_tok - (page + pp) * kPageTokens);
      if (!aborted) {
        const bool got = mbar_wait(bar0 + 8 * stage, phase);
        if (!__all_sync(FULL, got)) {
          aborted = true;
          *abort_flag = 1;
          if (lane == 0) atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
        }
      }
      if (!aborted) {
        const uint8_t* sp = smem + stage * sl.page_stride;
        // this lane's first byte in each region for the warp's tile 0 (tile u adds a constant)
        const uint8_t* sp_k = sp + lane_k;
        const uint8_t* sp_km = sp + lane_km;
        const uint8_t* sp_v = sp + lane_v;
        const uint8_t* sp_vm = sp + lane_vm;
        const bool tail_k = (KAXIS == 1) && (nv < kPageTokens);
        const int ntiles = (nv + 15) >> 4;

        // ---- channel-wise keys: per page, the operand of the integer MMAs is q_d * s_d in 22-bit fixed point
        // (scale from max|q| of the head times the page's largest channel scale).  Each warp makes the limbs of its
        // own slots, all warps exchange them through shared memory; sum_d q_d z_d is summed in fp32 the same way.
        float zq0 = 0.f, zq1 = 0.f;
        if constexpr (KAXIS == 1) {
          if (!tail_k) {
            const int buf = page_no & 1;
            const uint32_t* km = reinterpret_cast<const uint32_t*>(sp + g.k_meta_off);
            float smax = 0.f;
            if (4 * lane < D) {
              const uint4 mm = *reinterpret_cast<const uint4*>(km + 4 * lane);
              smax = fmaxf(fmaxf(meta_s(mm.x), meta_s(mm.y)), fmaxf(meta_s(mm.z), meta_s(mm.w)));
            }
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) smax = fmaxf(smax, __shfl_xor_sync(FULL, smax, off));
            int e = (int)((__float_as_uint(amax_h * smax) >> 23) & 0xFF) - 127;
            e = max(e, -60);
            const int k = 21 - e;
            const float scale = __uint_as_float((uint32_t)(127 + k) << 23);
            const float hs = c1 * __uint_as_float((uint32_t)(127 - k) << 23);
            hs0 = __shfl_sync(FULL, hs, (2 * tid) * 4);
            hs1 = __shfl_sync(FULL, hs, (2 * tid + 1) * 4);
            float zsum = 0.f;
#pragma unroll
            for (int i = 0; i < OWN; ++i) {
              const int r = warp * OWN + i;
              if (r < NR) {
                const uint4 mm = *reinterpret_cast<const uint4*>(km + 16 * r + 4 * tid);   // (s,z) of 4 channels
                const uint32_t mw[4] = {mm.x, mm.y, mm.z, mm.w};
                float t[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const float2 sz = __half22float2(as_h2(mw[j]));
                  t[j] = qk[i][j] * sz.x;
                  zsum = fmaf(qk[i][j], sz.y, zsum);
                }
                uint32_t w0, w1, w2;
                fixed_point_limbs(t, scale, w0, w1, w2);
                sB[((buf * NL + 0) * NR + r) * 32 + lane] = w0;
                sB[((buf * NL + 1) * NR + r) * 32 + lane] = w1;
                sB[((buf * NL + 2) * NR + r) * 32 + lane] = w2;
              }
            }
            zsum += __shfl_xor_sync(FULL, zsum, 1);
            zsum += __shfl_xor_sync(FULL, zsum, 2);
            if (tid == 0 && warp * OWN < NR) sZ[(buf * 8 + gid) * 8 + warp] = zsum;
          }
        }
      }
      if constexpr (KAXIS == 1) {
        // every warp takes part in the exchange barrier of a full page, also after a timeout
        const int nv_b = min(kPageTokens, n_tok - (page + pp) * kPageTokens);
        if (nv_b == kPageTokens) named_bar_sync(2, NCONS);
      }
      if (!aborted) {
        const uint8_t* sp = smem + stage * sl.page_stride;
        const uint8_t* sp_k = sp + lane_k;
        const uint8_t* sp_km = sp + lane_km;
        const uint8_t* sp_v = sp + lane_v;
        const uint8_t* sp_vm = sp + lane_vm;
        const bool tail_k = (KAXIS == 1) && (nv < kPageTokens);
        const int ntiles = (nv + 15) >> 4;
        float zq0 = 0.f, zq1 = 0.f;
        if constexpr (KAXIS == 1) {
          if (!tail_k) {
            const int buf = page_no & 1;
#pragma unroll
            for (int l = 0; l < NL; ++l) {
#pragma unroll
              for (int r = 0; r < NR; ++r) ql[l][r] = sB[((buf * NL + l) * NR + r) * 32 + lane];
            }
            constexpr int NWR = (NR / OWN < NW) ? NR / OWN : NW;      // warps that contributed
#pragma unroll
            for (int w = 0; w < NWR; ++w) {
              zq0 += sZ[(buf * 8 + 2 * tid) * 8 + w];
              zq1 += sZ[(buf * 8 + 2 * tid + 1) * 8 + w];
            }
            zq0 *= c1;
            zq1 *= c1;
          }
        }

        // The TPW tiles this warp owns in the page (tile = warp + NW * u) are processed together: logits of all
        // of them, one joint running-max check, then probabilities and PV.  MASKED handles a partial page.
        auto logits = [&](const int u, const int tok0, const bool v0, const bool v1, float (&L)[4]) {
          if (KAXIS == 1 && tail_k) {
            // tokens of the incomplete block: fp16 keys from the tail against q as fp16 high + low parts
            float S[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};   // two chains, summed below
            const uint16_t* tl = c.k_tail + ((size_t)stream * kPageTokens + tok0) * D;
#pragma unroll
            for (int r = 0; r < NR; ++r) {
              uint2 ra = make_uint2(0u, 0u), rb = make_uint2(0u, 0u);
              if (v0) ra = *reinterpret_cast<const uint2*>(tl + 16 * r + 4 * tid);
              if (v1) rb = *reinterpret_cast<const uint2*>(tl + 8 * D + 16 * r + 4 * tid);
              const float4 qq = sQ[r * 32 + lane];
              uint32_t h0, l0_, h1, l1_;
              split_h2(qq.x, qq.z, h0, l0_);
              split_h2(qq.y, qq.w, h1, l1_);
              const uint32_t a0 = __byte_perm(ra.x, ra.y, 0x5410), a1 = __byte_perm(rb.x, rb.y, 0x5410);
              const uint32_t a2 = __byte_perm(ra.x, ra.y, 0x7632), a3 = __byte_perm(rb.x, rb.y, 0x7632);
              mma16816(S[r & 1], a0, a1, a2, a3, h0, h1);
              mma16816(S[r & 1], a0, a1, a2, a3, l0_, l1_);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) L[i] = c1 * (S[0][i] + S[1][i]);
          } else {
            uint32_t ka[KW], kb2[KW];
            const uint8_t* krow = sp_k + u * (NW * 16 * K_ROW_BYTES);      // this lane's chunk of row tok0
            load_words<KW>(krow, 64, ka);
            load_words<KW>(krow + 8 * K_ROW_BYTES, 64, kb2);
            int S[NGK][NL][4];
#pragma unroll
            for (int j = 0; j < NGK; ++j) {
#pragma unroll
              for (int l = 0; l < NL; ++l) { S[j][l][0] = S[j][l][1] = S[j][l][2] = S[j][l][3] = 0; }
            }
#pragma unroll
            for (int s = 0; s < KS32; ++s) {
              const int j = s / (KS32 / NGK);
              const uint32_t a0 = key_slot<KB, KW>(ka, 2 * s), a1 = key_slot<KB, KW>(kb2, 2 * s);
              const uint32_t a2 = key_slot<KB, KW>(ka, 2 * s + 1), a3 = key_slot<KB, KW>(kb2, 2 * s + 1);
#pragma unroll
              for (int l = 0; l < NL; ++l) mma16832_u8s8(S[j][l], a0, a1, a2, a3, ql[l][2 * s], ql[l][2 * s + 1]);
            }
            const uint32_t* km = reinterpret_cast<const uint32_t*>(sp_km + u * (NW * 16 * 4 * NGK));   // row tok0
            L[0] = L[1] = L[2] = L[3] = 0.f;
#pragma unroll
            for (int j = 0; j < NGK; ++j) {
              float t[4];
#pragma unroll
              for (int i = 0; i < 4; ++i)       // sum_d code_d * Q_d = (S0 * 256 + S1) * 256 + S2, exact up to the last step
                t[i] = fmaf((float)(S[j][0][i] * 256 + S[j][1][i]), 256.f, (float)S[j][2][i]);
              if constexpr (KAXIS == 1) {       // scales are already inside Q; the zero-points are one sum per page
                L[0] = fmaf(t[0], hs0, zq0); L[1] = fmaf(t[1], hs1, zq1);
                L[2] = fmaf(t[2], hs0, zq0); L[3] = fmaf(t[3], hs1, zq1);
                continue;
              }
              const float2 ma = __half22float2(as_h2(km[j]));                       // (scale, zero)
              const float2 mb = __half22float2(as_h2(km[8 * NGK + j]));
              L[0] += fmaf(ma.x * hs0, t[0], ma.y * qsum[0][j]);
              L[1] += fmaf(ma.x * hs1, t[1], ma.y * qsum[1][j]);
              L[2] += fmaf(mb.x * hs0, t[2], mb.y * qsum[0][j]);
              L[3] += fmaf(mb.x * hs1, t[3], mb.y * qsum[1][j]);
            }
          }
          if (!v0) { L[0] = -INFINITY; L[1] = -INFINITY; }
          if (!v1) { L[2] = -INFINITY; L[3] = -INFINITY; }
        };

        // values of one tile: fold the scale into p, keep the zero-point term as a scalar per group
        auto values = [&](const int u, const bool v0, const bool v1, const float (&p)[4]) {
          const uint32_t* vm = reinterpret_cast<const uint32_t*>(sp_vm + u * (NW * 16 * 4 * NGV));   // row tok0
          const uint32_t pa01 = pack_h2(p[0], p[1]), pb01 = pack_h2(p[2], p[3]);
          uint32_t bw[NGV][2];
#pragma unroll
          for (int j = 0; j < NGV; ++j) {
            const uint32_t ma = v0 ? vm[j] : 0u;
            const uint32_t mb = v1 ? vm[8 * NGV + j] : 0u;
            // zero-point of the centred codes: z + s * MID
            const float za = fmaf(meta_s(ma), kCodeMid<VB>, meta_z(ma)), zb = fmaf(meta_s(mb), kCodeMid<VB>, meta_z(mb));
            zacc[0][j] += p[0] * za + p[2] * zb;
            zacc[1][j] += p[1] * za + p[3] * zb;
            // (p * s) in fp16: both heads of a row share the row's scale
            const uint32_t sa2 = __byte_perm(ma, ma, 0x1010), sb2 = __byte_perm(mb, mb, 0x1010);
            bw[j][0] = movmatrix_trans(as_u32(__hmul2(as_h2(pa01), as_h2(sa2))));
            bw[j][1] = movmatrix_trans(as_u32(__hmul2(as_h2(pb01), as_h2(sb2))));
          }
          // Codes become fp16 with one LOP3 (field bits into the mantissa of 1024.0) and one HFMA2 that strips the
          // 1024, undoes the field's bit position and centres the code on MID: the MMA then sums p*s*(code - MID),
          // which is small where sum p*s*code and sum p*z would cancel, and MID moves into the zero-point above.
          uint32_t vw[VW];
          load_words<VW>(sp_v + u * (NW * V_TILE_BYTES), 512, vw);
          uint32_t vh[VW];
#pragma unroll
          for (int w = 0; w < VW; ++w) vh[w] = vw[w] >> 8;        // tokens 8..15 of the tile
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const int j = mt / (MT / NGV);
            const uint32_t a0 = centered_pair<VB>(vw[(2 * mt) / NPOS], (2 * mt) % NPOS);
            const uint32_t a1 = centered_pair<VB>(vw[(2 * mt + 1) / NPOS], (2 * mt + 1) % NPOS);
            const uint32_t a2 = centered_pair<VB>(vh[(2 * mt) / NPOS], (2 * mt) % NPOS);
            const uint32_t a3 = centered_pair<VB>(vh[(2 * mt + 1) / NPOS], (2 * mt + 1) % NPOS);
            mma16816(O[mt], a0, a1, a2, a3, bw[j][0], bw[j][1]);
          }
        };

        auto do_tiles = [&](auto masked_tag) {
          constexpr bool MASKED = decltype(masked_tag)::value;
          float L[TPW][4];
          bool v0[TPW], v1[TPW];
          float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
          for (int u = 0; u < TPW; ++u) {
            const int tok0 = (warp + NW * u) * 16 + gid;        // page-local tokens of this lane's two rows
            v0[u] = !MASKED || tok0 < nv;
            v1[u] = !MASKED || tok0 + 8 < nv;
            if (!MASKED || (warp + NW * u) < ntiles) {
              logits(u, tok0, v0[u], v1[u], L[u]);
            } else {
              L[u][0] = L[u][1] = L[u][2] = L[u][3] = -INFINITY;
            }
            t0 = fmaxf(t0, fmaxf(L[u][0], L[u][2]));
            t1 = fmaxf(t1, fmaxf(L[u][1], L[u][3]));
          }
          // online softmax: rescale only when some logit exceeds the running max
          if (__any_sync(FULL, (t0 > m0) | (t1 > m1))) {
            float u0 = t0, u1 = t1;
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
              u0 = fmaxf(u0, __shfl_xor_sync(FULL, u0, off));
              u1 = fmaxf(u1, __shfl_xor_sync(FULL, u1, off));
            }
            const float n0 = fmaxf(m0, u0), n1 = fmaxf(m1, u1);
            const float a0 = (n0 == -INFINITY) ? 1.f : ex2(m0 - n0);
            const float a1 = (n1 == -INFINITY) ? 1.f : ex2(m1 - n1);
            m0 = n0; m1 = n1;
            l0 *= a0; l1 *= a1;
#pragma unroll
            for (int j = 0; j < NGV; ++j) { zacc[0][j] *= a0; zacc[1][j] *= a1; }
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) { O[mt][0] *= a0; O[mt][1] *= a1; O[mt][2] *= a0; O[mt][3] *= a1; }
          }
#pragma unroll
          for (int u = 0; u < TPW; ++u) {
            if (!MASKED || (warp + NW * u) < ntiles) {
              float p[4];
              p[0] = ex2(L[u][0] - m0); p[1] = ex2(L[u][1] - m1); p[2] = ex2(L[u][2] - m0); p[3] = ex2(L[u][3] - m1);
              l0 += p[0] + p[2];
              l1 += p[1] + p[3];
              values(u, v0[u], v1[u], p);
            }
          }
        };

        if (ntiles > warp) {                     // a short last page may leave this warp without a tile
          if (nv == kPageTokens) do_tiles(std::false_type{});
          else do_tiles(std::true_type{});
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar0 + 8 * (stages + stage));
      if (++stage == stages) { stage = 0; phase ^= 1; }
      ++page_no;
    }

    // ---- segment end: finish this warp's state, combine the NW warps, write the partial
    {
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(FULL, l0, off);
        l1 += __shfl_xor_sync(FULL, l1, off);
#pragma unroll
        for (int j = 0; j < NGV; ++j) {
          zacc[0][j] += __shfl_xor_sync(FULL, zacc[0][j], off);
          zacc[1][j] += __shfl_xor_sync(FULL, zacc[1][j], off);
        }
      }
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const int j = mt / (MT / NGV);
        O[mt][0] += zacc[0][j]; O[mt][1] += zacc[1][j]; O[mt][2] += zacc[0][j]; O[mt][3] += zacc[1][j];
      }
      constexpr int PER_LANE = MT * 4 + 4;
#pragma unroll
      for (int step = NW / 2; step >= 1; step >>= 1) {
        if (warp >= step && warp < 2 * step) {
          float* dst = sComb + (size_t)(warp - step) * PER_LANE * 32 + lane;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
            for (int r = 0; r < 4; ++r) dst[(mt * 4 + r) * 32] = O[mt][r];
          }
          dst[(MT * 4 + 0) * 32] = m0; dst[(MT * 4 + 1) * 32] = m1;
          dst[(MT * 4 + 2) * 32] = l0; dst[(MT * 4 + 3) * 32] = l1;
        }
        named_bar_sync(1, NCONS);
        if (warp < step) {
          const float* src = sComb + (size_t)warp * PER_LANE * 32 + lane;
          const float om0 = src[(MT * 4 + 0) * 32], om1 = src[(MT * 4 + 1) * 32];
          const float n0 = fmaxf(m0, om0), n1 = fmaxf(m1, om1);
          const float fa0 = (n0 == -INFINITY) ? 0.f : ex2(m0 - n0), fb0 = (n0 == -INFINITY) ? 0.f : ex2(om0 - n0);
          const float fa1 = (n1 == -INFINITY) ? 0.f : ex2(m1 - n1), fb1 = (n1 == -INFINITY) ? 0.f : ex2(om1 - n1);
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            O[mt][0] = O[mt][0] * fa0 + src[(mt * 4 + 0) * 32] * fb0;
            O[mt][1] = O[mt][1] * fa1 + src[(mt * 4 + 1) * 32] * fb1;
            O[mt][2] = O[mt][2] * fa0 + src[(mt * 4 + 2) * 32] * fb0;
            O[mt][3] = O[mt][3] * fa1 + src[(mt * 4 + 3) * 32] * fb1;
          }
          l0 = l0 * fa0 + src[(MT * 4 + 2) * 32] * fb0;
          l1 = l1 * fa1 + src[(MT * 4 + 3) * 32] * fb1;
          m0 = n0; m1 = n1;
        }
        named_bar_sync(1, NCONS);
      }
      if (warp == 0) {
        const long long xs = (long long)sPref[b] + (long long)h * pages_b;     // first page of this stream
        const int slot = (int)blockIdx.x - plan.cta_of(xs);
        if (slot >= 0 && slot < s_cap) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int head = 2 * tid + e;
            if (head < G) {
              float* dst = ws + (((size_t)stream * s_cap + slot) * G + head) * (D + 2);
              if (gid == 0) { dst[0] = e ? m1 : m0; dst[1] = e ? l1 : l0; }
#pragma unroll
              for (int mt = 0; mt < MT; ++mt) {
                // accumulator rows (gid, gid + 8) of m-tile mt are channels 64 (mt/4) + 8 gid + 2 (mt%4) + {0, 1}
                dst[2 + 64 * (mt >> 2) + 8 * gid + 2 * (mt & 3)] = O[mt][e];
                dst[2 + 64 * (mt >> 2) + 8 * gid + 2 * (mt & 3) + 1] = O[mt][2 + e];
              }
            }
          }
        }
      }
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
template <int D, int KB, int VB, int KAXIS, int NGK, int NGV, int NL, int NW, int MINB>
int launch_mma_inst(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap,
                    cudaStream_t stream) {
  const int budget = (227 * 1024) / MINB - 1024;            // shared memory per CTA for MINB resident CTAs per SM
  int stages = (budget - smem_layout(0, 0, NW, D, KAXIS == 1).total) / ((g.page_bytes + 127) & ~127);
  if (stages > 8) stages = 8;
  if (stages < 2) return KVQ_ERR_UNSUPPORTED;
  const SmemLayout sl = smem_layout(g.page_bytes, stages, NW, D, KAXIS == 1);
  auto kern = decode_mma_kernel<D, KB, VB, KAXIS, NGK, NGV, NL, NW, MINB>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sl.total) != cudaSuccess)
    return KVQ_ERR_CUDA_LAUNCH;
  kern<<<148 * MINB, (NW + 1) * 32, sl.total, stream>>>(g, c, static_cast<const uint16_t*>(q), c1, ws, s_cap,
                                                         stages);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace mma
}  // namespace kvq
