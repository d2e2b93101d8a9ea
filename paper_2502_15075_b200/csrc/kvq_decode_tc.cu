// Fused low-bit decode attention on the fifth-generation tensor cores (tcgen05, accumulators and the code
// operands in tensor memory): softmax(q K^T / sqrt(d)) V (App. A.1) over the packed cache with K^ = z + s*code and
// V^ likewise folded around the contractions, for head_dim 128, token-wise groups of 128, 4- or 8-bit keys,
// 2- or 4-bit values and up to four (virtual) query heads per KV head.
//
// One CTA = four consumer warps (thread x = token x of the page for QK^T and the softmax, = channel x for PV),
// a producer warp and an MMA warp; two or three CTAs per SM, each with 128 columns of tensor memory.
//  * The producer streams whole 128-token pages into a shared-memory ring with tiled TMA copies (the page seen
//    as rows of 64 bytes, 64-byte swizzle: row-per-thread 16-byte reads are then free of bank conflicts).
//  * A consumer thread turns its token's packed key row into the A operand of QK^T and stores it to tensor
//    memory (lane = token, 32 columns of four code bytes).  4-bit keys need ONE instruction per packed word:
//    the operand is the raw word (bytes lo + 16 hi) next to (word & 0xF0F0F0F0) (bytes 16 hi), and the query
//    side carries 16 Q_lo against the first and Q_hi - 16 Q_lo against the second, so that the int32 result is
//    exactly 16 sum_d code_d Q_d.  Likewise its channel's value codes (one mask per word: code * 2^(b f), the
//    factor removed when the accumulator is folded) become the A operand of PV (lane = channel, columns = tokens).
//  * One elected thread issues tcgen05.mma kind::i8 (M 128, N 16, K 32): S[token][(head, limb)] = codes . Q with q
//    as fixed point in three balanced signed byte limbs, and O[channel][(head, limb)] += codes^T . P with the
//    softmax weight times the value scale as unsigned 31-bit fixed point in four byte limbs (operand rows written
//    by the token threads, one 16-byte store each).  All sums are exact in int32.
//  * Scale and zero-point never touch the codes: q.K^_t = s_t (q.c_t) + z_t sum(q), o = sum_t (p_t s_t) c_t +
//    sum_t p_t z_t.
//  * The flat split over the grid, the partials and their merge by the last finisher are those of the warp-level
//    kernel (kvq_decode_mma_kernel.cuh), so both share one workspace format.
// Every wait is bounded; on expiry the kernel sets KVQ_STATUS_DEVICE_TIMEOUT, stops computing, keeps its block-wide
// barriers, waits for its own copies and MMAs in flight, frees its tensor memory and returns.
#include <cuda.h>   // CUtensorMap and its enums only; the encoder is looked up through the runtime (no libcuda link)

#include <mutex>

#include "kvq_decode_mma.cuh"

namespace kvq {
namespace tc {

using namespace mma;

constexpr int kThreads = 192;        // warps 0-3 consumers, 4 producer, 5 MMA issue + tensor-memory allocation
constexpr int kNCons = 128;
constexpr int kTmemCols = 128;       // per CTA; up to four CTAs per SM share the 512 columns
constexpr int kColKa = 0;            // key operand, 32 columns
constexpr int kColVa = 32;           // value operand, two buffers of 32 columns
constexpr int kColS = 96;            // logits accumulator, 16 columns
constexpr int kColO = 112;           // output accumulator, 16 columns
constexpr float kQFixTc = 32512.0f;  // largest |Q| of the 16-bit fixed-point q
constexpr float kPOne = 2147483648.0f;   // 2^31: the softmax weights are 31-bit fixed point
constexpr float kHeadroomTc = 6.0f;
constexpr int kFoldPages = 128;      // fold the int32 output accumulator at least this often (no overflow)

// Byte offset inside a ring stage after the 64-byte TMA swizzle (address bits 7-8 xor-ed into bits 4-5).
__host__ __device__ __forceinline__ constexpr int swz64(int off) { return off ^ ((off >> 3) & 0x30); }

struct SmemTc {
  int ring, qop, pop, sq, bars, pref, misc, red, total;
};
// ring | Q operand 2 KB | P operand 2 x 2 KB | fixed-point q [4][128] int | barriers | batch prefix | misc | reductions
__host__ __device__ inline SmemTc smem_tc(int page_bytes, int stages, int batch) {
  SmemTc s;
  s.ring = 0;
  s.qop = stages * page_bytes;
  s.pop = s.qop + 2048;
  s.sq = s.pop + 4096;
  s.bars = s.sq + 2048;
  s.pref = s.bars + 512;
  s.misc = (s.pref + (batch + 1) * 4 + 15) & ~15;
  s.red = s.misc + 64;
  s.total = s.red + 4 * 16 * 4 + 1024;          // + slack to align the ring to 1024 bytes
  return s;
}

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem descriptor], 8-bit integer operands, int32 accumulate.
__device__ __forceinline__ void tc_mma_i8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// barrier among the consumer threads that also ORs a predicate over them
__device__ __forceinline__ bool cons_bar_or(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "bar.red.or.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred) : "memory");
  return r != 0;
}

// Shared-memory matrix descriptors (no swizzle, version 1): start address, leading (K-direction) and stride
// (M/N-direction) byte offsets of the 8 x 16-byte core matrices, all in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFF) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | (1ull << 46);
}
// Instruction descriptors: int32 accumulate, A unsigned bytes (K-major, from tensor memory), M 128, N 16;
// QK^T: B signed bytes K-major; PV: B unsigned bytes N-major.
constexpr uint32_t kIdescQK = (2u << 4) | (0u << 7) | (1u << 10) | (0u << 16) | (2u << 17) | (8u << 24);
constexpr uint32_t kIdescPV = (2u << 4) | (0u << 7) | (0u << 10) | (1u << 16) | (2u << 17) | (8u << 24);

// Wait that also gives up early when another role of the CTA has already given up.
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, unsigned long long limit_ns,
                                              volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  while (true) {
    if (mbar_try_wait_hint(bar, parity, 2000u)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > limit_ns) return false;
  }
}

template <int KB, int VB, int MINB>
__global__ void __launch_bounds__(kThreads, MINB)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmap, Geom g, CachePtrs c, const uint16_t* __restrict__ q, float c1,
                 float* __restrict__ ws, int s_cap, int stages, int box_rows, void* __restrict__ out, int out_dtype,
                 unsigned long long call_id, unsigned long long wait_ns, long long skip_x) {
  constexpr int D = 128;
  constexpr int K_ROW = D * KB / 8;
  constexpr int K_META_OFF = kPageTokens * K_ROW;
  constexpr int V_CODES_OFF = K_META_OFF + kPageTokens * 4;
  constexpr int V_BLOCK = 4 * D * VB;
  constexpr int V_META_OFF = V_CODES_OFF + 4 * V_BLOCK;
  constexpr int PAGE = V_META_OFF + kPageTokens * 4;
  constexpr int FPBV = 8 / VB;
  constexpr int KMUL = KB == 4 ? 16 : 1;            // the key contraction yields KMUL * sum_d code_d Q_d
  constexpr uint32_t FULL = 0xffffffffu;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw_u32 + 1023u) & ~1023u) - raw_u32);      // the swizzle pattern follows address bits
  const SmemTc sl = smem_tc(PAGE, stages, g.B);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sl.bars);
  int* sPref = reinterpret_cast<int*>(smem + sl.pref);
  int* sMisc = reinterpret_cast<int*>(smem + sl.misc);       // [0] pages_max [1] abort [2] published [3] tmem base [4,5] fresh
  float* sRed = reinterpret_cast<float*>(smem + sl.red);     // [4 warps][16]
  int* sQ = reinterpret_cast<int*>(smem + sl.sq);            // [4][128] fixed-point q
  uint8_t* sQop = smem + sl.qop;
  uint8_t* sPop = smem + sl.pop;

  const int tid_ = threadIdx.x, lane = tid_ & 31, warp = tid_ >> 5;
  const int B = g.B, Hkv = g.Hkv, Gq = g.G, G = g.G * g.rows;
  // barrier map: full[s], empty[s], then k_ready, s_ready, p_ready[2], pv_done[2], drain
  const uint32_t bar0 = smem_u32(bars);
  const uint32_t bar_ops = bar0 + 8 * (2 * stages), bar_s = bar_ops + 16, bar_p = bar_ops + 32, bar_pv = bar_ops + 48,
                 bar_drain = bar_ops + 64;

  // ---- plan: pages per sequence, prefix over the batch
  if (tid_ == 0) { sPref[0] = 0; sMisc[0] = 0; sMisc[1] = 0; sMisc[4] = 0; sMisc[5] = 0; }
  __syncthreads();
  for (int b = tid_; b < B; b += blockDim.x) {
    int pages = (paged_len(c.seq_len, b, g.capacity, g.R) + kPageTokens - 1) >> 7;
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
      mbar_init(bar0 + 8 * s, 1);
      mbar_init(bar0 + 8 * (stages + s), 4);
    }
    mbar_init(bar_ops, 4);
    mbar_init(bar_s, 1);
    for (int k = 0; k < 2; ++k) {
      mbar_init(bar_p + 8 * k, 4);
      mbar_init(bar_pv + 8 * k, 1);
    }
    mbar_init(bar_drain, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {                       // tensor memory for this CTA (the permit is given up at once: nothing else allocates)
    tmem_alloc(smem_u32(&sMisc[3]), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&sMisc[3]);

  for (int bb = blockIdx.x; bb < B && g.R == 0; bb += gridDim.x) {       // sequences without pages: zero rows
    if (sPref[bb + 1] == sPref[bb]) {
      for (int i = tid_; i < g.rows * g.Hq * D; i += blockDim.x) {
        const size_t oi = (size_t)bb * g.rows * g.Hq * D + i;
        if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = 0.f;
        else static_cast<uint16_t*>(out)[oi] = 0;
      }
    }
  }
  const int s_plan = s_cap - (g.R ? 1 : 0);
  const FlatPlan plan = make_plan(sPref[B], sMisc[0], gridDim.x, s_plan);
  const bool active = plan.N != 0 && (int)blockIdx.x < plan.c_eff;
  unsigned long long* counts = reinterpret_cast<unsigned long long*>(ws + tag_offset_floats(B * Hkv, s_cap, G, D));
  const long long x_lo = active ? plan.lo(blockIdx.x) : 0, x_hi = active ? plan.lo(blockIdx.x + 1) : 0;

  int b = 0, pages_b = 1, h = 0, page = 0;
  if (active) {
    int lo_ = 0, hi_ = B - 1;
    while (lo_ < hi_) {
      int mid = (lo_ + hi_ + 1) >> 1;
      if (sPref[mid] <= x_lo) lo_ = mid; else hi_ = mid - 1;
    }
    b = lo_;
    pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
    h = (int)((x_lo - sPref[b]) / pages_b);
    page = (int)((x_lo - sPref[b]) % pages_b);
  }
  const uint32_t ring = smem_u32(smem);
  volatile int* abort_flag = sMisc + 1;
  volatile int* n_published = sMisc + 2;
  volatile int* sFresh = sMisc + 4;
  const unsigned long long id40 = (call_id & 0xFFFFFFFFFFull) ? (call_id & 0xFFFFFFFFFFull) : 1ull;

  // advance (b, h, page) by n pages inside the plan's page order (n never crosses more than the stream's end)
  auto advance = [&](int n) {
    page += n;
    if (page == pages_b) {
      page = 0;
      if (++h == Hkv) {
        h = 0;
        do { ++b; } while (b < B && sPref[b + 1] == sPref[b]);
        if (b < B) pages_b = (sPref[b + 1] - sPref[b]) / Hkv;
      }
    }
  };

  if (warp == 4) {
    // =========================================================== producer
    if (lane == 0 && active) {
      int it = 0, stage = 0;
      uint32_t phase = 1;
      bool ok = true;
      const uint64_t policy = l2_evict_first_policy();
      for (long long x = x_lo; x < x_hi; ++x, ++it) {
        if (it >= stages) {
          ok = wait_or_abort(bar0 + 8 * (stages + stage), phase, wait_ns, abort_flag);
          if (!ok) break;
        }
        const int gpage = (b * Hkv + h) * g.n_pages + page;
        const uint32_t fb = bar0 + 8 * stage;
        if (x != skip_x) {      // (skip_x: test hook - a page that never arrives makes the consumers' bounded wait expire)
          mbar_expect_tx(fb, (uint32_t)PAGE);
          const uint32_t dst = ring + stage * PAGE;
          tma_load_3d(dst, &tmap, 0, 0, gpage, fb, policy);
          if (box_rows * 64 < PAGE) tma_load_3d(dst + box_rows * 64, &tmap, 0, box_rows, gpage, fb, policy);
        }
        if (++stage == stages) { stage = 0; phase ^= 1; }
        advance(1);
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
      }
      // never leave while a copy may still be writing this CTA's shared memory
      for (int k = 1; k <= stages && k <= it; ++k) {
        const int j = it - k;
        if ((long long)(x_lo + j) == skip_x) continue;
        mbar_wait(bar0 + 8 * (j % stages), (j / stages) & 1, wait_ns);
      }
    }
  } else if (warp == 5) {
    // =========================================================== MMA issue
    if (lane == 0 && active) {
      bool ok = true;
      const int n_pages_cta = (int)(x_hi - x_lo);
      for (int it = 0; it < n_pages_cta; ++it) {
        const int buf = it & 1;
        ok = wait_or_abort(bar_ops, it & 1, wait_ns, abort_flag);               // the page's key operand is in tensor memory
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_i8_ts(tmem + kColS, tmem + kColKa + 8 * kk, smem_desc(smem_u32(sQop) + 512 * kk, 256, 128), kIdescQK,
                       kk > 0 ? 1u : 0u);
        tc_commit(bar_s);
        ok = wait_or_abort(bar_p + 8 * buf, (it >> 1) & 1, wait_ns, abort_flag);   // value operand and weights are ready
        if (!ok) break;
        tc_fence_after();
        const uint32_t fresh = (uint32_t)sFresh[buf];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_i8_ts(tmem + kColO, tmem + kColVa + 32 * buf + 8 * kk,
                       smem_desc(smem_u32(sPop) + 2048 * buf + 512 * kk, 128, 128), kIdescPV,
                       (kk > 0 || !fresh) ? 1u : 0u);
        tc_commit(bar_pv + 8 * buf);
      }
      if (!ok) {
        *abort_flag = 1;
        atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
      }
      // nothing of this CTA's may still run on the tensor cores when its tensor memory is freed
      tc_commit(bar_drain);
      mbar_wait(bar_drain, 0, wait_ns);
    }
  } else if (active) {
    // =========================================================== consumers: thread x = token x / channel x
    const int x_ = tid_;
    const uint32_t lane_taddr = tmem + ((uint32_t)(32 * warp) << 16);
    // value side: where this thread's channel lives in a value block
    const int v_mt = x_ >> 4, v_mw = v_mt / FPBV, v_f = v_mt % FPBV, v_rh = (x_ >> 3) & 1, v_gq = x_ & 7;
    const uint32_t v_mask = (((1u << VB) - 1u) * 0x01010101u) << (VB * v_f);
    const float v_unshift = 1.0f / (float)(1 << (VB * v_f));
    // row of the P operand this thread's token owns: the k-order of the value operand is (block, tq, half, byte)
    const int p_row = ((x_ >> 5) * 8 + ((x_ & 7) >> 1) * 2 + ((x_ >> 4) & 1)) * 4 + 2 * (x_ & 1) + ((x_ >> 3) & 1);

    int it = 0;                  // pages of this CTA consumed so far (buffer parity follows it)
    int stage = 0;
    uint32_t phase = 0;
    bool aborted = false;
    auto give_up = [&]() {
      aborted = true;
      *abort_flag = 1;
      if (lane == 0) atomicOr(c.status, KVQ_STATUS_DEVICE_TIMEOUT);
    };
    auto cons_wait = [&](uint32_t bar, uint32_t parity) {
      if (aborted) return;
      const bool got = wait_or_abort(bar, parity, wait_ns, abort_flag);
      if (!__all_sync(FULL, got)) give_up();
    };

    for (long long x = x_lo; x < x_hi;) {
      const int seg_pages = (int)min((long long)(pages_b - page), x_hi - x);
      const int n_tok = paged_len(c.seq_len, b, g.capacity, g.R);
      const int n_all = clamped_len(c.seq_len, b, g.capacity);
      const int stream = b * Hkv + h;

      // ---- segment start: the query operand of QK^T (no MMA of an earlier segment is still running: the
      // segment end waited for its last one)
      float hsc[4], qsf[4];
      {
        float qv[4], amax[4];
        int Qi[4];
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          qv[hv] = 0.f;
          if (hv < G) {
            const uint16_t* qrow = q + (((size_t)b * g.rows + hv / Gq) * g.Hq + (size_t)h * Gq + hv % Gq) * D;
            qv[hv] = bits16_to_f32(qrow[x_], g.in_dtype);
          }
          float a = fabsf(qv[hv]);
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) a = fmaxf(a, __shfl_xor_sync(FULL, a, off));
          if (lane == 0) sRed[warp * 16 + hv] = a;
        }
        named_bar_sync(1, kNCons);
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          amax[hv] = fmaxf(fmaxf(sRed[hv], sRed[16 + hv]), fmaxf(sRed[32 + hv], sRed[48 + hv]));
          const float scale = amax[hv] > 0.f ? kQFixTc / amax[hv] : 0.f;
          Qi[hv] = __float2int_rn(qv[hv] * scale);
          sQ[hv * D + x_] = Qi[hv];
          hsc[hv] = amax[hv] > 0.f ? c1 / (scale * (float)KMUL) : 0.f;
          int sum = Qi[hv];
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) sum += __shfl_xor_sync(FULL, sum, off);
          if (lane == 0) reinterpret_cast<int*>(sRed)[warp * 16 + 4 + hv] = sum;
        }
        named_bar_sync(1, kNCons);
        const int* sRedI = reinterpret_cast<const int*>(sRed);
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          // the zero-point term uses the sum of the same fixed-point q the MMAs see
          const int tot = sRedI[4 + hv] + sRedI[16 + 4 + hv] + sRedI[32 + 4 + hv] + sRedI[48 + 4 + hv];
          qsf[hv] = hsc[hv] * (float)KMUL * (float)tot;
        }
        // operand column k = x_: which channel(s) it multiplies
        const int cK = x_ >> 2, j = x_ & 3;
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          int val;
          if constexpr (KB == 4) {
            const int cch = cK >> 3, wd = (cK >> 1) & 3, plane = cK & 1;
            const int ch_lo = 32 * wd + 4 * cch + j;
            const int q_lo = sQ[hv * D + ch_lo], q_hi = sQ[hv * D + ch_lo + 16];
            val = plane == 0 ? 16 * q_lo : q_hi - 16 * q_lo;
          } else {
            const int half = cK >> 4, cch = (cK >> 2) & 3, w4 = cK & 3;
            val = sQ[hv * D + 16 * (4 * half + w4) + 4 * cch + j];
          }
          const int l0 = (int)(int8_t)(val & 0xFF);
          const int v1 = (val - l0) >> 8;
          const int l1 = (int)(int8_t)(v1 & 0xFF);
          const int l2 = (v1 - l1) >> 8;
          const int lim[3] = {l0, l1, l2};
#pragma unroll
          for (int li = 0; li < 3; ++li) {
            const int n = 3 * hv + li;
            sQop[(x_ >> 4) * 256 + (n >> 3) * 128 + (n & 7) * 16 + (x_ & 15)] = (uint8_t)(lim[li] & 0xFF);
          }
        }
#pragma unroll
        for (int n = 12; n < 16; ++n) sQop[(x_ >> 4) * 256 + (n >> 3) * 128 + (n & 7) * 16 + (x_ & 15)] = 0;
        fence_async_smem();
        named_bar_sync(1, kNCons);
      }

      float m_ref[4], l[4], zacc[4], master[4];
#pragma unroll
      for (int hv = 0; hv < 4; ++hv) { m_ref[hv] = -INFINITY; l[hv] = 0.f; zacc[hv] = 0.f; master[hv] = 0.f; }
      float sscale = kPOne / 9.094947e-13f;       // 2^31 / s_lim, s_lim a power of two above every value scale so far
      bool o_dirty = false;
      int since_fold = 0;
      int lim_hv[4];
#pragma unroll
      for (int hv = 0; hv < 4; ++hv) lim_hv[hv] = n_all - (g.rows - 1 - min(hv / Gq, g.rows - 1));

      // fold the int32 output accumulator into this thread's fp32 master (thread = channel) with the scale its
      // weights were made with
      auto fold_O = [&](int it_last) {
        if (!o_dirty) return;
        cons_wait(bar_pv + 8 * (it_last & 1), (it_last >> 1) & 1);
        tc_fence_after();
        uint32_t a[16];
        tmem_ld16(lane_taddr + kColO, a);
        tc_wait_ld();
        tc_fence_before();
        const float fw = v_unshift / sscale;
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          const float v = fmaf((float)(int)a[4 * hv + 3], 16777216.f,
                               fmaf((float)(int)a[4 * hv + 2], 65536.f,
                                    fmaf((float)(int)a[4 * hv + 1], 256.f, (float)(int)a[4 * hv])));
          master[hv] = fmaf(v, fw, master[hv]);
        }
        o_dirty = false;
        since_fold = 0;
      };

      for (int i = 0; i < seg_pages; ++i) {
        const int itp = it + i, buf = itp & 1;
        const int pg = page + i;                                  // page index inside the sequence
        const int nv = min(kPageTokens, n_tok - pg * kPageTokens);
        const int tokg = pg * kPageTokens + x_;
        // ------------------------------------------------------------ key operand (thread = token); the earlier
        // page's QK^T is complete and its logits are read: this thread waited for them in its softmax
        cons_wait(bar0 + 8 * stage, phase);
        tc_fence_after();
        const uint8_t* sp = smem + stage * PAGE;
        uint32_t r[32];
        if constexpr (KB == 4) {
#pragma unroll
          for (int cch = 0; cch < 4; ++cch) {
            const uint4 w = *reinterpret_cast<const uint4*>(sp + swz64(x_ * 64 + cch * 16));
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {
              r[cch * 8 + wd * 2] = ww[wd];
              r[cch * 8 + wd * 2 + 1] = ww[wd] & 0xF0F0F0F0u;
            }
          }
        } else {
#pragma unroll
          for (int half = 0; half < 2; ++half) {
#pragma unroll
            for (int cch = 0; cch < 4; ++cch) {
              const uint4 w = *reinterpret_cast<const uint4*>(sp + swz64(x_ * 128 + half * 64 + cch * 16));
              r[half * 16 + cch * 4 + 0] = w.x; r[half * 16 + cch * 4 + 1] = w.y;
              r[half * 16 + cch * 4 + 2] = w.z; r[half * 16 + cch * 4 + 3] = w.w;
            }
          }
        }
        tmem_st32(lane_taddr + kColKa, r);
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_ops);
        // ------------------------------------------------------------ value operand (thread = channel), while QK^T runs
        const uint32_t km_cur = *reinterpret_cast<const uint32_t*>(sp + swz64(K_META_OFF + 4 * x_));
        const uint32_t vm_cur = *reinterpret_cast<const uint32_t*>(sp + swz64(V_META_OFF + 4 * x_));
#pragma unroll
        for (int blk = 0; blk < 4; ++blk) {
#pragma unroll
          for (int tq = 0; tq < 4; ++tq) {
            const uint2 w = *reinterpret_cast<const uint2*>(
                sp + swz64(V_CODES_OFF + blk * V_BLOCK + v_mw * 512 + (4 * v_gq + tq) * 16 + 8 * v_rh));
            r[(blk * 4 + tq) * 2 + 0] = w.x & v_mask;
            r[(blk * 4 + tq) * 2 + 1] = w.y & v_mask;
          }
        }
        if (itp >= 2) cons_wait(bar_pv + 8 * buf, ((itp - 2) >> 1) & 1);       // the buffer's last reader is done
        tc_fence_after();
        tmem_st32(lane_taddr + kColVa + 32 * buf, r);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar0 + 8 * (stages + stage));               // the page's bytes are all in registers
        if (++stage == stages) { stage = 0; phase ^= 1; }
        // ------------------------------------------------------------ softmax (thread = token)
        {
          cons_wait(bar_s, itp & 1);
          tc_fence_after();
          uint32_t a[16];
          tmem_ld16(lane_taddr + kColS, a);
          tc_wait_ld();
          const bool tok_ok = x_ < nv;
          const float2 km = __half22float2(as_h2(tok_ok ? km_cur : 0u));
          const float2 vm = __half22float2(as_h2(tok_ok ? vm_cur : 0u));
          float L[4];
          bool trig = false;
#pragma unroll
          for (int hv = 0; hv < 4; ++hv) {
            const float sf = fmaf((float)(int)a[3 * hv + 2], 65536.f,
                                  fmaf((float)(int)a[3 * hv + 1], 256.f, (float)(int)a[3 * hv]));
            L[hv] = fmaf(km.x * hsc[hv], sf, km.y * qsf[hv]);
            if (!tok_ok || tokg >= lim_hv[hv]) L[hv] = -INFINITY;
            trig |= L[hv] > m_ref[hv];
          }
          trig |= vm.x * sscale >= kPOne;
          trig |= since_fold >= kFoldPages;
          if (cons_bar_or(trig)) {
            // rare: a new softmax reference, a larger value scale, or the periodic fold.  Block-wide maxima first.
            float red[5];
#pragma unroll
            for (int hv = 0; hv < 4; ++hv) red[hv] = L[hv];
            red[4] = vm.x;
#pragma unroll
            for (int k = 0; k < 5; ++k) {
#pragma unroll
              for (int off = 1; off < 32; off <<= 1) red[k] = fmaxf(red[k], __shfl_xor_sync(FULL, red[k], off));
              if (lane == 0) sRed[warp * 16 + 8 + k] = red[k];
            }
            named_bar_sync(1, kNCons);
#pragma unroll
            for (int k = 0; k < 5; ++k)
              red[k] = fmaxf(fmaxf(sRed[8 + k], sRed[16 + 8 + k]), fmaxf(sRed[32 + 8 + k], sRed[48 + 8 + k]));
            fold_O(itp - 1);
            if (tid_ == 0) sFresh[buf] = 1;
            if (red[4] * sscale >= kPOne)
              sscale = kPOne / __uint_as_float((__float_as_uint(red[4]) & 0x7F800000u) + 0x00800000u);
#pragma unroll
            for (int hv = 0; hv < 4; ++hv) {
              if (red[hv] > m_ref[hv]) {
                const float nref = red[hv] + kHeadroomTc;
                const float sc = (m_ref[hv] == -INFINITY) ? 0.f : ex2(m_ref[hv] - nref);
                m_ref[hv] = nref;
                l[hv] *= sc;
                zacc[hv] *= sc;
                master[hv] *= sc;
              }
            }
          } else if (tid_ == 0) {
            sFresh[buf] = 0;
          }
          uint4 pw;
          uint32_t* pwv = reinterpret_cast<uint32_t*>(&pw);
          const float sv = vm.x * sscale;
#pragma unroll
          for (int hv = 0; hv < 4; ++hv) {
            const float p = (L[hv] == -INFINITY) ? 0.f : ex2(L[hv] - m_ref[hv]);
            l[hv] += p;
            zacc[hv] = fmaf(p, vm.y, zacc[hv]);
            pwv[hv] = __float2uint_rn(p * sv);
          }
          *reinterpret_cast<uint4*>(sPop + 2048 * buf + 16 * p_row) = pw;
          fence_async_smem();
          tc_wait_st();                          // the value operand stored above
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_p + 8 * buf);
          o_dirty = true;
          ++since_fold;
        }
      }
      it += seg_pages;

      // ---- segment end: fold the last accumulations, combine the block, write the partial
      fold_O(it - 1);
      {
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          float a = l[hv], z = zacc[hv];
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            a += __shfl_xor_sync(FULL, a, off);
            z += __shfl_xor_sync(FULL, z, off);
          }
          if (lane == 0) { sRed[warp * 16 + hv] = a; sRed[warp * 16 + 4 + hv] = z; }
        }
        named_bar_sync(1, kNCons);
        float ltot[4], o[4];
#pragma unroll
        for (int hv = 0; hv < 4; ++hv) {
          ltot[hv] = (sRed[hv] + sRed[16 + hv]) + (sRed[32 + hv] + sRed[48 + hv]);
          const float ztot = (sRed[4 + hv] + sRed[16 + 4 + hv]) + (sRed[32 + 4 + hv] + sRed[48 + 4 + hv]);
          o[hv] = master[hv] + ztot;
        }
        const long long xs = (long long)sPref[b] + (long long)h * pages_b;
        const int c_first = plan.cta_of(xs);
        const int slot = (int)blockIdx.x - c_first;
        const int n_part = plan.cta_of(xs + pages_b - 1) - c_first + 1;
        const bool has_win = n_all > n_tok;
        if (slot >= 0 && slot < s_plan) {
          const int d = x_;
          if (n_part == 1 && !has_win) {
#pragma unroll
            for (int hv = 0; hv < 4; ++hv) {
              if (hv < G) {
                const float rr = ltot[hv] > 0.f ? o[hv] / ltot[hv] : 0.f;
                const size_t oi = (((size_t)b * g.rows + hv / Gq) * g.Hq + (size_t)h * Gq + hv % Gq) * D + d;
                if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = rr;
                else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(rr, out_dtype);
              }
            }
          } else {
#pragma unroll
            for (int hv = 0; hv < 4; ++hv) {
              if (hv < G) {
                float* dst = ws + (((size_t)stream * s_cap + slot) * G + hv) * (D + 2);
                if (d == 0) { dst[0] = m_ref[hv]; dst[1] = ltot[hv]; }
                dst[2 + d] = o[hv];
              }
            }
            __threadfence();
            named_bar_sync(1, kNCons);
            if (tid_ == 0) *n_published = (int)tagged_count(counts + stream, id40);
            named_bar_sync(1, kNCons);
            if (*n_published == n_part) {
              __threadfence();
              const int n_merge = n_part + (has_win ? 1 : 0);
              for (int hv = 0; hv < G; ++hv) {
                const float* base = ws + (((size_t)stream * s_cap) * G + hv) * (D + 2);
                const size_t slot_stride = (size_t)G * (D + 2);
                float mstar = -INFINITY, num = 0.f, den = 0.f;
                for (int j0 = 0; j0 < n_merge; j0 += 4) {
                  float mj[4], lj[4], oj[4];
#pragma unroll
                  for (int u = 0; u < 4; ++u) {
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
                const float rr = den > 0.f ? num / den : 0.f;
                const size_t oi = (((size_t)b * g.rows + hv / Gq) * g.Hq + (size_t)h * Gq + hv % Gq) * D + d;
                if (out_dtype == KVQ_FP32) static_cast<float*>(out)[oi] = rr;
                else static_cast<uint16_t*>(out)[oi] = f32_to_bits16(rr, out_dtype);
              }
              if (tid_ == 0) counts[stream] = 0ull;
            }
          }
        }
        named_bar_sync(1, kNCons);
      }
      x += seg_pages;
      advance(seg_pages);
    }
  }

  // ---- teardown: every role is done (or has given up and drained); free the tensor memory
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// The pages of a cache as a 3-D tensor [page][row of 64 bytes][64 bytes]; a box is (half of) one page.
static int make_page_map(const Geom& g, const CachePtrs& c, int box_rows, CUtensorMap* tm) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return KVQ_ERR_CUDA_LAUNCH;
  const cuuint64_t dims[3] = {64, (cuuint64_t)(g.page_bytes / 64), (cuuint64_t)g.B * g.Hkv * g.n_pages};
  const cuuint64_t strides[2] = {64, (cuuint64_t)g.page_bytes};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, c.pages, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

template <int KB, int VB, int MINB>
static int launch_inst(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap, void* out,
                       int out_dtype, unsigned long long call_id, unsigned long long wait_ns, long long skip_x,
                       cudaStream_t stream) {
  constexpr int kPage = kPageTokens * (128 * KB / 8 + 4) + kPageTokens * (128 * VB / 8 + 4);
  if (g.page_bytes != kPage) return KVQ_ERR_UNSUPPORTED;
  const int rows64 = g.page_bytes / 64;
  const int box_rows = rows64 <= 256 ? rows64 : rows64 / 2;
  if (g.page_bytes % 1024 || (box_rows * 64) % 512 || box_rows > 256) return KVQ_ERR_UNSUPPORTED;
  const int budget = (227 * 1024) / MINB - 1024;
  int stages = (budget - smem_tc(0, 0, g.B).total) / g.page_bytes;
  if (stages > 12) stages = 12;
  if (stages < 2) return KVQ_ERR_UNSUPPORTED;
  SmemTc sl = smem_tc(g.page_bytes, stages, g.B);
  // A CTA allocates 128 of the SM's 512 tensor-memory columns and would wait for ever as the fifth CTA on an SM:
  // asking for more than a fifth of the shared memory keeps the resident CTAs at four or fewer.
  if (sl.total < 48 * 1024) sl.total = 48 * 1024;
  CUtensorMap tm;
  int rc = make_page_map(g, c, box_rows, &tm);
  if (rc != KVQ_OK) return rc;
  auto kern = decode_tc_kernel<KB, VB, MINB>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, sl.total) != cudaSuccess)
    return KVQ_ERR_CUDA_LAUNCH;
  kern<<<148 * MINB, kThreads, sl.total, stream>>>(tm, g, c, static_cast<const uint16_t*>(q), c1, ws, s_cap, stages, box_rows,
                                               out, out_dtype, call_id, wait_ns, skip_x);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace tc

bool decode_tc_supported(const Geom& g, const CachePtrs& c) {
  if (g.D != 128 || g.k_axis != 0 || g.gk != 128 || g.gv != 128) return false;
  if ((g.kb != 4 && g.kb != 8) || (g.vb != 2 && g.vb != 4)) return false;
  if (g.G * g.rows > 4 || g.B > mma::kMaxBatchFlat) return false;
  if (c.k_signs != nullptr) return false;                       // rotated keys: the warp-level kernel
  if ((long long)g.B * g.Hkv * g.n_pages > 0x7fffffffLL) return false;
  return true;
}

int launch_decode_tc(const Geom& g, const CachePtrs& c, const void* q, float c1, float* ws, int s_cap, void* out,
                     int out_dtype, unsigned long long call_id, unsigned long long wait_ns, long long skip_x,
                     cudaStream_t stream) {
  if (g.kb == 4 && g.vb == 2) return tc::launch_inst<4, 2, 3>(g, c, q, c1, ws, s_cap, out, out_dtype, call_id, wait_ns, skip_x, stream);
  if (g.kb == 4 && g.vb == 4) return tc::launch_inst<4, 4, 3>(g, c, q, c1, ws, s_cap, out, out_dtype, call_id, wait_ns, skip_x, stream);
  if (g.kb == 8 && g.vb == 4) return tc::launch_inst<8, 4, 2>(g, c, q, c1, ws, s_cap, out, out_dtype, call_id, wait_ns, skip_x, stream);
  if (g.kb == 8 && g.vb == 2) return tc::launch_inst<8, 2, 2>(g, c, q, c1, ws, s_cap, out, out_dtype, call_id, wait_ns, skip_x, stream);
  return KVQ_ERR_UNSUPPORTED;
}

}  // namespace kvq
