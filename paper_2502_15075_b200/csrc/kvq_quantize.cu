// kvq_quantize_append kernels: group-wise asymmetric round-to-nearest
// quantization (App. B.1 quantizer per group; Sec. 4.1 grouping: token-wise
// groups along head_dim, or channel-wise groups over a 128-token block with an
// fp16 residual tail) and packing into the page layout.
//
// Token-wise kernel: one warp per block of 32 tokens (64 for head_dim 64 at 2 bits) of one
// stream and one side (keys or values).  A byte of the packed page holds codes of channels that
// lie 16 apart, so a lane loads, for each of its tokens, the 8/b 16-byte pieces whose codes share
// bytes: every output byte, and with four tokens (values) or four channels (keys) every output
// word, is then assembled in that lane's registers and stored directly - no shared memory, no
// atomics, no read-modify-write; a token that is not new is simply not stored (byte stores for
// values).  Group minima and maxima are reduced with a few shuffles between the lanes of a row.
// The kernel is bound by reading the 16-bit inputs from HBM.
#include "kvq_internal.h"

namespace kvq {

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = kThreads / 32;
constexpr uint32_t FULL = 0xffffffffu;
constexpr float kRoundMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds to nearest-even at integer precision

// Where the 16-bit row of a task-local token comes from: the call's input, or - for the first n_win tokens of a task
// when a residual window is kept - the window's ring of rows (token t in slot t % R; a task never wraps the ring).
struct RowSrc {
  const uint16_t* in;     // row of task-local token 0 in the input (never dereferenced before the first new token)
  int64_t st;             // input row stride in elements
  const uint16_t* win;    // window row of task-local token 0 (this side), or nullptr
  int n_win;              // task-local tokens [0, n_win) are read from the window
  int wst;                // window row stride in elements (2 D: key row, value row)
  __device__ __forceinline__ const uint16_t* row(int tau) const {
    return (tau < n_win) ? win + (size_t)tau * wst : in + (int64_t)tau * st;
  }
};

// Tokens handled by one warp task: 32, or 64 where 32 tokens would leave a lane fewer than the four tokens
// that make up a word of value codes.
__host__ __device__ constexpr int task_tokens(int D, int bits) { return (D == 64 && bits == 2) ? 64 : 32; }

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Four byte values held as exact float integers (0..255) -> one little-endian word.
__device__ __forceinline__ uint32_t pack_bytes(float b0, float b1, float b2, float b3) {
  const float lo = __fmaf_rn(b1, 256.0f, b0), hi = __fmaf_rn(b3, 256.0f, b2);        // < 65536: exact
  return prmt(__float_as_uint(__fadd_rn(lo, 8388608.0f)), __float_as_uint(__fadd_rn(hi, 8388608.0f)), 0x5410);
}

// Quantize one side of a task of TT tokens.  src: row of the task's first token in the input; tokens
// [lo, hi) of the task are new.  codes: keys - the page's key row of the task's first token; values - the
// page's value block of the task's first token.  meta_out: metadata row of the task's first token.
//
// Lane = (row slot rs, word column mw, row half rh): it owns, for each of its tokens, the FPB pieces of
// 8 channels 16 (FPB mw + f) + 8 rh + {0..7}, f < FPB, whose codes share bytes.
template <int BITS, bool IS_V, int D, int DTYPE, bool ROT>
__device__ __forceinline__ void quantize_task(const RowSrc& rsrc, int gsz, int lo, int hi,
                                              uint8_t* __restrict__ codes, uint32_t* __restrict__ meta_out,
                                              int lane, const int8_t* __restrict__ signs) {
  constexpr int FPB = 8 / BITS;
  constexpr int NMW = (D / 16) / FPB;        // word columns per row half
  constexpr int LR = 2 * NMW;                // lanes per token row
  constexpr int RS = 32 / LR;                // token rows per load instruction
  constexpr int TT = task_tokens(D, BITS);
  constexpr int TPL = TT / RS;               // tokens per lane
  constexpr int K_ROW_BYTES = D * BITS / 8;
  static_assert(TPL % 4 == 0, "a lane holds whole groups of four tokens");
  const int rs = lane / LR, cs = lane % LR, mw = cs >> 1, rh = cs & 1;
  const float qmax = (float)((1 << BITS) - 1);
  const int spg = gsz >> 4;                                  // 16-channel slices per group
  const bool split = FPB > spg;                              // a lane's fields belong to two groups (FPB 4, groups of 32)
  const int lpg = split ? 2 : 2 * spg / FPB;                 // lanes per group
  const int ng = D / gsz;

  // block-local token of token slot k
  auto token_of = [&](int k) {
    if constexpr (IS_V) {
      const int cmb = (k >> 2) * RS + rs, j = k & 3;         // cmb = (block, half, t) of the word; j = byte
      return 32 * (cmb >> 3) + 16 * ((cmb >> 2) & 1) + 2 * (cmb & 3) + (j >> 1) + 8 * (j & 1);
    } else {
      return k * RS + rs;
    }
  };

  // ---- all loads first (TPL * FPB 16-byte loads in flight per lane)
  uint4 raw[TPL][FPB];
#pragma unroll
  for (int k = 0; k < TPL; ++k) {
    const int tau = token_of(k);
    const bool valid = tau >= lo && tau < hi;
#pragma unroll
    for (int f = 0; f < FPB; ++f) {
      raw[k][f] = make_uint4(0u, 0u, 0u, 0u);
      if (valid) raw[k][f] = __ldcs(reinterpret_cast<const uint4*>(rsrc.row(tau) + 16 * (FPB * mw + f) + 8 * rh));
    }
  }

  float vbyte[4][8];      // values: byte values (exact float integers) of the four tokens of the words being built
#pragma unroll
  for (int k = 0; k < TPL; ++k) {
    const int tau = token_of(k);
    const bool valid = tau >= lo && tau < hi;
    float x[FPB][8];
#pragma unroll
    for (int f = 0; f < FPB; ++f) {
      const uint32_t rw[4] = {raw[k][f].x, raw[k][f].y, raw[k][f].z, raw[k][f].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if constexpr (DTYPE == KVQ_BF16) {
          x[f][2 * i] = __uint_as_float(rw[i] << 16);
          x[f][2 * i + 1] = __uint_as_float(rw[i] & 0xFFFF0000u);
        } else {
          const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&rw[i]));
          x[f][2 * i] = v.x;
          x[f][2 * i + 1] = v.y;
        }
      }
    }
    if constexpr (ROT) {
      // keys only: y = H (signs * x) / sqrt(D); channel d = 16 (FPB mw + f) + 8 rh + i.  Butterfly stages in
      // the order h = 1, 2, 4, ...: bits of i in the lane, rh across lanes, bits of f in the lane, bits of mw across lanes.
#pragma unroll
      for (int f = 0; f < FPB; ++f) {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[f][i] = __fmul_rn(x[f][i], (float)signs[16 * (FPB * mw + f) + 8 * rh + i]);
#pragma unroll
        for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if ((i & h) == 0) {
              const float a = x[f][i], b = x[f][i + h];
              x[f][i] = __fadd_rn(a, b);
              x[f][i + h] = __fsub_rn(a, b);
            }
          }
        }
      }
#pragma unroll
      for (int f = 0; f < FPB; ++f) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float o = __shfl_xor_sync(FULL, x[f][i], 1);
          x[f][i] = rh ? __fsub_rn(o, x[f][i]) : __fadd_rn(x[f][i], o);
        }
      }
#pragma unroll
      for (int hf = 1; hf < FPB; hf <<= 1) {
#pragma unroll
        for (int f = 0; f < FPB; ++f) {
          if ((f & hf) == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float a = x[f][i], b = x[f + hf][i];
              x[f][i] = __fadd_rn(a, b);
              x[f + hf][i] = __fsub_rn(a, b);
            }
          }
        }
      }
#pragma unroll
      for (int hm = 1; hm < NMW; hm <<= 1) {
        const bool upper = (mw & hm) != 0;
#pragma unroll
        for (int f = 0; f < FPB; ++f) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float o = __shfl_xor_sync(FULL, x[f][i], 2 * hm);
            x[f][i] = upper ? __fsub_rn(o, x[f][i]) : __fadd_rn(x[f][i], o);
          }
        }
      }
#pragma unroll
      for (int f = 0; f < FPB; ++f) {
#pragma unroll
        for (int i = 0; i < 8; ++i) x[f][i] = __fmul_rn(x[f][i], inv_sqrt_dim<D>());
      }
    }

    // ---- group minimum / maximum: fields in the lane, then the lanes of the group
    float mnf[FPB], mxf[FPB];
#pragma unroll
    for (int f = 0; f < FPB; ++f) {
      mnf[f] = fminf(fminf(fminf(x[f][0], x[f][1]), fminf(x[f][2], x[f][3])),
                     fminf(fminf(x[f][4], x[f][5]), fminf(x[f][6], x[f][7])));
      mxf[f] = fmaxf(fmaxf(fmaxf(x[f][0], x[f][1]), fmaxf(x[f][2], x[f][3])),
                     fmaxf(fmaxf(x[f][4], x[f][5]), fmaxf(x[f][6], x[f][7])));
    }
    float mnA = mnf[0], mxA = mxf[0], mnB = mnf[FPB - 1], mxB = mxf[FPB - 1];
    if constexpr (FPB == 2) {
      mnA = mnB = fminf(mnf[0], mnf[1]);
      mxA = mxB = fmaxf(mxf[0], mxf[1]);
    }
    if constexpr (FPB == 4) {
      mnA = fminf(mnf[0], mnf[1]); mxA = fmaxf(mxf[0], mxf[1]);
      mnB = fminf(mnf[2], mnf[3]); mxB = fmaxf(mxf[2], mxf[3]);
      if (!split) {
        mnA = mnB = fminf(mnA, mnB);
        mxA = mxB = fmaxf(mxA, mxB);
      }
    }
#pragma unroll
    for (int off = 1; off < LR; off <<= 1) {
      if (off < lpg) {
        mnA = fminf(mnA, __shfl_xor_sync(FULL, mnA, off));
        mxA = fmaxf(mxA, __shfl_xor_sync(FULL, mxA, off));
        if constexpr (FPB == 4) {
          if (split) {
            mnB = fminf(mnB, __shfl_xor_sync(FULL, mnB, off));
            mxB = fmaxf(mxB, __shfl_xor_sync(FULL, mxB, off));
          }
        }
      }
    }
    const GroupParams pA = group_params(mnA, mxA, qmax);
    GroupParams pB = pA;
    if constexpr (FPB == 4) {
      if (split) pB = group_params(mnB, mxB, qmax);
    }
    if (valid && (cs & (lpg - 1)) == 0) {
      const int gi = (16 * FPB * mw) / gsz;                 // group of the lane's first field
      meta_out[tau * ng + gi] = pA.meta;
      if constexpr (FPB == 4) {
        if (split) meta_out[tau * ng + gi + 1] = pB.meta;
      }
    }

    // ---- codes as exact float integers, the FPB fields of a byte combined: byte = sum_f code_f * 2^(BITS f)
    float bytev[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) bytev[i] = 0.f;
#pragma unroll
    for (int f = FPB - 1; f >= 0; --f) {
      const GroupParams& p = (FPB == 4 && f >= 2) ? pB : pA;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float u = __fmul_rn(__fsub_rn(x[f][i], p.z), p.inv);
        u = fminf(fmaxf(u, 0.0f), qmax);
        const float r = __fsub_rn(__fadd_rn(u, kRoundMagic), kRoundMagic);      // rint(u), exact
        bytev[i] = __fmaf_rn(bytev[i], (float)(1 << BITS), r);                  // exact: < 256
      }
    }

    if constexpr (!IS_V) {
      // keys: bytes 0..3 of a word are channels 4 hh + {0..3} of this lane's 8, chunk 2 rh + hh, word mw of the row
      if (valid) {
        constexpr int wpc = D * BITS / 128;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const uint32_t w = pack_bytes(bytev[4 * hh], bytev[4 * hh + 1], bytev[4 * hh + 2], bytev[4 * hh + 3]);
          *reinterpret_cast<uint32_t*>(codes + (size_t)tau * K_ROW_BYTES + chunk_word_byte(2 * rh + hh, mw, wpc, 4)) = w;
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) vbyte[k & 3][i] = bytev[i];
      if ((k & 3) == 3) {
        // the four tokens (bytes) of this lane's words are complete: word of channel slot i at lane chunk 4 i + t
        const int cmb = (k >> 2) * RS + rs;
        uint8_t* wbase = codes + (size_t)(cmb >> 3) * (4 * D * BITS) + mw * 512 + (cmb & 3) * 16 +
                         4 * (2 * rh + ((cmb >> 2) & 1));
        const int t4 = 32 * (cmb >> 3) + 16 * ((cmb >> 2) & 1) + 2 * (cmb & 3);   // token of byte 0; bytes 1..3: +8, +1, +9
        const bool v0 = t4 >= lo && t4 < hi, v1 = t4 + 8 >= lo && t4 + 8 < hi;
        const bool v2 = t4 + 1 >= lo && t4 + 1 < hi, v3 = t4 + 9 >= lo && t4 + 9 < hi;
        if (v0 && v1 && v2 && v3) {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint32_t*>(wbase + 64 * i) = pack_bytes(vbyte[0][i], vbyte[1][i], vbyte[2][i], vbyte[3][i]);
        } else if (v0 || v1 || v2 || v3) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (v0) wbase[64 * i + 0] = (uint8_t)vbyte[0][i];
            if (v1) wbase[64 * i + 1] = (uint8_t)vbyte[1][i];
            if (v2) wbase[64 * i + 2] = (uint8_t)vbyte[2][i];
            if (v3) wbase[64 * i + 3] = (uint8_t)vbyte[3][i];
          }
        }
      }
    }
  }
}

// Minimum and maximum of the eight 16-bit values of a 16-byte piece, taken in the 16-bit type itself (two at a
// time; exact, since every 16-bit value is an fp32 value and the order is the same).
template <int DTYPE>
__device__ __forceinline__ void minmax8(const uint4& r, float& mn, float& mx) {
  if constexpr (DTYPE == KVQ_BF16) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r);
    const __nv_bfloat162 lo = __hmin2(__hmin2(h[0], h[1]), __hmin2(h[2], h[3]));
    const __nv_bfloat162 hi = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
    mn = fminf(__low2float(lo), __high2float(lo));
    mx = fmaxf(__low2float(hi), __high2float(hi));
  } else {
    const __half2* h = reinterpret_cast<const __half2*>(&r);
    const __half2 lo = __hmin2(__hmin2(h[0], h[1]), __hmin2(h[2], h[3]));
    const __half2 hi = __hmax2(__hmax2(h[0], h[1]), __hmax2(h[2], h[3]));
    mn = fminf(__low2float(lo), __high2float(lo));
    mx = fmaxf(__low2float(hi), __high2float(hi));
  }
}

// quantize_task without rotation, four tokens per pass: the group minima / maxima of the four tokens are
// reduced with a shuffle reduce-scatter, so that the group parameters (two divisions) are computed once per
// group rather than once per lane, and are then broadcast to the lanes of the group.  FULLBLK: every token of
// the task is new (no predicates).  Same results as quantize_task, bit for bit.
template <int BITS, bool IS_V, int D, int DTYPE, bool FULLBLK>
__device__ __forceinline__ void quantize_task_fast(const RowSrc& rsrc, int gsz, int lo,
                                                   int hi, uint8_t* __restrict__ codes,
                                                   uint32_t* __restrict__ meta_out, int lane) {
  constexpr int FPB = 8 / BITS;
  constexpr int NMW = (D / 16) / FPB;
  constexpr int LR = 2 * NMW;
  constexpr int RS = 32 / LR;
  constexpr int TT = task_tokens(D, BITS);
  constexpr int TPL = TT / RS;
  constexpr int K_ROW_BYTES = D * BITS / 8;
  constexpr int NSET = FPB == 4 ? 2 : 1;      // a lane's fields may belong to two groups (groups of 32 at 2 bits)
  const int rs = lane / LR, cs = lane % LR, mw = cs >> 1, rh = cs & 1;
  const float qmax = (float)((1 << BITS) - 1);
  const int spg = gsz >> 4;
  const bool split = FPB > spg;
  const int lpg = split ? 2 : 2 * spg / FPB;                 // lanes per group: 2, 4, 8 or 16
  const int ng = D / gsz;
  const int b0 = cs & 1, b1 = (cs >> 1) & 1;
  const int gbase = lane & ~(lpg - 1);                       // first lane of this lane's group

  auto token_of = [&](int k) {
    if constexpr (IS_V) {
      const int cmb = (k >> 2) * RS + rs, j = k & 3;
      return 32 * (cmb >> 3) + 16 * ((cmb >> 2) & 1) + 2 * (cmb & 3) + (j >> 1) + 8 * (j & 1);
    } else {
      return k * RS + rs;
    }
  };

#pragma unroll 1
  for (int pass = 0; pass < TPL / 4; ++pass) {
    uint4 raw[4][FPB];
    bool valid[4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const int tau = token_of(4 * pass + kk);
      valid[kk] = FULLBLK || (tau >= lo && tau < hi);
#pragma unroll
      for (int f = 0; f < FPB; ++f) {
        raw[kk][f] = make_uint4(0u, 0u, 0u, 0u);
        if (valid[kk]) raw[kk][f] = __ldcs(reinterpret_cast<const uint4*>(rsrc.row(tau) + 16 * (FPB * mw + f) + 8 * rh));
      }
    }
    // ---- phase 1: minima / maxima of the lane's fields, per token and per set
    float mn[NSET][4], mx[NSET][4];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      float fm[FPB], fx[FPB];
#pragma unroll
      for (int f = 0; f < FPB; ++f) minmax8<DTYPE>(raw[kk][f], fm[f], fx[f]);
      if constexpr (FPB == 1) { mn[0][kk] = fm[0]; mx[0][kk] = fx[0]; }
      if constexpr (FPB == 2) { mn[0][kk] = fminf(fm[0], fm[1]); mx[0][kk] = fmaxf(fx[0], fx[1]); }
      if constexpr (FPB == 4) {
        mn[0][kk] = fminf(fm[0], fm[1]); mx[0][kk] = fmaxf(fx[0], fx[1]);
        mn[1][kk] = fminf(fm[2], fm[3]); mx[1][kk] = fmaxf(fx[2], fx[3]);
        if (!split) {
          mn[0][kk] = mn[1][kk] = fminf(mn[0][kk], mn[1][kk]);
          mx[0][kk] = mx[1][kk] = fmaxf(mx[0][kk], mx[1][kk]);
        }
      }
    }
    // ---- reduce-scatter over the lanes of the group: after lane bit 0 a lane holds tokens 2 b0 + {0, 1}, after
    // bit 1 (groups of 4 lanes or more) token 2 b0 + b1; higher bits are plain butterflies
    float pz[NSET][2], pinv[NSET][2];
    uint32_t pmeta[NSET][2];
#pragma unroll
    for (int e = 0; e < NSET; ++e) {
      if (e == 1 && !split) break;
      float a0, a1, c0, c1;
      {
        const float sm0 = b0 ? mn[e][0] : mn[e][2], sm1 = b0 ? mn[e][1] : mn[e][3];
        const float sx0 = b0 ? mx[e][0] : mx[e][2], sx1 = b0 ? mx[e][1] : mx[e][3];
        a0 = fminf(b0 ? mn[e][2] : mn[e][0], __shfl_xor_sync(FULL, sm0, 1));
        a1 = fminf(b0 ? mn[e][3] : mn[e][1], __shfl_xor_sync(FULL, sm1, 1));
        c0 = fmaxf(b0 ? mx[e][2] : mx[e][0], __shfl_xor_sync(FULL, sx0, 1));
        c1 = fmaxf(b0 ? mx[e][3] : mx[e][1], __shfl_xor_sync(FULL, sx1, 1));
      }
      if (lpg >= 4) {
        const float sm = b1 ? a0 : a1, sx = b1 ? c0 : c1;
        a0 = fminf(b1 ? a1 : a0, __shfl_xor_sync(FULL, sm, 2));
        c0 = fmaxf(b1 ? c1 : c0, __shfl_xor_sync(FULL, sx, 2));
      }
      if (lpg >= 8) {
        a0 = fminf(a0, __shfl_xor_sync(FULL, a0, 4));
        c0 = fmaxf(c0, __shfl_xor_sync(FULL, c0, 4));
      }
      if (lpg >= 16) {
        a0 = fminf(a0, __shfl_xor_sync(FULL, a0, 8));
        c0 = fmaxf(c0, __shfl_xor_sync(FULL, c0, 8));
      }
      const GroupParams p0 = group_params(a0, c0, qmax);
      pz[e][0] = p0.z; pinv[e][0] = p0.inv; pmeta[e][0] = p0.meta;
      pz[e][1] = 0.f; pinv[e][1] = 0.f; pmeta[e][1] = 0u;
      if (lpg == 2) {
        const GroupParams p1 = group_params(a1, c1, qmax);
        pz[e][1] = p1.z; pinv[e][1] = p1.inv; pmeta[e][1] = p1.meta;
      }
      // the lane (one per group) that holds a token's parameters stores its metadata word
      if ((cs & (lpg - 1) & ~3) == 0) {
        const int gi = (16 * FPB * mw) / gsz + e;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          if (i == 1 && lpg != 2) break;
          const int kk = 2 * b0 + (lpg >= 4 ? b1 : i);
          const int tau = token_of(4 * pass + kk);
          if (FULLBLK || (tau >= lo && tau < hi)) meta_out[tau * ng + gi] = pmeta[e][i];
        }
      }
    }
    // ---- phase 2: codes, token by token, with the group's parameters fetched from the lane that made them
    float vbyte[4][8];
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const int tau = token_of(4 * pass + kk);
      const int srcl = gbase + (lpg >= 4 ? (kk >> 1) + 2 * (kk & 1) : (kk >> 1));
      const int el = (lpg >= 4) ? 0 : (kk & 1);
      float zA, iA, zB, iB;
      zA = __shfl_sync(FULL, el ? pz[0][1] : pz[0][0], srcl);
      iA = __shfl_sync(FULL, el ? pinv[0][1] : pinv[0][0], srcl);
      zB = zA; iB = iA;
      if constexpr (NSET == 2) {
        if (split) {
          zB = __shfl_sync(FULL, el ? pz[1][1] : pz[1][0], srcl);
          iB = __shfl_sync(FULL, el ? pinv[1][1] : pinv[1][0], srcl);
        }
      }
      float bytev[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) bytev[i] = 0.f;
#pragma unroll
      for (int f = FPB - 1; f >= 0; --f) {
        const float z = (FPB == 4 && f >= 2) ? zB : zA, inv = (FPB == 4 && f >= 2) ? iB : iA;
        const uint32_t rw[4] = {raw[kk][f].x, raw[kk][f].y, raw[kk][f].z, raw[kk][f].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float xa, xb;
          if constexpr (DTYPE == KVQ_BF16) {
            xa = __uint_as_float(rw[i] << 16);
            xb = __uint_as_float(rw[i] & 0xFFFF0000u);
          } else {
            const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&rw[i]));
            xa = v.x; xb = v.y;
          }
          float ua = __fmul_rn(__fsub_rn(xa, z), inv), ub = __fmul_rn(__fsub_rn(xb, z), inv);
          ua = fminf(fmaxf(ua, 0.0f), qmax);
          ub = fminf(fmaxf(ub, 0.0f), qmax);
          const float ra = __fsub_rn(__fadd_rn(ua, kRoundMagic), kRoundMagic);
          const float rb = __fsub_rn(__fadd_rn(ub, kRoundMagic), kRoundMagic);
          bytev[2 * i] = __fmaf_rn(bytev[2 * i], (float)(1 << BITS), ra);
          bytev[2 * i + 1] = __fmaf_rn(bytev[2 * i + 1], (float)(1 << BITS), rb);
        }
      }
      if constexpr (!IS_V) {
        if (valid[kk]) {
          constexpr int wpc = D * BITS / 128;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const uint32_t w = pack_bytes(bytev[4 * hh], bytev[4 * hh + 1], bytev[4 * hh + 2], bytev[4 * hh + 3]);
            *reinterpret_cast<uint32_t*>(codes + (size_t)tau * K_ROW_BYTES + chunk_word_byte(2 * rh + hh, mw, wpc, 4)) = w;
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) vbyte[kk][i] = bytev[i];
      }
    }
    if constexpr (IS_V) {
      const int cmb = pass * RS + rs;
      uint8_t* wbase = codes + (size_t)(cmb >> 3) * (4 * D * BITS) + mw * 512 + (cmb & 3) * 16 +
                       4 * (2 * rh + ((cmb >> 2) & 1));
      if (FULLBLK || (valid[0] && valid[1] && valid[2] && valid[3])) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          *reinterpret_cast<uint32_t*>(wbase + 64 * i) = pack_bytes(vbyte[0][i], vbyte[1][i], vbyte[2][i], vbyte[3][i]);
      } else if (valid[0] || valid[1] || valid[2] || valid[3]) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            if (valid[kk]) wbase[64 * i + kk] = (uint8_t)vbyte[kk][i];
        }
      }
    }
  }
}

// Bit-plane widths (1, 3, 6 bits): a plain variant, one token row per warp step.  A lane holds 8 consecutive
// channels of a row, groups reduce by butterflies, and every code's plane fields are cleared and set with atomic
// AND / OR on the 32-bit words of the page (several lanes share a word).  Not tuned: these widths are served for
// the paper's 1-, 3- and 6-bit settings, the 2/4/8-bit path above is the fast one.
template <int D, int DTYPE>
__device__ __forceinline__ void quantize_task_planes(const RowSrc& rsrc, int gsz, int bits,
                                                     bool is_v, int lo, int hi, int tp0, uint8_t* __restrict__ region,
                                                     uint32_t* __restrict__ meta_out, int lane) {
  constexpr int LPR = D / 8, RPW = 32 / LPR;           // lanes per row, rows per warp step
  const int l = lane % LPR, r0 = lane / LPR;
  const int lpg = gsz >> 3, ng = D / gsz;
  const float qmax = (float)((1 << bits) - 1);
  for (int base = lo; base < hi; base += RPW) {
    const int tau = base + r0;                         // task-local token
    const bool valid = tau < hi;
    uint4 raw = make_uint4(0u, 0u, 0u, 0u);
    if (valid) raw = *reinterpret_cast<const uint4*>(rsrc.row(tau) + 8 * l);
    const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
    float x[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = bits16_to_f32((uint16_t)(rw[i] & 0xFFFF), DTYPE);
      x[2 * i + 1] = bits16_to_f32((uint16_t)(rw[i] >> 16), DTYPE);
    }
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
    if (!valid) continue;
    const int t = tp0 + tau;                           // page-local token
    if ((l & (lpg - 1)) == 0) meta_out[tau * ng + (8 * l) / gsz] = p.meta;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t code = code_of(x[i], p, qmax);
      int hb, lb;
      planes_of(bits, hb, lb);
#pragma unroll
      for (int plane = 0; plane < 2; ++plane) {
        if (plane == 1 && lb == 0) break;
        int wb, bit, pb;
        plane_pos(is_v, t, 8 * l + i, D, bits, plane, wb, bit, pb);
        const uint32_t field = (plane == 0 ? (code >> lb) : code) & ((1u << pb) - 1u);
        uint32_t* w = reinterpret_cast<uint32_t*>(region + wb);
        atomicAnd(w, ~(((1u << pb) - 1u) << bit));
        atomicOr(w, field << bit);
      }
    }
  }
}

// 16-bit passthrough of one side of a task: rows [lo, hi) copied to the page as they are.
__device__ __forceinline__ void copy_task_side(const RowSrc& rsrc, int D, int lo, int hi,
                                               uint16_t* __restrict__ dst_rows, int lane) {
  const int lpr = D >> 3, rps = 32 / lpr, l = lane & (lpr - 1);
  for (int row = lo + lane / lpr; row < hi; row += rps)
    *reinterpret_cast<uint4*>(dst_rows + (size_t)row * D + l * 8) =
        *reinterpret_cast<const uint4*>(rsrc.row(row) + l * 8);
}

// An append of t_new tokens at position t0 fits the cache; written without a sum that could overflow.
__host__ __device__ __forceinline__ bool append_fits(int t0, int t_new, int capacity) {
  return t0 >= 0 && t0 <= capacity - t_new;
}

// Token-wise quantization of V (blockIdx.z == 0) and of K (blockIdx.z == 1).  grid.y = stream, grid.x strides
// over the warp tasks touched by this append.
template <int D, int DTYPE, bool ROT>
__global__ void __launch_bounds__(kThreads, ROT ? 1 : 3)
quant_token_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                   int64_t sb, int64_t sh, int64_t st, int t_new) {
  const bool is_v = blockIdx.z == 0;
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (!append_fits(t0, t_new, g.capacity)) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int bits = is_v ? g.vb : g.kb;
  const int TT = (bits == 16 || is_plane_width(bits)) ? 32 : task_tokens(D, bits);
  // tokens to quantize: the new ones, or - with a residual window of R tokens - the blocks of R that this append
  // completes (their first tokens may come from the window, the rest from the input)
  const int R = g.R;
  const int qa = R ? (t0 / R) * R : t0, qb = R ? ((t0 + t_new) / R) * R : t0 + t_new;
  if (qb <= qa) return;
  const int first_task = qa / TT;
  const int n_tasks = (qb + TT - 1) / TT - first_task;
  const uint16_t* in = is_v ? v_new : k_new;
  const int gsz = is_v ? g.gv : g.gk;

  for (int j = blockIdx.x * kWarps + warp; j < n_tasks; j += gridDim.x * kWarps) {
    const int tk0 = (first_task + j) * TT;                     // first token of the task
    const int lo = max(qa, tk0) - tk0, hi = min(qb, tk0 + TT) - tk0;
    const int page = tk0 >> 7, tp0 = tk0 & 127;                // page-local token of the task's first row
    uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
    // row 0 of the task in the input (may lie before the first new token; never dereferenced there)
    RowSrc rs;
    rs.in = in + (int64_t)b * sb + (int64_t)h * sh + (int64_t)(tk0 - t0) * st;
    rs.st = st;
    rs.n_win = R ? max(0, min(TT, t0 - tk0)) : 0;
    rs.wst = 2 * D;
    rs.win = R ? c.kv_win + ((size_t)bh * R + (tk0 % R)) * (2 * D) + (is_v ? D : 0) : nullptr;
    if (is_v) {
      if (bits == 16) {
        copy_task_side(rs, D, lo, hi, reinterpret_cast<uint16_t*>(pg + g.v_codes_off) + (size_t)tp0 * D, lane);
        continue;
      }
      if (is_plane_width(bits)) {
        quantize_task_planes<D, DTYPE>(rs, gsz, bits, true, lo, hi, tp0, pg + g.v_codes_off,
                                       reinterpret_cast<uint32_t*>(pg + g.v_meta_off) + tp0 * (D / gsz), lane);
        continue;
      }
      uint8_t* vb = pg + g.v_codes_off + (size_t)(tp0 >> 5) * (4 * D * bits);
      uint32_t* vm = reinterpret_cast<uint32_t*>(pg + g.v_meta_off) + tp0 * (D / gsz);
      const bool full = lo == 0 && hi == TT;
      if (bits == 2) {
        if (full) quantize_task_fast<2, true, D, DTYPE, true>(rs, gsz, lo, hi, vb, vm, lane);
        else quantize_task_fast<2, true, D, DTYPE, false>(rs, gsz, lo, hi, vb, vm, lane);
      } else if (bits == 4) {
        if (full) quantize_task_fast<4, true, D, DTYPE, true>(rs, gsz, lo, hi, vb, vm, lane);
        else quantize_task_fast<4, true, D, DTYPE, false>(rs, gsz, lo, hi, vb, vm, lane);
      } else {
        if (full) quantize_task_fast<8, true, D, DTYPE, true>(rs, gsz, lo, hi, vb, vm, lane);
        else quantize_task_fast<8, true, D, DTYPE, false>(rs, gsz, lo, hi, vb, vm, lane);
      }
    } else {
      if (bits == 16) {
        copy_task_side(rs, D, lo, hi, reinterpret_cast<uint16_t*>(pg) + (size_t)tp0 * D, lane);
        continue;
      }
      if (is_plane_width(bits)) {
        quantize_task_planes<D, DTYPE>(rs, gsz, bits, false, lo, hi, tp0, pg,
                                       reinterpret_cast<uint32_t*>(pg + g.k_meta_off) + tp0 * (D / gsz), lane);
        continue;
      }
      uint8_t* kr = pg + (size_t)tp0 * (D * bits / 8);
      uint32_t* km = reinterpret_cast<uint32_t*>(pg + g.k_meta_off) + tp0 * (D / gsz);
      if constexpr (ROT) {
        if (bits == 2) quantize_task<2, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane, c.k_signs);
        else if (bits == 4) quantize_task<4, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane, c.k_signs);
        else quantize_task<8, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane, c.k_signs);
      } else {
        const bool full = lo == 0 && hi == TT;
        if (bits == 2) {
          if (full) quantize_task_fast<2, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane);
          else quantize_task_fast<2, false, D, DTYPE, false>(rs, gsz, lo, hi, kr, km, lane);
        } else if (bits == 4) {
          if (full) quantize_task_fast<4, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane);
          else quantize_task_fast<4, false, D, DTYPE, false>(rs, gsz, lo, hi, kr, km, lane);
        } else {
          if (full) quantize_task_fast<8, false, D, DTYPE, true>(rs, gsz, lo, hi, kr, km, lane);
          else quantize_task_fast<8, false, D, DTYPE, false>(rs, gsz, lo, hi, kr, km, lane);
        }
      }
    }
  }
}

// Pack K rows: `codes` holds bytes [ntok rows][D]; row r goes to page-local token slot0 + r.
__device__ __forceinline__ void pack_k_rows(const uint8_t* codes, int code_stride, int ntok, int slot0,
                                            uint8_t* kregion, int D, int b, int tid) {
  const int wpr = D * b / 32;    // words per row
  const int wpc = wpr / 4;       // words per chunk
  const int nf = 32 / b;
  for (int idx = tid; idx < ntok * wpr; idx += kThreads) {
    int r = idx / wpr, wi = idx % wpr;
    int chunk = wi / wpc, word = wi % wpc;
    uint32_t w = 0;
    for (int f = 0; f < nf; ++f) {
      int d = k_field_channel(chunk, word, f, b);
      w |= (uint32_t)codes[r * code_stride + d] << (f * b);
    }
    *reinterpret_cast<uint32_t*>(kregion + (size_t)(slot0 + r) * (D * b / 8) + chunk_word_byte(chunk, word, wpc, 4)) = w;
  }
}

// Channel-wise quantization of one complete 128-token block held as fp16 in shared memory, head_dim 128, 4- or
// 8-bit codes.  Thread = (token quarter, slice pair rp, channel pair pi): the four channels 32 rp + 2 pi + {0, 1}
// and 32 rp + 16 + 2 pi + {0, 1}, whose codes share two adjacent bytes (4 bits) or two adjacent byte pairs
// (8 bits) of every token row.  Minimum and maximum are taken two channels at a time in fp16 (exact), the
// parameters once per channel, and the codes are written as whole bytes into a shared image of the page's key
// region, which leaves with 16-byte stores.
template <int KB>
__device__ __forceinline__ void kchan_block_fast(const uint16_t* sX, uint8_t* sImg, uint8_t* pg, const Geom& g, int tid) {
  constexpr int D = 128, ROW = D * KB / 8;
  const __half2* sX2 = reinterpret_cast<const __half2*>(sX);            // [128][64]
  __half2* sRed = reinterpret_cast<__half2*>(sImg);                    // [4 quarters][32][4], dead before the image is written
  const int q = tid >> 5, l32 = tid & 31, rp = l32 >> 3, pi = l32 & 7;
  const int w_lo = 16 * rp + pi, w_hi = w_lo + 8;
  const float qmax = (float)((1 << KB) - 1);
  __half2 mn_lo = sX2[(32 * q) * 64 + w_lo], mx_lo = mn_lo, mn_hi = sX2[(32 * q) * 64 + w_hi], mx_hi = mn_hi;
#pragma unroll 8
  for (int t = 32 * q + 1; t < 32 * q + 32; ++t) {
    const __half2 a = sX2[t * 64 + w_lo], b = sX2[t * 64 + w_hi];
    mn_lo = __hmin2(mn_lo, a); mx_lo = __hmax2(mx_lo, a);
    mn_hi = __hmin2(mn_hi, b); mx_hi = __hmax2(mx_hi, b);
  }
  sRed[(q * 32 + l32) * 4 + 0] = mn_lo; sRed[(q * 32 + l32) * 4 + 1] = mx_lo;
  sRed[(q * 32 + l32) * 4 + 2] = mn_hi; sRed[(q * 32 + l32) * 4 + 3] = mx_hi;
  __syncthreads();
#pragma unroll
  for (int qq = 0; qq < 4; ++qq) {
    mn_lo = __hmin2(mn_lo, sRed[(qq * 32 + l32) * 4 + 0]); mx_lo = __hmax2(mx_lo, sRed[(qq * 32 + l32) * 4 + 1]);
    mn_hi = __hmin2(mn_hi, sRed[(qq * 32 + l32) * 4 + 2]); mx_hi = __hmax2(mx_hi, sRed[(qq * 32 + l32) * 4 + 3]);
  }
  const GroupParams p0 = group_params(__low2float(mn_lo), __low2float(mx_lo), qmax);     // channel 32 rp + 2 pi
  const GroupParams p1 = group_params(__high2float(mn_lo), __high2float(mx_lo), qmax);   // ... + 1
  const GroupParams p2 = group_params(__low2float(mn_hi), __low2float(mx_hi), qmax);     // ... + 16
  const GroupParams p3 = group_params(__high2float(mn_hi), __high2float(mx_hi), qmax);   // ... + 17
  if (q == 0) {
    uint32_t* meta = reinterpret_cast<uint32_t*>(pg + g.k_meta_off);
    const int d0 = 32 * rp + 2 * pi;
    meta[d0] = p0.meta; meta[d0 + 1] = p1.meta; meta[d0 + 16] = p2.meta; meta[d0 + 17] = p3.meta;
  }
  __syncthreads();                       // every thread has read the reduction scratch: the image may overwrite it
#pragma unroll 4
  for (int t = 32 * q; t < 32 * q + 32; ++t) {
    const float2 a = __half22float2(sX2[t * 64 + w_lo]), b = __half22float2(sX2[t * 64 + w_hi]);
    const uint32_t c0 = code_of_fast(a.x, p0, qmax), c1 = code_of_fast(a.y, p1, qmax);
    const uint32_t c2 = code_of_fast(b.x, p2, qmax), c3 = code_of_fast(b.y, p3, qmax);
    if constexpr (KB == 4) {
      // bytes 2 (pi % 2) + {0, 1} of word rp in chunk pi / 2: low nibble slice 2 rp, high nibble slice 2 rp + 1
      *reinterpret_cast<uint16_t*>(sImg + t * ROW + (pi >> 1) * 16 + rp * 4 + 2 * (pi & 1)) =
          (uint16_t)((c0 | (c2 << 4)) | ((c1 | (c3 << 4)) << 8));
    } else {
      const int wa = 2 * rp, wb = 2 * rp + 1;                      // words = slices 2 rp and 2 rp + 1
      *reinterpret_cast<uint16_t*>(sImg + t * ROW + (wa >> 2) * 64 + (pi >> 1) * 16 + (wa & 3) * 4 + 2 * (pi & 1)) =
          (uint16_t)(c0 | (c1 << 8));
      *reinterpret_cast<uint16_t*>(sImg + t * ROW + (wb >> 2) * 64 + (pi >> 1) * 16 + (wb & 3) * 4 + 2 * (pi & 1)) =
          (uint16_t)(c2 | (c3 << 8));
    }
  }
  __syncthreads();
  for (int i = tid; i < kPageTokens * ROW / 16; i += kThreads)
    reinterpret_cast<uint4*>(pg)[i] = reinterpret_cast<const uint4*>(sImg)[i];
}

// Channel-wise quantization of K over 128-token blocks with the fp16 tail.
// CTA j of a stream handles the j-th block touched by this append.  CTA 0 also
// handles the final block when that one is incomplete (it writes the tail, which
// CTA 0 must have finished reading first).
__global__ void __launch_bounds__(kThreads)
quant_kchan_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new,
                   int64_t sb, int64_t sh, int64_t st, int t_new) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int D = g.D;
  uint16_t* sX = reinterpret_cast<uint16_t*>(smem);          // [128][D] fp16 bits
  uint8_t* sC = smem + (size_t)kPageTokens * D * 2;           // [128][D] codes
  const int bh = blockIdx.y;
  const int b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (!append_fits(t0, t_new, g.capacity)) return;
  const int end = t0 + t_new;
  const int first_page = t0 >> 7;
  const int nblk = ((end + 127) >> 7) - first_page;
  const bool last_partial = (end & 127) != 0;
  const int tid = threadIdx.x;
  uint16_t* tail = c.k_tail + (size_t)bh * kPageTokens * D;
  const float qmax = (float)((1 << g.kb) - 1);

  for (int pass = 0; pass < 2; ++pass) {
    int j;
    if (pass == 0) {
      j = blockIdx.x;
      if (j >= nblk) return;
      if (j == nblk - 1 && last_partial && j != 0) return;   // done by CTA 0 in its second pass
    } else {
      if (blockIdx.x != 0 || nblk <= 1 || !last_partial) return;
      j = nblk - 1;
      __syncthreads();
    }
    const int page = first_page + j;
    const int tb = page << 7;
    const int lo = max(t0, tb) - tb, hi = min(end, tb + 128) - tb;   // new tokens occupy slots [lo, hi)
    const bool complete = (hi == 128);
    // gather the block: slots [0, lo) from the tail, [lo, hi) from the input (as saturated fp16)
    // (a row is handled by D/8 consecutive lanes, which is what the rotation's shuffles expect; every lane of a
    // warp runs the loop body, rows past the end are inactive)
    const int vec_per_row = D / 8;   // 16-byte vectors
    for (int base = 0; base < hi * vec_per_row; base += kThreads) {
      const int idx = base + tid;
      const bool active = idx < hi * vec_per_row;
      const int slot = idx / vec_per_row, v = idx % vec_per_row;
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      const bool is_new = active && slot >= lo;
      if (active && !is_new) val = *reinterpret_cast<const uint4*>(tail + (size_t)slot * D + v * 8);
      if (is_new)
        val = *reinterpret_cast<const uint4*>(k_new + (int64_t)b * sb + (int64_t)h * sh +
                                              (int64_t)(tb + slot - t0) * st + v * 8);
      if (c.k_signs != nullptr || g.in_dtype == KVQ_BF16) {
        // new tokens: to fp32, rotate if asked, store as saturated fp16
        uint32_t* w = reinterpret_cast<uint32_t*>(&val);
        float x[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[2 * i] = bits16_to_f32((uint16_t)(w[i] & 0xFFFF), g.in_dtype);
          x[2 * i + 1] = bits16_to_f32((uint16_t)(w[i] >> 16), g.in_dtype);
        }
        if (c.k_signs != nullptr) {
          if (D == 128) rotate_row8<128>(x, c.k_signs, v); else rotate_row8<64>(x, c.k_signs, v);
        }
        if (is_new) {
#pragma unroll
          for (int i = 0; i < 4; ++i)
            w[i] = (uint32_t)f32_to_fp16_sat_bits(x[2 * i]) | ((uint32_t)f32_to_fp16_sat_bits(x[2 * i + 1]) << 16);
        }
      }
      if (is_new && !complete) *reinterpret_cast<uint4*>(tail + (size_t)slot * D + v * 8) = val;
      if (active) *reinterpret_cast<uint4*>(sX + (size_t)slot * D + v * 8) = val;
    }
    if (!complete) continue;
    __syncthreads();
    uint8_t* pg = c.pages + ((size_t)bh * g.n_pages + page) * g.page_bytes;
    if (D == 128 && (g.kb == 4 || g.kb == 8)) {
      if (g.kb == 4) kchan_block_fast<4>(sX, sC, pg, g, tid); else kchan_block_fast<8>(sX, sC, pg, g, tid);
      continue;
    }
    for (int d = tid; d < D; d += kThreads) {
      float mn = INFINITY, mx = -INFINITY;
      for (int t = 0; t < kPageTokens; ++t) {
        float x = bits16_to_f32(sX[t * D + d], KVQ_FP16);
        mn = fminf(mn, x);
        mx = fmaxf(mx, x);
      }
      GroupParams p = group_params(mn, mx, qmax);
      reinterpret_cast<uint32_t*>(pg + g.k_meta_off)[d] = p.meta;
      for (int t = 0; t < kPageTokens; ++t)
        sC[t * D + d] = (uint8_t)code_of(bits16_to_f32(sX[t * D + d], KVQ_FP16), p, qmax);
    }
    __syncthreads();
    pack_k_rows(sC, D, kPageTokens, 0, pg, D, g.kb, tid);
  }
}

// Residual window: the new tokens that stay unquantized (positions >= the last complete block of R) are copied to
// the ring, key row and value row of token t in slot t % R.  Runs after the quantize kernel, which may still read
// the slots being replaced.
__global__ void __launch_bounds__(kThreads)
window_store_kernel(Geom g, CachePtrs c, const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                    int64_t sb, int64_t sh, int64_t st, int t_new) {
  const int bh = blockIdx.y, b = bh / g.Hkv, h = bh % g.Hkv;
  const int t0 = c.seq_len[b];
  if (!append_fits(t0, t_new, g.capacity)) return;
  const int R = g.R, D = g.D, vpr = D / 8;
  const int first = max(t0, ((t0 + t_new) / R) * R), n = t0 + t_new - first;     // tokens first .. first + n - 1 stay
  for (int idx = blockIdx.x * kThreads + threadIdx.x; idx < n * 2 * vpr; idx += gridDim.x * kThreads) {
    const int t = first + idx / (2 * vpr), side = (idx / vpr) & 1, vcol = idx % vpr;
    const uint16_t* src = (side ? v_new : k_new) + (int64_t)b * sb + (int64_t)h * sh + (int64_t)(t - t0) * st + 8 * vcol;
    uint16_t* dst = c.kv_win + (((size_t)bh * R + (t % R)) * 2 + side) * D + 8 * vcol;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
}

__global__ void bump_seq_len_kernel(Geom g, CachePtrs c, int t_new) {
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= g.B) return;
  int t0 = c.seq_len[b];
  if (!append_fits(t0, t_new, g.capacity)) {
    atomicOr(c.status, KVQ_STATUS_CAPACITY);
  } else {
    c.seq_len[b] = t0 + t_new;
  }
}

}  // namespace

int launch_quantize_append(const Geom& g, const CachePtrs& c, const void* k_new, const void* v_new,
                           int64_t sb, int64_t sh, int64_t st, int t_new, cudaStream_t stream) {
  const uint16_t* k = static_cast<const uint16_t*>(k_new);
  const uint16_t* v = static_cast<const uint16_t*>(v_new);
  // warp tasks touched per stream: at most ceil(t_new / 32) + 1; one warp per task, CTAs stride over them
  const int max_tasks = (t_new + 31) / 32 + 1;
  int gx = (max_tasks + kWarps - 1) / kWarps;
  const int streams = g.B * g.Hkv;
  const int want = (148 * 16 + streams - 1) / streams;       // enough CTAs to fill the GPU, not one per task
  if (gx > want) gx = want;
  dim3 grid1(gx, streams, g.k_axis == 0 ? 2 : 1);            // z = 0 values, z = 1 token-wise keys
  const bool rot = c.k_signs != nullptr && g.k_axis == 0;
#define KVQ_QLAUNCH(D_, T_)                                                                                  \
  do {                                                                                                       \
    if (rot) quant_token_kernel<D_, T_, true><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new); \
    else quant_token_kernel<D_, T_, false><<<grid1, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new);    \
  } while (0)
  if (g.D == 128 && g.in_dtype == KVQ_BF16) KVQ_QLAUNCH(128, KVQ_BF16);
  else if (g.D == 128) KVQ_QLAUNCH(128, KVQ_FP16);
  else if (g.in_dtype == KVQ_BF16) KVQ_QLAUNCH(64, KVQ_BF16);
  else KVQ_QLAUNCH(64, KVQ_FP16);
#undef KVQ_QLAUNCH
  if (g.k_axis == 1) {
    size_t smem = (size_t)kPageTokens * g.D * 3;
    cudaFuncSetAttribute(quant_kchan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 128 * 3);
    dim3 grid2((t_new + 127) / 128 + 1, streams);
    quant_kchan_kernel<<<grid2, kThreads, smem, stream>>>(g, c, k, sb, sh, st, t_new);
  }
  if (g.R) {
    dim3 grid3(1, streams);
    window_store_kernel<<<grid3, kThreads, 0, stream>>>(g, c, k, v, sb, sh, st, t_new);
  }
  bump_seq_len_kernel<<<(g.B + 127) / 128, 128, 0, stream>>>(g, c, t_new);
  return cudaGetLastError() == cudaSuccess ? KVQ_OK : KVQ_ERR_CUDA_LAUNCH;
}

}  // namespace kvq
