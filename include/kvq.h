/*
 * kvq - mixed-precision KV-cache quantization hot path for NVIDIA B200 (sm_100a).
 *
 * C-ABI of libkvq.so.  Plain C: POD structs, raw pointers, sizes.  No C++ or
 * torch types cross this boundary.  All `void*` / `int32_t*` data pointers in
 * kvq_cache and in the call arguments are DEVICE pointers owned by the caller;
 * kvq_config and kvq_cache structs themselves are HOST memory, read during the
 * call and never retained.  `cuda_stream` is a cudaStream_t passed as void*
 * (NULL = the legacy default stream).
 *
 * What is computed (arxiv 2502.15075, "Quantize What Counts: More for Keys,
 * Less for Values"): keys and values of the cache (K = X W^K, V = X W^V, one
 * L x d_head matrix per head, Sec. 3 / App. B.4) are stored with a uniform scalar
 * quantizer at independent bit widths b_K, b_V (Theorem 2: more bits for keys),
 * in groups of 32/64/128 elements, token-wise or channel-wise, with recent tokens
 * of an incomplete channel-wise block kept in 16-bit precision (Sec. 4.1).  A
 * decode step computes softmax(q K^T / sqrt(d)) V (App. A.1 notation) over the
 * reconstructed cache.
 *
 * Quantizer.  App. B.1 defines the symmetric uniform quantizer (alpha = M / (2^(b-1) - 1),
 * Q = round(A / alpha), A^ = alpha Q); this library applies the same uniform rounding per
 * group with the group minimum as offset (an asymmetric variant: scale = range / (2^b - 1)).
 * Fixed formula; every operation an individually rounded IEEE fp32 operation, ties to even:
 *     mn, mx  = min, max of the group, each + 0.0f   (-0 becomes +0)
 *     s16     = fp16_rn((mx - mn) / qmax), z16 = fp16_rn(mn), saturating at +-65504
 *     s, z    = (float)s16, (float)z16,  qmax = 2^b - 1
 *     code    = 0 if s == 0, else clamp(rintf((x - z) * (1.0f / s)), 0, qmax)
 *     x^      = fmaf(code, s, z)
 * Inputs must be finite.
 *
 * Packed page (layout version 2): 128 consecutive tokens of one
 * (batch, kv-head) stream, regions [K codes | K meta | V codes | V meta], each
 * a multiple of 16 bytes, little-endian.  Field f of a byte or word holds bits [f*b, f*b+b).
 *   K codes, b in {2,4,8}: rows of D*b/8 bytes per token, each holding 4 chunks of
 *     wpc = D*b/128 words; with fpb = 8/b fields per byte, channel d: chunk (d%16)/4,
 *     r = d/16, word r/fpb, bit 8*(d%4) + b*(r%fpb)  (byte j of a word holds channels
 *     16r + 4*chunk + j: one mask per field gives four consecutive channels as four bytes).
 *     (chunk, word) inside a row, with qw = min(wpc, 4):
 *     byte = (word/4)*(16*qw) + chunk*(4*qw) + (word%4)*4   (quads of words, quad-major).
 *   V codes, b in {2,4,8}: 4 blocks of 32 tokens, 4*D*b bytes each.  A byte holds the codes of
 *     one token for the fpb = 8/b channels that lie 16 apart.  With m = d/16, f = m%fpb,
 *     mw = m/fpb, rh = (d%16)/8, g = d%8 and, for block-local token tau, kh = tau/16,
 *     u = tau%16, t = (u%8)/2, j = 2*(u%2) + u/8:
 *     byte = block*(4*D*b) + mw*512 + (4*g + t)*16 + 4*(2*rh + kh) + j,  bit = b*f
 *     (the bytes of a word are tokens 2t, 2t+8, 2t+1, 2t+9 of one half of the block).
 *   b = 16: rows [token][D] of the input's 16-bit patterns, no meta.
 *   b in {1, 3, 6} (Table 1's 3-bit column; Sec. 4.1's 1- and 6-bit settings): bit planes.  A 3-bit code is a
 *     2-bit plane (code >> 1) followed by a 1-bit plane (code & 1), a 6-bit code a 4-bit plane (code >> 2)
 *     followed by a 2-bit plane (code & 3), a 1-bit code one 1-bit plane; every plane is a code region of its
 *     own width laid out as above, the high plane first (the region still holds 128*D*b/8 bytes).  Widths 1 and
 *     3 need head_dim 128; plane widths are token-wise only, are not combined with key rotation, and decode
 *     serves them through the plain-ALU kernel.
 *   Meta: (scale fp16, zero fp16) per group; per-token axis [128][D/g],
 *     per-channel K [D].
 * pages: [batch][n_kv_heads][capacity_tokens/128][page_bytes].
 * k_tail (k_axis == 1 only): fp16 [batch][n_kv_heads][128][head_dim]; holds
 *   fp16(x) of the keys of the incomplete last block; the block is quantized
 *   (one group per channel over its 128 tokens) when it fills up.
 */
#ifndef KVQ_H_
#define KVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVQ_LAYOUT_VERSION 2   /* changes whenever the bytes of a packed page change */
#define KVQ_PAGE_TOKENS 128

/* return codes (0 = success) */
#define KVQ_OK 0
#define KVQ_ERR_INVALID_ARG (-1)
#define KVQ_ERR_UNSUPPORTED (-2)
#define KVQ_ERR_MISALIGNED (-3)
#define KVQ_ERR_WORKSPACE_TOO_SMALL (-4)
#define KVQ_ERR_CAPACITY (-5)
#define KVQ_ERR_CUDA_LAUNCH (-6)
#define KVQ_ERR_DEVICE_TIMEOUT (-7)
#define KVQ_ERR_STATIC_SCRATCH (-8) /* problem needs more scratch than the library's built-in buffer */

/* bits that kernels OR into *kvq_cache.status (never trap) */
#define KVQ_STATUS_CAPACITY 1u       /* an append would exceed capacity_tokens; that sequence was skipped */
#define KVQ_STATUS_DEVICE_TIMEOUT 2u /* a bounded device-side wait expired */

/* dtypes */
#define KVQ_FP16 0
#define KVQ_BF16 1
#define KVQ_FP32 2 /* decode output only */

typedef struct {
  int32_t batch;
  int32_t n_q_heads;       /* multiple of n_kv_heads; query head h reads KV head h / (n_q_heads/n_kv_heads);
                              group size n_q_heads/n_kv_heads <= 8 */
  int32_t n_kv_heads;
  int32_t head_dim;        /* 64 or 128 */
  int32_t kb, vb;          /* 1, 2, 3, 4, 6, 8 quantized; 16 = unquantized passthrough */
  int32_t gk, gv;          /* group size along head_dim: 32, 64 or 128, dividing head_dim (per-token axis) */
  int32_t k_axis;          /* 0: keys token-wise; 1: keys channel-wise over 128-token blocks (needs kb != 16) */
  int32_t in_dtype;        /* KVQ_FP16 or KVQ_BF16: type of k_new, v_new, q and of dequantize's outputs */
  int32_t capacity_tokens; /* per sequence; multiple of 128 */
  int32_t residual_tokens; /* 0, or R = 64 or 128: the newest seq_len % R tokens of K and V stay in 16 bits in
                              kvq_cache.kv_win and are quantized as a block when R of them are complete (Sec. 4.1:
                              "a 64-token residual buffer ... periodically flushed").  Needs k_axis == 0. */
} kvq_config;

typedef struct {
  void* pages;      /* device; 16-byte aligned; see layout above */
  void* k_tail;     /* device fp16 tail, 16-byte aligned; NULL when k_axis == 0 */
  int32_t* seq_len; /* device [batch]: tokens stored per sequence (quantized + tail) */
  int32_t* status;  /* device, one word of KVQ_STATUS_* bits */
  const int8_t* k_signs; /* device [head_dim] of +1 / -1, or NULL.  Not NULL: keys are rotated before
                            quantization by y = H (signs * x) / sqrt(head_dim), H the Sylvester Hadamard matrix
                            (Sec. 4.4, key-only rotation, which the paper finds sufficient); decode applies the
                            same rotation to q, dequantize rotates back.  Needs kb != 16.  The transform is
                            computed in fp32 with butterfly stages h = 1, 2, 4, ... in this order, (a, b) ->
                            (a + b, a - b), then one multiplication by (float)(1/sqrt(head_dim)). */
  void* kv_win;     /* device, in_dtype [batch][n_kv_heads][residual_tokens][2][head_dim] (key row, value row of
                       token t in slot t % residual_tokens), 16-byte aligned; NULL when residual_tokens == 0 */
} kvq_cache;        /* one per layer.  The caller zeroes seq_len and status for a fresh cache;
                       pages must be zero-filled once before the first append. */

/* Layout queries (host only, no GPU work).  All return KVQ_OK or KVQ_ERR_INVALID_ARG /
 * KVQ_ERR_UNSUPPORTED for a config outside the documented ranges. */
int kvq_layout_version(void);
int kvq_page_bytes(const kvq_config* cfg, size_t* out);
int kvq_cache_bytes(const kvq_config* cfg, size_t* pages_bytes, size_t* k_tail_bytes);
int kvq_window_bytes(const kvq_config* cfg, size_t* kv_win_bytes);   /* 0 when residual_tokens == 0 */
/* Scratch needed by kvq_decode_attention for its split partial results. */
int kvq_workspace_bytes(const kvq_config* cfg, size_t* out);

/*
 * Quantize and pack t_new new tokens per sequence and append them at position
 * seq_len[b] (App. B.1 quantizer per group; Sec. 4.1 grouping and residual tail).
 *   k_new, v_new: device, in_dtype, logical shape [batch][n_kv_heads][t_new][head_dim];
 *     element (b,h,t,d) at offset b*stride_b + h*stride_h + t*stride_t + d (in elements);
 *     head_dim contiguous, base pointers and strides such that every row is 16-byte aligned.
 * With residual_tokens = R > 0 the new tokens first live in kv_win; the blocks of R tokens that this call completes
 * are quantized (their first tokens read from kv_win) and the tokens behind the last complete block are stored there.
 * Asynchronous on cuda_stream.  seq_len[b] += t_new for every sequence that fits; a sequence
 * with seq_len[b] + t_new > capacity_tokens is left untouched and KVQ_STATUS_CAPACITY is set.
 * Returns KVQ_OK or a host-detected argument / launch error (then nothing was launched).
 * Not safe to call concurrently on the same cache.
 */
int kvq_quantize_append(const kvq_config* cfg, const kvq_cache* cache,
                        const void* k_new, const void* v_new,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t,
                        int32_t t_new, void* cuda_stream);

/*
 * One decode step: out[b,h,:] = softmax_t(scale * q[b,h,:] . K^[b,h/G,t,:]) V^[b,h/G,t,:]
 * over t < seq_len[b] (App. A.1: S = Q K^T / sqrt(d), A = softmax(S), A V), streaming the
 * packed pages and reconstructing K^, V^ on the fly; tokens of an incomplete channel-wise
 * key block are read from the fp16 tail.  Split over the sequence, partial results merged by
 * log-sum-exp.  seq_len[b] == 0 gives zeros.  Tokens of a residual window (residual_tokens > 0) are attended in
 * full precision; that needs a configuration the tensor-core path serves (otherwise KVQ_ERR_UNSUPPORTED).
 *   q: device, in_dtype, [batch][n_q_heads][head_dim] contiguous.
 *   out: device, [batch][n_q_heads][head_dim] contiguous, out_dtype (KVQ_FP16/BF16/FP32).
 *   softmax_scale <= 0 selects 1/sqrt(head_dim).
 *   workspace: device scratch of at least kvq_workspace_bytes(), 16-byte aligned; contents
 *     need no initialisation and are undefined afterwards.  Calls that may overlap on the GPU
 *     need separate workspaces.
 * Asynchronous on cuda_stream; reads the cache only.
 */
int kvq_decode_attention(const kvq_config* cfg, const kvq_cache* cache,
                         const void* q, void* out, int32_t out_dtype, float softmax_scale,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Decode with several query rows per head (App. A.1: Q has one row per position, S = Q K^T / sqrt(d)), the shape
 * of speculative decoding and chunked prefill.  The n_rows rows are the queries of the LAST n_rows cached tokens of
 * each sequence (append their keys and values first), under a decoder's causal mask: row r attends to the tokens
 * t < seq_len[b] - (n_rows - 1 - r); a row whose token does not exist (seq_len[b] < n_rows - r) gives zeros.
 * n_rows = 1 is kvq_decode_attention.
 *   q, out: device, [batch][n_rows][n_q_heads][head_dim] contiguous (q in_dtype, out out_dtype).
 *   The (row, head) pairs of a KV head share its stream like query heads do: n_rows * (n_q_heads / n_kv_heads)
 *   may be up to 4 for every configuration the tensor-core path serves (2/4/8-bit codes, token-wise or
 *   channel-wise keys, head_dim 128, or head_dim 64 with K4V2 and groups of 64) and up to 8 for token-wise K4V2
 *   at head_dim 128; otherwise KVQ_ERR_UNSUPPORTED.  workspace: at least kvq_workspace_bytes_rows(cfg, n_rows).
 * Everything else as kvq_decode_attention.
 */
int kvq_workspace_bytes_rows(const kvq_config* cfg, int32_t n_rows, size_t* out);
int kvq_decode_attention_rows(const kvq_config* cfg, const kvq_cache* cache,
                              const void* q, int32_t n_rows, void* out, int32_t out_dtype, float softmax_scale,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Reconstruct tokens t_begin <= t < min(t_end, seq_len[b]) as x^ = fmaf(code, s, z) rounded to
 * in_dtype (App. B.1: A^ = scale * Q); tail keys are converted from fp16, tokens of a residual window are returned
 * as they were appended.
 *   k_out, v_out: device, in_dtype, [batch][n_kv_heads][capacity_tokens][head_dim] contiguous;
 *     either may be NULL to skip it.  Elements outside the token range are not written.
 * Asynchronous on cuda_stream; reads the cache only.
 */
int kvq_dequantize(const kvq_config* cfg, const kvq_cache* cache,
                   void* k_out, void* v_out, int32_t t_begin, int32_t t_end, void* cuda_stream);

/*
 * kvq_decode_attention for callers that cannot provide scratch memory.  (The paper has no
 * counterpart to this call; it exists for integration reasons only.)
 *
 * Some users of this library are not allowed to allocate device memory around a decode step:
 * a serving engine that hands all free HBM to its own arena at start-up and treats any allocator
 * call inside the token loop as a bug (cudaMalloc synchronises the whole device and fails once
 * memory is fully reserved), or a plug-in that is given only input and output pointers by its
 * host framework and has no allocator to ask.  For them this entry point takes the same inputs and
 * outputs as kvq_decode_attention but no workspace: the split partial results go to a buffer of
 * KVQ_STATIC_SCRATCH_BYTES that is part of the library image itself.  The call performs no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Consequences the caller has to know:
 *  - every GPU that loads libkvq.so holds those KVQ_STATIC_SCRATCH_BYTES until the process exits;
 *  - a configuration whose kvq_workspace_bytes() exceeds KVQ_STATIC_SCRATCH_BYTES is rejected with
 *    KVQ_ERR_STATIC_SCRATCH before anything is launched (use kvq_decode_attention then);
 *  - the first call on each device looks up the buffer's device address (a host-side query, made
 *    with that device current); make that first call before starting any stream capture;
 *  - all calls on a device share the one buffer, and it keeps whatever the previous call left in it.
 *    Nothing in it has to start at zero (each slot is written before it is read within a call), so
 *    back-to-back calls on one stream are fine, but two calls that may overlap on the GPU (different
 *    streams without an ordering between them) race on it and give wrong results.
 * Results are identical to kvq_decode_attention's.
 */
#define KVQ_STATIC_SCRATCH_BYTES (8u << 20)
int kvq_decode_attention_static(const kvq_config* cfg, const kvq_cache* cache,
                                const void* q, void* out, int32_t out_dtype, float softmax_scale,
                                void* cuda_stream);

/*
 * Reconstruction-error analysis of the quantizer (Sec. 4.1, experiment (i); Table 1 reports
 * MSE(A, A^) = ||A - A^||_F^2 / number of entries, App. B.4, of the dequantized K and V caches per head).
 * One pass over n_tokens tokens of K and V quantizes every token row in registers exactly as
 * kvq_quantize_append would (kb, vb, gk, gv of cfg; token-wise groups: k_axis must be 0), reconstructs
 * x^ = fmaf(code, scale, zero) and ADDS, per (batch, kv-head), to
 *   sums[b][h][0..3] = (sum k^2, sum (k - k^)^2, sum v^2, sum (v - v^)^2)      (device, double, 8-byte aligned).
 * The caller zeroes sums before the first call; several calls (chunks of tokens, layers) accumulate.  The MSE
 * of a head is sums[..][1] / (n_tokens * head_dim), its squared Frobenius norm sums[..][0].  k, v, strides: as
 * in kvq_quantize_append.  Writes nothing but sums.  Asynchronous on cuda_stream.
 */
int kvq_quant_error(const kvq_config* cfg, const void* k, const void* v,
                    int64_t stride_b, int64_t stride_h, int64_t stride_t, int32_t n_tokens,
                    double* sums, void* cuda_stream);

/*
 * Host only.  The difference of bit widths that equalises the Frobenius error bounds of App. B.4,
 * ||E||_F <~ sqrt(L d) / 2^b ||A||_F for keys and values:  b_K - b_V = log2(||K||_F / ||V||_F)
 * = 0.5 log2(sum_k2 / sum_v2).  (App. B.4 prints the ratio inverted, which contradicts its own conclusion
 * b_K > b_V; this is the form its preceding line implies.)  Both sums must be positive.
 */
int kvq_bit_balance(double sum_k2, double sum_v2, double* bk_minus_bv);

/* Synchronises cuda_stream, reads *cache->status and returns KVQ_OK, KVQ_ERR_CAPACITY,
 * KVQ_ERR_DEVICE_TIMEOUT or KVQ_ERR_CUDA_LAUNCH (a CUDA error surfaced by the sync). */
int kvq_check_status(const kvq_cache* cache, void* cuda_stream);

/* Static description of a return code. */
const char* kvq_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* KVQ_H_ */
