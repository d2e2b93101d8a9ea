// C-ABI layer of libkvq: argument validation, geometry, dispatch.  No device
// memory is allocated or retained here; all work is queued on the caller's stream.
#include <math.h>
#include <stdlib.h>

#include "kvq_debug.h"
#include "kvq_internal.h"

namespace kvq {

namespace {

bool is_bits(int b) { return b == 1 || b == 2 || b == 3 || b == 4 || b == 6 || b == 8 || b == 16; }
bool is_group(int g) { return g == 32 || g == 64 || g == 128; }

int make_geom(const kvq_config* cfg, Geom* out) {
  if (!cfg) return KVQ_ERR_INVALID_ARG;
  if (cfg->batch <= 0 || cfg->n_kv_heads <= 0 || cfg->n_q_heads <= 0) return KVQ_ERR_INVALID_ARG;
  if (cfg->n_q_heads % cfg->n_kv_heads != 0) return KVQ_ERR_INVALID_ARG;
  if (cfg->capacity_tokens <= 0 || cfg->capacity_tokens % kPageTokens != 0) return KVQ_ERR_INVALID_ARG;
  if (cfg->in_dtype != KVQ_FP16 && cfg->in_dtype != KVQ_BF16) return KVQ_ERR_INVALID_ARG;
  if (cfg->k_axis != 0 && cfg->k_axis != 1) return KVQ_ERR_INVALID_ARG;
  if (!is_bits(cfg->kb) || !is_bits(cfg->vb)) return KVQ_ERR_UNSUPPORTED;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return KVQ_ERR_UNSUPPORTED;
  // 1-bit planes (widths 1 and 3) fill whole bytes only at head_dim 128; plane widths are token-wise only
  if (cfg->head_dim != 128 && (cfg->kb == 1 || cfg->kb == 3 || cfg->vb == 1 || cfg->vb == 3)) return KVQ_ERR_UNSUPPORTED;
  if (cfg->k_axis == 1 && is_plane_width(cfg->kb)) return KVQ_ERR_UNSUPPORTED;
  if (cfg->n_q_heads / cfg->n_kv_heads > kMaxGroupHeads) return KVQ_ERR_UNSUPPORTED;
  if (cfg->kb != 16 && cfg->k_axis == 0 && (!is_group(cfg->gk) || cfg->head_dim % cfg->gk)) return KVQ_ERR_UNSUPPORTED;
  if (cfg->vb != 16 && (!is_group(cfg->gv) || cfg->head_dim % cfg->gv)) return KVQ_ERR_UNSUPPORTED;
  if (cfg->k_axis == 1 && cfg->kb == 16) return KVQ_ERR_UNSUPPORTED;
  if ((int64_t)cfg->batch * cfg->n_kv_heads > 65535) return KVQ_ERR_UNSUPPORTED;
  Geom g;
  g.B = cfg->batch; g.Hq = cfg->n_q_heads; g.Hkv = cfg->n_kv_heads; g.G = g.Hq / g.Hkv; g.D = cfg->head_dim;
  g.kb = cfg->kb; g.vb = cfg->vb;
  g.gk = (cfg->kb == 16 || cfg->k_axis == 1) ? g.D : cfg->gk;
  g.gv = (cfg->vb == 16) ? g.D : cfg->gv;
  g.k_axis = cfg->k_axis; g.in_dtype = cfg->in_dtype;
  g.capacity = cfg->capacity_tokens; g.n_pages = g.capacity / kPageTokens;
  g.k_codes_bytes = kPageTokens * g.D * g.kb / 8;
  g.k_meta_off = g.k_codes_bytes;
  g.k_meta_bytes = (g.kb == 16) ? 0 : (g.k_axis == 1 ? 4 * g.D : kPageTokens * (g.D / g.gk) * 4);
  g.v_codes_off = g.k_meta_off + g.k_meta_bytes;
  g.v_codes_bytes = kPageTokens * g.D * g.vb / 8;
  g.v_meta_off = g.v_codes_off + g.v_codes_bytes;
  g.v_meta_bytes = (g.vb == 16) ? 0 : kPageTokens * (g.D / g.gv) * 4;
  g.page_bytes = g.v_meta_off + g.v_meta_bytes;
  g.rows = 1;
  g.R = cfg->residual_tokens;
  if (g.R != 0 && g.R != 64 && g.R != 128) return KVQ_ERR_UNSUPPORTED;
  if (g.R != 0 && g.k_axis != 0) return KVQ_ERR_UNSUPPORTED;
  *out = g;
  return KVQ_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int make_cache(const Geom& g, const kvq_cache* cache, CachePtrs* out) {
  if (!cache || !cache->pages || !cache->seq_len || !cache->status) return KVQ_ERR_INVALID_ARG;
  if (g.k_axis == 1 && !cache->k_tail) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(cache->pages) || !aligned16(cache->k_tail)) return KVQ_ERR_MISALIGNED;
  out->pages = static_cast<uint8_t*>(cache->pages);
  out->k_tail = static_cast<uint16_t*>(cache->k_tail);
  out->seq_len = cache->seq_len;
  out->status = reinterpret_cast<uint32_t*>(cache->status);
  out->k_signs = cache->k_signs;
  out->kv_win = static_cast<uint16_t*>(cache->kv_win);
  if (g.R != 0 && !cache->kv_win) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(cache->kv_win)) return KVQ_ERR_MISALIGNED;
  if (cache->k_signs && (g.kb == 16 || is_plane_width(g.kb))) return KVQ_ERR_UNSUPPORTED;   // rotation: 2/4/8-bit keys only
  return KVQ_OK;
}

}  // namespace

int decode_num_splits(const Geom& g) {
  // Enough CTAs to fill the GPU a few times over, never more than one page per split.
  const int target_ctas = 148 * 4;
  const int streams = g.B * g.Hkv;
  int s = (target_ctas + streams - 1) / streams;
  if (s > g.n_pages) s = g.n_pages;
  if (s > 64) s = 64;
  if (s < 1) s = 1;
  return s;
}

size_t decode_workspace_bytes(const Geom& g) {
  size_t generic = (size_t)g.B * g.Hq * g.rows * decode_num_splits(g) * (g.D + 2) * sizeof(float);
  size_t flat = flat_workspace_bytes(g);
  return generic > flat ? generic : flat;
}

int launch_decode_attention(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype,
                            float softmax_scale, void* workspace, cudaStream_t stream, const DecodeDebug& dbg) {
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)g.D);
  const float scale_log2e = scale * 1.4426950408889634f;
  float* ws = static_cast<float*>(workspace);
  const bool use_mma = decode_mma_supported(g) && !dbg.force_generic;
  if (g.R != 0 && !use_mma) return KVQ_ERR_UNSUPPORTED;      // only the tensor-core path merges the residual window
  if (use_mma) return launch_decode_mma(g, c, q, out, out_dtype, scale_log2e, ws, dbg, stream);
  const int n_split = decode_num_splits(g);
  int rc = launch_decode_generic(g, c, q, scale_log2e, ws, n_split, stream);
  if (rc != KVQ_OK) return rc;
  return launch_merge(g, ws, out, out_dtype, n_split, stream);
}

}  // namespace kvq

using namespace kvq;

extern "C" {

int kvq_layout_version(void) { return KVQ_LAYOUT_VERSION; }

int kvq_page_bytes(const kvq_config* cfg, size_t* out) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (!out) return KVQ_ERR_INVALID_ARG;
  *out = (size_t)g.page_bytes;
  return KVQ_OK;
}

int kvq_cache_bytes(const kvq_config* cfg, size_t* pages_bytes, size_t* k_tail_bytes) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (pages_bytes) *pages_bytes = (size_t)g.B * g.Hkv * g.n_pages * g.page_bytes;
  if (k_tail_bytes) *k_tail_bytes = g.k_axis == 1 ? (size_t)g.B * g.Hkv * kPageTokens * g.D * 2 : 0;
  return KVQ_OK;
}

int kvq_window_bytes(const kvq_config* cfg, size_t* kv_win_bytes) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (!kv_win_bytes) return KVQ_ERR_INVALID_ARG;
  *kv_win_bytes = (size_t)g.B * g.Hkv * g.R * 2 * g.D * 2;
  return KVQ_OK;
}

int kvq_workspace_bytes(const kvq_config* cfg, size_t* out) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (!out) return KVQ_ERR_INVALID_ARG;
  *out = decode_workspace_bytes(g);
  return KVQ_OK;
}

int kvq_quantize_append(const kvq_config* cfg, const kvq_cache* cache, const void* k_new, const void* v_new,
                        int64_t stride_b, int64_t stride_h, int64_t stride_t, int32_t t_new, void* cuda_stream) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (t_new < 0 || !k_new || !v_new) return KVQ_ERR_INVALID_ARG;
  if (t_new == 0) return KVQ_OK;
  if (t_new > g.capacity) return KVQ_ERR_CAPACITY;
  if (stride_t < g.D || stride_h < 0 || stride_b < 0) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new) || (stride_b % 8) || (stride_h % 8) || (stride_t % 8))
    return KVQ_ERR_MISALIGNED;
  return launch_quantize_append(g, c, k_new, v_new, stride_b, stride_h, stride_t, t_new,
                                static_cast<cudaStream_t>(cuda_stream));
}

int kvq_decode_attention(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                         int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                         void* cuda_stream) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (!q || !out || !workspace) return KVQ_ERR_INVALID_ARG;
  if (out_dtype != KVQ_FP16 && out_dtype != KVQ_BF16 && out_dtype != KVQ_FP32) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return KVQ_ERR_MISALIGNED;
  if (workspace_bytes < decode_workspace_bytes(g)) return KVQ_ERR_WORKSPACE_TOO_SMALL;
  return launch_decode_attention(g, c, q, out, out_dtype, softmax_scale, workspace,
                                 static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------
// Decode without caller scratch: the split partials live in a buffer that is
// part of the library image (one copy per GPU that loads the library).
//
// `g_static_scratch` names a device variable.  In host code that name is only a
// handle for the runtime, not a device address, so it must never be passed to a
// kernel; the device address is looked up once per device below and that
// pointer is what the kernels receive.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[KVQ_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};   // device address per device ordinal, 0 = not looked up yet

// Device address of the built-in scratch on the current device.  The first call on a device
// performs the lookup (cudaGetSymbolAddress with that device current); later calls are a table read.
int static_scratch_ptr(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVQ_ERR_CUDA_LAUNCH;
  void* p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return KVQ_ERR_CUDA_LAUNCH;
    __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);   // idempotent: same value from any thread
  }
  *out = p;
  return KVQ_OK;
}
}  // namespace

int kvq_decode_attention_static(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                                int32_t out_dtype, float softmax_scale, void* cuda_stream) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (!q || !out) return KVQ_ERR_INVALID_ARG;
  if (out_dtype != KVQ_FP16 && out_dtype != KVQ_BF16 && out_dtype != KVQ_FP32) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return KVQ_ERR_MISALIGNED;
  if (decode_workspace_bytes(g) > (size_t)KVQ_STATIC_SCRATCH_BYTES) return KVQ_ERR_STATIC_SCRATCH;
  void* scratch = nullptr;
  rc = static_scratch_ptr(&scratch);
  if (rc != KVQ_OK) return rc;
  return launch_decode_attention(g, c, q, out, out_dtype, softmax_scale, scratch,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int kvq_workspace_bytes_rows(const kvq_config* cfg, int32_t n_rows, size_t* out) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (!out || n_rows < 1) return KVQ_ERR_INVALID_ARG;
  if (n_rows * g.G > kMaxGroupHeads) return KVQ_ERR_UNSUPPORTED;
  g.rows = n_rows;
  *out = decode_workspace_bytes(g);
  return KVQ_OK;
}

int kvq_decode_attention_rows(const kvq_config* cfg, const kvq_cache* cache, const void* q, int32_t n_rows,
                              void* out, int32_t out_dtype, float softmax_scale, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (!q || !out || !workspace || n_rows < 1) return KVQ_ERR_INVALID_ARG;
  if (out_dtype != KVQ_FP16 && out_dtype != KVQ_BF16 && out_dtype != KVQ_FP32) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return KVQ_ERR_MISALIGNED;
  if (n_rows * g.G > kMaxGroupHeads) return KVQ_ERR_UNSUPPORTED;
  g.rows = n_rows;
  if (n_rows > 1 && !decode_mma_supported(g)) return KVQ_ERR_UNSUPPORTED;      // only the fast path serves several rows
  if (workspace_bytes < decode_workspace_bytes(g)) return KVQ_ERR_WORKSPACE_TOO_SMALL;
  return launch_decode_attention(g, c, q, out, out_dtype, softmax_scale, workspace,
                                 static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------
// Test hooks (kvq_debug.h): the same validation and launch path as kvq_decode_attention with one knob turned.
// ---------------------------------------------------------------------------
static int decode_with(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out, int32_t out_dtype,
                       float softmax_scale, void* workspace, size_t workspace_bytes, void* cuda_stream,
                       const DecodeDebug& dbg, int n_rows = 1) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (n_rows * g.G > kMaxGroupHeads) return KVQ_ERR_UNSUPPORTED;
  g.rows = n_rows;
  if (n_rows > 1 && !decode_mma_supported(g)) return KVQ_ERR_UNSUPPORTED;
  if (!q || !out || !workspace) return KVQ_ERR_INVALID_ARG;
  if (out_dtype != KVQ_FP16 && out_dtype != KVQ_BF16 && out_dtype != KVQ_FP32) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(workspace)) return KVQ_ERR_MISALIGNED;
  if (workspace_bytes < decode_workspace_bytes(g)) return KVQ_ERR_WORKSPACE_TOO_SMALL;
  return launch_decode_attention(g, c, q, out, out_dtype, softmax_scale, workspace,
                                 static_cast<cudaStream_t>(cuda_stream), dbg);
}

int kvq_debug_decode_generic(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                             int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                             void* cuda_stream) {
  DecodeDebug dbg;
  dbg.force_generic = true;
  return decode_with(cfg, cache, q, out, out_dtype, softmax_scale, workspace, workspace_bytes, cuda_stream, dbg);
}

int kvq_debug_decode_impl(const kvq_config* cfg, const kvq_cache* cache, const void* q, int32_t n_rows, void* out,
                          int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                          int32_t impl, void* cuda_stream) {
  if (impl < 0 || impl > 2 || n_rows < 1) return KVQ_ERR_INVALID_ARG;
  DecodeDebug dbg;
  dbg.fast_impl = impl;
  return decode_with(cfg, cache, q, out, out_dtype, softmax_scale, workspace, workspace_bytes, cuda_stream, dbg, n_rows);
}

int kvq_debug_decode_stall(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out, int32_t out_dtype,
                           float softmax_scale, void* workspace, size_t workspace_bytes, int64_t skip_page,
                           uint32_t wait_us, void* cuda_stream) {
  if (wait_us == 0 || wait_us > 100000u) return KVQ_ERR_INVALID_ARG;      // the hook never waits longer than 0.1 s
  DecodeDebug dbg;
  dbg.skip_page = skip_page;
  dbg.wait_us = wait_us;
  return decode_with(cfg, cache, q, out, out_dtype, softmax_scale, workspace, workspace_bytes, cuda_stream, dbg);
}

int kvq_debug_decode_stall_impl(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                                int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                                int64_t skip_page, uint32_t wait_us, int32_t impl, void* cuda_stream) {
  if (wait_us == 0 || wait_us > 100000u || impl < 0 || impl > 2) return KVQ_ERR_INVALID_ARG;
  DecodeDebug dbg;
  dbg.skip_page = skip_page;
  dbg.wait_us = wait_us;
  dbg.fast_impl = impl;
  return decode_with(cfg, cache, q, out, out_dtype, softmax_scale, workspace, workspace_bytes, cuda_stream, dbg);
}

int kvq_dequantize(const kvq_config* cfg, const kvq_cache* cache, void* k_out, void* v_out, int32_t t_begin,
                   int32_t t_end, void* cuda_stream) {
  Geom g;
  CachePtrs c;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  rc = make_cache(g, cache, &c);
  if (rc != KVQ_OK) return rc;
  if (t_begin < 0 || t_end < t_begin || t_end > g.capacity) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(k_out) || !aligned16(v_out)) return KVQ_ERR_MISALIGNED;
  if (!k_out && !v_out) return KVQ_OK;
  return launch_dequantize(g, c, k_out, v_out, t_begin, t_end, static_cast<cudaStream_t>(cuda_stream));
}

int kvq_quant_error(const kvq_config* cfg, const void* k, const void* v, int64_t stride_b, int64_t stride_h,
                    int64_t stride_t, int32_t n_tokens, double* sums, void* cuda_stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != KVQ_OK) return rc;
  if (g.k_axis != 0) return KVQ_ERR_UNSUPPORTED;          // token-wise groups only
  if (!k || !v || !sums || n_tokens < 0) return KVQ_ERR_INVALID_ARG;
  if (n_tokens == 0) return KVQ_OK;
  if (stride_t < g.D || stride_h < 0 || stride_b < 0) return KVQ_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || (stride_b % 8) || (stride_h % 8) || (stride_t % 8) ||
      (reinterpret_cast<uintptr_t>(sums) & 7u))
    return KVQ_ERR_MISALIGNED;
  return launch_quant_error(g, k, v, stride_b, stride_h, stride_t, n_tokens, sums, static_cast<cudaStream_t>(cuda_stream));
}

int kvq_bit_balance(double sum_k2, double sum_v2, double* bk_minus_bv) {
  if (!bk_minus_bv || !(sum_k2 > 0.0) || !(sum_v2 > 0.0)) return KVQ_ERR_INVALID_ARG;
  *bk_minus_bv = 0.5 * log2(sum_k2 / sum_v2);
  return KVQ_OK;
}

int kvq_check_status(const kvq_cache* cache, void* cuda_stream) {
  if (!cache || !cache->status) return KVQ_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  uint32_t st = 0;
  if (cudaMemcpyAsync(&st, cache->status, sizeof(st), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return KVQ_ERR_CUDA_LAUNCH;
  if (cudaStreamSynchronize(s) != cudaSuccess) return KVQ_ERR_CUDA_LAUNCH;
  if (st & KVQ_STATUS_DEVICE_TIMEOUT) return KVQ_ERR_DEVICE_TIMEOUT;
  if (st & KVQ_STATUS_CAPACITY) return KVQ_ERR_CAPACITY;
  return KVQ_OK;
}

const char* kvq_strerror(int code) {
  switch (code) {
    case KVQ_OK: return "success";
    case KVQ_ERR_INVALID_ARG: return "invalid argument";
    case KVQ_ERR_UNSUPPORTED: return "unsupported configuration";
    case KVQ_ERR_MISALIGNED: return "pointer or stride not 16-byte aligned";
    case KVQ_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case KVQ_ERR_CAPACITY: return "append exceeds the cache capacity";
    case KVQ_ERR_CUDA_LAUNCH: return "CUDA launch or runtime error";
    case KVQ_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case KVQ_ERR_STATIC_SCRATCH:
      return "this configuration needs more split scratch than the library's built-in 8 MiB buffer; "
             "use kvq_decode_attention with a caller-provided workspace";
    default: return "unknown kvq error";
  }
}

}  // extern "C"
