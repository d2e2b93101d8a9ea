// Internal launch interface between the C-ABI layer (kvq_host.cu) and the kernels.
#pragma once

#include "kvq_common.cuh"

namespace kvq {

int launch_quantize_append(const Geom& g, const CachePtrs& c, const void* k_new, const void* v_new,
                           int64_t sb, int64_t sh, int64_t st, int t_new, cudaStream_t stream);

int launch_dequantize(const Geom& g, const CachePtrs& c, void* k_out, void* v_out, int t_begin, int t_end,
                      cudaStream_t stream);

int launch_quant_error(const Geom& g, const void* k, const void* v, int64_t sb, int64_t sh, int64_t st, int n_tokens,
                       double* sums, cudaStream_t stream);

// Number of sequence splits the decode kernels use for this geometry (also sizes the workspace).
int decode_num_splits(const Geom& g);
size_t decode_workspace_bytes(const Geom& g);
// Test hooks of a decode launch (all zero / -1 in the product path).
struct DecodeDebug {
  bool force_generic = false;    // run the plain-ALU kernel whatever the configuration
  int fast_impl = 0;             // fast path: 0 = the library's choice, 1 = the warp-level MMA kernel, 2 = the tcgen05 kernel
  uint32_t wait_us = 0;          // limit of every device-side wait in microseconds (0: the default, 2 s)
  long long skip_page = -1;      // flat page index whose copy is never issued (-1: none)
};
int launch_decode_attention(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype,
                            float softmax_scale, void* workspace, cudaStream_t stream,
                            const DecodeDebug& dbg = DecodeDebug{});

}  // namespace kvq

namespace kvq {
// kernels behind launch_decode_attention
int launch_decode_generic(const Geom& g, const CachePtrs& c, const void* q, float scale_log2e, float* ws,
                          int n_split, cudaStream_t stream);
int launch_merge(const Geom& g, const float* ws, void* out, int out_dtype, int n_split, cudaStream_t stream);
}  // namespace kvq

namespace kvq {
// fast (tensor-core) decode path: flat split over the grid
bool decode_mma_supported(const Geom& g);
size_t flat_workspace_bytes(const Geom& g);
// attention over the residual window's tokens: one partial per stream in slot s_cap - 1 of the flat workspace
int launch_decode_window(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype,
                         float scale_log2e, float* ws, int s_cap, cudaStream_t stream);
int launch_decode_mma(const Geom& g, const CachePtrs& c, const void* q, void* out, int out_dtype,
                      float scale_log2e, float* ws, const DecodeDebug& dbg, cudaStream_t stream);
// tcgen05 / tensor-memory variant of the fast path (same split, workspace and merge)
bool decode_tc_supported(const Geom& g, const CachePtrs& c);
int launch_decode_tc(const Geom& g, const CachePtrs& c, const void* q, float scale_log2e, float* ws, int s_cap,
                     void* out, int out_dtype, unsigned long long call_id, unsigned long long wait_ns, long long skip_x,
                     cudaStream_t stream);
}  // namespace kvq
