/*
 * Test hooks of libkvq.so.  Not part of the product API: they exist so that the test-suite can reach code
 * paths that a healthy run never takes.  Same argument conventions as kvq.h.  (The paper has no counterpart.)
 */
#ifndef KVQ_DEBUG_H_
#define KVQ_DEBUG_H_

#include "kvq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* kvq_decode_attention, but always through the plain-ALU kernel (the second implementation that the fast
 * tensor-core path is cross-checked against), whatever the configuration. */
int kvq_debug_decode_generic(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                             int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                             void* cuda_stream);

/* kvq_decode_attention_rows through a chosen implementation of the fast path: impl 0 = the library's own
 * choice, 1 = the warp-level integer-MMA kernel, 2 = the tcgen05 / tensor-memory kernel
 * (KVQ_ERR_UNSUPPORTED where that kernel does not serve the configuration).  Lets the tests hold both
 * kernels against the oracle on the same cache and the benchmark time them side by side. */
int kvq_debug_decode_impl(const kvq_config* cfg, const kvq_cache* cache, const void* q, int32_t n_rows, void* out,
                          int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                          int32_t impl, void* cuda_stream);

/* kvq_decode_attention on the fast path with every device-side wait limited to wait_us microseconds
 * (1 .. 100000) and the copy of flat page number skip_page (counted over all streams in (batch, kv-head, page)
 * order; -1: none) never issued.  The warps that wait for that page give up after wait_us, set
 * KVQ_STATUS_DEVICE_TIMEOUT in the cache's status word, keep their barrier protocol and return: the call
 * never hangs, kvq_check_status then reports KVQ_ERR_DEVICE_TIMEOUT, the output is undefined, and after the
 * caller clears the status word the next call on the same cache works.  Configurations that the fast path
 * does not serve run the generic kernel, which has no such waits. */
int kvq_debug_decode_stall(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                           int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                           int64_t skip_page, uint32_t wait_us, void* cuda_stream);

/* kvq_debug_decode_stall through a chosen kernel of the fast path (impl as in kvq_debug_decode_impl): the
 * tcgen05 kernel's bounded waits, its drain of copies and MMAs in flight and the release of its tensor memory
 * are exercised the same way as the warp-level kernel's. */
int kvq_debug_decode_stall_impl(const kvq_config* cfg, const kvq_cache* cache, const void* q, void* out,
                                int32_t out_dtype, float softmax_scale, void* workspace, size_t workspace_bytes,
                                int64_t skip_page, uint32_t wait_us, int32_t impl, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* KVQ_DEBUG_H_ */
