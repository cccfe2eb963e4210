// Internal entry points shared between spans_to_index.cu, decode_attn.cu and decode_step.cu.
#pragma once
#include "ssa_common.cuh"

namespace ssa {

// Defined in spans_to_index.cu: the index expansion of a decode step fused with the fetch of the step's inputs
// from page-locked host memory (used by ssa_decode_step).
int32_t fetch_and_index(const int32_t* host_span_offsets, const int32_t* host_spans, const int32_t* host_ctx_lens,
                        int32_t B, int32_t* index, int32_t index_stride, int32_t* counts, uint32_t* dev_status,
                        void* dst, const void* src, size_t bytes, cudaStream_t stream);

// Defined in spans_to_index.cu: ssa_spans_to_index with a list capacity below the row pitch and a bound on the
// spans taken per request (used where the span-list attention call falls back to an index list).
int32_t spans_to_index_capped(const int32_t* span_offsets, const int32_t* spans, const int32_t* ctx_lens, int32_t B,
                              int32_t* index, int32_t index_stride, int32_t capacity, int32_t span_cap,
                              int32_t* counts, uint32_t* dev_status, cudaStream_t stream);

// Defined in decode_attn.cu, for ssa_decode_step: the most spans per request the span-list attention kernel
// merges on chip, and whether a step is better served by that one kernel than by index + attention launches.
int32_t one_kernel_span_limit();
bool one_kernel_step_pays(const ssa_attn_desc* desc, int32_t max_selected, int32_t max_spans, size_t workspace_bytes);

// Defined in decode_attn.cu, for ssa_decode_step with copies done by kernels: the attention call that fetches the
// query rows itself (see there), and whether a step qualifies.
int32_t decode_attn_sparse_host_queries(const ssa_attn_desc* desc, void* q, const void* q_host, const void* k_cache,
                                        const void* v_cache, const int32_t* ctx_lens, const int32_t* index,
                                        int32_t index_stride, const int32_t* counts, int32_t max_selected, void* out,
                                        float* lse, void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                        void* stream);
bool host_queries_pay(const ssa_attn_desc* desc, int32_t max_selected);

}  // namespace ssa
