// Internal entry points defined in spans_to_index.cu and used by decode_step.cu and decode_attn.cu.
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

}  // namespace ssa
