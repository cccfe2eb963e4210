// Internal entry point shared by spans_to_index.cu (definition) and decode_step.cu (use).
#pragma once
#include "ssa_common.cuh"

namespace ssa {

// Defined in spans_to_index.cu: the index expansion of a decode step fused with the fetch of the step's inputs
// from page-locked host memory (used by ssa_decode_step).
int32_t fetch_and_index(const int32_t* host_span_offsets, const int32_t* host_spans, const int32_t* host_ctx_lens,
                        int32_t B, int32_t* index, int32_t index_stride, int32_t* counts, uint32_t* dev_status,
                        void* dst, const void* src, size_t bytes, cudaStream_t stream);

}  // namespace ssa
