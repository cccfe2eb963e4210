// ssa_decode_step: one decode step (optional copy in, span lists -> index
// lists -> span-restricted attention, optional copy out) enqueued by one call.
#include "ssa_common.cuh"

extern "C" int32_t ssa_decode_step(const ssa_attn_desc* desc, const ssa_step* s, void* stream) {
  if (!desc || !s) return SSA_ERR_NULL;
  if (s->host_in && (!s->dev_in || s->in_bytes == 0)) return SSA_ERR_NULL;
  if (s->host_out && (!s->dev_out || s->out_bytes == 0)) return SSA_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (s->host_in &&
      cudaMemcpyAsync(s->dev_in, s->host_in, s->in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return SSA_ERR_CUDA;
  int32_t rc = ssa_spans_to_index(s->span_offsets, s->spans, s->ctx_lens, desc->B, s->index, s->index_stride,
                                  s->counts, s->dev_status, stream);
  if (rc != SSA_OK) return rc;
  rc = ssa_decode_attn_sparse(desc, s->q, s->k_cache, s->v_cache, s->ctx_lens, s->index, s->index_stride,
                              s->counts, s->max_selected, s->out, s->lse, s->workspace, s->workspace_bytes,
                              s->dev_status, stream);
  if (rc != SSA_OK) return rc;
  if (s->host_out &&
      cudaMemcpyAsync(s->host_out, s->dev_out, s->out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return SSA_ERR_CUDA;
  return SSA_OK;
}
