// ssa_decode_step: one decode step (optional copy in, span lists -> index
// lists -> span-restricted attention, optional copy out) enqueued by one call.
#include <algorithm>

#include "fetch_index.cuh"

namespace ssa {

// Copy of n16 16-byte words between the device and page-locked host memory the
// device can address.  Every word is requested at once, so the transfer costs
// about one trip over the bus plus its bytes; a copy-engine transfer of the
// same few hundred KB pays several microseconds of set-up on top.
__global__ void __launch_bounds__(256) copy_words_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src,
                                                          size_t n16) {
  grid_dependency_wait();                      // the destination may still be read by the previous kernel
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) dst[i] = src[i];
}

// True when `p` is page-locked host memory that kernels can address under the same pointer.
static bool device_addressable_host(const void* p) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  return a.type == cudaMemoryTypeHost && a.devicePointer == p;
}

static int32_t copy_by_kernel(void* dst, const void* src, size_t bytes, cudaStream_t st) {
  const size_t n16 = bytes / 16;
  const unsigned blocks = (unsigned)std::min<size_t>((n16 + 255) / 256, (size_t)sm_count() * 4);
  const cudaError_t err = launch_pdl(copy_words_kernel, dim3(blocks), dim3(256), st, reinterpret_cast<uint4*>(dst),
                                     reinterpret_cast<const uint4*>(src), n16);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  note_launches(1);
  return SSA_OK;
}

static bool copy_aligned(const void* a, const void* b, size_t bytes) {
  return bytes % 16 == 0 && reinterpret_cast<uintptr_t>(a) % 16 == 0 && reinterpret_cast<uintptr_t>(b) % 16 == 0;
}

}  // namespace ssa

extern "C" int32_t ssa_decode_step(const ssa_attn_desc* desc, const ssa_step* s, void* stream) {
  if (!desc || !s) return SSA_ERR_NULL;
  if (s->host_in && (!s->dev_in || s->in_bytes == 0)) return SSA_ERR_NULL;
  if (s->host_out && (!s->dev_out || s->out_bytes == 0)) return SSA_ERR_NULL;
  if (s->flags & ~(uint32_t)(SSA_STEP_COPY_BY_KERNEL | SSA_STEP_ONE_KERNEL | SSA_STEP_TWO_KERNELS))
    return SSA_ERR_UNSUPPORTED;
  if ((s->flags & SSA_STEP_ONE_KERNEL) && (s->flags & SSA_STEP_TWO_KERNELS)) return SSA_ERR_UNSUPPORTED;
  const bool by_kernel = (s->flags & SSA_STEP_COPY_BY_KERNEL) != 0;
  if (by_kernel) {                             // everything is checked before anything is enqueued
    if (s->host_in && !ssa::copy_aligned(s->host_in, s->dev_in, s->in_bytes)) return SSA_ERR_ALIGN;
    if (s->host_out && !ssa::copy_aligned(s->host_out, s->dev_out, s->out_bytes)) return SSA_ERR_ALIGN;
    if (s->host_in && !ssa::device_addressable_host(s->host_in)) return SSA_ERR_UNSUPPORTED;
    if (s->host_out && !ssa::device_addressable_host(s->host_out)) return SSA_ERR_UNSUPPORTED;
  }
  cudaStream_t st = (cudaStream_t)stream;
  int32_t rc;
  // where a pointer into the device arena has its counterpart in the host arena (nullptr: not in the arena)
  auto host_twin = [&](const void* dev_ptr) -> const int32_t* {
    const char* d = static_cast<const char*>(dev_ptr);
    const char* base = static_cast<const char*>(s->dev_in);
    if (!s->host_in || d < base || d >= base + s->in_bytes) return nullptr;
    return reinterpret_cast<const int32_t*>(static_cast<const char*>(s->host_in) + (d - base));
  };
  const int32_t* h_off = by_kernel ? host_twin(s->span_offsets) : nullptr;
  const int32_t* h_spans = by_kernel ? host_twin(s->spans) : nullptr;
  const int32_t* h_ctx = by_kernel ? host_twin(s->ctx_lens) : nullptr;
  const bool fused_fetch = h_off && h_spans && h_ctx && desc->B > 0 && desc->B < 60000;
  bool one_kernel = (s->flags & SSA_STEP_ONE_KERNEL) != 0;
  if (one_kernel) {
    if (s->max_spans <= 0 || s->max_spans > ssa::one_kernel_span_limit()) return SSA_ERR_CAPACITY;
  } else if (!(s->flags & SSA_STEP_TWO_KERNELS) && !fused_fetch) {
    one_kernel = ssa::one_kernel_step_pays(desc, s->max_selected, s->max_spans, s->workspace_bytes);
  }
  if (one_kernel) {
    if (s->host_in) {
      if (by_kernel) {
        rc = ssa::copy_by_kernel(s->dev_in, s->host_in, s->in_bytes, st);
        if (rc != SSA_OK) return rc;
      } else if (cudaMemcpyAsync(s->dev_in, s->host_in, s->in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return SSA_ERR_CUDA;
      }
    }
    rc = ssa_decode_attn_spans(desc, s->q, s->k_cache, s->v_cache, s->ctx_lens, s->span_offsets, s->spans,
                               s->max_spans, s->max_selected, s->out, s->lse, s->index, s->index_stride, s->counts,
                               s->workspace, s->workspace_bytes, s->dev_status, stream);
    if (rc != SSA_OK) return rc;
  } else {
  const void* q_host = nullptr;                // set: the attention kernel fetches the query rows itself
  if (fused_fetch) {
    // The span lists are part of what is fetched: expand them straight from the host arena while the same
    // launch copies the arena in.  Where the query rows are the head or the tail of the arena and every request
    // is served by one thread block per head, that copy leaves them out: each attention block then fetches its
    // own row across the bus while it starts up (and writes the device copy), so the bulk of the input bytes
    // travels during the attention kernel instead of in front of it.
    const char* arena = static_cast<const char*>(s->dev_in);
    const char* q_dev = static_cast<const char*>(s->q);
    const size_t q_bytes = ((size_t)(desc->B - 1) * desc->q_stride_b + (size_t)(desc->H - 1) * desc->q_stride_h +
                            desc->D) * 2;
    size_t skip_head = 0, skip_tail = 0;
    if (host_twin(s->q) && q_bytes % 16 == 0 && q_bytes <= s->in_bytes && ssa::host_queries_pay(desc, s->max_selected)) {
      if (q_dev == arena) skip_head = q_bytes;
      else if (q_dev + q_bytes == arena + s->in_bytes) skip_tail = q_bytes;
    }
    if (skip_head + skip_tail > 0 && skip_head + skip_tail < s->in_bytes)
      q_host = static_cast<const char*>(s->host_in) + (q_dev - arena);
    else
      skip_head = skip_tail = 0;
    rc = ssa::fetch_and_index(h_off, h_spans, h_ctx, desc->B, s->index, s->index_stride, s->counts, s->dev_status,
                              static_cast<char*>(s->dev_in) + skip_head,
                              static_cast<const char*>(s->host_in) + skip_head,
                              s->in_bytes - skip_head - skip_tail, st);
    if (rc != SSA_OK) return rc;
  } else {
    if (s->host_in) {
      if (by_kernel) {
        rc = ssa::copy_by_kernel(s->dev_in, s->host_in, s->in_bytes, st);
        if (rc != SSA_OK) return rc;
      } else if (cudaMemcpyAsync(s->dev_in, s->host_in, s->in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return SSA_ERR_CUDA;
      }
    }
    rc = ssa_spans_to_index(s->span_offsets, s->spans, s->ctx_lens, desc->B, s->index, s->index_stride,
                            s->counts, s->dev_status, stream);
    if (rc != SSA_OK) return rc;
  }
  if (q_host)
    rc = ssa::decode_attn_sparse_host_queries(desc, const_cast<void*>(s->q), q_host, s->k_cache, s->v_cache,
                                              s->ctx_lens, s->index, s->index_stride, s->counts, s->max_selected,
                                              s->out, s->lse, s->workspace, s->workspace_bytes, s->dev_status, stream);
  else
    rc = ssa_decode_attn_sparse(desc, s->q, s->k_cache, s->v_cache, s->ctx_lens, s->index, s->index_stride,
                                s->counts, s->max_selected, s->out, s->lse, s->workspace, s->workspace_bytes,
                                s->dev_status, stream);
  if (rc != SSA_OK) return rc;
  }
  if (s->host_out) {
    if (by_kernel) {
      rc = ssa::copy_by_kernel(const_cast<void*>(s->host_out), s->dev_out, s->out_bytes, st);
      if (rc != SSA_OK) return rc;
    } else if (cudaMemcpyAsync(s->host_out, s->dev_out, s->out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
      return SSA_ERR_CUDA;
    }
  }
  return SSA_OK;
}
