// Anchors and references -> span lists (ssa_refs_to_spans).
//
// One warp per request.  The lanes take the request's references 32 at a
// time: each lane resolves one (lo, hi) pair to a first line and a count of
// lines, a shuffle prefix sum turns the counts into output offsets, and the
// lane writes its spans.  Slots past the last span are filled with (0, 0).
#include "refs_resolve.cuh"

namespace ssa {

constexpr int kRefWarps = 4;

__global__ void __launch_bounds__(kRefWarps * 32)
refs_to_spans_kernel(const ssa_anchor_tables t, int32_t B, int32_t* __restrict__ span_offsets_out,
                     int32_t* __restrict__ spans_out, int32_t span_stride, uint32_t* __restrict__ dev_status) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * kRefWarps + (threadIdx.x >> 5);
  grid_dependency_wait();
  if (b == 0 && lane == 0) span_offsets_out[B] = B * span_stride;
  if (b >= B) return;
  int2* row = reinterpret_cast<int2*>(spans_out) + (int64_t)b * span_stride;
  uint32_t flags = 0;
  if (lane == 0) span_offsets_out[b] = b * span_stride;
  // spans beyond the row are counted, not stored (overflow)
  const int written = resolve_refs_warp(t, b, lane, flags, [&](int at, int2 span) {
    if (at < span_stride) row[at] = span;
  });
  if (written > span_stride) flags |= SSA_DEV_OVERFLOW;
  for (int i = written + lane; i < span_stride; i += 32) row[i] = make_int2(0, 0);
  if (flags && dev_status) atomicOr(dev_status, flags);
}

}  // namespace ssa

extern "C" int32_t ssa_refs_to_spans(const ssa_anchor_tables* t, int32_t B, int32_t* span_offsets_out,
                                     int32_t* spans_out, int32_t span_stride, uint32_t* dev_status, void* stream) {
  if (!span_offsets_out || !spans_out) return SSA_ERR_NULL;
  const int32_t rc = ssa::check_anchor_tables(t);
  if (rc != SSA_OK) return rc;
  if (B <= 0 || span_stride < 2 || (long long)B * span_stride > 0x7fffffffll) return SSA_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(spans_out) % 8) return SSA_ERR_ALIGN;
  const unsigned blocks = (unsigned)((B + ssa::kRefWarps - 1) / ssa::kRefWarps);
  const cudaError_t err = ssa::launch_pdl(ssa::refs_to_spans_kernel, dim3(blocks), dim3(ssa::kRefWarps * 32),
                                          (cudaStream_t)stream, *t, B, span_offsets_out, spans_out, span_stride,
                                          dev_status);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  ssa::note_launches(1);
  return SSA_OK;
}
