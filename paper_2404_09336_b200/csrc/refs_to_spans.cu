// Anchors and references -> span lists (ssa_refs_to_spans).
//
// One warp per request.  The lanes take the request's references 32 at a
// time: each lane resolves one (lo, hi) pair to a first line and a count of
// lines, a shuffle prefix sum turns the counts into output offsets, and the
// lane writes its spans.  Slots past the last span are filled with (0, 0).
#include "ssa_common.cuh"

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
  const int l0 = t.line_offsets[b], n_lines = max(t.line_offsets[b + 1] - l0, 0);
  const int a0 = t.anchor_offsets[b], n_anchors = max(t.anchor_offsets[b + 1] - a0, 0);
  const int r0 = t.ref_offsets[b], n_refs = max(t.ref_offsets[b + 1] - r0, 0);
  const int2* lines = reinterpret_cast<const int2*>(t.lines) + l0;
  const int2* refs = reinterpret_cast<const int2*>(t.refs) + r0;
  uint32_t flags = 0;
  if (lane == 0) {
    span_offsets_out[b] = b * span_stride;
    row[0] = make_int2(0, t.prefix_len[b]);
    row[1] = make_int2(t.line_start[b], t.ctx_lens[b]);
  }
  int written = 2;                                      // spans placed so far (may exceed the row: overflow)
  for (int base = 0; base < n_refs; base += 32) {
    // this lane's reference: anchors [first, first + count) or one earlier line
    int first = 0, count = 0;
    bool by_anchor = false;
    if (base + lane < n_refs) {
      const int2 ref = refs[base + lane];
      if (ref.x == ref.y && ref.x < 0) {
        if (n_lines + ref.x >= 0) { first = n_lines + ref.x; count = 1; }
        else flags |= SSA_DEV_BAD_REF;
      } else if (ref.x >= 0 && ref.x <= ref.y) {
        first = ref.x;
        count = ref.y - ref.x + 1;
        by_anchor = true;
      } else {
        flags |= SSA_DEV_BAD_REF;
      }
    }
    // anchors that do not resolve are dropped, so count what each lane really emits
    int emit = 0;
    if (by_anchor) {
      for (int a = first; a < first + count; ++a) {
        const int li = a < n_anchors ? t.anchor_line[a0 + a] : -1;
        if (li >= 0 && li < n_lines) ++emit; else flags |= SSA_DEV_BAD_REF;
      }
    } else {
      emit = count;
    }
    int incl = emit;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    int at = written + incl - emit;
    if (by_anchor) {
      for (int a = first; a < first + count; ++a) {
        const int li = a < n_anchors ? t.anchor_line[a0 + a] : -1;
        if (li >= 0 && li < n_lines) {
          if (at < span_stride) row[at] = lines[li];
          ++at;
        }
      }
    } else if (count == 1) {
      if (at < span_stride) row[at] = lines[first];
    }
    written += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (written > span_stride) flags |= SSA_DEV_OVERFLOW;
  for (int i = written + lane; i < span_stride; i += 32) row[i] = make_int2(0, 0);
  if (flags && dev_status) atomicOr(dev_status, flags);
}

}  // namespace ssa

extern "C" int32_t ssa_refs_to_spans(const ssa_anchor_tables* t, int32_t B, int32_t* span_offsets_out,
                                     int32_t* spans_out, int32_t span_stride, uint32_t* dev_status, void* stream) {
  if (!t || !span_offsets_out || !spans_out) return SSA_ERR_NULL;
  if (!t->line_offsets || !t->lines || !t->anchor_offsets || !t->anchor_line || !t->ref_offsets || !t->refs ||
      !t->prefix_len || !t->line_start || !t->ctx_lens)
    return SSA_ERR_NULL;
  if (B <= 0 || span_stride < 2 || (long long)B * span_stride > 0x7fffffffll) return SSA_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(t->lines) % 8 || reinterpret_cast<uintptr_t>(t->refs) % 8 ||
      reinterpret_cast<uintptr_t>(spans_out) % 8)
    return SSA_ERR_ALIGN;
  const unsigned blocks = (unsigned)((B + ssa::kRefWarps - 1) / ssa::kRefWarps);
  const cudaError_t err = ssa::launch_pdl(ssa::refs_to_spans_kernel, dim3(blocks), dim3(ssa::kRefWarps * 32),
                                          (cudaStream_t)stream, *t, B, span_offsets_out, spans_out, span_stride,
                                          dev_status);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  ssa::note_launches(1);
  return SSA_OK;
}
