// Span list -> blocked span encoding (ssa_spans_to_blockmask): per request the
// ascending list of (block index, bitmask) of the blocks that hold a selected
// position.
//
// One thread block per request.  The request's spans are clamped into shared
// memory once; the context is then swept in windows of kWindowBits positions:
// the warps OR the spans, one span per warp at a time, into the window's bitmap
// in shared memory, the words of a block are tested for emptiness, a
// ballot scan numbers the non-empty blocks of the window after those of the
// earlier windows, and they are written out.
#include "ssa_common.cuh"

namespace ssa {

constexpr int kBmThreads = 256;
constexpr int kWindowBits = kBmThreads * 32;           // positions per sweep window
constexpr int kBmMaxSpans = SSA_MAX_SPANS_PER_SEQ;

__global__ void __launch_bounds__(kBmThreads)
spans_to_blockmask_kernel(const int32_t* __restrict__ span_offsets, const int32_t* __restrict__ spans,
                          const int32_t* __restrict__ ctx_lens, int32_t block_size,
                          int32_t* __restrict__ block_idx, uint32_t* __restrict__ block_mask,
                          int32_t block_stride, int32_t* __restrict__ block_counts,
                          uint32_t* __restrict__ dev_status) {
  __shared__ int2 s_span[kBmMaxSpans];
  __shared__ uint32_t s_word[kBmThreads];
  __shared__ int s_wcount[kBmThreads / 32];
  __shared__ uint32_t s_flags;

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  grid_dependency_wait();
  const int n = max(ctx_lens[b], 0);
  const int first = span_offsets[b];
  int S = span_offsets[b + 1] - first;
  uint32_t flags = 0;
  if (S < 0) S = 0;
  if (S > kBmMaxSpans) { S = kBmMaxSpans; flags |= SSA_DEV_TOO_MANY_SPANS; }
  if (tid == 0) s_flags = 0;
  for (int i = tid; i < S; i += kBmThreads) {
    const int2 se = reinterpret_cast<const int2*>(spans)[first + i];
    if (se.x < 0 || se.x > se.y) flags |= SSA_DEV_BAD_SPAN;
    if (se.y > n) flags |= SSA_DEV_CLIPPED;
    s_span[i] = make_int2(max(se.x, 0), min(se.y, n));  // empty when end <= start
  }
  __syncthreads();
  if (flags) atomicOr(&s_flags, flags);

  const int wpb = block_size / 32;                      // words per block
  const int blocks_per_window = kBmThreads / wpb;
  int listed = 0;                                       // non-empty blocks found so far
  for (int w0 = 0; w0 < n; w0 += kWindowBits) {
    // word t of the window's bitmap covers positions [w0 + 32 t, w0 + 32 t + 32).  A warp takes a span at a
    // time and its lanes OR the span's overlap into the words it touches, so the work follows the total
    // length of the spans, not spans x words.
    s_word[tid] = 0u;
    __syncthreads();
    for (int i = warp; i < S; i += kBmThreads / 32) {
      const int2 se = s_span[i];
      const int a = max(se.x, w0), e = min(se.y, w0 + kWindowBits);
      if (e <= a) continue;                             // warp-uniform
      const int last = (e - 1 - w0) >> 5;
      for (int w = ((a - w0) >> 5) + lane; w <= last; w += 32) {
        const int lo = w0 + w * 32;
        const int aa = max(a, lo), ee = min(e, lo + 32);
        atomicOr(&s_word[w], (ee - aa == 32) ? 0xffffffffu : (((1u << (ee - aa)) - 1u) << (aa - lo)));
      }
    }
    __syncthreads();
    // thread t < blocks_per_window owns block t of the window
    bool nonempty = false;
    if (tid < blocks_per_window)
      for (int k = 0; k < wpb; ++k) nonempty |= s_word[tid * wpb + k] != 0;
    const uint32_t ballot = __ballot_sync(0xffffffffu, nonempty);
    if (lane == 0) s_wcount[warp] = __popc(ballot);
    __syncthreads();
    int slot = listed + __popc(ballot & ((1u << lane) - 1u));
    int total = 0;
    for (int k = 0; k < kBmThreads / 32; ++k) {
      if (k < warp) slot += s_wcount[k];
      total += s_wcount[k];
    }
    if (nonempty && slot < block_stride) {
      const int64_t at = (int64_t)b * block_stride + slot;
      block_idx[at] = w0 / block_size + tid;
      for (int k = 0; k < wpb; ++k) block_mask[at * wpb + k] = s_word[tid * wpb + k];
    }
    listed += total;
    __syncthreads();                                    // s_word / s_wcount are rewritten next window
  }
  __syncthreads();                                      // every thread's flags are in
  if (tid == 0) {
    block_counts[b] = min(listed, block_stride);
    uint32_t f = s_flags;
    if (listed > block_stride) f |= SSA_DEV_OVERFLOW;
    if (f && dev_status) atomicOr(dev_status, f);
  }
}

}  // namespace ssa

extern "C" int32_t ssa_spans_to_blockmask(const int32_t* span_offsets, const int32_t* spans,
                                          const int32_t* ctx_lens, int32_t B, int32_t block_size,
                                          int32_t* block_idx, uint32_t* block_mask, int32_t block_stride,
                                          int32_t* block_counts, uint32_t* dev_status, void* stream) {
  if (!span_offsets || !spans || !ctx_lens || !block_idx || !block_mask || !block_counts) return SSA_ERR_NULL;
  if (B <= 0 || block_stride <= 0) return SSA_ERR_SHAPE;
  if (block_size != 32 && block_size != 64 && block_size != 128 && block_size != 256) return SSA_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(spans) % 8 != 0) return SSA_ERR_ALIGN;
  const cudaError_t err = ssa::launch_pdl(ssa::spans_to_blockmask_kernel, dim3((unsigned)B), dim3(ssa::kBmThreads),
                                          (cudaStream_t)stream, span_offsets, spans, ctx_lens, block_size,
                                          block_idx, block_mask, block_stride, block_counts, dev_status);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  ssa::note_launches(1);
  return SSA_OK;
}
