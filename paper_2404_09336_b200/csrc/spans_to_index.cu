// Span list -> sorted duplicate-free KV index list (ssa_spans_to_index).
//
// One thread block per (output slice, request).  The block
//   1. loads the request's spans, clamps them to [0, ctx_len) and packs each
//      non-empty one into a 64-bit key (start << 32 | end);
//   2. sorts the keys: up to 32 spans by rank counting inside one warp
//      (shuffles only), more by a bitonic network in shared memory;
//   3. has one warp walk the sorted spans 32 at a time with two shuffle
//      scans: a running maximum of the span ends seen so far, which trims
//      each span to the part no earlier span covers, and a prefix sum of the
//      trimmed lengths, which gives every span its offset in the output;
//   4. writes its slice of the output: slot k finds its span by binary
//      search over the offsets, so the stores are coalesced and balanced
//      however uneven the spans are.
// Blocks of one request repeat steps 1-3 (a few microseconds) instead of
// communicating.
//
// ssa_refs_to_index runs the same kernel with another step 1: one warp
// resolves the request's references into spans (as ssa_refs_to_spans does) and
// packs them straight into the keys in shared memory, so the span list never
// goes through global memory and the step is one launch instead of two.
#include <algorithm>

#include "fetch_index.cuh"
#include "refs_resolve.cuh"

namespace ssa {

constexpr int kIdxThreads = 128;
constexpr int kMaxSpans = SSA_MAX_SPANS_PER_SEQ;   // power of two
constexpr unsigned long long kEmptyKey = 0xffffffffffffffffull;

// Where the spans of a request come from: a span list in global memory, or the anchor tables.
struct SpanSource {
  const int32_t* span_offsets;
  const int32_t* spans;
  const int32_t* ctx_lens;
  ssa_anchor_tables tables;
};

// kFetch: rows of the grid from first_row on do not expand a request but copy n16 16-byte words from page-locked
// host memory to the device (the step's inputs), while the other rows read their span lists straight from
// that host memory: the fetch of a decode step's inputs and its index expansion overlap in one launch.
struct FetchJob {
  uint4* dst;
  const uint4* src;
  size_t n16;
  int32_t first_row;
};

template <bool kFromRefs, bool kFetch = false>
__global__ void __launch_bounds__(kIdxThreads)
spans_to_index_kernel(const SpanSource src, int32_t* __restrict__ index,
                      int32_t index_stride, int32_t slice, int32_t* __restrict__ counts,
                      uint32_t* __restrict__ dev_status, const FetchJob job,
                      int32_t capacity, int32_t span_cap) {
  // index_stride: distance between the rows of `index`; capacity <= index_stride: most positions a list keeps;
  // span_cap <= kMaxSpans: most spans a request may have
  if (kFetch && (int)blockIdx.y >= job.first_row) {
    grid_dependency_wait();                      // the destination may still be read by the previous kernel
    const size_t n_threads = (size_t)(gridDim.y - job.first_row) * gridDim.x * kIdxThreads;
    size_t i = ((size_t)(blockIdx.y - job.first_row) * gridDim.x + blockIdx.x) * kIdxThreads + threadIdx.x;
    for (; i + n_threads < job.n16; i += 2 * n_threads) {   // two requests in flight per thread
      const uint4 a = job.src[i], c = job.src[i + n_threads];
      job.dst[i] = a;
      job.dst[i + n_threads] = c;
    }
    if (i < job.n16) job.dst[i] = job.src[i];
    return;
  }
  __shared__ unsigned long long keys[kMaxSpans];
  __shared__ int32_t new_start[kMaxSpans];
  __shared__ int32_t offs[kMaxSpans + 1];
  __shared__ uint32_t s_flags;
  __shared__ int s_resolved;
  const int32_t* __restrict__ span_offsets = src.span_offsets;
  const int32_t* __restrict__ spans = src.spans;
  const int32_t* __restrict__ ctx_lens = kFromRefs ? src.tables.ctx_lens : src.ctx_lens;

  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  grid_dependency_wait();      // dependents are released when this grid completes: blocks of a large
                               // attention grid parked on the SMs during this kernel slowed it down
  const int n = max(ctx_lens[b], 0);
  uint32_t flags = 0;
  if (tid == 0) s_flags = 0;

  // clamp a span to the context and pack it; empty spans get the sentinel
  auto pack = [&](int2 se) -> unsigned long long {
    if (se.x < 0 || se.x > se.y) flags |= SSA_DEV_BAD_SPAN;
    if (se.y > n) flags |= SSA_DEV_CLIPPED;
    const int s = max(se.x, 0), e = min(se.y, n);
    return e > s ? ((unsigned long long)(uint32_t)s << 32) | (uint32_t)e : kEmptyKey;
  };

  int first = 0, S;
  if (kFromRefs) {
    // 1 (references): warp 0 resolves them and leaves the packed spans, unsorted, in keys[0, S)
    if (tid < 32) {
      const int resolved = resolve_refs_warp(src.tables, b, tid, flags, [&](int at, int2 span) {
        if (at < kMaxSpans) keys[at] = pack(span);
      });
      if (tid == 0) s_resolved = resolved;
    }
    __syncthreads();
    S = s_resolved;
  } else {
    first = span_offsets[b];
    S = span_offsets[b + 1] - first;
  }
  if (S < 0) S = 0;
  if (S > span_cap) { S = span_cap; flags |= SSA_DEV_TOO_MANY_SPANS; }
  int P = 32;
  while (P < S) P <<= 1;
  __syncthreads();

  auto load_key = [&](int i) -> unsigned long long {
    if (i >= S) return kEmptyKey;
    if (kFromRefs) return keys[i];
    return pack(reinterpret_cast<const int2*>(spans)[first + i]);
  };

  if (P == 32) {
    // 1+2 (up to 32 spans, the usual case): one warp ranks its keys with
    // shuffles, no block barrier needed
    if (tid < 32) {
      const unsigned long long key = load_key(tid);
      if (kFromRefs) __syncwarp();                  // every lane has read its key before any is overwritten
      int rank = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const unsigned long long kj = __shfl_sync(0xffffffffu, key, j);
        rank += (kj < key || (kj == key && j < tid)) ? 1 : 0;
      }
      keys[rank] = key;
      __syncwarp();
    }
  } else {
    // 1. load, clamp, pack (references: the keys are in place, only the padding is missing)
    for (int i = tid; i < P; i += kIdxThreads)
      if (!kFromRefs || i >= S) keys[i] = load_key(i);
    __syncthreads();
    // 2. bitonic sort, ascending by (start, end); empty keys sink to the end
    for (int k = 2; k <= P; k <<= 1) {
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int i = tid; i < P; i += kIdxThreads) {
          const int ixj = i ^ j;
          if (ixj > i) {
            const unsigned long long a = keys[i], c = keys[ixj];
            const bool up = (i & k) == 0;
            if ((a > c) == up) { keys[i] = c; keys[ixj] = a; }
          }
        }
        __syncthreads();
      }
    }
  }

  // 3. trim against the running maximum end and prefix-sum the lengths
  if (tid < 32) {
    int run_max = 0, run_sum = 0;
    for (int base = 0; base < P; base += 32) {
      const unsigned long long key = keys[base + tid];
      const bool live = key != kEmptyKey;
      const int s = live ? (int)(key >> 32) : 0;
      const int e = live ? (int)(uint32_t)key : 0;
      int mx = e;                                   // inclusive max-scan of ends
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, mx, d);
        if (tid >= d) mx = max(mx, o);
      }
      int prev = __shfl_up_sync(0xffffffffu, mx, 1);
      prev = (tid == 0) ? run_max : max(prev, run_max);
      const int ns = max(s, prev);
      const int len = live ? max(e - ns, 0) : 0;
      int sum = len;                                // inclusive sum-scan of lengths
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, sum, d);
        if (tid >= d) sum += o;
      }
      new_start[base + tid] = ns;
      offs[base + tid] = run_sum + sum - len;
      run_max = max(run_max, __shfl_sync(0xffffffffu, mx, 31));
      run_sum += __shfl_sync(0xffffffffu, sum, 31);
    }
    if (tid == 0) offs[P] = run_sum;
  }
  if (flags) atomicOr(&s_flags, flags);
  __syncthreads();

  const int total = offs[P];
  const int c = min(total, capacity);
  if (blockIdx.x == 0 && tid == 0) {
    counts[b] = c;
    uint32_t f = s_flags;
    if (total > capacity) f |= SSA_DEV_OVERFLOW;
    if (f && dev_status) atomicOr(dev_status, f);
  }

  // 4. write this block's slice of the list
  const int k_end = min(c, (int)(blockIdx.x + 1) * slice);
  int32_t* row = index + (size_t)b * index_stride;
  for (int k = blockIdx.x * slice + tid; k < k_end; k += kIdxThreads) {
    int lo = 0, hi = P;                             // last i with offs[i] <= k
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (offs[mid] <= k) lo = mid; else hi = mid;
    }
    row[k] = new_start[lo] + (k - offs[lo]);
  }
}

// ssa_spans_to_index with the span lists read from page-locked host memory (host_* are host addresses the
// device can use), fused with the copy of `bytes` bytes from src (the same kind of memory) to dst (device).
int32_t fetch_and_index(const int32_t* host_span_offsets, const int32_t* host_spans, const int32_t* host_ctx_lens,
                        int32_t B, int32_t* index, int32_t index_stride, int32_t* counts, uint32_t* dev_status,
                        void* dst, const void* src, size_t bytes, cudaStream_t stream) {
  if (!host_span_offsets || !host_spans || !host_ctx_lens || !index || !counts || !dst || !src) return SSA_ERR_NULL;
  if (B <= 0 || index_stride <= 0) return SSA_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(host_spans) % 8 != 0 || bytes % 16 != 0 ||
      reinterpret_cast<uintptr_t>(dst) % 16 != 0 || reinterpret_cast<uintptr_t>(src) % 16 != 0)
    return SSA_ERR_ALIGN;
  int slices = (index_stride + 511) / 512;
  if (slices > 32) slices = 32;
  const int32_t slice = (index_stride + slices - 1) / slices;
  const size_t n16 = bytes / 16;
  const size_t per_row = (size_t)slices * kIdxThreads * 2;            // two words per thread
  const int copy_rows = (int)std::min<size_t>((n16 + per_row - 1) / per_row, (size_t)sm_count() * 8);
  if (B + copy_rows > 65535) return SSA_ERR_SHAPE;
  SpanSource s = {};
  s.span_offsets = host_span_offsets; s.spans = host_spans; s.ctx_lens = host_ctx_lens;
  FetchJob job = {reinterpret_cast<uint4*>(dst), reinterpret_cast<const uint4*>(src), n16, B};
  dim3 grid((unsigned)slices, (unsigned)(B + std::max(copy_rows, 1)));
  const cudaError_t err = launch_pdl(spans_to_index_kernel<false, true>, grid, dim3(kIdxThreads), stream, s,
                                     index, index_stride, slice, counts, dev_status, job, index_stride, kMaxSpans);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  note_launches(1);
  return SSA_OK;
}

// ssa_spans_to_index with two more bounds: a list keeps at most `capacity` <= index_stride positions and a
// request at most `span_cap` <= SSA_MAX_SPANS_PER_SEQ spans.
int32_t spans_to_index_capped(const int32_t* span_offsets, const int32_t* spans, const int32_t* ctx_lens, int32_t B,
                              int32_t* index, int32_t index_stride, int32_t capacity, int32_t span_cap,
                              int32_t* counts, uint32_t* dev_status, cudaStream_t stream) {
  if (!span_offsets || !spans || !ctx_lens || !index || !counts) return SSA_ERR_NULL;
  if (B <= 0 || B > 65535 || index_stride <= 0) return SSA_ERR_SHAPE;
  if (capacity <= 0 || capacity > index_stride || span_cap <= 0 || span_cap > kMaxSpans) return SSA_ERR_CAPACITY;
  if (reinterpret_cast<uintptr_t>(spans) % 8 != 0) return SSA_ERR_ALIGN;
  int slices = (capacity + 511) / 512;               // blocks per request: 512 entries each, at most 32
  if (slices > 32) slices = 32;
  const int32_t slice = (capacity + slices - 1) / slices;
  dim3 grid((unsigned)slices, (unsigned)B);
  SpanSource src = {};
  src.span_offsets = span_offsets; src.spans = spans; src.ctx_lens = ctx_lens;
  const cudaError_t err = launch_pdl(spans_to_index_kernel<false>, grid, dim3(kIdxThreads), stream, src, index,
                                     index_stride, slice, counts, dev_status, FetchJob{}, capacity, span_cap);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  note_launches(1);
  return SSA_OK;
}

}  // namespace ssa

extern "C" int32_t ssa_spans_to_index(const int32_t* span_offsets, const int32_t* spans,
                                      const int32_t* ctx_lens, int32_t B, int32_t* index,
                                      int32_t index_stride, int32_t* counts,
                                      uint32_t* dev_status, void* stream) {
  return ssa::spans_to_index_capped(span_offsets, spans, ctx_lens, B, index, index_stride, index_stride,
                                    ssa::kMaxSpans, counts, dev_status, (cudaStream_t)stream);
}

extern "C" int32_t ssa_refs_to_index(const ssa_anchor_tables* tables, int32_t B, int32_t* index,
                                     int32_t index_stride, int32_t* counts, uint32_t* dev_status,
                                     void* stream) {
  if (!index || !counts) return SSA_ERR_NULL;
  const int32_t rc = ssa::check_anchor_tables(tables);
  if (rc != SSA_OK) return rc;
  if (B <= 0 || B > 65535 || index_stride <= 0) return SSA_ERR_SHAPE;
  int slices = (index_stride + 511) / 512;
  if (slices > 32) slices = 32;
  const int32_t slice = (index_stride + slices - 1) / slices;
  dim3 grid((unsigned)slices, (unsigned)B);
  ssa::SpanSource src = {};
  src.tables = *tables;
  const cudaError_t err = ssa::launch_pdl(ssa::spans_to_index_kernel<true>, grid, dim3(ssa::kIdxThreads),
                                          (cudaStream_t)stream, src, index, index_stride, slice, counts,
                                          dev_status, ssa::FetchJob{}, index_stride, ssa::kMaxSpans);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  ssa::note_launches(1);
  return SSA_OK;
}
