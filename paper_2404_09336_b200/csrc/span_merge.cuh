// A request's span list turned, inside one thread block, into the sorted and
// merged form from which the k-th attended position follows by arithmetic:
// disjoint runs in ascending order, each with the offset of its first
// position in the request's (virtual) index list.  This is what
// ssa_spans_to_index materialises as a list in global memory; the decode
// kernel that takes span lists directly (ssa_decode_attn_spans) keeps it in
// shared memory instead and never reads or writes an index list.
//
// The attended set is a per-position property (the union of the spans), so
// only the starts have to be ordered: walking the spans by ascending start
// with the running maximum of the ends seen so far trims every span to the
// part that no earlier span covers, whatever the order among equal starts.
#pragma once
#include "ssa_common.cuh"

namespace ssa {

constexpr int kDirectSpans = 128;           // most spans of one request the block-level merge takes
constexpr int32_t kNoSpan = 0x7fffffff;     // start of an empty span: sorts behind every real one

struct __align__(16) SpanRuns {
  int32_t start[kDirectSpans];              // sorted starts; after the scan: first position of run i not yet covered
  int32_t end[kDirectSpans];
  int32_t tmp_start[kDirectSpans];          // unsorted copy (only used above 32 spans; read four at a time)
  int32_t tmp_end[kDirectSpans];
  int32_t offs[kDirectSpans + 1];           // positions before run i; offs[P] = all positions
  int32_t P;                                // runs held (a multiple of 32)
  uint32_t flags;
};

// Clamp a span to [0, n); empty, reversed or out-of-range spans become (kNoSpan, kNoSpan).
__device__ __forceinline__ int2 clamp_span(int2 se, int n, uint32_t& flags) {
  if (se.x < 0 || se.x > se.y) flags |= SSA_DEV_BAD_SPAN;
  if (se.y > n) flags |= SSA_DEV_CLIPPED;
  const int s = max(se.x, 0), e = min(se.y, n);
  return e > s ? make_int2(s, e) : make_int2(kNoSpan, kNoSpan);
}

// Called by every thread of a block of kBlockThreads >= kDirectSpans threads.
// spans: (start, end) pairs of the request (first .. first + S); at most `cap`
// <= kDirectSpans are taken (SSA_DEV_TOO_MANY_SPANS beyond).  Returns the
// number of attended positions; r.flags then holds the status bits of the
// list.  Contains block barriers.
template <int kBlockThreads>
__device__ __forceinline__ int merge_spans_block(SpanRuns& r, const int2* __restrict__ spans, int S, int cap, int n) {
  static_assert(kBlockThreads >= kDirectSpans, "one thread per span");
  const int tid = threadIdx.x, lane = tid & 31;
  uint32_t flags = 0;
  if (S < 0) S = 0;
  if (S > cap) { S = cap; if (tid == 0) flags |= SSA_DEV_TOO_MANY_SPANS; }
  const int P = S <= 32 ? 32 : (S + 31) & ~31;
  if (tid == 0) { r.flags = 0; r.P = P; }
  if (P == 32) {
    // the usual case: one warp ranks the starts with shuffles
    if (tid < 32) {
      int2 se = make_int2(kNoSpan, kNoSpan);
      if (lane < S) se = clamp_span(spans[lane], n, flags);
      int rank = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const int sj = __shfl_sync(0xffffffffu, se.x, j);
        rank += (sj < se.x || (sj == se.x && j < lane)) ? 1 : 0;
      }
      r.start[rank] = se.x;
      r.end[rank] = se.y;
    }
    __syncthreads();                          // also publishes r.flags = 0
  } else {
    int2 se = make_int2(kNoSpan, kNoSpan);
    if (tid < P) {
      if (tid < S) se = clamp_span(spans[tid], n, flags);
      r.tmp_start[tid] = se.x;
      r.tmp_end[tid] = se.y;
    }
    __syncthreads();
    if (tid < P) {
      int rank = 0;
      for (int j = 0; j < P; j += 4) {        // every thread reads the same words: broadcasts
        const int4 s4 = *reinterpret_cast<const int4*>(&r.tmp_start[j]);
        rank += (s4.x < se.x || (s4.x == se.x && j < tid)) ? 1 : 0;
        rank += (s4.y < se.x || (s4.y == se.x && j + 1 < tid)) ? 1 : 0;
        rank += (s4.z < se.x || (s4.z == se.x && j + 2 < tid)) ? 1 : 0;
        rank += (s4.w < se.x || (s4.w == se.x && j + 3 < tid)) ? 1 : 0;
      }
      r.start[rank] = se.x;
      r.end[rank] = se.y;
    }
    __syncthreads();
  }
  if (flags) atomicOr(&r.flags, flags);
  // trim against the running maximum end and prefix-sum the lengths, 32 runs at a time
  if (tid < 32) {
    int run_max = 0, run_sum = 0;
    for (int base = 0; base < P; base += 32) {
      const int s0 = r.start[base + lane];
      const bool live = s0 != kNoSpan;
      const int s = live ? s0 : 0, e = live ? r.end[base + lane] : 0;
      int mx = e;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, mx, d);
        if (lane >= d) mx = max(mx, o);
      }
      int prev = __shfl_up_sync(0xffffffffu, mx, 1);
      prev = lane == 0 ? run_max : max(prev, run_max);
      const int ns = max(s, prev);
      const int len = live ? max(e - ns, 0) : 0;
      int sum = len;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, sum, d);
        if (lane >= d) sum += o;
      }
      r.start[base + lane] = ns;
      r.offs[base + lane] = run_sum + sum - len;
      run_max = max(run_max, __shfl_sync(0xffffffffu, mx, 31));
      run_sum += __shfl_sync(0xffffffffu, sum, 31);
    }
    if (lane == 0) r.offs[P] = run_sum;
  }
  __syncthreads();
  return r.offs[P];
}

// The same for up to 32 spans, done by ONE warp for itself: no block barrier and nothing shared with the other
// warps of the block, so a warp can go on to its cache rows as soon as its own lanes are done.  Lane i ends up
// owning run i of the sorted, trimmed list; the runs go to the warp's own `w`.
struct WarpRuns {
  int32_t start[32];                        // first position of run i that no earlier run covers
  int32_t offs[33];                         // positions before run i; offs[32] = all positions
};

// Called by all 32 lanes.  Lane i < S holds span i of the request in `my_span`; S <= P, P a power of two <= 32 (the work grows with P, not with 32:
// a request of the method names a handful of spans).  Returns the number of attended positions and ORs the
// status bits of the list into `flags` (every lane gets the same bits).
__device__ __forceinline__ int merge_spans_warp(WarpRuns& w, int2 my_span, int S, int P, int n, uint32_t& flags) {
  const int lane = threadIdx.x & 31;
  uint32_t f = 0;
  int2 se = make_int2(kNoSpan, kNoSpan);
  if (lane < S) se = clamp_span(my_span, n, f);
  // rank of this lane's span among the starts (ties by lane), then hand every span to the lane of its rank
  int rank = 0;
  for (int j = 0; j < P; ++j) {
    const int sj = __shfl_sync(0xffffffffu, se.x, j);
    rank += (sj < se.x || (sj == se.x && j < lane)) ? 1 : 0;
  }
  if (lane < P) {
    w.start[rank] = se.x;
    w.offs[rank] = se.y;
  }
  __syncwarp();
  const int s0 = lane < P ? w.start[lane] : kNoSpan;
  const bool live = s0 != kNoSpan;
  const int s = live ? s0 : 0, e = live ? w.offs[lane] : 0;
  __syncwarp();
  int mx = e;                               // running maximum of the ends up to and including this run
  for (int d = 1; d < P; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, mx, d);
    if (lane >= d) mx = max(mx, o);
  }
  const int prev = __shfl_up_sync(0xffffffffu, mx, 1);
  const int ns = lane == 0 ? s : max(s, prev);
  const int len = live ? max(e - ns, 0) : 0;
  int sum = len;
  for (int d = 1; d < P; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, sum, d);
    if (lane >= d) sum += o;
  }
  const int total = __shfl_sync(0xffffffffu, sum, P - 1);
  if (lane < P) {
    w.start[lane] = ns;
    w.offs[lane] = sum - len;
  }
  if (lane == 0) w.offs[P] = total;
  flags |= __reduce_or_sync(0xffffffffu, f);
  __syncwarp();
  return total;
}

// The k-th attended position (0 <= k < offs[P]) among P runs.
__device__ __forceinline__ int span_position(const WarpRuns& w, int P, int k) {
  int lo = 0;
  for (int step = P >> 1; step > 0; step >>= 1)
    if (w.offs[lo + step] <= k) lo += step;
  return w.start[lo] + (k - w.offs[lo]);
}

// The k-th attended position (0 <= k < offs[P]): the last run i with offs[i] <= k holds it.
__device__ __forceinline__ int span_position(const SpanRuns& r, int k) {
  int lo = 0, hi = r.P;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (r.offs[mid] <= k) lo = mid; else hi = mid;
  }
  return r.start[lo] + (k - r.offs[lo]);
}

}  // namespace ssa
