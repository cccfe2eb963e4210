// Split-KV decode attention over a KV index list (ssa_decode_attn_sparse) or
// over the full context (ssa_decode_attn_dense).
//
// Pass 1 (decode_partial_kernel): grid (chunk, head, request).  A block owns
// `chunk` consecutive entries of the request's index list (dense: `chunk`
// consecutive positions).  A cache row of D 16-bit values is read by a group
// of D/16 lanes, 32 bytes per lane (one 256-bit load where the cache is
// 32-byte aligned, else two 128-bit loads), so a warp covers 32/(D/16) rows
// per load and every 32-byte sector of a selected row is fetched exactly once.
// A warp keeps a tile of kU such loads of K and kU of V in flight, then
// reduces the kU dot products across each lane group with shuffles and folds
// them into a running (max, sum, accumulator) triple - the online form of the
// softmax.  The arithmetic is packed: two fp32 lanes per FMA (fma.rn.f32x2).
// Lane groups never talk to one another until the block ends, where their
// triples are combined through shared memory.  With one chunk per request the
// block normalises and stores the output itself; otherwise it stores the
// unnormalised triple to the workspace and
// Pass 2 (decode_merge_kernel) combines the chunks of one (request, head).
//
// The attended rows of a block come from one of four sources (kMode): every
// position (dense), a slice of the request's index list, a run of entries
// of the request's blocked (block index, bitmask) list, whose set bits the
// block expands into positions in shared memory before reading any row, or
// the request's span list itself, which the block sorts and merges in shared
// memory and turns into positions by arithmetic (no index list anywhere).
#include <algorithm>
#include <atomic>
#include <type_traits>

#include "fetch_index.cuh"
#include "span_merge.cuh"
#include "ssa_common.cuh"

namespace ssa {

#ifndef SSA_WARPS
#define SSA_WARPS 4
#endif
#ifndef SSA_U
#define SSA_U 4
#endif
#ifndef SSA_MIN_BLOCKS
#define SSA_MIN_BLOCKS 4
#endif

constexpr int kWarps = SSA_WARPS;      // warps per block in pass 1
constexpr int kThreads = kWarps * 32;
constexpr int kU = SSA_U;              // 32-byte loads in flight per lane, per tensor
constexpr int kMaxChunk = 512;         // index entries staged per block
constexpr int kIdxPerThread = kMaxChunk / kThreads;
constexpr int kMaskChunk = 512;        // positions a block expands from bitmasks
enum { kDense = 0, kIndex = 1, kBlockMask = 2, kSpans = 3 };

struct DecodeParams {
  const void* q_host;       // kHostQ only: the query rows in page-locked host memory the device addresses; every
                            // block fetches its own row across the bus and leaves a copy at q
  const void* q;
  const void* k;
  const void* v;
  const int32_t* ctx_lens;
  const int32_t* index;     // sparse only
  const int32_t* counts;    // list lengths: index entries or listed blocks (NULL selects the dense count)
  const int32_t* block_idx; // blocked list only
  const uint32_t* block_mask;
  int32_t block_size, block_stride;
  const int32_t* span_offsets;  // span lists only: [B+1]
  const int2* spans;            //   (start, end) pairs
  int32_t span_cap;             //   spans taken per request (<= kDirectSpans)
  int32_t* index_out;           //   optional copy of the positions, [B, index_stride]
  int32_t* counts_out;          //   optional number of positions per request
  int32_t* ws_counts;           //   the same for the second pass (when n_chunks > 1)
  void* out;
  float* lse;
  float* ws_acc;            // [B*H*n_chunks, D]
  float2* ws_ml;            // [B*H*n_chunks]  (max in log2 units, sum)
  uint32_t* dev_status;
  int64_t q_sb, q_sh, k_sb, k_sh, v_sb, v_sh, o_sb, o_sh;
  uint32_t k_row_bytes, v_row_bytes;   // token stride of the cache in bytes
  int32_t H, max_ctx, index_stride, max_selected, chunk, n_chunks, out_f32, early_release;
  int32_t kv_group;         // query heads per K/V head (1: multi-head attention)
  int32_t gqa_wide;         // row-sharing kernel with eight warps per block
  // paged cache (page_table != nullptr): logical position t of request b is row
  // page_table[b * page_table_stride + (t >> page_shift)] << page_shift | (t & page_mask) of the pool
  const int32_t* page_table;
  int32_t page_table_stride, page_shift, page_mask, n_pages;
  float scale_log2;         // softmax scale * log2(e)
};

// Number of list entries (dense: positions) of request b, clamped to what the
// host sized the launch for.
__device__ __forceinline__ void request_sizes(const DecodeParams& p, int b, int& n, int& c,
                                              uint32_t& flags) {
  n = p.ctx_lens[b];
  if (n > p.max_ctx) { n = p.max_ctx; flags |= SSA_DEV_BAD_COUNT; }
  if (n < 0) n = 0;
  if (p.counts) {
    c = p.counts[b];
    if (c > p.max_selected) { c = p.max_selected; flags |= SSA_DEV_BAD_COUNT; }
    if (c < 0) c = 0;
  } else {
    c = n;
  }
}

template <typename T>
__device__ __forceinline__ void store_out(const DecodeParams& p, int b, int h, int d, float val) {
  const int64_t o = (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + d;
  if (p.out_f32) reinterpret_cast<float*>(p.out)[o] = val;
  else reinterpret_cast<T*>(p.out)[o] = from_float<T>(val);
}

// A lane's piece of a cache row: 16 values as eight pairs.  16-bit storage: 32 bytes, a pair per word; 8-bit
// storage: 16 bytes in w[0..3], two pairs per word.
struct Piece { uint32_t w[8]; };

// A cache row is used once per launch, so the 256-bit loads mark its lines evict-first in L2 as well: they then
// do not push out what is re-read (index lists, query rows, partial results).  Measured: 4-5 % off every workload
// (cfg 2 attention 32.4 -> 30.7 us, full context at cfg 2 105 -> 100.5 us); prefetch-size hints on top: nothing.
// (The qualifier exists for 256-bit loads only, so the 128-bit fallback keeps the default L2 policy.)
template <bool kAligned32, bool kFp8 = false>
__device__ __forceinline__ void load_piece(Piece& r, const char* p) {
  if (kFp8) {
    const uint4 a = ld_stream_16B(p);
    r.w[0] = a.x; r.w[1] = a.y; r.w[2] = a.z; r.w[3] = a.w;
    r.w[4] = 0u; r.w[5] = 0u; r.w[6] = 0u; r.w[7] = 0u;
  } else if (kAligned32) {
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]),
                   "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                 : "l"(p));
  } else {
    const uint4 a = ld_stream_16B(p), b = ld_stream_16B(p + 16);
    r.w[0] = a.x; r.w[1] = a.y; r.w[2] = a.z; r.w[3] = a.w;
    r.w[4] = b.x; r.w[5] = b.y; r.w[6] = b.z; r.w[7] = b.w;
  }
}

// Pair i (0..7) of a piece as two floats.
template <typename T>
__device__ __forceinline__ float2 piece_pair(const Piece& r, int i) {
  if constexpr (kIsFp8<T>) return e4m3x2_to_float2(r.w[i >> 1] >> ((i & 1) * 16));
  else return unpack2<T>(r.w[i]);
}

__device__ __forceinline__ void zero_piece(Piece& r) {
#pragma unroll
  for (int i = 0; i < 8; ++i) r.w[i] = 0u;
}

// kPaged (index lists only): positions are translated through the page table while they are staged, and a
// missing list stands for 0, 1, 2, ...; kept out of the unpaged instantiations so that they stay as they are.
// kHostQ (index lists, one chunk per request): the query rows are still in page-locked host memory.  Each block
// asks for its row (D/8 threads, 16 bytes each) before anything else, so that the trip across the bus overlaps
// the block's start-up, shares it through shared memory and writes the device copy the caller expects at q.
template <typename T, int D, int kMode, bool kAligned32, bool kPaged = false, bool kHostQ = false>
__global__ void __launch_bounds__(kThreads, SSA_MIN_BLOCKS)
decode_partial_kernel(const DecodeParams p) {
  static_assert(!kPaged || kMode == kIndex, "a paged cache is read through staged positions");
  static_assert(!kHostQ || (kMode == kIndex && !kPaged), "host-resident queries: plain index lists only");
  using TQ = typename Storage<T>::Query;              // type of the query rows and of a stored output
  constexpr bool kFp8 = kIsFp8<T>;
  constexpr int kU = kFp8 ? 2 * SSA_U : SSA_U;        // 8-bit pieces are half as large: twice as many in flight
  constexpr bool kSparse = kMode != kDense;           // positions come from shared memory
  constexpr int kLanesPerRow = D / 16;                // 32-byte pieces per row
  constexpr int kRowsPerLoad = 32 / kLanesPerRow;     // rows one warp-wide load covers
  constexpr int kTileRows = kRowsPerLoad * kU;        // rows per warp per iteration
  constexpr int kGroups = kWarps * kRowsPerLoad;      // independent softmax streams
  static_assert(kThreads >= D, "the epilogue uses one thread per output element");
  static_assert(kMaxChunk == kIdxPerThread * kThreads && (32 * kIdxPerThread) % kTileRows == 0,
                "a warp stages whole tiles");

  __shared__ int32_t s_idx[kSparse ? kMaxChunk : 1];
  __shared__ __align__(16) float s_acc[kGroups][D];
  __shared__ float s_m[kGroups], s_l[kGroups];
  __shared__ int s_wcount[kWarps];
  __shared__ typename std::conditional<kMode == kSpans, SpanRuns, int>::type s_runs;
  __shared__ typename std::conditional<kMode == kSpans, WarpRuns, int>::type s_wruns[kMode == kSpans ? kWarps : 1];
  __shared__ uint4 s_qrow[kHostQ ? D / 8 : 1];

  const int chunk_id = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col = lane % kLanesPerRow, sub = lane / kLanesPerRow;
  const int start = chunk_id * p.chunk;

  grid_dependency_wait();
  if (p.early_release) grid_launch_dependents();      // small grid: let the next kernel's blocks move in now

  uint4 q_word = make_uint4(0u, 0u, 0u, 0u);          // kHostQ: this thread's 16 bytes of the query row
  if constexpr (kHostQ) {
    if (tid < D / 8)
      q_word = *(reinterpret_cast<const uint4*>(reinterpret_cast<const TQ*>(p.q_host) + (int64_t)b * p.q_sb +
                                                (int64_t)h * p.q_sh) + tid);
  }

  // Everything the block needs before it can request cache rows is loaded
  // here in one go: sizes, its slice of the index list, the query row.
  // A warp stages exactly the list entries of its own tiles (entry i of the
  // warp's share is row staged_row(i) of the block), so staging needs no block
  // barrier, only a warp one.
  auto staged_row = [&](int i) {
    return warp * kTileRows + (i / kTileRows) * (kWarps * kTileRows) + (i % kTileRows);
  };
  int32_t raw[kIdxPerThread];
  if (kMode == kIndex) {
    const bool listed = !kPaged || p.index != nullptr;
    const int32_t* row = listed ? p.index + (int64_t)b * p.index_stride + start : nullptr;
#pragma unroll
    for (int j = 0; j < kIdxPerThread; ++j) {
      const int r = staged_row(lane + 32 * j);
      raw[j] = (r < p.chunk && start + r < p.max_selected) ? (listed ? __ldg(row + r) : start + r) : -1;
    }
  }
  Piece qraw;                                         // re-read by every warp and chunk of the head: plain L2 policy
  if constexpr (!kHostQ) {
    const char* qp = reinterpret_cast<const char*>(
        reinterpret_cast<const TQ*>(p.q) + (int64_t)b * p.q_sb + (int64_t)h * p.q_sh + col * 16);
    const uint4 a = ld_stream_16B(qp), c4 = ld_stream_16B(qp + 16);
    qraw.w[0] = a.x; qraw.w[1] = a.y; qraw.w[2] = a.z; qraw.w[3] = a.w;
    qraw.w[4] = c4.x; qraw.w[5] = c4.y; qraw.w[6] = c4.z; qraw.w[7] = c4.w;
  }

  // span lists: where the request's list is; with up to 32 spans every lane asks for "its" span right away (a
  // fixed-stride table needs no offsets, so the spans then arrive together with the sizes and the query)
  int span_first = 0, span_n = 0;
  int2 my_span = make_int2(0, 0);
  const bool warp_merge = kMode == kSpans && p.span_cap <= 32;
  if constexpr (kMode == kSpans) {
    if (p.span_offsets) {
      span_first = __ldg(p.span_offsets + b);
      span_n = __ldg(p.span_offsets + b + 1) - span_first;
    } else {
      span_first = b * p.span_cap;
      span_n = p.span_cap;
    }
    if (warp_merge && lane < min(span_n, p.span_cap)) my_span = __ldg(p.spans + span_first + lane);
  }
  uint32_t flags = 0;
  int n, c;
  request_sizes(p, b, n, c, flags);
  int warp_runs = 1;                                  // span_cap rounded up to a power of two
  while (warp_merge && warp_runs < p.span_cap) warp_runs <<= 1;
  if constexpr (kMode == kSpans) {
    // the request's spans -> disjoint ascending runs in shared memory (every block of the request repeats this)
    int total;
    if (warp_merge) {                                 // up to 32 spans: every warp merges them for itself, no barrier
      int S = max(span_n, 0);
      if (S > p.span_cap) { S = p.span_cap; flags |= SSA_DEV_TOO_MANY_SPANS; }
      total = merge_spans_warp(s_wruns[warp], my_span, S, warp_runs, n, flags);
    } else {
      total = merge_spans_block<kThreads>(s_runs, p.spans + span_first, span_n, p.span_cap, n);
      if (tid == 0) flags |= s_runs.flags;
    }
    c = min(total, p.max_selected);
    if (total > p.max_selected) flags |= SSA_DEV_OVERFLOW;
  }
  if (start >= c && chunk_id > 0) return;             // chunk 0 always reports
  int cnt = max(0, min(p.chunk, c - start));          // list entries of this block; rows, except for bitmasks

  if (kMode == kBlockMask) {
    // expand the set bits of up to p.chunk listed blocks into positions, in list order
    const int wpb = p.block_size / 32;
    const int64_t entry0 = (int64_t)b * p.block_stride + start;
    int rows = 0;
    for (int base = 0; base < kMaskChunk; base += kThreads) {
      const int i = base + tid, r = i / p.block_size, bit = i % p.block_size;
      int pos = -1;
      if (r < cnt) {
        const int blk = __ldg(p.block_idx + entry0 + r);
        const uint32_t word = __ldg(p.block_mask + (entry0 + r) * wpb + (bit >> 5));
        if ((word >> (bit & 31)) & 1u) {
          if (blk >= 0 && blk <= (n - 1) / p.block_size && blk * p.block_size + bit < n)
            pos = blk * p.block_size + bit;
          else
            flags |= SSA_DEV_BAD_INDEX;
        }
      }
      const uint32_t ballot = __ballot_sync(0xffffffffu, pos >= 0);
      if (lane == 0) s_wcount[warp] = __popc(ballot);
      __syncthreads();
      int at = rows + __popc(ballot & ((1u << lane) - 1u));
#pragma unroll
      for (int k = 0; k < kWarps; ++k) {
        if (k < warp) at += s_wcount[k];
        rows += s_wcount[k];
      }
      if (pos >= 0) s_idx[at] = pos;
      __syncthreads();
    }
    cnt = rows;
  }
  if constexpr (kMode == kSpans) {
    // positions of this warp's tiles, by arithmetic on the runs; head 0 leaves a copy for callers that want the list
    int32_t* row = (h == 0 && p.index_out) ? p.index_out + (int64_t)b * p.index_stride + start : nullptr;
#pragma unroll
    for (int j = 0; j < kIdxPerThread; ++j) {
      const int r = staged_row(lane + 32 * j);
      if (r < cnt) {
        const int v = warp_merge ? span_position(s_wruns[warp], warp_runs, start + r) : span_position(s_runs, start + r);
        s_idx[r] = v;
        if (row) row[r] = v;
      }
    }
    __syncwarp();
    if (chunk_id == 0 && h == 0 && tid == 0) {
      if (p.counts_out) p.counts_out[b] = c;
      if (p.ws_counts) p.ws_counts[b] = c;
    }
  }
  bool any_bad = false;                               // warp-uniform: an entry of this warp's tiles is out of range
  if (kMode == kIndex) {
    bool bad = false;
#pragma unroll
    for (int j = 0; j < kIdxPerThread; ++j) {
      const int r = staged_row(lane + 32 * j);
      if (r < cnt) {
        int v = raw[j];
        if (v < 0 || v >= n) {
          v = -1; flags |= SSA_DEV_BAD_INDEX; bad = true;
        } else if (kPaged) {                          // logical position -> row of the pool
          const int page = __ldg(p.page_table + (int64_t)b * p.page_table_stride + (v >> p.page_shift));
          if ((unsigned)page < (unsigned)p.n_pages) v = (page << p.page_shift) | (v & p.page_mask);
          else { v = -1; flags |= SSA_DEV_BAD_INDEX; bad = true; }
        }
        s_idx[r] = v;
      }
    }
    any_bad = __any_sync(0xffffffffu, bad) != 0;      // also orders the stores before the warp's reads
    __syncwarp();
  }
  if (p.dev_status && h == 0) {
    const uint32_t f = (tid == 0 && chunk_id == 0) ? flags : (flags & SSA_DEV_BAD_INDEX);
    if (f) atomicOr(p.dev_status, f);
  }

  const char* kbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.k) + (int64_t)b * p.k_sb + (int64_t)(h / p.kv_group) * p.k_sh + col * 16);
  const char* vbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.v) + (int64_t)b * p.v_sb + (int64_t)(h / p.kv_group) * p.v_sh + col * 16);

  // Requests the K and V rows of the warp's tile that starts at row t of the block; returns whether the tile needs
  // the predicated path (a ragged tail or entries that were skipped).
  Piece kr[kU], vr[kU];
  float s[kU];
  auto request_tile = [&](int t) -> bool {
    // full tiles without bad entries take the unpredicated path
    const bool checked = any_bad || (t + kTileRows > cnt);
    if (!checked) {
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int r = t + u * kRowsPerLoad + sub;
        const uint32_t pos = (uint32_t)(kSparse ? s_idx[r] : start + r);
        load_piece<kAligned32, kFp8>(kr[u], kbase + (uint64_t)pos * p.k_row_bytes);
        load_piece<kAligned32, kFp8>(vr[u], vbase + (uint64_t)pos * p.v_row_bytes);
      }
    } else {
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const int r = t + u * kRowsPerLoad + sub;
        int pos = -1;
        if (r < cnt) pos = kSparse ? s_idx[r] : start + r;
        if (pos >= 0) {
          load_piece<kAligned32, kFp8>(kr[u], kbase + (uint64_t)(uint32_t)pos * p.k_row_bytes);
          load_piece<kAligned32, kFp8>(vr[u], vbase + (uint64_t)(uint32_t)pos * p.v_row_bytes);
          s[u] = 0.f;
        } else {
          zero_piece(kr[u]);
          zero_piece(vr[u]);
          s[u] = neg_inf();                           // marks the row as masked
        }
      }
    }
    return checked;
  };
  bool pre_issued = false, pre_checked = false;
  if constexpr (kHostQ) {
    // the first tile's rows are requested before the block waits for its query row
    if (warp * kTileRows < cnt) {
      pre_checked = request_tile(warp * kTileRows);
      pre_issued = true;
    }
    // the row has crossed the bus by now (or is about to): share it, and leave the device copy
    if (tid < D / 8) {
      s_qrow[tid] = q_word;
      *(reinterpret_cast<uint4*>(const_cast<TQ*>(reinterpret_cast<const TQ*>(p.q)) + (int64_t)b * p.q_sb +
                                 (int64_t)h * p.q_sh) + tid) = q_word;
    }
    __syncthreads();                                  // one chunk per request: every block gets here
    const uint4 a = s_qrow[2 * col], c4 = s_qrow[2 * col + 1];
    qraw.w[0] = a.x; qraw.w[1] = a.y; qraw.w[2] = a.z; qraw.w[3] = a.w;
    qraw.w[4] = c4.x; qraw.w[5] = c4.y; qraw.w[6] = c4.z; qraw.w[7] = c4.w;
  }
  float2 q2[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    q2[i] = unpack2<TQ>(qraw.w[i]);
    q2[i].x *= p.scale_log2;
    q2[i].y *= p.scale_log2;
  }
  float m = neg_inf(), l = 0.f;
  float2 acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = make_float2(0.f, 0.f);

  for (int t = warp * kTileRows; t < cnt; t += kWarps * kTileRows) {
    bool checked;
    if (kHostQ && pre_issued) {                         // the warp's first tile is already on its way
      checked = pre_checked;
      pre_issued = false;
    } else {
      checked = request_tile(t);
    }
    float mt = neg_inf();
#pragma unroll
    for (int u = 0; u < kU; ++u) {
      float2 d2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 8; ++i) d2 = fma2(q2[i], piece_pair<T>(kr[u], i), d2);
      float d = d2.x + d2.y;
#pragma unroll
      for (int o = kLanesPerRow / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      s[u] = checked ? d + s[u] : d;                  // -inf stays -inf
      mt = fmaxf(mt, s[u]);
    }
    const float m_new = fmaxf(m, mt);
    if (m_new > neg_inf()) {
      if (m_new > m) {                                // rare after the first tiles
        const float alpha = fast_exp2(m - m_new);     // m = -inf gives 0
        l *= alpha;
#pragma unroll
        for (int i = 0; i < 8; ++i) { acc[i].x *= alpha; acc[i].y *= alpha; }
        m = m_new;
      }
#pragma unroll
      for (int u = 0; u < kU; ++u) {
        const float pw = fast_exp2(s[u] - m);         // masked rows give 0
        l += pw;
        const float2 pw2 = make_float2(pw, pw);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = fma2(pw2, piece_pair<T>(vr[u], i), acc[i]);
      }
    }
  }

  // all cache rows of this block have been read: the next kernel of the stream
  // may start filling the SMs this grid is leaving
  if (!p.early_release) grid_launch_dependents();

  // combine the lane groups of the block
  const int g = warp * kRowsPerLoad + sub;
#pragma unroll
  for (int i = 0; i < 4; ++i)
    *reinterpret_cast<float4*>(&s_acc[g][col * 16 + 4 * i]) =
        make_float4(acc[2 * i].x, acc[2 * i].y, acc[2 * i + 1].x, acc[2 * i + 1].y);
  if (col == 0) { s_m[g] = m; s_l[g] = l; }
  __syncthreads();
  if (tid < D) {
    float M = neg_inf();
#pragma unroll
    for (int i = 0; i < kGroups; ++i) M = fmaxf(M, s_m[i]);
    float L = 0.f, A = 0.f;
#pragma unroll
    for (int i = 0; i < kGroups; ++i) {
      const float w = (s_m[i] > neg_inf()) ? fast_exp2(s_m[i] - M) : 0.f;
      L = fmaf(s_l[i], w, L);
      A = fmaf(s_acc[i][tid], w, A);
    }
    if (p.n_chunks == 1) {
      store_out<TQ>(p, b, h, tid, L > 0.f ? A / L : 0.f);
      if (tid == 0 && p.lse) p.lse[(int64_t)b * p.H + h] = L > 0.f ? (M + log2f(L)) * kLn2 : neg_inf();
    } else {
      const int64_t slot = ((int64_t)b * p.H + h) * p.n_chunks + chunk_id;
      p.ws_acc[slot * D + tid] = A;
      if (tid == 0) p.ws_ml[slot] = make_float2(M, L);
    }
  }
}

// Pass 2.  The kernel is pure latency (a few KB per block), so everything it may need is requested in one go,
// before the request's list length is known: the (max, sum) pairs of all n_chunks slots and the first eight
// accumulator rows.  Slots of chunks that do not exist were never written; what is read from them is not used.
constexpr int kMergeStage = 512;       // (max, sum) pairs staged in shared memory; more chunks: read in place
constexpr int kMergeAhead = 8;         // accumulator rows requested before the sizes are known

template <typename T, int D>
__global__ void __launch_bounds__(D)
decode_merge_kernel(const DecodeParams p) {
  __shared__ float2 s_ml[kMergeStage];
  const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
  grid_dependency_wait();
  grid_launch_dependents();
  const int64_t base = ((int64_t)b * p.H + h) * p.n_chunks;
  const bool staged = p.n_chunks <= kMergeStage;
  if (staged)
    for (int k = d; k < p.n_chunks; k += D) s_ml[k] = p.ws_ml[base + k];
  float ahead[kMergeAhead];
#pragma unroll
  for (int k = 0; k < kMergeAhead; ++k) ahead[k] = k < p.n_chunks ? p.ws_acc[(base + k) * D + d] : 0.f;
  uint32_t flags = 0;
  int n, c;
  request_sizes(p, b, n, c, flags);
  const int ns = c > 0 ? (c + p.chunk - 1) / p.chunk : 1;
  __syncthreads();
  auto pair = [&](int k) { return staged ? s_ml[k] : p.ws_ml[base + k]; };
  float M = neg_inf();
  for (int k = 0; k < ns; ++k) M = fmaxf(M, pair(k).x);
  float L = 0.f, A = 0.f;
#pragma unroll
  for (int k = 0; k < kMergeAhead; ++k) {
    if (k < ns) {
      const float2 ml = pair(k);
      const float w = (ml.x > neg_inf()) ? fast_exp2(ml.x - M) : 0.f;
      L = fmaf(ml.y, w, L);
      A = fmaf(ahead[k], w, A);
    }
  }
  for (int k0 = kMergeAhead; k0 < ns; k0 += kMergeAhead) {   // long requests: eight rows per trip
    float rows[kMergeAhead];
#pragma unroll
    for (int j = 0; j < kMergeAhead; ++j) rows[j] = k0 + j < ns ? p.ws_acc[(base + k0 + j) * D + d] : 0.f;
#pragma unroll
    for (int j = 0; j < kMergeAhead; ++j) {
      if (k0 + j < ns) {
        const float2 ml = pair(k0 + j);
        const float w = (ml.x > neg_inf()) ? fast_exp2(ml.x - M) : 0.f;
        L = fmaf(ml.y, w, L);
        A = fmaf(rows[j], w, A);
      }
    }
  }
  store_out<T>(p, b, h, d, L > 0.f ? A / L : 0.f);
  if (d == 0 && p.lse) p.lse[(int64_t)b * p.H + h] = L > 0.f ? (M + log2f(L)) * kLn2 : neg_inf();
}

}  // namespace ssa

#include "decode_gqa.cuh"

namespace ssa {

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
struct Plan { int chunk, n_chunks; size_t acc_bytes, total_bytes; bool wide; };   // wide: eight-warp row-sharing blocks

// Grouped query heads go to the kernel that reads a K/V row once for the whole group.
static bool shares_rows(const ssa_attn_desc* d) {
  const int group = d->H_kv > 0 ? d->H / d->H_kv : 1;
  return d->D == 128 && group >= 2 && group <= kGqaHeads && d->kv_dtype != SSA_FP8_E4M3;   // mma takes 16-bit rows
}

static bool make_plan(const ssa_attn_desc* d, int max_selected, Plan* pl) {
  if (!d || d->B <= 0 || d->H <= 0 || max_selected <= 0) return false;
  if (d->D != 64 && d->D != 128) return false;
  const long long out_units = (long long)d->B * d->H;                  // triples per chunk
  const long long units = shares_rows(d) ? (long long)d->B * d->H_kv   // blocks per chunk
                                         : out_units;
  // The second pass costs about as much as two rounds of a block, so a request is split only when that buys
  // parallelism: one chunk whenever the list fits a block's staging area and either every SM gets a block or
  // the list is short anyway; otherwise 256-entry chunks, halved while the grid has under two blocks per SM.
  const long long sms = sm_count();
  const long long want = sms * 2;
  int chunk = 256;
  if (max_selected <= kMaxChunk && (units >= sms || max_selected <= 256)) chunk = kMaxChunk;
  else while (chunk > 64 && units * ((max_selected + chunk - 1) / chunk) < want) chunk >>= 1;
  pl->wide = false;
  if (shares_rows(d) && 2 * units > sms && units <= sms && max_selected <= 2048) {
    // One unit for most SMs and a short list: the whole list is one eight-warp block's work, and the second pass
    // (about 3 us in the stream) is not needed (32 query heads over 4 K/V heads, 32 requests, 819 rows: 15.2 vs
    // 18.0 us).  With fewer units (2 K/V heads: 64) too many SMs would idle: 15.2 vs 14.4 us with four chunks.
    pl->wide = true;
    chunk = (max_selected + 63) / 64 * 64;
  } else if (shares_rows(d)) {
    // The row-sharing kernel leaves G triples per chunk, its blocks stream (a ring of tiles per warp) and two of
    // them fit an SM: about one block per resident slot, i.e. as few chunks as keep the SMs busy (measured,
    // B*H_kv = 64..256, context 8192: within 3 % of the best split for groups of 4, 8 and 16 heads).
    const long long target = sms * 2;
    long long n = target / units;                              // rounded down: never one block over a full wave
    n = std::max<long long>(1, std::min<long long>(n, (max_selected + 255) / 256));
    chunk = (int)(((max_selected + n - 1) / n + 63) / 64 * 64);
  }
  int n_chunks = (max_selected + chunk - 1) / chunk;
  if (n_chunks == 1) chunk = (max_selected + 31) / 32 * 32;
  pl->chunk = chunk;
  pl->n_chunks = n_chunks;
  pl->acc_bytes = ((size_t)out_units * n_chunks * d->D * sizeof(float) + 255) / 256 * 256;
  pl->total_bytes = pl->acc_bytes + ((size_t)out_units * n_chunks * sizeof(float2) + 255) / 256 * 256;
  return true;
}

// Blocked lists: a block of the grid expands as many list entries as fit kMaskChunk positions.
static bool make_plan_blockmask(const ssa_attn_desc* d, int block_size, int max_blocks, Plan* pl) {
  if (!d || d->B <= 0 || d->H <= 0 || max_blocks <= 0) return false;
  if (d->D != 64 && d->D != 128) return false;
  if (block_size != 32 && block_size != 64 && block_size != 128 && block_size != 256) return false;
  const long long units = (long long)d->B * d->H;
  pl->wide = false;
  pl->chunk = kMaskChunk / block_size;
  pl->n_chunks = (max_blocks + pl->chunk - 1) / pl->chunk;
  pl->acc_bytes = ((size_t)units * pl->n_chunks * d->D * sizeof(float) + 255) / 256 * 256;
  pl->total_bytes = pl->acc_bytes + ((size_t)units * pl->n_chunks * sizeof(float2) + 255) / 256 * 256;
  return true;
}

static bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

static int32_t check_desc(const ssa_attn_desc* d) {
  if (d->B <= 0 || d->H <= 0 || d->max_ctx <= 0 || d->B > 65535 || d->H > 65535) return SSA_ERR_SHAPE;
  if (d->D != 64 && d->D != 128) return SSA_ERR_UNSUPPORTED;
  if (d->H_kv <= 0 || d->H % d->H_kv != 0) return SSA_ERR_UNSUPPORTED;
  const bool fp8 = d->kv_dtype == SSA_FP8_E4M3;
  if (d->kv_dtype != SSA_F16 && d->kv_dtype != SSA_BF16 && !fp8) return SSA_ERR_DTYPE;
  const int32_t q_dtype = fp8 ? SSA_BF16 : d->kv_dtype;            // queries over an 8-bit cache are bf16
  if (d->out_dtype != q_dtype && d->out_dtype != SSA_F32) return SSA_ERR_DTYPE;
  const int64_t qo_strides[] = {d->q_stride_b, d->q_stride_h, d->o_stride_b, d->o_stride_h};
  const int64_t kv_strides[] = {d->k_stride_b, d->k_stride_t, d->k_stride_h, d->v_stride_b, d->v_stride_t, d->v_stride_h};
  for (int64_t s : qo_strides) {
    if (s < 0) return SSA_ERR_SHAPE;
    if (s % 8 != 0) return SSA_ERR_ALIGN;
  }
  for (int64_t s : kv_strides) {                                   // 16 bytes: 8 16-bit or 16 8-bit elements
    if (s < 0) return SSA_ERR_SHAPE;
    if (s % (fp8 ? 16 : 8) != 0) return SSA_ERR_ALIGN;
  }
  if (d->k_stride_t >= (1ll << 31) || d->v_stride_t >= (1ll << 31)) return SSA_ERR_SHAPE;
  return SSA_OK;
}

template <typename T, int D>
static int32_t launch(const DecodeParams& p, int B, int mode, bool aligned32, cudaStream_t st) {
  cudaEvent_t ev_b, ev_e;
  take_kernel_events(&ev_b, &ev_e);
  dim3 grid((unsigned)p.n_chunks, (unsigned)p.H, (unsigned)B);
  void (*kernel)(const DecodeParams);
  using TQ = typename Storage<T>::Query;
  constexpr bool kFp8 = kIsFp8<T>;
  size_t dynamic_smem = 0;
  unsigned block_threads = kThreads;
  bool share = false;
  if constexpr (!kFp8) {                                // the row-sharing kernel feeds 16-bit rows to the tensor cores
    share = D == 128 && p.kv_group >= 2 && p.kv_group <= kGqaHeads && mode != kBlockMask;
    if (share) {
      grid.y = (unsigned)(p.H / p.kv_group);            // one block per K/V head
      const bool hi = p.kv_group > 8;
      constexpr int kW8 = kGqaWideWarps;
      if (p.gqa_wide) {
        if (mode == kIndex)
          kernel = hi ? decode_partial_gqa_kernel<T, kIndex, true, kW8> : decode_partial_gqa_kernel<T, kIndex, false, kW8>;
        else if (mode == kSpans)
          kernel = hi ? decode_partial_gqa_kernel<T, kSpans, true, kW8> : decode_partial_gqa_kernel<T, kSpans, false, kW8>;
        else
          kernel = hi ? decode_partial_gqa_kernel<T, kDense, true, kW8> : decode_partial_gqa_kernel<T, kDense, false, kW8>;
        block_threads = kW8 * 32;
      } else if (mode == kIndex)
        kernel = hi ? decode_partial_gqa_kernel<T, kIndex, true> : decode_partial_gqa_kernel<T, kIndex, false>;
      else if (mode == kSpans)
        kernel = hi ? decode_partial_gqa_kernel<T, kSpans, true> : decode_partial_gqa_kernel<T, kSpans, false>;
      else
        kernel = hi ? decode_partial_gqa_kernel<T, kDense, true> : decode_partial_gqa_kernel<T, kDense, false>;
      dynamic_smem = (size_t)(block_threads / 32) * kStagedWarpBytes;
      if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dynamic_smem) != cudaSuccess)
        return SSA_ERR_CUDA;
    }
  }
  if (!share) {
    constexpr bool kWide = !kFp8;                       // 8-bit rows are read in 16-byte pieces: one instantiation
    const bool a32 = kWide && aligned32;
    if constexpr (!kFp8) {
      if (p.q_host)                                     // run() has checked: index lists, one chunk, no paging
        kernel = a32 ? decode_partial_kernel<T, D, kIndex, true, false, true>
                     : decode_partial_kernel<T, D, kIndex, false, false, true>;
    }
    if (p.q_host) {
    } else if (mode == kIndex && p.page_table)
      kernel = a32 ? decode_partial_kernel<T, D, kIndex, kWide, true> : decode_partial_kernel<T, D, kIndex, false, true>;
    else if (mode == kIndex)
      kernel = a32 ? decode_partial_kernel<T, D, kIndex, kWide> : decode_partial_kernel<T, D, kIndex, false>;
    else if (mode == kBlockMask)
      kernel = a32 ? decode_partial_kernel<T, D, kBlockMask, kWide> : decode_partial_kernel<T, D, kBlockMask, false>;
    else if (mode == kSpans)
      kernel = a32 ? decode_partial_kernel<T, D, kSpans, kWide> : decode_partial_kernel<T, D, kSpans, false>;
    else
      kernel = a32 ? decode_partial_kernel<T, D, kDense, kWide> : decode_partial_kernel<T, D, kDense, false>;
  }
  if (ev_b) cudaEventRecord(ev_b, st);
  cudaError_t err = launch_pdl_smem(kernel, grid, dim3(block_threads), dynamic_smem, st, p);
  if (ev_e) cudaEventRecord(ev_e, st);
  if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
  int launches = 1;
  if (p.n_chunks > 1) {
    DecodeParams pm = p;
    if (mode == kSpans) pm.counts = p.ws_counts;        // the first pass left the list lengths there
    err = launch_pdl(decode_merge_kernel<TQ, D>, dim3((unsigned)p.H, (unsigned)B), dim3(D), st, pm);
    if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return SSA_ERR_CUDA;
    ++launches;
  }
  note_launches(launches);
  return SSA_OK;
}

// A request's attended set in the blocked encoding (mode kBlockMask).
struct BlockList { const int32_t* block_idx; const uint32_t* block_mask; int32_t block_size; };

// The span lists themselves (mode kSpans), with the optional copies of what they expand to.
struct SpanLists { const int32_t* span_offsets; const int32_t* spans; int32_t span_cap; int32_t* index_out;
                   int32_t* counts_out; };

static size_t counts_bytes(const ssa_attn_desc* d) { return ((size_t)d->B * sizeof(int32_t) + 255) / 256 * 256; }

// mode kDense: index/counts unused.  kIndex: the index list.  kBlockMask: `counts`
// are the numbers of listed blocks, `index_stride` the list capacity in blocks,
// `max_selected` the host bound on listed blocks, `bl` the lists.  kSpans: `sl`
// the span lists, `index_stride` the pitch of sl->index_out; the workspace then
// ends with one int32 per request (list lengths for the second pass).
static int32_t run(const ssa_attn_desc* d, const void* q, const void* k, const void* v,
                   const int32_t* ctx_lens, const int32_t* index, int32_t index_stride,
                   const int32_t* counts, int32_t max_selected, void* out, float* lse,
                   void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream, int mode,
                   const BlockList* bl = nullptr, const ssa_paging* pg = nullptr,
                   const SpanLists* sl = nullptr, const void* q_host = nullptr) {
  // a paged cache is read through the staged-positions path; without a list the positions are 0 .. ctx_len-1
  const bool dense_paged = pg && mode == kDense;
  if (dense_paged) mode = kIndex;
  const bool sparse = mode == kIndex;
  if (!d || !q || !k || !v || !ctx_lens || !out) return SSA_ERR_NULL;
  if (sparse && !dense_paged && (!index || !counts)) return SSA_ERR_NULL;
  if (pg) {
    if (!pg->page_table) return SSA_ERR_NULL;
    if (mode == kBlockMask) return SSA_ERR_UNSUPPORTED;
    if (pg->page_size <= 0 || (pg->page_size & (pg->page_size - 1)) != 0 || pg->n_pages <= 0 ||
        pg->page_table_stride <= 0 || (long long)pg->n_pages * pg->page_size > 0x7fffffffll ||
        (long long)pg->page_table_stride * pg->page_size < d->max_ctx)
      return SSA_ERR_SHAPE;
  }
  if (mode == kBlockMask && (!bl || !bl->block_idx || !bl->block_mask || !counts)) return SSA_ERR_NULL;
  if (mode == kSpans) {
    if (!sl || !sl->spans) return SSA_ERR_NULL;           // no offsets: a fixed-stride table
    if (pg) return SSA_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(sl->spans) % 8 != 0) return SSA_ERR_ALIGN;
  }
  const int32_t rc = check_desc(d);
  if (rc != SSA_OK) return rc;
  if (dense_paged) {
    max_selected = d->max_ctx;
    index_stride = d->max_ctx;
  } else if (mode == kSpans) {
    if (max_selected <= 0 || sl->span_cap <= 0 || sl->span_cap > kDirectSpans) return SSA_ERR_CAPACITY;
    if (sl->index_out && max_selected > index_stride) return SSA_ERR_CAPACITY;
  } else if (mode != kDense) {
    if (index_stride <= 0 || max_selected <= 0 || max_selected > index_stride) return SSA_ERR_CAPACITY;
  } else {
    max_selected = d->max_ctx;
  }
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(ws)) return SSA_ERR_ALIGN;
  Plan pl;
  if (mode == kBlockMask) {
    if (bl->block_size != 32 && bl->block_size != 64 && bl->block_size != 128 && bl->block_size != 256)
      return SSA_ERR_UNSUPPORTED;
    if (!make_plan_blockmask(d, bl->block_size, max_selected, &pl)) return SSA_ERR_SHAPE;
  } else if (!make_plan(d, max_selected, &pl)) {
    return SSA_ERR_SHAPE;
  }
  if (!ws || ws_bytes < pl.total_bytes + (mode == kSpans ? counts_bytes(d) : 0)) return SSA_ERR_WORKSPACE;

  if (q_host && !(mode == kIndex && !pg && !dense_paged && pl.n_chunks == 1 && !shares_rows(d) &&
                  d->kv_dtype != SSA_FP8_E4M3 && aligned16(q_host)))
    return SSA_ERR_UNSUPPORTED;
  DecodeParams p;
  p.q_host = q_host;
  p.span_offsets = mode == kSpans ? sl->span_offsets : nullptr;
  p.spans = mode == kSpans ? reinterpret_cast<const int2*>(sl->spans) : nullptr;
  p.span_cap = mode == kSpans ? sl->span_cap : 0;
  p.index_out = mode == kSpans ? sl->index_out : nullptr;
  p.counts_out = mode == kSpans ? sl->counts_out : nullptr;
  p.ws_counts = mode == kSpans ? reinterpret_cast<int32_t*>(reinterpret_cast<char*>(ws) + pl.total_bytes) : nullptr;
  p.q = q; p.k = k; p.v = v;
  p.ctx_lens = ctx_lens;
  p.index = sparse && !dense_paged ? index : nullptr;
  p.counts = mode != kDense && mode != kSpans && !dense_paged ? counts : nullptr;
  p.page_table = pg ? pg->page_table : nullptr;
  p.page_table_stride = pg ? pg->page_table_stride : 0;
  p.n_pages = pg ? pg->n_pages : 0;
  p.page_mask = pg ? pg->page_size - 1 : 0;
  p.page_shift = 0;
  while (pg && (1 << p.page_shift) < pg->page_size) ++p.page_shift;
  p.block_idx = mode == kBlockMask ? bl->block_idx : nullptr;
  p.block_mask = mode == kBlockMask ? bl->block_mask : nullptr;
  p.block_size = mode == kBlockMask ? bl->block_size : 0;
  p.block_stride = mode == kBlockMask ? index_stride : 0;
  p.out = out; p.lse = lse;
  p.ws_acc = reinterpret_cast<float*>(ws);
  p.ws_ml = reinterpret_cast<float2*>(reinterpret_cast<char*>(ws) + pl.acc_bytes);
  p.dev_status = dev_status;
  p.q_sb = d->q_stride_b; p.q_sh = d->q_stride_h;
  p.kv_group = d->H / d->H_kv;
  p.k_sb = pg ? 0 : d->k_stride_b; p.k_sh = d->k_stride_h;      // a pool has no batch dimension
  p.v_sb = pg ? 0 : d->v_stride_b; p.v_sh = d->v_stride_h;
  const int kv_bytes = d->kv_dtype == SSA_FP8_E4M3 ? 1 : 2;
  p.k_row_bytes = (uint32_t)(d->k_stride_t * kv_bytes);
  p.v_row_bytes = (uint32_t)(d->v_stride_t * kv_bytes);
  p.o_sb = d->o_stride_b; p.o_sh = d->o_stride_h;
  p.H = d->H; p.max_ctx = d->max_ctx;
  p.index_stride = index_stride; p.max_selected = max_selected;
  p.chunk = pl.chunk; p.n_chunks = pl.n_chunks;
  p.gqa_wide = pl.wide ? 1 : 0;
  p.out_f32 = d->out_dtype == SSA_F32;
  // A grid of a few waves releases the next kernel at once (its blocks wait on
  // chip instead of being launched after the drain); a long grid does so only
  // as its blocks finish, so that waiting blocks do not crowd out its own.
  p.early_release = (long long)d->B * d->H * pl.n_chunks <= (long long)sm_count() * SSA_MIN_BLOCKS * 6;
  const float scale = d->scale > 0.f ? d->scale : 1.0f / sqrtf((float)d->D);
  p.scale_log2 = scale * kLog2e;

  // one 256-bit load per lane needs every cache row piece on a 32-byte boundary
  const bool a32 = reinterpret_cast<uintptr_t>(k) % 32 == 0 && reinterpret_cast<uintptr_t>(v) % 32 == 0 &&
                   p.k_sb % 16 == 0 && d->k_stride_t % 16 == 0 && d->k_stride_h % 16 == 0 &&
                   p.v_sb % 16 == 0 && d->v_stride_t % 16 == 0 && d->v_stride_h % 16 == 0;
  cudaStream_t st = (cudaStream_t)stream;
  if (d->kv_dtype == SSA_FP8_E4M3)
    return d->D == 128 ? launch<Fp8E4M3, 128>(p, d->B, mode, false, st) : launch<Fp8E4M3, 64>(p, d->B, mode, false, st);
  if (d->kv_dtype == SSA_BF16)
    return d->D == 128 ? launch<__nv_bfloat16, 128>(p, d->B, mode, a32, st)
                       : launch<__nv_bfloat16, 64>(p, d->B, mode, a32, st);
  return d->D == 128 ? launch<__half, 128>(p, d->B, mode, a32, st) : launch<__half, 64>(p, d->B, mode, a32, st);
}

int32_t one_kernel_span_limit() { return kDirectSpans; }

// ssa_decode_attn_sparse with the query rows still in page-locked host memory that the device addresses (q_host,
// laid out like q): every block fetches its own row across the bus and writes the device copy at q.  Offered
// where host_queries_pay() says so.
int32_t decode_attn_sparse_host_queries(const ssa_attn_desc* desc, void* q, const void* q_host, const void* k_cache,
                                        const void* v_cache, const int32_t* ctx_lens, const int32_t* index,
                                        int32_t index_stride, const int32_t* counts, int32_t max_selected, void* out,
                                        float* lse, void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                        void* stream) {
  if (!q_host) return SSA_ERR_NULL;
  return run(desc, q, k_cache, v_cache, ctx_lens, index, index_stride, counts, max_selected, out, lse, workspace,
             workspace_bytes, dev_status, stream, kIndex, nullptr, nullptr, nullptr, q_host);
}

// One chunk per request (every row then crosses the bus once), multi-head 16-bit cache.
bool host_queries_pay(const ssa_attn_desc* d, int32_t max_selected) {
  Plan pl;
  if (!d || check_desc(d) != SSA_OK || !make_plan(d, max_selected, &pl)) return false;
  return pl.n_chunks == 1 && !shares_rows(d) && d->kv_dtype != SSA_FP8_E4M3;
}

// Every block of the span-list kernel repeats the merge of its request's spans (about a microsecond per wave
// of blocks when a warp can do it alone), the index kernel does it once per request but costs a launch of its
// own (about 3 us exposed): one kernel up to three waves of blocks.
bool one_kernel_step_pays(const ssa_attn_desc* d, int32_t max_selected, int32_t max_spans, size_t ws_bytes) {
  Plan pl;
  if (max_spans <= 0 || max_spans > 32 || !d || check_desc(d) != SSA_OK || !make_plan(d, max_selected, &pl))
    return false;
  if (ws_bytes < pl.total_bytes + counts_bytes(d)) return false;
  const long long units = shares_rows(d) ? (long long)d->B * d->H_kv : (long long)d->B * d->H;
  return units * pl.n_chunks <= 3ll * SSA_MIN_BLOCKS * sm_count();
}

// Scratch of ssa_decode_attn_sparse_noalloc: part of the library's device image.
// In host code the name `g_static_scratch` is only a handle for
// cudaGetSymbolAddress, never a device address to pass to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[SSA_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device (its primary context), looked up once per device; threads
// that race on the first call all store the same value.  The address does not survive cudaDeviceReset.
static void* static_scratch_address() {
  constexpr int kMaxDevices = 64;
  static std::atomic<void*> address[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  void* ptr = address[dev].load(std::memory_order_acquire);
  if (!ptr) {
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return nullptr;
    address[dev].store(ptr, std::memory_order_release);
  }
  return ptr;
}

}  // namespace ssa

extern "C" {

int32_t ssa_decode_attn_sparse_noalloc(const ssa_attn_desc* desc, const void* q, const void* k_cache,
                                       const void* v_cache, const int32_t* ctx_lens, const int32_t* index,
                                       int32_t index_stride, const int32_t* counts, int32_t max_selected,
                                       void* out, float* lse, uint32_t* dev_status, void* stream) {
  // the checks of ssa_decode_attn_sparse in its order, so that a bad call gets the same status from both
  if (!desc || !q || !k_cache || !v_cache || !ctx_lens || !out || !index || !counts) return SSA_ERR_NULL;
  const int32_t rc = ssa::check_desc(desc);
  if (rc != SSA_OK) return rc;
  if (index_stride <= 0 || max_selected <= 0 || max_selected > index_stride) return SSA_ERR_CAPACITY;
  if (!ssa::aligned16(q) || !ssa::aligned16(k_cache) || !ssa::aligned16(v_cache) || !ssa::aligned16(out))
    return SSA_ERR_ALIGN;
  ssa::Plan pl;
  if (!ssa::make_plan(desc, max_selected, &pl)) return SSA_ERR_SHAPE;
  if (pl.total_bytes > SSA_STATIC_SCRATCH_BYTES) return SSA_ERR_WORKSPACE;   // beyond the built-in scratch
  void* scratch = ssa::static_scratch_address();
  if (!scratch) return SSA_ERR_CUDA;
  return ssa::run(desc, q, k_cache, v_cache, ctx_lens, index, index_stride, counts, max_selected, out, lse,
                  scratch, SSA_STATIC_SCRATCH_BYTES, dev_status, stream, ssa::kIndex);
}

// Layout of the workspace of ssa_decode_attn_spans: the partial results of the split pass, one int32 per
// request, and - only when the request may have more spans than a block merges in shared memory and the
// list is expanded by ssa_spans_to_index first - room for the index lists.
static size_t spans_index_pitch(int32_t max_selected) { return ((size_t)max_selected + 31) / 32 * 32; }

size_t ssa_decode_spans_workspace_bytes(const ssa_attn_desc* desc, int32_t max_selected, int32_t max_spans) {
  ssa::Plan pl;
  if (!desc || max_spans <= 0 || ssa::check_desc(desc) != SSA_OK || !ssa::make_plan(desc, max_selected, &pl))
    return 0;
  size_t need = pl.total_bytes + ssa::counts_bytes(desc);
  if (max_spans > ssa::kDirectSpans) need += (size_t)desc->B * spans_index_pitch(max_selected) * sizeof(int32_t);
  return need;
}

int32_t ssa_decode_attn_spans(const ssa_attn_desc* desc, const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* ctx_lens, const int32_t* span_offsets, const int32_t* spans,
                              int32_t max_spans, int32_t max_selected, void* out, float* lse, int32_t* index_out,
                              int32_t index_stride, int32_t* counts_out, void* workspace, size_t workspace_bytes,
                              uint32_t* dev_status, void* stream) {
  if (!desc || !spans) return SSA_ERR_NULL;
  if (max_spans <= 0) return SSA_ERR_CAPACITY;
  if (!span_offsets && max_spans > ssa::kDirectSpans) return SSA_ERR_UNSUPPORTED;
  if (max_spans <= ssa::kDirectSpans) {
    const ssa::SpanLists sl = {span_offsets, spans, max_spans, index_out, counts_out};
    return ssa::run(desc, q, k_cache, v_cache, ctx_lens, nullptr, index_stride, nullptr, max_selected, out, lse,
                    workspace, workspace_bytes, dev_status, stream, ssa::kSpans, nullptr, nullptr, &sl);
  }
  // More spans per request than a block merges on chip: expand the lists once (into the caller's buffers
  // when given, else into the workspace) and attend through them.
  if (!q || !k_cache || !v_cache || !ctx_lens || !out) return SSA_ERR_NULL;
  const int32_t rc = ssa::check_desc(desc);
  if (rc != SSA_OK) return rc;
  ssa::Plan pl;
  if (max_selected <= 0 || (index_out && max_selected > index_stride)) return SSA_ERR_CAPACITY;
  if (!ssa::make_plan(desc, max_selected, &pl)) return SSA_ERR_SHAPE;
  if (!workspace || workspace_bytes < ssa_decode_spans_workspace_bytes(desc, max_selected, max_spans))
    return SSA_ERR_WORKSPACE;
  if (!ssa::aligned16(workspace)) return SSA_ERR_ALIGN;
  char* ws = static_cast<char*>(workspace);
  int32_t* counts = counts_out ? counts_out : reinterpret_cast<int32_t*>(ws + pl.total_bytes);
  int32_t* index = index_out ? index_out : reinterpret_cast<int32_t*>(ws + pl.total_bytes + ssa::counts_bytes(desc));
  const int32_t pitch = index_out ? index_stride : (int32_t)spans_index_pitch(max_selected);
  const int32_t cap = max_spans < SSA_MAX_SPANS_PER_SEQ ? max_spans : SSA_MAX_SPANS_PER_SEQ;
  const int32_t rc2 = ssa::spans_to_index_capped(span_offsets, spans, ctx_lens, desc->B, index, pitch, max_selected,
                                                 cap, counts, dev_status, (cudaStream_t)stream);
  if (rc2 != SSA_OK) return rc2;
  return ssa::run(desc, q, k_cache, v_cache, ctx_lens, index, pitch, counts, max_selected, out, lse, workspace,
                  pl.total_bytes, dev_status, stream, ssa::kIndex);
}

// Several query tokens per head: (head, token) pairs become the heads of a wider descriptor over the same cache
// heads, so that the kernel for grouped query heads reads every selected row once for all of them.
static int32_t widen_for_tokens(const ssa_attn_desc* desc, int32_t n_q, int64_t q_stride_t, int64_t o_stride_t,
                                ssa_attn_desc* wide) {
  if (!desc) return SSA_ERR_NULL;
  if (n_q <= 0 || (long long)desc->H * n_q > 65535) return SSA_ERR_SHAPE;
  if (desc->q_stride_h != (int64_t)n_q * q_stride_t || desc->o_stride_h != (int64_t)n_q * o_stride_t)
    return SSA_ERR_UNSUPPORTED;                          // the rows of one head must lie side by side
  *wide = *desc;
  wide->H = desc->H * n_q;
  wide->q_stride_h = q_stride_t;
  wide->o_stride_h = o_stride_t;
  return SSA_OK;
}

size_t ssa_decode_multiq_workspace_bytes(const ssa_attn_desc* desc, int32_t n_q, int32_t max_selected) {
  ssa_attn_desc wide;
  if (!desc || widen_for_tokens(desc, n_q, desc->q_stride_h / (n_q > 0 ? n_q : 1),
                                desc->o_stride_h / (n_q > 0 ? n_q : 1), &wide) != SSA_OK)
    return 0;
  return ssa_decode_workspace_bytes(&wide, max_selected);
}

int32_t ssa_decode_attn_sparse_multiq(const ssa_attn_desc* desc, int32_t n_q, int64_t q_stride_t, int64_t o_stride_t,
                                      const void* q, const void* k_cache, const void* v_cache,
                                      const int32_t* ctx_lens, const int32_t* index, int32_t index_stride,
                                      const int32_t* counts, int32_t max_selected, void* out, float* lse,
                                      void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream) {
  ssa_attn_desc wide;
  const int32_t rc = widen_for_tokens(desc, n_q, q_stride_t, o_stride_t, &wide);
  if (rc != SSA_OK) return rc;
  return ssa::run(&wide, q, k_cache, v_cache, ctx_lens, index, index_stride, counts, max_selected, out, lse,
                  workspace, workspace_bytes, dev_status, stream, ssa::kIndex);
}

int32_t ssa_decode_attn_dense_multiq(const ssa_attn_desc* desc, int32_t n_q, int64_t q_stride_t, int64_t o_stride_t,
                                     const void* q, const void* k_cache, const void* v_cache,
                                     const int32_t* ctx_lens, void* out, float* lse, void* workspace,
                                     size_t workspace_bytes, uint32_t* dev_status, void* stream) {
  ssa_attn_desc wide;
  const int32_t rc = widen_for_tokens(desc, n_q, q_stride_t, o_stride_t, &wide);
  if (rc != SSA_OK) return rc;
  return ssa::run(&wide, q, k_cache, v_cache, ctx_lens, nullptr, 0, nullptr, 0, out, lse, workspace,
                  workspace_bytes, dev_status, stream, ssa::kDense);
}

size_t ssa_decode_blockmask_workspace_bytes(const ssa_attn_desc* desc, int32_t block_size, int32_t max_blocks) {
  ssa::Plan pl;
  if (!desc || ssa::check_desc(desc) != SSA_OK || !ssa::make_plan_blockmask(desc, block_size, max_blocks, &pl))
    return 0;
  return pl.total_bytes;
}

int32_t ssa_decode_attn_blockmask(const ssa_attn_desc* desc, const void* q, const void* k_cache,
                                  const void* v_cache, const int32_t* ctx_lens, const int32_t* block_idx,
                                  const uint32_t* block_mask, int32_t block_stride, const int32_t* block_counts,
                                  int32_t block_size, int32_t max_blocks, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream) {
  const ssa::BlockList bl = {block_idx, block_mask, block_size};
  return ssa::run(desc, q, k_cache, v_cache, ctx_lens, nullptr, block_stride, block_counts, max_blocks, out, lse,
                  workspace, workspace_bytes, dev_status, stream, ssa::kBlockMask, &bl);
}

size_t ssa_decode_workspace_bytes(const ssa_attn_desc* desc, int32_t max_selected) {
  ssa::Plan pl;
  if (!desc || ssa::check_desc(desc) != SSA_OK || !ssa::make_plan(desc, max_selected, &pl)) return 0;
  return pl.total_bytes;
}

int32_t ssa_decode_attn_sparse(const ssa_attn_desc* desc, const void* q, const void* k_cache,
                               const void* v_cache, const int32_t* ctx_lens, const int32_t* index,
                               int32_t index_stride, const int32_t* counts, int32_t max_selected,
                               void* out, float* lse, void* workspace, size_t workspace_bytes,
                               uint32_t* dev_status, void* stream) {
  return ssa::run(desc, q, k_cache, v_cache, ctx_lens, index, index_stride, counts, max_selected, out,
                  lse, workspace, workspace_bytes, dev_status, stream, ssa::kIndex);
}

int32_t ssa_decode_attn_dense(const ssa_attn_desc* desc, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* ctx_lens, void* out, float* lse,
                              void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                              void* stream) {
  return ssa::run(desc, q, k_cache, v_cache, ctx_lens, nullptr, 0, nullptr, 0, out, lse, workspace,
                  workspace_bytes, dev_status, stream, ssa::kDense);
}

int32_t ssa_decode_attn_sparse_paged(const ssa_attn_desc* desc, const void* q, const void* k_pool,
                                     const void* v_pool, const ssa_paging* paging, const int32_t* ctx_lens,
                                     const int32_t* index, int32_t index_stride, const int32_t* counts,
                                     int32_t max_selected, void* out, float* lse, void* workspace,
                                     size_t workspace_bytes, uint32_t* dev_status, void* stream) {
  if (!paging) return SSA_ERR_NULL;
  return ssa::run(desc, q, k_pool, v_pool, ctx_lens, index, index_stride, counts, max_selected, out, lse,
                  workspace, workspace_bytes, dev_status, stream, ssa::kIndex, nullptr, paging);
}

int32_t ssa_decode_attn_dense_paged(const ssa_attn_desc* desc, const void* q, const void* k_pool,
                                    const void* v_pool, const ssa_paging* paging, const int32_t* ctx_lens,
                                    void* out, float* lse, void* workspace, size_t workspace_bytes,
                                    uint32_t* dev_status, void* stream) {
  if (!paging) return SSA_ERR_NULL;
  return ssa::run(desc, q, k_pool, v_pool, ctx_lens, nullptr, 0, nullptr, 0, out, lse, workspace,
                  workspace_bytes, dev_status, stream, ssa::kDense, nullptr, paging);
}

}  // extern "C"
