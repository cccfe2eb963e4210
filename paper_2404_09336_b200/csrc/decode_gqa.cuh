// Pass 1 of the decode attention for grouped query heads (G = H / H_kv query
// heads share one K/V head, 2 <= G <= 16, D = 128; also several query tokens
// per head, which are served the same way): one block per (chunk, K/V head,
// request) reads every selected row ONCE and serves all G heads.
//
// With G heads per row the work per byte is G times that of multi-head
// attention and the packed-FMA path of decode_partial_kernel runs out of issue
// slots before it runs out of HBM bandwidth, so here the two contractions go
// to the tensor cores.  The shapes are far too small for tcgen05 tiles (G x 16
// rows x 128), so they are warp-level mma.sync.m16n8k16 (16-bit inputs, fp32
// accumulation) with the M dimension holding the query heads:
//   S[16 heads, 16 rows]  = Q . K_tile^T : A = Q (registers, loaded once),
//                           B = K tile via ldmatrix (rows are the n index);
//   O[16 heads, 128 dims] += P . V_tile  : A = P from the accumulators of S,
//                           B = V tile via ldmatrix.trans (rows are the k index).
// The rows travel global -> shared memory by asynchronous 16-byte copies
// (cp.async, evict-first in L2) into a ring of tiles that every warp keeps for
// itself, and the fragments come out of that ring with ldmatrix.  The bytes in
// flight are set by the ring (three tiles of 16 rows x (K + V) = 24 KB per
// warp, 96 KB per block, two blocks per SM), not by fragment registers, and a
// warp works on one tile while its next two are on their way; no block
// barrier inside the tile loop.  (An earlier version loaded the fragments
// straight from global memory into registers, one tile in flight per warp:
// 5-15 % slower on long lists.)
//
// Shared-memory tiles are [16 rows][256 bytes] with the 16-byte chunk index
// XOR-ed with (row & 7), so that the eight row addresses of an ldmatrix hit
// eight different bank groups.
// The softmax weights are the fp32 accumulators of S; they enter the second
// contraction as a 16-bit value plus a 16-bit residual (two mma passes), so
// the result keeps fp32-level accuracy instead of the 2^-9 of a bf16 weight.
// Included by decode_attn.cu after DecodeParams and its helpers.
#pragma once

namespace ssa {

template <typename T>
__device__ __forceinline__ uint32_t pack2(float lo, float hi);
template <>
__device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
template <>
__device__ __forceinline__ uint32_t pack2<__half>(float lo, float hi) {
  const __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// D(16x8, fp32) = A(16x16) . B(16x8) + C, 16-bit inputs of type T.
template <typename T>
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1, const float (&c)[4]);
template <>
__device__ __forceinline__ void mma_16816<__nv_bfloat16>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                         uint32_t a3, uint32_t b0, uint32_t b1,
                                                         const float (&c)[4]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
               "{%10,%11,%12,%13};"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
template <>
__device__ __forceinline__ void mma_16816<__half>(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1, const float (&c)[4]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
               "{%10,%11,%12,%13};"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

constexpr int kGqaRows = 16;            // rows per warp per iteration
constexpr int kGqaHeads = 16;           // M of the mma: most query heads one block serves
constexpr int kGqaPad = 4;              // floats of padding per head row of the block-level combine

constexpr int kStagedDepth = 3;                          // tiles per warp in the ring
constexpr int kStagedTileBytes = kGqaRows * 256;         // one tensor's tile
constexpr int kStagedWarpBytes = kStagedDepth * 2 * kStagedTileBytes;
constexpr int kStagedSmemBytes = kWarps * kStagedWarpBytes;   // four-warp blocks: 96 KB, two blocks per SM
constexpr int kGqaWideWarps = 8;                         // eight-warp blocks (192 KB, one per SM) for short lists of few units
// A chunk is worked through in windows: the block's warps meet at every window's end (and, for lists, stage
// the next window's positions).  Meeting often keeps the four warps on neighbouring rows, which the memory
// system rewards (full context at 32 query heads over 8 / 4 / 2 K/V heads: 6.9 / 6.3 / 5.4 TB/s with windows
// of 256 rows, 6.7 / 6.2 / 5.4 with 512, 6.5 / 6.0 / 5.4 with 1024, 6.3 / 5.8 / 5.2 without windows), but each
// meeting lets the ring run empty once (windows of 64 rows: 5.7 / 5.2 / 4.6 TB/s).
constexpr int kStagedWindow = 512;                       // list entries staged at a time ...
constexpr int kStagedShortList = 1024;                   // ... unless the whole chunk fits this many: then one window
constexpr int kStagedDenseWindow = 256;                  // full context: rows between two meetings of the warps

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte asynchronous copy global -> shared, not kept in L1, evict-first in L2; src_bytes = 0 writes zeros.
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, uint32_t src_bytes, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;"
               ::"r"(dst), "l"(src), "r"(src_bytes), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// byte offset of 16-byte chunk `chunk` of row `row` inside a swizzled [16][256 B] tile
__device__ __forceinline__ uint32_t tile_offset(int row, int chunk) {
  return (uint32_t)(row * 256 + ((chunk ^ (row & 7)) << 4));
}

// kW: warps per block.  Four is the rule (two blocks per SM).  Eight serve launches with at most one unit (request x
// K/V head) per SM and short lists: a whole list is then one block's work - no second pass - and eight warps stream it.
template <typename T, int kMode, bool kHi, int kW = kWarps>
__global__ void __launch_bounds__(kW * 32, kW == kWarps ? 2 : 1)
decode_partial_gqa_kernel(const DecodeParams p) {
  constexpr int kWarps = kW, kThreads = kW * 32;      // hide the library-wide four-warp constants in here
  constexpr int D = 128;
  constexpr bool kSparse = kMode != kDense;
  constexpr int kLiveHeads = kHi ? 16 : 8;
  static_assert(kMode == kDense || kMode == kIndex || kMode == kSpans,
                "blocked lists take the one-head-per-block kernel");
  static_assert(kLiveHeads * (D + kGqaPad) * 4 <= kStagedWarpBytes, "the combine reuses the ring");

  extern __shared__ __align__(128) unsigned char s_ring[];
  __shared__ int32_t s_idx[kSparse ? kStagedShortList : 1];
  __shared__ __align__(128) unsigned char s_qtile[kGqaHeads * 256];   // Q of the group, swizzled like a row tile
  __shared__ float s_m[kWarps][kLiveHeads], s_l[kWarps][kLiveHeads];
  __shared__ typename std::conditional<kMode == kSpans, SpanRuns, int>::type s_runs;

  const int chunk_id = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, j = lane & 3;
  const int G = p.kv_group;
  const int start = chunk_id * p.chunk;

  grid_dependency_wait();
  if (p.early_release) grid_launch_dependents();

  // One round trip for everything that does not depend on the list length: the first kStagedShortList list
  // entries of the chunk (within the host's bound, so inside the caller's row) and the group's query rows.
  constexpr int kAhead = kStagedShortList / kThreads;
  int32_t ahead[kAhead];
  const bool listed = kMode == kIndex && p.index != nullptr;
  if (listed) {
    const int32_t* row = p.index + (int64_t)b * p.index_stride + start;
#pragma unroll
    for (int jj = 0; jj < kAhead; ++jj) {
      const int i = tid + jj * kThreads;
      ahead[jj] = (i < p.chunk && start + i < p.max_selected) ? __ldg(row + i) : -1;
    }
  }
  uint4 q_lo = make_uint4(0u, 0u, 0u, 0u), q_hi = make_uint4(0u, 0u, 0u, 0u);
  {
    const int row = tid >> 3, c0 = (tid & 7) * 2;     // 16 rows x 8 threads; further threads have no part
    if (row < G) {
      const T* src = reinterpret_cast<const T*>(p.q) + (int64_t)b * p.q_sb + (int64_t)(kvh * G + row) * p.q_sh + 8 * c0;
      q_lo = ld_stream_16B(src);
      q_hi = ld_stream_16B(src + 8);
    }
  }
  uint32_t flags = 0;
  int n, c;
  request_sizes(p, b, n, c, flags);
  if constexpr (kMode == kSpans) {
    const int first = p.span_offsets ? __ldg(p.span_offsets + b) : b * p.span_cap;
    const int S = p.span_offsets ? __ldg(p.span_offsets + b + 1) - first : p.span_cap;
    const int total = merge_spans_block<kThreads>(s_runs, p.spans + first, S, p.span_cap, n);
    c = min(total, p.max_selected);
    if (total > p.max_selected) flags |= SSA_DEV_OVERFLOW;
    if (tid == 0) flags |= s_runs.flags;
    if (chunk_id == 0 && kvh == 0 && tid == 0) {
      if (p.counts_out) p.counts_out[b] = c;
      if (p.ws_counts) p.ws_counts[b] = c;
    }
  }
  if (start >= c && chunk_id > 0) return;
  const int cnt = max(0, min(p.chunk, c - start));

  auto stage_window = [&](int w0, int wn) {
    if constexpr (kMode == kSpans) {
      int32_t* out = (kvh == 0 && p.index_out) ? p.index_out + (int64_t)b * p.index_stride + start + w0 : nullptr;
      for (int i = tid; i < wn; i += kThreads) {
        const int v = span_position(s_runs, start + w0 + i);
        s_idx[i] = v;
        if (out) out[i] = v;
      }
      return;
    }
    // position -> what the tile loop uses: -1 for an entry outside the context, the pool row for a paged cache
    auto checked = [&](int v) {
      if (v < 0 || v >= n) {
        flags |= SSA_DEV_BAD_INDEX;
        return -1;
      }
      if (p.page_table) {
        const int page = __ldg(p.page_table + (int64_t)b * p.page_table_stride + (v >> p.page_shift));
        if ((unsigned)page < (unsigned)p.n_pages) return (page << p.page_shift) | (v & p.page_mask);
        flags |= SSA_DEV_BAD_INDEX;
        return -1;
      }
      return v;
    };
    if (listed && w0 == 0) {                             // the entries requested ahead cover any first window
#pragma unroll
      for (int jj = 0; jj < kAhead; ++jj) {
        const int i = tid + jj * kThreads;
        if (i < wn) s_idx[i] = checked(ahead[jj]);
      }
      return;
    }
    const int32_t* row = listed ? p.index + (int64_t)b * p.index_stride + start + w0 : nullptr;
    for (int i = tid; i < wn; i += kThreads)             // no list: the position itself (a paged full context)
      s_idx[i] = checked(row ? __ldg(row + i) : start + w0 + i);
  };
  // a list chunk of up to kStagedShortList entries is one window (no meeting in mid-chunk); longer ones go by 512
  const int window = kSparse ? (cnt <= kStagedShortList ? kStagedShortList : kStagedWindow) : kStagedDenseWindow;
  if (kSparse) stage_window(0, min(cnt, window));
  // the group's query rows -> shared memory (rows of heads that do not exist are zero)
  if (tid < kGqaHeads * 8) {
    const int row = tid >> 3, c0 = (tid & 7) * 2;
    *reinterpret_cast<uint4*>(s_qtile + tile_offset(row, c0)) = q_lo;
    *reinterpret_cast<uint4*>(s_qtile + tile_offset(row, c0 + 1)) = q_hi;
  }
  __syncthreads();
  // A fragments of Q for the eight k-steps: registers for the whole block's life
  uint32_t qa[8][4];
  {
    const int m = lane >> 3, r = lane & 7;
    const uint32_t base = smem_u32(s_qtile);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) ldmatrix_x4(qa[ks], base + tile_offset((m & 1) * 8 + r, 2 * ks + (m >> 1)));
  }
  uint64_t policy;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
  const char* kbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.k) + (int64_t)b * p.k_sb + (int64_t)kvh * p.k_sh);
  const char* vbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.v) + (int64_t)b * p.v_sb + (int64_t)kvh * p.v_sh);
  const uint32_t ring = smem_u32(s_ring) + warp * kStagedWarpBytes;

  // running softmax state of heads g (lo) and g+8 (hi); sums are per lane until the end.
  // o[nt][e]: dims 8 nt + 2j + (e & 1) of head g (e < 2) or g + 8 (e >= 2)
  float m_lo = neg_inf(), m_hi = neg_inf(), l_lo = 0.f, l_hi = 0.f;
  float o[16][4];
#pragma unroll
  for (int u = 0; u < 16; ++u) { o[u][0] = 0.f; o[u][1] = 0.f; o[u][2] = 0.f; o[u][3] = 0.f; }

  for (int w0 = 0; w0 < cnt; w0 += window) {
    const int wn = min(window, cnt - w0);
    if (kSparse && w0 > 0) {
      __syncthreads();                                 // every warp is done with the previous window
      stage_window(w0, wn);
      __syncthreads();
    }
    const int first_row = warp * kGqaRows;
    const int nk = wn > first_row ? (wn - first_row + kWarps * kGqaRows - 1) / (kWarps * kGqaRows) : 0;
    // position of row (lane & 15) of this warp's k-th tile, -1 if there is none
    auto tile_pos = [&](int k) {
      const int r = first_row + k * (kWarps * kGqaRows) + (lane & 15);
      return r < wn ? (kSparse ? s_idx[r] : start + w0 + r) : -1;
    };
    // requests tile k of the window (if it exists) into slot k % depth; always closes a copy group
    auto request = [&](int k) {
      if (k < nk) {
        const int my_pos = tile_pos(k);
        const uint32_t slot = ring + (uint32_t)(k % kStagedDepth) * (2 * kStagedTileBytes);
        const int chunk = lane & 15;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = 2 * i + (lane >> 4);
          const int pos = __shfl_sync(0xffffffffu, my_pos, r);
          const uint32_t bytes = pos >= 0 ? 16u : 0u;
          const uint64_t row = pos >= 0 ? (uint64_t)(uint32_t)pos : 0ull;
          const uint32_t off = tile_offset(r, chunk);
          cp_async_16(slot + off, kbase + row * p.k_row_bytes + chunk * 16, bytes, policy);
          cp_async_16(slot + kStagedTileBytes + off, vbase + row * p.v_row_bytes + chunk * 16, bytes, policy);
        }
      }
      cp_async_commit();
    };
#pragma unroll
    for (int k = 0; k < kStagedDepth - 1; ++k) request(k);
    for (int k = 0; k < nk; ++k) {
      __syncwarp();                                    // the slot about to be refilled has been read by every lane
      request(k + kStagedDepth - 1);
      cp_async_wait<kStagedDepth - 1>();               // tile k has landed (for this lane's copies) ...
      __syncwarp();                                    // ... and for every other lane's
      const uint32_t live = __ballot_sync(0xffffffffu, tile_pos(k) >= 0) & 0xffffu;
      if (live == 0u) continue;                        // warp-uniform: nothing to add
      const uint32_t kt = ring + (uint32_t)(k % kStagedDepth) * (2 * kStagedTileBytes), vt = kt + kStagedTileBytes;
      const int mm = lane >> 3, rr = lane & 7;

      // S = Q . K^T: two n-tiles of 8 rows
      float s[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) { s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f; }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t kb[4];                                // rows 0-7: k lo, k hi; rows 8-15: k lo, k hi
        ldmatrix_x4(kb, kt + tile_offset((mm >> 1) * 8 + rr, 2 * ks + (mm & 1)));
        mma_16816<T>(s[0], qa[ks][0], kHi ? qa[ks][1] : 0u, qa[ks][2], kHi ? qa[ks][3] : 0u, kb[0], kb[1], s[0]);
        mma_16816<T>(s[1], qa[ks][0], kHi ? qa[ks][1] : 0u, qa[ks][2], kHi ? qa[ks][3] : 0u, kb[2], kb[3], s[1]);
      }
      // lane (g, j) holds, for heads g (s[.][0..1]) and g+8 (s[.][2..3]), the rows nt*8 + 2j + {0, 1}
      float mt_lo = neg_inf(), mt_hi = neg_inf();
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool ok = (live >> (nt * 8 + 2 * j + e)) & 1u;
          s[nt][e] = ok ? s[nt][e] * p.scale_log2 : neg_inf();
          s[nt][2 + e] = ok ? s[nt][2 + e] * p.scale_log2 : neg_inf();
          mt_lo = fmaxf(mt_lo, s[nt][e]);
          mt_hi = fmaxf(mt_hi, s[nt][2 + e]);
        }
      mt_lo = fmaxf(mt_lo, __shfl_xor_sync(0xffffffffu, mt_lo, 1));
      mt_lo = fmaxf(mt_lo, __shfl_xor_sync(0xffffffffu, mt_lo, 2));
      if (kHi) {
        mt_hi = fmaxf(mt_hi, __shfl_xor_sync(0xffffffffu, mt_hi, 1));
        mt_hi = fmaxf(mt_hi, __shfl_xor_sync(0xffffffffu, mt_hi, 2));
      }
      const float mn_lo = fmaxf(m_lo, mt_lo), mn_hi = fmaxf(m_hi, mt_hi);
      if (mn_lo > m_lo) {
        const float alpha = fast_exp2(m_lo - mn_lo);
        l_lo *= alpha;
#pragma unroll
        for (int u = 0; u < 16; ++u) { o[u][0] *= alpha; o[u][1] *= alpha; }
        m_lo = mn_lo;
      }
      if (kHi && mn_hi > m_hi) {
        const float alpha = fast_exp2(m_hi - mn_hi);
        l_hi *= alpha;
#pragma unroll
        for (int u = 0; u < 16; ++u) { o[u][2] *= alpha; o[u][3] *= alpha; }
        m_hi = mn_hi;
      }
      // weights, split into a 16-bit value and a 16-bit residual: A fragments of P[16 heads, 16 rows]
      // (a0: head g, rows 2j..; a1: head g+8, rows 2j..; a2: head g, rows 8+2j..; a3: head g+8, rows 8+2j..)
      uint32_t pa[4], pr[4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const float w0 = fast_exp2(s[nt][0] - m_lo), w1 = fast_exp2(s[nt][1] - m_lo);   // -inf gives 0
        l_lo += w0 + w1;
        pa[2 * nt] = pack2<T>(w0, w1);
        const float2 back = unpack2<T>(pa[2 * nt]);
        pr[2 * nt] = pack2<T>(w0 - back.x, w1 - back.y);
        if (kHi) {
          const float x0 = fast_exp2(s[nt][2] - m_hi), x1 = fast_exp2(s[nt][3] - m_hi);
          l_hi += x0 + x1;
          pa[2 * nt + 1] = pack2<T>(x0, x1);
          const float2 bk = unpack2<T>(pa[2 * nt + 1]);
          pr[2 * nt + 1] = pack2<T>(x0 - bk.x, x1 - bk.y);
        } else {
          pa[2 * nt + 1] = 0u;
          pr[2 * nt + 1] = 0u;
        }
      }
      // O += P . V, sixteen dims (two n-tiles) per ldmatrix
#pragma unroll
      for (int dn = 0; dn < 8; ++dn) {
        uint32_t vb[4];                                // dims 16dn..+7: rows 0-7, rows 8-15; dims 16dn+8..+15: the same
        ldmatrix_x4_trans(vb, vt + tile_offset((mm & 1) * 8 + rr, 2 * dn + (mm >> 1)));
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int u = 2 * dn + half;
          if (kHi) {
            mma_16816<T>(o[u], pa[0], pa[1], pa[2], pa[3], vb[2 * half], vb[2 * half + 1], o[u]);
            mma_16816<T>(o[u], pr[0], pr[1], pr[2], pr[3], vb[2 * half], vb[2 * half + 1], o[u]);
          } else {
            // rows 8..15 of the M dimension are unused: feed zeros, drop what comes back
            float acc[4] = {o[u][0], o[u][1], 0.f, 0.f};
            mma_16816<T>(acc, pa[0], 0u, pa[2], 0u, vb[2 * half], vb[2 * half + 1], acc);
            mma_16816<T>(acc, pr[0], 0u, pr[2], 0u, vb[2 * half], vb[2 * half + 1], acc);
            o[u][0] = acc[0];
            o[u][1] = acc[1];
          }
        }
      }
    }
    cp_async_wait<0>();                                // only empty groups can be pending here
  }
  if (p.dev_status && kvh == 0) {
    const uint32_t f = (tid == 0 && chunk_id == 0) ? flags : (flags & SSA_DEV_BAD_INDEX);
    if (f) atomicOr(p.dev_status, f);
  }

  if (!p.early_release) grid_launch_dependents();

  // per-warp triples -> shared memory (the ring is free now)
  __syncthreads();
  float (*s_acc)[kLiveHeads][D + kGqaPad] = reinterpret_cast<float (*)[kLiveHeads][D + kGqaPad]>(s_ring);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  if (kHi) {
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  }
#pragma unroll
  for (int u = 0; u < 16; ++u) {
    *reinterpret_cast<float2*>(&s_acc[warp][g][8 * u + 2 * j]) = make_float2(o[u][0], o[u][1]);
    if (kHi) *reinterpret_cast<float2*>(&s_acc[warp][g + 8][8 * u + 2 * j]) = make_float2(o[u][2], o[u][3]);
  }
  if (j == 0) {
    s_m[warp][g] = m_lo; s_l[warp][g] = l_lo;
    if (kHi) { s_m[warp][g + 8] = m_hi; s_l[warp][g + 8] = l_hi; }
  }
  __syncthreads();
  // thread d finishes dim d of every head
  if (tid >= D) return;
  for (int i = 0; i < G; ++i) {
    const int h = kvh * G + i;
    float M = neg_inf();
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w][i]);
    float L = 0.f, A = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float wgt = (s_m[w][i] > neg_inf()) ? fast_exp2(s_m[w][i] - M) : 0.f;
      L = fmaf(s_l[w][i], wgt, L);
      A = fmaf(s_acc[w][i][tid], wgt, A);
    }
    if (p.n_chunks == 1) {
      store_out<T>(p, b, h, tid, L > 0.f ? A / L : 0.f);
      if (tid == 0 && p.lse) p.lse[(int64_t)b * p.H + h] = L > 0.f ? (M + log2f(L)) * kLn2 : neg_inf();
    } else {
      const int64_t slot = ((int64_t)b * p.H + h) * p.n_chunks + chunk_id;
      p.ws_acc[slot * D + tid] = A;
      if (tid == 0) p.ws_ml[slot] = make_float2(M, L);
    }
  }
}

}  // namespace ssa
