// Pass 1 of the decode attention for grouped query heads (G = H / H_kv query
// heads share one K/V head, 2 <= G <= 16, D = 128): one block per (chunk,
// K/V head, request) reads every selected row ONCE and serves all G heads.
//
// With G heads per row the work per byte is G times that of multi-head
// attention and the packed-FMA path of decode_partial_kernel runs out of issue
// slots before it runs out of HBM bandwidth, so here the two contractions go
// to the tensor cores.  The shapes are far too small for tcgen05 tiles (G x 16
// rows x 128), so they are warp-level mma.sync.m16n8k16 (16-bit inputs, fp32
// accumulation) with the M dimension holding the query heads:
//   S[16 heads, 16 rows]  = Q[16, 128] . K_tile^T          (2 x 8 mma)
//   O[16 heads, 128 dims] += P[16, 16] . V_tile[16, 128]   (16 mma, twice)
// Operands come straight from global memory into the fragment registers, no
// shared-memory staging and no ldmatrix: a dot product does not care in which
// order the dimensions are visited, so the k index of the mma is mapped to
// the head dimension such that every lane needs CONTIGUOUS bytes of a row:
//   Q/K:  lane (g = lane/4, j = lane%4) holds dims [32j, 32j+32) of head g
//         (and g+8) / of row g of each 8-row half of the tile; k-step s uses
//         its dims 32j+4s .. 32j+4s+3.
//   V:    lane (g, j) holds dims [16g, 16g+16) of tile rows 2j, 2j+1, 2j+8,
//         2j+9; n-tile u takes dim 16g+u, the two rows of a k pair are
//         interleaved with one byte-permute each.
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

__device__ __forceinline__ uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

constexpr int kGqaRows = 16;            // rows per warp per iteration
constexpr int kGqaHeads = 16;           // M of the mma: most query heads one block serves
constexpr int kGqaPad = 4;              // floats of padding per head row of the block-level combine

// kHi: more than 8 query heads per K/V head (rows 8..15 of the M dimension are live).
template <typename T, int kMode, bool kHi, bool kAligned32>
__global__ void __launch_bounds__(kThreads, kHi ? 2 : 3)
decode_partial_gqa_kernel(const DecodeParams p) {
  constexpr int D = 128;
  constexpr bool kSparse = kMode != kDense;
  constexpr int kLiveHeads = kHi ? 16 : 8;
  static_assert(kMode == kDense || kMode == kIndex || kMode == kSpans,
                "blocked lists take the one-head-per-block kernel");

  __shared__ int32_t s_idx[kSparse ? kMaxChunk : 1];
  __shared__ __align__(16) float s_acc[kWarps][kLiveHeads][D + kGqaPad];
  __shared__ float s_m[kWarps][kLiveHeads], s_l[kWarps][kLiveHeads];
  __shared__ uint32_t s_q[kHi ? 32 : 16][32];         // query fragments, [word][lane]: the same for every warp
  __shared__ typename std::conditional<kMode == kSpans, SpanRuns, int>::type s_runs;

  const int chunk_id = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, j = lane & 3;
  const int G = p.kv_group;
  const int start = chunk_id * p.chunk;

  grid_dependency_wait();
  if (p.early_release) grid_launch_dependents();

  uint32_t flags = 0;
  int n, c;
  request_sizes(p, b, n, c, flags);
  if constexpr (kMode == kSpans) {
    // the request's spans -> disjoint ascending runs in shared memory
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

  // A block may own more list entries than the staging area holds: it works through them in windows of
  // kMaxChunk entries (checked, translated for a paged cache, staged, consumed).
  auto stage_window = [&](int w0, int wn) {
    if constexpr (kMode == kSpans) {                  // positions by arithmetic on the runs
      int32_t* out = (kvh == 0 && p.index_out) ? p.index_out + (int64_t)b * p.index_stride + start + w0 : nullptr;
      for (int i = tid; i < wn; i += kThreads) {
        const int v = span_position(s_runs, start + w0 + i);
        s_idx[i] = v;
        if (out) out[i] = v;
      }
      return;
    }
    const int32_t* row = p.index ? p.index + (int64_t)b * p.index_stride + start + w0 : nullptr;
    for (int i = tid; i < wn; i += kThreads) {
      int v = row ? __ldg(row + i) : start + w0 + i;
      if (v < 0 || v >= n) {
        v = -1; flags |= SSA_DEV_BAD_INDEX;
      } else if (p.page_table) {
        const int page = __ldg(p.page_table + (int64_t)b * p.page_table_stride + (v >> p.page_shift));
        if ((unsigned)page < (unsigned)p.n_pages) v = (page << p.page_shift) | (v & p.page_mask);
        else { v = -1; flags |= SSA_DEV_BAD_INDEX; }
      }
      s_idx[i] = v;
    }
  };
  if (kSparse) stage_window(0, min(cnt, kMaxChunk));
  // query fragments: dims [32j, 32j+32) of heads g and g+8 of this K/V head.  They are the same for all
  // warps and live in shared memory: sixteen registers per lane are worth a third block per SM here.
  if (warp == 0) {
    const T* q0 = reinterpret_cast<const T*>(p.q) + (int64_t)b * p.q_sb + (int64_t)(kvh * G) * p.q_sh + 32 * j;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 a = make_uint4(0u, 0u, 0u, 0u), h8 = make_uint4(0u, 0u, 0u, 0u);
      if (g < G) a = ld_stream_16B(q0 + (int64_t)g * p.q_sh + 8 * i);
      if (kHi && g + 8 < G) h8 = ld_stream_16B(q0 + (int64_t)(g + 8) * p.q_sh + 8 * i);
      s_q[4 * i][lane] = a.x; s_q[4 * i + 1][lane] = a.y; s_q[4 * i + 2][lane] = a.z; s_q[4 * i + 3][lane] = a.w;
      if (kHi) {
        s_q[16 + 4 * i][lane] = h8.x; s_q[16 + 4 * i + 1][lane] = h8.y;
        s_q[16 + 4 * i + 2][lane] = h8.z; s_q[16 + 4 * i + 3][lane] = h8.w;
      }
    }
  }
  __syncthreads();
  const char* kbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.k) + (int64_t)b * p.k_sb + (int64_t)kvh * p.k_sh + 32 * j);
  const char* vbase = reinterpret_cast<const char*>(
      reinterpret_cast<const T*>(p.v) + (int64_t)b * p.v_sb + (int64_t)kvh * p.v_sh + 16 * g);

  // running softmax state of heads g (lo) and g+8 (hi); sums are per lane until the end
  float m_lo = neg_inf(), m_hi = neg_inf(), l_lo = 0.f, l_hi = 0.f;
  float o[16][4];
#pragma unroll
  for (int u = 0; u < 16; ++u) { o[u][0] = 0.f; o[u][1] = 0.f; o[u][2] = 0.f; o[u][3] = 0.f; }

  for (int w0 = 0; w0 < cnt; w0 += kMaxChunk) {
  const int wn = min(kMaxChunk, cnt - w0);
  if (kSparse && w0 > 0) {
    __syncthreads();                                   // every warp is done with the previous window
    stage_window(w0, wn);
    __syncthreads();
  }
  for (int t = warp * kGqaRows; t < wn; t += kWarps * kGqaRows) {
    // which of the tile's 16 rows exist (lane r and r+16 both answer for row r)
    int my_pos = -1;
    {
      const int r = t + (lane & 15);
      if (r < wn) my_pos = kSparse ? s_idx[r] : start + w0 + r;
    }
    const uint32_t live = __ballot_sync(0xffffffffu, my_pos >= 0) & 0xffffu;
    auto row_pos = [&](int r) { return __shfl_sync(0xffffffffu, my_pos, r); };

    // K: row g of each half (64 bytes per lane per row); V: rows 2j, 2j+1, 2j+8, 2j+9 (32 bytes each)
    uint32_t kf[2][16], vf[4][8];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int pos = row_pos(nt * 8 + g);
      if (pos >= 0) {
        const char* src = kbase + (uint64_t)(uint32_t)pos * p.k_row_bytes;
#pragma unroll
        for (int i = 0; i < 2; ++i) {                 // whole 32-byte sectors per request
          Piece pc;
          load_piece<kAligned32>(pc, src + 32 * i);
#pragma unroll
          for (int w = 0; w < 8; ++w) kf[nt][8 * i + w] = pc.w[w];
        }
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) kf[nt][i] = 0u;
      }
    }
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      const int pos = row_pos(2 * j + (rr & 1) + 8 * (rr >> 1));
      if (pos >= 0) {
        const char* src = vbase + (uint64_t)(uint32_t)pos * p.v_row_bytes;
        Piece pc;
        load_piece<kAligned32>(pc, src);
#pragma unroll
        for (int w = 0; w < 8; ++w) vf[rr][w] = pc.w[w];
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) vf[rr][i] = 0u;          // weight 0 times anything stored there must stay 0
      }
    }

    // S = Q . K^T for the two 8-row halves
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        mma_16816<T>(s[nt], s_q[2 * ks][lane], kHi ? s_q[16 + 2 * ks][lane] : 0u, s_q[2 * ks + 1][lane],
                     kHi ? s_q[16 + 2 * ks + 1][lane] : 0u, kf[nt][2 * ks], kf[nt][2 * ks + 1], s[nt]);
    }
    // lane (g, j) now holds, for heads g (s[.][0..1]) and g+8 (s[.][2..3]), the rows nt*8 + 2j + {0, 1}
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
    if (live == 0u) continue;                          // warp-uniform: nothing to add
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
    // weights, split into a 16-bit value and a 16-bit residual; A fragments of P[16 heads, 16 rows]
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
    // O += P . V, one n-tile (8 of this lane group's dims) at a time
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const uint32_t sel = (u & 1) ? 0x7632u : 0x5410u;
      const uint32_t b0 = byte_perm(vf[0][u >> 1], vf[1][u >> 1], sel);
      const uint32_t b1 = byte_perm(vf[2][u >> 1], vf[3][u >> 1], sel);
      if (kHi) {
        mma_16816<T>(o[u], pa[0], pa[1], pa[2], pa[3], b0, b1, o[u]);
        mma_16816<T>(o[u], pr[0], pr[1], pr[2], pr[3], b0, b1, o[u]);
      } else {
        // rows 8..15 of the M dimension are unused: feed zeros, drop what comes back
        float acc[4] = {o[u][0], o[u][1], 0.f, 0.f};
        mma_16816<T>(acc, pa[0], 0u, pa[2], 0u, b0, b1, acc);
        mma_16816<T>(acc, pr[0], 0u, pr[2], 0u, b0, b1, acc);
        o[u][0] = acc[0];
        o[u][1] = acc[1];
      }
    }
  }

  }                                                    // windows
  if (p.dev_status && kvh == 0) {
    const uint32_t f = (tid == 0 && chunk_id == 0) ? flags : (flags & SSA_DEV_BAD_INDEX);
    if (f) atomicOr(p.dev_status, f);
  }

  if (!p.early_release) grid_launch_dependents();

  // per-warp triples -> shared memory.  o[u][e] of lane (g, j) is dim 32j + 16e + u of head g (+8 for e+2).
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  if (kHi) {
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  }
#pragma unroll
  for (int u = 0; u < 16; ++u) {
    s_acc[warp][g][32 * j + u] = o[u][0];
    s_acc[warp][g][32 * j + 16 + u] = o[u][1];
    if (kHi) {
      s_acc[warp][g + 8][32 * j + u] = o[u][2];
      s_acc[warp][g + 8][32 * j + 16 + u] = o[u][3];
    }
  }
  if (j == 0) {
    s_m[warp][g] = m_lo; s_l[warp][g] = l_lo;
    if (kHi) { s_m[warp][g + 8] = m_hi; s_l[warp][g + 8] = l_hi; }
  }
  __syncthreads();
  // thread d finishes dim d of every head
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
