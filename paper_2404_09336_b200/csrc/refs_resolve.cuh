// Resolution of one request's references into token spans, shared by
// ssa_refs_to_spans (spans written to global memory) and ssa_refs_to_index
// (spans kept in shared memory and expanded at once).
#pragma once
#include "ssa_common.cuh"

namespace ssa {

// Called by all 32 lanes of one warp for request b.  Span 0 is the
// instruction prefix, span 1 the line being generated; then the lanes take the
// references 32 at a time: each lane resolves one (lo, hi) pair to a first
// line and a count of lines, a shuffle prefix sum turns the counts into output
// positions, and the lane hands its spans to put(position, span).  Returns the
// number of spans the request resolves to (put decides what to do with
// positions beyond its capacity).
template <typename Put>
__device__ __forceinline__ int resolve_refs_warp(const ssa_anchor_tables& t, int b, int lane, uint32_t& flags,
                                                 Put put) {
  const int l0 = t.line_offsets[b], n_lines = max(t.line_offsets[b + 1] - l0, 0);
  const int a0 = t.anchor_offsets[b], n_anchors = max(t.anchor_offsets[b + 1] - a0, 0);
  const int r0 = t.ref_offsets[b], n_refs = max(t.ref_offsets[b + 1] - r0, 0);
  const int2* lines = reinterpret_cast<const int2*>(t.lines) + l0;
  const int2* refs = reinterpret_cast<const int2*>(t.refs) + r0;
  if (lane == 0) {
    put(0, make_int2(0, t.prefix_len[b]));
    put(1, make_int2(t.line_start[b], t.ctx_lens[b]));
  }
  int written = 2;
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
        // anchors past the end of the table do not exist: flag them and walk only the ones that do, so the
        // work per reference is bounded by the table whatever the pair says
        int hi = ref.y;
        if (hi >= n_anchors) { hi = n_anchors - 1; flags |= SSA_DEV_BAD_REF; }
        first = ref.x;
        count = max(hi - ref.x + 1, 0);
        by_anchor = true;
      } else {
        flags |= SSA_DEV_BAD_REF;
      }
    }
    // anchors that do not resolve are dropped, so count what each lane really emits (table reads four at a
    // time: a lane's walk over its anchors is a chain of dependent-looking loads otherwise)
    int emit = 0;
    if (by_anchor) {
      for (int a = first; a < first + count; a += 4) {
        int li[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          li[k] = (a + k < first + count && a + k < n_anchors) ? __ldg(t.anchor_line + a0 + a + k) : -1;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (a + k >= first + count) break;
          if (li[k] >= 0 && li[k] < n_lines) ++emit; else flags |= SSA_DEV_BAD_REF;
        }
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
      for (int a = first; a < first + count; a += 4) {
        int li[4];
        int2 span[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          li[k] = (a + k < first + count && a + k < n_anchors) ? __ldg(t.anchor_line + a0 + a + k) : -1;
#pragma unroll
        for (int k = 0; k < 4; ++k)
          span[k] = (li[k] >= 0 && li[k] < n_lines) ? __ldg(lines + li[k]) : make_int2(0, 0);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (li[k] >= 0 && li[k] < n_lines) put(at++, span[k]);
      }
    } else if (count == 1) {
      put(at, lines[first]);
    }
    written += __shfl_sync(0xffffffffu, incl, 31);
  }
  return written;
}

// Host-side check of the tables shared by both entry points.
inline int32_t check_anchor_tables(const ssa_anchor_tables* t) {
  if (!t) return SSA_ERR_NULL;
  if (!t->line_offsets || !t->lines || !t->anchor_offsets || !t->anchor_line || !t->ref_offsets || !t->refs ||
      !t->prefix_len || !t->line_start || !t->ctx_lens)
    return SSA_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(t->lines) % 8 || reinterpret_cast<uintptr_t>(t->refs) % 8) return SSA_ERR_ALIGN;
  return SSA_OK;
}

}  // namespace ssa
