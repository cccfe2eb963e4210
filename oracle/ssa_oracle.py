"""Plain fp64 CPU statement of span-restricted decode attention.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product path.  It shares no code
with the CUDA library (own storage decoders, own status constants).

What is stated here, and where the paper defines it:

* ``spans_to_index``      the set of context positions a request may attend
                          to, as the sorted list of positions covered by its
                          token spans (Sec. "Self-selected attention span":
                          groups of contiguous tokens; Sec. "CUDA Kernel
                          Design": the span may be non-contiguous, and a
                          per-token binary mask records what is attended).
* ``attn_set_form``       masked attention for the single query row of a
                          decode step (Background, equations for S, A and O;
                          "Token generation": one row of S and A per step),
                          with the mask 0 on the selected set and -inf
                          elsewhere.
* ``attn_dense``          the same with every position kept.
* ``attn_additive_mask``  the background equations taken literally: all
                          scores, plus a 0/-inf mask, softmax, times V.
* ``attn_alg1_blocked``   Algorithm 1 (blocked span encoding: block index +
                          block bitmask, empty blocks omitted) with the
                          readings listed below.
* ``spans_to_blockmask``  the paper's blocked span encoding (Sec. "CUDA Kernel
                          Design", Attention span encoding): block index and
                          block bitmask of every block of ``bs`` positions that
                          holds a selected position, empty blocks omitted;
                          ``blockmask_to_index`` is its decoding.
* ``resolve_references``  anchors and references to token spans (Sec.
                          "Self-selected attention span": anchors identify
                          groups of contiguous tokens, the model names anchors,
                          generation attends to the named groups; the worked
                          examples of the arithmetic and summarization figures:
                          "[-1]" is the previous line, the instruction is always
                          attended, the line being generated attends to itself).
                          The paper gives no algorithm; the rules are stated in
                          the function.
* ``decode_attn_sparse_multiq``  several query rows per head over one
                          selected set (outside the paper, which decodes one
                          token per step): the set form applied row by row.
* ``decode_e4m3``         the 8-bit cache storage format (outside the paper),
                          from the format's definition.
* ``merge_partials``      recombination of (max, sum, accumulator) partial
                          results of disjoint subsets; not in the paper (its
                          kernel runs one thread block per head and request),
                          it is the algebra of the softmax itself.

Readings of Algorithm 1 where its printed form cannot be taken literally:
  - the mask conversion on the block bitmask is read from the prose next to
    it: bit 1 adds 0 to the score, bit 0 adds -inf;
  - scores of blocks absent from the metadata are -inf (the text says
    attention is computed only over the selected span), not the initial 0;
  - the output is a d-vector accumulated over all selected tokens
    (O = A V), not an n-vector assigned per token;
  - whether the metadata holds a bitmask or start/end offsets inside the
    block is immaterial to the result; the bitmask form is used.
The softmax scale is exposed as an argument; callers pass 1/sqrt(head_dim).
An empty selection (never produced by the method, which always keeps the
instruction and the previous line) yields a zero row and lse = -inf.

Pins (tests marked "not gpu"): hand-enumerated index lists and a set
brute force; the worked anchor/reference examples of the paper as span
structure; closed forms of the softmax (one token, two tokens, uniform
weights, weights 1/6 2/6 3/6); agreement of the three formulations above;
a library scaled-dot-product attention in fp64; convexity, shift, permutation
and split/merge invariants; independence from unselected rows.
"""
from __future__ import annotations

import numpy as np

# Status bits a span list can raise (diagnostics; the index list itself always
# follows the set definition).
ST_BAD_SPAN = 1    # start < 0 or start > end
ST_CLIPPED = 2     # end > context length
ST_OVERFLOW = 4    # more selected positions than the index row can hold
ST_BAD_REF = 64    # a reference named an anchor or line that does not exist


# --------------------------------------------------------------------------
# storage decoders (16-bit patterns -> float64, exact)
# --------------------------------------------------------------------------
def decode_bits(u16, dtype: str) -> np.ndarray:
    """Exact value of 16-bit storage patterns as float64.

    ``bf16``: the pattern is the upper half of an IEEE binary32.
    ``f16`` : IEEE binary16.
    ``e4m3``: 8-bit patterns (uint8), see ``decode_e4m3``.
    """
    if dtype == "e4m3":
        return decode_e4m3(u16)
    a = np.ascontiguousarray(u16)
    if a.dtype != np.uint16:
        raise TypeError("expected uint16 bit patterns")
    if dtype == "bf16":
        with np.errstate(invalid="ignore"):      # signalling NaN patterns
            return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    if dtype == "f16":
        return a.view(np.float16).astype(np.float64)
    raise ValueError(f"unknown storage dtype {dtype!r}")


def decode_e4m3(u8) -> np.ndarray:
    """Exact value of 8-bit "e4m3" storage patterns (1 sign bit, 4 exponent
    bits with bias 7, 3 mantissa bits; the format has no infinities and its
    only NaN is exponent 15 with mantissa 7) as float64, written out from the
    format's definition bit field by bit field:
      exponent 0      : (mantissa / 8) * 2^-6           (subnormal, and zero)
      otherwise       : (1 + mantissa / 8) * 2^(exponent - 7), up to 448.
    The paper stores the cache in 16 bits; 8-bit storage is outside it."""
    a = np.ascontiguousarray(u8)
    if a.dtype != np.uint8:
        raise TypeError("expected uint8 bit patterns")
    sign = np.where(a >> 7, -1.0, 1.0)
    e = ((a >> 3) & 0xF).astype(np.int64)
    m = (a & 0x7).astype(np.float64)
    val = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    val = np.where((e == 15) & ((a & 0x7) == 7), np.nan, val)
    return sign * val


# --------------------------------------------------------------------------
# spans -> index list
# --------------------------------------------------------------------------
def spans_to_index(spans, n: int) -> np.ndarray:
    """Sorted positions j in [0, n) covered by at least one span [s, e).

    Definition by marking: a per-position boolean "may attend" array is
    filled span by span and the marked positions are emitted in increasing
    order.  Order, overlap and repetition of spans therefore cannot matter.
    """
    n = int(n)
    mark = np.zeros(max(n, 0), dtype=bool)
    for s, e in np.asarray(spans, dtype=np.int64).reshape(-1, 2):
        lo = max(int(s), 0)
        hi = min(int(e), n)
        if hi > lo:
            mark[lo:hi] = True
    return np.flatnonzero(mark).astype(np.int32)


def spans_status(spans, n: int, index_stride: int | None = None) -> int:
    """Diagnostic bits for one request's span list (see ST_* above)."""
    st = 0
    for s, e in np.asarray(spans, dtype=np.int64).reshape(-1, 2):
        if s < 0 or s > e:
            st |= ST_BAD_SPAN
        if e > n:
            st |= ST_CLIPPED
    if index_stride is not None and len(spans_to_index(spans, n)) > index_stride:
        st |= ST_OVERFLOW
    return st


def spans_to_index_batch(span_offsets, spans, ctx_lens, index_stride: int):
    """Batch form with the padded row layout of the library interface.

    Returns (index[B, index_stride] int32 filled with -1 past the count,
    counts[B] int32, status bits OR-ed over the batch).  A request whose list
    is longer than ``index_stride`` keeps its first ``index_stride`` positions.
    """
    span_offsets = np.asarray(span_offsets, dtype=np.int64)
    spans = np.asarray(spans, dtype=np.int64).reshape(-1, 2)
    B = len(ctx_lens)
    index = np.full((B, index_stride), -1, dtype=np.int32)
    counts = np.zeros(B, dtype=np.int32)
    status = 0
    for b in range(B):
        sp = spans[span_offsets[b]:span_offsets[b + 1]]
        idx = spans_to_index(sp, int(ctx_lens[b]))
        status |= spans_status(sp, int(ctx_lens[b]), index_stride)
        c = min(len(idx), index_stride)
        index[b, :c] = idx[:c]
        counts[b] = c
    return index, counts, status


# --------------------------------------------------------------------------
# attention for one (request, head): q[D], K[n, D], V[n, D] in float64
# --------------------------------------------------------------------------
def attn_partial(q, K, V, idx, scale: float):
    """(m, l, acc) over the positions ``idx``: m = max score,
    l = sum exp(score - m), acc[d] = sum exp(score - m) V[j, d]."""
    idx = np.asarray(idx, dtype=np.int64)
    D = V.shape[-1]
    if idx.size == 0:
        return -np.inf, 0.0, np.zeros(D)
    s = scale * (K[idx] @ q)
    m = float(np.max(s))
    w = np.exp(s - m)
    return m, float(np.sum(w)), w @ V[idx]


def attn_set_form(q, K, V, idx, scale: float):
    """out[d] = sum_j softmax_j(scale q.K_j) V[j, d] over j in ``idx``;
    lse = log sum_j exp(scale q.K_j).  Rows outside ``idx`` are never read."""
    m, l, acc = attn_partial(q, K, V, idx, scale)
    if l == 0.0:
        return np.zeros(V.shape[-1]), -np.inf
    return acc / l, m + np.log(l)


def attn_dense(q, K, V, n: int, scale: float):
    """Every position 0..n-1 kept (the full-context step)."""
    D = V.shape[-1]
    if n <= 0:
        return np.zeros(D), -np.inf
    s = (K[:n] @ q) * scale
    m = np.max(s)
    a = np.exp(s - m)
    z = np.sum(a)
    return (a / z) @ V[:n], float(m + np.log(z))


def attn_additive_mask(q, K, V, n: int, keep, scale: float):
    """The background equations as printed: S = qK^T scaled, M is 0 where
    attention is permitted and -inf where it is prohibited, A = softmax(M+S),
    O = A V.  ``keep`` is a boolean array over the n positions."""
    keep = np.asarray(keep, dtype=bool)[:n]
    S = (K[:n] @ q) * scale
    M = np.where(keep, 0.0, -np.inf)
    Z = M + S
    zmax = np.max(Z) if n > 0 else -np.inf
    if not np.isfinite(zmax):
        return np.zeros(V.shape[-1]), -np.inf
    E = np.exp(Z - zmax)
    A = E / np.sum(E)
    return A @ V[:n], float(zmax + np.log(np.sum(E)))


def encode_blocked(idx, bs: int):
    """Blocked span encoding: for every block of ``bs`` consecutive positions
    holding at least one selected position, (block index, bs-bit mask of the
    selected positions inside it); empty blocks are omitted."""
    meta = {}
    for j in np.asarray(idx, dtype=np.int64):
        blk, off = divmod(int(j), bs)
        meta.setdefault(blk, np.zeros(bs, dtype=bool))[off] = True
    return [(blk, meta[blk]) for blk in sorted(meta)]


def attn_alg1_blocked(q, K, V, n: int, metadata, bs: int, scale: float):
    """Attention from the blocked span encoding, in the two phases of
    Algorithm 1 (scores of the listed blocks, one softmax over the context,
    weighted sum of the listed blocks' value rows), with the readings stated
    in the module header.  ``metadata``: (block index, boolean mask of ``bs``
    positions) pairs as ``encode_blocked`` returns them."""
    n = max(int(n), 0)
    scores = np.full(n, -np.inf)              # a position of no listed block stays excluded
    listed = []
    for block, mask in metadata:
        first = int(block) * bs
        inside = np.arange(first, min(first + bs, n))
        listed.append(inside)
        # every position of a listed block gets its score; the block's mask then
        # leaves selected positions as they are and sends the others to -inf
        penalty = np.where(np.asarray(mask, dtype=bool)[: len(inside)], 0.0, -np.inf)
        scores[inside] = scale * (K[inside] @ q) + penalty
    top = np.max(scores) if n else -np.inf
    if not np.isfinite(top):
        return np.zeros(V.shape[-1]), -np.inf
    weights = np.exp(scores - top)
    total = np.sum(weights)
    weights = weights / total
    out = np.zeros(V.shape[-1])
    for inside in listed:                     # only listed blocks contribute value rows
        live = inside[weights[inside] != 0.0]  # weight exactly zero: the row is not touched
        out += weights[live] @ V[live]
    return out, float(top + np.log(total))


def resolve_references(lines, anchor_line, refs, prefix_len: int, line_start: int, ctx_len: int,
                       span_stride: int | None = None):
    """Token spans a request attends to while it generates its current line.

    ``lines``       (start, end) of the completed lines (groups) of the context,
                    in order of appearance;
    ``anchor_line`` anchor id -> index into ``lines`` of the line it identifies;
    ``refs``        (lo, hi) pairs.  0 <= lo <= hi: the anchors lo..hi; lo == hi
                    == -k (k >= 1): the k-th line before the current one, i.e.
                    ``lines[len(lines) - k]``.
    Result, in this order: the always-attended prefix [0, prefix_len), the
    current line [line_start, ctx_len), then for each reference in turn one span
    per named line.  References to anchors or lines that do not exist, and
    pairs of any other form, are skipped and flagged.  With ``span_stride`` the
    list is cut to that many spans (flag ST_OVERFLOW) and padded with (0, 0).
    Returns (spans int32 [k, 2], status bits)."""
    lines = np.asarray(lines, dtype=np.int64).reshape(-1, 2)
    out = [(0, int(prefix_len)), (int(line_start), int(ctx_len))]
    status = 0
    for lo, hi in np.asarray(refs, dtype=np.int64).reshape(-1, 2):
        lo, hi = int(lo), int(hi)
        if lo == hi and lo < 0:
            k = len(lines) + lo
            if k < 0:
                status |= ST_BAD_REF
            else:
                out.append(tuple(int(x) for x in lines[k]))
        elif 0 <= lo <= hi:
            for a in range(lo, hi + 1):
                if a >= len(anchor_line) or not (0 <= int(anchor_line[a]) < len(lines)):
                    status |= ST_BAD_REF
                else:
                    out.append(tuple(int(x) for x in lines[int(anchor_line[a])]))
        else:
            status |= ST_BAD_REF
    if span_stride is not None:
        if len(out) > span_stride:
            status |= ST_OVERFLOW
            out = out[:span_stride]
        out = out + [(0, 0)] * (span_stride - len(out))
    return np.asarray(out, dtype=np.int32).reshape(-1, 2), status


def spans_to_blockmask(spans, n: int, bs: int):
    """Blocked encoding of the positions selected by ``spans`` in a context of
    ``n`` rows: (block_idx int32[nb] ascending, words uint32[nb, bs // 32]).
    Bit ``i`` of word ``w`` of a block stands for position
    ``block * bs + 32 * w + i``."""
    if bs % 32 != 0 or bs <= 0:
        raise ValueError("block size must be a positive multiple of 32")
    meta = encode_blocked(spans_to_index(spans, n), bs)
    block_idx = np.array([blk for blk, _ in meta], dtype=np.int32)
    words = np.zeros((len(meta), bs // 32), dtype=np.uint32)
    for r, (_, bm) in enumerate(meta):
        for i in np.flatnonzero(bm):
            words[r, i // 32] |= np.uint32(1) << np.uint32(i % 32)
    return block_idx, words


def blockmask_to_index(block_idx, words, bs: int) -> np.ndarray:
    """Positions named by a blocked encoding, in the order of the list."""
    out = []
    for blk, row in zip(np.asarray(block_idx, dtype=np.int64), np.asarray(words, dtype=np.uint32)):
        for w, word in enumerate(row):
            for i in range(32):
                if (int(word) >> i) & 1:
                    out.append(int(blk) * bs + 32 * w + i)
    return np.asarray(out, dtype=np.int32)


def spans_to_blockmask_batch(span_offsets, spans, ctx_lens, bs: int, block_stride: int):
    """Batch form in the library's padded layout: block_idx[B, block_stride]
    (-1 past the count), words[B, block_stride, bs // 32], counts[B], status
    bits.  A request with more than ``block_stride`` blocks keeps the first."""
    span_offsets = np.asarray(span_offsets, dtype=np.int64)
    spans = np.asarray(spans, dtype=np.int64).reshape(-1, 2)
    B = len(ctx_lens)
    block_idx = np.full((B, block_stride), -1, dtype=np.int32)
    words = np.zeros((B, block_stride, bs // 32), dtype=np.uint32)
    counts = np.zeros(B, dtype=np.int32)
    status = 0
    for b in range(B):
        sp = spans[span_offsets[b]:span_offsets[b + 1]]
        status |= spans_status(sp, int(ctx_lens[b]))
        bi, wd = spans_to_blockmask(sp, int(ctx_lens[b]), bs)
        if len(bi) > block_stride:
            status |= ST_OVERFLOW
        c = min(len(bi), block_stride)
        block_idx[b, :c], words[b, :c], counts[b] = bi[:c], wd[:c], c
    return block_idx, words, counts, status


def merge_partials(ms, ls, accs):
    """Combine partial results of disjoint position subsets:
    m = max m_k, l = sum l_k e^(m_k - m), out = sum acc_k e^(m_k - m) / l."""
    ms = np.asarray(ms, dtype=np.float64)
    ls = np.asarray(ls, dtype=np.float64)
    accs = np.asarray(accs, dtype=np.float64)
    m = np.max(ms) if ms.size else -np.inf
    if not np.isfinite(m):
        return np.zeros(accs.shape[-1]), -np.inf
    f = np.where(np.isfinite(ms), np.exp(ms - m), 0.0)
    l = float(np.sum(ls * f))
    return (f[:, None] * accs).sum(axis=0) / l, float(m + np.log(l))


# --------------------------------------------------------------------------
# batch forms over a KV cache (logical layout [B, H, T, D])
# --------------------------------------------------------------------------
def _as_f64(a, dtype):
    """dtype may name two storage types, "query/cache" (e.g. "bf16/e4m3": 16-bit
    queries over an 8-bit cache); uint8 arrays are always e4m3 patterns."""
    a = np.asarray(a)
    if a.dtype == np.uint8:
        return decode_e4m3(a)
    if a.dtype == np.uint16:
        return decode_bits(a, dtype.split("/")[0])
    return a.astype(np.float64)


def decode_attn_sparse(q, k_cache, v_cache, ctx_lens, index, counts, scale,
                       dtype: str = "bf16", heads=None, seqs=None):
    """Span-restricted decode attention for a batch.

    q[B, H, D]; k_cache, v_cache[B, H, T, D] (uint16 storage patterns of
    ``dtype`` or floats; any numpy strides); index[B, stride] with counts[B]
    valid entries per request, shared by all heads of the request.  Entries
    outside [0, ctx_lens[b]) are skipped.  ``seqs`` / ``heads`` restrict the
    work to a sample; untouched rows of the result are NaN.
    Returns out[B, H, D] float64 and lse[B, H] float64.
    """
    B, H, D = q.shape
    out = np.full((B, H, D), np.nan)
    lse = np.full((B, H), np.nan)
    for b in (range(B) if seqs is None else seqs):
        n = int(ctx_lens[b])
        idx = np.asarray(index[b][: int(counts[b])], dtype=np.int64)
        idx = idx[(idx >= 0) & (idx < n)]
        for h in (range(H) if heads is None else heads):
            qv = _as_f64(q[b, h], dtype)
            # decode only the gathered rows; the others are never touched
            Ks = _as_f64(np.asarray(k_cache[b, h])[idx], dtype)
            Vs = _as_f64(np.asarray(v_cache[b, h])[idx], dtype)
            o, e = attn_set_form(qv, Ks, Vs, np.arange(len(idx)), scale)
            out[b, h] = o
            lse[b, h] = e
    return out, lse


def decode_attn_sparse_multiq(q, k_cache, v_cache, ctx_lens, index, counts, scale, dtype: str = "bf16"):
    """Several query tokens per request and head in one step, all attending
    to the request's one selected set (the paper decodes one token per step,
    "Token generation"; with several, every query row is its own instance of
    the Background equations over the same mask row).

    q[B, H, Tq, D]; cache, lists and conventions as ``decode_attn_sparse``;
    query heads may outnumber cache heads (head h reads cache head
    h // (H / H_kv)).  Returns out[B, H, Tq, D] and lse[B, H, Tq]."""
    B, H, Tq, D = q.shape
    group = H // np.asarray(k_cache).shape[1]
    out = np.full((B, H, Tq, D), np.nan)
    lse = np.full((B, H, Tq), np.nan)
    for b in range(B):
        n = int(ctx_lens[b])
        idx = np.asarray(index[b][: int(counts[b])], dtype=np.int64)
        idx = idx[(idx >= 0) & (idx < n)]
        for h in range(H):
            Ks = _as_f64(np.asarray(k_cache[b, h // group])[idx], dtype)
            Vs = _as_f64(np.asarray(v_cache[b, h // group])[idx], dtype)
            for t in range(Tq):
                out[b, h, t], lse[b, h, t] = attn_set_form(_as_f64(q[b, h, t], dtype), Ks, Vs,
                                                           np.arange(len(idx)), scale)
    return out, lse


def decode_attn_blockmask(q, k_cache, v_cache, ctx_lens, block_idx, words, counts, bs: int, scale,
                          dtype: str = "bf16", heads=None, seqs=None):
    """Span-restricted decode attention from the blocked encoding: the
    positions it names (those inside the context) are attended.  Same
    conventions as ``decode_attn_sparse``."""
    B = q.shape[0]
    stride = max(int(np.max(counts)) * bs if B else 0, 1)
    index = np.full((B, stride), -1, dtype=np.int32)
    cnt = np.zeros(B, dtype=np.int32)
    for b in range(B):
        pos = blockmask_to_index(block_idx[b][: int(counts[b])], words[b][: int(counts[b])], bs)
        index[b, : len(pos)], cnt[b] = pos, len(pos)
    return decode_attn_sparse(q, k_cache, v_cache, ctx_lens, index, cnt, scale, dtype, heads, seqs)


def decode_attn_dense(q, k_cache, v_cache, ctx_lens, scale,
                      dtype: str = "bf16", heads=None, seqs=None):
    """Full-context decode attention for a batch (same conventions)."""
    B, H, D = q.shape
    out = np.full((B, H, D), np.nan)
    lse = np.full((B, H), np.nan)
    for b in (range(B) if seqs is None else seqs):
        n = int(ctx_lens[b])
        for h in (range(H) if heads is None else heads):
            qv = _as_f64(q[b, h], dtype)
            Kf = _as_f64(np.asarray(k_cache[b, h])[:n], dtype)
            Vf = _as_f64(np.asarray(v_cache[b, h])[:n], dtype)
            o, e = attn_dense(qv, Kf, Vf, n, scale)
            out[b, h] = o
            lse[b, h] = e
    return out, lse


def gather_pages(pool, page_table, page_size: int, max_ctx: int) -> np.ndarray:
    """The contiguous cache [B, H, max_ctx, D] that a paged cache stands for.

    ``pool`` [n_pages, page_size, H, D]; ``page_table`` [B, pages per request].
    Logical position t of request b is row t % page_size of page
    page_table[b, t // page_size].  (The paper pre-allocates a contiguous cache
    per request, so paging has no passage there; this is only the definition of
    the layout, after which the attention definitions above apply unchanged.)
    Positions whose page id lies outside the pool are left zero; a test must not
    select them when it compares with this function's result.
    """
    pool = np.asarray(pool)
    page_table = np.asarray(page_table)
    B = page_table.shape[0]
    n_pages, ps, H, D = pool.shape
    assert ps == page_size
    cache = np.zeros((B, H, max_ctx, D), dtype=pool.dtype)
    for b in range(B):
        for t in range(max_ctx):
            page = int(page_table[b, t // page_size])
            if 0 <= page < n_pages:
                cache[b, :, t, :] = pool[page, t % page_size]
    return cache
