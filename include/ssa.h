/*
 * ssa.h - span-restricted ("self-selected attention span") decode attention
 *         for NVIDIA B200 (sm_100a).  C ABI of libssa.
 *
 * One decode step of the method: every request of a batch attends, with its
 * single query row per head, only to the KV-cache rows of the token spans
 * currently selected for it (Sec. "Self-selected attention span", "Token
 * generation"; Sec. "CUDA Kernel Design").  The result is exactly masked
 * attention (Background: S = q K^T / sqrt(d), A = softmax(M + S), O = A V)
 * with M = 0 on the selected positions and -inf elsewhere.
 *
 * General conventions
 *  - Every pointer marked "dev" is a DEVICE pointer owned by the caller; the
 *    library never allocates or frees device memory, and keeps none between
 *    calls except the fixed array named at ssa_decode_attn_sparse_noalloc.
 *    Pointers marked "host" are ordinary host pointers read during the call.
 *  - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *    the default stream).  No call synchronises or reads device memory back,
 *    so everything data-dependent (selected counts, context lengths) stays on
 *    the device and host-side sizes are upper bounds.
 *  - Return value: an ssa_status.  Non-zero means nothing was launched.
 *  - Data-dependent problems never fault: they set bits in the caller's
 *    device status word (`dev_status`, may be NULL) and take the defined
 *    fallback (clip / skip / truncate).
 *  - Selection is per request and shared by all heads of the request (the
 *    paper keeps separate metadata per request of a batch).
 */
#ifndef SSA_H_
#define SSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SSA_OK = 0,
  SSA_ERR_NULL = 1,        /* a required pointer is NULL                          */
  SSA_ERR_SHAPE = 2,       /* a size is non-positive or out of the supported range */
  SSA_ERR_DTYPE = 3,       /* unsupported kv_dtype / out_dtype                     */
  SSA_ERR_ALIGN = 4,       /* pointer or stride not 16-byte aligned                */
  SSA_ERR_CAPACITY = 5,    /* index_stride / max_selected inconsistent             */
  SSA_ERR_WORKSPACE = 6,   /* workspace missing or too small                       */
  SSA_ERR_CUDA = 7,        /* a CUDA runtime call or launch failed                 */
  SSA_ERR_UNSUPPORTED = 8  /* valid request outside the implemented set            */
} ssa_status;

/* Bits OR-ed into *dev_status by kernels. */
enum {
  SSA_DEV_BAD_SPAN = 1,    /* a span had start < 0 or start > end                  */
  SSA_DEV_CLIPPED = 2,     /* a span had end > ctx_len and was clipped             */
  SSA_DEV_OVERFLOW = 4,    /* a request selected more than index_stride positions;
                              its list was truncated to the first index_stride     */
  SSA_DEV_BAD_INDEX = 8,   /* an index entry was outside [0, ctx_len): skipped     */
  SSA_DEV_BAD_COUNT = 16,  /* counts[b] > max_selected or ctx_lens[b] > max_ctx:
                              clamped                                              */
  SSA_DEV_TOO_MANY_SPANS = 32, /* a request had more than SSA_MAX_SPANS_PER_SEQ
                              spans; the surplus was ignored                       */
  SSA_DEV_BAD_REF = 64     /* a reference named an anchor or line that does not
                              exist, or was malformed: skipped                     */
};

#define SSA_MAX_SPANS_PER_SEQ 2048

typedef enum { SSA_F16 = 0, SSA_BF16 = 1, SSA_F32 = 2, SSA_FP8_E4M3 = 3 } ssa_dtype;

/*
 * Geometry of q, the KV cache and the output.  Strides are in ELEMENTS; the
 * head dimension is contiguous in every tensor.  Both the per-head layout
 * [B, H, T, D] and the token-major layout [B, T, H, D] are expressible.
 *   q   [b, h, :]    at q   + b*q_stride_b + h*q_stride_h
 *   K   [b, t, h, :] at k   + b*k_stride_b + t*k_stride_t + h*k_stride_h
 *   V   likewise with the v_* strides
 *   out [b, h, :]    at out + b*o_stride_b + h*o_stride_h
 * Row t = ctx_lens[b]-1 is the current token's own K/V, appended by the
 * caller before the call; it is attended only if selected.
 * Supported: D in {64, 128}; kv_dtype F16 or BF16 (q has the same type);
 * out_dtype equal to kv_dtype or F32; H_kv == H (multi-head attention, as in
 * the paper's LLaMA-7B) or H_kv dividing H (grouped queries, not in the paper:
 * query head h reads K/V head h / (H/H_kv); the cache then has H_kv heads).
 * Every base pointer and every stride * element size
 * must be a multiple of 16 bytes.
 * kv_dtype SSA_FP8_E4M3 (not in the paper, whose cache is 16-bit): K and V are
 * stored as 8-bit e4m3 values (1 sign, 4 exponent, 3 mantissa bits, bias 7, no
 * infinities), one byte per element, read as they are - a caller that keeps a
 * scale with the cache folds K's into `scale` and applies V's to the output;
 * q is then BF16 and out_dtype BF16 or F32.  Such a cache halves the bytes per
 * selected row; grouped query heads over it are served one head per thread
 * block (each head re-reads the rows, mostly from L2).
 */
typedef struct {
  int32_t B, H, H_kv, D;
  int32_t max_ctx;          /* rows allocated per request in the cache            */
  int32_t kv_dtype;         /* ssa_dtype                                          */
  int32_t out_dtype;        /* ssa_dtype                                          */
  float   scale;            /* softmax scale; <= 0 selects 1/sqrt(D)              */
  int64_t q_stride_b, q_stride_h;
  int64_t k_stride_b, k_stride_t, k_stride_h;
  int64_t v_stride_b, v_stride_t, v_stride_h;
  int64_t o_stride_b, o_stride_h;
} ssa_attn_desc;

/*
 * Span list -> compact KV index list (the "on the fly" conversion of the
 * selected references into an attention mask, Abstract and Sec. "CUDA Kernel
 * Design", Attention span encoding; here the mask is kept as the sorted list
 * of attended positions instead of block bitmasks).
 *
 * For request b with spans (s_i, e_i), i in [span_offsets[b], span_offsets[b+1]):
 *   index[b*index_stride + 0 .. counts[b]) = ascending { j : 0 <= j < ctx_lens[b]
 *                                             and s_i <= j < e_i for some i }.
 * Spans may be unsorted, overlapping, adjacent, repeated or empty: the result
 * is the sorted duplicate-free union.  Entries past counts[b] are left
 * untouched.  start < 0 is clamped to 0 and start > end contributes nothing
 * (both set SSA_DEV_BAD_SPAN); end > ctx_lens[b] is clipped (SSA_DEV_CLIPPED);
 * more than index_stride positions keep the first index_stride
 * (SSA_DEV_OVERFLOW).
 *
 *   span_offsets dev int32 [B+1], non-decreasing, span_offsets[0] >= 0
 *   spans        dev int32 [2 * span_offsets[B]]  (start, end) pairs, 8-byte
 *                aligned, non-NULL even when there are no spans
 *   ctx_lens     dev int32 [B]
 *   index        dev int32 [B * index_stride]     (written)
 *   counts       dev int32 [B]                    (written)
 *   dev_status   dev uint32 [1] or NULL           (bits OR-ed in)
 * Errors: SSA_ERR_NULL, SSA_ERR_SHAPE (B <= 0, B > 65535 or
 * index_stride <= 0), SSA_ERR_ALIGN, SSA_ERR_CUDA.
 */
int32_t ssa_spans_to_index(const int32_t* span_offsets, const int32_t* spans,
                           const int32_t* ctx_lens, int32_t B,
                           int32_t* index, int32_t index_stride,
                           int32_t* counts, uint32_t* dev_status, void* stream);

/*
 * Bytes of device workspace the two attention calls need for `desc` when no
 * request selects more than `max_selected` positions (for the dense call pass
 * desc->max_ctx).  Returns 0 for an invalid descriptor.  The workspace holds
 * the per-split partial results (running max, running sum, fp32 accumulator)
 * of the split-KV pass (the paper's kernel runs one thread block per head and
 * request and has no such step); its contents need no initialisation and are
 * dead after the call's work has run.
 */
size_t ssa_decode_workspace_bytes(const ssa_attn_desc* desc, int32_t max_selected);

/*
 * Span-restricted decode attention (Algorithm 1; Background equations with a
 * 0 / -inf mask): for every request b and head h
 *   s_j = scale * <q[b,h,:], K[b,j,h,:]>          j in the request's index list
 *   out[b,h,:] = sum_j softmax_j(s) * V[b,j,h,:]
 *   lse[b,h]   = log sum_j exp(s_j)               (natural log; optional)
 * computed with fp32 accumulation.  Only the selected rows of K and V are
 * read.  The list is index[b*index_stride .. + counts[b]); entries need not be
 * sorted; a duplicated entry is counted twice; an entry outside
 * [0, ctx_lens[b]) is skipped (SSA_DEV_BAD_INDEX).  counts[b] == 0 gives a
 * zero output row and lse = -inf.  `max_selected` is a host-side upper bound
 * on every counts[b] (1 <= max_selected <= index_stride); a larger count is
 * clamped to it (SSA_DEV_BAD_COUNT).
 *
 *   desc       host
 *   q, k_cache, v_cache  dev, kv_dtype
 *   ctx_lens   dev int32 [B]
 *   index      dev int32 [B * index_stride];  counts dev int32 [B]
 *   out        dev, out_dtype (written);  lse dev float [B*H] or NULL (written)
 *              (both are only ever stored to, once per element, so they may
 *              also be page-locked host memory that the device addresses: a
 *              row then crosses the bus as soon as it is finished)
 *   workspace  dev, >= ssa_decode_workspace_bytes(desc, max_selected) bytes,
 *              16-byte aligned; always required (the size query never returns
 *              0 for a valid descriptor, also when every request fits one
 *              thread block and nothing is written to it)
 * Errors: SSA_ERR_NULL, SSA_ERR_SHAPE, SSA_ERR_DTYPE, SSA_ERR_ALIGN,
 * SSA_ERR_CAPACITY, SSA_ERR_WORKSPACE, SSA_ERR_UNSUPPORTED, SSA_ERR_CUDA.
 */
int32_t ssa_decode_attn_sparse(const ssa_attn_desc* desc, const void* q,
                               const void* k_cache, const void* v_cache,
                               const int32_t* ctx_lens, const int32_t* index,
                               int32_t index_stride, const int32_t* counts,
                               int32_t max_selected, void* out, float* lse,
                               void* workspace, size_t workspace_bytes,
                               uint32_t* dev_status, void* stream);

/*
 * Span-restricted decode attention straight from the span lists: the result of
 * ssa_spans_to_index followed by ssa_decode_attn_sparse, in one kernel and
 * without an index list in memory (Sec. "CUDA Kernel Design": the attention
 * span "might consist of non-contiguous token spans"; Sec. "Self-selected
 * attention span", Token generation; Algorithm 1 with the span list as the
 * metadata).  Every thread block sorts and merges its request's spans in
 * shared memory - the union, exactly as ssa_spans_to_index defines it - and
 * derives the positions of the rows it reads by arithmetic on the merged runs.
 *
 * Same span semantics and status bits as ssa_spans_to_index (unsorted,
 * overlapping, empty, reversed or out-of-range spans), same result and
 * options as ssa_decode_attn_sparse.  Two host-side bounds size the launch:
 *   max_spans     >= the number of spans of any request (a caller knows it: it
 *                 built the lists).  A request with more keeps its first
 *                 max_spans spans (SSA_DEV_TOO_MANY_SPANS).  Up to 128 spans
 *                 per request are merged on chip (up to 32 by every warp for
 *                 itself, without a block barrier); with a larger bound (up to
 *                 SSA_MAX_SPANS_PER_SEQ, beyond which it is treated as that)
 *                 the call expands the lists with the kernel of
 *                 ssa_spans_to_index first and attends through them - two
 *                 launches, same results.
 *   max_selected  >= the number of positions any request attends to.  A
 *                 request with more keeps the first max_selected, in
 *                 ascending order (SSA_DEV_OVERFLOW).
 * Optional outputs, for callers that also want what ssa_spans_to_index would
 * have written (the lists are bit-identical to its output):
 *   index_out   dev int32 [B * index_stride] or NULL; index_stride >=
 *               max_selected when given; entries past the count untouched
 *   counts_out  dev int32 [B] or NULL
 *   span_offsets, spans, ctx_lens  dev, as in ssa_spans_to_index.  span_offsets
 *               may be NULL when max_spans <= 128: the lists are then a table
 *               of exactly max_spans pairs per request (request b owns pairs
 *               b*max_spans .. (b+1)*max_spans - 1, unused ones empty, e.g.
 *               (0, 0) - the layout ssa_refs_to_spans writes), which saves the
 *               blocks one dependent read (SSA_ERR_UNSUPPORTED above 128)
 *   workspace   dev, >= ssa_decode_spans_workspace_bytes(desc, max_selected,
 *               max_spans) bytes, 16-byte aligned, no initialisation needed
 * A paged cache is not supported by this call.
 * Errors: those of ssa_decode_attn_sparse; SSA_ERR_CAPACITY also for
 * max_spans <= 0.
 */
size_t ssa_decode_spans_workspace_bytes(const ssa_attn_desc* desc, int32_t max_selected,
                                        int32_t max_spans);
int32_t ssa_decode_attn_spans(const ssa_attn_desc* desc, const void* q,
                              const void* k_cache, const void* v_cache,
                              const int32_t* ctx_lens, const int32_t* span_offsets,
                              const int32_t* spans, int32_t max_spans,
                              int32_t max_selected, void* out, float* lse,
                              int32_t* index_out, int32_t index_stride,
                              int32_t* counts_out, void* workspace,
                              size_t workspace_bytes, uint32_t* dev_status,
                              void* stream);

/*
 * Full-context decode attention, the baseline the method is compared with
 * (Background equations with M = 0; the paper's "determine attention span"
 * steps attend to all preceding context): as above with the implicit list
 * 0 .. ctx_lens[b]-1 read as one contiguous stream.  ctx_lens[b] > max_ctx is
 * clamped (SSA_DEV_BAD_COUNT).  Workspace: ssa_decode_workspace_bytes(desc,
 * desc->max_ctx).
 */
int32_t ssa_decode_attn_dense(const ssa_attn_desc* desc, const void* q,
                              const void* k_cache, const void* v_cache,
                              const int32_t* ctx_lens, void* out, float* lse,
                              void* workspace, size_t workspace_bytes,
                              uint32_t* dev_status, void* stream);

/*
 * The two attention calls over a PAGED cache (the paper pre-allocates one
 * contiguous cache per request, Experimental results; paging has no
 * counterpart there - it is what serving stacks use to avoid that
 * reservation).  K and V live in pools of n_pages pages of page_size rows;
 * logical position t of request b is pool row
 *     page_table[b * page_table_stride + t / page_size] * page_size + t % page_size,
 * whose head h starts at pool + row * k_stride_t + (h / (H/H_kv)) * k_stride_h
 * elements (desc->k_stride_b / v_stride_b are ignored; a pool laid out
 * [n_pages, page_size, H_kv, D] has k_stride_t = H_kv*D, k_stride_h = D).
 * desc->max_ctx bounds the logical context.  Everything else - index lists,
 * counts, results, workspace size, status bits - is as for
 * ssa_decode_attn_sparse / ssa_decode_attn_dense; a page-table entry outside
 * [0, n_pages) makes the positions it covers be skipped (SSA_DEV_BAD_INDEX).
 * The position -> row translation happens once per block, while it stages its
 * list entries, and costs one extra page-table read per entry.
 *   page_table  dev int32 [B * page_table_stride]
 * Errors as for the unpaged calls, plus SSA_ERR_NULL for a missing paging
 * struct or table and SSA_ERR_SHAPE for page_size not a power of two,
 * n_pages <= 0, n_pages * page_size >= 2^31 or
 * page_table_stride * page_size < desc->max_ctx.
 */
typedef struct {
  const int32_t* page_table;
  int32_t page_table_stride;   /* entries per request */
  int32_t page_size;           /* rows per page, a power of two */
  int32_t n_pages;             /* pages in the pool */
} ssa_paging;

int32_t ssa_decode_attn_sparse_paged(const ssa_attn_desc* desc, const void* q, const void* k_pool,
                                     const void* v_pool, const ssa_paging* paging,
                                     const int32_t* ctx_lens, const int32_t* index,
                                     int32_t index_stride, const int32_t* counts,
                                     int32_t max_selected, void* out, float* lse, void* workspace,
                                     size_t workspace_bytes, uint32_t* dev_status, void* stream);
int32_t ssa_decode_attn_dense_paged(const ssa_attn_desc* desc, const void* q, const void* k_pool,
                                    const void* v_pool, const ssa_paging* paging,
                                    const int32_t* ctx_lens, void* out, float* lse, void* workspace,
                                    size_t workspace_bytes, uint32_t* dev_status, void* stream);

/*
 * Several query tokens per request in one step (the paper decodes one token
 * per step, Sec. "Self-selected attention span", Token generation; this has
 * no counterpart there - it is what speculative or multi-token decoding
 * needs): n_q query rows per head, all attending to the request's ONE
 * selected set, each row its own instance of the Background equations over
 * the same mask row.  Row t of head h is at q + b*q_stride_b + h*q_stride_h +
 * t*q_stride_t, its output at out + b*o_stride_b + h*o_stride_h +
 * t*o_stride_t, its lse at lse[(b*H + h)*n_q + t].  The rows of one head
 * must lie side by side: desc->q_stride_h == n_q*q_stride_t and
 * desc->o_stride_h == n_q*o_stride_t (q and out laid out [B, H, n_q, D]),
 * else SSA_ERR_UNSUPPORTED.  Everything else - desc, cache, lists, counts,
 * status bits, errors - is as for ssa_decode_attn_sparse /
 * ssa_decode_attn_dense.  The (head, token) pairs that share a K/V head are
 * served like grouped query heads: while (H/H_kv)*n_q <= 16 and D = 128
 * every selected row is read once for all of them.  H*n_q <= 65535.
 * Workspace: ssa_decode_multiq_workspace_bytes(desc, n_q, max_selected)
 * (max_selected = desc->max_ctx for the dense call).
 */
size_t ssa_decode_multiq_workspace_bytes(const ssa_attn_desc* desc, int32_t n_q, int32_t max_selected);
int32_t ssa_decode_attn_sparse_multiq(const ssa_attn_desc* desc, int32_t n_q, int64_t q_stride_t,
                                      int64_t o_stride_t, const void* q, const void* k_cache,
                                      const void* v_cache, const int32_t* ctx_lens, const int32_t* index,
                                      int32_t index_stride, const int32_t* counts, int32_t max_selected,
                                      void* out, float* lse, void* workspace, size_t workspace_bytes,
                                      uint32_t* dev_status, void* stream);
int32_t ssa_decode_attn_dense_multiq(const ssa_attn_desc* desc, int32_t n_q, int64_t q_stride_t,
                                     int64_t o_stride_t, const void* q, const void* k_cache,
                                     const void* v_cache, const int32_t* ctx_lens, void* out, float* lse,
                                     void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                     void* stream);

/*
 * Anchors and references -> span lists: the step before ssa_spans_to_index
 * (Sec. "Self-selected attention span": anchors identify groups of contiguous
 * tokens, the model names the anchors it needs, generation attends to the
 * named groups; the worked arithmetic and summarization examples: "[-1]" is
 * the previous line, the instruction is always attended, the line being
 * generated attends to itself).  The paper gives no algorithm; the rules are:
 * request b attends to
 *   - its prefix           [0, prefix_len[b])                 (instruction)
 *   - its current line     [line_start[b], ctx_lens[b])
 *   - for every reference (lo, hi) in refs[ref_offsets[b] .. ref_offsets[b+1]):
 *       0 <= lo <= hi      the lines identified by anchors lo..hi: line
 *                          anchor_line[anchor_offsets[b] + a] of the request
 *       lo == hi == -k     the k-th completed line before the current one
 *     where the request's completed lines are the (start, end) pairs
 *     lines[line_offsets[b] .. line_offsets[b+1]) in order of appearance.
 * Output, ready for ssa_spans_to_index: span_offsets_out[b] = b*span_stride
 * (B+1 entries) and, in row b of spans_out, the spans in the order above,
 * padded with (0, 0) to span_stride pairs.  References to anchors or lines
 * that do not exist and pairs of any other form are skipped
 * (SSA_DEV_BAD_REF); more than span_stride spans keep the first
 * (SSA_DEV_OVERFLOW).  All pointers dev int32; pair arrays 8-byte aligned.
 * Errors: SSA_ERR_NULL, SSA_ERR_SHAPE (B <= 0, span_stride < 2),
 * SSA_ERR_ALIGN, SSA_ERR_CUDA.
 */
typedef struct {
  const int32_t* line_offsets;    /* [B+1] */
  const int32_t* lines;           /* (start, end) pairs */
  const int32_t* anchor_offsets;  /* [B+1] */
  const int32_t* anchor_line;     /* anchor id -> index of its line within the request */
  const int32_t* ref_offsets;     /* [B+1] */
  const int32_t* refs;            /* (lo, hi) pairs */
  const int32_t* prefix_len;      /* [B] */
  const int32_t* line_start;      /* [B] */
  const int32_t* ctx_lens;        /* [B] */
} ssa_anchor_tables;

int32_t ssa_refs_to_spans(const ssa_anchor_tables* tables, int32_t B, int32_t* span_offsets_out,
                          int32_t* spans_out, int32_t span_stride, uint32_t* dev_status, void* stream);

/*
 * ssa_refs_to_spans and ssa_spans_to_index in one launch (same passages of the
 * paper): the lists index[b, 0 .. counts[b]) are exactly those the two calls
 * produce with span_stride = SSA_MAX_SPANS_PER_SEQ, but the span list stays in
 * shared memory.  The device status bits are those of the two calls
 * (SSA_DEV_BAD_REF; SSA_DEV_BAD_SPAN / SSA_DEV_CLIPPED for lines, prefixes or
 * current lines that do not fit the context; SSA_DEV_OVERFLOW for more than
 * index_stride positions); a request that resolves to more than
 * SSA_MAX_SPANS_PER_SEQ spans keeps the first ones
 * (SSA_DEV_TOO_MANY_SPANS).  index, counts as for ssa_spans_to_index.
 * Errors: SSA_ERR_NULL, SSA_ERR_SHAPE (B <= 0, B > 65535, index_stride <= 0),
 * SSA_ERR_ALIGN, SSA_ERR_CUDA.
 */
int32_t ssa_refs_to_index(const ssa_anchor_tables* tables, int32_t B, int32_t* index,
                          int32_t index_stride, int32_t* counts, uint32_t* dev_status,
                          void* stream);

/*
 * The paper's own metadata format (Sec. "CUDA Kernel Design", Attention span
 * encoding): the context is cut into blocks of `block_size` positions; for
 * every block that holds at least one selected position the list records the
 * block index and a bitmask of the selected positions inside it; blocks
 * without selected positions are omitted; every request has its own list.
 *
 * ssa_spans_to_blockmask builds it from span lists (same span semantics and
 * status bits as ssa_spans_to_index):
 *   block_idx  [b*block_stride + 0 .. block_counts[b])  ascending block indices
 *   block_mask [(b*block_stride + r) * (block_size/32) + w]  32-bit words of
 *              list entry r; bit i of word w stands for position
 *              block_idx*block_size + 32*w + i
 * Entries past block_counts[b] are left untouched; more than block_stride
 * blocks keep the first block_stride (SSA_DEV_OVERFLOW).
 * block_size in {32, 64, 128, 256}.  All pointers dev; span_offsets, spans,
 * ctx_lens as in ssa_spans_to_index.
 * Errors: SSA_ERR_NULL, SSA_ERR_SHAPE, SSA_ERR_UNSUPPORTED (block_size),
 * SSA_ERR_ALIGN, SSA_ERR_CUDA.
 */
int32_t ssa_spans_to_blockmask(const int32_t* span_offsets, const int32_t* spans,
                               const int32_t* ctx_lens, int32_t B, int32_t block_size,
                               int32_t* block_idx, uint32_t* block_mask, int32_t block_stride,
                               int32_t* block_counts, uint32_t* dev_status, void* stream);

/*
 * Span-restricted decode attention from that format (Algorithm 1): same
 * result, options and errors as ssa_decode_attn_sparse, with the attended set
 * of request b given by its first block_counts[b] list entries.  Only the rows
 * whose bit is set are read (the bitmask is expanded on chip; a partially
 * selected block costs its selected rows, not the whole block).  Bits naming
 * positions outside [0, ctx_lens[b]) are skipped (SSA_DEV_BAD_INDEX); a block
 * listed twice counts twice.  `max_blocks` is a host-side upper bound on every
 * block_counts[b] (1 <= max_blocks <= block_stride); larger counts are clamped
 * (SSA_DEV_BAD_COUNT).  Workspace: ssa_decode_blockmask_workspace_bytes.
 */
size_t ssa_decode_blockmask_workspace_bytes(const ssa_attn_desc* desc, int32_t block_size,
                                            int32_t max_blocks);
int32_t ssa_decode_attn_blockmask(const ssa_attn_desc* desc, const void* q, const void* k_cache,
                                  const void* v_cache, const int32_t* ctx_lens,
                                  const int32_t* block_idx, const uint32_t* block_mask,
                                  int32_t block_stride, const int32_t* block_counts,
                                  int32_t block_size, int32_t max_blocks, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                                  void* stream);

/*
 * One decode step of the method in one call (Sec. "Self-selected attention
 * span", Inference: token generation restricted to the selected spans):
 * ssa_spans_to_index followed by ssa_decode_attn_sparse on `stream`, with the
 * same arguments, meanings and errors as those two calls.  Optionally the
 * step's host-resident inputs are copied in first and its results copied out
 * afterwards, on the same stream: when host_in is non-NULL, in_bytes bytes go
 * from host_in to dev_in before the index kernel (a caller lays out query rows,
 * context lengths, span offsets and spans back to back in one device arena and
 * one pinned host arena, so that a single copy brings in everything that
 * changes per step); when host_out is non-NULL, out_bytes bytes go from dev_out
 * to host_out after the attention kernels.  Host arenas should be page-locked,
 * otherwise the copies are not asynchronous.  The call does not wait for any of
 * this work.  The KV cache is resident state and is never copied.
 *
 * flags = 0: both copies are cudaMemcpyAsync transfers (copy engine).
 * flags = SSA_STEP_COPY_BY_KERNEL: both copies are done by kernels of the
 * library that read / write the host arena across the bus (when span_offsets,
 * spans and ctx_lens lie inside the input arena, the copy in is done by extra
 * blocks of the index kernel, whose other blocks read the span lists from the
 * host arena meanwhile; where, besides, the query rows are the head or the
 * tail of the input arena and every request is served by one thread block per
 * head, each attention block fetches its own query row across the bus while it
 * starts up and writes the device copy itself, so that most of the input
 * bytes travel during the attention kernel instead of in front of it).  For the few
 * hundred KB that change per decode step this is faster than a copy-engine
 * transfer, whose set-up time dominates at that size.  The host arenas must
 * then be page-locked memory that the device addresses under the same pointer
 * (cudaHostAlloc / cudaMallocHost under unified addressing; checked with
 * cudaPointerGetAttributes, else SSA_ERR_UNSUPPORTED), all four arena pointers
 * 16-byte aligned and both sizes multiples of 16 (else SSA_ERR_ALIGN); these
 * checks come first, so a refused call has enqueued nothing.
 * In either mode `out` and `lse` may themselves point into such host memory:
 * the attention kernels then store each finished row straight across the bus
 * while the rest of the batch is still being read, and the copy out only has
 * to carry what kernels also read back (counts, the status word).
 *
 * Which kernels run.  The lists index / counts are always written and the
 * results are always those of the two calls, bit for bit.  When the caller
 * states a bound on the spans per request (max_spans > 0) the step may run as
 * ONE kernel instead - ssa_decode_attn_spans with index / counts as its
 * optional outputs - which removes the index launch from short steps:
 *   SSA_STEP_ONE_KERNEL   always (needs 0 < max_spans <= 128 and a workspace
 *                         of ssa_decode_spans_workspace_bytes(desc,
 *                         max_selected, max_spans) bytes, else
 *                         SSA_ERR_CAPACITY / SSA_ERR_WORKSPACE)
 *   SSA_STEP_TWO_KERNELS  never
 *   neither               the library decides: one kernel when max_spans <= 32,
 *                         the workspace suffices, the inputs are not fetched by
 *                         kernel (that fetch is fused with the index launch)
 *                         and the attention grid is at most three waves of
 *                         thread blocks - where every block repeating the merge
 *                         of its request's spans costs less than a launch.
 * Errors: SSA_ERR_NULL for a NULL desc/step or an inconsistent copy request,
 * SSA_ERR_UNSUPPORTED for unknown or contradictory flag bits, otherwise those
 * of the calls made; nothing after a failing stage is enqueued.
 */
#define SSA_STEP_COPY_BY_KERNEL 1u
#define SSA_STEP_ONE_KERNEL 2u
#define SSA_STEP_TWO_KERNELS 4u
typedef struct {
  const int32_t* span_offsets;  /* dev [B+1]                                   */
  const int32_t* spans;         /* dev (start, end) pairs                      */
  const int32_t* ctx_lens;      /* dev [B]                                     */
  int32_t* index;               /* dev [B * index_stride]  (written)           */
  int32_t* counts;              /* dev [B]                 (written)           */
  const void* q;                /* dev                                         */
  const void* k_cache;          /* dev                                         */
  const void* v_cache;          /* dev                                         */
  void* out;                    /* dev, or host the device addresses (written) */
  float* lse;                   /* same, [B*H], or NULL    (written)           */
  void* workspace;              /* dev                                         */
  size_t workspace_bytes;
  uint32_t* dev_status;         /* dev [1] or NULL                             */
  int32_t index_stride;
  int32_t max_selected;
  const void* host_in;          /* host (pinned) or NULL                       */
  void* dev_in;                 /* dev                                         */
  size_t in_bytes;
  void* host_out;               /* host (pinned) or NULL                       */
  const void* dev_out;          /* dev                                         */
  size_t out_bytes;
  uint32_t flags;               /* OR of SSA_STEP_* bits                       */
  int32_t max_spans;            /* host bound on spans per request; 0: unknown */
} ssa_step;

int32_t ssa_decode_step(const ssa_attn_desc* desc, const ssa_step* step, void* stream);

/*
 * ssa_decode_attn_sparse for callers that cannot hand the library a
 * workspace.  (The paper has no counterpart: its kernel runs one thread block
 * per head and request and needs no scratch memory.)
 *
 * Who needs it: code that may not allocate device memory at the point of the
 * call - a plug-in running inside a host application that owns the device
 * allocator, a serving loop that has frozen its memory pool after start-up,
 * or a latency-critical path where cudaMalloc (which can synchronise the whole
 * device) is off limits.  Such a caller still passes all inputs and outputs;
 * only the split-KV scratch comes from the library: a fixed array of
 * SSA_STATIC_SCRATCH_BYTES bytes that lives in the library's device image, so
 * every GPU that loads the library holds it until the process exits.
 *
 * Same arguments and results as ssa_decode_attn_sparse, minus the workspace.
 * Differences:
 *  - a request whose scratch need (what ssa_decode_workspace_bytes reports
 *    for desc and max_selected) exceeds SSA_STATIC_SCRATCH_BYTES is rejected
 *    with SSA_ERR_WORKSPACE and nothing is launched;
 *  - the first call on each device looks up the array's device address (the
 *    device must be current); make that first call outside any stream
 *    capture.  The address is kept per device ordinal for the device's
 *    primary context (the one the runtime API uses) and is stale after
 *    cudaDeviceReset.  No call allocates or frees memory;
 *  - all calls share the one array, and it keeps whatever the previous call
 *    left in it.  Nothing in it needs to start at zero (every slot is written
 *    before it is read within a call), but two calls whose kernels overlap on
 *    the GPU - different streams, or graphs launched concurrently - race on
 *    it and corrupt each other's results.  Issue them on one stream, or order
 *    them with events.
 */
#define SSA_STATIC_SCRATCH_BYTES (8u << 20)
int32_t ssa_decode_attn_sparse_noalloc(const ssa_attn_desc* desc, const void* q,
                                       const void* k_cache, const void* v_cache,
                                       const int32_t* ctx_lens, const int32_t* index,
                                       int32_t index_stride, const int32_t* counts,
                                       int32_t max_selected, void* out, float* lse,
                                       uint32_t* dev_status, void* stream);

/*
 * Optional timing hook for harnesses (no counterpart in the paper): the next
 * attention call made by the calling thread records `ev_begin` immediately
 * before and `ev_end` immediately after its main (split-KV) kernel on the
 * call's stream, then forgets them.  Both are cudaEvent_t passed as void*;
 * passing NULLs clears the hook.  Has no effect on results.
 */
void ssa_set_kernel_events(void* ev_begin, void* ev_end);

/* Number of kernels the calling thread's calls have launched so far. */
uint64_t ssa_launch_count(void);

const char* ssa_status_string(int32_t status);
int32_t ssa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SSA_H_ */
