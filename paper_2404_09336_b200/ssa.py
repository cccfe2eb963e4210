"""ctypes binding of libssa (include/ssa.h): argument marshalling only.

Every function takes torch CUDA tensors (used purely as device memory) and
hands their addresses, sizes and strides to the C entry point of the same
name.  Nothing is computed here, and there is no fallback: if the shared
library cannot be loaded the import fails.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

# ---- status codes / bits (mirror include/ssa.h) -----------------------------------
OK = 0
ERR_NULL, ERR_SHAPE, ERR_DTYPE, ERR_ALIGN, ERR_CAPACITY, ERR_WORKSPACE, ERR_CUDA, ERR_UNSUPPORTED = range(1, 9)
DEV_BAD_SPAN, DEV_CLIPPED, DEV_OVERFLOW, DEV_BAD_INDEX, DEV_BAD_COUNT, DEV_TOO_MANY_SPANS = 1, 2, 4, 8, 16, 32
DEV_BAD_REF = 64
MAX_SPANS_PER_SEQ = 2048
F16, BF16, F32, FP8_E4M3 = 0, 1, 2, 3
_DTYPES = {torch.float16: F16, torch.bfloat16: BF16, torch.float32: F32, torch.float8_e4m3fn: FP8_E4M3}


class AttnDesc(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("H", C.c_int32), ("H_kv", C.c_int32), ("D", C.c_int32),
        ("max_ctx", C.c_int32), ("kv_dtype", C.c_int32), ("out_dtype", C.c_int32), ("scale", C.c_float),
        ("q_stride_b", C.c_int64), ("q_stride_h", C.c_int64),
        ("k_stride_b", C.c_int64), ("k_stride_t", C.c_int64), ("k_stride_h", C.c_int64),
        ("v_stride_b", C.c_int64), ("v_stride_t", C.c_int64), ("v_stride_h", C.c_int64),
        ("o_stride_b", C.c_int64), ("o_stride_h", C.c_int64),
    ]


class Step(C.Structure):
    """ssa_step: the arguments of one decode step (see include/ssa.h)."""
    _fields_ = [
        ("span_offsets", C.c_void_p), ("spans", C.c_void_p), ("ctx_lens", C.c_void_p),
        ("index", C.c_void_p), ("counts", C.c_void_p),
        ("q", C.c_void_p), ("k_cache", C.c_void_p), ("v_cache", C.c_void_p),
        ("out", C.c_void_p), ("lse", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("dev_status", C.c_void_p), ("index_stride", C.c_int32), ("max_selected", C.c_int32),
        ("host_in", C.c_void_p), ("dev_in", C.c_void_p), ("in_bytes", C.c_size_t),
        ("host_out", C.c_void_p), ("dev_out", C.c_void_p), ("out_bytes", C.c_size_t),
        ("flags", C.c_uint32), ("max_spans", C.c_int32),
    ]


class Paging(C.Structure):
    """ssa_paging (see include/ssa.h)."""
    _fields_ = [("page_table", C.c_void_p), ("page_table_stride", C.c_int32), ("page_size", C.c_int32),
                ("n_pages", C.c_int32)]


class AnchorTables(C.Structure):
    """ssa_anchor_tables (see include/ssa.h)."""
    _fields_ = [(n, C.c_void_p) for n in ("line_offsets", "lines", "anchor_offsets", "anchor_line", "ref_offsets",
                                          "refs", "prefix_len", "line_start", "ctx_lens")]


class SsaError(RuntimeError):
    def __init__(self, fn, code):
        self.code = code
        super().__init__(f"{fn}: {status_string(code)} (status {code})")


def _load():
    path = os.environ.get("SSA_LIBRARY") or _build.LIB
    if path == _build.LIB:
        _build.build_library()          # no-op when the in-tree library is current
    lib = C.CDLL(path)
    vp = C.c_void_p
    lib.ssa_spans_to_index.restype = C.c_int32
    lib.ssa_spans_to_index.argtypes = [vp, vp, vp, C.c_int32, vp, C.c_int32, vp, vp, vp]
    lib.ssa_decode_workspace_bytes.restype = C.c_size_t
    lib.ssa_decode_workspace_bytes.argtypes = [C.POINTER(AttnDesc), C.c_int32]
    lib.ssa_decode_attn_sparse.restype = C.c_int32
    lib.ssa_decode_attn_sparse.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, vp, vp, C.c_int32, vp, C.c_int32,
                                           vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_decode_spans_workspace_bytes.restype = C.c_size_t
    lib.ssa_decode_spans_workspace_bytes.argtypes = [C.POINTER(AttnDesc), C.c_int32, C.c_int32]
    lib.ssa_decode_attn_spans.restype = C.c_int32
    lib.ssa_decode_attn_spans.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, C.c_int32, C.c_int32, vp, vp,
                                          vp, C.c_int32, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_decode_multiq_workspace_bytes.restype = C.c_size_t
    lib.ssa_decode_multiq_workspace_bytes.argtypes = [C.POINTER(AttnDesc), C.c_int32, C.c_int32]
    lib.ssa_decode_attn_sparse_multiq.restype = C.c_int32
    lib.ssa_decode_attn_sparse_multiq.argtypes = [C.POINTER(AttnDesc), C.c_int32, C.c_int64, C.c_int64, vp, vp, vp, vp,
                                                  vp, C.c_int32, vp, C.c_int32, vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_decode_attn_dense_multiq.restype = C.c_int32
    lib.ssa_decode_attn_dense_multiq.argtypes = [C.POINTER(AttnDesc), C.c_int32, C.c_int64, C.c_int64, vp, vp, vp, vp,
                                                 vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_spans_to_blockmask.restype = C.c_int32
    lib.ssa_spans_to_blockmask.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, vp, vp, C.c_int32, vp, vp, vp]
    lib.ssa_decode_blockmask_workspace_bytes.restype = C.c_size_t
    lib.ssa_decode_blockmask_workspace_bytes.argtypes = [C.POINTER(AttnDesc), C.c_int32, C.c_int32]
    lib.ssa_decode_attn_blockmask.restype = C.c_int32
    lib.ssa_decode_attn_blockmask.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, C.c_int32, vp, C.c_int32,
                                              C.c_int32, vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_refs_to_spans.restype = C.c_int32
    lib.ssa_refs_to_spans.argtypes = [C.POINTER(AnchorTables), C.c_int32, vp, vp, C.c_int32, vp, vp]
    lib.ssa_decode_attn_sparse_paged.restype = C.c_int32
    lib.ssa_decode_attn_sparse_paged.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, C.POINTER(Paging), vp, vp, C.c_int32,
                                                 vp, C.c_int32, vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_decode_attn_dense_paged.restype = C.c_int32
    lib.ssa_decode_attn_dense_paged.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, C.POINTER(Paging), vp, vp, vp, vp,
                                                C.c_size_t, vp, vp]
    lib.ssa_refs_to_index.restype = C.c_int32
    lib.ssa_refs_to_index.argtypes = [C.POINTER(AnchorTables), C.c_int32, vp, C.c_int32, vp, vp, vp]
    lib.ssa_decode_step.restype = C.c_int32
    lib.ssa_decode_step.argtypes = [C.POINTER(AttnDesc), C.POINTER(Step), vp]
    lib.ssa_decode_attn_sparse_noalloc.restype = C.c_int32
    lib.ssa_decode_attn_sparse_noalloc.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, vp, vp, C.c_int32, vp, C.c_int32,
                                                   vp, vp, vp, vp]
    lib.ssa_decode_attn_dense.restype = C.c_int32
    lib.ssa_decode_attn_dense.argtypes = [C.POINTER(AttnDesc), vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
    lib.ssa_set_kernel_events.restype = None
    lib.ssa_set_kernel_events.argtypes = [vp, vp]
    lib.ssa_launch_count.restype = C.c_uint64
    lib.ssa_launch_count.argtypes = []
    lib.ssa_status_string.restype = C.c_char_p
    lib.ssa_status_string.argtypes = [C.c_int32]
    lib.ssa_version.restype = C.c_int32
    lib.ssa_version.argtypes = []
    return lib


lib = _load()
LIBRARY_PATH = lib._name


def status_string(code: int) -> str:
    return lib.ssa_status_string(int(code)).decode()


def version() -> int:
    return lib.ssa_version()


def launch_count() -> int:
    return int(lib.ssa_launch_count())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _row_stride(index):
    """Elements between consecutive rows of index[B, n] (a one-row tensor may
    carry an arbitrary stride for its size-1 dimension)."""
    return int(index.stride(0) if index.shape[0] > 1 else index.shape[1])


def _check(fn, rc, check):
    if check and rc != OK:
        raise SsaError(fn, rc)
    return rc


def make_desc(q, k_cache, v_cache, out, max_ctx=None, scale: float = 0.0) -> AttnDesc:
    """Descriptor for q[B,H,D], k_cache/v_cache[B,H,T,D] (any batch, head and
    token strides: a token-major cache is the permuted view) and out[B,H,D]."""
    B, H, D = q.shape
    d = AttnDesc()
    d.B, d.H, d.H_kv, d.D = B, H, k_cache.shape[1], D
    d.max_ctx = int(k_cache.shape[2] if max_ctx is None else max_ctx)
    d.kv_dtype = _DTYPES.get(k_cache.dtype, -1)
    d.out_dtype = _DTYPES.get(out.dtype, -1)
    d.scale = float(scale)
    d.q_stride_b, d.q_stride_h = q.stride(0), q.stride(1)
    d.k_stride_b, d.k_stride_h, d.k_stride_t = k_cache.stride(0), k_cache.stride(1), k_cache.stride(2)
    d.v_stride_b, d.v_stride_h, d.v_stride_t = v_cache.stride(0), v_cache.stride(1), v_cache.stride(2)
    d.o_stride_b, d.o_stride_h = out.stride(0), out.stride(1)
    for t in (q, k_cache, v_cache, out):
        if t.stride(-1) != 1:
            raise ValueError("the head dimension must be contiguous")
    return d


def spans_to_index(span_offsets, spans, ctx_lens, index, counts, dev_status=None, stream=None, check=True):
    """ssa_spans_to_index: index[B, index_stride] and counts[B] are written."""
    rc = lib.ssa_spans_to_index(_ptr(span_offsets), _ptr(spans), _ptr(ctx_lens), int(ctx_lens.numel()),
                                _ptr(index), _row_stride(index), _ptr(counts), _ptr(dev_status),
                                _stream(stream))
    return _check("ssa_spans_to_index", rc, check)


def decode_workspace_bytes(desc: AttnDesc, max_selected: int) -> int:
    return int(lib.ssa_decode_workspace_bytes(C.byref(desc), int(max_selected)))


def decode_attn_sparse(desc, q, k_cache, v_cache, ctx_lens, index, counts, max_selected, out, lse=None,
                       workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_sparse: out (and lse) are written."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_sparse(C.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens),
                                    _ptr(index), _row_stride(index) if index is not None else 0,
                                    _ptr(counts), int(max_selected), _ptr(out), _ptr(lse), _ptr(workspace),
                                    ws_bytes, _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_sparse", rc, check)


DIRECT_SPANS = 128      # spans per request the span-list attention call merges on chip


def decode_spans_workspace_bytes(desc: AttnDesc, max_selected: int, max_spans: int) -> int:
    return int(lib.ssa_decode_spans_workspace_bytes(C.byref(desc), int(max_selected), int(max_spans)))


def decode_attn_spans(desc, q, k_cache, v_cache, ctx_lens, span_offsets, spans, max_spans, max_selected, out, lse=None,
                      index_out=None, counts_out=None, workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_spans: span lists -> attention output in one call; index_out / counts_out optional."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_spans(C.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens),
                                   _ptr(span_offsets), _ptr(spans), int(max_spans), int(max_selected), _ptr(out),
                                   _ptr(lse), _ptr(index_out), _row_stride(index_out) if index_out is not None else 0,
                                   _ptr(counts_out), _ptr(workspace), ws_bytes, _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_spans", rc, check)


def make_desc_multiq(q, k_cache, v_cache, out, max_ctx=None, scale: float = 0.0):
    """Descriptor for q[B,H,Tq,D], out[B,H,Tq,D] (several query tokens per head) over k_cache/v_cache[B,H_kv,T,D].
    Returns (desc, n_q, q_stride_t, o_stride_t)."""
    d = make_desc(q[:, :, 0], k_cache, v_cache, out[:, :, 0], max_ctx, scale)
    return d, int(q.shape[2]), int(q.stride(2)), int(out.stride(2))


def decode_multiq_workspace_bytes(desc: AttnDesc, n_q: int, max_selected: int) -> int:
    return int(lib.ssa_decode_multiq_workspace_bytes(C.byref(desc), int(n_q), int(max_selected)))


def decode_attn_sparse_multiq(desc, n_q, q_stride_t, o_stride_t, q, k_cache, v_cache, ctx_lens, index, counts,
                              max_selected, out, lse=None, workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_sparse_multiq: n_q query rows per head over one selected set; out / lse are written."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_sparse_multiq(C.byref(desc), int(n_q), int(q_stride_t), int(o_stride_t), _ptr(q),
                                           _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens), _ptr(index),
                                           _row_stride(index) if index is not None else 0, _ptr(counts),
                                           int(max_selected), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                           _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_sparse_multiq", rc, check)


def decode_attn_dense_multiq(desc, n_q, q_stride_t, o_stride_t, q, k_cache, v_cache, ctx_lens, out, lse=None,
                             workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_dense_multiq: n_q query rows per head over the full context."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_dense_multiq(C.byref(desc), int(n_q), int(q_stride_t), int(o_stride_t), _ptr(q),
                                          _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens), _ptr(out), _ptr(lse),
                                          _ptr(workspace), ws_bytes, _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_dense_multiq", rc, check)


def spans_to_blockmask(span_offsets, spans, ctx_lens, block_size, block_idx, block_mask, block_counts,
                       dev_status=None, stream=None, check=True):
    """ssa_spans_to_blockmask: block_idx[B, stride], block_mask[B, stride, block_size/32] and
    block_counts[B] are written."""
    rc = lib.ssa_spans_to_blockmask(_ptr(span_offsets), _ptr(spans), _ptr(ctx_lens), int(ctx_lens.numel()),
                                    int(block_size), _ptr(block_idx), _ptr(block_mask), _row_stride(block_idx),
                                    _ptr(block_counts), _ptr(dev_status), _stream(stream))
    return _check("ssa_spans_to_blockmask", rc, check)


def decode_blockmask_workspace_bytes(desc: AttnDesc, block_size: int, max_blocks: int) -> int:
    return int(lib.ssa_decode_blockmask_workspace_bytes(C.byref(desc), int(block_size), int(max_blocks)))


def decode_attn_blockmask(desc, q, k_cache, v_cache, ctx_lens, block_idx, block_mask, block_counts, block_size,
                          max_blocks, out, lse=None, workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_blockmask: out (and lse) are written."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_blockmask(C.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens),
                                       _ptr(block_idx), _ptr(block_mask),
                                       _row_stride(block_idx) if block_idx is not None else 0, _ptr(block_counts),
                                       int(block_size), int(max_blocks), _ptr(out), _ptr(lse), _ptr(workspace),
                                       ws_bytes, _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_blockmask", rc, check)


def make_desc_paged(q, k_pool, v_pool, out, max_ctx: int, scale: float = 0.0) -> AttnDesc:
    """Descriptor for q[B,H,D], out[B,H,D] and K/V pools [n_pages, page_size, H_kv, D] whose rows are evenly
    spaced over the whole pool (pages back to back)."""
    B, H, D = q.shape
    d = AttnDesc()
    d.B, d.H, d.H_kv, d.D = B, H, k_pool.shape[2], D
    d.max_ctx = int(max_ctx)
    d.kv_dtype = _DTYPES.get(k_pool.dtype, -1)
    d.out_dtype = _DTYPES.get(out.dtype, -1)
    d.scale = float(scale)
    d.q_stride_b, d.q_stride_h = q.stride(0), q.stride(1)
    d.o_stride_b, d.o_stride_h = out.stride(0), out.stride(1)
    for pool in (k_pool, v_pool):
        if pool.stride(-1) != 1 or pool.stride(0) != pool.shape[1] * pool.stride(1):
            raise ValueError("pool rows must be evenly spaced and the head dimension contiguous")
    d.k_stride_b = d.v_stride_b = 0
    d.k_stride_t, d.k_stride_h = k_pool.stride(1), k_pool.stride(2)
    d.v_stride_t, d.v_stride_h = v_pool.stride(1), v_pool.stride(2)
    return d


def make_paging(page_table, page_size: int, n_pages: int) -> Paging:
    """ssa_paging for page_table[B, pages per request] (int32, device); keep the tensor alive."""
    pg = Paging()
    pg.page_table, pg.page_table_stride = page_table.data_ptr(), _row_stride(page_table)
    pg.page_size, pg.n_pages = int(page_size), int(n_pages)
    return pg


def decode_attn_sparse_paged(desc, q, k_pool, v_pool, paging, ctx_lens, index, counts, max_selected, out, lse=None,
                             workspace=None, dev_status=None, stream=None, check=True):
    """ssa_decode_attn_sparse_paged: as decode_attn_sparse over a paged cache."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_sparse_paged(C.byref(desc), _ptr(q), _ptr(k_pool), _ptr(v_pool),
                                          C.byref(paging) if paging is not None else None, _ptr(ctx_lens),
                                          _ptr(index), _row_stride(index) if index is not None else 0, _ptr(counts),
                                          int(max_selected), _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes,
                                          _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_sparse_paged", rc, check)


def decode_attn_dense_paged(desc, q, k_pool, v_pool, paging, ctx_lens, out, lse=None, workspace=None,
                            dev_status=None, stream=None, check=True):
    """ssa_decode_attn_dense_paged: full-context attention over a paged cache."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_dense_paged(C.byref(desc), _ptr(q), _ptr(k_pool), _ptr(v_pool),
                                         C.byref(paging) if paging is not None else None, _ptr(ctx_lens), _ptr(out),
                                         _ptr(lse), _ptr(workspace), ws_bytes, _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_dense_paged", rc, check)


def _anchor_tables(line_offsets, lines, anchor_offsets, anchor_line, ref_offsets, refs, prefix_len, line_start,
                   ctx_lens) -> AnchorTables:
    t = AnchorTables()
    for name, ten in (("line_offsets", line_offsets), ("lines", lines), ("anchor_offsets", anchor_offsets),
                      ("anchor_line", anchor_line), ("ref_offsets", ref_offsets), ("refs", refs),
                      ("prefix_len", prefix_len), ("line_start", line_start), ("ctx_lens", ctx_lens)):
        setattr(t, name, None if ten is None else ten.data_ptr())
    return t


def refs_to_index(line_offsets, lines, anchor_offsets, anchor_line, ref_offsets, refs, prefix_len, line_start,
                  ctx_lens, index, counts, dev_status=None, stream=None, check=True):
    """ssa_refs_to_index: references -> index[B, index_stride] and counts[B] in one launch."""
    t = _anchor_tables(line_offsets, lines, anchor_offsets, anchor_line, ref_offsets, refs, prefix_len, line_start,
                       ctx_lens)
    rc = lib.ssa_refs_to_index(C.byref(t), int(ctx_lens.numel()), _ptr(index), _row_stride(index), _ptr(counts),
                               _ptr(dev_status), _stream(stream))
    return _check("ssa_refs_to_index", rc, check)


def refs_to_spans(line_offsets, lines, anchor_offsets, anchor_line, ref_offsets, refs, prefix_len, line_start,
                  ctx_lens, span_offsets_out, spans_out, dev_status=None, stream=None, check=True):
    """ssa_refs_to_spans: spans_out[B, span_stride, 2] and span_offsets_out[B+1] are written."""
    t = _anchor_tables(line_offsets, lines, anchor_offsets, anchor_line, ref_offsets, refs, prefix_len, line_start,
                       ctx_lens)
    rc = lib.ssa_refs_to_spans(C.byref(t), int(ctx_lens.numel()), _ptr(span_offsets_out), _ptr(spans_out),
                               int(spans_out.shape[1]), _ptr(dev_status), _stream(stream))
    return _check("ssa_refs_to_spans", rc, check)


STEP_COPY_BY_KERNEL, STEP_ONE_KERNEL, STEP_TWO_KERNELS = 1, 2, 4


def make_step(span_offsets, spans, ctx_lens, index, counts, q, k_cache, v_cache, max_selected, out, lse=None,
              workspace=None, dev_status=None, host_in=None, dev_in=None, host_out=None, dev_out=None,
              copy_by_kernel=False, max_spans=0, kernels="auto") -> Step:
    """Fill an ssa_step from tensors (addresses only; keep the tensors alive)."""
    addr = lambda t: None if t is None else t.data_ptr()
    nbytes = lambda t: 0 if t is None else t.numel() * t.element_size()
    s = Step()
    s.span_offsets, s.spans, s.ctx_lens = addr(span_offsets), addr(spans), addr(ctx_lens)
    s.index, s.counts = addr(index), addr(counts)
    s.q, s.k_cache, s.v_cache = addr(q), addr(k_cache), addr(v_cache)
    s.out, s.lse, s.workspace, s.workspace_bytes = addr(out), addr(lse), addr(workspace), nbytes(workspace)
    s.dev_status, s.index_stride, s.max_selected = addr(dev_status), _row_stride(index), int(max_selected)
    s.host_in, s.dev_in, s.in_bytes = addr(host_in), addr(dev_in), nbytes(host_in)
    s.host_out, s.dev_out, s.out_bytes = addr(host_out), addr(dev_out), nbytes(host_out)
    s.flags = (STEP_COPY_BY_KERNEL if copy_by_kernel else 0) | {"auto": 0, "one": STEP_ONE_KERNEL,
                                                                 "two": STEP_TWO_KERNELS}[kernels]
    s.max_spans = int(max_spans)
    return s


def decode_step(desc: AttnDesc, step: Step, stream=None, check=True):
    """ssa_decode_step: [copy in] -> span lists to index lists and attention (one kernel or two) -> [copy out]."""
    return _check("ssa_decode_step", lib.ssa_decode_step(C.byref(desc), C.byref(step), _stream(stream)), check)


STATIC_SCRATCH_BYTES = 8 << 20


def decode_attn_sparse_noalloc(desc, q, k_cache, v_cache, ctx_lens, index, counts, max_selected, out, lse=None,
                               dev_status=None, stream=None, check=True):
    """ssa_decode_attn_sparse_noalloc: as decode_attn_sparse, with the scratch
    memory taken from the library's built-in array instead of a workspace
    tensor (for callers that must not allocate; see include/ssa.h)."""
    rc = lib.ssa_decode_attn_sparse_noalloc(C.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens),
                                            _ptr(index), _row_stride(index) if index is not None else 0,
                                            _ptr(counts), int(max_selected), _ptr(out), _ptr(lse),
                                            _ptr(dev_status), _stream(stream))
    return _check("ssa_decode_attn_sparse_noalloc", rc, check)


def decode_attn_dense(desc, q, k_cache, v_cache, ctx_lens, out, lse=None, workspace=None, dev_status=None,
                      stream=None, check=True):
    """ssa_decode_attn_dense: out (and lse) are written."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.ssa_decode_attn_dense(C.byref(desc), _ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(ctx_lens),
                                   _ptr(out), _ptr(lse), _ptr(workspace), ws_bytes, _ptr(dev_status),
                                   _stream(stream))
    return _check("ssa_decode_attn_dense", rc, check)


def set_kernel_events(begin=None, end=None):
    """ssa_set_kernel_events with torch.cuda.Event objects that have been
    recorded at least once (so that they own a CUDA event), or None."""
    lib.ssa_set_kernel_events(None if begin is None else C.c_void_p(begin.cuda_event),
                              None if end is None else C.c_void_p(end.cuda_event))
