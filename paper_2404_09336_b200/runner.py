"""Device-side plumbing around the C-ABI calls: buffers for one workload and
the decode step (span lists -> index lists -> attention).

Only allocation, host<->device copies and calls of ``ssa.*`` happen here.
"""
from __future__ import annotations

import concurrent.futures as _cf
import os

import numpy as np
import torch

from . import ssa
from .inputs import Workload

_TORCH_DTYPE = {"bf16": torch.bfloat16, "f16": torch.float16}


def bits_to_tensor(bits: np.ndarray, dtype: str) -> torch.Tensor:
    """uint16 storage patterns -> CPU tensor of the storage type (no copy)."""
    return torch.from_numpy(bits.view(np.int16)).view(_TORCH_DTYPE[dtype])


def tensor_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def _nbytes(shape, dt):
    return int(np.prod(shape)) * torch.empty((), dtype=dt).element_size()


def _views(buf, specs):
    """Tensors of the given (shape, dtype) laid back to back at 256-byte boundaries in the uint8 buffer."""
    views, o = [], 0
    for shape, dt in specs:
        n = _nbytes(shape, dt)
        views.append(buf[o:o + n].view(dt).view(shape))
        o += (n + 255) // 256 * 256
    return views


def _arena(device, specs):
    """One uint8 device buffer holding tensors of the given (shape, dtype)
    back to back at 256-byte boundaries; returns (buffer, views)."""
    total = sum((_nbytes(shape, dt) + 255) // 256 * 256 for shape, dt in specs)
    buf = torch.zeros(total, dtype=torch.uint8, device=device)
    return buf, _views(buf, specs)


class DecodeStep:
    """Buffers of one workload on one GPU.

    layout "bhtd": cache stored [B, H, T, D] (one contiguous plane per head);
    layout "bthd": cache stored [B, T, H, D] (token-major).  Either way
    ``self.k`` / ``self.v`` are the logical [B, H, T, D] views.
    ``kv_copies`` > 1 keeps several copies of the cache so that consecutive
    timed steps read different memory.  ``query_heads`` (a multiple of the
    workload's H) gives the query, output and lse that many heads over the
    workload's H cache heads (grouped query heads).
    """

    def __init__(self, wl: Workload, device="cuda:0", layout="bhtd", out_dtype=None, kv_copies=1,
                 index_stride=None, max_selected=None, gen_threads=None,
                 span_capacity=0, query_heads=None):
        self.wl, self.device, self.layout = wl, torch.device(device), layout
        dt = _TORCH_DTYPE[wl.dtype]
        dev = self.device
        B, H, D, T = wl.B, wl.H, wl.D, wl.max_ctx
        shape = (B, H, T, D) if layout == "bhtd" else (B, T, H, D)
        self.k_store = [torch.empty(shape, dtype=dt, device=dev) for _ in range(kv_copies)]
        self.v_store = [torch.empty(shape, dtype=dt, device=dev) for _ in range(kv_copies)]
        threads = gen_threads or max(1, min(B, (os.cpu_count() or 2) // 2, 8))
        with _cf.ThreadPoolExecutor(threads) as ex:          # draw on several cores, upload in order
            pending = []
            for i in range(B):
                pending.append(ex.submit(wl.kv_bits_seq, i))
                if len(pending) >= threads or i == B - 1:
                    first = i - len(pending) + 1
                    for j, fut in enumerate(pending):
                        kb, vb = fut.result()
                        kt, vt = bits_to_tensor(kb, wl.dtype), bits_to_tensor(vb, wl.dtype)
                        if layout == "bthd":
                            kt, vt = kt.permute(1, 0, 2), vt.permute(1, 0, 2)
                        self.k_store[0][first + j].copy_(kt)
                        self.v_store[0][first + j].copy_(vt)
                    pending = []
        for c in range(1, kv_copies):
            self.k_store[c].copy_(self.k_store[0])
            self.v_store[c].copy_(self.v_store[0])
        self.select_copy(0)
        spans = wl.spans if len(wl.spans) else np.zeros((1, 2), np.int32)
        self.max_selected = int(max_selected or max(wl.selected_upper_bound(), 1))
        self.index_stride = int(index_stride or (self.max_selected + 31) // 32 * 32)
        odt = out_dtype or dt
        QH = int(query_heads or H)
        if QH % H != 0:
            raise ValueError("query_heads must be a multiple of the workload's heads")
        # what changes every decode step lives in one input arena and one result
        # arena, so that a host-driven step is one copy in and one copy out
        self.in_arena, (self.q, self.ctx_lens, self.span_offsets, self.spans) = _arena(
            dev, [((B, QH, D), dt), ((B,), torch.int32), ((B + 1,), torch.int32), ((max(len(spans), span_capacity), 2), torch.int32)])
        self._out_specs = [((B, QH, D), odt), ((B, QH), torch.float32), ((B,), torch.int32), ((1,), torch.int32)]
        self.out_arena, (self.out, self.lse, self.counts, self.status) = _arena(dev, self._out_specs)
        self.q.copy_(bits_to_tensor(wl.q_bits(QH), wl.dtype))
        self.ctx_lens.copy_(torch.from_numpy(wl.ctx_lens.copy()))
        self.span_offsets.copy_(torch.from_numpy(wl.span_offsets.copy()))
        self.spans[: len(spans)].copy_(torch.from_numpy(np.ascontiguousarray(spans)))
        self.out.zero_()
        self.lse.zero_()
        self.counts.fill_(-7)
        self.status.zero_()
        self.index = torch.full((B, self.index_stride), -7, dtype=torch.int32, device=dev)
        self.desc = ssa.make_desc(self.q, self.k, self.v, self.out, max_ctx=T)
        self.max_spans = int(max(1, np.diff(wl.span_offsets).max() if wl.B else 1))
        need = max(ssa.decode_workspace_bytes(self.desc, self.max_selected),
                   ssa.decode_workspace_bytes(self.desc, T),
                   ssa.decode_spans_workspace_bytes(self.desc, self.index_stride, ssa.MAX_SPANS_PER_SEQ))
        if need == 0:
            raise RuntimeError("ssa_decode_workspace_bytes rejected the descriptor")
        self.workspace = torch.empty(need, dtype=torch.uint8, device=dev)
        self._steps = {}

    def select_copy(self, c: int):
        ks, vs = self.k_store[c % len(self.k_store)], self.v_store[c % len(self.v_store)]
        self.k = ks if self.layout == "bhtd" else ks.permute(0, 2, 1, 3)
        self.v = vs if self.layout == "bhtd" else vs.permute(0, 2, 1, 3)

    # ---- the calls ------------------------------------------------------------------
    def build_index(self, stream=None):
        return ssa.spans_to_index(self.span_offsets, self.spans, self.ctx_lens, self.index, self.counts,
                                  self.status, stream)

    def attend_sparse(self, stream=None):
        return ssa.decode_attn_sparse(self.desc, self.q, self.k, self.v, self.ctx_lens, self.index,
                                      self.counts, self.max_selected, self.out, self.lse, self.workspace,
                                      self.status, stream)

    def attend_spans(self, stream=None, want_lists=False):
        """Span lists -> attention output in one call (no index list unless want_lists)."""
        return ssa.decode_attn_spans(self.desc, self.q, self.k, self.v, self.ctx_lens, self.span_offsets, self.spans,
                                     self.max_spans, self.max_selected, self.out, self.lse,
                                     self.index if want_lists else None, self.counts if want_lists else None,
                                     self.workspace, self.status, stream)

    def attend_dense(self, stream=None):
        return ssa.decode_attn_dense(self.desc, self.q, self.k, self.v, self.ctx_lens, self.out, self.lse,
                                     self.workspace, self.status, stream)

    # ---- the paper's blocked encoding as the metadata format ---------------------------
    def enable_blockmask(self, block_size: int = 256):
        """Buffers for the (block index, bitmask) lists of every request."""
        B, dev = self.wl.B, self.device
        self.block_size = block_size
        self.block_stride = (self.wl.max_ctx + block_size - 1) // block_size
        self._bound_blocks()
        self.block_idx = torch.full((B, self.block_stride), -7, dtype=torch.int32, device=dev)
        self.block_mask = torch.zeros((B, self.block_stride, block_size // 32), dtype=torch.int32, device=dev)
        self.block_counts = torch.zeros((B,), dtype=torch.int32, device=dev)
        need = ssa.decode_blockmask_workspace_bytes(self.desc, block_size, self.block_stride)
        if need > self.workspace.numel():
            self.workspace = torch.empty(need, dtype=torch.uint8, device=dev)
            self._steps = {}

    def _bound_blocks(self):
        """Host-side bound on the listed blocks of any request: no more than its context spans."""
        longest = int(self.wl.ctx_lens.max()) if len(self.wl.ctx_lens) else 1
        self.max_blocks = max(1, min(self.block_stride, (longest + self.block_size - 1) // self.block_size))

    def build_blockmask(self, stream=None):
        return ssa.spans_to_blockmask(self.span_offsets, self.spans, self.ctx_lens, self.block_size, self.block_idx,
                                      self.block_mask, self.block_counts, self.status, stream)

    def attend_blockmask(self, stream=None):
        return ssa.decode_attn_blockmask(self.desc, self.q, self.k, self.v, self.ctx_lens, self.block_idx,
                                         self.block_mask, self.block_counts, self.block_size, self.max_blocks,
                                         self.out, self.lse, self.workspace, self.status, stream)

    def step_blockmask(self, stream=None):
        self.build_blockmask(stream)
        self.attend_blockmask(stream)

    def step_two_calls(self, stream=None):
        """One decode step as two calls: span lists -> index lists -> attention."""
        self.build_index(stream)
        self.attend_sparse(stream)

    def step(self, stream=None, kernels="auto"):
        """One decode step of the method through ssa_decode_step with everything resident on the
        device: index lists, counts and the attention output are written.  kernels: "auto" (the
        library picks one kernel or index + attention launches), "one" or "two"."""
        key = ("resident", self.k.data_ptr(), self.max_selected, self.max_spans, kernels)
        st = self._steps.get(key)
        if st is None:
            st = ssa.make_step(self.span_offsets, self.spans, self.ctx_lens, self.index, self.counts, self.q, self.k,
                               self.v, self.max_selected, self.out, self.lse, self.workspace, self.status,
                               max_spans=self.max_spans, kernels=kernels)
            self._steps[key] = st
        return ssa.decode_step(self.desc, st, stream)

    # ---- host-buffer form (end-to-end timing) -----------------------------------------
    def make_host_buffers(self):
        """Pinned host copy of what changes every decode step (query rows,
        context lengths, span lists) and a pinned landing buffer for what the
        caller reads back (output rows, lse, counts, status word).
        Returns (host-to-device bytes, device-to-host bytes) per step."""
        self.h_in = self.in_arena.cpu().pin_memory()
        self.h_out = torch.empty(self.out_arena.shape, dtype=torch.uint8).pin_memory()
        self.h_out_rows, self.h_lse, self.h_counts, self.h_status = _views(self.h_out, self._out_specs)
        return self.h_in.numel(), self.h_out.numel()

    def step_from_host(self, stream=None, direct=False):
        """Decode step whose per-step inputs start in pinned host memory and
        whose result ends there (ssa_decode_step with both copies); the KV
        cache is the resident state.

        direct=False: one copy-engine transfer in, the kernels, one out.
        direct=True: the inputs are fetched by a kernel, the attention kernels
        store output rows and lse straight into the pinned landing buffer, and
        a kernel carries counts and the status word over
        (SSA_STEP_COPY_BY_KERNEL).  Same bytes, same result, less latency."""
        if not hasattr(self, "h_in"):
            raise RuntimeError("call make_host_buffers() before step_from_host()")
        key = ("host", self.k.data_ptr(), self.max_selected, self.max_spans, bool(direct))
        st = self._steps.get(key)
        if st is None:
            if direct:
                tail = self.counts.data_ptr() - self.out_arena.data_ptr()   # counts + status: kernels read them too
                st = ssa.make_step(self.span_offsets, self.spans, self.ctx_lens, self.index, self.counts, self.q,
                                   self.k, self.v, self.max_selected, self.h_out_rows, self.h_lse, self.workspace,
                                   self.status, host_in=self.h_in, dev_in=self.in_arena,
                                   host_out=self.h_out[tail:], dev_out=self.out_arena[tail:], copy_by_kernel=True,
                                   max_spans=self.max_spans)
            else:
                st = ssa.make_step(self.span_offsets, self.spans, self.ctx_lens, self.index, self.counts, self.q,
                                   self.k, self.v, self.max_selected, self.out, self.lse, self.workspace, self.status,
                                   host_in=self.h_in, dev_in=self.in_arena, host_out=self.h_out, dev_out=self.out_arena,
                                   max_spans=self.max_spans)
            self._steps[key] = st
        return ssa.decode_step(self.desc, st, stream)

    def set_spans(self, wl: Workload):
        """Replace the span lists (same geometry, same cache)."""
        assert (wl.B, wl.H, wl.D, wl.max_ctx) == (self.wl.B, self.wl.H, self.wl.D, self.wl.max_ctx)
        assert wl.spans.shape[0] <= self.spans.shape[0] and wl.selected_upper_bound() <= self.index_stride
        self.spans[: wl.spans.shape[0]].copy_(torch.from_numpy(np.ascontiguousarray(wl.spans)))
        self.span_offsets.copy_(torch.from_numpy(wl.span_offsets.copy()))
        self.ctx_lens.copy_(torch.from_numpy(wl.ctx_lens.copy()))
        self.max_selected = max(wl.selected_upper_bound(), 1)
        self.max_spans = int(max(1, np.diff(wl.span_offsets).max()))
        self.wl = wl
        if hasattr(self, "block_size"):
            self._bound_blocks()

    # ---- results ---------------------------------------------------------------------
    def out_f64(self) -> np.ndarray:
        return self.out.detach().to(torch.float64).cpu().numpy()

    def selected_bytes(self) -> int:
        return int(self.counts.clamp(min=0).sum().item()) * self.wl.kv_bytes_per_token()
