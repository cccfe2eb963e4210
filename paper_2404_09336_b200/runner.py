"""Device-side plumbing around the C-ABI calls: buffers for one workload and
the two-call decode step (span list -> index list -> attention).

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


class DecodeStep:
    """Buffers of one workload on one GPU.

    layout "bhtd": cache stored [B, H, T, D] (one contiguous plane per head);
    layout "bthd": cache stored [B, T, H, D] (token-major).  Either way
    ``self.k`` / ``self.v`` are the logical [B, H, T, D] views.
    ``kv_copies`` > 1 keeps several copies of the cache so that consecutive
    timed steps read different memory.
    """

    def __init__(self, wl: Workload, device="cuda:0", layout="bhtd", out_dtype=None, kv_copies=1,
                 index_stride=None, max_selected=None, gen_threads=None):
        self.wl, self.device, self.layout = wl, torch.device(device), layout
        dt = _TORCH_DTYPE[wl.dtype]
        dev = self.device
        B, H, D, T = wl.B, wl.H, wl.D, wl.max_ctx
        self.q = bits_to_tensor(wl.q_bits(), wl.dtype).to(dev)
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
        self.ctx_lens = torch.from_numpy(wl.ctx_lens.copy()).to(dev)
        self.span_offsets = torch.from_numpy(wl.span_offsets.copy()).to(dev)
        spans = wl.spans if len(wl.spans) else np.zeros((1, 2), np.int32)
        self.spans = torch.from_numpy(np.ascontiguousarray(spans)).to(dev)
        self.max_selected = int(max_selected or max(wl.selected_upper_bound(), 1))
        self.index_stride = int(index_stride or (self.max_selected + 31) // 32 * 32)
        self.index = torch.full((B, self.index_stride), -7, dtype=torch.int32, device=dev)
        self.counts = torch.full((B,), -7, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out = torch.zeros((B, H, D), dtype=out_dtype or dt, device=dev)
        self.lse = torch.zeros((B, H), dtype=torch.float32, device=dev)
        self.desc = ssa.make_desc(self.q, self.k, self.v, self.out, max_ctx=T)
        need = max(ssa.decode_workspace_bytes(self.desc, self.max_selected),
                   ssa.decode_workspace_bytes(self.desc, T))
        if need == 0:
            raise RuntimeError("ssa_decode_workspace_bytes rejected the descriptor")
        self.workspace = torch.empty(need, dtype=torch.uint8, device=dev)

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

    def attend_dense(self, stream=None):
        return ssa.decode_attn_dense(self.desc, self.q, self.k, self.v, self.ctx_lens, self.out, self.lse,
                                     self.workspace, self.status, stream)

    def step(self, stream=None):
        """One decode step of the method: span lists -> index lists -> attention."""
        self.build_index(stream)
        self.attend_sparse(stream)

    # ---- host-buffer form (end-to-end timing) -----------------------------------------
    def make_host_buffers(self):
        """Pinned host copies of what changes every decode step (query rows and
        span lists) and pinned landing buffers for what the caller reads back.
        Returns (host-to-device bytes, device-to-host bytes) per step."""
        pin = lambda t: t.detach().cpu().pin_memory()
        self.h_q, self.h_spans = pin(self.q), pin(self.spans)
        self.h_offsets, self.h_ctx = pin(self.span_offsets), pin(self.ctx_lens)
        self.h_out = torch.empty(self.out.shape, dtype=self.out.dtype).pin_memory()
        self.h_counts = torch.empty(self.counts.shape, dtype=torch.int32).pin_memory()
        self.h_status = torch.empty(1, dtype=torch.int32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in (self.h_q, self.h_spans, self.h_offsets, self.h_ctx))
        d2h = sum(t.numel() * t.element_size() for t in (self.h_out, self.h_counts, self.h_status))
        return h2d, d2h

    def step_from_host(self, stream=None):
        """Decode step whose per-step inputs start in (pinned) host memory and
        whose result ends there; the KV cache is the resident state."""
        self.q.copy_(self.h_q, non_blocking=True)
        self.spans.copy_(self.h_spans, non_blocking=True)
        self.span_offsets.copy_(self.h_offsets, non_blocking=True)
        self.ctx_lens.copy_(self.h_ctx, non_blocking=True)
        self.step(stream)
        self.h_out.copy_(self.out, non_blocking=True)
        self.h_counts.copy_(self.counts, non_blocking=True)
        self.h_status.copy_(self.status, non_blocking=True)

    # ---- results ---------------------------------------------------------------------
    def out_f64(self) -> np.ndarray:
        return self.out.detach().to(torch.float64).cpu().numpy()

    def selected_bytes(self) -> int:
        return int(self.counts.clamp(min=0).sum().item()) * self.wl.kv_bytes_per_token()
