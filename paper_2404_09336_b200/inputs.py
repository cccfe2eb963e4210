"""Seeded synthetic decode-attention workloads.

This module only draws inputs: context lengths, span lists and the 16-bit
storage patterns of Q, K and V.  It holds none of the method's arithmetic and
is the one module that both the CUDA path's callers and the CPU checker may
use, so that the two see identical bits.

The five workloads stand in for the paper's tasks (its datasets and
fine-tuned weights are not available): LLaMA-7B attention geometry (32 heads
of 128), an always-attended instruction prefix, a few referenced groups of
contiguous tokens, and the most recent tokens.  Q, K and V are i.i.d. N(0, 1)
drawn in fp32 and rounded to nearest-even into the storage type.  Every row
of the cache up to ``max_ctx`` is filled, also past a request's context
length, so that an over-read changes the result.

Streams: request ``b`` of workload seed ``s`` draws its spans from
``PCG64(SeedSequence([s, b, 0]))``, K and V from stream 1 and q from stream 2,
so any single request can be regenerated without the others.
"""
from __future__ import annotations

import concurrent.futures as _cf
import os
from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20240409

DENSITIES = (0.01, 0.05, 0.10, 0.25, 0.50, 1.00)


def _rng(seed, b, stream):
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(b), int(stream)])))


def round_to_storage(x32: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 -> 16-bit storage pattern (uint16), round to nearest even."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    if dtype == "f16":
        return x32.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        u = x32.view(np.uint32)
        t = u >> np.uint32(16)              # u + 0x7FFF + (bit 16 of u), then keep the upper half
        t &= np.uint32(1)
        t += np.uint32(0x7FFF)
        t += u
        return (t >> np.uint32(16)).astype(np.uint16)
    raise ValueError(dtype)


def _normal_bits(rng, shape, dtype):
    return round_to_storage(rng.standard_normal(shape, dtype=np.float32), dtype)


def _place_disjoint(rng, lo, hi, lengths, placed=None):
    """Rejection-sample start positions so that spans [s, s+len) lie inside
    [lo, hi) and do not overlap one another (they may touch)."""
    placed = [] if placed is None else placed
    for ln in lengths:
        for _ in range(100000):
            s = int(rng.integers(lo, hi - ln + 1))
            if all(s + ln <= a or s >= b for a, b in placed):
                placed.append((s, s + ln))
                break
        else:
            raise RuntimeError("could not place disjoint spans")
    return placed


@dataclass
class Workload:
    name: str
    seed: int
    B: int
    H: int
    D: int
    max_ctx: int
    dtype: str                       # "bf16" | "f16"
    ctx_lens: np.ndarray             # int32 [B]
    span_offsets: np.ndarray         # int32 [B+1]
    spans: np.ndarray                # int32 [S_total, 2]  (start, end)
    seq_ids: np.ndarray = field(default=None)   # global request ids (stream selectors)

    def __post_init__(self):
        if self.seq_ids is None:
            self.seq_ids = np.arange(self.B, dtype=np.int64)

    # ---- inputs ------------------------------------------------------------
    def q_bits(self, heads: int | None = None) -> np.ndarray:
        """uint16 [B, heads, D]; ``heads`` defaults to H (more query heads than
        cache heads: grouped query heads, which the paper's model does not have)."""
        heads = heads or self.H
        out = np.empty((self.B, heads, self.D), np.uint16)
        for i, b in enumerate(self.seq_ids):
            out[i] = _normal_bits(_rng(self.seed, b, 2), (heads, self.D), self.dtype)
        return out

    def kv_bits_seq(self, i: int):
        """(k, v) uint16 [H, max_ctx, D] of the i-th request of this workload."""
        r = _rng(self.seed, self.seq_ids[i], 1)
        k = _normal_bits(r, (self.H, self.max_ctx, self.D), self.dtype)
        v = _normal_bits(r, (self.H, self.max_ctx, self.D), self.dtype)
        return k, v

    def kv_bits(self, threads: int | None = None):
        """(k, v) uint16 [B, H, max_ctx, D]."""
        k = np.empty((self.B, self.H, self.max_ctx, self.D), np.uint16)
        v = np.empty_like(k)

        def one(i):
            k[i], v[i] = self.kv_bits_seq(i)

        threads = threads or min(self.B, os.cpu_count() or 1, 16)
        if threads <= 1:
            for i in range(self.B):
                one(i)
        else:
            with _cf.ThreadPoolExecutor(threads) as ex:
                list(ex.map(one, range(self.B)))
        return k, v

    # ---- bookkeeping ----------------------------------------------------------
    def spans_of(self, i: int) -> np.ndarray:
        return self.spans[self.span_offsets[i]:self.span_offsets[i + 1]]

    def selected_upper_bound(self) -> int:
        """Host-side bound on any request's selected count: the sum of its span
        lengths (what a generation loop knows without reading the device)."""
        best = 0
        for i in range(self.B):
            sp = self.spans_of(i)
            if len(sp):
                best = max(best, int(np.clip(sp[:, 1] - sp[:, 0], 0, None).sum()))
        return min(best, int(self.max_ctx))

    def kv_bytes_per_token(self) -> int:
        """K + V bytes of one selected position over all heads."""
        return 2 * self.H * self.D * 2

    def shard(self, rank: int, world: int) -> "Workload":
        """Requests [lo, hi) of an even split across ``world`` ranks; requests
        are independent, so a shard is a workload of its own."""
        lo = (self.B * rank) // world
        hi = (self.B * (rank + 1)) // world
        s0, s1 = int(self.span_offsets[lo]), int(self.span_offsets[hi])
        return Workload(f"{self.name}[{rank}/{world}]", self.seed, hi - lo, self.H, self.D, self.max_ctx,
                        self.dtype, self.ctx_lens[lo:hi].copy(),
                        (self.span_offsets[lo:hi + 1] - s0).astype(np.int32),
                        self.spans[s0:s1].copy(), self.seq_ids[lo:hi].copy())


def _finish(name, seed, B, H, D, max_ctx, dtype, ctx_lens, per_seq_spans, first_id=0):
    offs = np.zeros(B + 1, np.int32)
    offs[1:] = np.cumsum([len(s) for s in per_seq_spans])
    spans = np.asarray([p for s in per_seq_spans for p in s], dtype=np.int32).reshape(-1, 2)
    return Workload(name, seed, B, H, D, max_ctx, dtype, np.asarray(ctx_lens, np.int32), offs, spans,
                    np.arange(first_id, first_id + B, dtype=np.int64))


def _shuffled(rng, spans):
    order = rng.permutation(len(spans))
    return [spans[i] for i in order]


def make_config(cfg: int, density: float | None = None, B: int | None = None, H: int | None = None,
                first_id: int = 0) -> Workload:
    """Workload ``cfg`` in 1..5.  ``B`` / ``H`` override the batch size and head
    count (smaller copies of the same recipe, for checks the CPU can finish);
    ``first_id`` offsets the request ids (distinct data per rank in a
    multi-process run).  ``density`` selects the point of the sweep (cfg 5)."""
    sub = 0 if density is None else int(round(density * 1000))
    seed = BASE_SEED + 1000 * cfg + sub
    per_seq, ctx = [], []
    if cfg == 1:
        B, H, D, T, dtype, name = B or 1, H or 8, 64, 512, "f16", "tiny"
        for b in range(first_id, first_id + B):
            r = _rng(seed, b, 0)
            mid = _place_disjoint(r, 32, 496, [int(x) for x in r.integers(8, 17, size=3)])
            per_seq.append(_shuffled(r, [(0, 32)] + mid + [(496, 512)]))
            ctx.append(512)
    elif cfg == 2:
        B, H, D, T, dtype, name = B or 64, H or 32, 128, 1024, "bf16", "arithmetic"
        for b in range(first_id, first_id + B):
            r = _rng(seed, b, 0)
            n = int(r.integers(256, 1025))
            k = int(r.integers(1, 5))
            mid = _place_disjoint(r, 64, n - 32, [int(x) for x in r.integers(4, 33, size=k)])
            per_seq.append(_shuffled(r, [(0, 64)] + mid + [(n - 32, n)]))
            ctx.append(n)
    elif cfg == 3:
        B, H, D, T, dtype, name = B or 16, H or 32, 128, 4096, "bf16", "summarization"
        n_lines = -(-(3968 - 64) // 40)                     # 97 full lines + a 24-token tail line
        for b in range(first_id, first_id + B):
            r = _rng(seed, b, 0)
            sp = [(0, 64), (4032, 4096)]
            for _ in range(int(r.integers(2, 11))):
                cnt = int(r.integers(1, 6))
                first = int(r.integers(0, n_lines - cnt + 1))
                sp.append((64 + 40 * first, min(64 + 40 * (first + cnt), 3968)))
            per_seq.append(_shuffled(r, sp))
            ctx.append(4096)
    elif cfg == 4:
        B, H, D, T, dtype, name = B or 8, H or 32, 128, 16384, "bf16", "long_context"
        for b in range(first_id, first_id + B):
            r = _rng(seed, b, 0)
            mid = _place_disjoint(r, 64, 16256, [int(x) for x in r.integers(32, 257, size=16)])
            per_seq.append(_shuffled(r, [(0, 64)] + mid + [(16256, 16384)]))
            ctx.append(16384)
    elif cfg == 5:
        if density is None:
            raise ValueError("cfg 5 needs a density")
        B, H, D, T, dtype = B or 32, H or 32, 128, 8192, "bf16"
        name = f"density_{int(round(density * 100))}pct"
        target = int(round(density * 8192))
        for b in range(first_id, first_id + B):
            r = _rng(seed, b, 0)
            if target >= 8192:
                per_seq.append([(0, 8192)])
            else:
                total, placed = 64, []
                while total < target:
                    ln = min(int(r.integers(16, 257)), target - total)
                    _place_disjoint(r, 0, 8128, [ln], placed)
                    total += ln
                per_seq.append(_shuffled(r, [(8128, 8192)] + placed))
            ctx.append(8192)
    else:
        raise ValueError(f"no workload {cfg}")
    return _finish(name, seed, B, H, D, T, dtype, ctx, per_seq, first_id)


def make_mixed(every: int, B: int | None = None, H: int | None = None, first_id: int = 0) -> Workload:
    """Workload 2 with every ``every``-th request at a "determine span" step of
    the method (Sec. "Self-selected attention span", Inference: such a step
    attends to the whole preceding context): its list is the single span
    [0, ctx_len); the other requests keep their selected spans."""
    base = make_config(2, B=B, H=H, first_id=first_id)
    per_seq = []
    for i in range(base.B):
        if i % every == 0:
            per_seq.append([(0, int(base.ctx_lens[i]))])
        else:
            per_seq.append([tuple(int(x) for x in p) for p in base.spans_of(i)])
    return _finish(f"mixed_every_{every}", base.seed, base.B, base.H, base.D, base.max_ctx, base.dtype,
                   base.ctx_lens, per_seq, first_id)


def make_microbench(ctx: int, sparsity_block: int, B: int = 64, H: int = 32, max_ctx: int | None = None,
                    first_id: int = 0) -> Workload:
    """The paper's kernel micro-benchmark (Sec. "Custom CUDA kernel
    benchmarking"): one new token over ``ctx`` preceding tokens of which half
    are ignored; the binary mask is made of blocks of ones of size
    ``sparsity_block`` (exactly half of the aligned blocks, drawn at random
    per request); batch 64; LLaMA-7B heads.  ``max_ctx`` lets several context
    lengths share one cache allocation."""
    if ctx % sparsity_block:
        raise ValueError("the context must be a multiple of the sparsity block")
    seed = BASE_SEED + 6000
    n_blocks = ctx // sparsity_block
    per_seq = []
    for b in range(first_id, first_id + B):
        r = _rng(seed + ctx + sparsity_block, b, 0)
        keep = np.sort(r.permutation(n_blocks)[: n_blocks // 2])
        per_seq.append(_shuffled(r, [(int(k) * sparsity_block, (int(k) + 1) * sparsity_block) for k in keep]))
    wl = _finish(f"paper_microbench_ctx{ctx}_sb{sparsity_block}", seed, B, H, 128, max_ctx or ctx, "bf16",
                 [ctx] * B, per_seq, first_id)
    return wl
