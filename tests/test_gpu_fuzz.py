"""Randomised shapes through the restricted and the full-context call against
the oracle: head counts and groupings, head sizes, storage types, cache
layouts, list lengths (empty, one entry, everything), sorted and unsorted
lists, loose and tight host bounds, output in fp32 or the storage type."""
import random

import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O

from gpu_util import Problem, random_bits
from parity import parity_report

pytestmark = pytest.mark.gpu


def one_case(case):
    rnd = random.Random(case)
    D = rnd.choice([64, 128])
    dtype = rnd.choice(["bf16", "f16"])
    Hkv = rnd.choice([1, 2, 3, 4])
    G = rnd.choice([1, 1, 2, 3, 4, 8, 16, 20])
    H = Hkv * G
    B = rnd.choice([1, 2, 5, 17, 40, 150]) if H < 40 else rnd.choice([1, 2, 5, 17])
    T = rnd.choice([1, 7, 64, 65, 255, 513, 700, 1500, 2600])
    if B * Hkv * T * D > 40e6:
        T = max(1, int(40e6 // (B * Hkv * D)))
    layout = rnd.choice(["bhtd", "bthd"])
    p = Problem(B, Hkv, T, D, dtype, seed=case, layout=layout)
    rng = np.random.default_rng(case)
    p.q_bits = random_bits(rng, (B, H, D), dtype)
    p.H = H
    p.upload()
    ctx = [int(rng.integers(1, T + 1)) for _ in range(B)]
    counts = [int(rng.integers(0, n + 1)) if rnd.random() < 0.8 else rnd.choice([0, 1, n]) for n in ctx]
    stride = max(counts + [1]) + rnd.choice([0, 3, 40])
    index = np.full((B, stride), -1, np.int32)
    for b in range(B):
        sel = rng.choice(ctx[b], counts[b], replace=False)
        index[b, :counts[b]] = np.sort(sel) if rnd.random() < 0.7 else sel
    ms = rnd.choice([stride, max(counts + [1])])
    native = rnd.random() < 0.3
    what = f"case {case}: B={B} H={H} Hkv={Hkv} D={D} {dtype} T={T} {layout} ms={ms} stride={stride} native={native}"
    out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=ms, out_dtype=None if native else torch.float32)
    sample = sorted(set(rng.integers(0, B, size=min(B, 6)).tolist()))
    kr, vr = np.repeat(p.k_bits, G, axis=1), np.repeat(p.v_bits, G, axis=1)
    scale = 1 / np.sqrt(D)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, kr, vr, ctx, index, counts, scale, dtype, seqs=sample)
    r = parity_report(out[sample], ref[sample])
    assert status == 0 and np.all(np.isfinite(out)), what
    assert (r["fails"] == 0) if native else (r["max_abs"] <= 2e-3 and r["max_rel"] <= 1e-2), f"{what}: {r}"
    fin = np.isfinite(ref_lse[sample])
    np.testing.assert_allclose(lse[sample][fin], ref_lse[sample][fin], rtol=1e-5, atol=1e-5, err_msg=what)
    assert np.all(np.isneginf(lse[sample][~fin])), what
    out_d, _, st_d = p.dense(ctx)
    ref_d, _ = O.decode_attn_dense(p.q_bits, kr, vr, ctx, scale, dtype, seqs=sample)
    rd = parity_report(out_d[sample], ref_d[sample])
    assert st_d == 0 and rd["max_abs"] <= 2e-3 and rd["max_rel"] <= 1e-2, f"{what}, dense: {rd}"


@pytest.mark.parametrize("first", range(0, 48, 8))
def test_random_shapes(first):
    for case in range(first, first + 8):
        one_case(case)
        torch.cuda.empty_cache()


def one_span_case(case):
    """Random span lists straight to attention (ssa_decode_attn_spans): list lengths around the 32- and 128-span
    limits of the two on-chip merges, offsets or a fixed-stride table, with and without the lists written out."""
    from paper_2404_09336_b200 import ssa
    from gpu_util import DEV
    rnd = random.Random(1000 + case)
    D = rnd.choice([64, 128])
    dtype = rnd.choice(["bf16", "f16"])
    Hkv = rnd.choice([1, 2, 4])
    G = rnd.choice([1, 1, 2, 4])
    H = Hkv * G
    B = rnd.choice([1, 3, 9, 33])
    T = rnd.choice([40, 300, 1100, 2300])
    p = Problem(B, Hkv, T, D, dtype, seed=1000 + case)
    rng = np.random.default_rng(1000 + case)
    p.q_bits = random_bits(rng, (B, H, D), dtype)
    p.H = H
    p.upload()
    ctx = [int(rng.integers(1, T + 1)) for _ in range(B)]
    max_spans = rnd.choice([1, 3, 8, 9, 31, 32, 33, 100, 128])
    lists = []
    for b in range(B):
        k = int(rng.integers(0, max_spans + 1))
        lists.append([(int(a), int(a + rng.integers(0, max(2, T // 8)))) for a in rng.integers(-2, ctx[b] + 3, size=k)])
    fixed = rnd.random() < 0.4
    if fixed:
        table = np.zeros((B, max_spans, 2), np.int32)
        for b, sp in enumerate(lists):
            for i, pair in enumerate(sp):
                table[b, i] = pair
        d_sp, d_off = torch.from_numpy(table).to(DEV), None
    else:
        offs = np.cumsum([0] + [len(s) for s in lists]).astype(np.int32)
        flat = np.asarray([x for s in lists for x in s] or [(0, 0)], np.int32).reshape(-1, 2)
        d_sp, d_off = torch.from_numpy(flat).to(DEV), torch.from_numpy(offs).to(DEV)
    ref_idx = [O.spans_to_index(s, n) for s, n in zip(lists, ctx)]
    ms = max(max(len(i) for i in ref_idx), 1) + rnd.choice([0, 5])
    stride = (ms + 31) // 32 * 32
    want_lists = rnd.random() < 0.5
    index = torch.full((B, stride), -7, dtype=torch.int32, device=DEV)
    counts = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    out = torch.full((B, H, D), 5.0, dtype=torch.float32, device=DEV)
    lse = torch.zeros((B, H), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_spans_workspace_bytes(desc, ms, max_spans), dtype=torch.uint8, device=DEV)
    ssa.decode_attn_spans(desc, p.q, p.k, p.v, d_ctx, d_off, d_sp, max_spans, ms, out, lse,
                          index if want_lists else None, counts if want_lists else None, ws, status)
    torch.cuda.synchronize()
    what = f"span case {case}: B={B} H={H} Hkv={Hkv} D={D} {dtype} T={T} spans<={max_spans} fixed={fixed} lists={want_lists}"
    ri = np.full((B, ms), -1, np.int32)
    rc = np.zeros(B, np.int32)
    for b, idx in enumerate(ref_idx):
        ri[b, :len(idx)], rc[b] = idx, len(idx)
        if want_lists:
            assert int(counts[b]) == len(idx) and index[b, :len(idx)].cpu().numpy().tolist() == idx.tolist(), what
    kr, vr = np.repeat(p.k_bits, G, axis=1), np.repeat(p.v_bits, G, axis=1)
    ref, _ = O.decode_attn_sparse(p.q_bits, kr, vr, ctx, ri, rc, 1 / np.sqrt(D), dtype)
    r = parity_report(out.double().cpu().numpy(), ref)
    assert np.all(np.isfinite(out.cpu().numpy())) and r["max_abs"] <= 2e-3 and r["max_rel"] <= 1e-2, f"{what}: {r}"


@pytest.mark.parametrize("first", range(0, 40, 8))
def test_random_span_lists(first):
    for case in range(first, first + 8):
        one_span_case(case)
        torch.cuda.empty_cache()
