"""ssa_refs_to_spans against the oracle (bit-exact span rows), ssa_refs_to_index
(the same plus the index expansion in one launch, bit-exact lists), and the whole
chain references -> spans -> index lists -> attention on the device."""
import random

import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import ssa

from gpu_util import DEV, Problem
from parity import assert_parity

pytestmark = pytest.mark.gpu


def flat(lists, width):
    offs = np.zeros(len(lists) + 1, np.int32)
    offs[1:] = np.cumsum([len(x) for x in lists])
    data = np.asarray([v for x in lists for v in x], np.int32).reshape(-1, width) if offs[-1] else \
        np.zeros((1, width), np.int32)
    return torch.from_numpy(offs).to(DEV), torch.from_numpy(np.ascontiguousarray(data)).to(DEV)


def run_refs(reqs, stride):
    """reqs: list of dicts(lines, anchors, refs, prefix, start, ctx)."""
    B = len(reqs)
    lo, ld = flat([r["lines"] for r in reqs], 2)
    ao, ad = flat([[(a,) for a in r["anchors"]] for r in reqs], 1)
    ro, rd = flat([r["refs"] for r in reqs], 2)
    i32 = lambda k: torch.tensor([r[k] for r in reqs], dtype=torch.int32, device=DEV)
    prefix, start, ctx = i32("prefix"), i32("start"), i32("ctx")
    so = torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)
    sp = torch.full((B, stride, 2), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ssa.refs_to_spans(lo, ld, ao, ad.view(-1), ro, rd, prefix, start, ctx, so, sp, status)
    torch.cuda.synchronize()
    return so, sp, ctx, int(status.item())


def compare(reqs, stride):
    so, sp, ctx, status = run_refs(reqs, stride)
    want_status = 0
    for b, r in enumerate(reqs):
        ref, st = O.resolve_references(r["lines"], r["anchors"], r["refs"], r["prefix"], r["start"], r["ctx"], stride)
        want_status |= st
        assert sp[b].cpu().numpy().tolist() == ref.tolist(), f"request {b}"
    assert so.cpu().numpy().tolist() == [b * stride for b in range(len(reqs) + 1)]
    gpu_bits = {O.ST_OVERFLOW: ssa.DEV_OVERFLOW, O.ST_BAD_REF: ssa.DEV_BAD_REF}
    assert status == sum(v for k, v in gpu_bits.items() if want_status & k)
    return so, sp, ctx


def fuzz_requests(seed):
    rnd = random.Random(seed)
    reqs = []
    for _ in range(rnd.randint(1, 30)):
        n_lines = rnd.randint(0, 50)
        pos, lines = rnd.randint(0, 20), []
        prefix = pos
        for _ in range(n_lines):
            ln = rnd.randint(1, 30)
            lines.append((pos, pos + ln))
            pos += ln + rnd.randint(0, 2)
        anchors = [rnd.randint(-1, n_lines) for _ in range(rnd.randint(0, 20))]
        refs = []
        for _ in range(rnd.randint(0, 40)):
            if rnd.random() < 0.3:
                k = -rnd.randint(1, n_lines + 2)
                refs.append((k, k))
            else:
                a = rnd.randint(-1, len(anchors) + 1)
                refs.append((a, a + rnd.randint(-1, 4)))
        reqs.append(dict(lines=lines, anchors=anchors, refs=refs, prefix=prefix, start=pos, ctx=pos + rnd.randint(0, 9)))
    return reqs


def run_refs_index(reqs, index_stride):
    B = len(reqs)
    lo, ld = flat([r["lines"] for r in reqs], 2)
    ao, ad = flat([[(a,) for a in r["anchors"]] for r in reqs], 1)
    ro, rd = flat([r["refs"] for r in reqs], 2)
    i32 = lambda k: torch.tensor([r[k] for r in reqs], dtype=torch.int32, device=DEV)
    index = torch.full((B, index_stride), -7, dtype=torch.int32, device=DEV)
    counts = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ssa.refs_to_index(lo, ld, ao, ad.view(-1), ro, rd, i32("prefix"), i32("start"), i32("ctx"), index, counts, status)
    torch.cuda.synchronize()
    return index.cpu().numpy(), counts.cpu().numpy(), int(status.item())


def compare_index(reqs, index_stride, max_spans=2048):
    """One launch against the oracle's resolver followed by its span -> index definition."""
    index, counts, status = run_refs_index(reqs, index_stride)
    want_status = 0
    for b, r in enumerate(reqs):
        spans, st = O.resolve_references(r["lines"], r["anchors"], r["refs"], r["prefix"], r["start"], r["ctx"])
        if len(spans) > max_spans:
            spans, st = spans[:max_spans], st | 1 << 20          # marker for "too many spans"
        want_status |= st | O.spans_status(spans, r["ctx"], index_stride)
        idx = O.spans_to_index(spans, r["ctx"])[:index_stride]
        assert counts[b] == len(idx), f"request {b}"
        assert index[b, :len(idx)].tolist() == idx.tolist(), f"request {b}"
        assert np.all(index[b, len(idx):] == -7)                 # nothing written past the list
    gpu_bits = {O.ST_BAD_SPAN: ssa.DEV_BAD_SPAN, O.ST_CLIPPED: ssa.DEV_CLIPPED, O.ST_OVERFLOW: ssa.DEV_OVERFLOW,
                O.ST_BAD_REF: ssa.DEV_BAD_REF, 1 << 20: ssa.DEV_TOO_MANY_SPANS}
    assert status == sum(v for k, v in gpu_bits.items() if want_status & k)
    return index, counts


def test_paper_examples_and_flags():
    arith = dict(lines=[(0, 14), (14, 40), (40, 54), (54, 66)], anchors=[0, 2, 3], refs=[(0, 0), (1, 1), (2, 2)],
                 prefix=0, start=66, ctx=69)
    summ = dict(lines=[(12 + 8 * i, 20 + 8 * i) for i in range(31)] + [(260, 280)], anchors=list(range(31)),
                refs=[(17, 19), (-1, -1)], prefix=12, start=280, ctx=291)
    so, sp, ctx = compare([arith, summ], 8)
    # union of the resolved spans = the positions the paper's examples attend to
    assert O.spans_to_index(sp[0].cpu().numpy(), 69).tolist() == list(range(0, 14)) + list(range(40, 69))
    assert O.spans_to_index(sp[1].cpu().numpy(), 291).tolist() == \
        list(range(0, 12)) + list(range(148, 172)) + list(range(260, 291))
    compare([dict(arith, refs=[(0, 2), (-1, -1), (-2, -2), (-4, -4)])], 5)          # overflow: 2 + 6 spans
    for bad in ([(5, 5)], [(-9, -9)], [(1, 0)], [(-1, 2)], [(0, 7)]):
        compare([dict(arith, refs=bad)], 8)
    compare([dict(lines=[], anchors=[], refs=[], prefix=3, start=3, ctx=9)], 2)
    compare([dict(arith, anchors=[0, 9, 3])], 8)                                    # an anchor that points nowhere


def test_one_launch_paper_examples_and_flags():
    arith = dict(lines=[(0, 14), (14, 40), (40, 54), (54, 66)], anchors=[0, 2, 3], refs=[(0, 0), (1, 1), (2, 2)],
                 prefix=0, start=66, ctx=69)
    summ = dict(lines=[(12 + 8 * i, 20 + 8 * i) for i in range(31)] + [(260, 280)], anchors=list(range(31)),
                refs=[(17, 19), (-1, -1)], prefix=12, start=280, ctx=291)
    index, counts = compare_index([arith, summ], 320)
    assert index[0, :counts[0]].tolist() == list(range(0, 14)) + list(range(40, 69))
    assert index[1, :counts[1]].tolist() == list(range(0, 12)) + list(range(148, 172)) + list(range(260, 291))
    compare_index([arith, summ], 40)                                                # lists cut at index_stride
    for bad in ([(5, 5)], [(-9, -9)], [(1, 0)], [(-1, 2)], [(0, 7)]):
        compare_index([dict(arith, refs=bad)], 96)
    compare_index([dict(lines=[], anchors=[], refs=[], prefix=3, start=3, ctx=9)], 16)
    compare_index([dict(arith, anchors=[0, 9, 3])], 96)                             # an anchor that points nowhere
    compare_index([dict(arith, ctx=60)], 96)                                        # lines beyond the context: clipped
    compare_index([dict(arith, prefix=-2), dict(arith, start=80)], 96)              # malformed prefix / current line
    # many references: more than 32 spans (sorted in shared memory by the whole block), and more than the
    # 2048 a request may resolve to (the first 2048 are kept)
    lines = [(4 * i, 4 * i + 3) for i in range(700)]
    many = dict(lines=lines, anchors=list(range(700)), refs=[(i, i + 2) for i in range(0, 690, 7)], prefix=0,
                start=2800, ctx=2810)
    compare_index([many, arith], 2816)
    too_many = dict(many, refs=[(0, 699)] * 3)
    compare_index([too_many, summ], 2816)
    # several output slices per request
    compare_index([dict(many, refs=[(0, 699)])], 2816)


def test_references_far_beyond_the_anchor_table_cost_nothing_and_are_flagged():
    """A pair (lo, hi) with hi in the billions must neither be walked anchor by anchor nor lose its flag.
    The oracle walks every named anchor, so it is given the same pair cut one anchor past the table: the
    anchors beyond the table contribute nothing but the flag, and that one anchor already raises it."""
    arith = dict(lines=[(0, 14), (14, 40), (40, 54), (54, 66)], anchors=[0, 2, 3], prefix=0, start=66, ctx=69)
    for lo in (0, 1, 3, 5):
        for hi in (1 << 30, 2 ** 31 - 1):
            on_device = [dict(arith, refs=[(lo, hi), (-1, -1)])]
            for_oracle = dict(arith, refs=[(lo, max(lo, 3)), (-1, -1)])
            so, sp, ctx, status = run_refs(on_device, 8)
            ref, st = O.resolve_references(for_oracle["lines"], for_oracle["anchors"], for_oracle["refs"], 0, 66, 69, 8)
            assert st & O.ST_BAD_REF
            assert sp[0].cpu().numpy().tolist() == ref.tolist()
            assert status == ssa.DEV_BAD_REF
            index, counts, status = run_refs_index(on_device, 96)
            want = O.spans_to_index(ref, 69)
            assert counts[0] == len(want) and index[0, :len(want)].tolist() == want.tolist()
            assert status == ssa.DEV_BAD_REF


@pytest.mark.parametrize("seed", range(5))
def test_one_launch_fuzz(seed):
    reqs = fuzz_requests(seed + 100)
    compare_index(reqs, random.Random(seed).choice([64, 700, 2000]))


@pytest.mark.parametrize("seed", range(5))
def test_fuzz(seed):
    reqs = fuzz_requests(seed)
    compare(reqs, random.Random(seed + 50).choice([4, 32, 100]))


def test_references_to_attention_on_the_device():
    rnd = random.Random(3)
    B, H, T, D = 4, 2, 900, 128
    p = Problem(B, H, T, D, "bf16", seed=5)
    reqs = []
    for b in range(B):
        lines = [(20 + 40 * i, 60 + 40 * i) for i in range(18)]
        refs = [(rnd.randint(0, 8), rnd.randint(9, 17)), (-1, -1)] if b else [(3, 3)]
        reqs.append(dict(lines=lines, anchors=list(range(18)), refs=refs, prefix=20, start=740, ctx=760 + 30 * b))
    stride = 32
    so, sp, ctx, status = run_refs(reqs, stride)
    assert status == 0
    index = torch.full((B, T), -7, dtype=torch.int32, device=DEV)
    counts = torch.zeros(B, dtype=torch.int32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    ssa.spans_to_index(so, sp.view(-1, 2), ctx, index, counts, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ctx_l = [r["ctx"] for r in reqs]
    out, lse, status, _ = p.sparse(ctx_l, index.cpu().numpy(), counts.cpu().numpy().tolist(), max_selected=T)
    want_idx = np.full((B, T), -1, np.int32)
    want_cnt = []
    for b, r in enumerate(reqs):
        spans, _ = O.resolve_references(r["lines"], r["anchors"], r["refs"], r["prefix"], r["start"], r["ctx"])
        idx = O.spans_to_index(spans, r["ctx"])
        want_idx[b, :len(idx)] = idx
        want_cnt.append(len(idx))
    assert counts.cpu().numpy().tolist() == want_cnt
    ref, _ = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, ctx_l, want_idx, want_cnt, 1 / np.sqrt(D), "bf16")
    assert_parity(out, ref, False, "references to attention")


def test_generation_loop_with_growing_context():
    # several consecutive decode steps as a generation loop makes them: the context grows by one row per
    # step, the current line grows with it, every third step is a "determine span" step over everything
    B, H, T, D = 3, 2, 400, 128
    p = Problem(B, H, T, D, "bf16", seed=8)
    lines = [(16 + 30 * i, 46 + 30 * i) for i in range(8)]                     # completed lines, 16..256
    reqs = [dict(lines=lines, anchors=list(range(8)), refs=[(b, b + 2), (-1, -1)], prefix=16, start=256,
                 ctx=300 + 7 * b) for b in range(B)]
    lo, ld = flat([r["lines"] for r in reqs], 2)
    ao, ad = flat([[(a,) for a in r["anchors"]] for r in reqs], 1)
    ro, rd = flat([r["refs"] for r in reqs], 2)
    full_ro = torch.zeros(B + 1, dtype=torch.int32, device=DEV)                # no references: prefix + line only
    i32 = lambda vals: torch.tensor(vals, dtype=torch.int32, device=DEV)
    prefix, start = i32([r["prefix"] for r in reqs]), i32([r["start"] for r in reqs])
    zero = i32([0] * B)
    ctx = i32([r["ctx"] for r in reqs])
    stride = 16
    so = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
    sp = torch.zeros((B, stride, 2), dtype=torch.int32, device=DEV)
    index = torch.zeros((B, T), dtype=torch.int32, device=DEV)
    counts = torch.zeros(B, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = torch.zeros((B, H, D), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_workspace_bytes(desc, T), dtype=torch.uint8, device=DEV)
    for step in range(7):
        determine = step % 3 == 0
        if determine:       # the whole context: an empty prefix and a "line" that starts at 0
            ssa.refs_to_spans(lo, ld, ao, ad.view(-1), full_ro, rd, zero, zero, ctx, so, sp, status)
        else:
            ssa.refs_to_spans(lo, ld, ao, ad.view(-1), ro, rd, prefix, start, ctx, so, sp, status)
        ssa.spans_to_index(so, sp.view(-1, 2), ctx, index, counts, status)
        ssa.decode_attn_sparse(desc, p.q, p.k, p.v, ctx, index, counts, T, out, None, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ctx_l = ctx.cpu().tolist()
        want_idx, want_cnt = np.full((B, T), -1, np.int32), []
        for b, r in enumerate(reqs):
            if determine:
                idx = np.arange(ctx_l[b], dtype=np.int32)
            else:
                spans, _ = O.resolve_references(r["lines"], r["anchors"], r["refs"], r["prefix"], r["start"], ctx_l[b])
                idx = O.spans_to_index(spans, ctx_l[b])
            want_idx[b, :len(idx)] = idx
            want_cnt.append(len(idx))
        assert counts.cpu().tolist() == want_cnt
        ref, _ = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, ctx_l, want_idx, want_cnt, 1 / np.sqrt(D), "bf16")
        assert_parity(out.double().cpu().numpy(), ref, False, f"step {step}")
        ctx += 1                                                               # the next token's row is appended
