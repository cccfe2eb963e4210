"""Pins for the oracle's span -> index list (CPU only)."""
import os
import random

import numpy as np
import pytest

from oracle import ssa_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def ranges(text):
    out = []
    for part in text.split():
        a, b = part.split("-")
        out.extend(range(int(a), int(b) + 1))
    return out


# ---- hand cases -----------------------------------------------------------
def test_hand_cases():
    assert O.spans_to_index([], 10).tolist() == []
    assert O.spans_to_index([(0, 10)], 10).tolist() == list(range(10))
    assert O.spans_to_index([(3, 5), (4, 9)], 20).tolist() == [3, 4, 5, 6, 7, 8]
    assert O.spans_to_index([(7, 30)], 10).tolist() == [7, 8, 9]          # clipped
    assert O.spans_to_index([(5, 5)], 10).tolist() == []                  # empty span
    assert O.spans_to_index([(6, 2)], 10).tolist() == []                  # reversed
    assert O.spans_to_index([(-4, 3)], 10).tolist() == [0, 1, 2]          # negative start
    assert O.spans_to_index([(8, 9), (0, 1), (4, 6)], 10).tolist() == [0, 4, 5, 8]
    assert O.spans_to_index([(2, 4), (4, 6)], 10).tolist() == [2, 3, 4, 5]  # adjacent
    assert O.spans_to_index([(12, 14)], 10).tolist() == []                # beyond n
    assert O.spans_to_index([(0, 3)], 0).tolist() == []
    assert O.spans_to_index([(2, 4)], 10).dtype == np.int32


def test_status_bits():
    assert O.spans_status([(0, 4)], 10) == 0
    assert O.spans_status([(6, 2)], 10) == O.ST_BAD_SPAN
    assert O.spans_status([(-1, 2)], 10) == O.ST_BAD_SPAN
    assert O.spans_status([(3, 11)], 10) == O.ST_CLIPPED
    assert O.spans_status([(0, 10)], 10, index_stride=9) == O.ST_OVERFLOW
    assert O.spans_status([(0, 10)], 10, index_stride=10) == 0
    assert O.spans_status([(5, 5)], 10) == 0


# ---- brute force with a different data structure --------------------------
def brute(spans, n):
    return sorted({j for s, e in spans for j in range(max(s, 0), min(e, n))})


@pytest.mark.parametrize("seed", range(40))
def test_against_set_brute_force(seed):
    rnd = random.Random(seed)
    n = rnd.randint(0, 300)
    spans = []
    for _ in range(rnd.randint(0, 12)):
        s = rnd.randint(-10, n + 10)
        spans.append((s, s + rnd.randint(-5, 60)))
    assert O.spans_to_index(spans, n).tolist() == brute(spans, n)


# ---- invariants ------------------------------------------------------------
@pytest.mark.parametrize("seed", range(20))
def test_invariants(seed):
    rnd = random.Random(1000 + seed)
    n = rnd.randint(50, 400)
    spans = []
    for _ in range(rnd.randint(1, 10)):
        s = rnd.randint(0, n - 1)
        spans.append((s, min(n, s + rnd.randint(1, 50))))
    idx = O.spans_to_index(spans, n)
    # strictly ascending, in range, count = number of marked positions
    assert np.all(np.diff(idx) > 0)
    assert idx.min() >= 0 and idx.max() < n
    mark = np.zeros(n, bool)
    for s, e in spans:
        mark[s:e] = True
    assert len(idx) == int(mark.sum())
    # idempotent: feeding the result back as unit spans
    unit = [(int(j), int(j) + 1) for j in idx]
    assert O.spans_to_index(unit, n).tolist() == idx.tolist()
    # order of spans
    shuffled = spans[:]
    rnd.shuffle(shuffled)
    assert O.spans_to_index(shuffled, n).tolist() == idx.tolist()
    # splitting one span in two
    s, e = spans[0]
    if e - s >= 2:
        mid = rnd.randint(s + 1, e - 1)
        assert O.spans_to_index([(s, mid), (mid, e)] + spans[1:], n).tolist() == idx.tolist()
    # adding a span contained in another, or a duplicate
    s, e = spans[-1]
    inner = (s + (e - s) // 3, e - (e - s) // 3)
    assert O.spans_to_index(spans + [inner, spans[0]], n).tolist() == idx.tolist()


def test_batch_layout_and_truncation():
    offsets = [0, 2, 2, 3]
    spans = [(0, 3), (5, 7), (0, 9)]
    index, counts, st = O.spans_to_index_batch(offsets, spans, [10, 10, 6], index_stride=5)
    assert counts.tolist() == [5, 0, 5]
    assert index[0].tolist() == [0, 1, 2, 5, 6]
    assert index[1].tolist() == [-1] * 5
    assert index[2].tolist() == [0, 1, 2, 3, 4]          # 6 positions, row holds 5
    assert st == (O.ST_CLIPPED | O.ST_OVERFLOW)


# ---- the paper's worked reference examples, as span structure ---------------
def test_golden_arithmetic_references():
    lines, anchors, cases = {}, {}, []
    for raw in open(os.path.join(GOLDEN, "arith_references.txt")):
        t = raw.split("#")[0].split()
        if not t:
            continue
        if t[0] == "line":
            lines[int(t[1])] = (int(t[2]), int(t[3]))
        elif t[0] == "anchor":
            anchors[int(t[1])] = int(t[2])
        elif t[0] == "case":
            n = int(t[t.index("n") + 1])
            prev = int(t[t.index("prev") + 1])
            refs = t[t.index("refs") + 1]
            expect = " ".join(t[t.index("expect") + 1:])
            cases.append((n, prev, refs, expect))
    assert len(cases) == 3
    for n, prev, refs, expect in cases:
        cur = max(k for k, (s, e) in lines.items() if s < n)      # line being generated
        spans = [lines[cur]]                                      # its own tokens (clipped at n)
        if prev:
            spans.append(lines[cur - 1])
        if refs != "-":
            spans += [lines[anchors[int(r)]] for r in refs.split(",")]
        assert O.spans_to_index(spans, n).tolist() == ranges(expect)


def test_golden_summarization_references():
    art, summ, cases, instr = None, {}, [], None
    for raw in open(os.path.join(GOLDEN, "summarization_references.txt")):
        t = raw.split("#")[0].split()
        if not t:
            continue
        if t[0] == "instruction":
            instr = (int(t[1]), int(t[2]))
        elif t[0] == "article_lines":
            art = (int(t[1]), int(t[3]), int(t[5]))
        elif t[0] == "summary":
            summ[int(t[1])] = (int(t[2]), int(t[3]))
        elif t[0] == "case":
            n = int(t[t.index("n") + 1])
            lo, hi = map(int, t[t.index("refs") + 1].split("-"))
            prev = t[t.index("prev") + 1]
            expect = " ".join(t[t.index("expect") + 1:])
            cases.append((n, lo, hi, prev, expect))
    count, first, each = art
    assert count == 31 and len(cases) == 3
    for n, lo, hi, prev, expect in cases:
        cur = max(k for k, (s, e) in summ.items() if s < n)
        spans = [summ[cur], (first + lo * each, first + (hi + 1) * each), instr]
        if prev != "-":
            spans.append(summ[int(prev)])
        assert O.spans_to_index(spans, n).tolist() == ranges(expect)
