"""Pins for the oracle's reference resolution (CPU only): the paper's two worked
examples, as recorded in tests/golden/, must come out of the anchor tables."""
import os

import numpy as np

from oracle import ssa_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def ranges(text):
    out = []
    for part in text.split():
        a, b = part.split("-")
        out.extend(range(int(a), int(b) + 1))
    return out


def test_arithmetic_example():
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
            cases.append((int(t[t.index("n") + 1]), int(t[t.index("prev") + 1]), t[t.index("refs") + 1],
                          " ".join(t[t.index("expect") + 1:])))
    order = sorted(lines)
    for n, prev, refs, expect in cases:
        cur = max(k for k in order if lines[k][0] < n)                 # the line being generated
        done = [lines[k] for k in order if k < cur]                    # completed lines
        anchor_line = [order.index(anchors[a]) for a in sorted(anchors) if anchors[a] < cur]
        pairs = [(-1, -1)] if prev else []
        if refs != "-":
            pairs += [(int(r), int(r)) for r in refs.split(",")]
        spans, st = O.resolve_references(done, anchor_line, pairs, 0, lines[cur][0], n)
        assert st == 0
        assert O.spans_to_index(spans, n).tolist() == ranges(expect)


def test_summarization_example():
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
            lo, hi = map(int, t[t.index("refs") + 1].split("-"))
            cases.append((int(t[t.index("n") + 1]), lo, hi, t[t.index("prev") + 1],
                          " ".join(t[t.index("expect") + 1:])))
    count, first, each = art
    article = [(first + i * each, first + (i + 1) * each) for i in range(count)]
    for n, lo, hi, prev, expect in cases:
        cur = max(k for k, (s, e) in summ.items() if s < n)
        done = article + [summ[k] for k in sorted(summ) if k < cur]    # article lines, then finished sentences
        pairs = [(lo, hi)] + ([(-1, -1)] if prev != "-" else [])       # the line numbers are the anchors
        spans, st = O.resolve_references(done, list(range(count)), pairs, instr[1], summ[cur][0], n)
        assert st == 0
        assert O.spans_to_index(spans, n).tolist() == ranges(expect)


def test_order_padding_and_flags():
    lines = [(10, 20), (20, 35), (40, 50)]
    spans, st = O.resolve_references(lines, [2, 0], [(0, 1), (-2, -2)], 4, 60, 66, span_stride=6)
    assert st == 0
    assert spans.tolist() == [[0, 4], [60, 66], [40, 50], [10, 20], [20, 35], [0, 0]]
    spans, st = O.resolve_references(lines, [2, 0], [(0, 1), (-1, -1), (-3, -3)], 4, 60, 66, span_stride=4)
    assert st == O.ST_OVERFLOW and spans.tolist() == [[0, 4], [60, 66], [40, 50], [10, 20]]
    for bad in ([(5, 5)], [(-4, -4)], [(1, 0)], [(-1, 2)], [(-2, -1)]):
        spans, st = O.resolve_references(lines, [2, 0], bad, 4, 60, 66)
        assert st == O.ST_BAD_REF and spans.tolist() == [[0, 4], [60, 66]]
    spans, st = O.resolve_references(lines, [7], [(0, 0)], 0, 0, 0)                  # anchor points nowhere
    assert st == O.ST_BAD_REF and spans.tolist() == [[0, 0], [0, 0]]
    spans, st = O.resolve_references([], [], [], 3, 3, 9)
    assert st == 0 and O.spans_to_index(spans, 9).tolist() == list(range(9))
