"""ssa_spans_to_index against the oracle: bit-exact lists and counts."""
import random

import numpy as np
import pytest

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs, ssa

from gpu_util import run_index

pytestmark = pytest.mark.gpu


def compare(span_lists, ctx_lens, index_stride, expect_status=None):
    index, counts, status, (offs, flat) = run_index(span_lists, ctx_lens, index_stride)
    ref_index, ref_counts, ref_status = O.spans_to_index_batch(offs, flat[: offs[-1]], ctx_lens, index_stride)
    assert counts.tolist() == ref_counts.tolist()
    for b in range(len(span_lists)):
        c = int(ref_counts[b])
        assert index[b, :c].tolist() == ref_index[b, :c].tolist(), f"request {b}"
        assert np.all(index[b, c:] == -7)                    # padding left untouched
    assert status == (ref_status if expect_status is None else expect_status)
    return index, counts, status


def wl_lists(wl):
    return [wl.spans_of(i).tolist() for i in range(wl.B)]


@pytest.mark.parametrize("cfg", [1, 2, 3, 4])
def test_configs(cfg):
    wl = inputs.make_config(cfg)
    stride = (wl.selected_upper_bound() + 31) // 32 * 32
    _, counts, status = compare(wl_lists(wl), wl.ctx_lens.tolist(), stride)
    assert status == 0 and counts.min() > 0


@pytest.mark.parametrize("f", inputs.DENSITIES)
def test_density_sweep(f):
    wl = inputs.make_config(5, density=f)
    _, counts, status = compare(wl_lists(wl), wl.ctx_lens.tolist(), 8192)
    assert status == 0 and np.all(counts == round(f * 8192))


def test_hand_cases():
    lists = [
        [],                                   # no spans
        [(0, 10)],                            # whole context
        [(3, 5), (4, 9)],                     # overlap
        [(8, 9), (0, 1), (4, 6)],             # unsorted
        [(2, 4), (4, 6)],                     # adjacent
        [(5, 5)],                             # empty span
        [(1, 3), (1, 3), (1, 3)],             # repeated
        [(0, 10), (2, 4)],                    # contained
        [(9, 10)],                            # last position only
    ]
    compare(lists, [10] * len(lists), 16, expect_status=0)


def test_flags_and_clipping():
    compare([[(6, 2)]], [10], 16, expect_status=ssa.DEV_BAD_SPAN)
    compare([[(-4, 3)]], [10], 16, expect_status=ssa.DEV_BAD_SPAN)
    compare([[(7, 30)]], [10], 16, expect_status=ssa.DEV_CLIPPED)
    compare([[(12, 14)]], [10], 16, expect_status=ssa.DEV_CLIPPED)
    compare([[(0, 3)]], [0], 16, expect_status=ssa.DEV_CLIPPED)
    compare([[(0, 5)], [(0, 40)], [(2, 3)]], [50, 50, 50], 32, expect_status=ssa.DEV_OVERFLOW)
    index, counts, _ = compare([[(0, 64)]], [64], 64)          # exactly full row: no overflow
    assert counts[0] == 64


def test_many_spans_and_long_lists():
    rnd = random.Random(5)
    for n_spans in (31, 32, 33, 100, 1000, 2048):
        n = 20000
        sp = []
        for _ in range(n_spans):
            s = rnd.randint(0, n - 1)
            sp.append((s, s + rnd.randint(0, 40)))
        compare([sp, sp[: n_spans // 2], sp[::-1]], [n, n // 2, n], 20000)
    # one span over a very long context, written by several blocks
    compare([[(5, 100000)]], [99999], 100032)
    # more spans than one request may have: the surplus is ignored and flagged
    sp = [(2 * i, 2 * i + 1) for i in range(2049)]
    index, counts, status, _ = run_index([sp], [10000], 4096)
    assert status & ssa.DEV_TOO_MANY_SPANS
    assert counts[0] == 2048 and index[0, :2048].tolist() == [2 * i for i in range(2048)]


@pytest.mark.parametrize("seed", range(8))
def test_fuzz(seed):
    rnd = random.Random(100 + seed)
    lists, ctx = [], []
    for _ in range(rnd.randint(1, 40)):
        n = rnd.randint(0, 3000)
        sp = []
        for _ in range(rnd.randint(0, 70)):
            s = rnd.randint(-20, n + 20)
            sp.append((s, s + rnd.randint(-10, 200)))
        lists.append(sp)
        ctx.append(n)
    compare(lists, ctx, rnd.choice([64, 512, 3008]))


def test_invariance_to_order_and_splitting():
    wl = inputs.make_config(3)
    lists = wl_lists(wl)
    stride = 4096
    base, counts, _, _ = run_index(lists, wl.ctx_lens.tolist(), stride)
    rnd = random.Random(1)
    alt = []
    for sp in lists:
        sp = [tuple(x) for x in sp]
        s, e = sp[0]
        mid = (s + e) // 2
        sp = [(s, mid), (mid, e)] + sp[1:] + [sp[-1]]
        rnd.shuffle(sp)
        alt.append(sp)
    again, counts2, _, _ = run_index(alt, wl.ctx_lens.tolist(), stride)
    assert np.array_equal(counts, counts2)
    for b in range(wl.B):
        assert np.array_equal(base[b, :counts[b]], again[b, :counts[b]])
