"""Pins for the oracle's blocked span encoding (CPU only)."""
import random

import numpy as np
import pytest

from oracle import ssa_oracle as O


def test_hand_example():
    # block size 32, context 100: positions 1, 2, 40..43, 99
    bi, wd = O.spans_to_blockmask([(1, 3), (40, 44), (99, 120)], 100, 32)
    assert bi.tolist() == [0, 1, 3]                              # block 2 (64..95) is empty: omitted
    assert wd[:, 0].tolist() == [0b110, 0b1111 << 8, 1 << 3]
    # block size 64: two words per block
    bi, wd = O.spans_to_blockmask([(1, 3), (40, 44), (99, 120)], 100, 64)
    assert bi.tolist() == [0, 1]
    assert wd.tolist() == [[0b110, 0b1111 << 8], [0, 1 << 3]]
    # a block-aligned span gives an all-ones mask; nothing selected gives an empty list
    bi, wd = O.spans_to_blockmask([(64, 128)], 200, 64)
    assert bi.tolist() == [1] and wd.tolist() == [[0xFFFFFFFF, 0xFFFFFFFF]]
    bi, wd = O.spans_to_blockmask([], 200, 64)
    assert len(bi) == 0 and wd.shape == (0, 2)
    with pytest.raises(ValueError):
        O.spans_to_blockmask([(0, 1)], 10, 48)


@pytest.mark.parametrize("seed", range(24))
def test_round_trip_and_structure(seed):
    rnd = random.Random(seed)
    n = rnd.randint(1, 2000)
    bs = rnd.choice([32, 64, 128, 256])
    spans = []
    for _ in range(rnd.randint(0, 15)):
        s = rnd.randint(-5, n + 5)
        spans.append((s, s + rnd.randint(-3, 150)))
    idx = O.spans_to_index(spans, n)
    bi, wd = O.spans_to_blockmask(spans, n, bs)
    assert O.blockmask_to_index(bi, wd, bs).tolist() == idx.tolist()        # decoding gives back the set
    assert np.all(np.diff(bi) > 0)                                           # ascending, no repeats
    assert np.all(wd.any(axis=1)) if len(bi) else True                       # no empty block is listed
    assert bi.tolist() == sorted({int(j) // bs for j in idx})                # exactly the touched blocks
    pop = sum(bin(int(w)).count("1") for w in wd.ravel())
    assert pop == len(idx)


def test_batch_layout_and_truncation():
    offsets = [0, 1, 1, 3]
    spans = [(0, 70), (10, 20), (500, 600)]
    bi, wd, counts, st = O.spans_to_blockmask_batch(offsets, spans, [100, 50, 550], 32, 2)
    assert counts.tolist() == [2, 0, 2]
    assert bi[0].tolist() == [0, 1] and bi[1].tolist() == [-1, -1] and bi[2].tolist() == [0, 15]
    assert st == (O.ST_OVERFLOW | O.ST_CLIPPED)                  # request 0 has 3 blocks; request 2's span is clipped
    assert wd[2, 1, 0] == ((1 << 32) - 1) ^ ((1 << 20) - 1)      # positions 500..511 of block 15 (480..511)


def test_attention_from_the_encoding_equals_algorithm_1():
    rng = np.random.default_rng(3)
    B, H, T, D, bs = 2, 2, 300, 8, 32
    q = rng.standard_normal((B, H, D))
    K = rng.standard_normal((B, H, T, D))
    V = rng.standard_normal((B, H, T, D))
    ctx = [300, 170]
    offsets, spans = [0, 2, 4], [(5, 40), (100, 131), (0, 3), (160, 400)]
    bi, wd, counts, _ = O.spans_to_blockmask_batch(offsets, spans, ctx, bs, 16)
    out, lse = O.decode_attn_blockmask(q, K, V, ctx, bi, wd, counts, bs, 0.35)
    for b in range(B):
        idx = O.spans_to_index(spans[offsets[b]:offsets[b + 1]], ctx[b])
        meta = O.encode_blocked(idx, bs)
        for h in range(H):
            o, l = O.attn_alg1_blocked(q[b, h], K[b, h], V[b, h], ctx[b], meta, bs, 0.35)
            np.testing.assert_allclose(out[b, h], o, rtol=1e-12, atol=1e-14)
            assert lse[b, h] == pytest.approx(l, rel=1e-13)
