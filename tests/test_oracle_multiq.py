"""Pins of the oracle's several-query-tokens form: it is the single-query set form row by row.  What fixes it
without re-typing its formula: one query token reproduces the single-query call; rows do not influence one
another; permuting the query rows permutes the outputs; a one-token selection returns that V row for every
query row; a zero query row returns the mean of the selected V rows; a library scaled-dot-product attention
in fp64 with the selection as a boolean mask agrees; grouped heads read the cache head they belong to."""
import numpy as np
import torch

from oracle import ssa_oracle as O


def problem(B=2, H=3, Tq=4, T=50, D=8, seed=0, Hkv=None):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, Tq, D))
    k = rng.standard_normal((B, Hkv or H, T, D))
    v = rng.standard_normal((B, Hkv or H, T, D))
    ctx = np.array([T, T - 7][:B])
    index = np.full((B, 16), -1, np.int32)
    counts = np.zeros(B, np.int32)
    for b in range(B):
        c = int(rng.integers(3, 15))
        index[b, :c] = np.sort(rng.choice(int(ctx[b]), c, replace=False))
        counts[b] = c
    return q, k, v, ctx, index, counts


def test_one_query_token_is_the_single_query_call():
    q, k, v, ctx, index, counts = problem(Tq=1)
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.3)
    ref, ref_lse = O.decode_attn_sparse(q[:, :, 0], k, v, ctx, index, counts, 0.3)
    assert np.array_equal(out[:, :, 0], ref) and np.array_equal(lse[:, :, 0], ref_lse)


def test_rows_are_independent_and_permute_with_the_queries():
    q, k, v, ctx, index, counts = problem()
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.3)
    q2 = q.copy()
    q2[:, :, 1] = 100.0                                        # another query row changes: the rest stays
    out2, _ = O.decode_attn_sparse_multiq(q2, k, v, ctx, index, counts, 0.3)
    keep = [0, 2, 3]
    assert np.array_equal(out2[:, :, keep], out[:, :, keep]) and not np.allclose(out2[:, :, 1], out[:, :, 1])
    perm = [2, 0, 3, 1]
    outp, lsep = O.decode_attn_sparse_multiq(q[:, :, perm], k, v, ctx, index, counts, 0.3)
    assert np.array_equal(outp, out[:, :, perm]) and np.array_equal(lsep, lse[:, :, perm])
    # each row equals the single-query call on that row
    for t in range(q.shape[2]):
        ref, _ = O.decode_attn_sparse(q[:, :, t], k, v, ctx, index, counts, 0.3)
        assert np.array_equal(out[:, :, t], ref)


def test_closed_forms():
    q, k, v, ctx, index, counts = problem(B=1, H=2, Tq=3)
    index[0, 0], counts[0] = 11, 1                             # one selected token: weight 1, whatever the query
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.7)
    for t in range(3):
        assert np.array_equal(out[0, :, t], v[0, :, 11])
        np.testing.assert_allclose(lse[0, :, t], 0.7 * np.einsum("hd,hd->h", q[0, :, t], k[0, :, 11]), rtol=1e-14)
    q, k, v, ctx, index, counts = problem(B=1, H=2, Tq=2, seed=3)
    q[0, :, 1] = 0.0                                           # zero query: uniform weights
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.7)
    sel = index[0, :counts[0]]
    np.testing.assert_allclose(out[0, :, 1], v[0][:, sel].mean(axis=1), rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(lse[0, :, 1], np.log(counts[0]), rtol=1e-14)
    counts[0] = 0                                              # empty selection: zero rows, lse = -inf
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.7)
    assert not out.any() and np.all(np.isneginf(lse))


def test_library_attention_with_a_boolean_mask_agrees():
    q, k, v, ctx, index, counts = problem(B=2, H=3, Tq=5, T=40, D=16, seed=5)
    out, _ = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.25)
    for b in range(2):
        mask = torch.zeros(5, 40, dtype=torch.bool)
        mask[:, index[b, :counts[b]].astype(np.int64)] = True
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[b]), torch.from_numpy(k[b]), torch.from_numpy(v[b]), attn_mask=mask, scale=0.25)
        np.testing.assert_allclose(out[b], ref.numpy(), rtol=1e-12, atol=1e-13)


def test_grouped_heads_read_their_cache_head():
    q, k, v, ctx, index, counts = problem(B=2, H=6, Tq=2, Hkv=2, seed=7)
    out, lse = O.decode_attn_sparse_multiq(q, k, v, ctx, index, counts, 0.3)
    ref, ref_lse = O.decode_attn_sparse_multiq(q, np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1), ctx, index,
                                               counts, 0.3)
    assert np.array_equal(out, ref) and np.array_equal(lse, ref_lse)
    # a planted mistake in the head mapping (h % H_kv instead of h // group) would read other rows
    wrong, _ = O.decode_attn_sparse_multiq(q, np.tile(k, (1, 3, 1, 1)), np.tile(v, (1, 3, 1, 1)), ctx, index, counts, 0.3)
    assert not np.allclose(wrong, out)
