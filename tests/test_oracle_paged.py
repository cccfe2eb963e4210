"""The oracle's definition of a paged cache layout, pinned by what fixes it:
an identity table over a pool cut from a contiguous cache gives the cache back,
and scattering a cache's rows to shuffled pages and gathering them restores it."""
import numpy as np

from oracle import ssa_oracle as O


def test_identity_table_returns_the_contiguous_cache():
    rng = np.random.default_rng(0)
    B, H, T, D, ps = 3, 2, 64, 4, 16
    cache = rng.integers(0, 65536, size=(B, H, T, D)).astype(np.uint16)
    # request b owns pages b*T/ps .. (b+1)*T/ps - 1, in order
    pool = cache.transpose(0, 2, 1, 3).reshape(B * T // ps, ps, H, D)
    table = np.arange(B * T // ps, dtype=np.int32).reshape(B, T // ps)
    assert np.array_equal(O.gather_pages(pool, table, ps, T), cache)


def test_scatter_to_shuffled_pages_then_gather_restores_every_row():
    rng = np.random.default_rng(1)
    B, H, T, D, ps, n_pages = 2, 3, 40, 2, 8, 17
    cache = rng.integers(0, 65536, size=(B, H, T, D)).astype(np.uint16)
    perm = rng.permutation(n_pages)[: B * T // ps].astype(np.int32).reshape(B, T // ps)
    pool = np.full((n_pages, ps, H, D), 0xFFFF, np.uint16)
    for b in range(B):
        for t in range(T):                                     # written out position by position
            pool[perm[b, t // ps], t % ps] = cache[b, :, t, :]
    assert np.array_equal(O.gather_pages(pool, perm, ps, T), cache)
    # a table entry outside the pool leaves its positions zero and touches nothing else
    bad = perm.copy()
    bad[1, 2] = n_pages
    got = O.gather_pages(pool, bad, ps, T)
    assert not got[1, :, 2 * ps:3 * ps].any()
    got[1, :, 2 * ps:3 * ps] = cache[1, :, 2 * ps:3 * ps]
    assert np.array_equal(got, cache)
