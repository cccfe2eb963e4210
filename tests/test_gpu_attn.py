"""ssa_decode_attn_sparse / ssa_decode_attn_dense against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs, ssa
from paper_2404_09336_b200.runner import DecodeStep

from gpu_util import DEV, Problem, random_bits, run_index
from parity import assert_parity

pytestmark = pytest.mark.gpu


def scale_of(D):
    return 1.0 / np.sqrt(D)


def oracle_for(wl, ds, seqs=None, heads=None):
    """Oracle output for a workload from the generator's own bits (never from
    device memory): index lists by the oracle, attention in set form."""
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    seqs = list(range(wl.B)) if seqs is None else list(seqs)
    q = wl.q_bits()
    out = np.full((wl.B, wl.H, wl.D), np.nan)
    lse = np.full((wl.B, wl.H), np.nan)
    dense = np.full((wl.B, wl.H, wl.D), np.nan)
    for b in seqs:
        k, v = wl.kv_bits_seq(b)
        o, l = O.decode_attn_sparse(q[b:b + 1], k[None], v[None], wl.ctx_lens[b:b + 1], index[b:b + 1],
                                    counts[b:b + 1], scale_of(wl.D), wl.dtype, heads=heads)
        out[b], lse[b] = o[0], l[0]
        od, _ = O.decode_attn_dense(q[b:b + 1], k[None], v[None], wl.ctx_lens[b:b + 1], scale_of(wl.D),
                                    wl.dtype, heads=heads)
        dense[b] = od[0]
    return out, lse, dense, index, counts


def run_and_compare(wl, layout="bhtd", out_dtype=None, seqs=None, heads=None):
    ds = DecodeStep(wl, layout=layout, out_dtype=out_dtype)
    ref, ref_lse, ref_dense, ref_index, ref_counts = oracle_for(wl, ds, seqs, heads)
    ds.step()
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    counts = ds.counts.cpu().numpy()
    assert counts.tolist() == ref_counts.tolist()
    idx = ds.index.cpu().numpy()
    for b in range(wl.B):
        assert np.array_equal(idx[b, :counts[b]], ref_index[b, :counts[b]])
    got, got_lse = ds.out_f64(), ds.lse.double().cpu().numpy()
    native = out_dtype is None
    sel = ~np.isnan(ref)
    r = assert_parity(got[sel], ref[sel], native, f"{wl.name} sparse {layout}")
    sel_l = ~np.isnan(ref_lse)
    np.testing.assert_allclose(got_lse[sel_l], ref_lse[sel_l], rtol=1e-5, atol=1e-5)
    ds.out.fill_(55.0)
    ds.attend_dense()
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    assert_parity(ds.out_f64()[sel], ref_dense[sel], native, f"{wl.name} dense {layout}")
    return r


# ---- the five workloads, scaled so that the oracle covers every output ----------------
@pytest.mark.parametrize("layout", ["bhtd", "bthd"])
@pytest.mark.parametrize("out_dtype", [None, torch.float32])
def test_cfg1_tiny_full(layout, out_dtype):
    run_and_compare(inputs.make_config(1), layout, out_dtype)


@pytest.mark.parametrize("layout", ["bhtd", "bthd"])
@pytest.mark.parametrize("out_dtype", [None, torch.float32])
def test_cfg2_reduced(layout, out_dtype):
    run_and_compare(inputs.make_config(2, B=6, H=4), layout, out_dtype)


@pytest.mark.parametrize("out_dtype", [None, torch.float32])
def test_cfg3_reduced(out_dtype):
    run_and_compare(inputs.make_config(3, B=3, H=3), "bhtd", out_dtype)


def test_cfg4_reduced():
    run_and_compare(inputs.make_config(4, B=2, H=2), "bhtd", torch.float32)
    run_and_compare(inputs.make_config(4, B=1, H=2), "bthd", None)


@pytest.mark.parametrize("f", [0.01, 0.10, 1.00])
def test_cfg5_reduced(f):
    run_and_compare(inputs.make_config(5, density=f, B=2, H=2), "bhtd", torch.float32)


# ---- full sizes, in the launch configuration the benchmark times; sampled outputs -----
@pytest.mark.parametrize("cfg,density", [(2, None), (3, None), (4, None), (5, 0.01), (5, 0.05), (5, 0.10), (5, 0.25),
                                         (5, 0.50), (5, 1.00)])
def test_full_size_sampled(cfg, density):
    wl = inputs.make_config(cfg, density=density)
    rng = np.random.default_rng(cfg)
    seqs = sorted(rng.choice(wl.B, size=2, replace=False).tolist())
    heads = sorted(rng.choice(wl.H, size=3, replace=False).tolist())
    run_and_compare(wl, "bhtd", None, seqs=seqs, heads=heads)


# ---- edge cases on hand-made problems ----------------------------------------------------
def oracle_sparse(p, ctx, index, counts, scale=None):
    return O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, ctx, index, counts,
                                scale_of(p.D) if scale is None else scale, p.dtype)


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f16", 128), ("bf16", 64), ("f16", 64)])
@pytest.mark.parametrize("layout", ["bhtd", "bthd"])
def test_counts_zero_one_and_ragged(dtype, D, layout):
    B, H, T = 5, 3, 700
    p = Problem(B, H, T, D, dtype, seed=D, layout=layout)
    ctx = [700, 1, 513, 64, 300]
    rng = np.random.default_rng(0)
    index = np.full((B, 704), -1, np.int32)
    counts = [0, 1, 513, 17, 300]
    index[1, 0] = 0
    index[2, :513] = np.arange(513)
    index[3, :17] = np.sort(rng.choice(64, 17, replace=False))
    index[4, :300] = rng.permutation(300)                     # unsorted list
    for out_dtype in (torch.float32, None):
        out, lse, status, _ = p.sparse(ctx, index, counts, out_dtype=out_dtype)
        ref, ref_lse = oracle_sparse(p, ctx, index, counts)
        assert status == 0
        assert not out[0].any() and np.all(np.isneginf(lse[0]))            # empty selection
        assert_parity(out, ref, out_dtype is None, "edge")
        np.testing.assert_allclose(lse[1:], ref_lse[1:], rtol=1e-5, atol=1e-5)
    # a single selected row is returned exactly
    out, _, _, _ = p.sparse(ctx, index, counts, out_dtype=torch.float32)
    assert np.array_equal(out[1], O.decode_bits(p.v_bits[1, :, 0, :], dtype))


def test_multi_chunk_merge_and_tail_sizes():
    # sizes around the tile, chunk and split boundaries
    B, H, T, D = 1, 2, 3000, 128
    p = Problem(B, H, T, D, "bf16", seed=7)
    rng = np.random.default_rng(3)
    for c in (1, 15, 16, 17, 63, 64, 65, 255, 256, 257, 511, 513, 1000, 2999, 3000):
        index = np.full((B, 3008), -1, np.int32)
        index[0, :c] = np.sort(rng.choice(T, c, replace=False))
        for ms in {c, 3000}:
            out, lse, status, _ = p.sparse([T], index, [c], max_selected=ms)
            ref, ref_lse = oracle_sparse(p, [T], index, [c])
            assert status == 0
            assert_parity(out, ref, False, f"c={c} ms={ms}")
            np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("B,H", [(2, 2), (5, 32)])
def test_one_chunk_or_several_on_both_sides_of_the_switch(B, H):
    # the host picks one chunk per request or several from (B*H, max_selected): list lengths and contexts
    # right below and above the sizes where that choice changes, for few and for many (request, head) pairs
    D = 128
    rng = np.random.default_rng(B)
    for T in (256, 257, 512, 513):
        p = Problem(B, H, T, D, "bf16", seed=T + B)
        ctx = [T] * B
        counts = [T] + [int(rng.integers(1, T + 1)) for _ in range(B - 1)]
        index = np.full((B, T + 7), -1, np.int32)
        for b in range(B):
            index[b, :counts[b]] = np.sort(rng.choice(T, counts[b], replace=False))
        out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=T)
        ref, ref_lse = oracle_sparse(p, ctx, index, counts)
        assert status == 0
        assert_parity(out, ref, False, f"sparse T={T}")
        np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
        out_d, lse_d, st_d = p.dense(ctx)
        ref_d, ref_lse_d = O.decode_attn_dense(p.q_bits, p.k_bits, p.v_bits, ctx, scale_of(D), "bf16")
        assert st_d == 0
        assert_parity(out_d, ref_d, False, f"dense T={T}")
        np.testing.assert_allclose(lse_d, ref_lse_d, rtol=1e-5, atol=1e-5)


def test_large_batch_of_short_ragged_requests():
    # thousands of requests, one head each, lengths 0..600: several chunks per request, many empty ones
    B, H, T, D = 4100, 1, 600, 64
    p = Problem(B, H, T, D, "bf16", seed=29)
    rng = np.random.default_rng(9)
    ctx = rng.integers(1, T + 1, size=B).tolist()
    counts = [int(rng.integers(0, n + 1)) for n in ctx]
    counts[0], counts[1], counts[2] = 0, ctx[1], 1
    index = np.full((B, 608), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(ctx[b], counts[b], replace=False))
    out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=600)
    ref, ref_lse = oracle_sparse(p, ctx, index, counts)
    assert status == 0
    assert_parity(out, ref, False, "large batch")
    ok = np.isfinite(ref_lse)
    np.testing.assert_allclose(lse[ok], ref_lse[ok], rtol=1e-5, atol=1e-5)
    assert np.all(np.isneginf(lse[~ok]))
    out_d, _, st_d = p.dense(ctx)
    ref_d, _ = O.decode_attn_dense(p.q_bits, p.k_bits, p.v_bits, ctx, scale_of(D), "bf16")
    assert st_d == 0
    assert_parity(out_d, ref_d, False, "large batch dense")


def test_full_span_equals_dense():
    B, H, T, D = 3, 2, 1500, 128
    p = Problem(B, H, T, D, "bf16", seed=11)
    ctx = [1500, 777, 1]
    index = np.tile(np.arange(1504, dtype=np.int32), (B, 1))
    out_s, lse_s, st, _ = p.sparse(ctx, index, ctx, max_selected=1500)
    out_d, lse_d, st_d = p.dense(ctx)
    ref, ref_lse = O.decode_attn_dense(p.q_bits, p.k_bits, p.v_bits, ctx, scale_of(D), "bf16")
    assert st == 0 and st_d == 0
    assert_parity(out_s, ref, False, "sparse full span")
    assert_parity(out_d, ref, False, "dense")
    np.testing.assert_allclose(out_s, out_d, rtol=0, atol=1e-5)
    np.testing.assert_allclose(lse_d, ref_lse, rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(lse_s, ref_lse, rtol=1e-5, atol=1e-5)


def test_unselected_rows_do_not_matter():
    B, H, T, D = 2, 2, 600, 128
    p = Problem(B, H, T, D, "bf16", seed=13)
    ctx = [600, 400]
    rng = np.random.default_rng(1)
    index = np.full((B, 608), -1, np.int32)
    counts = [150, 90]
    index[0, :150] = np.sort(rng.choice(600, 150, replace=False))
    index[1, :90] = np.sort(rng.choice(400, 90, replace=False))
    base, base_lse, _, _ = p.sparse(ctx, index, counts)
    for b in range(B):                                         # poison everything unselected
        keep = np.zeros(T, bool)
        keep[index[b, :counts[b]]] = True
        p.k_bits[b][:, ~keep, :] = 0x7FC0                      # NaN
        p.v_bits[b][:, ~keep, :] = 0x7F80                      # +inf
    p.upload()
    out, lse, status, _ = p.sparse(ctx, index, counts)
    assert status == 0
    assert np.array_equal(out, base) and np.array_equal(lse, base_lse)
    ref, _ = oracle_sparse(p, ctx, index, counts)
    assert_parity(out, ref, False, "poisoned")


def test_bad_entries_are_skipped_and_flagged():
    B, H, T, D = 2, 2, 300, 64
    p = Problem(B, H, T, D, "f16", seed=17)
    ctx = [200, 300]
    index = np.full((B, 64), -1, np.int32)
    index[0, :6] = [5, 250, 7, -3, 199, 200]                  # 250, -3, 200 are outside [0, 200)
    index[1, :4] = [1, 1, 2, 299]                             # a duplicate counts twice
    counts = [6, 4]
    out, lse, status, _ = p.sparse(ctx, index, counts)
    assert status == ssa.DEV_BAD_INDEX
    ref, ref_lse = oracle_sparse(p, ctx, index, counts)
    assert_parity(out, ref, False, "bad entries")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    # a count above the host bound is clamped and flagged
    index[0, :40] = np.arange(40)
    out, _, status, _ = p.sparse(ctx, index, [40, 4], max_selected=32)
    assert status & ssa.DEV_BAD_COUNT
    ref, _ = oracle_sparse(p, ctx, index, [32, 4])
    assert_parity(out, ref, False, "clamped count")
    # a context length above the allocated rows is clamped and flagged (dense)
    out, _, status = p.dense([999, 300])
    assert status & ssa.DEV_BAD_COUNT
    ref, _ = O.decode_attn_dense(p.q_bits, p.k_bits, p.v_bits, [300, 300], scale_of(D), "f16")
    assert_parity(out, ref, False, "clamped ctx")


def test_explicit_scale_and_large_scores():
    B, H, T, D = 1, 2, 256, 128
    p = Problem(B, H, T, D, "bf16", seed=19)
    index = np.arange(256, dtype=np.int32)[None]
    for scale in (1.0, 0.01):                                 # scale 1: nearly one-hot softmax
        out, lse, _, _ = p.sparse([256], index, [256], scale=scale)
        ref, ref_lse = oracle_sparse(p, [256], index, [256], scale=scale)
        assert_parity(out, ref, False, f"scale {scale}")
        np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-4)


def test_strided_views_and_launch_counter():
    # q and out as slices of larger buffers (strides differ from the packed ones)
    B, H, T, D = 2, 3, 128, 128
    p = Problem(B, H, T, D, "bf16", seed=23)
    big_q = torch.zeros((B, H, 2 * D), dtype=torch.bfloat16, device="cuda:0")
    big_q[:, :, :D] = p.q
    p.q = big_q[:, :, :D]
    index = np.tile(np.arange(0, 128, 2, dtype=np.int32), (B, 1))
    before = ssa.launch_count()
    out, _, status, _ = p.sparse([128, 128], index, [64, 64])
    assert ssa.launch_count() > before
    ref, _ = oracle_sparse(p, [128, 128], index, [64, 64])
    assert_parity(out, ref, False, "strided q")


@pytest.mark.parametrize("H,Hkv", [(3, 3), (8, 2)])
@pytest.mark.parametrize("how", ["base", "row_stride"])
def test_cache_aligned_to_16_but_not_32_bytes(H, Hkv, how):
    # the 256-bit row loads need 32-byte alignment; a cache that only has the 16 bytes the interface asks for
    # (base address, or a row stride of D + 8 elements) takes the path with two 128-bit loads per piece
    B, T, D = 2, 300, 128
    p = Problem(B, Hkv, T, D, "bf16", seed=41 + H)
    rng = np.random.default_rng(H)
    p.q_bits = random_bits(rng, (B, H, D), "bf16")
    p.H = H
    p.upload()
    def carve(t):
        if how == "base":
            flat = torch.zeros(t.numel() + 8, dtype=t.dtype, device=t.device)
            view = flat[8:].view(t.shape)
        else:
            wide = torch.zeros((B, Hkv, T, D + 8), dtype=t.dtype, device=t.device)
            view = wide[..., :D]
        view.copy_(t)
        return view
    p.k, p.v = carve(p.k), carve(p.v)
    assert p.k.data_ptr() % 16 == 0 and (p.k.data_ptr() % 32 == 16 or p.k.stride(2) % 16 == 8)
    ctx = [300, 177]
    counts = [150, 60]
    index = np.full((B, 304), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(ctx[b], counts[b], replace=False))
    g = H // Hkv
    k_rep, v_rep = np.repeat(p.k_bits, g, axis=1), np.repeat(p.v_bits, g, axis=1)
    out, lse, status, _ = p.sparse(ctx, index, counts)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, k_rep, v_rep, ctx, index, counts, scale_of(D), "bf16")
    assert status == 0
    assert_parity(out, ref, False, "16-byte aligned cache, sparse")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    out_d, _, _ = p.dense(ctx)
    ref_d, _ = O.decode_attn_dense(p.q_bits, k_rep, v_rep, ctx, scale_of(D), "bf16")
    assert_parity(out_d, ref_d, False, "16-byte aligned cache, dense")


@pytest.mark.parametrize("H,Hkv,D,dtype", [(8, 2, 128, "bf16"), (8, 4, 128, "f16"), (16, 2, 128, "bf16"),
                                           (12, 1, 128, "f16"), (32, 2, 128, "bf16"), (6, 2, 128, "bf16"),
                                           (40, 2, 128, "bf16"), (8, 2, 64, "bf16")])
def test_grouped_query_heads_share_a_kv_head(H, Hkv, D, dtype):
    # not in the paper (LLaMA-7B is multi-head): H query heads over H_kv cache heads.  Groups of 2..16 heads with
    # D = 128 run on the kernel that reads a row once per group (2, 3, 6, 8, 12, 16 heads here); larger groups
    # and D = 64 on the one-head-per-block kernel.  Poisoned unselected rows, ragged and empty lists, bad entries.
    B, T = 4, 700
    p = Problem(B, Hkv, T, D, dtype, seed=31 + H)              # cache with H_kv heads
    rng = np.random.default_rng(H)
    p.q_bits = random_bits(rng, (B, H, D), dtype)
    p.H = H
    ctx = [700, 333, 64, 500]
    counts = [300, 120, 64, 0]
    index = np.full((B, 704), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(ctx[b], counts[b], replace=False))
    nan = 0x7FC0 if dtype == "bf16" else 0x7E00
    for b in range(B):                                         # rows nobody selects hold NaN
        unselected = np.setdiff1d(np.arange(T), index[b, :counts[b]])
        p.k_bits[b][:, unselected] = nan
        p.v_bits[b][:, unselected] = nan
    p.upload()
    g = H // Hkv
    k_rep, v_rep = np.repeat(p.k_bits, g, axis=1), np.repeat(p.v_bits, g, axis=1)
    for ms in (700, 300):                                      # several chunks per request / one
        out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=ms)
        ref, ref_lse = O.decode_attn_sparse(p.q_bits, k_rep, v_rep, ctx, index, counts, scale_of(D), dtype)
        assert status == 0
        assert not out[3].any() and np.all(np.isneginf(lse[3]))
        assert_parity(out, ref, False, f"grouped queries ms={ms}")
        np.testing.assert_allclose(lse[:3], ref_lse[:3], rtol=1e-5, atol=1e-5)
    out, _, _, _ = p.sparse(ctx, index, counts, max_selected=700, out_dtype=None)
    assert_parity(out, ref, True, "grouped queries, output in the storage type")
    # an entry outside the context is skipped and flagged
    bad = index.copy()
    bad[0, 5], bad[1, 0] = 700, -3
    out, lse, status, _ = p.sparse(ctx, bad, counts, max_selected=700)
    keep = [np.delete(bad[0, :300], 5), bad[1, 1:120], bad[2, :64], bad[3, :0]]
    want = np.full((B, 704), -1, np.int32)
    for b in range(B):
        want[b, :len(keep[b])] = keep[b]
    ref_b, _ = O.decode_attn_sparse(p.q_bits, k_rep, v_rep, ctx, want, [len(x) for x in keep], scale_of(D), dtype)
    assert status == ssa.DEV_BAD_INDEX
    assert_parity(out, ref_b, False, "grouped queries, bad entries")
    # full context (clean cache)
    q = Problem(B, Hkv, T, D, dtype, seed=77 + H)
    q.q_bits = random_bits(rng, (B, H, D), dtype)
    q.H = H
    q.upload()
    out_d, lse_d, _ = q.dense(ctx)
    ref_d, ref_lse_d = O.decode_attn_dense(q.q_bits, np.repeat(q.k_bits, g, axis=1), np.repeat(q.v_bits, g, axis=1),
                                           ctx, scale_of(D), dtype)
    assert_parity(out_d, ref_d, False, "grouped queries, dense")
    np.testing.assert_allclose(lse_d, ref_lse_d, rtol=1e-5, atol=1e-5)


def test_grouped_query_heads_large_ragged_batch():
    # every tile shape of the row-sharing kernel: list lengths 0..600 over 300 requests, 8 heads on 2
    B, H, Hkv, T, D = 300, 8, 2, 600, 128
    p = Problem(B, Hkv, T, D, "bf16", seed=5)
    rng = np.random.default_rng(6)
    p.q_bits = random_bits(rng, (B, H, D), "bf16")
    p.H = H
    p.upload()
    ctx = rng.integers(1, T + 1, size=B).tolist()
    counts = [int(rng.integers(0, n + 1)) for n in ctx]
    index = np.full((B, 608), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = rng.permutation(ctx[b])[:counts[b]]        # unsorted lists
    out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=600)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, np.repeat(p.k_bits, 4, axis=1), np.repeat(p.v_bits, 4, axis=1),
                                        ctx, index, counts, scale_of(D), "bf16")
    assert status == 0
    assert_parity(out, ref, False, "grouped queries, ragged batch")
    ok = np.isfinite(ref_lse)
    np.testing.assert_allclose(lse[ok], ref_lse[ok], rtol=1e-5, atol=1e-5)
    assert np.all(np.isneginf(lse[~ok]))


@pytest.mark.parametrize("B,H,Hkv,T", [(350, 4, 2, 1100), (80, 32, 2, 1200)])
def test_grouped_heads_chunks_longer_than_the_staging_area(B, H, Hkv, T):
    # with many (request, K/V head) pairs the row-sharing kernel takes chunks of more than 512 entries and walks
    # them in windows: lists up to the whole context, a bad entry in a late window, sparse and full-context calls
    D = 128
    p = Problem(B, Hkv, T, D, "bf16", seed=B)
    rng = np.random.default_rng(B + 1)
    p.q_bits = random_bits(rng, (B, H, D), "bf16")
    p.H = H
    p.upload()
    ctx = rng.integers(T // 2, T + 1, size=B).tolist()
    ctx[0] = T
    counts = [int(rng.integers(0, n + 1)) for n in ctx]
    counts[0], counts[1] = T, 1
    index = np.full((B, T + 4), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(ctx[b], counts[b], replace=False))
    g = H // Hkv
    k_rep, v_rep = np.repeat(p.k_bits, g, axis=1), np.repeat(p.v_bits, g, axis=1)
    sample = sorted(set([0, 1, 2, B // 2, B - 1] + rng.integers(0, B, size=12).tolist()))
    out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=T)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, k_rep, v_rep, ctx, index, counts, scale_of(D), "bf16", seqs=sample)
    assert status == 0
    assert_parity(out[sample], ref[sample], False, "long chunks")
    ok = np.isfinite(ref_lse[sample])
    np.testing.assert_allclose(lse[sample][ok], ref_lse[sample][ok], rtol=1e-5, atol=1e-5)
    bad = index.copy()
    bad[0, T - 3] = T + 9                                       # last window of the longest list
    out, _, status, _ = p.sparse(ctx, bad, counts, max_selected=T)
    want = index.copy()
    want[0, :T - 1] = np.delete(index[0, :T], T - 3)
    cnt2 = list(counts)
    cnt2[0] = T - 1
    ref_b, _ = O.decode_attn_sparse(p.q_bits, k_rep, v_rep, ctx, want, cnt2, scale_of(D), "bf16", seqs=[0])
    assert status == ssa.DEV_BAD_INDEX
    assert_parity(out[[0]], ref_b[[0]], False, "long chunks, bad entry")
    out_d, _, _ = p.dense(ctx)
    ref_d, _ = O.decode_attn_dense(p.q_bits, k_rep, v_rep, ctx, scale_of(D), "bf16", seqs=sample)
    assert_parity(out_d[sample], ref_d[sample], False, "long chunks, dense")


def test_mixed_batch_of_full_context_and_restricted_requests():
    # requests at a "determine span" step attend to everything, the others to their spans, in one launch
    wl = inputs.make_config(2, B=6, H=4)
    spans, offs = [], [0]
    for i in range(wl.B):
        sp = [(0, int(wl.ctx_lens[i]))] if i % 2 == 0 else wl.spans_of(i).tolist()
        spans += sp
        offs.append(len(spans))
    wl.spans, wl.span_offsets = np.asarray(spans, np.int32), np.asarray(offs, np.int32)
    ds = DecodeStep(wl, out_dtype=torch.float32)
    assert ds.max_selected == int(wl.ctx_lens[::2].max())
    ds.step()
    torch.cuda.synchronize()
    got = ds.out_f64()
    k, v = wl.kv_bits()
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    ref, _ = O.decode_attn_sparse(wl.q_bits(), k, v, wl.ctx_lens, index, counts, scale_of(wl.D), wl.dtype)
    refd, _ = O.decode_attn_dense(wl.q_bits(), k, v, wl.ctx_lens, scale_of(wl.D), wl.dtype)
    assert int(ds.status.item()) == 0
    assert_parity(got, ref, False, "mixed batch")
    assert_parity(got[::2], refd[::2], False, "full-context requests")
    ds.attend_dense()
    torch.cuda.synchronize()
    np.testing.assert_allclose(ds.out_f64()[::2], got[::2], rtol=0, atol=1e-5)


def test_decode_step_in_one_call_with_host_copies():
    # ssa_decode_step: copy in, index, attention, copy out - against the two separate calls
    wl = inputs.make_config(2, B=5, H=4)
    ds = DecodeStep(wl, out_dtype=torch.float32)
    ds.step_two_calls()
    torch.cuda.synchronize()
    want_out, want_lse = ds.out.clone(), ds.lse.clone()
    want_counts = ds.counts.clone()
    ds.make_host_buffers()
    ds.in_arena.zero_()                                        # the device copy of the inputs is wiped:
    ds.out_arena.fill_(7)                                      # everything must come from the host arena
    ds.index.fill_(-7)
    ds.status.zero_()
    before = ssa.launch_count()
    ds.step_from_host()
    torch.cuda.synchronize()
    assert ssa.launch_count() - before >= 1
    assert torch.equal(ds.out, want_out) and torch.equal(ds.lse, want_lse) and torch.equal(ds.counts, want_counts)
    host = ds.h_out.clone()
    assert torch.equal(host, ds.out_arena.cpu())               # results landed in the pinned arena
    assert int(ds.status.item()) == 0
    # argument checks of the composite call
    st = ssa.make_step(ds.span_offsets, ds.spans, ds.ctx_lens, ds.index, ds.counts, ds.q, ds.k, ds.v,
                       ds.max_selected, ds.out, ds.lse, ds.workspace, ds.status, host_in=ds.h_in, dev_in=None)
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_NULL
    st = ssa.make_step(ds.span_offsets, ds.spans, ds.ctx_lens, ds.index, ds.counts, ds.q, ds.k, ds.v,
                       ds.max_selected, ds.out, ds.lse, None, ds.status)
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_WORKSPACE


@pytest.mark.parametrize("cfg,B,H", [(2, 5, 4), (3, 2, 4)])
def test_decode_step_with_copies_done_by_kernels_and_rows_stored_into_host_memory(cfg, B, H):
    # SSA_STEP_COPY_BY_KERNEL with out / lse pointing into the pinned landing buffer (one chunk per request
    # at cfg 2, several plus the second pass at cfg 3): same bits as the device-resident step, and as the oracle
    wl = inputs.make_config(cfg, B=B, H=H)
    ds = DecodeStep(wl, out_dtype=torch.float32)
    ds.step()
    torch.cuda.synchronize()
    want_out, want_lse, want_counts = ds.out.cpu(), ds.lse.cpu(), ds.counts.cpu()
    ds.make_host_buffers()
    for rep in range(2):                                       # twice: the second call overwrites the first
        ds.in_arena.zero_()
        ds.out_arena.fill_(7)
        ds.status.zero_()
        ds.h_out.fill_(9)
        ds.index.fill_(-7)
        before = ssa.launch_count()
        ds.step_from_host(direct=True)
        torch.cuda.synchronize()
        assert ssa.launch_count() - before >= 3                # fetch + index in one launch, attention, copy out
        assert torch.equal(ds.h_out_rows, want_out) and torch.equal(ds.h_lse, want_lse)
        assert torch.equal(ds.h_counts, want_counts) and int(ds.h_status.item()) == 0
        assert torch.equal(ds.in_arena.cpu(), ds.h_in)         # inputs arrived on the device
        assert bool((ds.out.view(torch.uint8) == 7).all())     # the device-side output rows were not used
    ref, _ = O.decode_attn_sparse(wl.q_bits(), *wl.kv_bits(), wl.ctx_lens,
                                  *O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)[:2],
                                  scale_of(wl.D), wl.dtype)
    assert_parity(ds.h_out_rows.to(torch.float64).numpy(), ref, False, "direct to host")
    # refusals come before anything is enqueued
    pageable = torch.empty(ds.h_in.numel(), dtype=torch.uint8)
    mk = lambda **kw: ssa.make_step(ds.span_offsets, ds.spans, ds.ctx_lens, ds.index, ds.counts, ds.q, ds.k, ds.v,
                                    ds.max_selected, ds.out, ds.lse, ds.workspace, ds.status, **kw)
    before = ssa.launch_count()
    st = mk(host_in=pageable, dev_in=ds.in_arena, copy_by_kernel=True)
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_UNSUPPORTED      # not page-locked
    st = mk(host_in=ds.h_in[8:264], dev_in=ds.in_arena, copy_by_kernel=True)
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_ALIGN
    st = mk(host_in=ds.h_in, dev_in=ds.in_arena)
    st.flags = 8
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_UNSUPPORTED      # unknown flag bits
    st.flags = ssa.STEP_ONE_KERNEL | ssa.STEP_TWO_KERNELS
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_UNSUPPORTED      # contradictory
    assert ssa.launch_count() == before


@pytest.mark.parametrize("cfg,kw", [(2, dict(B=5, H=4)), (3, dict(B=2, H=3)), (5, dict(density=0.25, B=2, H=2))])
def test_decode_step_runs_as_one_kernel_or_two_with_the_same_bits(cfg, kw):
    """ssa_decode_step: forced to one kernel, forced to index + attention launches, and left to decide;
    index lists, counts, output and lse agree bit for bit, and with the oracle."""
    wl = inputs.make_config(cfg, **kw)
    ds = DecodeStep(wl, out_dtype=torch.float32)
    got = {}
    for kernels in ("two", "one", "auto"):
        ds.out.fill_(5.0)
        ds.lse.fill_(5.0)
        ds.index.fill_(-7)
        ds.counts.fill_(-7)
        before = ssa.launch_count()
        ds.step(kernels=kernels)
        torch.cuda.synchronize()
        got[kernels] = (ds.out.clone(), ds.lse.clone(), ds.index.clone(), ds.counts.clone(),
                        ssa.launch_count() - before)
        assert int(ds.status.item()) == 0
    chunks = got["two"][4] - 1                                  # attention launches of the two-kernel form
    assert got["one"][4] == chunks                              # the same without the index launch
    assert got["auto"][4] in (chunks, chunks + 1)
    for kernels in ("one", "auto"):
        for a, b in zip(got[kernels][:4], got["two"][:4]):
            assert torch.equal(a, b)
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    assert got["one"][3].cpu().numpy().tolist() == counts.tolist()
    for b in range(wl.B):
        assert np.array_equal(got["one"][2][b, :counts[b]].cpu().numpy(), index[b, :counts[b]])
    ref, _ = O.decode_attn_sparse(wl.q_bits(), *wl.kv_bits(), wl.ctx_lens, index, counts, scale_of(wl.D), wl.dtype)
    assert_parity(got["one"][0].double().cpu().numpy(), ref, False, "one-kernel step")
    # forcing one kernel without a usable span bound is refused
    st = ssa.make_step(ds.span_offsets, ds.spans, ds.ctx_lens, ds.index, ds.counts, ds.q, ds.k, ds.v,
                       ds.max_selected, ds.out, ds.lse, ds.workspace, ds.status, kernels="one", max_spans=0)
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_CAPACITY
    st.max_spans = 129
    assert ssa.decode_step(ds.desc, st, check=False) == ssa.ERR_CAPACITY


def test_side_stream_graph_replay_and_determinism():
    wl = inputs.make_config(3, B=2, H=4)
    ds = DecodeStep(wl, out_dtype=torch.float32)
    ds.step()
    torch.cuda.synchronize()
    first = ds.out.clone()
    # twice the same call: bit-identical (no atomics in the accumulation)
    ds.out.zero_()
    ds.step()
    torch.cuda.synchronize()
    assert torch.equal(ds.out, first)
    # on a side stream, handed over explicitly and as torch's current stream
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    ds.out.zero_()
    torch.cuda.synchronize()
    ds.step(stream=side)
    side.synchronize()
    assert torch.equal(ds.out, first)
    ds.out.zero_()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        ds.step()
    side.synchronize()
    assert torch.equal(ds.out, first)
    # captured into a CUDA graph and replayed
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ds.step()
    ds.out.zero_()
    ds.counts.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(ds.out, first) and int(ds.status.item()) == 0
    # the no-workspace and the dense calls through the same graph mechanism
    g2 = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g2, stream=side):
        ds.attend_dense()
    g2.replay()
    torch.cuda.synchronize()
    k, v = wl.kv_bits()
    refd, _ = O.decode_attn_dense(wl.q_bits(), k, v, wl.ctx_lens, scale_of(wl.D), wl.dtype)
    assert_parity(ds.out_f64(), refd, False, "dense from a graph")


def test_host_driven_step_replayed_from_a_graph_with_new_inputs():
    # ssa_decode_step with kernel copies captured once; between replays the host rewrites the pinned input
    # arena (other query rows, other spans) and the cache changes: every replay must pick the new bytes up
    kw = dict(out_dtype=torch.float32, span_capacity=40, index_stride=256, max_selected=256)
    steps = {name: DecodeStep(inputs.make_config(2, B=6, H=4, first_id=fid), **kw) for name, fid in (("a", 0), ("b", 50))}
    want, arena, cache = {}, {}, {}
    for name, d in steps.items():
        d.step()
        torch.cuda.synchronize()
        want[name] = (d.out.cpu(), d.lse.cpu(), d.counts.cpu())
        arena[name] = d.in_arena.cpu()
        cache[name] = (d.k.clone(), d.v.clone())
    assert not torch.equal(want["a"][0], want["b"][0]) and arena["a"].shape == arena["b"].shape
    ds = steps["a"]
    ds.make_host_buffers()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    ds.step_from_host(direct=True, stream=side)                # first call outside the capture
    side.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        ds.step_from_host(direct=True)
    for name in ("a", "b", "a"):
        ds.h_in.copy_(arena[name])
        ds.k.copy_(cache[name][0])
        ds.v.copy_(cache[name][1])
        ds.h_out.fill_(9)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        out, lse, counts = want[name]
        assert torch.equal(ds.h_counts, counts), name
        assert torch.equal(ds.h_out_rows, out) and torch.equal(ds.h_lse, lse), name
        assert int(ds.h_status.item()) == 0


def test_decode_step_with_more_query_heads_than_cache_heads():
    # the runner's buffers with grouped query heads: span lists -> index lists -> attention, 8 query heads on 2
    wl = inputs.make_config(3, B=2, H=2)
    ds = DecodeStep(wl, out_dtype=torch.float32, query_heads=8)
    ds.step()
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    k, v = wl.kv_bits()
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    ref, ref_lse = O.decode_attn_sparse(wl.q_bits(8), np.repeat(k, 4, axis=1), np.repeat(v, 4, axis=1), wl.ctx_lens,
                                        index, counts, scale_of(wl.D), wl.dtype)
    assert_parity(ds.out_f64(), ref, False, "runner, grouped heads")
    np.testing.assert_allclose(ds.lse.double().cpu().numpy(), ref_lse, rtol=1e-5, atol=1e-5)
    ds.attend_dense()
    torch.cuda.synchronize()
    refd, _ = O.decode_attn_dense(wl.q_bits(8), np.repeat(k, 4, axis=1), np.repeat(v, 4, axis=1), wl.ctx_lens,
                                  scale_of(wl.D), wl.dtype)
    assert_parity(ds.out_f64(), refd, False, "runner, grouped heads, dense")


def test_largest_batch_the_grid_allows():
    # 65535 requests (the launch grid's limit in that dimension), one head, tiny contexts: index expansion,
    # restricted and full-context attention on sampled requests; one request more is refused on the host
    B, H, T, D = 65535, 1, 8, 64
    rng = np.random.default_rng(12)
    q_bits = random_bits(rng, (B, H, D), "f16")
    k_bits = random_bits(rng, (B, H, T, D), "f16")
    v_bits = random_bits(rng, (B, H, T, D), "f16")
    from paper_2404_09336_b200.runner import bits_to_tensor
    q, k, v = (bits_to_tensor(x, "f16").to("cuda:0") for x in (q_bits, k_bits, v_bits))
    ctx = rng.integers(1, T + 1, size=B).astype(np.int32)
    starts = rng.integers(0, T, size=B)
    spans = np.stack([starts, np.minimum(starts + rng.integers(1, 5, size=B), T + 2)], axis=1).astype(np.int32)
    offs = np.arange(B + 1, dtype=np.int32)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")
    d_ctx, d_sp, d_off = dev(ctx), dev(spans), dev(offs)
    index = torch.full((B, 8), -7, dtype=torch.int32, device="cuda:0")
    counts = torch.full((B,), -7, dtype=torch.int32, device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    ssa.spans_to_index(d_off, d_sp, d_ctx, index, counts, status)
    out = torch.zeros((B, H, D), dtype=torch.float32, device="cuda:0")
    lse = torch.zeros((B, H), dtype=torch.float32, device="cuda:0")
    desc = ssa.make_desc(q, k, v, out)
    ws = torch.empty(max(ssa.decode_workspace_bytes(desc, 8), 16), dtype=torch.uint8, device="cuda:0")
    ssa.decode_attn_sparse(desc, q, k, v, d_ctx, index, counts, 8, out, lse, ws, status)
    torch.cuda.synchronize()
    sample = sorted(set([0, 1, B // 2, B - 2, B - 1] + rng.integers(0, B, size=40).tolist()))
    want_index, want_counts, want_status = O.spans_to_index_batch(offs, spans, ctx, 8)
    assert torch.equal(counts.cpu(), torch.from_numpy(want_counts))
    got_index = index.cpu().numpy()
    for b in sample:
        assert got_index[b, :want_counts[b]].tolist() == want_index[b, :want_counts[b]].tolist()
    assert int(status.item()) == (ssa.DEV_CLIPPED if want_status & O.ST_CLIPPED else 0)
    ref, _ = O.decode_attn_sparse(q_bits, k_bits, v_bits, ctx, want_index, want_counts, scale_of(D), "f16", seqs=sample)
    assert_parity(out.double().cpu().numpy()[sample], ref[sample], False, "largest batch, sparse")
    ssa.decode_attn_dense(desc, q, k, v, d_ctx, out, lse, ws, status)
    torch.cuda.synchronize()
    ref_d, _ = O.decode_attn_dense(q_bits, k_bits, v_bits, ctx, scale_of(D), "f16", seqs=sample)
    assert_parity(out.double().cpu().numpy()[sample], ref_d[sample], False, "largest batch, dense")
    desc.B = 65536
    assert ssa.decode_attn_dense(desc, q, k, v, d_ctx, out, lse, ws, status, check=False) == ssa.ERR_SHAPE


def test_one_long_context_with_hundreds_of_spans():
    # a single request, 300 000 cached tokens, ~250 spans covering ~45 000 of them: the shared-memory sort of the
    # index kernel, 32 output slices, hundreds of chunks and the second pass
    B, H, T, D = 1, 2, 300_000, 64
    p = Problem(B, H, T, D, "f16", seed=77)
    rng = np.random.default_rng(5)
    starts = np.sort(rng.integers(0, T - 400, size=250))
    spans = [(int(s), int(s + rng.integers(1, 400))) for s in starts]
    rng.shuffle(spans)
    stride = 65536
    index, counts, status, _ = run_index([spans], [T], stride)
    want = O.spans_to_index(spans, T)
    assert status == 0 and counts[0] == len(want) and 30_000 < len(want) <= stride
    assert np.array_equal(index[0, :len(want)], want)
    out, lse, st, _ = p.sparse([T], index, counts.tolist(), max_selected=stride)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, [T], index, counts, scale_of(D), "f16")
    assert st == 0
    assert_parity(out, ref, False, "long context")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    out_d, lse_d, _ = p.dense([T])
    ref_d, ref_lse_d = O.decode_attn_dense(p.q_bits, p.k_bits, p.v_bits, [T], scale_of(D), "f16")
    assert_parity(out_d, ref_d, False, "long context, dense")
    np.testing.assert_allclose(lse_d, ref_lse_d, rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("order", ["q first", "q last", "q in the middle"])
def test_host_driven_step_wherever_the_query_rows_sit_in_the_input_arena(order):
    """SSA_STEP_COPY_BY_KERNEL with hand-laid arenas: with the query rows at the head or the tail of the arena the
    attention blocks fetch them from the pinned copy themselves (one chunk per request here); in the middle the
    whole arena is fetched in front of the kernels.  Either way: the oracle's output, and the device arena ends up
    a copy of the host arena."""
    wl = inputs.make_config(2, B=5, H=4)
    B, H, D = wl.B, wl.H, wl.D
    n_spans = len(wl.spans)
    sizes = {"q": B * H * D * 2, "ctx": B * 4, "offs": (B + 1) * 4, "spans": n_spans * 8}
    pad = lambda n: (n + 255) // 256 * 256
    names = {"q first": ["q", "ctx", "offs", "spans"], "q last": ["ctx", "offs", "spans", "q"],
             "q in the middle": ["ctx", "q", "offs", "spans"]}[order]
    at, total = {}, 0
    for i, name in enumerate(names):
        at[name] = total
        total += sizes[name] if i == len(names) - 1 else pad(sizes[name])   # nothing behind the last tensor
    total = (total + 15) // 16 * 16
    h_in = torch.zeros(total, dtype=torch.uint8).pin_memory()
    view = lambda buf, name, dt, shape: buf[at[name]:at[name] + sizes[name]].view(dt).view(shape)
    view(h_in, "q", torch.bfloat16, (B, H, D)).copy_(torch.from_numpy(wl.q_bits().view(np.int16)).view(torch.bfloat16))
    view(h_in, "ctx", torch.int32, (B,)).copy_(torch.from_numpy(wl.ctx_lens.copy()))
    view(h_in, "offs", torch.int32, (B + 1,)).copy_(torch.from_numpy(wl.span_offsets.copy()))
    view(h_in, "spans", torch.int32, (n_spans, 2)).copy_(torch.from_numpy(np.ascontiguousarray(wl.spans)))
    d_in = torch.full((total,), 0xAB, dtype=torch.uint8, device=DEV)
    q = view(d_in, "q", torch.bfloat16, (B, H, D))
    ctx, offs = view(d_in, "ctx", torch.int32, (B,)), view(d_in, "offs", torch.int32, (B + 1,))
    spans = view(d_in, "spans", torch.int32, (n_spans, 2))
    ds = DecodeStep(wl, out_dtype=torch.float32)              # the cache, and buffers to borrow
    h_out = torch.zeros(ds.counts.numel() * 4 + 256, dtype=torch.uint8).pin_memory()
    ds.index.fill_(-7)
    ds.status.zero_()
    desc = ssa.make_desc(q, ds.k, ds.v, ds.out)
    st = ssa.make_step(offs, spans, ctx, ds.index, ds.counts, q, ds.k, ds.v, ds.max_selected, ds.out, ds.lse,
                       ds.workspace, ds.status, host_in=h_in, dev_in=d_in, copy_by_kernel=True, max_spans=ds.max_spans)
    for _ in range(2):
        ds.out.fill_(3.0)
        ssa.decode_step(desc, st)
        torch.cuda.synchronize()
        assert torch.equal(d_in.cpu(), h_in)                  # every input byte arrived on the device
        assert int(ds.status.item()) == 0
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    assert ds.counts.cpu().numpy().tolist() == counts.tolist()
    ref, _ = O.decode_attn_sparse(wl.q_bits(), *wl.kv_bits(), wl.ctx_lens, index, counts, scale_of(D), wl.dtype)
    assert_parity(ds.out_f64(), ref, False, order)
