"""Attention over a paged cache (ssa_decode_attn_sparse_paged / _dense_paged)
against the oracle: the pool is random, the oracle gathers the pages into the
contiguous cache they stand for and applies its plain definitions."""
import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import ssa
from paper_2404_09336_b200.runner import bits_to_tensor

from gpu_util import DEV, TORCH_DT, random_bits
from parity import assert_parity

pytestmark = pytest.mark.gpu


class PagedProblem:
    def __init__(self, B, H, H_kv, D, T, page_size, spare_pages, dtype="bf16", seed=0):
        rng = np.random.default_rng(seed)
        self.B, self.H, self.H_kv, self.D, self.T, self.ps, self.dtype = B, H, H_kv, D, T, page_size, dtype
        per_req = (T + page_size - 1) // page_size
        self.n_pages = B * per_req + spare_pages
        self.table = rng.permutation(self.n_pages)[: B * per_req].astype(np.int32).reshape(B, per_req)
        self.q_bits = random_bits(rng, (B, H, D), dtype)
        self.k_pool = random_bits(rng, (self.n_pages, page_size, H_kv, D), dtype)
        self.v_pool = random_bits(rng, (self.n_pages, page_size, H_kv, D), dtype)
        self.q = bits_to_tensor(self.q_bits, dtype).to(DEV)
        self.kp = bits_to_tensor(self.k_pool, dtype).to(DEV)
        self.vp = bits_to_tensor(self.v_pool, dtype).to(DEV)

    def logical(self, table=None):
        """The contiguous caches the pools stand for, query heads' view: [B, H, T, D]."""
        t = self.table if table is None else table
        g = self.H // self.H_kv
        k = O.gather_pages(self.k_pool, t, self.ps, self.T)
        v = O.gather_pages(self.v_pool, t, self.ps, self.T)
        return np.repeat(k, g, axis=1), np.repeat(v, g, axis=1)

    def run(self, ctx, index=None, counts=None, table=None, out_dtype=torch.float32, max_selected=None):
        B, H, D = self.B, self.H, self.D
        d_tab = torch.from_numpy(np.ascontiguousarray(self.table if table is None else table)).to(DEV)
        d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
        out = torch.full((B, H, D), 777.0, dtype=out_dtype or TORCH_DT[self.dtype], device=DEV)
        lse = torch.full((B, H), 777.0, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        desc = ssa.make_desc_paged(self.q, self.kp, self.vp, out, max_ctx=self.T)
        pg = ssa.make_paging(d_tab, self.ps, self.n_pages)
        if index is None:
            ws = torch.empty(ssa.decode_workspace_bytes(desc, self.T), dtype=torch.uint8, device=DEV)
            ssa.decode_attn_dense_paged(desc, self.q, self.kp, self.vp, pg, d_ctx, out, lse, ws, status)
        else:
            d_idx = torch.from_numpy(np.ascontiguousarray(index, dtype=np.int32)).to(DEV)
            d_cnt = torch.tensor(counts, dtype=torch.int32, device=DEV)
            ms = int(max_selected or index.shape[1])
            ws = torch.empty(ssa.decode_workspace_bytes(desc, ms), dtype=torch.uint8, device=DEV)
            ssa.decode_attn_sparse_paged(desc, self.q, self.kp, self.vp, pg, d_ctx, d_idx, d_cnt, ms, out, lse, ws,
                                         status)
        torch.cuda.synchronize()
        return out.to(torch.float64).cpu().numpy(), lse.to(torch.float64).cpu().numpy(), int(status.item())


def random_lists(rng, ctx, stride):
    B = len(ctx)
    index = np.full((B, stride), -1, np.int32)
    counts = []
    for b, n in enumerate(ctx):
        c = int(rng.integers(1, min(n, stride) + 1))
        index[b, :c] = np.sort(rng.choice(n, c, replace=False))
        counts.append(c)
    return index, counts


@pytest.mark.parametrize("page_size", [1, 16, 128])
@pytest.mark.parametrize("B,H,H_kv,D,dtype", [(3, 4, 4, 128, "bf16"), (40, 4, 2, 64, "f16"), (5, 8, 2, 128, "bf16"),
                                              (3, 12, 1, 128, "f16")])
def test_sparse_and_dense_over_shuffled_pages(page_size, B, H, H_kv, D, dtype):
    T = 700
    p = PagedProblem(B, H, H_kv, D, T, page_size, spare_pages=5, dtype=dtype, seed=page_size + B)
    rng = np.random.default_rng(B)
    ctx = [T] + [int(rng.integers(1, T + 1)) for _ in range(B - 1)]
    k, v = p.logical()
    scale = 1 / np.sqrt(D)
    index, counts = random_lists(rng, ctx, 704)
    out, lse, status = p.run(ctx, index, counts)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, k, v, ctx, index, counts, scale, dtype)
    assert status == 0
    assert_parity(out, ref, False, "paged sparse")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    out, lse, status = p.run(ctx)
    ref, ref_lse = O.decode_attn_dense(p.q_bits, k, v, ctx, scale, dtype)
    assert status == 0
    assert_parity(out, ref, False, "paged dense")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    out, _, _ = p.run(ctx, index, counts, out_dtype=None)                  # output in the storage type
    assert_parity(out, O.decode_attn_sparse(p.q_bits, k, v, ctx, index, counts, scale, dtype)[0], True, "paged bf16/f16 out")


def test_paged_equals_contiguous_bit_for_bit():
    # the same rows through a page table and through a contiguous cache: identical arithmetic, identical bits
    B, H, D, T, ps = 4, 8, 128, 1024, 64
    p = PagedProblem(B, H, H, D, T, ps, spare_pages=3, seed=11)
    rng = np.random.default_rng(2)
    ctx = [T, 777, 1000, 64]
    index, counts = random_lists(rng, ctx, T)
    out_p, lse_p, _ = p.run(ctx, index, counts)
    k, v = p.logical()
    kt, vt = bits_to_tensor(k, "bf16").to(DEV), bits_to_tensor(v, "bf16").to(DEV)
    out = torch.zeros((B, H, D), dtype=torch.float32, device=DEV)
    lse = torch.zeros((B, H), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc(p.q, kt, vt, out)
    ws = torch.empty(ssa.decode_workspace_bytes(desc, T), dtype=torch.uint8, device=DEV)
    ssa.decode_attn_sparse(desc, p.q, kt, vt, torch.tensor(ctx, dtype=torch.int32, device=DEV),
                           torch.from_numpy(index).to(DEV), torch.tensor(counts, dtype=torch.int32, device=DEV), T,
                           out, lse, ws)
    torch.cuda.synchronize()
    assert np.array_equal(out_p, out.to(torch.float64).cpu().numpy())
    assert np.array_equal(lse_p, lse.to(torch.float64).cpu().numpy())


def test_page_ids_outside_the_pool_are_skipped_and_flagged():
    B, H, D, T, ps = 2, 2, 128, 256, 32
    p = PagedProblem(B, H, H, D, T, ps, spare_pages=0, seed=4)
    bad = p.table.copy()
    bad[0, 3] = p.n_pages                                     # positions 96..127 of request 0
    bad[1, 0] = -1                                            # positions 0..31 of request 1
    ctx = [T, T]
    index = np.tile(np.arange(T, dtype=np.int32), (B, 1))
    out, lse, status = p.run(ctx, index, [T, T], table=bad)
    assert status == ssa.DEV_BAD_INDEX
    k, v = p.logical()
    keep0 = np.r_[0:96, 128:T].astype(np.int32)
    keep1 = np.arange(32, T, dtype=np.int32)
    want = np.full((B, T), -1, np.int32)
    want[0, :len(keep0)], want[1, :len(keep1)] = keep0, keep1
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, k, v, ctx, want, [len(keep0), len(keep1)], 1 / np.sqrt(D), "bf16")
    assert_parity(out, ref, False, "bad pages skipped")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    out, lse, status = p.run(ctx, table=bad)                  # the full-context call skips them too
    assert status == ssa.DEV_BAD_INDEX
    assert_parity(out, ref, False, "bad pages skipped, dense")


def test_argument_checks():
    p = PagedProblem(2, 2, 2, 128, 128, 16, spare_pages=0, seed=1)
    out = torch.zeros((2, 2, 128), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc_paged(p.q, p.kp, p.vp, out, max_ctx=128)
    tab = torch.from_numpy(p.table).to(DEV)
    ctx = torch.tensor([128, 128], dtype=torch.int32, device=DEV)
    ws = torch.empty(ssa.decode_workspace_bytes(desc, 128), dtype=torch.uint8, device=DEV)
    call = lambda pg: ssa.decode_attn_dense_paged(desc, p.q, p.kp, p.vp, pg, ctx, out, None, ws, check=False)
    before = ssa.launch_count()
    assert call(None) == ssa.ERR_NULL
    assert call(ssa.make_paging(tab, 24, p.n_pages)) == ssa.ERR_SHAPE          # not a power of two
    assert call(ssa.make_paging(tab, 16, 0)) == ssa.ERR_SHAPE
    assert call(ssa.make_paging(tab, 8, p.n_pages)) == ssa.ERR_SHAPE           # table too short for max_ctx
    assert ssa.launch_count() == before
    assert call(ssa.make_paging(tab, 16, p.n_pages)) == ssa.OK
    torch.cuda.synchronize()
