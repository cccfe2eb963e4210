"""The paper's blocked span encoding on the GPU: ssa_spans_to_blockmask (bit-exact
against the oracle) and ssa_decode_attn_blockmask (parity with the oracle and
with the index-list path)."""
import random

import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs, ssa
from paper_2404_09336_b200.runner import bits_to_tensor

from gpu_util import DEV, Problem
from parity import assert_parity

pytestmark = pytest.mark.gpu


def run_blockmask(span_lists, ctx_lens, bs, stride, fill=-7):
    B = len(span_lists)
    offs = np.zeros(B + 1, np.int32)
    offs[1:] = np.cumsum([len(s) for s in span_lists])
    flat = np.asarray([p for s in span_lists for p in s], np.int32).reshape(-1, 2)
    if len(flat) == 0:
        flat = np.zeros((1, 2), np.int32)
    d_off, d_sp = torch.from_numpy(offs).to(DEV), torch.from_numpy(flat).to(DEV)
    d_ctx = torch.tensor(ctx_lens, dtype=torch.int32, device=DEV)
    bidx = torch.full((B, stride), fill, dtype=torch.int32, device=DEV)
    bmask = torch.full((B, stride, bs // 32), fill, dtype=torch.int32, device=DEV)
    bcnt = torch.full((B,), fill, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ssa.spans_to_blockmask(d_off, d_sp, d_ctx, bs, bidx, bmask, bcnt, status)
    torch.cuda.synchronize()
    return (bidx.cpu().numpy(), bmask.cpu().numpy().view(np.uint32), bcnt.cpu().numpy(), int(status.item()),
            (offs, flat), (bidx, bmask, bcnt, d_ctx))


def compare_encoding(span_lists, ctx_lens, bs, stride):
    bidx, bmask, bcnt, status, (offs, flat), dev = run_blockmask(span_lists, ctx_lens, bs, stride)
    r_idx, r_mask, r_cnt, r_status = O.spans_to_blockmask_batch(offs, flat[: offs[-1]], ctx_lens, bs, stride)
    assert bcnt.tolist() == r_cnt.tolist()
    for b in range(len(span_lists)):
        c = int(r_cnt[b])
        assert bidx[b, :c].tolist() == r_idx[b, :c].tolist(), f"request {b}"
        assert np.array_equal(bmask[b, :c], r_mask[b, :c]), f"request {b}"
        assert np.all(bidx[b, c:] == -7)                       # padding left untouched
    assert status == r_status
    return dev


@pytest.mark.parametrize("bs", [32, 64, 128, 256])
def test_encoding_of_the_workloads(bs):
    for cfg, dens in [(1, None), (2, None), (3, None), (4, None), (5, 0.25)]:
        wl = inputs.make_config(cfg, density=dens, B=None if cfg < 5 else 4)
        lists = [wl.spans_of(i).tolist() for i in range(wl.B)]
        stride = (wl.max_ctx + bs - 1) // bs
        compare_encoding(lists, wl.ctx_lens.tolist(), bs, stride)


def test_encoding_hand_cases_and_flags():
    lists = [[], [(0, 100)], [(1, 3), (40, 44), (99, 120)], [(5, 5)], [(63, 65)], [(-4, 2)], [(9, 3)]]
    compare_encoding(lists, [100] * len(lists), 32, 8)
    compare_encoding(lists, [100] * len(lists), 64, 8)
    compare_encoding([[(0, 1000)]], [1000], 32, 8)             # 32 blocks, 8 kept: overflow flag
    compare_encoding([[(5, 70000)]], [66000], 256, 300)        # several sweep windows
    compare_encoding([[(0, 10)]], [0], 32, 4)


@pytest.mark.parametrize("seed", range(6))
def test_encoding_fuzz(seed):
    rnd = random.Random(seed)
    lists, ctx = [], []
    for _ in range(rnd.randint(1, 20)):
        n = rnd.randint(0, 20000)
        sp = []
        for _ in range(rnd.randint(0, 60)):
            s = rnd.randint(-20, n + 20)
            sp.append((s, s + rnd.randint(-10, 700)))
        lists.append(sp)
        ctx.append(n)
    bs = rnd.choice([32, 64, 128, 256])
    compare_encoding(lists, ctx, bs, rnd.choice([4, 64, 640]))


def attention_from_lists(p, ctx, bidx, bmask, bcnt, bs, max_blocks, out_dtype=torch.float32):
    B, H, D = p.B, p.H, p.D
    d_idx = torch.from_numpy(np.ascontiguousarray(bidx, dtype=np.int32)).to(DEV)
    d_mask = torch.from_numpy(np.ascontiguousarray(bmask).view(np.int32)).to(DEV)
    d_cnt = torch.tensor(list(bcnt), dtype=torch.int32, device=DEV)
    d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
    out = torch.full((B, H, D), 777.0, dtype=out_dtype, device=DEV)
    lse = torch.full((B, H), 777.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_blockmask_workspace_bytes(desc, bs, max_blocks), dtype=torch.uint8, device=DEV)
    ssa.decode_attn_blockmask(desc, p.q, p.k, p.v, d_ctx, d_idx, d_mask, d_cnt, bs, max_blocks, out, lse, ws, status)
    torch.cuda.synchronize()
    return out.double().cpu().numpy(), lse.double().cpu().numpy(), int(status.item())


@pytest.mark.parametrize("bs", [32, 64, 128, 256])
@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f16", 64)])
def test_attention_from_blocked_lists(bs, dtype, D):
    B, H, T = 4, 3, 2500
    p = Problem(B, H, T, D, dtype, seed=bs + D)
    ctx = [2500, 1, 1300, 700]
    rnd = random.Random(bs)
    lists = [[(0, 64), (100, 130), (900, 1500), (2400, 2500)], [(0, 1)], [],
             [(rnd.randint(0, 600), rnd.randint(0, 800)) for _ in range(12)]]
    lists[3] = [(min(a, b), max(a, b)) for a, b in lists[3]]
    offs = np.zeros(B + 1, np.int64)
    offs[1:] = np.cumsum([len(s) for s in lists])
    flat = [q for s in lists for q in s]
    stride = (T + bs - 1) // bs
    r_idx, r_mask, r_cnt, _ = O.spans_to_blockmask_batch(offs, flat, ctx, bs, stride)
    ref, ref_lse = O.decode_attn_blockmask(p.q_bits, p.k_bits, p.v_bits, ctx, r_idx, r_mask, r_cnt, bs,
                                           1 / np.sqrt(D), dtype)
    for max_blocks in (int(r_cnt.max()), stride):
        out, lse, status = attention_from_lists(p, ctx, r_idx, r_mask, r_cnt, bs, max_blocks)
        assert status == 0
        assert_parity(out, ref, False, f"bs={bs}")
        ok = np.isfinite(ref_lse)
        np.testing.assert_allclose(lse[ok], ref_lse[ok], rtol=1e-5, atol=1e-5)
        assert not out[2].any() and np.all(np.isneginf(lse[2]))           # request 2 selected nothing
    # same attended set through the index list: the two paths agree
    index, counts, _ = O.spans_to_index_batch(offs, flat, ctx, T)
    out_i, _, _, _ = p.sparse(ctx, index, counts.tolist(), max_selected=T)
    np.testing.assert_allclose(out, out_i, rtol=0, atol=2e-6)


def test_blocked_lists_with_grouped_query_heads():
    # 8 query heads on 2 cache heads through the blocked lists (served by the one-head-per-block kernel)
    from gpu_util import random_bits
    B, H, Hkv, T, D, bs = 3, 8, 2, 1000, 128, 64
    p = Problem(B, Hkv, T, D, "bf16", seed=9)
    p.q_bits = random_bits(np.random.default_rng(1), (B, H, D), "bf16")
    p.H = H
    p.upload()
    ctx = [1000, 400, 77]
    lists = [[(0, 64), (300, 420), (900, 1000)], [(10, 390)], [(0, 77)]]
    offs = np.zeros(B + 1, np.int64)
    offs[1:] = np.cumsum([len(s) for s in lists])
    flat = [q for s in lists for q in s]
    stride = (T + bs - 1) // bs
    r_idx, r_mask, r_cnt, _ = O.spans_to_blockmask_batch(offs, flat, ctx, bs, stride)
    k_rep, v_rep = np.repeat(p.k_bits, H // Hkv, axis=1), np.repeat(p.v_bits, H // Hkv, axis=1)
    ref, ref_lse = O.decode_attn_blockmask(p.q_bits, k_rep, v_rep, ctx, r_idx, r_mask, r_cnt, bs, 1 / np.sqrt(D), "bf16")
    out, lse, status = attention_from_lists(p, ctx, r_idx, r_mask, r_cnt, bs, stride)
    assert status == 0
    assert_parity(out, ref, False, "blocked lists, grouped heads")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)


def test_end_to_end_on_device_and_bad_bits():
    # spans -> blocked lists -> attention without leaving the device
    wl = inputs.make_config(2, B=5, H=4)
    lists = [wl.spans_of(i).tolist() for i in range(wl.B)]
    bs, stride = 64, 16
    _, _, _, status, _, (bidx, bmask, bcnt, d_ctx) = run_blockmask(lists, wl.ctx_lens.tolist(), bs, stride)
    assert status == 0
    k, v = wl.kv_bits()
    p = Problem.__new__(Problem)
    p.B, p.H, p.T, p.D, p.dtype, p.layout = wl.B, wl.H, wl.max_ctx, wl.D, wl.dtype, "bhtd"
    p.q_bits, p.k_bits, p.v_bits = wl.q_bits(), k, v
    p.upload()
    out, lse, st = attention_from_lists(p, wl.ctx_lens.tolist(), bidx.cpu().numpy(),
                                        bmask.cpu().numpy().view(np.uint32), bcnt.cpu().numpy(), bs, stride)
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, 256)
    ref, _ = O.decode_attn_sparse(p.q_bits, k, v, wl.ctx_lens, index, counts, 1 / np.sqrt(wl.D), wl.dtype)
    assert st == 0
    assert_parity(out, ref, False, "device pipeline")
    # bits beyond the context, a negative block index, a count above the bound: skipped / clamped and flagged
    hb = bidx.cpu().numpy().copy()
    hm = bmask.cpu().numpy().view(np.uint32).copy()
    hc = bcnt.cpu().numpy().copy()
    n0 = int(wl.ctx_lens[0])
    hb[0, hc[0]] = (n0 + bs - 1) // bs + 3                     # a block wholly outside the context
    hm[0, hc[0]] = 0xFFFFFFFF
    hb[1, hc[1]] = -2
    hm[1, hc[1]] = 1
    hc[0] += 1
    hc[1] += 1
    out2, _, st2 = attention_from_lists(p, wl.ctx_lens.tolist(), hb, hm, hc, bs, stride)
    assert st2 == ssa.DEV_BAD_INDEX
    np.testing.assert_array_equal(out2, out)
    hc[2] = stride + 5
    _, _, st3 = attention_from_lists(p, wl.ctx_lens.tolist(), hb, hm, hc, bs, stride)
    assert st3 & ssa.DEV_BAD_COUNT


def test_full_size_workload_through_the_blocked_lists():
    # cfg 3 at full size in the launch configuration of the benchmark; sampled outputs against the oracle
    from paper_2404_09336_b200.runner import DecodeStep
    wl = inputs.make_config(3)
    ds = DecodeStep(wl)
    ds.enable_blockmask(256)
    ds.step_blockmask()
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    got = ds.out_f64()
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, 4096)
    q = wl.q_bits()
    for b in (3, 12):
        k, v = wl.kv_bits_seq(b)
        ref, _ = O.decode_attn_sparse(q[b:b + 1], k[None], v[None], wl.ctx_lens[b:b + 1], index[b:b + 1],
                                      counts[b:b + 1], 1 / np.sqrt(wl.D), wl.dtype, heads=[0, 17, 31])
        for h in (0, 17, 31):
            assert_parity(got[b, h], ref[0, h], True, f"request {b} head {h}")
    ds.step()
    torch.cuda.synchronize()
    np.testing.assert_allclose(ds.out_f64(), got, rtol=0, atol=4e-3)       # bf16 outputs of the two paths
