"""ssa_decode_attn_spans (span lists -> attention output in one kernel, no index
list) against the fp64 oracle: the oracle's span -> index definition followed by
its set-form attention.  The optional index / counts outputs are compared bit
for bit with the oracle's lists, the status word with the oracle's status."""
import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs, ssa
from paper_2404_09336_b200.runner import DecodeStep

from gpu_util import DEV, Problem
from parity import assert_parity
from test_gpu_attn import oracle_for

pytestmark = pytest.mark.gpu

GPU_BITS = {O.ST_BAD_SPAN: ssa.DEV_BAD_SPAN, O.ST_CLIPPED: ssa.DEV_CLIPPED, O.ST_OVERFLOW: ssa.DEV_OVERFLOW}


def run_workload(wl, layout="bhtd", out_dtype=None, seqs=None, heads=None, want_lists=True, query_heads=None):
    ds = DecodeStep(wl, layout=layout, out_dtype=out_dtype)
    ref, ref_lse, _, ref_index, ref_counts = oracle_for(wl, ds, seqs, heads)
    ds.attend_spans(want_lists=want_lists)
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    if want_lists:
        counts = ds.counts.cpu().numpy()
        assert counts.tolist() == ref_counts.tolist()
        idx = ds.index.cpu().numpy()
        for b in range(wl.B):
            assert np.array_equal(idx[b, :counts[b]], ref_index[b, :counts[b]])
            assert np.all(idx[b, counts[b]:] == -7)            # nothing written past the list
    else:
        assert np.all(ds.index.cpu().numpy() == -7) and np.all(ds.counts.cpu().numpy() == -7)
    sel = ~np.isnan(ref)
    assert_parity(ds.out_f64()[sel], ref[sel], out_dtype is None, f"{wl.name} spans {layout}")
    sel_l = ~np.isnan(ref_lse)
    np.testing.assert_allclose(ds.lse.double().cpu().numpy()[sel_l], ref_lse[sel_l], rtol=1e-5, atol=1e-5)
    return ds


# ---- the five workloads, reduced so that the oracle covers every output ----------------------------------
@pytest.mark.parametrize("layout", ["bhtd", "bthd"])
@pytest.mark.parametrize("out_dtype", [None, torch.float32])
def test_cfg1_tiny_full(layout, out_dtype):
    run_workload(inputs.make_config(1), layout, out_dtype)


@pytest.mark.parametrize("layout", ["bhtd", "bthd"])
@pytest.mark.parametrize("want_lists", [True, False])
def test_cfg2_reduced(layout, want_lists):
    run_workload(inputs.make_config(2, B=6, H=4), layout, torch.float32, want_lists=want_lists)
    run_workload(inputs.make_config(2, B=3, H=2), layout, None, want_lists=want_lists)


def test_cfg3_cfg4_reduced():
    run_workload(inputs.make_config(3, B=3, H=3), "bhtd", torch.float32)
    run_workload(inputs.make_config(4, B=2, H=2), "bhtd", torch.float32)
    run_workload(inputs.make_config(4, B=1, H=2), "bthd", None, want_lists=False)


@pytest.mark.parametrize("f", [0.01, 0.10, 0.50, 1.00])
def test_cfg5_reduced(f):
    run_workload(inputs.make_config(5, density=f, B=2, H=2), "bhtd", torch.float32)


# ---- full sizes, in the launch configuration the benchmark times; sampled outputs ----------------------------
@pytest.mark.parametrize("cfg,density", [(2, None), (3, None), (4, None), (5, 0.05), (5, 0.10), (5, 0.50), (5, 1.00)])
def test_full_size_sampled(cfg, density):
    wl = inputs.make_config(cfg, density=density)
    rng = np.random.default_rng(100 + cfg)
    seqs = sorted(rng.choice(wl.B, size=2, replace=False).tolist())
    heads = sorted(rng.choice(wl.H, size=3, replace=False).tolist())
    run_workload(wl, "bhtd", None, seqs=seqs, heads=heads, want_lists=(cfg != 2))


# ---- hand-made span lists: every case the index path is tested on ------------------------------------------
def run_spans(p, span_lists, ctx_lens, max_selected, max_spans=None, index_stride=None, out_dtype=torch.float32,
              want_lists=True, fill=-7):
    B = p.B
    offs = np.zeros(B + 1, np.int32)
    offs[1:] = np.cumsum([len(s) for s in span_lists])
    flat = np.asarray([x for s in span_lists for x in s], np.int32).reshape(-1, 2)
    if len(flat) == 0:
        flat = np.zeros((1, 2), np.int32)
    d_off, d_sp = torch.from_numpy(offs).to(DEV), torch.from_numpy(flat).to(DEV)
    d_ctx = torch.tensor(ctx_lens, dtype=torch.int32, device=DEV)
    stride = index_stride or (max_selected + 31) // 32 * 32
    index = torch.full((B, stride), fill, dtype=torch.int32, device=DEV)
    counts = torch.full((B,), fill, dtype=torch.int32, device=DEV)
    out = torch.full((B, p.H, p.D), 777.0, dtype=out_dtype, device=DEV)
    lse = torch.full((B, p.H), 777.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ms = max_spans or max(1, max(len(s) for s in span_lists))
    ws = torch.empty(ssa.decode_spans_workspace_bytes(desc, max_selected, ms), dtype=torch.uint8, device=DEV)
    before = ssa.launch_count()
    ssa.decode_attn_spans(desc, p.q, p.k, p.v, d_ctx, d_off, d_sp, ms, max_selected, out, lse,
                          index if want_lists else None, counts if want_lists else None, ws, status)
    launches = ssa.launch_count() - before
    torch.cuda.synchronize()
    return (out.double().cpu().numpy(), lse.double().cpu().numpy(), index.cpu().numpy(), counts.cpu().numpy(),
            int(status.item()), launches)


def check_spans(p, span_lists, ctx_lens, max_selected, max_spans=None, out_dtype=torch.float32, want_lists=True):
    """Runs the call and compares everything with the oracle; max_spans cuts the lists the oracle sees."""
    got, lse, index, counts, status, launches = run_spans(p, span_lists, ctx_lens, max_selected, max_spans,
                                                         out_dtype=out_dtype, want_lists=want_lists)
    want_status = 0
    ref_index = np.full((p.B, max_selected), -1, np.int32)
    ref_counts = np.zeros(p.B, np.int32)
    for b in range(p.B):
        sp = np.asarray(span_lists[b], np.int64).reshape(-1, 2)
        cap = None if max_spans is None else min(max_spans, ssa.MAX_SPANS_PER_SEQ)
        if cap is not None and len(sp) > cap:
            sp, want_status = sp[:cap], want_status | (1 << 20)
        want_status |= O.spans_status(sp, ctx_lens[b], max_selected)
        idx = O.spans_to_index(sp, ctx_lens[b])[:max_selected]
        ref_index[b, :len(idx)], ref_counts[b] = idx, len(idx)
        if want_lists:
            assert counts[b] == len(idx), f"request {b}"
            assert index[b, :len(idx)].tolist() == idx.tolist(), f"request {b}"
            assert np.all(index[b, len(idx):] == -7)
    bits = dict(GPU_BITS)
    bits[1 << 20] = ssa.DEV_TOO_MANY_SPANS
    assert status == sum(v for k, v in bits.items() if want_status & k)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, np.asarray(ctx_lens), ref_index, ref_counts,
                                        1.0 / np.sqrt(p.D), p.dtype)
    assert_parity(got, ref, out_dtype != torch.float32, "spans")
    live = ref_counts > 0
    np.testing.assert_allclose(lse[live], ref_lse[live], rtol=1e-5, atol=1e-5)
    assert np.all(got[~live] == 0) and np.all(np.isneginf(lse[~live]))
    return launches


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f16", 64)])
def test_empty_one_token_overlapping_unsorted_clipped(dtype, D):
    B, H, T = 8, 3, 700
    p = Problem(B, H, T, D, dtype, seed=3)
    ctx = [700, 1, 513, 64, 300, 700, 40, 700]
    lists = [
        [],                                             # no spans: empty selection
        [(0, 1)],                                       # one token
        [(0, 513)],                                     # the full context
        [(30, 40), (5, 9), (35, 50), (5, 9), (8, 8)],    # unsorted, overlapping, repeated, empty
        [(250, 400), (-5, 3), (9, 2)],                  # clipped at the context, negative start, reversed
        [(3, 5), (4, 9), (9, 12), (100, 700), (0, 1)],  # adjacent and overlapping
        [(50, 60)],                                     # entirely beyond the context: nothing left
        [(i, i + 1) for i in range(0, 64, 2)],          # 32 one-token spans
    ]
    assert check_spans(p, lists, ctx, 700) == 2         # several chunks: split pass + merge, no index kernel
    assert check_spans(p, lists[3:4] * 8, [64] * 8, 32, want_lists=False) == 1


@pytest.mark.parametrize("stride", [1, 7, 32, 33, 128])
def test_fixed_stride_table_without_offsets(stride):
    """span_offsets = NULL: request b owns `stride` pairs of the table, unused ones empty."""
    B, H, T, D = 5, 3, 900, 128
    p = Problem(B, H, T, D, "bf16", seed=30 + stride)
    rng = np.random.default_rng(stride)
    ctx = [900, 17, 500, 900, 64]
    table = np.zeros((B, stride, 2), np.int32)
    lists = []
    for b in range(B):
        k = int(rng.integers(0, stride + 1)) if b else stride          # request 0 uses every slot
        sp = [(int(a), int(a + rng.integers(0, 40))) for a in rng.integers(-3, ctx[b], size=k)]
        slots = rng.permutation(stride)[:k]                              # padding anywhere in the row
        for slot, pair in zip(slots, sp):
            table[b, slot] = pair
        lists.append([tuple(int(x) for x in row) for row in table[b]])
    max_selected = 900
    d_tab = torch.from_numpy(table).to(DEV)
    d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
    index = torch.full((B, 928), -7, dtype=torch.int32, device=DEV)
    counts = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    out = torch.full((B, H, D), 777.0, dtype=torch.float32, device=DEV)
    lse = torch.full((B, H), 777.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_spans_workspace_bytes(desc, max_selected, stride), dtype=torch.uint8, device=DEV)
    ssa.decode_attn_spans(desc, p.q, p.k, p.v, d_ctx, None, d_tab, stride, max_selected, out, lse, index, counts, ws,
                          status)
    torch.cuda.synchronize()
    want_status = 0
    ref_index = np.full((B, max_selected), -1, np.int32)
    ref_counts = np.zeros(B, np.int32)
    for b in range(B):
        want_status |= O.spans_status(lists[b], ctx[b], max_selected)
        idx = O.spans_to_index(lists[b], ctx[b])
        ref_index[b, :len(idx)], ref_counts[b] = idx, len(idx)
        assert int(counts[b]) == len(idx) and index[b, :len(idx)].cpu().numpy().tolist() == idx.tolist()
    assert int(status.item()) == sum(v for k, v in GPU_BITS.items() if want_status & k)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, np.asarray(ctx), ref_index, ref_counts,
                                        1.0 / np.sqrt(D), "bf16")
    live = ref_counts > 0
    assert_parity(out.double().cpu().numpy(), ref, False, "fixed-stride table")
    np.testing.assert_allclose(lse.double().cpu().numpy()[live], ref_lse[live], rtol=1e-5, atol=1e-5)


def test_more_than_32_and_more_than_128_spans():
    B, H, T, D = 3, 2, 3000, 128
    p = Problem(B, H, T, D, "bf16", seed=4)
    rng = np.random.default_rng(5)

    def random_spans(k, hi):
        s = rng.integers(0, hi - 20, size=k)
        return [(int(a), int(a + rng.integers(0, 20))) for a in s]

    # 33 .. 128 spans: merged by the whole block in shared memory; one launch (+ merge)
    lists = [random_spans(33, 3000), random_spans(128, 2000), random_spans(70, 900)]
    assert check_spans(p, lists, [3000, 2000, 900], 2560) <= 2
    # the bound says up to 500 spans: the lists are expanded by the index kernel first
    lists = [random_spans(500, 3000), random_spans(129, 2000), random_spans(2, 900)]
    assert check_spans(p, lists, [3000, 2000, 900], 3000, max_spans=500) == 3
    assert check_spans(p, lists, [3000, 2000, 900], 3000, max_spans=500, want_lists=False) == 3
    # more spans than the bound, on chip and through the index kernel: the surplus is dropped and flagged
    check_spans(p, lists, [3000, 2000, 900], 3000, max_spans=100)
    check_spans(p, lists, [3000, 2000, 900], 3000, max_spans=200)
    # more than SSA_MAX_SPANS_PER_SEQ
    lists = [random_spans(2100, 3000), [(0, 10)], []]
    check_spans(p, lists, [3000, 2000, 900], 3000, max_spans=4000)


def test_more_positions_than_max_selected_keep_the_first():
    B, H, T, D = 2, 2, 1200, 128
    p = Problem(B, H, T, D, "bf16", seed=6)
    lists = [[(100, 900), (0, 50)], [(0, 64)]]
    check_spans(p, lists, [1200, 1200], 300)            # 850 positions -> the first 300, overflow flagged
    check_spans(p, lists, [1200, 1200], 64)


def test_unselected_rows_do_not_matter():
    B, H, T, D = 2, 2, 600, 128
    p = Problem(B, H, T, D, "bf16", seed=7)
    lists = [[(10, 20), (300, 340)], [(0, 5), (590, 600)]]
    base = run_spans(p, lists, [600, 600], 64)[0]
    keep = np.zeros((B, T), bool)
    for b, sp in enumerate(lists):
        for s, e in sp:
            keep[b, s:e] = True
    nan16 = np.uint16(0x7FC0)
    for b in range(B):
        p.k_bits[b][:, ~keep[b]] = nan16
        p.v_bits[b][:, ~keep[b]] = nan16
    p.upload()
    again = run_spans(p, lists, [600, 600], 64)[0]
    assert np.array_equal(base, again)


def test_span_order_and_splitting_leave_the_output_bit_identical():
    B, H, T, D = 1, 4, 2048, 128
    p = Problem(B, H, T, D, "bf16", seed=8)
    a = [[(0, 64), (500, 800), (1900, 2048)]]
    b = [[(1900, 2048), (600, 800), (0, 30), (500, 600), (30, 64), (550, 650)]]
    ra, rb = run_spans(p, a, [2048], 1024), run_spans(p, b, [2048], 1024)
    assert np.array_equal(ra[0], rb[0]) and np.array_equal(ra[2], rb[2]) and ra[3].tolist() == rb[3].tolist()


def test_matches_the_two_call_path_bit_for_bit():
    """Same rows in the same order through the same arithmetic: the one-kernel path and
    ssa_spans_to_index + ssa_decode_attn_sparse give identical bits."""
    for wl in (inputs.make_config(2, B=8, H=4), inputs.make_config(5, density=0.25, B=2, H=4)):
        ds = DecodeStep(wl, out_dtype=torch.float32)
        ds.step()
        torch.cuda.synchronize()
        two_call, lse2 = ds.out.clone(), ds.lse.clone()
        ds.out.fill_(3.0)
        ds.attend_spans()
        torch.cuda.synchronize()
        assert torch.equal(ds.out, two_call) and torch.equal(ds.lse, lse2)


def test_mixed_batch_of_full_context_and_restricted_requests():
    """Requests at a "determine span" step attend to everything (one span over the context),
    the others to their spans, in one launch."""
    wl = inputs.make_config(2, B=6, H=4)
    spans, offs = [], [0]
    for b in range(wl.B):
        sp = [(0, int(wl.ctx_lens[b]))] if b % 2 == 0 else [tuple(x) for x in wl.spans_of(b)]
        spans += sp
        offs.append(len(spans))
    mixed = inputs.Workload("mixed", wl.seed, wl.B, wl.H, wl.D, wl.max_ctx, wl.dtype, wl.ctx_lens,
                            np.asarray(offs, np.int32), np.asarray(spans, np.int32), wl.seq_ids)
    ds = run_workload(mixed, "bhtd", torch.float32)
    got = ds.out_f64()
    ds.attend_dense()
    torch.cuda.synchronize()
    dense = ds.out_f64()
    np.testing.assert_allclose(got[0::2], dense[0::2], rtol=0, atol=2e-6)


@pytest.mark.parametrize("H,Hkv", [(8, 2), (16, 1), (6, 3)])
def test_grouped_query_heads(H, Hkv):
    wl = inputs.make_config(3, B=2, H=Hkv)
    ds = DecodeStep(wl, out_dtype=torch.float32, query_heads=H)
    ds.attend_spans(want_lists=True)
    torch.cuda.synchronize()
    assert int(ds.status.item()) == 0
    index, counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, ds.index_stride)
    assert ds.counts.cpu().numpy().tolist() == counts.tolist()
    k, v = wl.kv_bits()
    g = H // Hkv
    ref, _ = O.decode_attn_sparse(wl.q_bits(H), np.repeat(k, g, axis=1), np.repeat(v, g, axis=1), wl.ctx_lens, index,
                                  counts, 1.0 / np.sqrt(wl.D), wl.dtype)
    assert_parity(ds.out_f64(), ref, False, "grouped heads from span lists")


def test_argument_checks_launch_nothing():
    p = Problem(1, 2, 64, 128, "bf16", seed=9)
    out = torch.zeros((1, 2, 128), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    off = torch.tensor([0, 1], dtype=torch.int32, device=DEV)
    sp = torch.tensor([[0, 8]], dtype=torch.int32, device=DEV)
    ctx = torch.tensor([64], dtype=torch.int32, device=DEV)
    ws = torch.empty(ssa.decode_spans_workspace_bytes(desc, 64, 1), dtype=torch.uint8, device=DEV)
    idx = torch.zeros((1, 32), dtype=torch.int32, device=DEV)
    call = lambda **kw: ssa.decode_attn_spans(desc, p.q, p.k, p.v, ctx, kw.get("off", off), kw.get("sp", sp), kw.get("ms", 1),
                                              kw.get("sel", 64), out, None, kw.get("idx"), None, kw.get("ws", ws),
                                              None, check=False)
    before = ssa.launch_count()
    assert call(sp=None) == ssa.ERR_NULL
    assert call(off=None, ms=129) == ssa.ERR_UNSUPPORTED    # a fixed-stride table holds at most 128 pairs per request
    assert call(ms=0) == ssa.ERR_CAPACITY
    assert call(sel=0) == ssa.ERR_CAPACITY
    assert call(idx=idx) == ssa.ERR_CAPACITY            # list pitch 32 below max_selected 64
    assert call(ws=ws[:64]) == ssa.ERR_WORKSPACE
    assert call(ws=None) == ssa.ERR_WORKSPACE
    assert ssa.launch_count() == before
    assert call() == ssa.OK
