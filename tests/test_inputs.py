"""The seeded workload generators follow their recipes (CPU only)."""
import numpy as np
import pytest

from paper_2404_09336_b200 import inputs


def covered(sp, n):
    m = np.zeros(n, bool)
    for s, e in sp:
        m[s:e] = True
    return int(m.sum())


def test_cfg1_recipe():
    wl = inputs.make_config(1)
    assert (wl.B, wl.H, wl.D, wl.max_ctx, wl.dtype) == (1, 8, 64, 512, "f16")
    sp = wl.spans_of(0).tolist()
    assert [0, 32] in sp and [496, 512] in sp and len(sp) == 5
    mids = [s for s in sp if s not in ([0, 32], [496, 512])]
    assert all(8 <= e - s <= 16 and 32 <= s and e <= 496 for s, e in mids)
    assert 32 + 16 + 24 <= covered(sp, 512) <= 32 + 16 + 48


def test_cfg2_recipe():
    wl = inputs.make_config(2)
    assert (wl.B, wl.H, wl.D, wl.max_ctx, wl.dtype) == (64, 32, 128, 1024, "bf16")
    assert wl.ctx_lens.min() >= 256 and wl.ctx_lens.max() <= 1024 and len(set(wl.ctx_lens.tolist())) > 30
    for i in range(wl.B):
        n = int(wl.ctx_lens[i])
        sp = wl.spans_of(i).tolist()
        assert [0, 64] in sp and [n - 32, n] in sp and 3 <= len(sp) <= 6
        tot = sum(e - s for s, e in sp)
        assert tot == covered(sp, n)                       # non-overlapping
        assert 100 <= tot <= 224
    assert 100 <= wl.selected_upper_bound() <= 224


def test_cfg3_recipe():
    wl = inputs.make_config(3)
    assert (wl.B, wl.H, wl.D, wl.max_ctx) == (16, 32, 128, 4096)
    for i in range(wl.B):
        sp = wl.spans_of(i).tolist()
        assert [0, 64] in sp and [4032, 4096] in sp and 4 <= len(sp) <= 12
        for s, e in sp:
            if [s, e] not in ([0, 64], [4032, 4096]):
                assert (s - 64) % 40 == 0 and 64 <= s < e <= 3968 and e - s <= 200
        assert 128 + 40 <= covered(sp, 4096) <= 128 + 2000


def test_cfg4_recipe():
    wl = inputs.make_config(4)
    assert (wl.B, wl.H, wl.D, wl.max_ctx) == (8, 32, 128, 16384)
    for i in range(wl.B):
        sp = wl.spans_of(i).tolist()
        assert len(sp) == 18 and [0, 64] in sp and [16256, 16384] in sp
        tot = sum(e - s for s, e in sp)
        assert tot == covered(sp, 16384) and 192 + 16 * 32 <= tot <= 192 + 16 * 256


@pytest.mark.parametrize("f", inputs.DENSITIES)
def test_cfg5_hits_the_density_exactly(f):
    wl = inputs.make_config(5, density=f, B=4)
    for i in range(wl.B):
        sp = wl.spans_of(i).tolist()
        assert covered(sp, 8192) == round(f * 8192) == sum(e - s for s, e in sp)
        if f < 1:
            assert [8128, 8192] in sp


def test_determinism_and_independent_streams():
    a, b = inputs.make_config(2, B=3, H=2), inputs.make_config(2, B=3, H=2)
    assert np.array_equal(a.spans, b.spans) and np.array_equal(a.ctx_lens, b.ctx_lens)
    ka, va = a.kv_bits_seq(1)
    kb, vb = b.kv_bits_seq(1)
    assert np.array_equal(ka, kb) and np.array_equal(va, vb) and not np.array_equal(ka, va)
    assert np.array_equal(a.q_bits(), b.q_bits())
    k_all, v_all = a.kv_bits(threads=2)
    assert np.array_equal(k_all[1], ka) and np.array_equal(v_all[1], va)
    assert ka.shape == (2, 1024, 128) and ka.dtype == np.uint16
    # request ids select the streams: a later window of the same workload
    c = inputs.make_config(2, B=2, H=2, first_id=1)
    assert np.array_equal(c.spans_of(0), a.spans_of(1)) and np.array_equal(c.kv_bits_seq(0)[0], ka)


def test_rounding_to_storage():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 1.0 + 2 ** -8 + 2 ** -20], np.float32)
    b = inputs.round_to_storage(x, "bf16")
    # ties to even: 1 + 2^-8 -> 1.0, 1 + 3*2^-8 -> 1 + 2^-6; above the tie rounds up
    assert b.tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x3F81]
    h = inputs.round_to_storage(np.array([1.0, 65504.0, 2.0 ** -24], np.float32), "f16")
    assert h.tolist() == [0x3C00, 0x7BFF, 0x0001]


def test_value_distribution():
    wl = inputs.make_config(1)
    k, v = wl.kv_bits_seq(0)
    x = k.view(np.float16).astype(np.float64)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01


def test_shard_partitions_the_batch():
    wl = inputs.make_config(2, B=7, H=2)
    parts = [wl.shard(r, 3) for r in range(3)]
    assert sum(p.B for p in parts) == 7
    assert np.array_equal(np.concatenate([p.ctx_lens for p in parts]), wl.ctx_lens)
    assert np.array_equal(np.concatenate([p.spans for p in parts]), wl.spans)
    assert np.array_equal(np.concatenate([p.seq_ids for p in parts]), wl.seq_ids)
    p = parts[1]
    g = int(p.seq_ids[0])
    assert np.array_equal(p.spans_of(0), wl.spans_of(g))
    assert np.array_equal(p.kv_bits_seq(0)[0], wl.kv_bits_seq(g)[0])
    assert np.array_equal(p.q_bits()[0], wl.q_bits()[g])


def test_mixed_workload_replaces_every_kth_list_by_the_full_context():
    base = inputs.make_config(2, B=9, H=2)
    mixed = inputs.make_mixed(4, B=9, H=2)
    assert np.array_equal(mixed.ctx_lens, base.ctx_lens) and mixed.seed == base.seed
    for b in range(9):
        if b % 4 == 0:
            assert mixed.spans_of(b).tolist() == [[0, int(base.ctx_lens[b])]]
        else:
            assert mixed.spans_of(b).tolist() == base.spans_of(b).tolist()
    assert mixed.selected_upper_bound() == int(base.ctx_lens[[0, 4, 8]].max())
