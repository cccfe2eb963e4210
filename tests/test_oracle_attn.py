"""Pins for the oracle's attention functions (CPU only).

Each pin is something the mathematics fixes without reference to the oracle's
own code: closed forms, a library routine, structurally different
formulations, invariants.  The last test plants mistakes in copies of the
oracle and checks that the pins catch each of them.
"""
import math

import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O


def rand_case(seed, n=97, D=16, frac=0.3):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal(D)
    K = rng.standard_normal((n, D))
    V = rng.standard_normal((n, D))
    idx = np.flatnonzero(rng.random(n) < frac)
    if idx.size == 0:
        idx = np.array([n // 2])
    return q, K, V, idx


# ---- the pins, as functions of the implementation under test ----------------
def pin_single_token(attn):
    q, K, V, _ = rand_case(1)
    for j in (0, 13, 96):
        out, lse = attn(q, K, V, np.array([j]), 0.25)
        assert np.array_equal(out, V[j])                  # weight exactly 1
        assert lse == pytest.approx(0.25 * float(K[j] @ q), rel=1e-14)


def pin_two_tokens(attn):
    q, K, V, _ = rand_case(2)
    a, b, scale = 5, 40, 0.3
    s1, s2 = scale * float(K[a] @ q), scale * float(K[b] @ q)
    sig = 1.0 / (1.0 + math.exp(-(s1 - s2)))
    out, lse = attn(q, K, V, np.array([a, b]), scale)
    np.testing.assert_allclose(out, sig * V[a] + (1 - sig) * V[b], rtol=1e-13, atol=1e-15)
    assert lse == pytest.approx(math.log(math.exp(s1) + math.exp(s2)), rel=1e-13)


def pin_uniform(attn):
    q, K, V, idx = rand_case(3)
    out, lse = attn(np.zeros_like(q), K, V, idx, 0.7)     # q = 0: all scores equal
    np.testing.assert_allclose(out, V[idx].mean(axis=0), rtol=1e-13, atol=1e-15)
    assert lse == pytest.approx(math.log(len(idx)), rel=1e-13)
    K2 = K.copy()
    K2[idx] = K[idx[0]]                                   # identical selected keys
    out, _ = attn(q, K2, V, idx, 0.7)
    np.testing.assert_allclose(out, V[idx].mean(axis=0), rtol=1e-12, atol=1e-14)


def pin_log_weights(attn):
    # D = 2, scale 1, q = (1, 0), k_j = (ln j, 0): weights j / 6 for j = 1, 2, 3
    q = np.array([1.0, 0.0])
    K = np.array([[9.0, 9.0]] + [[math.log(j), 0.0] for j in (1, 2, 3)] + [[-3.0, 1.0]])
    V = np.array([[100.0, 100.0], [1.0, 0.0], [0.0, 1.0], [2.0, -2.0], [50.0, 50.0]])
    out, lse = attn(q, K, V, np.array([1, 2, 3]), 1.0)
    np.testing.assert_allclose(out, [1 / 6 + 3 / 6 * 2, 2 / 6 - 3 / 6 * 2], rtol=1e-14)
    assert lse == pytest.approx(math.log(6.0), rel=1e-14)
    # the softmax scale multiplies the score: scale 2 -> weights j^2 / 14
    out, lse = attn(q, K, V, np.array([1, 2, 3]), 2.0)
    np.testing.assert_allclose(out, [1 / 14 + 9 / 14 * 2, 4 / 14 - 9 / 14 * 2], rtol=1e-13)
    assert lse == pytest.approx(math.log(14.0), rel=1e-14)


def pin_library_sdpa(attn):
    for seed in range(3):
        q, K, V, idx = rand_case(10 + seed, n=130, D=32)
        scale = 1.0 / math.sqrt(32)
        keep = np.zeros(130, bool)
        keep[idx] = True
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q)[None, None, None, :], torch.from_numpy(K)[None, None],
            torch.from_numpy(V)[None, None], attn_mask=torch.from_numpy(keep)[None, None, None, :],
            scale=scale)[0, 0, 0].numpy()
        out, _ = attn(q, K, V, idx, scale)
        np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-14)


def pin_invariants(attn):
    q, K, V, idx = rand_case(20, n=200, D=24)
    scale = 0.2
    out, lse = attn(q, K, V, idx, scale)
    # convex combination of the selected value rows
    assert np.all(out <= V[idx].max(axis=0) + 1e-12) and np.all(out >= V[idx].min(axis=0) - 1e-12)
    # unselected rows with huge values must not move the hull
    # a constant added to every score leaves the output unchanged, lse shifts
    q2 = np.append(q, 1.0)
    K2 = np.hstack([K, np.full((K.shape[0], 1), 3.5)])
    out2, lse2 = attn(q2, K2, V, idx, scale)
    np.testing.assert_allclose(out2, out, rtol=1e-12, atol=1e-14)
    assert lse2 == pytest.approx(lse + scale * 3.5, rel=1e-13)
    # order of the selected positions
    perm = np.random.default_rng(0).permutation(idx)
    out3, lse3 = attn(q, K, V, perm, scale)
    np.testing.assert_allclose(out3, out, rtol=1e-13, atol=1e-15)
    assert lse3 == pytest.approx(lse, rel=1e-14)
    # unselected rows are irrelevant, even when poisoned
    Kp, Vp = K.copy(), V.copy()
    unsel = np.setdiff1d(np.arange(K.shape[0]), idx)
    Kp[unsel] = np.nan
    Vp[unsel] = np.inf
    out4, lse4 = attn(q, Kp, Vp, idx, scale)
    assert np.array_equal(out4, out) and lse4 == lse
    # adding a key far below the others changes nothing visible; far above takes over
    Kx = np.vstack([K, 1e3 * q / (q @ q)])
    Vx = np.vstack([V, np.full((1, V.shape[1]), 7.0)])
    out5, _ = attn(q, Kx, Vx, np.append(idx, K.shape[0]), 1.0)
    np.testing.assert_allclose(out5, 7.0, rtol=1e-12)


def pin_empty(attn):
    q, K, V, _ = rand_case(30)
    out, lse = attn(q, K, V, np.array([], dtype=np.int64), 0.5)
    assert np.array_equal(out, np.zeros(V.shape[1])) and lse == -np.inf


ALL_PINS = [pin_single_token, pin_two_tokens, pin_uniform, pin_log_weights,
            pin_library_sdpa, pin_invariants, pin_empty]


@pytest.mark.parametrize("pin", ALL_PINS, ids=lambda f: f.__name__)
def test_set_form_pins(pin):
    pin(O.attn_set_form)


# ---- the other formulations -------------------------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_formulations_agree(seed):
    n = [1, 31, 97, 256, 300, 513][seed]
    q, K, V, idx = rand_case(100 + seed, n=n, D=16, frac=[1.0, 0.5, 0.1, 0.3, 0.7, 0.02][seed])
    scale = 0.25
    out, lse = O.attn_set_form(q, K, V, idx, scale)
    keep = np.zeros(n, bool)
    keep[idx] = True
    o4, l4 = O.attn_additive_mask(q, K, V, n, keep, scale)
    np.testing.assert_allclose(o4, out, rtol=1e-12, atol=1e-14)
    assert l4 == pytest.approx(lse, rel=1e-13, abs=1e-13)
    for bs in (32, 256):
        meta = O.encode_blocked(idx, bs)
        assert all(bm.any() for _, bm in meta)                   # empty blocks omitted
        assert sorted({int(j) // bs for j in idx}) == [blk for blk, _ in meta]
        o5, l5 = O.attn_alg1_blocked(q, K, V, n, meta, bs, scale)
        np.testing.assert_allclose(o5, out, rtol=1e-12, atol=1e-14)
        assert l5 == pytest.approx(lse, rel=1e-13, abs=1e-13)


@pytest.mark.parametrize("pin", [pin_two_tokens, pin_log_weights, pin_library_sdpa, pin_uniform],
                         ids=lambda f: f.__name__)
def test_additive_mask_and_blocked_pins(pin):
    def additive(q, K, V, idx, scale):
        keep = np.zeros(K.shape[0], bool)
        keep[idx] = True
        return O.attn_additive_mask(q, K, V, K.shape[0], keep, scale)

    def blocked(q, K, V, idx, scale):
        return O.attn_alg1_blocked(q, K, V, K.shape[0], O.encode_blocked(idx, 32), 32, scale)

    pin(additive)
    pin(blocked)


def test_full_span_equals_dense():
    for n in (1, 2, 77, 300):
        q, K, V, _ = rand_case(200 + n, n=n + 5, D=16)        # rows beyond n exist
        out, lse = O.attn_set_form(q, K, V, np.arange(n), 0.25)
        od, ld = O.attn_dense(q, K, V, n, 0.25)
        np.testing.assert_allclose(od, out, rtol=1e-13, atol=1e-15)
        assert ld == pytest.approx(lse, rel=1e-14)
    od, ld = O.attn_dense(q, K, V, 0, 0.25)
    assert not od.any() and ld == -np.inf


def test_dense_pins():
    def dense_as_attn(q, K, V, idx, scale):
        idx = np.asarray(idx, dtype=np.int64)
        return O.attn_dense(q, K[idx], V[idx], len(idx), scale)
    for pin in (pin_single_token, pin_two_tokens, pin_uniform, pin_log_weights, pin_library_sdpa):
        pin(dense_as_attn)


@pytest.mark.parametrize("seed", range(5))
def test_split_merge(seed):
    q, K, V, idx = rand_case(300 + seed, n=400, D=16, frac=0.4)
    scale = 0.25
    out, lse = O.attn_set_form(q, K, V, idx, scale)
    rng = np.random.default_rng(seed)
    cuts = np.sort(rng.choice(np.arange(1, len(idx)), size=min(4, len(idx) - 1), replace=False))
    parts = np.split(idx, cuts) + [np.array([], dtype=np.int64)]        # an empty part too
    ms, ls, accs = zip(*[O.attn_partial(q, K, V, p, scale) for p in parts])
    om, lm = O.merge_partials(ms, ls, accs)
    np.testing.assert_allclose(om, out, rtol=1e-13, atol=1e-15)
    assert lm == pytest.approx(lse, rel=1e-14)
    o0, l0 = O.merge_partials([-np.inf, -np.inf], [0.0, 0.0], np.zeros((2, 16)))
    assert not o0.any() and l0 == -np.inf


# ---- storage decoders ----------------------------------------------------------
def test_decoders_known_patterns():
    bf = np.array([0x3F80, 0xC000, 0x0000, 0x8000, 0x3F81, 0x7F80, 0x0001], np.uint16)
    v = O.decode_bits(bf, "bf16")
    assert v[:5].tolist() == [1.0, -2.0, 0.0, -0.0, 1.0 + 2.0 ** -7]
    assert np.isinf(v[5]) and v[6] == 2.0 ** -133
    hf = np.array([0x3C00, 0xC000, 0x0001, 0x7BFF, 0x3555, 0xFC00], np.uint16)
    w = O.decode_bits(hf, "f16")
    assert w[:4].tolist() == [1.0, -2.0, 2.0 ** -24, 65504.0]
    assert w[4] == (1 + 0x155 / 1024) * 2.0 ** -2 and w[5] == -np.inf


def test_decoders_against_library():
    bits = np.arange(0, 65536, dtype=np.uint16)
    t = torch.from_numpy(bits.view(np.int16).copy())
    ref_bf = t.view(torch.bfloat16).to(torch.float64).numpy()
    ref_hf = t.view(torch.float16).to(torch.float64).numpy()
    np.testing.assert_array_equal(O.decode_bits(bits, "bf16"), ref_bf)
    np.testing.assert_array_equal(O.decode_bits(bits, "f16"), ref_hf)


# ---- batch wrappers -------------------------------------------------------------
def test_batch_wrappers_match_single():
    rng = np.random.default_rng(5)
    B, H, T, D = 2, 3, 40, 8
    q = rng.standard_normal((B, H, D))
    Kc = rng.standard_normal((B, H, T, D))
    Vc = rng.standard_normal((B, H, T, D))
    ctx = np.array([33, 40])
    index, counts, _ = O.spans_to_index_batch([0, 2, 3], [(0, 4), (20, 50), (5, 9)], ctx, 64)
    index[1, 3] = 77                                             # out of range: skipped
    out, lse = O.decode_attn_sparse(q, Kc, Vc, ctx, index, counts, 0.3)
    for b in range(B):
        idx = [j for j in index[b, :counts[b]] if 0 <= j < ctx[b]]
        for h in range(H):
            o, l = O.attn_set_form(q[b, h], Kc[b, h], Vc[b, h], idx, 0.3)
            np.testing.assert_array_equal(out[b, h], o)
            assert lse[b, h] == l
    od, ld = O.decode_attn_dense(q, Kc, Vc, ctx, 0.3)
    o, l = O.attn_dense(q[1, 2], Kc[1, 2], Vc[1, 2], 40, 0.3)
    np.testing.assert_array_equal(od[1, 2], o)
    # a token-major cache seen through a transposed view gives the same result
    Kt = np.ascontiguousarray(Kc.transpose(0, 2, 1, 3)).transpose(0, 2, 1, 3)
    out2, _ = O.decode_attn_sparse(q, Kt, Vc, ctx, index, counts, 0.3)
    np.testing.assert_array_equal(out2, out)


# ---- planted mistakes must be caught ---------------------------------------------
def _mutants():
    def no_scale(q, K, V, idx, scale):
        return O.attn_set_form(q, K, V, idx, 1.0)

    def k_v_swapped(q, K, V, idx, scale):
        return O.attn_set_form(q, V, K, idx, scale)

    def wrong_sign(q, K, V, idx, scale):
        return O.attn_set_form(-q, K, V, idx, scale)

    def not_normalised(q, K, V, idx, scale):
        m, l, acc = O.attn_partial(q, K, V, idx, scale)
        return acc, m + np.log(l) if l else -np.inf

    def off_by_one(q, K, V, idx, scale):
        idx = np.asarray(idx, dtype=np.int64)
        return O.attn_set_form(q, K, V, np.minimum(idx + 1, K.shape[0] - 1), scale)

    def values_off_by_one(q, K, V, idx, scale):
        return O.attn_set_form(q, K, np.roll(V, 1, axis=0), idx, scale)

    def reads_everything(q, K, V, idx, scale):
        return O.attn_dense(q, K, V, K.shape[0], scale)

    def sqrt_scale(q, K, V, idx, scale):
        return O.attn_set_form(q, K, V, idx, math.sqrt(scale))

    def drops_last(q, K, V, idx, scale):
        idx = np.asarray(idx)
        return O.attn_set_form(q, K, V, idx[:-1] if len(idx) > 1 else idx, scale)

    def lse_without_max(q, K, V, idx, scale):
        out, lse = O.attn_set_form(q, K, V, idx, scale)
        m, _, _ = O.attn_partial(q, K, V, idx, scale)
        return out, lse - m

    return [no_scale, k_v_swapped, wrong_sign, not_normalised, off_by_one, values_off_by_one,
            reads_everything, sqrt_scale, drops_last, lse_without_max]


@pytest.mark.parametrize("mutant", _mutants(), ids=lambda f: f.__name__)
def test_pins_catch_planted_mistakes(mutant):
    caught = 0
    for pin in ALL_PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError, IndexError):
            caught += 1
    assert caught >= 1
