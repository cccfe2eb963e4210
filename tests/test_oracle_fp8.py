"""Pins of the oracle's e4m3 decoder: all 256 patterns against a library's conversion (torch.float8_e4m3fn),
hand values from the format's definition, symmetry and monotonicity; and that the batch attention functions
take an 8-bit cache (exactly the attention over the decoded values)."""
import numpy as np
import torch

from oracle import ssa_oracle as O


def test_all_256_patterns_against_the_library_type():
    bits = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(bits.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = O.decode_e4m3(bits)
    assert np.array_equal(np.isnan(got), np.isnan(ref)) and np.isnan(got).sum() == 2      # 0x7f and 0xff
    ok = ~np.isnan(ref)
    assert np.array_equal(got[ok], ref[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(ref[ok]))                       # -0 stays -0


def test_hand_values_from_the_definition():
    val = lambda b: float(O.decode_e4m3(np.array([b], np.uint8))[0])
    assert val(0x00) == 0.0 and val(0x38) == 1.0 and val(0xB8) == -1.0
    assert val(0x40) == 2.0 and val(0xC0) == -2.0 and val(0x3C) == 1.5
    assert val(0x01) == 2.0 ** -9                      # smallest subnormal: 1/8 * 2^-6
    assert val(0x07) == 7 / 8 * 2.0 ** -6              # largest subnormal
    assert val(0x08) == 2.0 ** -6                      # smallest normal
    assert val(0x7E) == 448.0 and val(0xFE) == -448.0  # largest finite: 1.75 * 2^8
    assert np.isnan(val(0x7F)) and np.isnan(val(0xFF))
    assert val(0x78) == 256.0                          # exponent 15 is an ordinary binade, not infinity


def test_order_and_symmetry():
    pos = O.decode_e4m3(np.arange(0x00, 0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)                    # patterns ascend with their values
    neg = O.decode_e4m3(np.arange(0x80, 0xFF, dtype=np.uint8))
    assert np.array_equal(neg, -pos)


def test_attention_over_an_8_bit_cache_is_attention_over_its_values():
    rng = np.random.default_rng(0)
    B, H, T, D = 2, 2, 40, 8
    k8 = rng.integers(0, 0x7F, size=(B, H, T, D)).astype(np.uint8)          # finite patterns
    v8 = rng.integers(0x80, 0xFF, size=(B, H, T, D)).astype(np.uint8)
    q16 = (rng.standard_normal((B, H, D)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)   # bf16 patterns
    index = np.stack([np.sort(rng.choice(T, 10, replace=False)) for _ in range(B)]).astype(np.int32)
    counts = np.array([10, 7], np.int32)
    ctx = np.array([T, T])
    got, lse = O.decode_attn_sparse(q16, k8, v8, ctx, index, counts, 0.2, "bf16/e4m3")
    ref, ref_lse = O.decode_attn_sparse(O.decode_bits(q16, "bf16"), O.decode_e4m3(k8), O.decode_e4m3(v8), ctx, index,
                                        counts, 0.2)
    assert np.array_equal(got, ref) and np.array_equal(lse, ref_lse)
    gotd, _ = O.decode_attn_dense(q16, k8, v8, ctx, 0.2, "bf16/e4m3")
    refd, _ = O.decode_attn_dense(O.decode_bits(q16, "bf16"), O.decode_e4m3(k8), O.decode_e4m3(v8), ctx, 0.2)
    assert np.array_equal(gotd, refd)
