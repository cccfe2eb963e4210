"""Randomised shapes through the restricted and the full-context call against
the oracle: head counts and groupings, head sizes, storage types, cache
layouts, list lengths (empty, one entry, everything), sorted and unsorted
lists, loose and tight host bounds, output in fp32 or the storage type."""
import random

import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O

from gpu_util import Problem, random_bits
from parity import parity_report

pytestmark = pytest.mark.gpu


def one_case(case):
    rnd = random.Random(case)
    D = rnd.choice([64, 128])
    dtype = rnd.choice(["bf16", "f16"])
    Hkv = rnd.choice([1, 2, 3, 4])
    G = rnd.choice([1, 1, 2, 3, 4, 8, 16, 20])
    H = Hkv * G
    B = rnd.choice([1, 2, 5, 17, 40, 150]) if H < 40 else rnd.choice([1, 2, 5, 17])
    T = rnd.choice([1, 7, 64, 65, 255, 513, 700, 1500, 2600])
    if B * Hkv * T * D > 40e6:
        T = max(1, int(40e6 // (B * Hkv * D)))
    layout = rnd.choice(["bhtd", "bthd"])
    p = Problem(B, Hkv, T, D, dtype, seed=case, layout=layout)
    rng = np.random.default_rng(case)
    p.q_bits = random_bits(rng, (B, H, D), dtype)
    p.H = H
    p.upload()
    ctx = [int(rng.integers(1, T + 1)) for _ in range(B)]
    counts = [int(rng.integers(0, n + 1)) if rnd.random() < 0.8 else rnd.choice([0, 1, n]) for n in ctx]
    stride = max(counts + [1]) + rnd.choice([0, 3, 40])
    index = np.full((B, stride), -1, np.int32)
    for b in range(B):
        sel = rng.choice(ctx[b], counts[b], replace=False)
        index[b, :counts[b]] = np.sort(sel) if rnd.random() < 0.7 else sel
    ms = rnd.choice([stride, max(counts + [1])])
    native = rnd.random() < 0.3
    what = f"case {case}: B={B} H={H} Hkv={Hkv} D={D} {dtype} T={T} {layout} ms={ms} stride={stride} native={native}"
    out, lse, status, _ = p.sparse(ctx, index, counts, max_selected=ms, out_dtype=None if native else torch.float32)
    sample = sorted(set(rng.integers(0, B, size=min(B, 6)).tolist()))
    kr, vr = np.repeat(p.k_bits, G, axis=1), np.repeat(p.v_bits, G, axis=1)
    scale = 1 / np.sqrt(D)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, kr, vr, ctx, index, counts, scale, dtype, seqs=sample)
    r = parity_report(out[sample], ref[sample])
    assert status == 0 and np.all(np.isfinite(out)), what
    assert (r["fails"] == 0) if native else (r["max_abs"] <= 2e-3 and r["max_rel"] <= 1e-2), f"{what}: {r}"
    fin = np.isfinite(ref_lse[sample])
    np.testing.assert_allclose(lse[sample][fin], ref_lse[sample][fin], rtol=1e-5, atol=1e-5, err_msg=what)
    assert np.all(np.isneginf(lse[sample][~fin])), what
    out_d, _, st_d = p.dense(ctx)
    ref_d, _ = O.decode_attn_dense(p.q_bits, kr, vr, ctx, scale, dtype, seqs=sample)
    rd = parity_report(out_d[sample], ref_d[sample])
    assert st_d == 0 and rd["max_abs"] <= 2e-3 and rd["max_rel"] <= 1e-2, f"{what}, dense: {rd}"


@pytest.mark.parametrize("first", range(0, 48, 8))
def test_random_shapes(first):
    for case in range(first, first + 8):
        one_case(case)
        torch.cuda.empty_cache()
