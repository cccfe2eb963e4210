"""ssa_decode_attn_sparse_noalloc: the variant for callers that cannot allocate.

Some users of the library cannot give it a workspace: a plug-in inside a host
application that owns the device allocator, a serving loop that froze its
memory pool after start-up, a path where cudaMalloc (which may synchronise
the device) is forbidden.  For them the split-KV scratch comes from a fixed
array inside the library.  This file checks, through the C ABI, that the
variant returns what ssa_decode_attn_sparse returns - on two calls in a row,
because the array is shared and keeps the previous call's contents - that both
agree with the fp64 oracle, and that it refuses requests larger than the
array.  It sorts last on purpose: a run
that stops at the first failure has then already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2404_09336_b200 import ssa


def _desc(B, H, D, T):
    d = ssa.AttnDesc()
    d.B, d.H, d.H_kv, d.D, d.max_ctx = B, H, H, D, T
    d.kv_dtype, d.out_dtype, d.scale = ssa.BF16, ssa.BF16, 0.0
    d.q_stride_b, d.q_stride_h = H * D, D
    d.k_stride_b, d.k_stride_h, d.k_stride_t = H * T * D, T * D, D
    d.v_stride_b, d.v_stride_h, d.v_stride_t = H * T * D, T * D, D
    d.o_stride_b, d.o_stride_h = H * D, D
    return d


def test_requests_beyond_the_builtin_scratch_are_refused():
    """Host-side check only: the pointers are never dereferenced because the
    size test fails first, so this also runs without a GPU."""
    d = _desc(8192, 32, 128, 8192)
    assert ssa.decode_workspace_bytes(d, 8192) > ssa.STATIC_SCRATCH_BYTES
    P = C.c_void_p(0x1000)
    before = ssa.launch_count()
    rc = ssa.lib.ssa_decode_attn_sparse_noalloc(C.byref(d), P, P, P, P, P, 8192, P, 8192, P, None, None, None)
    assert rc == ssa.ERR_WORKSPACE and ssa.launch_count() == before
    assert "workspace" in ssa.status_string(rc)
    # and the usual argument checks still apply
    assert ssa.lib.ssa_decode_attn_sparse_noalloc(None, P, P, P, P, P, 64, P, 64, P, None, None, None) == ssa.ERR_NULL
    d.D = 96
    assert ssa.lib.ssa_decode_attn_sparse_noalloc(C.byref(d), P, P, P, P, P, 64, P, 64, P, None, None, None) \
        == ssa.ERR_UNSUPPORTED


@pytest.mark.gpu
def test_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    from gpu_util import Problem
    from parity import assert_parity

    dev = "cuda:0"
    B, H, T, D = 2, 4, 3000, 128
    rng = np.random.default_rng(42)
    for call, seed in enumerate((101, 202)):           # second call: new data over the first call's leftovers
        p = Problem(B, H, T, D, "bf16", seed=seed)
        counts = [2500 - 700 * call, 1300 + 400 * call]
        index = np.full((B, 3008), -1, np.int32)
        for b in range(B):
            index[b, :counts[b]] = np.sort(rng.choice(T, counts[b], replace=False))
        d_idx = torch.from_numpy(index).to(dev)
        d_cnt = torch.tensor(counts, dtype=torch.int32, device=dev)
        d_ctx = torch.tensor([T, T], dtype=torch.int32, device=dev)
        outs, lses = [], []
        for variant in ("workspace", "noalloc"):
            out = torch.full((B, H, D), 9.0, dtype=torch.float32, device=dev)
            lse = torch.full((B, H), 9.0, dtype=torch.float32, device=dev)
            status = torch.zeros(1, dtype=torch.int32, device=dev)
            desc = ssa.make_desc(p.q, p.k, p.v, out)
            need = ssa.decode_workspace_bytes(desc, 3000)
            assert 0 < need <= ssa.STATIC_SCRATCH_BYTES
            if variant == "workspace":
                ws = torch.empty(need, dtype=torch.uint8, device=dev)
                ssa.decode_attn_sparse(desc, p.q, p.k, p.v, d_ctx, d_idx, d_cnt, 3000, out, lse, ws, status)
            else:
                ssa.decode_attn_sparse_noalloc(desc, p.q, p.k, p.v, d_ctx, d_idx, d_cnt, 3000, out, lse, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            outs.append(out.double().cpu().numpy())
            lses.append(lse.double().cpu().numpy())
        # same kernels, same split, same order of operations: the results agree to the
        # last bit; the parity rule of the other tests is the stated bound
        assert_parity(outs[1], outs[0], native_out=False, what=f"call {call}")
        np.testing.assert_allclose(lses[1], lses[0], rtol=1e-5, atol=1e-5)
        assert np.array_equal(outs[1], outs[0])
        # and both are right: the oracle's set-form attention over the same lists
        from oracle import ssa_oracle as O
        ref, ref_lse = O.decode_attn_sparse(p.q_bits, p.k_bits, p.v_bits, np.array([T, T]), index,
                                            np.asarray(counts, np.int32), 1.0 / np.sqrt(D), "bf16")
        assert_parity(outs[1], ref, native_out=False, what=f"call {call} against the oracle")
        np.testing.assert_allclose(lses[1], ref_lse, rtol=1e-5, atol=1e-5)


@pytest.mark.gpu
@pytest.mark.parametrize("H,Hkv,D,dtype,T,sel", [
    (4, 4, 128, "bf16", 400, 200),      # every request fits one thread block: the scratch is not touched
    (8, 2, 128, "bf16", 2600, 2000),    # grouped query heads, several chunks
    (3, 3, 64, "f16", 1500, 1200),      # fp16 storage, head dimension 64, output in the storage type
])
def test_other_shapes_against_the_workspace_call_and_the_oracle(H, Hkv, D, dtype, T, sel):
    from gpu_util import TORCH_DT, Problem, random_bits
    from oracle import ssa_oracle as O
    from paper_2404_09336_b200.runner import bits_to_tensor
    from parity import assert_parity

    dev = "cuda:0"
    B = 3
    rng = np.random.default_rng(7 + H)
    p = Problem(B, Hkv, T, D, dtype, seed=300 + H)
    q_bits = random_bits(rng, (B, H, D), dtype)
    q = bits_to_tensor(q_bits, dtype).to(dev)
    counts = [sel, sel // 3, 1]
    stride = (sel + 31) // 32 * 32
    index = np.full((B, stride), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(T, counts[b], replace=False))
    d_idx = torch.from_numpy(index).to(dev)
    d_cnt = torch.tensor(counts, dtype=torch.int32, device=dev)
    d_ctx = torch.tensor([T] * B, dtype=torch.int32, device=dev)
    native = dtype == "f16"
    odt = TORCH_DT[dtype] if native else torch.float32
    got = {}
    for variant in ("workspace", "noalloc", "noalloc again"):
        out = torch.full((B, H, D), 9.0, dtype=odt, device=dev)
        lse = torch.full((B, H), 9.0, dtype=torch.float32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        desc = ssa.make_desc(q, p.k, p.v, out)
        if variant == "workspace":
            ws = torch.empty(ssa.decode_workspace_bytes(desc, sel), dtype=torch.uint8, device=dev)
            ssa.decode_attn_sparse(desc, q, p.k, p.v, d_ctx, d_idx, d_cnt, sel, out, lse, ws, status)
        else:
            ssa.decode_attn_sparse_noalloc(desc, q, p.k, p.v, d_ctx, d_idx, d_cnt, sel, out, lse, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got[variant] = (out.double().cpu().numpy(), lse.double().cpu().numpy())
    g = H // Hkv
    ref, ref_lse = O.decode_attn_sparse(q_bits, np.repeat(p.k_bits, g, axis=1), np.repeat(p.v_bits, g, axis=1),
                                        np.array([T] * B), index, np.asarray(counts, np.int32), 1.0 / np.sqrt(D), dtype)
    for variant in ("noalloc", "noalloc again"):
        assert np.array_equal(got[variant][0], got["workspace"][0])
        assert_parity(got[variant][0], ref, native_out=native, what=variant)
        np.testing.assert_allclose(got[variant][1], ref_lse, rtol=1e-5, atol=1e-5)
