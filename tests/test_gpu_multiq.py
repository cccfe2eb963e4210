"""ssa_decode_attn_sparse_multiq / ssa_decode_attn_dense_multiq (several query tokens per head over one selected
set) against the fp64 oracle's row-by-row set form."""
import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import ssa
from paper_2404_09336_b200.runner import bits_to_tensor

from gpu_util import DEV, TORCH_DT, Problem, random_bits
from parity import assert_parity

pytestmark = pytest.mark.gpu


def setup(B, H, Hkv, Tq, T, D, dtype, seed, counts):
    rng = np.random.default_rng(seed)
    p = Problem(B, Hkv, T, D, dtype, seed=seed)
    q_bits = random_bits(rng, (B, H, Tq, D), dtype)
    stride = (max(max(counts), 1) + 31) // 32 * 32
    index = np.full((B, stride), -1, np.int32)
    for b in range(B):
        index[b, :counts[b]] = np.sort(rng.choice(T, counts[b], replace=False))
    return p, q_bits, index


@pytest.mark.parametrize("Tq", [1, 2, 4])
@pytest.mark.parametrize("G", [1, 4])
def test_sparse_against_the_oracle(Tq, G):
    B, Hkv, T, D = 3, 2, 1500, 128
    H = Hkv * G
    counts = [1200, 333, 1]
    p, q_bits, index = setup(B, H, Hkv, Tq, T, D, "bf16", 50 + 10 * Tq + G, counts)
    q = bits_to_tensor(q_bits, "bf16").to(DEV)
    out = torch.full((B, H, Tq, D), 7.0, dtype=torch.float32, device=DEV)
    lse = torch.full((B, H, Tq), 7.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc, n_q, qst, ost = ssa.make_desc_multiq(q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_multiq_workspace_bytes(desc, n_q, 1200), dtype=torch.uint8, device=DEV)
    d_idx, d_cnt = torch.from_numpy(index).to(DEV), torch.tensor(counts, dtype=torch.int32, device=DEV)
    d_ctx = torch.tensor([T] * B, dtype=torch.int32, device=DEV)
    ssa.decode_attn_sparse_multiq(desc, n_q, qst, ost, q, p.k, p.v, d_ctx, d_idx, d_cnt, 1200, out, lse, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref, ref_lse = O.decode_attn_sparse_multiq(q_bits, p.k_bits, p.v_bits, [T] * B, index, counts, 1 / np.sqrt(D), "bf16")
    assert_parity(out.double().cpu().numpy(), ref, False, f"Tq={Tq} G={G}")
    np.testing.assert_allclose(lse.double().cpu().numpy(), ref_lse, rtol=1e-5, atol=1e-5)
    if Tq == 1 and G == 1:                                      # one token: the single-query call, bit for bit
        p.q = q[:, :, 0].contiguous()
        got1, _, _, _ = p.sparse([T] * B, index, counts, 1200)
        assert np.array_equal(got1, out[:, :, 0].double().cpu().numpy())


@pytest.mark.parametrize("H,Hkv,Tq,D,dtype", [(3, 3, 3, 128, "bf16"), (8, 2, 8, 128, "f16"), (2, 2, 2, 64, "f16")])
def test_dense_and_other_shapes(H, Hkv, Tq, D, dtype):
    """An odd token count, (heads per K/V head) x tokens above 16 (each pair its own block), head dimension 64;
    native output type; the dense call; ragged contexts."""
    B, T = 2, 700
    counts = [600, 45]
    ctx = [700, 90]
    p, q_bits, index = setup(B, H, Hkv, Tq, T, D, dtype, 90 + H + Tq, counts)
    index[1, :45] = np.sort(np.random.default_rng(1).choice(90, 45, replace=False))
    q = bits_to_tensor(q_bits, dtype).to(DEV)
    out = torch.full((B, H, Tq, D), 7.0, dtype=TORCH_DT[dtype], device=DEV)
    lse = torch.full((B, H, Tq), 7.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc, n_q, qst, ost = ssa.make_desc_multiq(q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_multiq_workspace_bytes(desc, n_q, T), dtype=torch.uint8, device=DEV)
    d_idx, d_cnt = torch.from_numpy(index).to(DEV), torch.tensor(counts, dtype=torch.int32, device=DEV)
    d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
    ssa.decode_attn_sparse_multiq(desc, n_q, qst, ost, q, p.k, p.v, d_ctx, d_idx, d_cnt, 600, out, lse, ws, status)
    torch.cuda.synchronize()
    ref, ref_lse = O.decode_attn_sparse_multiq(q_bits, p.k_bits, p.v_bits, ctx, index, counts, 1 / np.sqrt(D), dtype)
    assert_parity(out.double().cpu().numpy(), ref, True, "sparse")
    np.testing.assert_allclose(lse.double().cpu().numpy(), ref_lse, rtol=1e-5, atol=1e-5)
    ssa.decode_attn_dense_multiq(desc, n_q, qst, ost, q, p.k, p.v, d_ctx, out, lse, ws, status)
    torch.cuda.synchronize()
    full = np.stack([np.arange(T, dtype=np.int32)] * B)
    refd, refd_lse = O.decode_attn_sparse_multiq(q_bits, p.k_bits, p.v_bits, ctx, full, ctx, 1 / np.sqrt(D), dtype)
    assert_parity(out.double().cpu().numpy(), refd, True, "dense")
    np.testing.assert_allclose(lse.double().cpu().numpy(), refd_lse, rtol=1e-5, atol=1e-5)
    assert int(status.item()) == 0


def test_layout_and_size_checks():
    p = Problem(1, 2, 64, 128, "bf16", seed=1)
    q = torch.zeros((1, 2, 4, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros((1, 2, 4, 128), dtype=torch.float32, device=DEV)
    desc, n_q, qst, ost = ssa.make_desc_multiq(q, p.k, p.v, out)
    ctx = torch.tensor([64], dtype=torch.int32, device=DEV)
    idx = torch.zeros((1, 64), dtype=torch.int32, device=DEV)
    cnt = torch.tensor([8], dtype=torch.int32, device=DEV)
    ws = torch.empty(ssa.decode_multiq_workspace_bytes(desc, 4, 64), dtype=torch.uint8, device=DEV)
    call = lambda n, a, b: ssa.decode_attn_sparse_multiq(desc, n, a, b, q, p.k, p.v, ctx, idx, cnt, 64, out, None, ws,
                                                         None, check=False)
    before = ssa.launch_count()
    assert call(0, qst, ost) == ssa.ERR_SHAPE
    assert call(2, qst, ost) == ssa.ERR_UNSUPPORTED            # heads' rows not side by side for this count
    assert call(4, qst * 2, ost) == ssa.ERR_UNSUPPORTED
    assert ssa.decode_multiq_workspace_bytes(desc, 0, 64) == 0
    assert ssa.launch_count() == before
    assert call(4, qst, ost) == ssa.OK
