"""8-bit (e4m3) cache storage: the attention calls over a cache of uint8 patterns against the fp64 oracle, whose
decoder is written from the format's definition.  Queries are bf16; outputs fp32 or bf16."""
import numpy as np
import pytest
import torch

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import ssa
from paper_2404_09336_b200.inputs import round_to_storage

from gpu_util import DEV
from parity import assert_parity

pytestmark = pytest.mark.gpu


def to_e4m3_bits(x32):
    return torch.from_numpy(np.ascontiguousarray(x32, np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()


class Fp8Problem:
    def __init__(self, B, H, Hkv, T, D, seed, layout="bhtd"):
        rng = np.random.default_rng(seed)
        self.B, self.H, self.Hkv, self.T, self.D = B, H, Hkv, T, D
        self.q_bits = round_to_storage(rng.standard_normal((B, H, D), dtype=np.float32), "bf16")
        self.k_bits = to_e4m3_bits(rng.standard_normal((B, Hkv, T, D), dtype=np.float32))
        self.v_bits = to_e4m3_bits(rng.standard_normal((B, Hkv, T, D), dtype=np.float32))
        self.q = torch.from_numpy(self.q_bits.view(np.int16)).view(torch.bfloat16).to(DEV)
        k = torch.from_numpy(self.k_bits).view(torch.float8_e4m3fn)
        v = torch.from_numpy(self.v_bits).view(torch.float8_e4m3fn)
        if layout == "bthd":
            self.k = k.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
            self.v = v.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
        else:
            self.k, self.v = k.to(DEV), v.to(DEV)

    def oracle_kv(self):
        g = self.H // self.Hkv
        return np.repeat(self.k_bits, g, axis=1), np.repeat(self.v_bits, g, axis=1)


@pytest.mark.parametrize("H,Hkv,D,layout,out_dtype", [
    (4, 4, 128, "bhtd", torch.float32), (3, 3, 64, "bthd", torch.float32), (8, 2, 128, "bhtd", torch.bfloat16),
    (2, 2, 128, "bthd", torch.bfloat16)])
def test_sparse_dense_and_span_calls_against_the_oracle(H, Hkv, D, layout, out_dtype):
    B, T = 3, 2000
    p = Fp8Problem(B, H, Hkv, T, D, seed=11 * H + D, layout=layout)
    ctx = [2000, 1333, 300]
    spans = [[(0, 64), (700, 1500), (1990, 2000)], [(5, 9), (100, 130), (1300, 1333), (128, 140)], [(17, 18)]]
    counts, index = [], np.full((B, 1024), -1, np.int32)
    for b in range(B):
        idx = O.spans_to_index(spans[b], ctx[b])
        index[b, :len(idx)] = idx
        counts.append(len(idx))
    d_idx, d_cnt = torch.from_numpy(index).to(DEV), torch.tensor(counts, dtype=torch.int32, device=DEV)
    d_ctx = torch.tensor(ctx, dtype=torch.int32, device=DEV)
    out = torch.full((B, H, D), 7.0, dtype=out_dtype, device=DEV)
    lse = torch.full((B, H), 7.0, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    assert desc.kv_dtype == ssa.FP8_E4M3
    ws = torch.empty(max(ssa.decode_workspace_bytes(desc, T), ssa.decode_spans_workspace_bytes(desc, 1024, 8)),
                     dtype=torch.uint8, device=DEV)
    ko, vo = p.oracle_kv()
    native = out_dtype != torch.float32
    scale = 1 / np.sqrt(D)
    ref, ref_lse = O.decode_attn_sparse(p.q_bits, ko, vo, ctx, index, counts, scale, "bf16/e4m3")

    ssa.decode_attn_sparse(desc, p.q, p.k, p.v, d_ctx, d_idx, d_cnt, 1024, out, lse, ws, status)
    torch.cuda.synchronize()
    assert_parity(out.double().cpu().numpy(), ref, native, "index lists over an 8-bit cache")
    np.testing.assert_allclose(lse.double().cpu().numpy(), ref_lse, rtol=1e-5, atol=1e-5)

    out.fill_(7.0)
    offs = torch.tensor(np.cumsum([0] + [len(s) for s in spans]), dtype=torch.int32, device=DEV)
    flat = torch.tensor([x for s in spans for x in s], dtype=torch.int32, device=DEV)
    ssa.decode_attn_spans(desc, p.q, p.k, p.v, d_ctx, offs, flat, 4, 1024, out, lse, None, None, ws, status)
    torch.cuda.synchronize()
    assert_parity(out.double().cpu().numpy(), ref, native, "span lists over an 8-bit cache")

    ssa.decode_attn_dense(desc, p.q, p.k, p.v, d_ctx, out, lse, ws, status)
    torch.cuda.synchronize()
    refd, refd_lse = O.decode_attn_dense(p.q_bits, ko, vo, ctx, scale, "bf16/e4m3")
    assert_parity(out.double().cpu().numpy(), refd, native, "full context over an 8-bit cache")
    np.testing.assert_allclose(lse.double().cpu().numpy(), refd_lse, rtol=1e-5, atol=1e-5)
    assert int(status.item()) == 0


def test_every_e4m3_pattern_is_read_exactly():
    """One selected row per head holding all finite patterns: the output row is that V row, exactly."""
    B, H, T, D = 1, 2, 32, 128
    p = Fp8Problem(B, H, H, T, D, seed=1)
    pats = np.array([x for x in range(256) if x not in (0x7F, 0xFF)], np.uint8)
    v = p.v_bits.copy()
    v[0, 0, 5], v[0, 1, 5] = pats[:128], pats[126:254]
    p.v = torch.from_numpy(v).view(torch.float8_e4m3fn).to(DEV)
    out = torch.zeros((B, H, D), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    ws = torch.empty(ssa.decode_workspace_bytes(desc, 32), dtype=torch.uint8, device=DEV)
    idx = torch.full((1, 32), 5, dtype=torch.int32, device=DEV)
    ssa.decode_attn_sparse(desc, p.q, p.k, p.v, torch.tensor([T], dtype=torch.int32, device=DEV), idx,
                           torch.tensor([1], dtype=torch.int32, device=DEV), 32, out, None, ws, None)
    torch.cuda.synchronize()
    want = O.decode_e4m3(v[0, :, 5])
    assert np.array_equal(out.double().cpu().numpy()[0], want)


def test_descriptor_checks():
    p = Fp8Problem(1, 2, 2, 64, 128, seed=2)
    out16 = torch.zeros((1, 2, 128), dtype=torch.float16, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out16)                  # fp16 output with an 8-bit cache: not offered
    assert ssa.decode_workspace_bytes(desc, 64) == 0
    out = torch.zeros((1, 2, 128), dtype=torch.float32, device=DEV)
    desc = ssa.make_desc(p.q, p.k, p.v, out)
    assert ssa.decode_workspace_bytes(desc, 64) > 0
    desc.k_stride_t = 136                                       # 136 bytes: not a multiple of 16
    assert ssa.decode_workspace_bytes(desc, 64) == 0
