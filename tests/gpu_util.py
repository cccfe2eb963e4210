"""Helpers of the GPU parity tests: run the C-ABI calls on hand-made inputs."""
import numpy as np
import torch

from paper_2404_09336_b200 import ssa
from paper_2404_09336_b200.inputs import round_to_storage
from paper_2404_09336_b200.runner import bits_to_tensor

DEV = "cuda:0"
TORCH_DT = {"bf16": torch.bfloat16, "f16": torch.float16}


def run_index(span_lists, ctx_lens, index_stride, fill=-7):
    """span_lists: per request a list of (start, end).  Returns index, counts, status."""
    B = len(span_lists)
    offs = np.zeros(B + 1, np.int32)
    offs[1:] = np.cumsum([len(s) for s in span_lists])
    flat = np.asarray([p for s in span_lists for p in s], np.int32).reshape(-1, 2)
    if len(flat) == 0:
        flat = np.zeros((1, 2), np.int32)
    d_off = torch.from_numpy(offs).to(DEV)
    d_sp = torch.from_numpy(flat).to(DEV)
    d_ctx = torch.tensor(ctx_lens, dtype=torch.int32, device=DEV)
    index = torch.full((B, index_stride), fill, dtype=torch.int32, device=DEV)
    counts = torch.full((B,), fill, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ssa.spans_to_index(d_off, d_sp, d_ctx, index, counts, status)
    torch.cuda.synchronize()
    return index.cpu().numpy(), counts.cpu().numpy(), int(status.item()), (offs, flat)


def random_bits(rng, shape, dtype):
    return round_to_storage(rng.standard_normal(shape, dtype=np.float32), dtype)


class Problem:
    """q[B,H,D], K/V[B,H,T,D] bit patterns on the host plus their device copies."""

    def __init__(self, B, H, T, D, dtype="bf16", seed=0, layout="bhtd"):
        rng = np.random.default_rng(seed)
        self.B, self.H, self.T, self.D, self.dtype = B, H, T, D, dtype
        self.q_bits = random_bits(rng, (B, H, D), dtype)
        self.k_bits = random_bits(rng, (B, H, T, D), dtype)
        self.v_bits = random_bits(rng, (B, H, T, D), dtype)
        self.layout = layout
        self.upload()

    def upload(self):
        self.q = bits_to_tensor(self.q_bits, self.dtype).to(DEV)
        k, v = bits_to_tensor(self.k_bits, self.dtype), bits_to_tensor(self.v_bits, self.dtype)
        if self.layout == "bthd":
            self.k = k.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
            self.v = v.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
        else:
            self.k, self.v = k.to(DEV), v.to(DEV)

    def sparse(self, ctx_lens, index, counts, max_selected=None, out_dtype=torch.float32, scale=0.0,
               check=True):
        B, H, D = self.B, self.H, self.D
        index = np.ascontiguousarray(index, dtype=np.int32)
        d_idx = torch.from_numpy(index).to(DEV)
        d_cnt = torch.tensor(counts, dtype=torch.int32, device=DEV)
        d_ctx = torch.tensor(ctx_lens, dtype=torch.int32, device=DEV)
        out = torch.full((B, H, D), 777.0, dtype=out_dtype or TORCH_DT[self.dtype], device=DEV)
        lse = torch.full((B, H), 777.0, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        desc = ssa.make_desc(self.q, self.k, self.v, out, scale=scale)
        ms = int(max_selected if max_selected is not None else index.shape[1])
        ws = torch.empty(max(ssa.decode_workspace_bytes(desc, ms), 16), dtype=torch.uint8, device=DEV)
        rc = ssa.decode_attn_sparse(desc, self.q, self.k, self.v, d_ctx, d_idx, d_cnt, ms, out, lse, ws,
                                    status, check=check)
        torch.cuda.synchronize()
        return (out.to(torch.float64).cpu().numpy(), lse.to(torch.float64).cpu().numpy(),
                int(status.item()), rc)

    def dense(self, ctx_lens, out_dtype=torch.float32, scale=0.0):
        B, H, D = self.B, self.H, self.D
        d_ctx = torch.tensor(ctx_lens, dtype=torch.int32, device=DEV)
        out = torch.full((B, H, D), 777.0, dtype=out_dtype or TORCH_DT[self.dtype], device=DEV)
        lse = torch.full((B, H), 777.0, dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        desc = ssa.make_desc(self.q, self.k, self.v, out, scale=scale)
        ws = torch.empty(ssa.decode_workspace_bytes(desc, self.T), dtype=torch.uint8, device=DEV)
        ssa.decode_attn_dense(desc, self.q, self.k, self.v, d_ctx, out, lse, ws, status)
        torch.cuda.synchronize()
        return out.to(torch.float64).cpu().numpy(), lse.to(torch.float64).cpu().numpy(), int(status.item())
