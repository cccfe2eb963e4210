"""A few decode steps of one workload, for use under a profiler.

    python -m paper_2404_09336_b200.profile_step --cfg 2 [--density 0.1] [--batch B] [--steps 5] [--dense]
                                                 [--heads H_kv --query-heads H]

Runs `steps` times: ssa_spans_to_index, ssa_decode_attn_sparse and (with
--dense) ssa_decode_attn_dense on one copy of the workload's KV cache, then
synchronises.  Nothing is timed here.
"""
from __future__ import annotations

import argparse

import torch

from . import inputs
from .runner import DecodeStep


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cfg", type=int, default=2)
    ap.add_argument("--density", type=float, default=None)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--dense", action="store_true")
    ap.add_argument("--layout", default="bhtd", choices=["bhtd", "bthd"])
    ap.add_argument("--heads", type=int, default=None, help="cache heads (default: the workload's)")
    ap.add_argument("--query-heads", type=int, default=None, help="query heads, a multiple of the cache heads")
    a = ap.parse_args()
    wl = inputs.make_config(a.cfg, density=a.density, B=a.batch, H=a.heads)
    ds = DecodeStep(wl, layout=a.layout, kv_copies=1, query_heads=a.query_heads)
    for _ in range(a.steps):
        ds.step()
        if a.dense:
            ds.attend_dense()
    torch.cuda.synchronize()
    print(f"{wl.name}: {a.steps} steps, status {int(ds.status.item())}, {ds.selected_bytes()} selected KV bytes per step")


if __name__ == "__main__":
    main()
