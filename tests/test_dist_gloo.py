"""The multi-process path on CPU (gloo, world size 2): the batch is sharded by
request with no exchange on the data path, every rank's shard reproduces its
part of the unsharded result, and the benchmark's reductions (time = max over
ranks, bytes = sum over ranks) behave."""
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
import numpy as np
import torch
import torch.distributed as dist
sys.path.insert(0, os.environ["SSA_ROOT"])
import bench
from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
wl = inputs.make_config(2, B=5, H=2)
mine = wl.shard(rank, world)
k, v = mine.kv_bits()
index, counts, _ = O.spans_to_index_batch(mine.span_offsets, mine.spans, mine.ctx_lens, 256)
out, _ = O.decode_attn_sparse(mine.q_bits(), k, v, mine.ctx_lens, index, counts, 1 / np.sqrt(wl.D), wl.dtype)
parts = [None] * world
dist.all_gather_object(parts, (mine.seq_ids.tolist(), out, int(counts.sum())))
timer = bench.Timer(torch, dist, world, device="cpu")
slowest = timer.max_over_ranks(10.0 + rank)
total = timer.total(int(counts.sum()) * mine.kv_bytes_per_token())
# ranks of a weak-scaling run draw different requests
other = inputs.make_config(2, B=5, H=2, first_id=1000 * rank)
first_ctx = [None] * world
dist.all_gather_object(first_ctx, other.ctx_lens.tolist())
if rank == 0:
    ids = sum((p[0] for p in parts), [])
    assert ids == list(range(wl.B)), ids
    full = np.concatenate([p[1] for p in parts])
    kf, vf = wl.kv_bits()
    fi, fc, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, 256)
    ref, _ = O.decode_attn_sparse(wl.q_bits(), kf, vf, wl.ctx_lens, fi, fc, 1 / np.sqrt(wl.D), wl.dtype)
    assert np.array_equal(full, ref)
    assert slowest == 10.0 + world - 1
    assert total == int(fc.sum()) * wl.kv_bytes_per_token()
    assert first_ctx[0] != first_ctx[1]
    print("GLOO_OK")
dist.barrier()
dist.destroy_process_group()
"""


def test_two_ranks_shard_the_batch(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), SSA_ROOT=ROOT, OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            o, _ = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            p.kill()
            o, _ = p.communicate()
        outs.append(o)
    assert all(p.returncode == 0 for p in procs), "\n".join(outs)
    assert "GLOO_OK" in outs[0]
