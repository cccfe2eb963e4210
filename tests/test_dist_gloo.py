"""The multi-process path on CPU (gloo, world size 2): the batch is sharded by
request with no exchange on the data path, every rank's shard reproduces its
part of the unsharded result, and the benchmark's reductions (time = max over
ranks, bytes = sum over ranks) behave."""
import json
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


def test_bench_starts_its_own_ranks_when_run_as_a_plain_script():
    """`python bench.py --gpus 2` without torchrun: the script re-launches itself as two ranks.  With
    SSA_BENCH_DRY_RUN=1 the ranks use gloo and a stand-in measurement (rank r: 10 + r ms for
    1000 * (r + 1) bytes per step), so the reductions can be checked: time = max, bytes = sum."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    env.update(SSA_BENCH_DRY_RUN="1", OMP_NUM_THREADS="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "20", "--warmup", "3"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout                         # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["steps"] == 20 and line["dry_run"] is True
    assert line["ms_per_step"] == 11.0 / 20                    # the slower rank's time
    assert abs(line["value"] - 3000.0 * 20 / 11e-3 / 1e9) < 1e-12   # both ranks' bytes


def test_clock_samples_between_the_first_and_last_region_count_as_under_load():
    """Timed regions are far shorter than nvidia-smi's sampling period; the record must not come out empty."""
    import bench
    assert bench.host_cores() >= 1
    rows = [(100.0 + 0.05 * i, "3996, 1965, 1965, 400.0, 0x0, Not Active, Not Active, Not Active, Active")
            for i in range(40)]
    # regions far shorter than the sampling period: every sample between the first and the last region counts
    windows = [(100.5 + 0.001 * i, 100.5005 + 0.001 * i) for i in range(500)]
    c = bench.summarize_clock_rows(rows, windows)
    assert c["samples"] == 40 and c["samples_under_load"] >= 10
    assert c["sm_mhz"] == 1965 and c["sm_max_mhz"] == 1965 and c["reasons"] == ["sw_power_cap"]
