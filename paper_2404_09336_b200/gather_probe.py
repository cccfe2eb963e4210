"""Gather micro-benchmark (bench.py --probe gather): the decode kernel's row gather alone, with per-lane
256-bit loads against bulk asynchronous copies (cp.async.bulk + mbarrier) into a shared-memory ring.

One launch gathers 36 864 stages of 32 rows x 256 bytes (302 MB, more than twice the L2) placed at random in a
2 GiB buffer; three different lists rotate between launches.  Lists are made of runs of 1, 4 or 32 consecutive
rows (256 B, 1 KB, 8 KB: single rows, the short spans of the arithmetic-style workload, long spans).  Timed with
CUDA events around back-to-back launches; every variant's checksum is compared with the plain-load one.
Single GPU only; no multicast; every copy reads this GPU's own memory.
"""
from __future__ import annotations

import ctypes as C
import json
import statistics

import numpy as np
import torch

from . import build as _build

ROW_BYTES, STAGE_ROWS = 256, 32


def _load():
    lib = C.CDLL(_build.build_probe())
    vp = C.c_void_p
    lib.ssa_probe_gather.restype = C.c_int
    lib.ssa_probe_gather.argtypes = [C.c_int, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp]
    return lib


def make_lists(n_rows_buf, n_stages, run_rows, seed):
    """int32 [n_stages * 32] row numbers: runs of run_rows consecutive rows at random places."""
    rng = np.random.default_rng(seed)
    n_runs = n_stages * STAGE_ROWS // run_rows
    starts = rng.integers(0, n_rows_buf // run_rows, size=n_runs, dtype=np.int64) * run_rows
    rows = (starts[:, None] + np.arange(run_rows)[None, :]).reshape(-1)
    return torch.from_numpy(rows.astype(np.int32))


def main():
    if not torch.cuda.is_available():
        raise SystemExit("the gather probe needs a CUDA device")
    lib = _load()
    dev = torch.device("cuda", 0)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    buf_bytes = 2 << 30
    buf = torch.empty(buf_bytes // 4, dtype=torch.int32, device=dev)
    buf.random_(0, 2 ** 31 - 1)
    n_rows_buf = buf_bytes // ROW_BYTES
    n_stages = 36864
    nbytes = n_stages * STAGE_ROWS * ROW_BYTES
    checksum = torch.zeros(1, dtype=torch.int32, device=dev)
    error = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def launch(mode, rows, grid, stages=1, run_rows=1):
        rc = lib.ssa_probe_gather(mode, buf.data_ptr(), rows.data_ptr(), n_stages, grid, stages, run_rows,
                                  checksum.data_ptr(), error.data_ptr(), stream)
        if rc != 0:
            raise RuntimeError(f"ssa_probe_gather refused the launch ({rc})")

    def timed(mode, lists, grid, stages=1, run_rows=1, n=12, reps=5):
        for r in lists:
            launch(mode, r, grid, stages, run_rows)
        out = []
        for _ in range(reps):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(n):
                launch(mode, lists[i % len(lists)], grid, stages, run_rows)
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / n * 1e3)
        return statistics.median(out)

    def checksum_of(mode, rows, grid, stages=1, run_rows=1):
        checksum.zero_()
        launch(mode, rows, grid, stages, run_rows)
        torch.cuda.synchronize()
        return int(checksum.item())

    results = []
    for run_rows in (1, 4, 32):
        lists = [make_lists(n_rows_buf, n_stages, run_rows, 100 * run_rows + s).to(dev) for s in range(3)]
        want = checksum_of(0, lists[0], sms * 8)
        for blocks_per_sm in (4, 8, 16):
            us = timed(0, lists, sms * blocks_per_sm)
            results.append({"run_bytes": run_rows * ROW_BYTES, "how": "256-bit loads", "blocks_per_sm": blocks_per_sm,
                            "in_flight_per_sm_kb": blocks_per_sm * 4 * 8, "us": round(us, 1),
                            "gbs": round(nbytes / us / 1e3)})
        for copy_rows in sorted({1, run_rows}):
            for blocks_per_sm, stages in ((1, 27), (2, 13), (4, 6), (8, 2), (8, 3), (16, 1)):
                got = checksum_of(1, lists[0], sms * blocks_per_sm, stages, copy_rows)
                if got != want or int(error.item()) != 0:
                    raise SystemExit(f"bulk-copy gather disagrees with the plain loads (run {run_rows}, copies of "
                                     f"{copy_rows} rows, {blocks_per_sm} blocks/SM): checksum {got:#x} vs {want:#x}, "
                                     f"error flag {int(error.item())}")
                us = timed(1, lists, sms * blocks_per_sm, stages, copy_rows)
                results.append({"run_bytes": run_rows * ROW_BYTES, "how": f"bulk copies of {copy_rows * ROW_BYTES} B",
                                "blocks_per_sm": blocks_per_sm, "in_flight_per_sm_kb": blocks_per_sm * stages * 8,
                                "us": round(us, 1), "gbs": round(nbytes / us / 1e3)})
        del lists
    if int(error.item()) != 0:
        raise SystemExit("a bounded wait expired in the bulk-copy gather")
    print("| run length | how | blocks/SM | KB in flight per SM | us per launch | GB/s |")
    print("|---|---|---|---|---|---|")
    for r in results:
        print(f"| {r['run_bytes']} B | {r['how']} | {r['blocks_per_sm']} | {r['in_flight_per_sm_kb']} | {r['us']} | {r['gbs']} |")
    print(json.dumps({"probe": "gather", "bytes_per_launch": nbytes, "rows": results}))


if __name__ == "__main__":
    main()
