"""The C ABI used from plain C: a C99 program (tests/c_client/ssa_client.c, gcc,
CUDA runtime for memory, no Python in the process) runs the three calls on a
small problem; its results are compared with the oracle here."""
import os
import shutil
import struct
import subprocess

import numpy as np
import pytest

from oracle import ssa_oracle as O
from paper_2404_09336_b200 import inputs, ssa

from parity import assert_parity

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CUDA = os.environ.get("CUDA_HOME", "/usr/local/cuda")


def build_client(tmp_path):
    gcc = shutil.which("gcc")
    if gcc is None or not os.path.exists(os.path.join(CUDA, "include", "cuda_runtime_api.h")):
        pytest.skip("gcc or the CUDA runtime headers are not installed")
    exe = str(tmp_path / "ssa_client")
    libdir = os.path.dirname(ssa.LIBRARY_PATH)
    cmd = [gcc, "-std=c99", "-Wall", "-Werror", "-O1", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(CUDA, "include"), os.path.join(ROOT, "tests", "c_client", "ssa_client.c"), "-o", exe,
           "-L", libdir, "-l:" + os.path.basename(ssa.LIBRARY_PATH), "-L", os.path.join(CUDA, "lib64"), "-lcudart",
           "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(CUDA, "lib64")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    return exe


@pytest.mark.parametrize("cfg,B,H", [(1, 2, 4), (2, 3, 4)])
def test_c_program_matches_the_oracle(tmp_path, cfg, B, H):
    exe = build_client(tmp_path)
    wl = inputs.make_config(cfg, B=B, H=H)
    k, v = wl.kv_bits()
    q = wl.q_bits()
    stride = (wl.selected_upper_bound() + 31) // 32 * 32
    spans = np.ascontiguousarray(wl.spans, dtype=np.int32)
    src, dst = tmp_path / "in.bin", tmp_path / "out.bin"
    with open(src, "wb") as f:
        f.write(struct.pack("<7i", wl.B, wl.H, wl.D, wl.max_ctx, 1 if wl.dtype == "bf16" else 0, stride, len(spans)))
        for a in (wl.ctx_lens.astype(np.int32), wl.span_offsets.astype(np.int32), spans, q, k, v):
            f.write(np.ascontiguousarray(a).tobytes())
    res = subprocess.run([exe, str(src), str(dst)], capture_output=True, text=True)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "kernels launched" in res.stdout
    raw = np.fromfile(dst, dtype=np.uint8)
    o = 0

    def take(n, dt):
        nonlocal o
        a = raw[o:o + n * np.dtype(dt).itemsize].view(dt)
        o += n * np.dtype(dt).itemsize
        return a

    nq = wl.B * wl.H * wl.D
    counts = take(wl.B, np.int32)
    index = take(wl.B * stride, np.int32).reshape(wl.B, stride)
    status = int(take(1, np.uint32)[0])
    out_sparse = take(nq, np.float32).reshape(wl.B, wl.H, wl.D)
    lse = take(wl.B * wl.H, np.float32).reshape(wl.B, wl.H)
    out_dense = take(nq, np.float32).reshape(wl.B, wl.H, wl.D)
    assert o == raw.size and status == 0
    want_index, want_counts, _ = O.spans_to_index_batch(wl.span_offsets, wl.spans, wl.ctx_lens, stride)
    assert counts.tolist() == want_counts.tolist()
    for b in range(wl.B):
        assert index[b, :counts[b]].tolist() == want_index[b, :counts[b]].tolist()
    scale = 1 / np.sqrt(wl.D)
    ref, ref_lse = O.decode_attn_sparse(q, k, v, wl.ctx_lens, want_index, want_counts, scale, wl.dtype)
    assert_parity(out_sparse.astype(np.float64), ref, False, "C client, sparse")
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-5, atol=1e-5)
    ref_d, _ = O.decode_attn_dense(q, k, v, wl.ctx_lens, scale, wl.dtype)
    assert_parity(out_dense.astype(np.float64), ref_d, False, "C client, dense")
