"""The C-ABI library loads, exports what include/ssa.h declares, and rejects
bad arguments on the host before anything is launched (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2404_09336_b200 import ssa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ssa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ssa_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_symbols()
    assert {"ssa_spans_to_index", "ssa_decode_attn_sparse", "ssa_decode_attn_dense",
            "ssa_decode_workspace_bytes"} <= set(names)
    raw = C.CDLL(ssa.LIBRARY_PATH)
    for n in names:
        assert hasattr(raw, n), n


def test_library_is_in_tree():
    assert os.path.dirname(ssa.LIBRARY_PATH) == os.path.join(ROOT, "paper_2404_09336_b200")


def test_version_and_strings():
    assert ssa.version() >= 100
    assert ssa.status_string(ssa.OK) == "ok"
    assert "aligned" in ssa.status_string(ssa.ERR_ALIGN)
    assert "unknown" in ssa.status_string(12345)


def good_desc():
    d = ssa.AttnDesc()
    d.B, d.H, d.H_kv, d.D, d.max_ctx = 2, 4, 4, 128, 512
    d.kv_dtype, d.out_dtype, d.scale = ssa.BF16, ssa.BF16, 0.0
    d.q_stride_b, d.q_stride_h = 4 * 128, 128
    d.k_stride_b, d.k_stride_h, d.k_stride_t = 4 * 512 * 128, 512 * 128, 128
    d.v_stride_b, d.v_stride_h, d.v_stride_t = 4 * 512 * 128, 512 * 128, 128
    d.o_stride_b, d.o_stride_h = 4 * 128, 128
    return d


def test_workspace_query():
    d = good_desc()
    small = ssa.decode_workspace_bytes(d, 64)
    full = ssa.decode_workspace_bytes(d, 512)
    assert 0 < small <= full
    assert full >= 2 * 4 * (512 // 256) * (128 * 4 + 8)
    d.D = 96
    assert ssa.decode_workspace_bytes(d, 64) == 0
    d = good_desc()
    assert ssa.decode_workspace_bytes(d, 0) == 0


P = C.c_void_p(0x1000)      # never dereferenced: validation fails first
NUL = None


def sparse(d, q=P, k=P, v=P, ctx=P, idx=P, stride=64, cnt=P, max_sel=64, out=P, ws=P, ws_bytes=1 << 30):
    return ssa.lib.ssa_decode_attn_sparse(C.byref(d), q, k, v, ctx, idx, stride, cnt, max_sel, out, NUL, ws,
                                          ws_bytes, NUL, NUL)


def test_sparse_rejects_bad_arguments_without_launching():
    before = ssa.launch_count()
    d = good_desc()
    assert ssa.lib.ssa_decode_attn_sparse(None, P, P, P, P, P, 64, P, 64, P, NUL, P, 1 << 30, NUL, NUL) == ssa.ERR_NULL
    assert sparse(d, q=NUL) == ssa.ERR_NULL
    assert sparse(d, idx=NUL) == ssa.ERR_NULL
    assert sparse(d, out=NUL) == ssa.ERR_NULL
    assert sparse(d, max_sel=65) == ssa.ERR_CAPACITY
    assert sparse(d, max_sel=0) == ssa.ERR_CAPACITY
    assert sparse(d, stride=0) == ssa.ERR_CAPACITY
    assert sparse(d, k=C.c_void_p(0x1008)) == ssa.ERR_ALIGN
    assert sparse(d, ws=NUL) == ssa.ERR_WORKSPACE
    assert sparse(d, ws_bytes=16) == ssa.ERR_WORKSPACE
    for field, val, err in [("D", 96, ssa.ERR_UNSUPPORTED), ("H_kv", 3, ssa.ERR_UNSUPPORTED),
                            ("kv_dtype", ssa.F32, ssa.ERR_DTYPE), ("out_dtype", ssa.F16, ssa.ERR_DTYPE),
                            ("k_stride_t", 132, ssa.ERR_ALIGN), ("B", 0, ssa.ERR_SHAPE),
                            ("max_ctx", 0, ssa.ERR_SHAPE), ("v_stride_h", -128, ssa.ERR_SHAPE)]:
        d = good_desc()
        setattr(d, field, val)
        assert sparse(d) == err, field
    assert ssa.launch_count() == before


def test_dense_and_index_reject_bad_arguments():
    before = ssa.launch_count()
    d = good_desc()
    f = ssa.lib.ssa_decode_attn_dense
    assert f(C.byref(d), P, P, P, NUL, P, NUL, P, 1 << 30, NUL, NUL) == ssa.ERR_NULL
    assert f(C.byref(d), P, P, P, P, P, NUL, P, 64, NUL, NUL) == ssa.ERR_WORKSPACE
    d.D = 32
    assert f(C.byref(d), P, P, P, P, P, NUL, P, 1 << 30, NUL, NUL) == ssa.ERR_UNSUPPORTED
    g = ssa.lib.ssa_spans_to_index
    assert g(NUL, P, P, 4, P, 64, P, NUL, NUL) == ssa.ERR_NULL
    assert g(P, P, P, 0, P, 64, P, NUL, NUL) == ssa.ERR_SHAPE
    assert g(P, P, P, 4, P, 0, P, NUL, NUL) == ssa.ERR_SHAPE
    assert g(P, C.c_void_p(0x1004), P, 4, P, 64, P, NUL, NUL) == ssa.ERR_ALIGN
    assert ssa.launch_count() == before


def test_error_raises_through_binding():
    with pytest.raises(ssa.SsaError) as e:
        ssa._check("ssa_decode_attn_sparse", ssa.ERR_WORKSPACE, True)
    assert "workspace" in str(e.value)


def test_step_rejects_bad_copy_requests_before_enqueuing_anything():
    d = good_desc()
    st = ssa.Step()
    assert ssa.lib.ssa_decode_step(None, C.byref(st), None) == ssa.ERR_NULL
    st.host_in, st.dev_in, st.in_bytes = 0x1000, None, 256
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_NULL         # a copy without a destination
    st.dev_in = 0x2000
    st.flags = 8
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_UNSUPPORTED  # unknown flag bit
    st.flags = ssa.STEP_ONE_KERNEL | ssa.STEP_TWO_KERNELS
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_UNSUPPORTED  # contradictory
    st.flags = ssa.STEP_COPY_BY_KERNEL
    st.host_in = 0x1008
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_ALIGN
    st.host_in, st.in_bytes = 0x1000, 250
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_ALIGN
    import numpy as np
    buf = np.zeros(4096 + 64, np.uint8)                                          # ordinary pageable memory
    addr = (buf.ctypes.data + 63) // 64 * 64
    st.host_in, st.in_bytes = addr, 256
    assert ssa.decode_step(d, st, stream=0, check=False) == ssa.ERR_UNSUPPORTED  # kernels cannot address it


def test_refs_to_index_rejects_bad_arguments():
    t = ssa.AnchorTables()
    for name, _ in t._fields_:
        setattr(t, name, 0x1000)
    call = lambda tab, B, index, stride, counts: ssa.lib.ssa_refs_to_index(
        C.byref(tab) if tab is not None else None, B, index, stride, counts, None, None)
    assert call(None, 1, 0x2000, 64, 0x3000) == ssa.ERR_NULL
    assert call(t, 1, None, 64, 0x3000) == ssa.ERR_NULL
    assert call(t, 0, 0x2000, 64, 0x3000) == ssa.ERR_SHAPE
    assert call(t, 70000, 0x2000, 64, 0x3000) == ssa.ERR_SHAPE
    assert call(t, 1, 0x2000, 0, 0x3000) == ssa.ERR_SHAPE
    t.refs = 0x1004
    assert call(t, 1, 0x2000, 64, 0x3000) == ssa.ERR_ALIGN
    t.refs, t.lines = 0x1000, None
    assert call(t, 1, 0x2000, 64, 0x3000) == ssa.ERR_NULL


def test_header_is_plain_c_and_cpp(tmp_path):
    # the boundary is a C ABI: the header must compile as C99 and as C++ with nothing but the standard headers
    import shutil
    import subprocess
    src = tmp_path / "use_ssa.c"
    src.write_text('#include "ssa.h"\n'
                   "int main(void) {\n"
                   "  ssa_attn_desc d; ssa_step s; ssa_anchor_tables t; ssa_paging p;\n"
                   "  (void)d; (void)s; (void)t; (void)p;\n"
                   "  return (int)(sizeof(ssa_step) == 0) + (SSA_MAX_SPANS_PER_SEQ != 2048);\n"
                   "}\n")
    inc = os.path.join(ROOT, "include")
    for cc, std in (("gcc", "-std=c99"), ("g++", "-std=c++11")):
        exe = shutil.which(cc)
        if exe is None:
            pytest.skip(f"{cc} not installed")
        args = [exe, std, "-Wall", "-Werror", "-pedantic", "-I", inc, "-fsyntax-only"]
        args += ["-x", "c++"] if cc == "g++" else []
        res = subprocess.run(args + [str(src)], capture_output=True, text=True)
        assert res.returncode == 0, res.stderr


def test_struct_layouts_of_the_binding_match_the_header(tmp_path):
    # sizes and a few offsets of the ctypes mirrors against what the C compiler lays out
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("gcc not installed")
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "ssa.h"\n'
                   "int main(void) {\n"
                   '  printf("%zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(ssa_attn_desc), sizeof(ssa_step),\n'
                   "         sizeof(ssa_anchor_tables), sizeof(ssa_paging), offsetof(ssa_attn_desc, scale),\n"
                   "         offsetof(ssa_step, flags), offsetof(ssa_step, host_in), offsetof(ssa_paging, n_pages));\n"
                   "  return 0;\n}\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    want = [C.sizeof(ssa.AttnDesc), C.sizeof(ssa.Step), C.sizeof(ssa.AnchorTables), C.sizeof(ssa.Paging),
            ssa.AttnDesc.scale.offset, ssa.Step.flags.offset, ssa.Step.host_in.offset, ssa.Paging.n_pages.offset]
    assert got == want
