"""Host-side checks of the C ABI that need no GPU: the library loads, exports what the header
declares, the ctypes mirrors match the C structs, and every argument error is reported by
status before anything is launched (none of these calls reaches a CUDA launch).
"""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import paper_2410_06577_b200 as rd
from paper_2410_06577_b200 import build as rd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "rodimus_ddts.h")


@pytest.fixture(scope="module")
def lib():
    rd_build.build()
    return rd.load_library()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rodimus_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert set(names) == set(rd.EXPORTED_SYMBOLS)
    for name in names:
        assert hasattr(lib, name), name


def test_struct_layout_matches_header(tmp_path):
    src = tmp_path / "sz.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "rodimus_ddts.h"\n'
        "int main(void){printf(\"%zu %zu %zu %zu %zu %zu\\n\", sizeof(rodimus_ddts_fwd_params),"
        " offsetof(rodimus_ddts_fwd_params,q), offsetof(rodimus_ddts_fwd_params,stream),"
        " sizeof(rodimus_ddts_step_params), offsetof(rodimus_ddts_step_params,q),"
        " offsetof(rodimus_ddts_step_params,stream));"
        "printf(\"%zu %zu %zu %zu\\n\", sizeof(rodimus_ddts_bwd_params),"
        " offsetof(rodimus_ddts_bwd_params,q), offsetof(rodimus_ddts_bwd_params,d_s0),"
        " offsetof(rodimus_ddts_bwd_params,stream));"
        "printf(\"%zu %zu %zu\\n\", sizeof(rodimus_swska_fwd_params),"
        " offsetof(rodimus_swska_fwd_params,q), offsetof(rodimus_swska_fwd_params,stream));return 0;}\n")
    exe = tmp_path / "sz"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    got = [int(t) for t in out]
    want = [ctypes.sizeof(rd.FwdParams), rd.FwdParams.q.offset, rd.FwdParams.stream.offset,
            ctypes.sizeof(rd.StepParams), rd.StepParams.q.offset, rd.StepParams.stream.offset,
            ctypes.sizeof(rd.BwdParams), rd.BwdParams.q.offset, rd.BwdParams.d_s0.offset,
            rd.BwdParams.stream.offset,
            ctypes.sizeof(rd.SwskaParams), rd.SwskaParams.q.offset, rd.SwskaParams.stream.offset]
    assert got == want


def test_version_and_status_strings(lib):
    assert rd.version() >= 100
    seen = {rd.status_str(s) for s in range(10)}
    assert len(seen) == 10 and "unknown status" not in seen
    assert rd.status_str(12345) == "unknown status"


FAKE = 0x7F0000001000  # 16-byte aligned address that is never dereferenced: every call below
                       # is rejected by the host checks first


def _fwd(**kw):
    p = rd.FwdParams()
    p.struct_size = ctypes.sizeof(rd.FwdParams)
    p.dtype, p.ingate = rd.BF16, rd.INGATE_POW_G
    p.B, p.H, p.T, p.dk, p.dv = 2, 2, 64, 128, 256
    p.scale = 1.0
    for name in ("q", "k", "gate_x", "temp_y", "v", "o"):
        setattr(p, name, FAKE)
    p.workspace = 0
    p.workspace_bytes = 0
    for key, val in kw.items():
        setattr(p, key, val)
    return p


def test_fwd_argument_errors(lib):
    assert lib.rodimus_ddts_fwd(None) == rd.ERR_NULL
    assert rd.fwd_raw(_fwd(struct_size=8)) == rd.ERR_DTYPE
    assert rd.fwd_raw(_fwd(dtype=7)) == rd.ERR_DTYPE
    assert rd.fwd_raw(_fwd(ingate=2)) == rd.ERR_DTYPE
    assert rd.fwd_raw(_fwd(T=-1)) == rd.ERR_SHAPE
    assert rd.fwd_raw(_fwd(dk=120)) == rd.ERR_UNSUPPORTED
    assert rd.fwd_raw(_fwd(dk=512)) == rd.ERR_UNSUPPORTED
    assert rd.fwd_raw(_fwd(dv=0)) == rd.ERR_SHAPE
    assert rd.fwd_raw(_fwd(B=1 << 15, H=1 << 10, T=1 << 10)) == rd.ERR_SHAPE
    assert rd.fwd_raw(_fwd(q=0)) == rd.ERR_NULL
    assert rd.fwd_raw(_fwd(o=0)) == rd.ERR_NULL
    assert rd.fwd_raw(_fwd(k=FAKE + 2)) == rd.ERR_ALIGN
    assert rd.fwd_raw(_fwd(s0=FAKE + 8)) == rd.ERR_ALIGN
    assert rd.fwd_raw(_fwd()) == rd.ERR_WORKSPACE                       # no workspace
    assert rd.fwd_raw(_fwd(workspace=FAKE, workspace_bytes=16)) == rd.ERR_WORKSPACE
    assert rd.fwd_raw(_fwd(workspace=FAKE + 16, workspace_bytes=4096)) == rd.ERR_ALIGN
    # varlen: B must be 1, host copy is checked before launch
    cu = np.array([0, 10, 5, 64], dtype=np.int32)
    cup = cu.ctypes.data
    assert rd.fwd_raw(_fwd(cu_seqlens=FAKE, N=3)) == rd.ERR_SHAPE        # B = 2
    bad = _fwd(B=1, cu_seqlens=FAKE, cu_seqlens_host=cup, N=3, workspace=FAKE - 0x1000 + 0x1000,
               workspace_bytes=4096)
    bad.workspace = 0x7F0000002000
    assert rd.fwd_raw(bad) == rd.ERR_SEQLENS
    cu2 = np.array([0, 10, 20, 63], dtype=np.int32)                      # does not end at T
    bad.cu_seqlens_host = cu2.ctypes.data
    assert rd.fwd_raw(bad) == rd.ERR_SEQLENS
    cu3 = np.array([1, 10, 20, 64], dtype=np.int32)                      # does not start at 0
    bad.cu_seqlens_host = cu3.ctypes.data
    assert rd.fwd_raw(bad) == rd.ERR_SEQLENS
    assert rd.fwd_raw(_fwd(cu_seqlens_host=cup)) == rd.ERR_NULL          # host copy alone
    # empty problem: accepted, nothing launched
    ok = _fwd(B=0, workspace=0x7F0000002000, workspace_bytes=4096)
    assert rd.fwd_raw(ok) == rd.OK and rd.last_launch_count() == 0


def test_workspace_bytes_and_kernel_choice(lib):
    p = _fwd()
    assert rd.fwd_workspace_bytes(p) == 256
    pv = _fwd(B=1, cu_seqlens=FAKE, N=100)
    assert rd.fwd_workspace_bytes(pv) == 256 + 512
    assert rd.fwd_workspace_bytes(_fwd(dk=7)) == 0
    assert rd.fwd_kernel_name(_fwd(dk=7)) == "invalid"
    assert rd.fwd_kernel_name(_fwd(dtype=rd.F32)) == "simt"
    assert rd.fwd_kernel_name(_fwd(dk=64)) == "simt"
    assert rd.fwd_kernel_name(_fwd()) in ("tcgen05", "simt")


def _step(**kw):
    p = rd.StepParams()
    p.struct_size = ctypes.sizeof(rd.StepParams)
    p.dtype, p.ingate = rd.BF16, rd.INGATE_POW_G
    p.Nseq, p.H, p.dk, p.dv = 4, 2, 128, 256
    p.scale = 1.0
    for name in ("q", "k", "gate_x", "temp_y", "v", "o", "state"):
        setattr(p, name, FAKE)
    for key, val in kw.items():
        setattr(p, key, val)
    return p


def test_step_argument_errors(lib):
    assert lib.rodimus_ddts_step(None) == rd.ERR_NULL
    assert rd.step_raw(_step(struct_size=4)) == rd.ERR_DTYPE
    assert rd.step_raw(_step(dtype=-1)) == rd.ERR_DTYPE
    assert rd.step_raw(_step(ingate=9)) == rd.ERR_DTYPE
    assert rd.step_raw(_step(Nseq=-3)) == rd.ERR_SHAPE
    assert rd.step_raw(_step(dk=100)) == rd.ERR_UNSUPPORTED
    assert rd.step_raw(_step(dv=2048)) == rd.ERR_UNSUPPORTED
    assert rd.step_raw(_step(state=0)) == rd.ERR_NULL
    assert rd.step_raw(_step(v=FAKE + 4)) == rd.ERR_ALIGN
    assert rd.step_raw(_step(Nseq=0)) == rd.OK and rd.last_launch_count() == 0


def _bwd(**kw):
    p = rd.BwdParams()
    p.struct_size = ctypes.sizeof(rd.BwdParams)
    p.dtype, p.ingate = rd.BF16, rd.INGATE_POW_G
    p.B, p.H, p.T, p.dk, p.dv = 2, 2, 64, 128, 256
    p.scale = 1.0
    for name in ("q", "k", "gate_x", "temp_y", "v", "d_o", "d_q", "d_k", "d_gate_x", "d_temp_y",
                 "d_v"):
        setattr(p, name, FAKE)
    p.workspace = 0
    p.workspace_bytes = 0
    for key, val in kw.items():
        setattr(p, key, val)
    return p


def test_bwd_argument_errors_and_workspace_size(lib):
    assert lib.rodimus_ddts_bwd(None) == rd.ERR_NULL
    assert rd.bwd_raw(_bwd(struct_size=8)) == rd.ERR_DTYPE
    assert rd.bwd_raw(_bwd(dtype=5)) == rd.ERR_DTYPE
    assert rd.bwd_raw(_bwd(ingate=2)) == rd.ERR_DTYPE
    assert rd.bwd_raw(_bwd(T=-1)) == rd.ERR_SHAPE
    assert rd.bwd_raw(_bwd(dk=64)) == rd.ERR_UNSUPPORTED      # widths the kernel is not built for
    assert rd.bwd_raw(_bwd(dv=128)) == rd.ERR_UNSUPPORTED
    assert rd.bwd_raw(_bwd(d_o=0)) == rd.ERR_NULL
    assert rd.bwd_raw(_bwd(d_v=0)) == rd.ERR_NULL
    assert rd.bwd_raw(_bwd(d_k=FAKE + 4)) == rd.ERR_ALIGN
    assert rd.bwd_raw(_bwd(d_sT=FAKE + 8)) == rd.ERR_ALIGN
    assert rd.bwd_raw(_bwd()) == rd.ERR_WORKSPACE
    # header + two fp32 scratch rows of dk per token and head + one per (sequence, head)
    # + six 64 x 256 fp32 state slices per (sequence, head) and their flags (a multiple of 256 bytes)
    want = 256 + 4 * (2 * 2 * 2 * 64 * 128 + 2 * 2 * 128) + 2 * 2 * 6 * 65536 + 256
    assert rd.bwd_workspace_bytes(_bwd()) == want
    assert rd.bwd_raw(_bwd(workspace=0x7F0000002000, workspace_bytes=want - 256)) == rd.ERR_WORKSPACE
    assert rd.bwd_workspace_bytes(_bwd(dk=64)) == 0
    assert rd.bwd_raw(_bwd(cu_seqlens=FAKE, N=3)) == rd.ERR_SHAPE       # packed needs B = 1
    cu = np.array([0, 10, 5, 64], dtype=np.int32)
    pv = _bwd(B=1, cu_seqlens=FAKE, cu_seqlens_host=cu.ctypes.data, N=3)
    pv.workspace, pv.workspace_bytes = 0x7F0000002000, rd.bwd_workspace_bytes(pv)
    assert pv.workspace_bytes == 256 + 256 + 4 * (2 * 2 * 64 * 128 + 3 * 2 * 128) + 3 * 2 * 6 * 65536 + 256
    assert rd.bwd_raw(pv) == rd.ERR_SEQLENS
    ok = _bwd(B=0, workspace=0x7F0000002000, workspace_bytes=4096)
    assert rd.bwd_raw(ok) == rd.OK and rd.last_launch_count() == 0


def test_swska_argument_errors(lib):
    def mk(**kw):
        p = rd.SwskaParams()
        p.struct_size = ctypes.sizeof(rd.SwskaParams)
        p.dtype, p.B, p.H, p.T, p.d, p.window, p.scale = rd.BF16, 2, 2, 64, 128, 16, 0.1
        p.q = p.k = p.v = p.o = FAKE
        for key, val in kw.items():
            setattr(p, key, val)
        return p
    assert lib.rodimus_swska_fwd(None) == rd.ERR_NULL
    assert rd.swska_raw(mk(struct_size=4)) == rd.ERR_DTYPE
    assert rd.swska_raw(mk(dtype=3)) == rd.ERR_DTYPE
    assert rd.swska_raw(mk(window=0)) == rd.ERR_SHAPE
    assert rd.swska_raw(mk(T=-2)) == rd.ERR_SHAPE
    assert rd.swska_raw(mk(d=64)) == rd.ERR_UNSUPPORTED
    assert rd.swska_raw(mk(k=0)) == rd.ERR_NULL
    assert rd.swska_raw(mk(o=FAKE + 8)) == rd.ERR_ALIGN
    assert rd.swska_raw(mk(T=0)) == rd.OK and rd.last_launch_count() == 0


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(rd, "_lib", None)
    monkeypatch.setattr(rd, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        rd.load_library()


def test_noalloc_entry_point_argument_errors_need_no_device(lib):
    """The checks that come before the built-in scratch array is looked up."""
    h = ctypes.c_void_p(1)
    assert lib.rodimus_ddts_fwd_noalloc(None, ctypes.byref(h)) == rd.ERR_NULL and h.value is None
    p = _fwd(struct_size=8)
    assert rd.fwd_noalloc_raw(p) == (rd.ERR_DTYPE, None)
    p = _fwd(B=1, N=rd.NOALLOC_MAX_SEQS + 1, cu_seqlens=FAKE)
    assert rd.fwd_noalloc_raw(p) == (rd.ERR_WORKSPACE, None)
