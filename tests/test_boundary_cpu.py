"""CPU-side checks of the C-ABI boundary: the library loads, exports every symbol the header
declares, tail_select agrees with the oracle's exact-rational evaluation, and host-detectable
argument errors are reported before any GPU work (none of these needs a device)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2608_30310_b200 as gdn
from paper_2608_30310_b200 import _binding as B
from paper_2608_30310_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_library()
    return gdn.load_library()


def header_functions():
    text = open(os.path.join(ROOT, "include", "gdn_tail_replay.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return re.findall(r"GDN_API\s+[\w\s\*]+?\b(\w+)\s*\(", text)


def test_header_symbols_are_exported(lib):
    names = header_functions()
    assert {"gdn_tail_replay", "gdn_full_prefill", "tail_select", "gdn_workspace_size",
            "gdn_status_string", "gdn_last_launch_count"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_desc_layout_matches_header():
    # 6 int32, int64, 4 int32, 2 pointers, size_t, 2 pointers on LP64
    assert ctypes.sizeof(B.GdnDesc) == 6 * 4 + 8 + 4 * 4 + 8 + 8 + 8 + 8 + 8
    assert B.GdnDesc.total_tokens.offset == 24 and B.GdnDesc.input_stage.offset == 40
    assert B.GdnDesc.init_state.offset == 48 and B.GdnDesc.stream.offset == 80


def test_tail_select_matches_oracle_and_table(lib):
    for line in open(os.path.join(ROOT, "tests", "golden", "tail_select_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        m, r, k = line.split()
        assert gdn.tail_select(int(m), float(r)) == int(k), line
    for m in list(range(0, 300)) + [8192, 16384, 32768, 131072, 8225, 16418, 31366, 31847, 10 ** 6]:
        for pct in range(0, 101):
            assert gdn.tail_select(m, pct / 100.0) == oracle.tail_select(m, pct / 100.0), (m, pct)
    # exact at any size: a genuine fraction is never swallowed, an exact product never rounded up
    for m in (10 ** 7 + 1, 10 ** 9 + 7, 10 ** 12 + 1, 3 * 10 ** 15 + 11, 2 ** 62 + 1):
        for r in (0.05, 0.1, 0.07, 0.0333, 1e-9, 0.999999, 1e-300, 0.3):
            assert gdn.tail_select(m, r) == oracle.tail_select(m, r), (m, r)
    assert gdn.tail_select(-1, 0.1) == -1
    assert gdn.tail_select(5, -0.1) == -1
    assert gdn.tail_select(5, float("nan")) == -1
    assert gdn.tail_select(5, 2.0) == 5


def test_status_strings(lib):
    assert gdn.status_string(0) == "ok"
    for s in range(-5, 0):
        assert gdn.status_string(s) not in ("ok", "unknown status")
    assert gdn.status_string(-99) == "unknown status"


def _desc(**kw):
    d = B.GdnDesc()
    d.num_qk_heads, d.num_v_heads, d.head_k_dim, d.head_v_dim = 2, 4, 64, 64
    d.io_dtype, d.num_seqs, d.total_tokens = B.GDN_F32, 1, 16
    d.memory, d.kernel = B.GDN_MEM_DEVICE, B.GDN_KERNEL_AUTO
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def _call(lib, d, ptrs=None, chunk=64, fn="gdn_tail_replay"):
    buf = np.zeros(1 << 16, dtype=np.uint8)                 # never dereferenced: errors come first
    base = buf.ctypes.data + (-buf.ctypes.data) % 256
    p = [base] * 8 if ptrs is None else ptrs
    return getattr(lib, fn)(ctypes.byref(d), p[0], p[1], p[2], p[3], p[4], p[5], chunk, p[6], p[7]), buf


def test_host_detectable_errors_need_no_gpu(lib):
    assert lib.gdn_tail_replay(None, 1, 1, 1, 1, 1, 1, 64, 1, 1) == -1
    rc, _ = _call(lib, _desc(num_v_heads=3))
    assert rc == -1                                           # Hv not a multiple of Hq
    rc, _ = _call(lib, _desc(num_seqs=-1))
    assert rc == -1
    rc, _ = _call(lib, _desc(io_dtype=7))
    assert rc == -1
    rc, _ = _call(lib, _desc(head_k_dim=96))
    assert rc == -2                                           # unsupported head dim
    rc, _ = _call(lib, _desc(), chunk=32)
    assert rc == -2                                           # unsupported chunk
    rc, _ = _call(lib, _desc(kernel=B.GDN_KERNEL_TCGEN05))
    assert rc == -2                                           # tensor-core path needs bf16, d = 128
    rc, _ = _call(lib, _desc())
    assert rc == -3                                           # no workspace
    d = _desc()
    buf = np.zeros(4096, dtype=np.uint8)
    base = buf.ctypes.data + (-buf.ctypes.data) % 256
    d.workspace, d.workspace_bytes = base, 8
    rc, _ = _call(lib, d)
    assert rc == -3                                           # workspace too small
    rc, _ = _call(lib, _desc(), ptrs=[0] + [base] * 7)
    assert rc == -1                                           # null q
    rc, _ = _call(lib, _desc(), ptrs=[base + 4] + [base] * 7)
    assert rc == -1                                           # misaligned q
    for fn in ("gdn_tail_replay", "gdn_full_prefill"):
        rc, _ = _call(lib, _desc(num_seqs=0, total_tokens=0), fn=fn)
        assert rc == 0                                        # empty batch: nothing to do


def test_host_mode_checks_cu_before_any_copy(lib):
    d = _desc(memory=B.GDN_MEM_HOST, num_seqs=2, total_tokens=16)
    need = lib.gdn_workspace_size(ctypes.byref(d))
    assert need > 0
    buf = np.zeros(need + 512, dtype=np.uint8)
    base = buf.ctypes.data + (-buf.ctypes.data) % 256
    d.workspace, d.workspace_bytes = base, need
    cu = np.array([0, 10, 8, 0], dtype=np.int32)            # decreasing, and cu[N] != T
    data = np.zeros(1 << 16, dtype=np.uint8)
    dp = data.ctypes.data + (-data.ctypes.data) % 256
    rc = lib.gdn_tail_replay(ctypes.byref(d), dp, dp, dp, dp, dp, cu.ctypes.data, 64, dp, dp)
    assert rc == -1


def test_workspace_size(lib):
    d = _desc(num_seqs=32)
    dev = lib.gdn_workspace_size(ctypes.byref(d))
    assert dev >= 256 + 32 * 4 and dev % 256 == 0
    d.memory = B.GDN_MEM_HOST
    assert lib.gdn_workspace_size(ctypes.byref(d)) > dev
    assert lib.gdn_workspace_size(ctypes.byref(_desc(num_v_heads=3))) == 0
    assert lib.gdn_workspace_size(None) == 0
