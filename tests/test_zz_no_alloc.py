"""The no-allocation entry point, gdn_tail_replay_static_scratch, against the ordinary one.

Some callers of this library cannot give it a workspace: a serving process that has already handed all of
the GPU's memory to its own cache pool, or code that only receives raw device pointers from someone else's
allocator.  For them the library carries its scheduler scratch inside its own device image.  This test calls
that entry point through the C ABI, twice in a row on the same stream (the second call finds the array
filled by the first and must not be disturbed by it), and requires the same outputs and final states as
gdn_tail_replay with a caller-owned workspace, under the tolerances the other GPU tests use (the two are
in fact expected to agree bit for bit, since only the address of the scratch differs).  It also checks the
documented size limit.  The file sorts last on purpose: if it fails under -x, everything else has run.
"""
import ctypes

import numpy as np
import pytest

import oracle
from gdn_workloads import make_inputs
from gpu_utils import run_library, assert_parity, TOL, state_rel_fro

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("io,dk,kernel", [("bf16", 128, 0), ("f32", 64, 0)])
def test_static_scratch_matches_workspace_entry_twice(io, dk, kernel):
    lens_a = [130, 0, 65, 410, 7]
    lens_b = [64, 300, 1]                                  # second call: different batch, fewer requests
    for lens, seed in ((lens_a, 301), (lens_b, 302)):
        inp = make_inputs(lens, 2, 4, dk, dk, io, seed=seed)
        o_ref, st_ref, _ = run_library(inp, kernel=kernel, fn="gdn_tail_replay")
        o_new, st_new, launches = run_library(inp, kernel=kernel, fn="gdn_tail_replay_static_scratch")
        assert launches >= 2
        tol = TOL[io]
        assert np.isfinite(o_new).all() and np.isfinite(st_new).all()
        assert np.abs(o_new - o_ref).max() <= tol["o_max_abs"]
        assert state_rel_fro(st_new, st_ref)[0] <= tol["state_rel_fro"]
        np.testing.assert_array_equal(o_new, o_ref)        # same kernels, same order: bitwise equal
        np.testing.assert_array_equal(st_new, st_ref)
        ro, rst = oracle.gdn_forward_inputs(inp)             # and directly against the oracle
        assert_parity(inp, o_new, st_new, ro, rst)


def test_static_scratch_at_its_request_limit_and_with_one_request():
    """4,096 requests fill the built-in array to its last byte (the order list ends exactly there); a single
    request on the tensor-core path runs without the scheduler kernel, i.e. without touching the array."""
    lens = [(i * 7) % 4 for i in range(4096)]              # lengths 0..3
    inp = make_inputs(lens, 1, 2, 64, 64, "f32", seed=303)
    o_ref, st_ref, _ = run_library(inp, fn="gdn_tail_replay")
    o_new, st_new, _ = run_library(inp, fn="gdn_tail_replay_static_scratch")
    np.testing.assert_array_equal(o_new, o_ref)
    np.testing.assert_array_equal(st_new, st_ref)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o_new, st_new, ro, rst)
    one = make_inputs([200], 2, 4, 128, 128, "bf16", seed=304)
    o1, st1, launches = run_library(one, fn="gdn_tail_replay_static_scratch")
    assert launches == 1
    ro, rst = oracle.gdn_forward_inputs(one)
    assert_parity(one, o1, st1, ro, rst)


def test_static_scratch_rejects_oversize_and_host_memory():
    import paper_2608_30310_b200 as gdn
    from paper_2608_30310_b200 import _binding as B
    lib = gdn.load_library()
    d = B.GdnDesc()
    d.num_qk_heads, d.num_v_heads, d.head_k_dim, d.head_v_dim = 2, 4, 64, 64
    d.io_dtype, d.total_tokens, d.kernel = B.GDN_F32, 16, B.GDN_KERNEL_AUTO
    buf = np.zeros(4096, dtype=np.uint8)                   # never dereferenced: the checks come first
    p = buf.ctypes.data + (-buf.ctypes.data) % 256
    d.num_seqs, d.memory = 4097, B.GDN_MEM_DEVICE
    rc = lib.gdn_tail_replay_static_scratch(ctypes.byref(d), p, p, p, p, p, p, 64, p, p)
    assert rc == -6 and "built-in scratch" in gdn.status_string(rc)
    d.num_seqs, d.memory = 1, B.GDN_MEM_HOST
    rc = lib.gdn_tail_replay_static_scratch(ctypes.byref(d), p, p, p, p, p, p, 64, p, p)
    assert rc == -2
