"""ctypes binding of libgdn_tail_replay.so: argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libgdn_tail_replay.so")
_lib = None

GDN_OK = 0
GDN_F32, GDN_BF16 = 0, 1
GDN_MEM_DEVICE, GDN_MEM_HOST = 0, 1
GDN_KERNEL_AUTO, GDN_KERNEL_FP32_SIMT, GDN_KERNEL_TCGEN05 = 0, 1, 2
GDN_INPUT_READY, GDN_INPUT_RAW = 0, 1


class GdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


class GdnDesc(ctypes.Structure):
    """Mirror of ``struct gdn_desc`` in include/gdn_tail_replay.h."""
    _fields_ = [
        ("num_qk_heads", ctypes.c_int32), ("num_v_heads", ctypes.c_int32),
        ("head_k_dim", ctypes.c_int32), ("head_v_dim", ctypes.c_int32),
        ("io_dtype", ctypes.c_int32), ("num_seqs", ctypes.c_int32),
        ("total_tokens", ctypes.c_int64),
        ("memory", ctypes.c_int32), ("kernel", ctypes.c_int32),
        ("input_stage", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("init_state", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
        ("status_word", ctypes.c_void_p), ("stream", ctypes.c_void_p),
    ]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load the CUDA library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            "libgdn_tail_replay.so is missing at %s: build it with "
            "`python -m paper_2608_30310_b200.build` (nvcc, sm_100a). There is no CPU fallback." % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    vp, dp = ctypes.c_void_p, ctypes.POINTER(GdnDesc)
    fwd_args = [dp, vp, vp, vp, vp, vp, vp, ctypes.c_int32, vp, vp]
    lib.gdn_workspace_size.restype = ctypes.c_size_t
    lib.gdn_workspace_size.argtypes = [dp]
    for name in ("gdn_tail_replay", "gdn_full_prefill", "gdn_tail_replay_static_scratch"):
        fn = getattr(lib, name)
        fn.restype = ctypes.c_int32
        fn.argtypes = fwd_args
    lib.gdn_decode_step.restype = ctypes.c_int32
    lib.gdn_decode_step.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.tail_select.restype = ctypes.c_int64
    lib.tail_select.argtypes = [ctypes.c_int64, ctypes.c_double]
    lib.gdn_status_string.restype = ctypes.c_char_p
    lib.gdn_status_string.argtypes = [ctypes.c_int32]
    lib.gdn_last_launch_count.restype = ctypes.c_int32
    lib.gdn_last_launch_count.argtypes = []
    lib.gdn_test_hooks.restype = None
    lib.gdn_test_hooks.argtypes = [ctypes.c_uint64, ctypes.c_int32]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().gdn_status_string(int(status)).decode()


def tail_select(prefix_len: int, budget_frac: float) -> int:
    """k = ceil(budget_frac * prefix_len); the replay window is rows [prefix_len - k, prefix_len)."""
    return int(load_library().tail_select(int(prefix_len), float(budget_frac)))


def last_launch_count() -> int:
    return int(load_library().gdn_last_launch_count())


def test_hooks(wait_timeout_ns: int = 0, skip_kq_load_of_chunk: int = -1) -> None:
    """Testing aid: bound of the device-side waits and an optional K/Q tile copy to leave out (see the header)."""
    load_library().gdn_test_hooks(int(wait_timeout_ns), int(skip_kq_load_of_chunk))


def workspace_size(desc: GdnDesc) -> int:
    return int(load_library().gdn_workspace_size(ctypes.byref(desc)))


class Workspace:
    """A caller-owned device scratch buffer (a torch uint8 tensor), grown on demand."""

    def __init__(self, device="cuda"):
        self.device = device
        self.buf = None

    def ensure(self, nbytes: int):
        import torch
        if self.buf is None or self.buf.numel() < nbytes:
            self.buf = torch.empty(max(int(nbytes), 256) + 256, dtype=torch.uint8, device=self.device)
        base = self.buf.data_ptr()
        off = (-base) % 256
        return base + off, self.buf.numel() - off


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _forward(fn_name, q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, *, total_tokens=None,
             init_state=None, workspace: Optional[Workspace] = None, status_word=None,
             kernel: int = GDN_KERNEL_AUTO, stream=None, check: bool = True, raw_inputs: bool = False) -> int:
    import torch
    lib = load_library()
    host = not q.is_cuda
    T, Hq, dk = q.shape
    Tv, Hv, dv = v.shape
    N = cu_tail_lens.numel() - 1
    if q.dtype == torch.bfloat16:
        io = GDN_BF16
    elif q.dtype == torch.float32:
        io = GDN_F32
    else:
        raise TypeError("q, k, v must be bfloat16 or float32")
    for name, t, dt in (("k", k, q.dtype), ("v", v, q.dtype), ("g", g, torch.float32),
                        ("beta", beta, torch.float32), ("cu_tail_lens", cu_tail_lens, torch.int32)):
        if t.dtype != dt:
            raise TypeError("%s has dtype %s, expected %s" % (name, t.dtype, dt))
    for name, t in (("q", q), ("k", k), ("v", v), ("g", g), ("beta", beta), ("cu_tail_lens", cu_tail_lens),
                    ("out_o", out_o), ("out_state", out_state), ("init_state", init_state)):
        if t is not None and (not t.is_contiguous() or t.is_cuda == host):
            raise ValueError("%s must be contiguous and on the same side (host/device) as q" % name)
    if k.shape != q.shape or Tv != T or tuple(g.shape) != (T, Hv) or tuple(beta.shape) != (T, Hv):
        raise ValueError("inconsistent input shapes")
    if out_o is not None and (tuple(out_o.shape) != (T, Hv, dv) or out_o.dtype != q.dtype):
        raise ValueError("out_o must be [T, Hv, dv] in the io dtype")
    if out_state is not None and (tuple(out_state.shape) != (N, Hv, dk, dv) or out_state.dtype != torch.float32):
        raise ValueError("out_state must be [N, Hv, dk, dv] fp32")
    desc = GdnDesc()
    desc.num_qk_heads, desc.num_v_heads, desc.head_k_dim, desc.head_v_dim = Hq, Hv, dk, dv
    desc.io_dtype, desc.num_seqs = io, N
    desc.total_tokens = T if total_tokens is None else int(total_tokens)
    desc.memory = GDN_MEM_HOST if host else GDN_MEM_DEVICE
    desc.kernel = kernel
    desc.input_stage = GDN_INPUT_RAW if raw_inputs else GDN_INPUT_READY
    desc.init_state = _ptr(init_state)
    if fn_name == "gdn_tail_replay_static_scratch":
        desc.workspace, desc.workspace_bytes = None, 0          # ignored: the library's built-in scratch is used
    else:
        need = int(lib.gdn_workspace_size(ctypes.byref(desc)))
        if workspace is None:
            workspace = Workspace(device="cuda" if host else q.device)
        desc.workspace, desc.workspace_bytes = workspace.ensure(need)
    desc.status_word = _ptr(status_word)
    if stream is None:
        stream = torch.cuda.current_stream()
    desc.stream = int(stream.cuda_stream)
    rc = int(getattr(lib, fn_name)(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta),
                                   _ptr(cu_tail_lens), int(chunk), _ptr(out_o), _ptr(out_state)))
    if check and rc != GDN_OK:
        raise GdnError(rc, fn_name)
    return rc


def gdn_tail_replay(q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw) -> int:
    """Tail replay (paper Eq. 2) on torch tensors; see include/gdn_tail_replay.h for layouts.

    All tensors on the GPU (device call) or all on the host (host call: the library stages
    through its workspace and copies results back on the stream).  Asynchronous on the current
    (or given) stream.  Keyword arguments: init_state, workspace, status_word, kernel, stream,
    check, raw_inputs (q, k, g, beta are raw projection outputs: the fused input stage of the header).
    """
    return _forward("gdn_tail_replay", q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw)


def gdn_tail_replay_static_scratch(q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw) -> int:
    """``gdn_tail_replay`` for callers with no device memory to spare: the scheduler scratch comes from an
    array built into the library instead of a workspace, and the call allocates nothing (this binding passes
    no workspace and creates no tensor).  Device tensors only, at most 4096 requests per call, and calls
    must not overlap on the GPU because they all share that one array.  Make the first call on a device
    outside any stream capture: it looks up the array's address once."""
    return _forward("gdn_tail_replay_static_scratch", q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw)


def gdn_full_prefill(q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw) -> int:
    """Full prefill (paper Eq. 1 over whole prefixes); same arguments as ``gdn_tail_replay``."""
    return _forward("gdn_full_prefill", q, k, v, g, beta, cu_tail_lens, chunk, out_o, out_state, **kw)


def gdn_decode_step(q, k, v, g, beta, state_in, out_o, state_out, *, stream=None, check: bool = True) -> int:
    """One token per request from a given state (Eq. 1 continued after the replay); see the header.

    q, k [N, Hq, dk], v [N, Hv, dv], g, beta [N, Hv], state_in / state_out [N, Hv, dk, dv] fp32 (may be the
    same tensor), out_o [N, Hv, dv] or None.  Device tensors only."""
    import torch
    lib = load_library()
    N, Hq, dk = q.shape
    _, Hv, dv = v.shape
    if q.dtype == torch.bfloat16:
        io = GDN_BF16
    elif q.dtype == torch.float32:
        io = GDN_F32
    else:
        raise TypeError("q, k, v must be bfloat16 or float32")
    for name, t, shape, dt in (("k", k, (N, Hq, dk), q.dtype), ("v", v, (N, Hv, dv), q.dtype), ("g", g, (N, Hv), torch.float32),
                               ("beta", beta, (N, Hv), torch.float32), ("state_in", state_in, (N, Hv, dk, dv), torch.float32),
                               ("state_out", state_out, (N, Hv, dk, dv), torch.float32)):
        if tuple(t.shape) != shape or t.dtype != dt or not t.is_contiguous() or not t.is_cuda:
            raise ValueError("%s must be a contiguous device tensor of shape %s and dtype %s" % (name, shape, dt))
    if out_o is not None and (tuple(out_o.shape) != (N, Hv, dv) or out_o.dtype != q.dtype or not out_o.is_cuda):
        raise ValueError("out_o must be [N, Hv, dv] in the io dtype on the device")
    desc = GdnDesc()
    desc.num_qk_heads, desc.num_v_heads, desc.head_k_dim, desc.head_v_dim = Hq, Hv, dk, dv
    desc.io_dtype, desc.num_seqs, desc.total_tokens = io, N, N
    desc.memory, desc.kernel = GDN_MEM_DEVICE, GDN_KERNEL_AUTO
    if stream is None:
        stream = torch.cuda.current_stream()
    desc.stream = int(stream.cuda_stream)
    rc = int(lib.gdn_decode_step(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(state_in),
                                 _ptr(out_o), _ptr(state_out)))
    if check and rc != GDN_OK:
        raise GdnError(rc, "gdn_decode_step")
    return rc
