"""CPU oracle for the GDN tail-replay path.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference legs may use
this package; the product never routes through it and shares no code with it.

* ``gdn_forward``  — fp64 token-by-token GDN recurrence (paper Eq. 1; Eq. 2 when started from
  zero on a tail), implemented in plain C in ``gdn_oracle.c`` and threaded over
  (request, v-head) chains only.
* ``tail_select``  — replay-window arithmetic k = ceil(r * m) (paper, Method section),
  evaluated in exact rational arithmetic.
* ``prologue``     — the input pipeline in front of the recurrence (L2-normalised q and k,
  sigmoid gate and beta from raw projection outputs; paper, Method section), plain numpy fp64;
  ``gdn_forward_f64`` runs the same recurrence on its fp64 results.

Every function is pinned by the CPU tests; none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from fractions import Fraction
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gdn_oracle.c")
_LIB = os.path.join(_HERE, "libgdn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no special flags: it is meant to be plain)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-pthread",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.gdn_oracle_forward.restype = ctypes.c_int
        lib.gdn_oracle_forward.argtypes = [fp, fp, fp, fp, fp, ip] + [ctypes.c_int32] * 5 + [dp, dp, dp, ctypes.c_int32]
        lib.gdn_oracle_forward_f64.restype = ctypes.c_int
        lib.gdn_oracle_forward_f64.argtypes = [dp, dp, dp, dp, dp, ip] + [ctypes.c_int32] * 5 + [dp, dp, dp, ctypes.c_int32]
        _lib = lib
    return _lib


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1))


def gdn_forward(q, k, v, g, beta, cu_tail_lens, init_state: Optional[np.ndarray] = None,
                threads: Optional[int] = None, want_o: bool = True
                ) -> Tuple[Optional[np.ndarray], np.ndarray]:
    """Run the recurrence over every request and v-head.

    q, k: [T, Hq, dk]; v: [T, Hv, dv]; g, beta: [T, Hv] (fp32 values, widened exactly to fp64
    inside); cu_tail_lens: [N+1].  ``init_state`` [N, Hv, dk, dv] fp64 or None for the zero
    start of Eq. 2.  Returns (o [T, Hv, dv] fp64 or None, state [N, Hv, dk, dv] fp64) where
    state[n, h, a, b] = S[b, a] for the dv x dk state S of the recurrence.
    """
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.float32)
    k = np.ascontiguousarray(k, dtype=np.float32)
    v = np.ascontiguousarray(v, dtype=np.float32)
    g = np.ascontiguousarray(g, dtype=np.float32)
    beta = np.ascontiguousarray(beta, dtype=np.float32)
    cu = np.ascontiguousarray(cu_tail_lens, dtype=np.int32)
    T, Hq, dk = q.shape
    Tv, Hv, dv = v.shape
    N = cu.shape[0] - 1
    assert k.shape == q.shape and Tv == T and g.shape == (T, Hv) and beta.shape == (T, Hv)
    assert cu[0] == 0 and cu[-1] == T
    o = np.zeros((T, Hv, dv), dtype=np.float64) if want_o else None
    st = np.zeros((N, Hv, dk, dv), dtype=np.float64)
    init = None
    if init_state is not None:
        init = np.ascontiguousarray(init_state, dtype=np.float64)
        assert init.shape == st.shape
    fp = ctypes.POINTER(ctypes.c_float)
    dp = ctypes.POINTER(ctypes.c_double)
    ip = ctypes.POINTER(ctypes.c_int32)
    rc = lib.gdn_oracle_forward(
        q.ctypes.data_as(fp), k.ctypes.data_as(fp), v.ctypes.data_as(fp), g.ctypes.data_as(fp),
        beta.ctypes.data_as(fp), cu.ctypes.data_as(ip), N, Hq, Hv, dk, dv,
        init.ctypes.data_as(dp) if init is not None else None,
        o.ctypes.data_as(dp) if o is not None else None,
        st.ctypes.data_as(dp), int(threads if threads is not None else default_threads()))
    if rc != 0:
        raise ValueError("gdn_oracle_forward rejected its arguments")
    return o, st


def prologue(q_raw, k_raw, gate_raw, beta_raw, eps: float = 1e-6):
    """The input pipeline in front of the recurrence (paper, Method section: the cached hiddens are fed through the
    linear-attention layers, "which produce k, v, T and beta at each replay step"), from raw projection outputs, in
    fp64.  The paper fixes neither normalisation nor gate parametrisation; the reading taken here:

        q, k   L2-normalised over the head dimension:  x / sqrt(sum(x^2) + eps)
        alpha  = sigmoid(gate_raw)   so that alpha in (0, 1), i.e.  g = log alpha = -log(1 + exp(-gate_raw))
        beta   = sigmoid(beta_raw)   in (0, 1)

    Returns (q, k, g, beta) as fp64 arrays."""
    q = np.asarray(q_raw, dtype=np.float64)
    k = np.asarray(k_raw, dtype=np.float64)
    a = np.asarray(gate_raw, dtype=np.float64)
    b = np.asarray(beta_raw, dtype=np.float64)
    qn = q / np.sqrt(np.sum(q * q, axis=-1, keepdims=True) + eps)
    kn = k / np.sqrt(np.sum(k * k, axis=-1, keepdims=True) + eps)
    g = -np.logaddexp(0.0, -a)
    beta = 1.0 / (1.0 + np.exp(-b))
    return qn, kn, g, beta


def gdn_forward_f64(q, k, v, g, beta, cu_tail_lens, init_state: Optional[np.ndarray] = None,
                    threads: Optional[int] = None, want_o: bool = True):
    """``gdn_forward`` on inputs that are already fp64 (no widening step): same C routine, same recurrence."""
    lib = _load()
    q, k, v, g, beta = (np.ascontiguousarray(x, dtype=np.float64) for x in (q, k, v, g, beta))
    cu = np.ascontiguousarray(cu_tail_lens, dtype=np.int32)
    T, Hq, dk = q.shape
    Tv, Hv, dv = v.shape
    N = cu.shape[0] - 1
    assert k.shape == q.shape and Tv == T and g.shape == (T, Hv) and beta.shape == (T, Hv)
    assert cu[0] == 0 and cu[-1] == T
    o = np.zeros((T, Hv, dv), dtype=np.float64) if want_o else None
    st = np.zeros((N, Hv, dk, dv), dtype=np.float64)
    init = None
    if init_state is not None:
        init = np.ascontiguousarray(init_state, dtype=np.float64)
        assert init.shape == st.shape
    dp = ctypes.POINTER(ctypes.c_double)
    ip = ctypes.POINTER(ctypes.c_int32)
    rc = lib.gdn_oracle_forward_f64(
        q.ctypes.data_as(dp), k.ctypes.data_as(dp), v.ctypes.data_as(dp), g.ctypes.data_as(dp),
        beta.ctypes.data_as(dp), cu.ctypes.data_as(ip), N, Hq, Hv, dk, dv,
        init.ctypes.data_as(dp) if init is not None else None,
        o.ctypes.data_as(dp) if o is not None else None,
        st.ctypes.data_as(dp), int(threads if threads is not None else default_threads()))
    if rc != 0:
        raise ValueError("gdn_oracle_forward_f64 rejected its arguments")
    return o, st


def gdn_forward_inputs(inp, init_state=None, threads=None, want_o=True):
    """Convenience: run on a ``gdn_workloads.GdnInputs`` batch."""
    return gdn_forward(inp.q, inp.k, inp.v, inp.g, inp.beta, inp.cu_tail_lens,
                       init_state=init_state, threads=threads, want_o=want_o)


def tail_select(prefix_len: int, budget_frac) -> int:
    """Replay-window length k = ceil(r * m), clamped to [0, m]; the window is [m - k, m).

    The ratio is read as the decimal it was written as (its shortest round-trip decimal
    string) and the ceiling is taken over exact rationals, so that e.g. r = 0.07, m = 100
    gives 7 and not the 8 that binary64 multiplication would.  Returns -1 for m < 0, r < 0
    or NaN.
    """
    m = int(prefix_len)
    r = float(budget_frac)
    if m < 0 or r != r or r < 0:
        return -1
    if r >= 1.0:
        return m
    x = Fraction(repr(r)) * m
    k = -((-x.numerator) // x.denominator)
    return max(0, min(m, int(k)))
