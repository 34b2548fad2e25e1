"""Helpers for the GPU parity tests: run the C-ABI library on a GdnInputs batch and compare
with the oracle under the stated tolerances."""
import numpy as np

# Tolerances (benchmark statement): bf16 io with fp32 state: final state relative Frobenius
# error <= 5e-3, outputs max abs error <= 2e-2; fp32 io: 1e-4 on both.
TOL = {"bf16": {"state_rel_fro": 5e-3, "o_max_abs": 2e-2},
       "f32": {"state_rel_fro": 1e-4, "o_max_abs": 1e-4}}


def to_torch(inp, device="cuda", pin=False):
    import torch

    def t(a, bits=None):
        if bits is not None:
            x = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
        else:
            x = torch.from_numpy(a)
        if device == "cpu":
            return x.pin_memory() if pin else x.contiguous()
        return x.to(device)
    bf = inp.io_dtype == "bf16"
    q = t(inp.q, inp.q_bits if bf else None)
    k = t(inp.k, inp.k_bits if bf else None)
    v = t(inp.v, inp.v_bits if bf else None)
    return q, k, v, t(inp.g), t(inp.beta), t(inp.cu_tail_lens)


GUARD_ROWS = 64                     # guard rows on each side of out_o (one guard state on each side of out_state)
GUARD_BF16 = 0x7BCD                 # bit pattern of the guards (a large finite bf16; as fp32 halves 0x7BCD7BCD)


def run_library(inp, kernel=0, host=False, fn="gdn_tail_replay", want_o=True, init_state=None,
                canary=False, raw_inputs=False, workspace=None):
    """Returns (o [T,Hv,dv] float64 or None, state [N,Hv,dk,dv] float64, launches).

    With ``canary`` the outputs are carved out of larger device buffers whose surrounding guard
    rows / guard states hold a fixed bit pattern, rows of the outputs start from the same pattern,
    and the call asserts afterwards that every guard byte is untouched.
    """
    import torch
    import paper_2608_30310_b200 as gdn
    dev = "cpu" if host else "cuda"
    q, k, v, g, beta, cu = to_torch(inp, dev, pin=host)
    T, Hv, dv = v.shape
    dk = q.shape[2]
    N = cu.numel() - 1
    o_full = st_full = None
    if canary:
        assert not host
        esz = 2 if q.dtype == torch.bfloat16 else 4
        o_full = torch.full(((T + 2 * GUARD_ROWS) * Hv * dv * esz // 2,), GUARD_BF16, dtype=torch.int16, device=dev)
        st_full = torch.full(((N + 2) * Hv * dk * dv * 2,), GUARD_BF16, dtype=torch.int16, device=dev)
        o = o_full.view(q.dtype).view(T + 2 * GUARD_ROWS, Hv, dv)[GUARD_ROWS:GUARD_ROWS + T] if want_o else None
        st = st_full.view(torch.float32).view(N + 2, Hv, dk, dv)[1:N + 1]
    else:
        o = torch.full((T, Hv, dv), float("nan"), dtype=q.dtype, device=dev) if want_o else None
        st = torch.full((N, Hv, dk, dv), float("nan"), dtype=torch.float32, device=dev)
    if host:
        o = o.pin_memory() if o is not None else None
        st = st.pin_memory()
    init = None
    if init_state is not None:
        init = torch.from_numpy(np.ascontiguousarray(init_state, dtype=np.float32))
        init = init.pin_memory() if host else init.cuda()
    getattr(gdn, fn)(q, k, v, g, beta, cu, 64, o, st, kernel=kernel, init_state=init, raw_inputs=raw_inputs,
                     workspace=workspace)
    torch.cuda.synchronize()
    launches = gdn.last_launch_count()
    if canary:
        og = o_full.view(torch.int16).view(T + 2 * GUARD_ROWS, -1)
        assert bool((og[:GUARD_ROWS] == GUARD_BF16).all()) and bool((og[GUARD_ROWS + T:] == GUARD_BF16).all()), \
            "guard rows around out_o were written"
        sg = st_full.view(N + 2, -1)
        assert bool((sg[0] == GUARD_BF16).all()) and bool((sg[N + 1] == GUARD_BF16).all()), \
            "guard states around out_state were written"
    o_np = None if o is None else o.float().cpu().numpy().astype(np.float64)
    return o_np, st.cpu().numpy().astype(np.float64), launches


def state_rel_fro(got, ref):
    """Worst per-(request, head) relative Frobenius error and the whole-tensor one."""
    N, H = ref.shape[:2]
    worst = 0.0
    for n in range(N):
        for h in range(H):
            den = np.linalg.norm(ref[n, h])
            num = np.linalg.norm(got[n, h] - ref[n, h])
            if den == 0:
                worst = max(worst, 0.0 if num == 0 else np.inf)
            else:
                worst = max(worst, num / den)
    den = np.linalg.norm(ref)
    total = 0.0 if den == 0 else np.linalg.norm(got - ref) / den
    return worst, total


def assert_parity(inp, got_o, got_state, ref_o, ref_state, tol=None):
    tol = tol or TOL[inp.io_dtype]
    assert np.isfinite(got_state).all(), "non-finite state"
    worst, total = state_rel_fro(got_state, ref_state)
    assert worst <= tol["state_rel_fro"], "state rel-Frobenius %.3e (whole %.3e)" % (worst, total)
    if got_o is not None and ref_o is not None and ref_o.size:
        assert np.isfinite(got_o).all(), "non-finite output"
        err = np.abs(got_o - ref_o).max()
        assert err <= tol["o_max_abs"], "output max abs err %.3e" % err
    return worst


def assert_parity_lean(inp, got_o, got_state, ref_o, ref_state):
    """assert_parity for very large outputs: the output comparison walks the rows in blocks so that no
    temporary of the full size is made."""
    tol = TOL[inp.io_dtype]
    assert np.isfinite(got_state).all(), "non-finite state"
    worst, total = state_rel_fro(got_state, ref_state)
    assert worst <= tol["state_rel_fro"], "state rel-Frobenius %.3e (whole %.3e)" % (worst, total)
    err = 0.0
    for a in range(0, ref_o.shape[0], 8192):
        blk = got_o[a:a + 8192]
        assert np.isfinite(blk).all(), "non-finite output"
        err = max(err, float(np.abs(blk - ref_o[a:a + 8192]).max()))
    assert err <= tol["o_max_abs"], "output max abs err %.3e" % err
    return worst
