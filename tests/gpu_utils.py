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


def run_library(inp, kernel=0, host=False, fn="gdn_tail_replay", want_o=True, init_state=None,
                canary=False):
    """Returns (o [T,Hv,dv] float64 or None, state [N,Hv,dk,dv] float64, launches)."""
    import torch
    import paper_2608_30310_b200 as gdn
    dev = "cpu" if host else "cuda"
    q, k, v, g, beta, cu = to_torch(inp, dev, pin=host)
    T, Hv, dv = v.shape
    dk = q.shape[2]
    N = cu.numel() - 1
    o = torch.full((T, Hv, dv), float("nan"), dtype=q.dtype, device=dev) if want_o else None
    st = torch.full((N, Hv, dk, dv), float("nan"), dtype=torch.float32, device=dev)
    if host:
        o = o.pin_memory() if o is not None else None
        st = st.pin_memory()
    init = None
    if init_state is not None:
        init = torch.from_numpy(np.ascontiguousarray(init_state, dtype=np.float32))
        init = init.pin_memory() if host else init.cuda()
    getattr(gdn, fn)(q, k, v, g, beta, cu, 64, o, st, kernel=kernel, init_state=init)
    torch.cuda.synchronize()
    launches = gdn.last_launch_count()
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
