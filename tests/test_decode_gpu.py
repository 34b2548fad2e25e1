"""The single-token step from a given state (what serving does after the replay), through the C ABI, against the oracle
started from the same state; and a replay followed by decode steps against one oracle pass over the whole sequence."""
import numpy as np
import pytest

import oracle
from gdn_workloads import make_inputs
from gpu_utils import TOL, state_rel_fro, run_library

pytestmark = pytest.mark.gpu


def _decode(inp, state_in, in_place=False):
    import torch
    import paper_2608_30310_b200 as gdn
    from gpu_utils import to_torch
    q, k, v, g, beta, _ = to_torch(inp, "cuda")
    N = inp.num_seqs
    st_in = torch.from_numpy(np.ascontiguousarray(state_in, dtype=np.float32)).cuda()
    st_out = st_in if in_place else torch.full_like(st_in, float("nan"))
    o = torch.full((N, inp.num_v_heads, inp.head_v_dim), float("nan"), dtype=q.dtype, device="cuda")
    gdn.gdn_decode_step(q, k, v, g, beta, st_in, o, st_out)
    torch.cuda.synchronize()
    assert gdn.last_launch_count() == 1
    return o.float().cpu().numpy().astype(np.float64), st_out.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("io", ["bf16", "f32"])
@pytest.mark.parametrize("dk,dv", [(128, 128), (64, 128), (128, 64), (64, 64)])
def test_decode_step_matches_oracle(io, dk, dv):
    N = 37
    inp = make_inputs([1] * N, 2, 6, dk, dv, io, seed=500 + dk + 2 * dv)
    rng = np.random.default_rng(7)
    st0 = rng.standard_normal((N, 6, dk, dv)).astype(np.float32)
    ro, rst = oracle.gdn_forward_inputs(inp, init_state=st0.astype(np.float64))
    for in_place in (False, True):
        o, st = _decode(inp, st0, in_place=in_place)
        # the state is carried in fp32 whatever the io dtype: fp32 tolerance; outputs are rounded to the io dtype
        assert state_rel_fro(st, rst)[0] <= 1e-5
        assert np.abs(o - ro).max() <= (TOL[io]["o_max_abs"] if io == "bf16" else 1e-4)


def test_replay_then_decode_equals_one_pass():
    """Rebuild the states from a tail, then serve three more tokens one at a time: states and outputs must match the
    oracle run over tail + suffix in one go (many requests, ragged tails)."""
    lens = [int(x) for x in np.random.default_rng(3).integers(1, 200, size=64)]
    steps = 3
    full = make_inputs([l + steps for l in lens], 2, 4, 128, 128, "bf16", seed=777)
    ro, rst = oracle.gdn_forward_inputs(full)
    cu = full.cu_tail_lens
    tail_rows = np.concatenate([np.arange(cu[n], cu[n] + lens[n]) for n in range(len(lens))])
    tail = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=1)
    for name in ("q", "k", "v", "g", "beta", "q_bits", "k_bits", "v_bits"):
        setattr(tail, name, np.ascontiguousarray(getattr(full, name)[tail_rows]))
    _, st, _ = run_library(tail, kernel=0)
    for s in range(steps):
        rows = np.array([cu[n] + lens[n] + s for n in range(len(lens))])
        tok = make_inputs([1] * len(lens), 2, 4, 128, 128, "bf16", seed=2)
        for name in ("q", "k", "v", "g", "beta", "q_bits", "k_bits", "v_bits"):
            setattr(tok, name, np.ascontiguousarray(getattr(full, name)[rows]))
        o, st = _decode(tok, st)
        assert np.abs(o - ro[rows]).max() <= TOL["bf16"]["o_max_abs"]
    assert state_rel_fro(st, rst)[0] <= TOL["bf16"]["state_rel_fro"]
