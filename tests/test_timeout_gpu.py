"""Failure detection without a GPU fault: a device-side wait that can never be satisfied runs out after its
bound, the kernel stops blocking and returns, the status word carries GDN_ERR_TIMEOUT, and the context stays
usable for the next, healthy call."""
import numpy as np
import pytest

import oracle
from gdn_workloads import make_inputs
from gpu_utils import run_library, assert_parity, to_torch

pytestmark = pytest.mark.gpu


def test_expired_wait_sets_status_and_context_survives():
    import torch
    import paper_2608_30310_b200 as gdn
    inp = make_inputs([200], 1, 1, 128, 128, "bf16", seed=91)
    q, k, v, g, beta, cu = to_torch(inp, "cuda")
    o = torch.zeros((200, 1, 128), dtype=torch.bfloat16, device="cuda")
    st = torch.zeros((1, 1, 128, 128), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        # the K/Q tile of chunk 1 is never copied, so the wait for it runs out after 2 ms
        gdn.test_hooks(wait_timeout_ns=2_000_000, skip_kq_load_of_chunk=1)
        rc = gdn.gdn_tail_replay(q, k, v, g, beta, cu, 64, o, st, kernel=2, status_word=status)
        torch.cuda.synchronize()
        assert rc == 0                                       # the launch itself succeeded
        assert int(status.item()) == -5                      # GDN_ERR_TIMEOUT reported by the device
    finally:
        gdn.test_hooks(0, -1)
    # same inputs again with the hooks cleared: correct results, status untouched
    status.zero_()
    o2, st2, _ = run_library(inp, kernel=2)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o2, st2, ro, rst)
    gdn.gdn_tail_replay(q, k, v, g, beta, cu, 64, o, st, kernel=2, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
