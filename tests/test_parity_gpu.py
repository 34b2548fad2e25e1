"""GPU parity: the CUDA path, called through the C-ABI, against the fp64 oracle on the same
seeded inputs, element by element, at sizes the oracle finishes in seconds but that span
several chunks and a ragged tail; plus edge cases and full-size sampled checks."""
import numpy as np
import pytest

import oracle
from gdn_workloads import (make_inputs, config_tiny_f32, config_single_layer, config_concurrent_hits,
                           config_budget_sweep_tails, config_budget_sweep_layer, config_full_prefill)
from gpu_utils import run_library, assert_parity, state_rel_fro, TOL

pytestmark = pytest.mark.gpu

SIMT, TC = 1, 2


def check(inp, kernel, **kw):
    o, st, launches = run_library(inp, kernel=kernel, **kw)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert launches >= 1
    return assert_parity(inp, o, st, ro, rst)


def test_config0_tiny_fp32():
    check(config_tiny_f32(), SIMT)
    check(config_tiny_f32(), 0)


@pytest.mark.parametrize("dk,dv", [(64, 64), (64, 128), (128, 64), (128, 128)])
@pytest.mark.parametrize("io", ["f32", "bf16"])
def test_simt_shapes(dk, dv, io):
    inp = make_inputs([150, 0, 1, 64, 65, 17], 2, 4, dk, dv, io, seed=11 + dk + 2 * dv)
    check(inp, SIMT)


def test_simt_fp32_tolerance_is_fp32_tight():
    inp = make_inputs([300], 2, 4, 128, 128, "f32", seed=3)
    o, st, _ = run_library(inp, kernel=SIMT)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert np.abs(o - ro).max() < 1e-5
    assert state_rel_fro(st, rst)[0] < 1e-5


def test_simt_init_state_resume():
    """Resume identity on the GPU: run(prefix + tail) == run(tail, init = run(prefix))."""
    inp = make_inputs([200], 2, 4, 64, 64, "f32", seed=21)
    _, st_full, _ = run_library(inp, kernel=SIMT)
    pre, tail = inp.take_rows(0, 120), inp.take_rows(120, 200)
    _, st_pre, _ = run_library(pre, kernel=SIMT)
    o_tail, st_res, _ = run_library(tail, kernel=SIMT, init_state=st_pre)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert state_rel_fro(st_res, rst)[0] < 1e-4
    assert np.abs(o_tail - ro[120:]).max() < 1e-4


@pytest.mark.parametrize("kernel", [SIMT, TC, 0])
def test_bf16_d128_ragged_batch(kernel):
    lens = [130, 64, 1, 0, 63, 65, 127, 128, 129, 410, 5]
    inp = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=77)
    check(inp, kernel)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_config1_single_layer(kernel):
    check(config_single_layer(), kernel)


@pytest.mark.parametrize("kernel", [TC])
def test_gqa_group_sizes(kernel):
    for Hq, Hv in [(1, 1), (1, 4), (3, 3), (2, 6)]:
        inp = make_inputs([200, 77], Hq, Hv, 128, 128, "bf16", seed=5 + Hq * 10 + Hv)
        check(inp, kernel)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_outputs_only_touch_valid_rows_and_are_deterministic(kernel):
    inp = make_inputs([100, 37, 200], 2, 4, 128, 128, "bf16", seed=9)
    o1, s1, _ = run_library(inp, kernel=kernel)
    o2, s2, _ = run_library(inp, kernel=kernel)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(s1, s2)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_state_only_and_full_prefill_entry(kernel):
    inp = make_inputs([333, 64], 2, 4, 128, 128, "bf16", seed=15)
    ro, rst = oracle.gdn_forward_inputs(inp)
    _, st, _ = run_library(inp, kernel=kernel, want_o=False)
    assert_parity(inp, None, st, None, rst)
    o, st, _ = run_library(inp, kernel=kernel, fn="gdn_full_prefill")
    assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_host_memory_call(kernel):
    inp = make_inputs([150, 90], 2, 4, 128, 128, "bf16", seed=31)
    o, st, _ = run_library(inp, kernel=kernel, host=True)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_strong_decay_and_beta_zero(kernel):
    """alpha -> 0 keeps only the last token's rank-1 update; beta = 0 keeps the state at zero."""
    inp = make_inputs([130], 1, 2, 128, 128, "bf16", seed=41)
    inp.g[:] = -1000.0
    o, st, _ = run_library(inp, kernel=kernel)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o, st, ro, rst)
    inp = make_inputs([130], 1, 2, 128, 128, "bf16", seed=42)
    inp.beta[:] = 0.0
    o, st, _ = run_library(inp, kernel=kernel)
    assert np.all(st == 0) and np.all(o == 0)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_weak_decay_long_memory(kernel):
    inp = make_inputs([700], 1, 2, 128, 128, "bf16", seed=43, g_lo=-0.002, g_hi=-0.0001)
    check(inp, kernel)


def _sampled_chain_parity(inp, o, st, chains):
    for (n, h) in chains:
        sub = inp.take_chain(n, h)
        ro, rst = oracle.gdn_forward_inputs(sub, threads=1)
        a, b = int(inp.cu_tail_lens[n]), int(inp.cu_tail_lens[n + 1])
        assert_parity(inp, o[a:b, h:h + 1], st[n:n + 1, h:h + 1], ro, rst)


@pytest.mark.parametrize("kernel", [TC])
def test_config3_concurrent_hits_full_size_sampled(kernel):
    """Full-size 32-request batch in the benchmark's launch configuration; the oracle checks a
    sample of whole chains (shortest, longest and a few others) and every state for finiteness."""
    inp = config_concurrent_hits()
    o, st, _ = run_library(inp, kernel=kernel)
    assert np.isfinite(st).all() and np.isfinite(o).all()
    lens = inp.tail_lens()
    chains = [(int(np.argmin(lens)), 0), (int(np.argmax(lens)), 31), (7, 13), (19, 2), (31, 30)]
    _sampled_chain_parity(inp, o, st, chains)


@pytest.mark.parametrize("kernel", [TC])
def test_config2_budget_sweep_tails(kernel):
    for i, cfg in enumerate(config_budget_sweep_tails()):
        inp = config_budget_sweep_layer(cfg["tail"], layer=i)
        o, st, _ = run_library(inp, kernel=kernel)
        _sampled_chain_parity(inp, o, st, [(0, 0), (0, 17), (0, 31)])


@pytest.mark.parametrize("kernel", [TC])
def test_config4_full_prefill_and_alpha_product_bound(kernel):
    """Zero-state forward over a whole 32K prefix vs the oracle on sampled heads, and the
    tail-vs-full state difference against prod(alpha over the tail) * ||S_prefix||_F."""
    full = config_full_prefill(32768)
    o, st, _ = run_library(full, kernel=kernel, fn="gdn_full_prefill")
    _sampled_chain_parity(full, o, st, [(0, 0), (0, 21)])
    for tail_len in (1639, 3277):
        tail = full.take_rows(32768 - tail_len, 32768)
        _, st_tail, _ = run_library(tail, kernel=kernel)
        _, st_pre, _ = run_library(full.take_rows(0, 32768 - tail_len), kernel=kernel,
                                   fn="gdn_full_prefill", want_o=False)
        for h in (0, 13, 31):
            prod_alpha = np.exp(np.sum(full.g[32768 - tail_len:, h].astype(np.float64)))
            bound = prod_alpha * np.linalg.norm(st_pre[0, h])
            diff = np.linalg.norm(st[0, h] - st_tail[0, h])
            slack = 2 * TOL["bf16"]["state_rel_fro"] * np.linalg.norm(st[0, h])
            assert diff <= bound + slack


@pytest.mark.parametrize("kernel", [TC])
def test_config4_full_prefill_128k_sampled(kernel):
    """The largest named size: zero-state forward over a 131,072-token prefix (2,048 serial chunks per head);
    one whole chain is checked against the oracle, every state for finiteness."""
    full = config_full_prefill(131072)
    o, st, _ = run_library(full, kernel=kernel, fn="gdn_full_prefill")
    assert np.isfinite(st).all()
    _sampled_chain_parity(full, o, st, [(0, 5)])


@pytest.mark.parametrize("kernel", [TC])
def test_weak_decay_tail_vs_full_bound_has_teeth(kernel):
    full = config_full_prefill(600, g_lo=-0.002, g_hi=-0.0001, num_qk_heads=2, num_v_heads=4)
    _, st, _ = run_library(full, kernel=kernel)
    tail = full.take_rows(300, 600)
    _, st_tail, _ = run_library(tail, kernel=kernel)
    _, st_pre, _ = run_library(full.take_rows(0, 300), kernel=kernel)
    for h in range(4):
        bound = np.exp(np.sum(full.g[300:, h].astype(np.float64))) * np.linalg.norm(st_pre[0, h])
        diff = np.linalg.norm(st[0, h] - st_tail[0, h])
        assert diff <= bound + 2 * TOL["bf16"]["state_rel_fro"] * np.linalg.norm(st[0, h])
        assert bound > 0.1                                   # the bound is not vacuous here


@pytest.mark.parametrize("kernel", [TC])
def test_randomised_ragged_batches(kernel):
    """Seeded sweep over ragged batches: request counts 1-11, lengths 0-330 (plus runs of lengths around one chunk and
    one long request), seven head configurations, four decay ranges from very weak to very strong.  The pipeline of
    the tensor-core kernel runs across chain boundaries, so short and empty chains in odd mixes are its edge cases."""
    rng = np.random.default_rng(2608030310)
    heads = [(1, 1), (1, 2), (2, 2), (2, 4), (4, 1), (3, 2), (16, 2)]
    decay = [(-0.1, -0.001), (-2.0, -0.1), (-0.002, -0.0001), (-8.0, -0.4)]
    for it in range(24):
        nreq = int(rng.integers(1, 12))
        lens = [int(x) for x in rng.integers(0, 330, size=nreq)]
        if it % 7 == 0:
            lens = [int(x) for x in rng.integers(60, 70, size=nreq)]
        if it % 11 == 0:
            lens[0] = int(rng.integers(700, 1500))
        if sum(lens) == 0:
            lens[0] = 5
        hq, g = heads[it % 7]
        g_lo, g_hi = decay[it % 4]
        inp = make_inputs(lens, hq, hq * g, 128, 128, "bf16", seed=2608030310 + 50_000 + it, g_lo=g_lo, g_hi=g_hi)
        check(inp, kernel)
