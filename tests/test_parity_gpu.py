"""GPU parity: the CUDA path, called through the C-ABI, against the fp64 oracle on the same
seeded inputs, element by element, at sizes the oracle finishes in seconds but that span
several chunks and a ragged tail; plus edge cases, guard regions around the outputs, poisoned neighbour
rows, and every chain of the full-size configurations."""
import numpy as np
import pytest

import oracle
from gdn_workloads import (make_inputs, make_raw_inputs, config_tiny_f32, config_single_layer, config_concurrent_hits,
                           config_budget_sweep_tails, config_budget_sweep_layer, config_full_prefill)
from gpu_utils import run_library, assert_parity, assert_parity_lean, state_rel_fro, TOL

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
    for Hq, Hv in [(1, 1), (1, 4), (3, 3), (2, 6), (2, 8)]:
        inp = make_inputs([200, 77], Hq, Hv, 128, 128, "bf16", seed=5 + Hq * 10 + Hv)
        check(inp, kernel)


@pytest.mark.parametrize("kernel", [TC])
def test_tc_init_state_resume_ragged(kernel):
    """Resume identity on the tensor-core path: run(prefix + tail) == run(tail, init = run(prefix)), request by
    request on a ragged batch that includes empty tails (whose final state must equal the start state) and
    tails shorter than a chunk; the resumed outputs and states are also compared with the oracle."""
    lens = [200, 64, 0, 1, 129, 330, 63, 0]
    cut = [120, 64, 0, 0, 1, 200, 10, 0]                   # rows of each request that form the prefix
    inp = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=23)
    pre_lens = cut
    tail_lens = [l - c for l, c in zip(lens, cut)]
    def split(lens_part, offs):
        rows = np.concatenate([np.arange(int(inp.cu_tail_lens[n]) + o, int(inp.cu_tail_lens[n]) + o + l)
                               for n, (l, o) in enumerate(zip(lens_part, offs))]).astype(np.int64)
        sub = make_inputs(lens_part, 2, 4, 128, 128, "bf16", seed=1)
        for name in ("q", "k", "v", "g", "beta", "q_bits", "k_bits", "v_bits"):
            setattr(sub, name, np.ascontiguousarray(getattr(inp, name)[rows]))
        return sub, rows
    pre, _ = split(pre_lens, [0] * len(lens))
    tail, tail_rows = split(tail_lens, cut)
    ro, rst = oracle.gdn_forward_inputs(inp)
    _, st_pre, _ = run_library(pre, kernel=kernel)
    o_tail, st_res, _ = run_library(tail, kernel=kernel, init_state=st_pre, canary=True)
    assert_parity(inp, None, st_res, None, rst)
    assert np.abs(o_tail - ro[tail_rows]).max() <= TOL["bf16"]["o_max_abs"]
    # and against the oracle started from the same (GPU-made, fp32) prefix state
    ro2, rst2 = oracle.gdn_forward_inputs(tail, init_state=st_pre.astype(np.float32).astype(np.float64))
    assert_parity(tail, o_tail, st_res, ro2, rst2)
    for n, l in enumerate(tail_lens):
        if l == 0:
            np.testing.assert_array_equal(st_res[n], st_pre[n].astype(np.float32).astype(np.float64))


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_run_to_run_bitwise_determinism(kernel):
    inp = make_inputs([100, 37, 200], 2, 4, 128, 128, "bf16", seed=9)
    o1, s1, _ = run_library(inp, kernel=kernel)
    o2, s2, _ = run_library(inp, kernel=kernel)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(s1, s2)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_guard_rows_around_outputs_stay_untouched(kernel):
    """out_o sits between 64 guard rows on each side and out_state between two guard states, all filled with a
    bit pattern; ragged last chunks (whose 64-row tiles reach past the request and past the end of the batch)
    must leave every guard byte alone, and the rows in between must match the oracle."""
    for lens in ([100, 37, 200], [1], [63, 0, 65], [129]):
        inp = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=9 + len(lens))
        o, st, _ = run_library(inp, kernel=kernel, canary=True)
        ro, rst = oracle.gdn_forward_inputs(inp)
        assert_parity(inp, o, st, ro, rst)
        _, st2, _ = run_library(inp, kernel=kernel, canary=True, want_o=False)
        np.testing.assert_array_equal(st, st2)


def _poison_other_requests(inp, keep):
    """Copy of the batch in which every row that does not belong to request `keep` holds large finite values
    (keys and queries far from unit norm, a huge beta, a strong gate)."""
    import copy
    from gdn_workloads import f32_to_bf16_bits, bf16_bits_to_f32
    p = copy.deepcopy(inp)
    a, b = int(inp.cu_tail_lens[keep]), int(inp.cu_tail_lens[keep + 1])
    mask = np.ones(inp.total_tokens, dtype=bool)
    mask[a:b] = False
    for name in ("q", "k", "v"):
        x = getattr(p, name)
        x[mask] = np.float32(-3.0e4) if name == "v" else np.float32(1.0e4)
        bits = f32_to_bf16_bits(x)
        setattr(p, name + "_bits", bits)
        setattr(p, name, bf16_bits_to_f32(bits))
    p.g[mask] = np.float32(-7.0)
    p.beta[mask] = np.float32(50.0)
    return p


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_poisoned_neighbour_rows_do_not_leak(kernel):
    """The 64-row tiles of a request's ragged last chunk overlap the first rows of the next request (and a
    short request sits inside tiles of its neighbours).  Filling every foreign row with large finite values
    must not change a request's outputs or final state by a single bit."""
    lens = [100, 37, 200, 5, 64, 1]
    inp = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=19)
    o, st, _ = run_library(inp, kernel=kernel, canary=True)
    for keep in range(len(lens)):
        pinp = _poison_other_requests(inp, keep)
        po, pst, _ = run_library(pinp, kernel=kernel, canary=True)
        a, b = int(inp.cu_tail_lens[keep]), int(inp.cu_tail_lens[keep + 1])
        np.testing.assert_array_equal(po[a:b], o[a:b])
        np.testing.assert_array_equal(pst[keep], st[keep])


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
def test_host_memory_groups_with_dirty_workspace(kernel):
    """Host-memory mode pipelines the batch by groups of requests through the caller's workspace.  The workspace here
    starts out filled with NaN bit patterns and the requests end inside tiles (ragged tails), so a group's last tile
    hangs over rows that have not arrived yet: the results must not depend on what the workspace held."""
    import torch
    import paper_2608_30310_b200 as gdn
    rng = np.random.default_rng(41)
    lens = [int(x) for x in rng.integers(1, 200, size=40)]
    lens[7] = 0
    inp = make_inputs(lens, 2, 4, 128, 128, "bf16", seed=32)
    st0 = rng.standard_normal((len(lens), 4, 128, 128)).astype(np.float32)
    ws = gdn.Workspace(device="cuda")
    ws.ensure(64 << 20)
    ws.buf.fill_(0xFF)
    torch.cuda.synchronize()
    o, st, _ = run_library(inp, kernel=kernel, host=True, init_state=st0, workspace=ws)
    ro, rst = oracle.gdn_forward_inputs(inp, init_state=st0.astype(np.float64))
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
    # alpha = 0 exactly (g = -inf) on single tokens: inside a chunk, on a chunk's first and on its last token
    inp = make_inputs([200], 1, 2, 128, 128, "bf16", seed=44)
    for t, h in ((37, 0), (64, 1), (127, 0), (128, 1)):
        inp.g[t, h] = -np.inf
    o, st, _ = run_library(inp, kernel=kernel)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_weak_decay_long_memory(kernel):
    inp = make_inputs([700], 1, 2, 128, 128, "bf16", seed=43, g_lo=-0.002, g_hi=-0.0001)
    check(inp, kernel)


@pytest.mark.parametrize("kernel", [TC])
def test_config3_concurrent_hits_full_size_all_chains(kernel):
    """Full-size 32-request batch in the benchmark's launch configuration: every one of the 1,024 chains
    (all outputs, all final states) against the oracle."""
    inp = config_concurrent_hits()
    o, st, _ = run_library(inp, kernel=kernel, canary=True)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity_lean(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [TC])
def test_config2_budget_sweep_tails_all_chains(kernel):
    for i, cfg in enumerate(config_budget_sweep_tails()):
        inp = config_budget_sweep_layer(cfg["tail"], layer=i)
        o, st, launches = run_library(inp, kernel=kernel, canary=True)
        assert launches == 1                                  # a single request needs no scheduler kernel
        ro, rst = oracle.gdn_forward_inputs(inp)
        assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [TC])
def test_paper_matched_prefix_tails_ragged_batch(kernel):
    """The tails of the matched-prefix lengths the paper's serving-efficiency table prints at 32K
    (31,366 and 31,847 tokens at 5 % and 10 %: 1,569 / 1,593 / 3,137 / 3,185) as one ragged batch."""
    import paper_2608_30310_b200 as gdn
    lens = [gdn.tail_select(m, r) for m in (31366, 31847) for r in (0.05, 0.10)]
    assert sorted(lens) == [1569, 1593, 3137, 3185]
    inp = make_inputs(lens, 16, 32, 128, 128, "bf16", seed=2608030310 + 117)
    o, st, _ = run_library(inp, kernel=kernel, canary=True)
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity_lean(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [TC])
def test_config4_full_prefill_and_alpha_product_bound(kernel):
    """Zero-state forward over a whole 32K prefix vs the oracle on every chain, and the
    tail-vs-full state difference against prod(alpha over the tail) * ||S_prefix||_F."""
    full = config_full_prefill(32768)
    o, st, _ = run_library(full, kernel=kernel, fn="gdn_full_prefill")
    ro, rst = oracle.gdn_forward_inputs(full)
    assert_parity_lean(full, o, st, ro, rst)
    del o, ro
    for tail_len in (1639, 3277):
        tail = full.take_rows(32768 - tail_len, 32768)
        _, st_tail, _ = run_library(tail, kernel=kernel)
        _, st_pre, _ = run_library(full.take_rows(0, 32768 - tail_len), kernel=kernel,
                                   fn="gdn_full_prefill", want_o=False)
        for h in range(32):
            prod_alpha = np.exp(np.sum(full.g[32768 - tail_len:, h].astype(np.float64)))
            bound = prod_alpha * np.linalg.norm(st_pre[0, h])
            diff = np.linalg.norm(st[0, h] - st_tail[0, h])
            slack = 2 * TOL["bf16"]["state_rel_fro"] * np.linalg.norm(st[0, h])
            assert diff <= bound + slack


@pytest.mark.parametrize("kernel", [TC])
def test_config4_full_prefill_128k_all_chains(kernel):
    """The largest named size: zero-state forward over a 131,072-token prefix (2,048 serial chunks per head),
    every chain against the oracle."""
    full = config_full_prefill(131072)
    o, st, _ = run_library(full, kernel=kernel, fn="gdn_full_prefill")
    ro, rst = oracle.gdn_forward_inputs(full)
    assert_parity_lean(full, o, st, ro, rst)


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


@pytest.mark.parametrize("kernel", [TC])
def test_many_short_requests(kernel):
    """2,000 requests of 0-130 tokens (4,000 chains, 27 rounds of the snake schedule over 148 CTAs): almost every chunk is
    the first and the last of its chain, a quarter of the requests fit no full chunk and some are empty, so the chain
    switches (start, final-state store, first-chunk shortcuts) are exercised back to back."""
    rng = np.random.default_rng(2608030310 + 7)
    lens = [int(x) for x in rng.integers(0, 131, size=2000)]
    lens[3] = lens[1500] = 0
    inp = make_inputs(lens, 1, 2, 128, 128, "bf16", seed=2608030310 + 70_000)
    o, st, launches = run_library(inp, kernel=kernel, canary=True)
    assert launches == 2                                     # scheduler kernel + forward kernel
    ro, rst = oracle.gdn_forward_inputs(inp)
    assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [TC])
def test_group_parallel_packing_equals_per_layer_calls(kernel):
    """The paper rebuilds every group independently: the current layer of G groups can therefore go into one call as
    G pseudo-requests.  The packed call must reproduce the G single-request calls bit for bit (a chain's arithmetic does
    not depend on what else is in the batch) and match the oracle."""
    G, L = 12, 410
    layers = [config_budget_sweep_layer(L, layer=i) for i in range(G)]
    packed = make_inputs([L] * G, 16, 32, 128, 128, "bf16", seed=1)
    for name in ("q", "k", "v", "g", "beta", "q_bits", "k_bits", "v_bits"):
        setattr(packed, name, np.ascontiguousarray(np.concatenate([getattr(x, name) for x in layers], axis=0)))
    o, st, launches = run_library(packed, kernel=kernel, canary=True)
    ro, rst = oracle.gdn_forward_inputs(packed)
    assert_parity(packed, o, st, ro, rst)
    for i in (0, 5, G - 1):
        oi, sti, _ = run_library(layers[i], kernel=kernel)
        np.testing.assert_array_equal(o[i * L:(i + 1) * L], oi)
        np.testing.assert_array_equal(st[i], sti[0])


def _check_raw(inp, kernel):
    o, st, _ = run_library(inp, kernel=kernel, raw_inputs=True, canary=True)
    qn, kn, g, beta = oracle.prologue(inp.q, inp.k, inp.g, inp.beta)
    ro, rst = oracle.gdn_forward_f64(qn, kn, inp.v, g, beta, inp.cu_tail_lens)
    return assert_parity(inp, o, st, ro, rst)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_fused_input_stage_bf16(kernel):
    """Raw projection outputs in (un-normalised q and k of varying scale, gate and beta pre-activations): the kernels
    apply the input stage in their load path; the oracle applies its plain fp64 version first."""
    _check_raw(make_raw_inputs([130, 64, 1, 0, 63, 65, 410, 5], 2, 4, 128, 128, "bf16", seed=61), kernel)
    _check_raw(make_raw_inputs([700], 1, 2, 128, 128, "bf16", seed=62), kernel)
    _check_raw(make_raw_inputs([1638], 16, 32, 128, 128, "bf16", seed=63), kernel)


@pytest.mark.parametrize("kernel", [SIMT, TC])
def test_fused_input_stage_with_start_state(kernel):
    """The input stage and a non-zero start state together (a suffix served from raw projection outputs after a
    replay): the oracle applies its fp64 input stage and starts the recurrence from the same state."""
    lens = [130, 0, 64, 1, 200]
    inp = make_raw_inputs(lens, 2, 4, 128, 128, "bf16", seed=66)
    st0 = np.random.default_rng(66).standard_normal((len(lens), 4, 128, 128)).astype(np.float32)
    o, st, _ = run_library(inp, kernel=kernel, raw_inputs=True, init_state=st0, canary=True)
    qn, kn, g, beta = oracle.prologue(inp.q, inp.k, inp.g, inp.beta)
    ro, rst = oracle.gdn_forward_f64(qn, kn, inp.v, g, beta, inp.cu_tail_lens, init_state=st0.astype(np.float64))
    assert_parity(inp, o, st, ro, rst)
    np.testing.assert_array_equal(st[1], st0[1].astype(np.float64))      # the empty request returns its start state


def test_fused_input_stage_fp32():
    _check_raw(make_raw_inputs([150, 0, 1, 64, 65, 17], 2, 4, 64, 64, "f32", seed=64), SIMT)
    _check_raw(make_raw_inputs([300], 2, 4, 128, 64, "f32", seed=65), 0)
