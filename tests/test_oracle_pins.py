"""Pins for the CPU oracle: facts that the paper's definitions (Eq. 1, Eq. 2, k = ceil(r m))
and plain mathematics fix, chosen so that a dropped term, a wrong sign or index, a transposed
operand or a wrong head mapping in the oracle fails at least one of them.  CPU only."""
import json
import os

import numpy as np
import pytest

import oracle
from gdn_workloads import make_inputs, config_tiny_f32
from chunked_form import chunked_forward

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def run(q, k, v, g, beta, cu=None, init=None):
    q, k, v = (np.asarray(x, dtype=np.float32) for x in (q, k, v))
    g, beta = np.asarray(g, dtype=np.float32), np.asarray(beta, dtype=np.float32)
    if cu is None:
        cu = [0, q.shape[0]]
    return oracle.gdn_forward(q, k, v, g, beta, np.asarray(cu, dtype=np.int32), init_state=init, threads=2)


def rand_case(rng, L, Hq, Hv, dk, dv, unit=True):
    q = rng.standard_normal((L, Hq, dk))
    k = rng.standard_normal((L, Hq, dk))
    if unit:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((L, Hv, dv))
    g = rng.uniform(-0.3, -0.001, (L, Hv))
    beta = 1 / (1 + np.exp(-rng.standard_normal((L, Hv))))
    return [x.astype(np.float32) for x in (q, k, v, g, beta)]


# --- hand-worked examples (golden file) --------------------------------------------------

@pytest.mark.parametrize("name", ["scalar", "two_by_two"])
def test_hand_examples(name):
    ex = json.load(open(os.path.join(GOLD, "hand_examples.json")))[name]
    k = np.array(ex["k"])[:, None, :]
    q = np.array(ex["q"])[:, None, :]
    v = np.array(ex["v"])[:, None, :]
    g = np.log(np.array(ex["alpha"]))[:, None]
    beta = np.array(ex["beta"])[:, None]
    o, st = run(q, k, v, g, beta)
    S = np.array(ex["S_final"])                      # dv x dk
    np.testing.assert_allclose(st[0, 0], S.T, rtol=0, atol=5e-7)   # inputs pass through fp32 (0.6, 0.8, log 0.5)
    np.testing.assert_allclose(o[:, 0, :], np.array(ex["o"]), rtol=0, atol=5e-7)


# --- P1: beta = 0 keeps the state at zero -------------------------------------------------

def test_beta_zero_state_stays_zero():
    rng = np.random.default_rng(1)
    q, k, v, g, beta = rand_case(rng, 50, 2, 4, 8, 6)
    o, st = run(q, k, v, np.zeros_like(g), np.zeros_like(beta))      # alpha = 1, beta = 0
    assert np.all(st == 0) and np.all(o == 0)
    o, st = run(q, k, v, g, np.zeros_like(beta))
    assert np.all(st == 0) and np.all(o == 0)


# --- P2: alpha -> 0 leaves only the last token's rank-1 update ----------------------------

def test_alpha_to_zero_keeps_last_rank1_update():
    rng = np.random.default_rng(2)
    L, Hq, Hv, dk, dv = 20, 2, 4, 8, 6
    q, k, v, g, beta = rand_case(rng, L, Hq, Hv, dk, dv, unit=False)
    g[:] = -1000.0                                               # exp underflows to exactly 0
    o, st = run(q, k, v, g, beta)
    G = Hv // Hq
    for h in range(Hv):
        kk, vv, bb = k[-1, h // G].astype(np.float64), v[-1, h].astype(np.float64), float(beta[-1, h])
        np.testing.assert_allclose(st[0, h], bb * np.outer(kk, vv), rtol=1e-14, atol=0)   # H = S^T = beta k v^T
        for t in range(L):
            kq = float(k[t, h // G].astype(np.float64) @ q[t, h // G].astype(np.float64))
            np.testing.assert_allclose(o[t, h], float(beta[t, h]) * kq * v[t, h].astype(np.float64),
                                       rtol=1e-13, atol=1e-300)


# --- P3: recall identity S_t k_t = alpha(1 - beta |k|^2) S_{t-1} k_t + beta |k|^2 v_t -------

def test_recall_identity_unit_keys_beta_one():
    rng = np.random.default_rng(3)
    L, dk, dv = 30, 8, 5
    q, k, v, g, beta = rand_case(rng, L, 1, 1, dk, dv)
    beta[:] = 1.0
    q = k.copy()                                                  # o_t = S_t k_t
    o, st = run(q, k, v, g, beta)
    k64 = k.astype(np.float64)
    nrm2 = np.sum(k64 * k64, axis=-1)                             # ~1 up to fp32 rounding of k
    # with beta = 1: S_t k_t = alpha (1 - |k|^2) S_{t-1} k_t + |k|^2 v_t; the first term is ~1e-7
    np.testing.assert_allclose(o[:, 0], nrm2 * v[:, 0].astype(np.float64), rtol=0, atol=5e-6)


def test_recall_identity_general_form():
    rng = np.random.default_rng(4)
    L, dk, dv = 12, 6, 4
    q, k, v, g, beta = rand_case(rng, L, 1, 1, dk, dv, unit=False)
    k *= 0.5
    # state before the last token
    _, s_prev = run(q[:-1], k[:-1], v[:-1], g[:-1], beta[:-1])
    _, s_full = run(q, k, v, g, beta)
    kk = k[-1, 0].astype(np.float64)
    a, b = np.exp(np.float64(g[-1, 0])), np.float64(beta[-1, 0])
    n2 = kk @ kk
    lhs = s_full[0, 0].T @ kk                                     # S_t k_t
    rhs = a * (1 - b * n2) * (s_prev[0, 0].T @ kk) + b * n2 * v[-1, 0].astype(np.float64)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12, atol=1e-14)


# --- P4: chunked (WY) form == token form, brute force on small inputs -----------------------

@pytest.mark.parametrize("L,Hq,Hv,dk,dv,C", [
    (7, 1, 1, 4, 3, 4), (37, 2, 4, 8, 8, 8), (150, 1, 2, 16, 16, 64), (130, 1, 1, 64, 64, 64),
    (1, 1, 1, 4, 4, 64), (63, 1, 1, 8, 4, 64), (64, 1, 1, 8, 4, 64), (65, 1, 1, 8, 4, 64),
])
def test_chunked_form_matches_token_form(L, Hq, Hv, dk, dv, C):
    rng = np.random.default_rng(100 + L)
    q, k, v, g, beta = rand_case(rng, L, Hq, Hv, dk, dv)
    o, st = run(q, k, v, g, beta)
    o2, st2 = chunked_forward(q, k, v, g, beta, [0, L], C)
    np.testing.assert_allclose(o, o2, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(st, st2, rtol=1e-10, atol=1e-12)


def test_chunked_form_varlen_batch():
    rng = np.random.default_rng(5)
    lens = [5, 0, 70, 1, 64]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v, g, beta = rand_case(rng, int(cu[-1]), 2, 4, 8, 8)
    o, st = run(q, k, v, g, beta, cu)
    o2, st2 = chunked_forward(q, k, v, g, beta, cu, 16)
    np.testing.assert_allclose(o, o2, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(st, st2, rtol=1e-10, atol=1e-12)
    assert np.all(st[1] == 0)                                      # zero-length request: zero state


# --- P5: resume identity and the contraction (alpha-product) bound ---------------------------

def test_resume_identity_and_alpha_product_bound():
    rng = np.random.default_rng(6)
    m, tail, Hq, Hv, dk, dv = 400, 120, 2, 4, 16, 16
    q, k, v, g, beta = rand_case(rng, m, Hq, Hv, dk, dv)
    g = rng.uniform(-0.004, -0.0002, g.shape).astype(np.float32)   # weak decay: the bound has teeth
    cut = m - tail
    _, s_full = run(q, k, v, g, beta)
    _, s_prefix = run(q[:cut], k[:cut], v[:cut], g[:cut], beta[:cut])
    _, s_tail = run(q[cut:], k[cut:], v[cut:], g[cut:], beta[cut:])
    _, s_resumed = run(q[cut:], k[cut:], v[cut:], g[cut:], beta[cut:], init=s_prefix)
    np.testing.assert_allclose(s_resumed, s_full, rtol=1e-12, atol=1e-14)
    # unit keys (|k|^2 <= 1 + 1e-6 after fp32 rounding) and beta in (0,1): each (I - beta k k^T)
    # is a contraction, so ||S_full - S_tail||_F <= prod(alpha over the replayed tail) ||S_prefix||_F
    for h in range(Hv):
        prod_alpha = np.exp(np.sum(g[cut:, h].astype(np.float64)))
        diff = np.linalg.norm(s_full[0, h] - s_tail[0, h])
        bound = prod_alpha * np.linalg.norm(s_prefix[0, h])
        assert diff <= bound * (1 + 1e-5)
        assert diff > 0
    # tail of length 0: the difference is the whole prefix state (empty product = 1)
    _, s_none = run(q[:0], k[:0], v[:0], g[:0], beta[:0])
    assert np.all(s_none == 0)


# --- P6: closed form for orthonormal keys (fixes the state layout H = S^T) --------------------

def test_orthonormal_keys_closed_form():
    rng = np.random.default_rng(7)
    dk, dv = 8, 5
    L = dk
    perm = rng.permutation(dk)
    k = np.zeros((L, 1, dk), dtype=np.float32)
    k[np.arange(L), 0, perm] = 1.0
    q = rng.standard_normal((L, 1, dk)).astype(np.float32)
    v = rng.standard_normal((L, 1, dv)).astype(np.float32)
    g = rng.uniform(-0.5, -0.01, (L, 1)).astype(np.float32)
    beta = rng.uniform(0.1, 0.9, (L, 1)).astype(np.float32)
    o, st = run(q, k, v, g, beta)
    a = np.exp(g[:, 0].astype(np.float64))
    H = np.zeros((dk, dv))
    for i in range(L):
        H[perm[i]] = np.prod(a[i + 1:]) * np.float64(beta[i, 0]) * v[i, 0].astype(np.float64)
    np.testing.assert_allclose(st[0, 0], H, rtol=1e-13, atol=1e-15)
    for t in range(L):
        ot = np.zeros(dv)
        for i in range(t + 1):
            ot += np.prod(a[i + 1:t + 1]) * np.float64(beta[i, 0]) * np.float64(q[t, 0, perm[i]]) * v[i, 0].astype(np.float64)
        np.testing.assert_allclose(o[t, 0], ot, rtol=1e-12, atol=1e-14)


# --- P7: repeated unit key, alpha = 1: exponential moving average of v ------------------------

def test_repeated_key_is_moving_average():
    rng = np.random.default_rng(8)
    L, dk, dv = 25, 4, 3
    kvec = np.array([0.5, 0.5, 0.5, 0.5], dtype=np.float32)      # exactly unit in fp32
    k = np.tile(kvec, (L, 1, 1))
    q = k.copy()
    v = rng.standard_normal((L, 1, dv)).astype(np.float32)
    beta = rng.uniform(0.1, 0.9, (L, 1)).astype(np.float32)
    o, _ = run(q, k, v, np.zeros((L, 1), dtype=np.float32), beta)
    ema = np.zeros(dv)
    for t in range(L):
        b = np.float64(beta[t, 0])
        ema = (1 - b) * ema + b * v[t, 0].astype(np.float64)
        np.testing.assert_allclose(o[t, 0], ema, rtol=1e-13, atol=1e-15)


# --- P8: linear in v ---------------------------------------------------------------------------

def test_linear_in_v():
    rng = np.random.default_rng(9)
    q, k, v, g, beta = rand_case(rng, 40, 1, 2, 8, 8)
    v2 = rng.standard_normal(v.shape).astype(np.float32)
    o1, s1 = run(q, k, v, g, beta)
    o2, s2 = run(q, k, v2, g, beta)
    vs = (2.0 * v.astype(np.float64) - 3.0 * v2.astype(np.float64))
    # the combination is not exactly representable in fp32; run it through the chunked fp64 form
    o3, s3 = chunked_forward(q, k, vs, g, beta, [0, 40], 8)
    np.testing.assert_allclose(2 * o1 - 3 * o2, o3, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(2 * s1 - 3 * s2, s3, rtol=1e-10, atol=1e-12)


# --- head mapping, batching, permutation ---------------------------------------------------------

def test_v_head_reads_qk_head_h_div_group():
    rng = np.random.default_rng(10)
    L, Hq, Hv, dk, dv = 20, 2, 6, 4, 4
    q, k, v, g, beta = rand_case(rng, L, Hq, Hv, dk, dv)
    o, st = run(q, k, v, g, beta)
    for h in range(Hv):
        hq = h // (Hv // Hq)                                        # consecutive v-heads share a q/k head
        o1, s1 = run(q[:, hq:hq + 1], k[:, hq:hq + 1], v[:, h:h + 1], g[:, h:h + 1], beta[:, h:h + 1])
        np.testing.assert_array_equal(o[:, h], o1[:, 0])
        np.testing.assert_array_equal(st[0, h], s1[0, 0])
    # an interleaved mapping (h % Hq) would give something else
    o_wrong, _ = run(q[:, 1:2], k[:, 1:2], v[:, 1:2], g[:, 1:2], beta[:, 1:2])
    assert np.abs(o_wrong[:, 0] - o[:, 1]).max() > 1e-3


def test_requests_are_independent_of_batching():
    rng = np.random.default_rng(11)
    lens = [13, 40, 7]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v, g, beta = rand_case(rng, int(cu[-1]), 1, 2, 8, 8)
    o, st = run(q, k, v, g, beta, cu)
    for n in range(3):
        a, b = cu[n], cu[n + 1]
        o1, s1 = run(q[a:b], k[a:b], v[a:b], g[a:b], beta[a:b])
        np.testing.assert_array_equal(o[a:b], o1)
        np.testing.assert_array_equal(st[n], s1[0])


def test_threads_do_not_change_result():
    inp = make_inputs([33, 70], 2, 4, 16, 16, "bf16", seed=5)
    o1, s1 = oracle.gdn_forward_inputs(inp, threads=1)
    o8, s8 = oracle.gdn_forward_inputs(inp, threads=8)
    np.testing.assert_array_equal(o1, o8)
    np.testing.assert_array_equal(s1, s8)


def test_config0_scale_statistics():
    """Sanity on the named tiny configuration: finite, and of the magnitude the tolerances assume."""
    inp = config_tiny_f32()
    o, st = oracle.gdn_forward_inputs(inp)
    assert o.shape == (512, 4, 64) and st.shape == (1, 4, 64, 64)
    assert np.isfinite(o).all() and np.isfinite(st).all()
    assert 1.0 < np.linalg.norm(st[0, 0]) < 100.0
    o2, st2 = chunked_forward(inp.q, inp.k, inp.v, inp.g, inp.beta, inp.cu_tail_lens, 64)
    np.testing.assert_allclose(o, o2, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(st, st2, rtol=1e-9, atol=1e-11)


def test_oracle_rejects_bad_arguments():
    with pytest.raises(ValueError):
        z = np.zeros((2, 1, 4), dtype=np.float32)
        oracle.gdn_forward(z, z, z, np.zeros((2, 1), np.float32), np.zeros((2, 1), np.float32),
                           np.array([0, 3, 2], dtype=np.int32))


# --- replay-window arithmetic ------------------------------------------------------------------

def test_tail_select_table():
    for line in open(os.path.join(GOLD, "tail_select_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        m, r, k = line.split()
        assert oracle.tail_select(int(m), float(r)) == int(k), line


def test_tail_select_matches_integer_ceiling():
    for m in list(range(0, 400)) + [8192, 16384, 32768, 131072, 31366, 31847]:
        for pct in range(0, 101):
            assert oracle.tail_select(m, pct / 100.0) == -(-m * pct // 100)


def test_tail_select_errors():
    assert oracle.tail_select(-1, 0.05) == -1
    assert oracle.tail_select(10, -0.1) == -1
    assert oracle.tail_select(10, float("nan")) == -1


# ---- the input stage in front of the recurrence (oracle.prologue) -------------------------------------

def test_prologue_hand_values_and_identities():
    """3-4-5 triangle, sigmoid symmetry, log-sigmoid at 0 and far out, scale invariance of the normalisation."""
    q = np.array([[[3.0, 4.0]]]); k = np.array([[[0.0, -2.0]]])
    a = np.array([[0.0, 40.0, -40.0]]); b = np.array([[0.0, 1.5, -1.5]])
    qn, kn, g, beta = oracle.prologue(q, k, a, b, eps=0.0)
    np.testing.assert_allclose(qn, [[[0.6, 0.8]]], rtol=0, atol=1e-15)
    np.testing.assert_allclose(kn, [[[0.0, -1.0]]], rtol=0, atol=1e-15)
    np.testing.assert_allclose(g[0, 0], -np.log(2.0), rtol=1e-15)
    assert abs(g[0, 1]) < 1e-17 and abs(g[0, 2] + 40.0) < 1e-15          # log sigmoid(a): ~0 far right, ~a far left
    assert beta[0, 0] == 0.5 and abs(beta[0, 1] + beta[0, 2] - 1.0) < 1e-15
    rng = np.random.default_rng(1)
    x = rng.standard_normal((5, 3, 16))
    n1 = oracle.prologue(x, x, np.zeros((5, 2)), np.zeros((5, 2)), eps=0.0)[0]
    n2 = oracle.prologue(7.5 * x, x, np.zeros((5, 2)), np.zeros((5, 2)), eps=0.0)[0]
    np.testing.assert_allclose(n1, n2, rtol=1e-14)
    np.testing.assert_allclose(np.sum(n1 * n1, axis=-1), 1.0, rtol=1e-14)
    aa = rng.standard_normal((4, 3)) * 3
    ga = oracle.prologue(x[:4], x[:4], aa, aa)[2]
    gb = oracle.prologue(x[:4], x[:4], -aa, aa)[2]
    np.testing.assert_allclose(np.exp(ga) + np.exp(gb), 1.0, rtol=1e-14)  # sigmoid(a) + sigmoid(-a) = 1


def test_prologue_composed_with_recurrence_reduces_to_ready_inputs():
    """Feeding ready-made inputs through the stage changes nothing it should not: unit-norm q, k stay (eps = 0), the
    logit of alpha gives back g, the logit of beta gives back beta; and the fp64-input entry of the recurrence is the
    same routine as the fp32-input one (bitwise on fp32-representable values)."""
    inp = make_inputs([23, 0, 9], 2, 4, 8, 4, "f32", seed=77)
    alpha = np.exp(inp.g.astype(np.float64)); beta = inp.beta.astype(np.float64)
    qn, kn, g, b = oracle.prologue(inp.q, inp.k, np.log(alpha / (1 - alpha)), np.log(beta / (1 - beta)), eps=0.0)
    np.testing.assert_allclose(g, inp.g.astype(np.float64), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(b, beta, rtol=1e-12)
    o1, s1 = oracle.gdn_forward_inputs(inp)
    o2, s2 = oracle.gdn_forward_f64(inp.q, inp.k, inp.v, inp.g, inp.beta, inp.cu_tail_lens)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(s1, s2)
    o3, s3 = oracle.gdn_forward_f64(qn, kn, inp.v, g, b, inp.cu_tail_lens)
    np.testing.assert_allclose(o3, o1, rtol=0, atol=1e-6)                 # q, k of the recipe are unit rows up to fp32 rounding
    np.testing.assert_allclose(s3, s1, rtol=0, atol=1e-6)
