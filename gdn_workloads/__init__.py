"""Seeded synthetic inputs for the GDN tail-replay path.

This module is the only code shared by the CUDA path and the CPU oracle.  It
holds none of the method's arithmetic: it draws random numbers, normalises keys
and queries (the caller's job in a real model), rounds to the storage dtype and
lays the arrays out as the C-ABI expects them.

Recipe (per token, per head), following the configurations the benchmark names:
    q, k ~ N(0,1), L2-normalised over the head dimension in fp32, then rounded
           to the io dtype;
    v    ~ N(0,1), rounded to the io dtype;
    g    = log(alpha) ~ U(g_lo, g_hi)   (fp32, <= 0);
    beta = sigmoid(N(0,1))              (fp32, in (0,1)).
The matched-prefix lengths and replay budgets are those of the paper's
serving-efficiency table (8K/16K/32K prefixes, 5 % and 10 % budgets); the
dataset the paper drew its prefixes from is not available, so only shapes and
distributions are imitated.

Layouts (row-major, packed varlen, no batch dimension):
    q, k   [T, Hq, dk]      v [T, Hv, dv]      g, beta [T, Hv]
    cu_tail_lens [N+1] int32 prefix sums of the tail lengths, cu[0] = 0.
bf16 arrays are carried as uint16 bit patterns (numpy has no bf16) next to an
exactly-widened fp32 copy, so both sides read the same stored values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

BASE_SEED = 2608030310

__all__ = [
    "BASE_SEED", "GdnInputs", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "make_inputs", "make_raw_inputs", "tail_lengths_uniform", "config_tiny_f32", "config_single_layer",
    "config_budget_sweep_tails", "config_budget_sweep_layer", "config_concurrent_hits", "config_full_prefill",
    "PAPER_PREFIX_LENGTHS", "NOMINAL_PREFIX_LENGTHS", "REPLAY_BUDGETS",
]

# Matched-prefix lengths printed in the paper's TTFT table, and the nominal ones.
PAPER_PREFIX_LENGTHS = (8225, 8226, 16417, 16418, 31366, 31847)
NOMINAL_PREFIX_LENGTHS = (8192, 16384, 32768)
REPLAY_BUDGETS = (0.05, 0.10)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class GdnInputs:
    """One batch of packed varlen GDN inputs.

    ``q, k, v`` hold the values both sides compute with, as fp32 (for bf16 io
    they are exactly the widened bf16 values).  ``q_bits, k_bits, v_bits`` are
    the uint16 bf16 patterns when ``io_dtype == 'bf16'`` and None otherwise.
    """
    q: np.ndarray
    k: np.ndarray
    v: np.ndarray
    g: np.ndarray
    beta: np.ndarray
    cu_tail_lens: np.ndarray
    num_qk_heads: int
    num_v_heads: int
    head_k_dim: int
    head_v_dim: int
    io_dtype: str
    q_bits: Optional[np.ndarray] = None
    k_bits: Optional[np.ndarray] = None
    v_bits: Optional[np.ndarray] = None
    meta: Dict[str, object] = field(default_factory=dict)

    @property
    def num_seqs(self) -> int:
        return int(self.cu_tail_lens.shape[0] - 1)

    @property
    def total_tokens(self) -> int:
        return int(self.cu_tail_lens[-1])

    def tail_lens(self) -> np.ndarray:
        return np.diff(self.cu_tail_lens)

    def take_chain(self, n: int, h: int) -> "GdnInputs":
        """The single chain (request n, v-head h) as a 1-request, 1-head batch."""
        G = self.num_v_heads // self.num_qk_heads
        a, b = int(self.cu_tail_lens[n]), int(self.cu_tail_lens[n + 1])
        hq = h // G
        sub = GdnInputs(
            q=np.ascontiguousarray(self.q[a:b, hq:hq + 1]),
            k=np.ascontiguousarray(self.k[a:b, hq:hq + 1]),
            v=np.ascontiguousarray(self.v[a:b, h:h + 1]),
            g=np.ascontiguousarray(self.g[a:b, h:h + 1]),
            beta=np.ascontiguousarray(self.beta[a:b, h:h + 1]),
            cu_tail_lens=np.array([0, b - a], dtype=np.int32),
            num_qk_heads=1, num_v_heads=1,
            head_k_dim=self.head_k_dim, head_v_dim=self.head_v_dim,
            io_dtype=self.io_dtype, meta=dict(self.meta, chain=(n, h)),
        )
        return sub

    def take_rows(self, start: int, stop: int) -> "GdnInputs":
        """Rows [start, stop) of a single-request batch as a new single request."""
        assert self.num_seqs == 1

        def cut(x):
            return None if x is None else np.ascontiguousarray(x[start:stop])
        return GdnInputs(
            q=cut(self.q), k=cut(self.k), v=cut(self.v), g=cut(self.g), beta=cut(self.beta),
            cu_tail_lens=np.array([0, stop - start], dtype=np.int32),
            num_qk_heads=self.num_qk_heads, num_v_heads=self.num_v_heads,
            head_k_dim=self.head_k_dim, head_v_dim=self.head_v_dim, io_dtype=self.io_dtype,
            q_bits=cut(self.q_bits), k_bits=cut(self.k_bits), v_bits=cut(self.v_bits),
            meta=dict(self.meta, rows=(start, stop)),
        )


def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(size=shape, dtype=np.float32)


def _unit_rows(x: np.ndarray) -> np.ndarray:
    n = np.sqrt(np.sum(x.astype(np.float32) ** 2, axis=-1, keepdims=True, dtype=np.float32))
    return (x / np.maximum(n, np.float32(1e-20))).astype(np.float32)


def make_inputs(tail_lens: Sequence[int], num_qk_heads: int, num_v_heads: int,
                head_k_dim: int, head_v_dim: int, io_dtype: str = "bf16",
                seed: int = BASE_SEED, g_lo: float = -0.1, g_hi: float = -0.001,
                meta: Optional[Dict[str, object]] = None) -> GdnInputs:
    """Draw one batch with the recipe in the module docstring."""
    assert io_dtype in ("bf16", "f32")
    assert num_v_heads % num_qk_heads == 0
    lens = np.asarray(list(tail_lens), dtype=np.int64)
    assert (lens >= 0).all()
    cu = np.zeros(len(lens) + 1, dtype=np.int64)
    np.cumsum(lens, out=cu[1:])
    assert cu[-1] < 2 ** 31
    T = int(cu[-1])
    rng = np.random.Generator(np.random.Philox(key=int(seed)))
    q = _unit_rows(_normal(rng, (T, num_qk_heads, head_k_dim)))
    k = _unit_rows(_normal(rng, (T, num_qk_heads, head_k_dim)))
    v = _normal(rng, (T, num_v_heads, head_v_dim))
    g = rng.uniform(g_lo, g_hi, size=(T, num_v_heads)).astype(np.float32)
    z = _normal(rng, (T, num_v_heads))
    beta = (1.0 / (1.0 + np.exp(-z.astype(np.float64)))).astype(np.float32)
    qb = kb = vb = None
    if io_dtype == "bf16":
        qb, kb, vb = f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)
        q, k, v = bf16_bits_to_f32(qb), bf16_bits_to_f32(kb), bf16_bits_to_f32(vb)
    m = {"seed": int(seed), "g_range": (g_lo, g_hi)}
    if meta:
        m.update(meta)
    return GdnInputs(q=q, k=k, v=v, g=g, beta=beta, cu_tail_lens=cu.astype(np.int32),
                     num_qk_heads=num_qk_heads, num_v_heads=num_v_heads,
                     head_k_dim=head_k_dim, head_v_dim=head_v_dim, io_dtype=io_dtype,
                     q_bits=qb, k_bits=kb, v_bits=vb, meta=m)


def make_raw_inputs(tail_lens: Sequence[int], num_qk_heads: int, num_v_heads: int,
                    head_k_dim: int, head_v_dim: int, io_dtype: str = "bf16",
                    seed: int = BASE_SEED, gate_lo: float = 2.2, gate_hi: float = 7.0) -> GdnInputs:
    """One batch of RAW projection outputs for the fused input stage: q, k ~ N(0, s^2) with a per-token scale
    s ~ U(0.5, 3) and no normalisation, v ~ N(0,1), the gate pre-activation ~ U(gate_lo, gate_hi) (sigmoid of it
    in about (0.90, 0.999), the range of the ready-made recipe) and the beta pre-activation ~ N(0,1).  The fields
    ``q, k, g, beta`` of the result hold these raw values; nothing here applies the input stage."""
    assert io_dtype in ("bf16", "f32")
    lens = np.asarray(list(tail_lens), dtype=np.int64)
    cu = np.zeros(len(lens) + 1, dtype=np.int64)
    np.cumsum(lens, out=cu[1:])
    T = int(cu[-1])
    rng = np.random.Generator(np.random.Philox(key=int(seed) ^ 0x0A57A6E))
    sq = rng.uniform(0.5, 3.0, size=(T, num_qk_heads, 1)).astype(np.float32)
    sk = rng.uniform(0.5, 3.0, size=(T, num_qk_heads, 1)).astype(np.float32)
    q = _normal(rng, (T, num_qk_heads, head_k_dim)) * sq
    k = _normal(rng, (T, num_qk_heads, head_k_dim)) * sk
    v = _normal(rng, (T, num_v_heads, head_v_dim))
    gate = rng.uniform(gate_lo, gate_hi, size=(T, num_v_heads)).astype(np.float32)
    braw = _normal(rng, (T, num_v_heads))
    qb = kb = vb = None
    if io_dtype == "bf16":
        qb, kb, vb = f32_to_bf16_bits(q), f32_to_bf16_bits(k), f32_to_bf16_bits(v)
        q, k, v = bf16_bits_to_f32(qb), bf16_bits_to_f32(kb), bf16_bits_to_f32(vb)
    return GdnInputs(q=q, k=k, v=v, g=gate, beta=braw, cu_tail_lens=cu.astype(np.int32),
                     num_qk_heads=num_qk_heads, num_v_heads=num_v_heads,
                     head_k_dim=head_k_dim, head_v_dim=head_v_dim, io_dtype=io_dtype,
                     q_bits=qb, k_bits=kb, v_bits=vb, meta={"seed": int(seed), "raw": True})


def tail_lengths_uniform(num_seqs: int, lo: int, hi: int, seed: int) -> List[int]:
    """Integer tail lengths ~ U{lo..hi}, seeded."""
    rng = np.random.Generator(np.random.Philox(key=int(seed) ^ 0x5EED))
    return [int(x) for x in rng.integers(lo, hi + 1, size=num_seqs)]


# --- the five named configurations -------------------------------------------------------

def config_tiny_f32(seed_offset: int = 0) -> GdnInputs:
    """Config 0: 1 request, 4 heads, dk = dv = 64, tail 512, fp32 io."""
    return make_inputs([512], 4, 4, 64, 64, "f32", seed=BASE_SEED + seed_offset,
                       meta={"config": 0})


def config_single_layer(seed_offset: int = 0, tail: int = 1638) -> GdnInputs:
    """Config 1: 1 request, 16 q/k heads shared by 32 v heads, dk = dv = 128, bf16, tail 1,638."""
    return make_inputs([tail], 16, 32, 128, 128, "bf16", seed=BASE_SEED + 1000 + seed_offset,
                       meta={"config": 1})


def config_budget_sweep_tails() -> List[Dict[str, int]]:
    """Config 2: (prefix, budget) grid; tails come from ceil(r*m) over the nominal prefixes."""
    out = []
    for m in NOMINAL_PREFIX_LENGTHS:
        for r_pct in (5, 10):
            # integer arithmetic: ceil(m * pct / 100); 8192 -> 410/820, 32768 -> 1639/3277
            out.append({"prefix": m, "budget_pct": r_pct, "tail": -(-m * r_pct // 100)})
    return out


def config_budget_sweep_layer(tail: int, layer: int) -> GdnInputs:
    """Config 2: one of the 36 layers of a batch-1 rebuild, fresh seeded inputs per layer."""
    return make_inputs([tail], 16, 32, 128, 128, "bf16", seed=BASE_SEED + 2000 + layer,
                       meta={"config": 2, "layer": layer})


def config_concurrent_hits(num_seqs: int = 32, lo: int = 400, hi: int = 3300,
                           seed_offset: int = 0) -> GdnInputs:
    """Config 3: 32 requests packed varlen, tails ~ U{400..3300}, 16/32 heads, d = 128, bf16."""
    seed = BASE_SEED + 3000 + seed_offset
    lens = tail_lengths_uniform(num_seqs, lo, hi, seed)
    return make_inputs(lens, 16, 32, 128, 128, "bf16", seed=seed, meta={"config": 3})


def config_full_prefill(prefix_len: int = 32768, seed_offset: int = 0,
                        g_lo: float = -0.1, g_hi: float = -0.001,
                        num_qk_heads: int = 16, num_v_heads: int = 32) -> GdnInputs:
    """Config 4: zero-state forward over a whole prefix (32K or 128K tokens), 16/32 heads, bf16."""
    return make_inputs([prefix_len], num_qk_heads, num_v_heads, 128, 128, "bf16",
                       seed=BASE_SEED + 4000 + seed_offset, g_lo=g_lo, g_hi=g_hi,
                       meta={"config": 4})
