"""Seeded synthetic inputs shaped like the paper's workloads (Llama-2-7B, Llama-3-8B,
Mistral-7B attention layers at 4k-32k context, Section 4.1 / Table 1 / Table 2).

This module only *draws data*: it holds none of the method's arithmetic, and both
the CUDA path and the CPU oracle are fed from it.  numpy only; no torch import.

Recipe, per unit (sequence b, kv head h) with a counter-based Philox stream keyed by
(seed, layer, unit, purpose):
  * anchor a ~ N(0, I_d);
  * keys ~ N(0,1), four outlier channels (drawn per unit) multiplied by 8;
    values ~ N(0,1);
  * n_hh "heavy-hitter" rows overwritten by r*(0.6 a^ + 0.8 z^), z^ a random unit
    vector orthogonal to a^, r the mean key norm (cosine 0.6 to the anchor);
  * queries q_{t,g} = 0.9 a + sqrt(0.19) eps_{t,g}; eps iid N(0,I), or AR(1) in t
    with coefficient rho (slow drift) when the workload asks for it;
  * appended tokens: keys from the same key law (no new heavy hitters), values N(0,1);
  * everything is rounded to bf16 (round-to-nearest-even) before anyone sees it.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H_q: int
    H_kv: int
    d: int
    N: int                      # initial context (max over sequences when ragged)
    budget_ratio: float
    period: int                 # compression period P (decode steps)
    steps: int                  # decode steps of the protocol
    n_hh: int                   # planted heavy hitters per unit
    seed: int
    ar_rho: float = 0.0         # AR(1) coefficient of the query noise (0 = iid)
    n_min: int = 0              # ragged lengths uniform in [n_min, N] when > 0
    layers: int = 1
    n_sink: int = 4
    recent_frac: float = 0.8    # recent : heavy = 4 : 1 of the budget left after the sinks

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def U(self) -> int:
        return self.B * self.H_kv

    def budget(self, n: int | None = None) -> int:
        """Entries kept: floor(ratio * N + 1/2) (ratio = budget / prompt length)."""
        n = self.N if n is None else n
        return int(np.floor(self.budget_ratio * n + 0.5))

    def n_recent(self, b: int | None = None) -> int:
        b = self.budget() if b is None else b
        return int(np.floor(self.recent_frac * max(b - self.n_sink, 0)))


CONFIGS = {
    # tiny correctness case: one compression, 32 decode steps
    "C1": Workload("C1", B=1, H_q=8, H_kv=2, d=64, N=512, budget_ratio=0.10, period=32, steps=32, n_hh=16, seed=0),
    # Llama-3-8B-shaped layer
    "C2": Workload("C2", B=8, H_q=32, H_kv=8, d=128, N=8192, budget_ratio=0.20, period=128, steps=1024, n_hh=64,
                   seed=1000),
    # Llama-2-7B-shaped MHA layer, slowly drifting queries
    "C3": Workload("C3", B=16, H_q=32, H_kv=32, d=128, N=4096, budget_ratio=0.10, period=64, steps=512, n_hh=64,
                   seed=2000, ar_rho=0.95),
    # Mistral-7B-shaped long context, 32 layers with independent seeds
    "C4": Workload("C4", B=2, H_q=32, H_kv=8, d=128, N=32768, budget_ratio=0.10, period=256, steps=512, n_hh=64,
                   seed=3000, layers=32),
    # serving-scale decode with ragged lengths
    "C5": Workload("C5", B=64, H_q=64, H_kv=8, d=128, N=16384, budget_ratio=0.10, period=128, steps=2048, n_hh=64,
                   seed=4000, n_min=4096),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller/larger variant of a workload with the same recipe."""
    return replace(w, **kw)


# ------------------------------------------------------------------ bf16 helpers

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array rounded onto the bf16 grid (still float32)."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# ------------------------------------------------------------------ generators

_PROFILE, _KEYS, _VALUES, _QUERIES, _APPEND, _LENGTHS = range(6)


def _rng(w: Workload, layer: int, unit: int, purpose: int) -> np.random.Generator:
    key = ((int(w.seed) + int(layer)) << 40) | ((int(unit) & 0xFFFFFF) << 8) | int(purpose)
    return np.random.Generator(np.random.Philox(key=key))


def seq_lens(w: Workload, layer: int = 0) -> np.ndarray:
    """Initial context length per sequence, int32 [B]."""
    if w.n_min <= 0:
        return np.full(w.B, w.N, dtype=np.int32)
    g = _rng(w, layer, 0, _LENGTHS)
    return g.integers(w.n_min, w.N + 1, size=w.B).astype(np.int32)


def unit_profile(w: Workload, layer: int, unit: int) -> dict:
    g = _rng(w, layer, unit, _PROFILE)
    a = g.standard_normal(w.d).astype(np.float32)
    ch = g.choice(w.d, size=4, replace=False)
    z = g.standard_normal(w.d).astype(np.float32)
    a_hat = a / np.linalg.norm(a)
    z = z - (z @ a_hat) * a_hat
    z_hat = z / np.linalg.norm(z)
    return dict(anchor=a, a_hat=a_hat, z_seed=z_hat, outlier_channels=np.sort(ch))


def _draw_keys(g: np.random.Generator, n: int, d: int, channels: np.ndarray) -> np.ndarray:
    k = g.standard_normal((n, d), dtype=np.float32)
    k[:, channels] *= 8.0
    return k


def make_unit(w: Workload, layer: int, unit: int, n: int) -> dict:
    """Prompt cache of one unit: K, V float32 [n, d] holding bf16 values."""
    prof = unit_profile(w, layer, unit)
    gk = _rng(w, layer, unit, _KEYS)
    K = _draw_keys(gk, n, w.d, prof["outlier_channels"])
    rbar = float(np.mean(np.linalg.norm(K, axis=1))) if n > 0 else 0.0
    n_hh = min(w.n_hh, n)
    if n_hh > 0:
        rows = np.sort(gk.choice(n, size=n_hh, replace=False))
        z = gk.standard_normal((n_hh, w.d)).astype(np.float32)
        z -= np.outer(z @ prof["a_hat"], prof["a_hat"])
        z /= np.linalg.norm(z, axis=1, keepdims=True)
        K[rows] = rbar * (0.6 * prof["a_hat"][None, :] + 0.8 * z)
    else:
        rows = np.zeros(0, dtype=np.int64)
    V = _rng(w, layer, unit, _VALUES).standard_normal((n, w.d), dtype=np.float32)
    return dict(K=round_bf16(K), V=round_bf16(V), hh_rows=rows, anchor=prof["anchor"])


def make_queries(w: Workload, layer: int, unit: int, t0: int, t1: int) -> np.ndarray:
    """Queries of the unit's G heads for decode steps t0..t1-1: float32 [t1-t0, G, d], bf16 values."""
    prof = unit_profile(w, layer, unit)
    g = _rng(w, layer, unit, _QUERIES)
    eta = g.standard_normal((t1, w.G, w.d), dtype=np.float32)   # drawn from step 0 so any window is reproducible
    if w.ar_rho > 0.0:
        eps = np.empty_like(eta)
        eps[0] = eta[0]
        c = np.float32(np.sqrt(1.0 - w.ar_rho ** 2))
        for t in range(1, t1):
            eps[t] = np.float32(w.ar_rho) * eps[t - 1] + c * eta[t]
    else:
        eps = eta
    q = np.float32(0.9) * prof["anchor"][None, None, :] + np.float32(np.sqrt(0.19)) * eps
    return round_bf16(q[t0:t1])


def make_appends(w: Workload, layer: int, unit: int, t0: int, t1: int):
    """New tokens' key/value rows for decode steps t0..t1-1: two float32 [t1-t0, d] arrays."""
    prof = unit_profile(w, layer, unit)
    g = _rng(w, layer, unit, _APPEND)
    k = _draw_keys(g, t1, w.d, prof["outlier_channels"])
    v = g.standard_normal((t1, w.d), dtype=np.float32)
    return round_bf16(k[t0:t1]), round_bf16(v[t0:t1])


def make_cache(w: Workload, layer: int = 0, n_cap: int | None = None, units=None):
    """Whole prompt cache as bf16 bit patterns: K, V uint16 [U, n_cap, d] (rows past a
    sequence's length are zero), seq_len int32 [B].  ``units`` restricts generation to a
    subset of unit indices (the others stay zero)."""
    lens = seq_lens(w, layer)
    n_cap = int(n_cap if n_cap is not None else w.N + w.period)
    K = np.zeros((w.U, n_cap, w.d), dtype=np.uint16)
    V = np.zeros((w.U, n_cap, w.d), dtype=np.uint16)
    for u in (range(w.U) if units is None else units):
        n = int(lens[u // w.H_kv])
        c = make_unit(w, layer, u, n)
        K[u, :n] = f32_to_bf16_bits(c["K"])
        V[u, :n] = f32_to_bf16_bits(c["V"])
    return K, V, lens


def make_step_inputs(w: Workload, layer: int, t0: int, t1: int):
    """Queries and appended rows for all units and steps t0..t1-1, as bf16 bit patterns:
    q uint16 [T, B, H_q, d], k_new, v_new uint16 [T, B, H_kv, d]."""
    T = t1 - t0
    q = np.empty((T, w.B, w.H_q, w.d), dtype=np.uint16)
    kn = np.empty((T, w.B, w.H_kv, w.d), dtype=np.uint16)
    vn = np.empty((T, w.B, w.H_kv, w.d), dtype=np.uint16)
    for u in range(w.U):
        b, h = divmod(u, w.H_kv)
        q[:, b, h * w.G:(h + 1) * w.G, :] = f32_to_bf16_bits(make_queries(w, layer, u, t0, t1))
        k, v = make_appends(w, layer, u, t0, t1)
        kn[:, b, h, :] = f32_to_bf16_bits(k)
        vn[:, b, h, :] = f32_to_bf16_bits(v)
    return q, kn, vn
