"""KeepKV CPU oracle -- TEST INFRASTRUCTURE, not part of the product path.

Thin ctypes/numpy binding over ``keepkv_oracle.c`` (plain C, fp64).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and this package never touches the CUDA
library.  All arrays are float64 (cache, votes, lscore, queries) or int32.

Every function works on ONE unit = one (sequence, kv-head) pair unless its name
ends in ``_batch``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "keepkv_oracle.c")
_SO = os.path.join(_HERE, "libkeepkv_oracle.so")


def _cpu_has_fma() -> bool:
    try:
        with open("/proc/cpuinfo") as f:
            return " fma " in f.read().replace("\n", " ")
    except OSError:
        return False


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no contraction: fmaf is the only fused op)."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared"]
        if _cpu_has_fma():
            cmd.append("-mfma")
        cmd += ["-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


class _Params(C.Structure):
    _fields_ = [
        ("G", C.c_int32), ("d", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32),
        ("storage_faithful", C.c_int32), ("pad_", C.c_int32),
        ("sm_scale", C.c_double), ("ema_alpha", C.c_double), ("merge_threshold", C.c_double),
        ("gamma_min", C.c_double), ("gamma_max", C.c_double),
    ]


class _Stats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_retained", "n_evicted", "n_merged", "n_below_T", "n_guard_groups", "n_groups", "max_group", "pad_")]


STATS_DTYPE = np.dtype([(n, np.int32) for n in
                        ("n_retained", "n_evicted", "n_merged", "n_below_T", "n_guard_groups", "n_groups",
                         "max_group", "pad_")])


@dataclass
class Params:
    """Per-unit parameters.  Defaults: 4 sinks, T = 0.8 (the paper's settings); no recent window;
    guard (0, 4] on the key rescale factor; ideal (unrounded fp64) storage."""
    G: int
    d: int
    n_sink: int = 4
    n_recent: int = 0
    storage_faithful: bool = False
    sm_scale: float | None = None
    ema_alpha: float = 0.9
    merge_threshold: float = 0.8
    gamma_min: float = 0.0
    gamma_max: float = 4.0

    def c(self) -> _Params:
        s = self.sm_scale if self.sm_scale is not None else 1.0 / np.sqrt(self.d)
        return _Params(self.G, self.d, self.n_sink, self.n_recent, int(self.storage_faithful), 0, s,
                       self.ema_alpha, self.merge_threshold, self.gamma_min, self.gamma_max)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build(force=not _cpu_has_fma())  # a library built with -mfma elsewhere must not run here
        try:
            _lib = C.CDLL(_SO)
        except OSError:
            build(force=True)
            _lib = C.CDLL(_SO)
        _lib.okv_round_bf16.restype = C.c_double
        _lib.okv_round_bf16.argtypes = [C.c_double]
        _lib.okv_cosine.restype = C.c_float
        _lib.okv_merge_group.restype = C.c_double
        for n in ("okv_select", "okv_select_sorted", "okv_compress", "okv_compress_keyed", "okv_merge_similar", "okv_compress_inplace", "okv_append",
                  "okv_num_threads"):
            getattr(_lib, n).restype = C.c_int32
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a, t=C.c_double):
    return a.ctypes.data_as(C.POINTER(t))


def _pi(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def round_bf16(x):
    """Round-to-nearest-even onto the bf16 grid, directly from float64."""
    x = np.asarray(x, dtype=np.float64)
    f = lib().okv_round_bf16
    return np.vectorize(lambda v: f(float(v)), otypes=[np.float64])(x)


def logits(P: Params, q, K):
    q, K = _f64(q), _f64(K)
    n = K.shape[0]
    ell = np.empty((P.G, n), dtype=np.float64)
    cp = P.c()
    lib().okv_logits(C.byref(cp), C.c_int32(n), _p(q), _p(K), _p(ell))
    return ell


def decode(P: Params, q, K, V, votes):
    """Eq. 6 for one unit.  q [G,d], K,V [len,d], votes [len] -> (out [G,d], lse [G])."""
    q, K, V, votes = _f64(q), _f64(K), _f64(V), _f64(votes)
    n = K.shape[0]
    out = np.empty((P.G, P.d), dtype=np.float64)
    lse = np.empty((P.G,), dtype=np.float64)
    cp = P.c()
    lib().okv_decode(C.byref(cp), C.c_int32(n), _p(q), _p(K), _p(V), _p(votes), _p(out), _p(lse))
    return out, lse


def score_update(P: Params, q, K, lscore):
    """Eq. 8 recursive case for one unit; returns the new lscore [len]."""
    q, K = _f64(q), _f64(K)
    ls = _f64(lscore).copy()
    cp = P.c()
    lib().okv_score_update(C.byref(cp), C.c_int32(K.shape[0]), _p(q), _p(K), _p(ls))
    return ls


def prefill_scores(P: Params, q_window, K):
    """Eq. 8 first case for one unit: q_window [W, G, d] (oldest first), K [len, d] -> lscore [len]."""
    q, K = _f64(q_window), _f64(K)
    ls = np.empty(K.shape[0], dtype=np.float64)
    cp = P.c()
    lib().okv_prefill_scores(C.byref(cp), C.c_int32(K.shape[0]), C.c_int32(q.shape[0]), _p(q), _p(K), _p(ls))
    return ls


def kappa(votes, lscore):
    votes, lscore = _f64(votes), _f64(lscore)
    k = np.empty(votes.shape[0], dtype=np.float32)
    lib().okv_kappa(C.c_int32(votes.shape[0]), _p(votes), _p(lscore), _p(k, C.c_float))
    return k


def select(kap, budget: int, n_sink: int, n_recent: int, sorted_impl: bool = False):
    kap = np.ascontiguousarray(kap, dtype=np.float32)
    n = kap.shape[0]
    ret = np.empty(max(n, 1), dtype=np.int32)
    f = lib().okv_select_sorted if sorted_impl else lib().okv_select
    m = f(C.c_int32(n), _p(kap, C.c_float), C.c_int32(budget), C.c_int32(n_sink), C.c_int32(n_recent), _pi(ret))
    return ret[:m].copy()


def cosine(ke, kc):
    ke, kc = _f64(ke), _f64(kc)
    return float(lib().okv_cosine(_p(ke), _p(kc), C.c_int32(ke.shape[0])))


def match(P: Params, K, ret_idx):
    """Algorithm 1, similarity and arg-max steps.  Returns (target [len] int32, umax [len] f32, second [len] f32)."""
    K = _f64(K)
    ret_idx = np.ascontiguousarray(ret_idx, dtype=np.int32)
    n = K.shape[0]
    target = np.empty(max(n, 1), dtype=np.int32)
    umax = np.empty(max(n, 1), dtype=np.float32)
    second = np.empty(max(n, 1), dtype=np.float32)
    cp = P.c()
    lib().okv_match(C.byref(cp), C.c_int32(n), _p(K), C.c_int32(ret_idx.shape[0]), _pi(ret_idx), _pi(target),
                    _p(umax, C.c_float), _p(second, C.c_float))
    return target[:n], umax[:n], second[:n]


def merge_group(d: int, idx, K, V, votes, lscore):
    """Eq. (A.3) with s_hat for the group idx (target included).
    Returns dict(k_r, v_r, p_r, lambda_r, gamma, lambda_bar)."""
    K, V, votes, lscore = _f64(K), _f64(V), _f64(votes), _f64(lscore)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    kr = np.empty(d, dtype=np.float64)
    vr = np.empty(d, dtype=np.float64)
    pr, lr, lb = C.c_double(), C.c_double(), C.c_double()
    g = lib().okv_merge_group(C.c_int32(d), C.c_int32(idx.shape[0]), _pi(idx), _p(K), _p(V), _p(votes), _p(lscore),
                              _p(kr), _p(vr), C.byref(pr), C.byref(lr), C.byref(lb))
    return dict(k_r=kr, v_r=vr, p_r=pr.value, lambda_r=lr.value, gamma=float(g), lambda_bar=lb.value)


def compress(P: Params, budget: int, K, V, votes, lscore, sorted_select: bool = False, select_key=None):
    """Algorithm 1 end to end for one unit.  Returns a dict with the compacted cache
    (K, V, votes, lscore: n_ret rows), ret_idx, target [len], gammas [n_ret], stats.
    select_key: optional fp32 importance scores [len] that replace kappa in the selection (Section 3.4:
    any token selection may designate the retained and evicted sets)."""
    K, V, votes, lscore = _f64(K), _f64(V), _f64(votes), _f64(lscore)
    n, d = K.shape[0], P.d
    m = max(min(n, max(budget, 0)), 1)
    dK = np.zeros((m, d)); dV = np.zeros((m, d)); dv = np.zeros(m); dl = np.zeros(m)
    ret = np.empty(max(n, 1), dtype=np.int32)
    target = np.empty(max(n, 1), dtype=np.int32)
    gam = np.empty(m, dtype=np.float64)
    st = _Stats()
    cp = P.c()
    if select_key is None:
        n_ret = lib().okv_compress(C.byref(cp), C.c_int32(n), C.c_int32(budget), _p(K), _p(V), _p(votes), _p(lscore),
                                   _p(dK), _p(dV), _p(dv), _p(dl), _pi(ret), _pi(target), _p(gam), C.byref(st),
                                   C.c_int32(int(sorted_select)))
    else:
        key = np.ascontiguousarray(select_key, dtype=np.float32)
        assert key.shape == (n,)
        n_ret = lib().okv_compress_keyed(C.byref(cp), C.c_int32(n), C.c_int32(budget), _p(K), _p(V), _p(votes),
                                         _p(lscore), _p(key, C.c_float), _p(dK), _p(dV), _p(dv), _p(dl), _pi(ret),
                                         _pi(target), _p(gam), C.byref(st), C.c_int32(int(sorted_select)))
    return dict(K=dK[:n_ret], V=dV[:n_ret], votes=dv[:n_ret], lscore=dl[:n_ret], ret_idx=ret[:n_ret].copy(),
                target=target[:n].copy(), gammas=gam[:n_ret],
                stats={f: getattr(st, f) for f, _ in _Stats._fields_ if f != "pad_"})


def compress_inplace(P: Params, budget: int, K, V, votes, lscore, pos):
    """Algorithm 1 in place for one unit whose rows are not in token order (pos[i] = token position of row i).
    Returns a dict with the arrays after the call (K, V, votes, lscore, pos: n_ret rows), moved_from [n_ret] (the row
    each final row came from), target [len] (row of the target before the placement, -1, -2), gammas [len], stats."""
    K, V, votes, lscore = (_f64(a).copy() for a in (K, V, votes, lscore))
    pos = np.ascontiguousarray(pos, dtype=np.int32).copy()
    n = K.shape[0]
    m = max(n, 1)
    moved = np.empty(m, dtype=np.int32); target = np.empty(m, dtype=np.int32); gam = np.empty(m, dtype=np.float64)
    st = _Stats()
    cp = P.c()
    n_ret = lib().okv_compress_inplace(C.byref(cp), C.c_int32(n), C.c_int32(budget), _p(K), _p(V), _p(votes), _p(lscore),
                                       _pi(pos), _pi(moved), _pi(target), _p(gam), C.byref(st))
    return dict(K=K[:n_ret], V=V[:n_ret], votes=votes[:n_ret], lscore=lscore[:n_ret], pos=pos[:n_ret],
                moved_from=moved[:n_ret].copy(), target=target[:n].copy(), gammas=gam[:n],
                stats={f: getattr(st, f) for f, _ in _Stats._fields_ if f != "pad_"})


def merge_similar(P: Params, K, V, votes, lscore):
    """Prefill merge-first policy (Section 3.4; App. B, Table 3) for one unit: entries whose most similar other
    key exceeds T are merged into that (earlier) entry; nothing else is evicted.  Returns the same dict as
    compress(): the merged cache (n_ret rows), ret_idx, target [len] (slot for a member, -1 guard, -2 kept),
    gammas, stats."""
    K, V, votes, lscore = _f64(K), _f64(V), _f64(votes), _f64(lscore)
    n, d = K.shape[0], P.d
    m = max(n, 1)
    dK = np.zeros((m, d)); dV = np.zeros((m, d)); dv = np.zeros(m); dl = np.zeros(m)
    ret = np.empty(m, dtype=np.int32)
    target = np.empty(m, dtype=np.int32)
    gam = np.empty(m, dtype=np.float64)
    st = _Stats()
    cp = P.c()
    n_ret = lib().okv_merge_similar(C.byref(cp), C.c_int32(n), _p(K), _p(V), _p(votes), _p(lscore), _p(dK), _p(dV),
                                    _p(dv), _p(dl), _pi(ret), _pi(target), _p(gam), C.byref(st))
    return dict(K=dK[:n_ret], V=dV[:n_ret], votes=dv[:n_ret], lscore=dl[:n_ret], ret_idx=ret[:n_ret].copy(),
                target=target[:n].copy(), gammas=gam[:n_ret],
                stats={f: getattr(st, f) for f, _ in _Stats._fields_ if f != "pad_"})


def append(K, V, votes, lscore, length: int, k_new, v_new) -> int:
    """Eq. 2 in place on capacity-sized arrays; returns the new length."""
    assert K.dtype == np.float64 and K.flags.c_contiguous
    k_new, v_new = _f64(k_new), _f64(v_new)
    return lib().okv_append(C.c_int32(K.shape[1]), C.c_int32(length), _p(K), _p(V), _p(votes), _p(lscore),
                            _p(k_new), _p(v_new))


def decode_batch(P: Params, lens, q, K, V, votes, lscore, update_scores: bool):
    """U units, arrays [U, n_cap, ...]; lscore is updated IN PLACE when update_scores.
    Returns (out [U,G,d], lse [U,G]).  OpenMP over units."""
    for a in (q, K, V, votes, lscore):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    U, n_cap = K.shape[0], K.shape[1]
    out = np.empty((U, P.G, P.d)); lse = np.empty((U, P.G))
    cp = P.c()
    lib().okv_decode_batch(C.byref(cp), C.c_int32(U), C.c_int32(n_cap), _pi(lens), _p(q), _p(K), _p(V), _p(votes),
                           _p(lscore), C.c_int32(int(update_scores)), _p(out), _p(lse))
    return out, lse


def compress_batch(P: Params, lens, budgets, K, V, votes, lscore):
    """U units, arrays [U, n_cap, ...].  Returns dict of dst arrays (same shapes), ret_idx, target,
    new_lens, stats (structured array).  OpenMP over units, sort-based selection."""
    for a in (K, V, votes, lscore):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    budgets = np.ascontiguousarray(budgets, dtype=np.int32)
    U, n_cap = K.shape[0], K.shape[1]
    dK = np.zeros_like(K); dV = np.zeros_like(V); dv = np.zeros_like(votes); dl = np.zeros_like(lscore)
    ret = np.full((U, n_cap), -1, dtype=np.int32)
    target = np.full((U, n_cap), -3, dtype=np.int32)
    new_lens = np.zeros(U, dtype=np.int32)
    stats = np.zeros(U, dtype=STATS_DTYPE)
    cp = P.c()
    lib().okv_compress_batch(C.byref(cp), C.c_int32(U), C.c_int32(n_cap), _pi(lens), _pi(budgets), _p(K), _p(V),
                             _p(votes), _p(lscore), _p(dK), _p(dV), _p(dv), _p(dl), _pi(ret), _pi(target),
                             _pi(new_lens), stats.ctypes.data_as(C.c_void_p))
    return dict(K=dK, V=dV, votes=dv, lscore=dl, ret_idx=ret, target=target, new_lens=new_lens, stats=stats)


def num_threads() -> int:
    return int(lib().okv_num_threads())
