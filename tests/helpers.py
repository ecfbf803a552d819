"""Shared helpers of the GPU parity tests: move data between numpy (oracle side, float64) and
torch CUDA tensors (library side, bf16/fp32), and the comparison rules.

Tolerances (bf16 storage, fp32 accumulation on the GPU, fp64 in the oracle):
  max-abs   |gpu - ref| <= 2e-2 * max(1, |ref|)      (2e-2 absolute near 1; keys carry channels of
                                                      magnitude ~30 where one bf16 ulp is 0.125)
  mean-rel  mean|gpu - ref| / mean|ref| <= 1e-3
  ulp       every stored bf16 value within one bf16 ulp of the oracle's value rounded to bf16
"""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle as O
from paper_2504_09936_b200 import binding as kb
from paper_2504_09936_b200 import workloads as W

MAX_ABS = 2e-2
MEAN_REL = 1e-3


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 CUDA tensor."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def f32_to_dev_bf16(x: np.ndarray) -> torch.Tensor:
    return bits_to_dev(W.f32_to_bf16_bits(np.asarray(x, dtype=np.float32)))


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    ax = np.maximum(np.abs(x), 2.0 ** -6)      # below 1/64 the rule becomes absolute (1.2e-4)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def check_close(gpu: np.ndarray, ref: np.ndarray, what: str, ulps: float | None = 1.0, max_abs=MAX_ABS,
                mean_rel=MEAN_REL):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert gpu.shape == ref.shape, (what, gpu.shape, ref.shape)
    if gpu.size == 0:
        return
    fin = np.isfinite(ref)
    assert np.array_equal(np.isfinite(gpu), fin), f"{what}: non-finite pattern differs"
    assert np.array_equal(gpu[~fin], ref[~fin]), f"{what}: infinities differ"
    g, r = gpu[fin], ref[fin]
    if g.size == 0:
        return
    err = np.abs(g - r)
    worst = np.max(err / np.maximum(1.0, np.abs(r)))
    assert worst <= max_abs, f"{what}: max-abs {worst:.3e} > {max_abs}"
    denom = np.mean(np.abs(r))
    if denom > 0:
        mr = np.mean(err) / denom
        assert mr <= mean_rel, f"{what}: mean-rel {mr:.3e} > {mean_rel}"
    if ulps is not None:
        bad = err > ulps * bf16_ulp(r) * (1 + 1e-9)
        assert not bad.any(), f"{what}: {bad.sum()} of {bad.size} values beyond {ulps} bf16 ulp"


def oracle_params(p: kb.keepkv_params, storage_faithful=True, n_recent=None) -> O.Params:
    return O.Params(G=p.H_q // p.H_kv, d=p.d, n_sink=p.n_sink, n_recent=p.n_recent if n_recent is None else n_recent,
                    storage_faithful=storage_faithful, sm_scale=float(np.float32(p.sm_scale)),
                    ema_alpha=float(np.float32(p.ema_alpha)), merge_threshold=float(p.merge_threshold),
                    gamma_min=float(p.gamma_min), gamma_max=float(p.gamma_max))


class HostCache:
    """float64 mirror of a device cache for the oracle: arrays [U, N_cap, ...]."""

    def __init__(self, cache: kb.Cache):
        B, H, N, d = cache.K.shape
        self.K = to_f64(cache.K).reshape(B * H, N, d)
        self.V = to_f64(cache.V).reshape(B * H, N, d)
        self.votes = to_f64(cache.votes).reshape(B * H, N)
        self.lscore = to_f64(cache.lscore).reshape(B * H, N)
        self.seq_len = cache.seq_len.cpu().numpy().astype(np.int64)
        self.H = H

    def unit(self, u):
        n = int(self.seq_len[u // self.H])
        return self.K[u, :n], self.V[u, :n], self.votes[u, :n], self.lscore[u, :n]


def random_cache(p: kb.keepkv_params, lens, seed=0, vote_max=1, scored_frac=1.0, scale=1.0) -> kb.Cache:
    """A cache with N(0, scale) keys, N(0,1) values, integer votes in [1, vote_max], and lscore either
    N(0, 2) (scored) or -inf."""
    rng = np.random.default_rng(seed)
    U, N, d = p.B * p.H_kv, p.N_cap, p.d
    K = rng.standard_normal((U, N, d)).astype(np.float32) * scale
    V = rng.standard_normal((U, N, d)).astype(np.float32)
    votes = rng.integers(1, vote_max + 1, (U, N)).astype(np.float32)
    ls = (rng.standard_normal((U, N)) * 2.0).astype(np.float32)
    ls[rng.random((U, N)) > scored_frac] = -np.inf
    c = kb.Cache(f32_to_dev_bf16(K).view(p.B, p.H_kv, N, d), f32_to_dev_bf16(V).view(p.B, p.H_kv, N, d),
                 torch.from_numpy(votes).cuda().view(p.B, p.H_kv, N), torch.from_numpy(ls).cuda().view(p.B, p.H_kv, N),
                 torch.tensor(np.asarray(lens, dtype=np.int32)).cuda())
    return c


def workload_cache(w: W.Workload, n_cap=None, layer=0, units=None) -> kb.Cache:
    K, V, lens = W.make_cache(w, layer=layer, n_cap=n_cap, units=units)
    N = K.shape[1]
    return kb.Cache(bits_to_dev(K).view(w.B, w.H_kv, N, w.d), bits_to_dev(V).view(w.B, w.H_kv, N, w.d),
                    torch.ones(w.B, w.H_kv, N, dtype=torch.float32, device="cuda"),
                    torch.full((w.B, w.H_kv, N), -math.inf, dtype=torch.float32, device="cuda"),
                    torch.from_numpy(lens).cuda())


def workload_params(w: W.Workload, n_cap=None, **kw) -> kb.keepkv_params:
    n_cap = int(n_cap if n_cap is not None else -(-(w.N + w.period) // 64) * 64)
    args = dict(B=w.B, H_q=w.H_q, H_kv=w.H_kv, d=w.d, N_cap=n_cap, period=w.period, n_sink=w.n_sink,
                n_recent=w.n_recent(), ema_alpha=0.9, merge_threshold=0.8)
    args.update(kw)
    return kb.make_params(**args)


def check_decode_unit(p, u, hc: HostCache, q64, out_gpu64, lse_gpu, lscore_after=None, what=""):
    """Compare one unit of a decode call with the oracle (pre-call state in hc)."""
    P = oracle_params(p)
    G = P.G
    K, V, votes, ls = hc.unit(u)
    b, h = divmod(u, p.H_kv)
    qu = q64[b, h * G:(h + 1) * G]
    o_ref, lse_ref = O.decode(P, qu, K, V, votes)
    check_close(out_gpu64[b, h * G:(h + 1) * G], O.round_bf16(o_ref), f"{what} out u={u}")
    if lse_gpu is not None:
        check_close(lse_gpu[b, h * G:(h + 1) * G], lse_ref, f"{what} lse u={u}", ulps=None, max_abs=1e-4, mean_rel=1e-5)
    if lscore_after is not None:
        ls_ref = O.score_update(P, qu, K, ls)
        check_close(lscore_after[u, :len(ls_ref)], ls_ref, f"{what} lscore u={u}", ulps=None, max_abs=1e-4,
                    mean_rel=1e-5)


def check_compress_unit(p, u, budget, n_recent, hc_src: HostCache, hc_dst: HostCache, ret_idx, target, stats=None,
                        what="", sorted_select=True, select_key=None, max_tolerated=0):
    """Teacher-forced staged check of one unit of a compress call: the oracle is fed the same source
    state; index sets and merge targets must match exactly, tensors within the bf16 rules.

    The only tolerated difference is a group whose rescale factor sits on the edge of the gamma guard
    in the oracle (within 1e-3 relative): the two sides may then disagree on whether that ONE slot is
    merged, so the targets of its members and the row of that slot are excused.  Every other slot is
    still compared.  Returns (oracle result, number of excused source entries); more than
    `max_tolerated` of them fail the check."""
    P = oracle_params(p, n_recent=n_recent)
    K, V, votes, ls = hc_src.unit(u)
    n = K.shape[0]
    ref = O.compress(P, budget, K, V, votes, ls, sorted_select=sorted_select,
                     select_key=None if select_key is None else select_key[u, :n])
    m = len(ref["ret_idx"])
    b = u // p.H_kv
    assert int(hc_dst.seq_len[b]) == m, f"{what} u={u}: new seq_len {hc_dst.seq_len[b]} != {m}"
    assert np.array_equal(ret_idx[u, :m], ref["ret_idx"]), f"{what} u={u}: retained set differs"
    tg, tr = target[u, :n], ref["target"]
    excused_slots = set()
    diff = np.nonzero(tg != tr)[0]
    gam = ref["gammas"]
    for e in diff:
        slots = [int(s) for s in (tg[e], tr[e]) if s >= 0]
        # the entry's target itself must agree wherever both sides name one: only "merged or not" may differ
        assert len(slots) == 1 or slots[0] == slots[1], f"{what} u={u}: target of entry {e}: gpu {tg[e]} oracle {tr[e]}"
        s = slots[0] if slots else -1
        edge = s >= 0 and np.isfinite(gam[s]) and (min(abs(gam[s] - P.gamma_min), abs(gam[s] - P.gamma_max))
                                                   < 1e-3 * max(1.0, abs(gam[s])))
        assert edge, f"{what} u={u}: target of entry {e}: gpu {tg[e]} oracle {tr[e]} (not on the guard's edge)"
        excused_slots.add(s)
    n_tol = int(len(diff))
    assert n_tol <= max_tolerated, f"{what} u={u}: {n_tol} entries excused by the guard edge (> {max_tolerated})"
    keep = np.ones(m, dtype=bool)
    keep[list(excused_slots)] = False
    dK, dV, dvotes, dls = hc_dst.unit(u)
    assert np.array_equal(dvotes[keep], ref["votes"][keep]), f"{what} u={u}: votes differ"
    check_close(dK[keep], ref["K"][keep], f"{what} K u={u}")
    check_close(dV[keep], ref["V"][keep], f"{what} V u={u}")
    check_close(dls[keep], ref["lscore"][keep], f"{what} lscore u={u}", ulps=None, max_abs=1e-4, mean_rel=1e-5)
    if stats is not None:
        exact = ("n_retained", "n_evicted") if n_tol else ("n_retained", "n_evicted", "n_merged", "n_below_T",
                                                           "n_guard_groups", "n_groups", "max_group")
        for f in exact:
            assert int(stats[u][kb.STATS_FIELDS.index(f)]) == ref["stats"][f], (what, u, f, stats[u], ref["stats"])
    return ref, n_tol
