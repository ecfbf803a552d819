"""GPU parity at the sizes and launch configurations the benchmark times, on sampled units the oracle
can afford, plus the shapes that reach the less common code paths: ragged per-sequence budgets with
G = 8, hundreds of short units, one very long unit (partial results of hundreds of CTAs, group keys
sorted in global memory), the largest supported capacity."""
import math

import numpy as np
import pytest
import torch

import oracle as O
from helpers import (bits_to_dev, check_close, check_compress_unit, f32_to_dev_bf16, oracle_params, random_cache, to_f64,
                     workload_cache, workload_params)
from paper_2504_09936_b200 import binding as kb
from paper_2504_09936_b200 import workloads as W

pytestmark = pytest.mark.gpu


class UnitView:
    """float64 copy of a few units of a device cache, with the interface check_compress_unit expects."""

    def __init__(self, cache: kb.Cache, units):
        B, H, N, d = cache.K.shape
        self.H = H
        self.seq_len = cache.seq_len.cpu().numpy().astype(np.int64)
        self._u = {}
        for u in units:
            b, h = divmod(u, H)
            self._u[u] = (to_f64(cache.K[b, h]), to_f64(cache.V[b, h]), to_f64(cache.votes[b, h]), to_f64(cache.lscore[b, h]))

    def unit(self, u):
        n = int(self.seq_len[u // self.H])
        K, V, p, ls = self._u[u]
        return K[:n], V[:n], p[:n], ls[:n]


def _check_decode(p, view: UnitView, units, q, out, lscore_after, what, lse=None):
    P = oracle_params(p)
    G = P.G
    q64, o64 = to_f64(q), to_f64(out)
    for u in units:
        K, V, votes, ls = view.unit(u)
        b, h = divmod(u, p.H_kv)
        qu = q64[b, h * G:(h + 1) * G]
        o_ref, lse_ref = O.decode(P, qu, K, V, votes)
        check_close(o64[b, h * G:(h + 1) * G], O.round_bf16(o_ref), f"{what} out u={u}", ulps=2.0)
        if lse is not None:
            check_close(to_f64(lse)[b, h * G:(h + 1) * G], lse_ref, f"{what} lse u={u}", ulps=None, max_abs=1e-3,
                        mean_rel=1e-5)
        if lscore_after is not None:
            ls_ref = O.score_update(P, qu, K, ls)
            got = to_f64(lscore_after[b, h, :len(ls_ref)])
            check_close(got, ls_ref, f"{what} lscore u={u}", ulps=None, max_abs=1e-3, mean_rel=1e-4)


def _compress(p, src, budget, n_recent_dev=None):
    dst = kb.Cache.empty(p)
    ws, st = kb.new_workspace(p), kb.new_status()
    U = p.B * p.H_kv
    ret = torch.full((U, p.N_cap), -7, dtype=torch.int32, device="cuda")
    tgt = torch.full((U, p.N_cap), -7, dtype=torch.int32, device="cuda")
    stats = torch.zeros(U, 8, dtype=torch.int32, device="cuda")
    kb.keepkv_compress(p, src, dst, budget, ws, st, n_recent_dev=n_recent_dev, retained_idx=ret, target=tgt, stats=stats)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return dst, ret.cpu().numpy(), tgt.cpu().numpy(), stats.cpu().numpy()


def test_c2_benchmark_size_sampled_units():
    """Workload C2 exactly as bench.py runs it (8 x 8 units, 8192 entries, capacity 8320, budget 1638,
    period 128): prompt scoring, the first compression, one whole period, the steady-state compression.
    Three units are compared with the oracle at every stage (teacher-forced)."""
    w = W.CONFIGS["C2"]
    p = workload_params(w)
    units = [0, 27, 63]
    cache = workload_cache(w, n_cap=p.N_cap)
    ws, st = kb.new_workspace(p), kb.new_status()
    P_ = w.period
    q_all, kn_all, vn_all = W.make_step_inputs(w, 0, 0, P_ + 1)
    out = torch.empty(w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(w.B, w.H_q, dtype=torch.float32, device="cuda")
    # step 0 on the full prompt
    before = UnitView(cache, units)
    q0 = bits_to_dev(q_all[0])
    kb.keepkv_decode_attention(p, cache, q0, out, lse, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, units, q0, out, cache.lscore, "C2 step 0", lse=lse)
    # first compression 8192 -> 1638
    b = w.budget()
    src = UnitView(cache, units)
    dst, ret, tgt, stats = _compress(p, cache, b)
    dview = UnitView(dst, units)
    assert list(dst.seq_len.cpu()) == [b] * w.B
    for u in units:
        check_compress_unit(p, u, b, p.n_recent, src, dview, ret, tgt, stats, what="C2 first compress")
    # one period on the compressed cache
    cur = dst
    for t in range(1, P_ + 1):
        if t == P_:
            before = UnitView(cur, units)          # state before the last step's append
        q = bits_to_dev(q_all[t])
        kb.keepkv_append(p, cur, bits_to_dev(kn_all[t]), bits_to_dev(vn_all[t]), st)
        if t == P_:
            after_append = UnitView(cur, units)
        kb.keepkv_decode_attention(p, cur, q, out, None, True, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and list(cur.seq_len.cpu()) == [b + P_] * w.B
    _check_decode(p, after_append, units, q, out, cur.lscore, "C2 last step of the period")
    # the appended row itself (Eq. 2)
    kn64, vn64 = to_f64(bits_to_dev(kn_all[P_])), to_f64(bits_to_dev(vn_all[P_]))
    for u in units:
        bb, h = divmod(u, w.H_kv)
        K, V, votes, _ = after_append.unit(u)
        assert np.array_equal(K[-1], kn64[bb, h]) and np.array_equal(V[-1], vn64[bb, h]) and votes[-1] == 1.0
    # steady-state compression 1766 -> 1638
    src = UnitView(cur, units)
    dst2, ret, tgt, stats = _compress(p, cur, b)
    dview = UnitView(dst2, units)
    for u in units:
        check_compress_unit(p, u, b, p.n_recent, src, dview, ret, tgt, stats, what="C2 steady compress")


def test_ragged_budgets_g8_like_c5():
    """The serving-scale workload's structure at a size the oracle checks in full: G = 8, ragged prompt
    lengths, per-sequence budgets (10 %) and recent windows, first compression then a short period."""
    w = W.scaled(W.CONFIGS["C5"], B=6, N=1536, n_min=384, period=32)
    p = workload_params(w)
    cache = workload_cache(w, n_cap=p.N_cap)
    lens = cache.seq_len.cpu().numpy()
    assert len(set(lens.tolist())) > 1
    bud = np.array([w.budget(int(n)) for n in lens], dtype=np.int32)
    nrec = np.array([w.n_recent(int(x)) for x in bud], dtype=np.int32)
    bud_d, nrec_d = torch.from_numpy(bud).cuda(), torch.from_numpy(nrec).cuda()
    units = list(range(w.U))
    ws, st = kb.new_workspace(p), kb.new_status()
    q_all, kn_all, vn_all = W.make_step_inputs(w, 0, 0, w.period + 1)
    out = torch.empty(w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
    before = UnitView(cache, units)
    q0 = bits_to_dev(q_all[0])
    kb.keepkv_decode_attention(p, cache, q0, out, None, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, units, q0, out, cache.lscore, "ragged step 0")
    src = UnitView(cache, units)
    dst, ret, tgt, stats = _compress(p, cache, bud_d, nrec_d)
    assert list(dst.seq_len.cpu().numpy()) == list(bud)
    dview = UnitView(dst, units)
    for u in units:
        bb = u // w.H_kv
        check_compress_unit(p, u, int(bud[bb]), int(nrec[bb]), src, dview, ret, tgt, stats, what="ragged first compress")
    cur = dst
    for t in range(1, w.period + 1):
        kb.keepkv_append(p, cur, bits_to_dev(kn_all[t]), bits_to_dev(vn_all[t]), st)
        if t == w.period:
            before = UnitView(cur, units)
        q = bits_to_dev(q_all[t])
        kb.keepkv_decode_attention(p, cur, q, out, None, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, units, q, out, cur.lscore, "ragged last step")
    src = UnitView(cur, units)
    dst2, ret, tgt, stats = _compress(p, cur, bud_d, nrec_d)
    dview = UnitView(dst2, units)
    for u in units:
        bb = u // w.H_kv
        check_compress_unit(p, u, int(bud[bb]), int(nrec[bb]), src, dview, ret, tgt, stats, what="ragged steady compress")
    assert int(st.item()) == 0


def test_many_short_units_like_c3():
    """512 units (16 sequences x 32 heads, G = 1) of 474 entries, as workload C3 in steady state: every
    CTA of the decode grid crosses unit boundaries; compression 474 -> 410 on every unit."""
    B, H, d = 16, 32, 128
    p = kb.make_params(B=B, H_q=H, H_kv=H, d=d, N_cap=512, period=64, n_sink=4, n_recent=324, merge_threshold=0.3)
    lens = [474] * B
    lens[3], lens[9] = 0, 411
    cache = random_cache(p, lens, seed=77, vote_max=3, scored_frac=0.9)
    units = [0, 1, 31, 32, 100, 3 * 32 + 5, 9 * 32 + 7, 255, 256, 511]
    rng = np.random.default_rng(5)
    q = f32_to_dev_bf16(rng.standard_normal((B, H, d)).astype(np.float32))
    out = torch.empty_like(q)
    lse = torch.empty(B, H, dtype=torch.float32, device="cuda")
    ws, st = kb.new_workspace(p), kb.new_status()
    before = UnitView(cache, units)
    kb.keepkv_decode_attention(p, cache, q, out, lse, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, [u for u in units if lens[u // H] > 0], q, out, cache.lscore, "C3-like decode", lse=lse)
    assert torch.all(out[3] == 0) and torch.all(torch.isinf(lse[3]))      # the empty sequence
    src = UnitView(cache, units)
    dst, ret, tgt, stats = _compress(p, cache, 410)
    dview = UnitView(dst, units)
    for u in units:
        check_compress_unit(p, u, 410, p.n_recent, src, dview, ret, tgt, stats, what="C3-like compress")


@pytest.mark.parametrize("T", [-math.inf, 0.8])
def test_one_long_unit_many_ctas(T):
    """One unit of 36 000 entries: its tiles spread over the whole decode grid (hundreds of partial
    results for one output), the similarity search splits its columns into chunks, several CTAs
    resolve the unit, and with T = -inf more than 32768 entries are merged, so the group keys are
    sorted in global memory."""
    N, d, budget = 36000, 64, 96
    p = kb.make_params(B=1, H_q=2, H_kv=1, d=d, N_cap=36864, period=0, n_sink=4, n_recent=40, merge_threshold=T,
                       gamma_min=0.0, gamma_max=4.0)
    cache = random_cache(p, [N], seed=13, vote_max=2, scored_frac=1.0)
    cache.lscore.mul_(0.25).add_(1.5)          # positive log-scores keep most rescale factors inside the guard
    rng = np.random.default_rng(1)
    q = f32_to_dev_bf16(rng.standard_normal((1, 2, d)).astype(np.float32))
    out = torch.empty_like(q)
    lse = torch.empty(1, 2, dtype=torch.float32, device="cuda")
    ws, st = kb.new_workspace(p), kb.new_status()
    before = UnitView(cache, [0])
    kb.keepkv_decode_attention(p, cache, q, out, lse, True, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    _check_decode(p, before, [0], q, out, cache.lscore, "long unit decode", lse=lse)
    src = UnitView(cache, [0])
    dst, ret, tgt, stats = _compress(p, cache, budget)
    dview = UnitView(dst, [0])
    check_compress_unit(p, 0, budget, p.n_recent, src, dview, ret, tgt, stats, what=f"long unit compress T={T}")
    if T == -math.inf:
        assert int(stats[0][2]) + int(stats[0][4]) > 0 and int(stats[0][3]) <= N - budget


def test_largest_capacity():
    """N_cap = 49152, the largest capacity the selection kernel's shared memory holds."""
    N = 49152
    p = kb.make_params(B=1, H_q=4, H_kv=1, d=64, N_cap=N, period=0, n_sink=4, n_recent=100, merge_threshold=0.35)
    cache = random_cache(p, [N], seed=3, scored_frac=1.0)
    rng = np.random.default_rng(2)
    q = f32_to_dev_bf16(rng.standard_normal((1, 4, 64)).astype(np.float32))
    out = torch.empty_like(q)
    ws, st = kb.new_workspace(p), kb.new_status()
    before = UnitView(cache, [0])
    kb.keepkv_decode_attention(p, cache, q, out, None, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, [0], q, out, cache.lscore, "largest capacity decode")
    src = UnitView(cache, [0])
    dst, ret, tgt, stats = _compress(p, cache, 160)
    check_compress_unit(p, 0, 160, p.n_recent, src, UnitView(dst, [0]), ret, tgt, stats, what="largest capacity compress")
    assert int(st.item()) == 0
