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


# ---------------------------------------------------------------------------------------------------
# The remaining workloads at their stated shapes, in the launch configuration the benchmark times:
# capacity, parameters, per-sequence budgets and the steady-state flag exactly as bench.py sets them.
# Every stage runs on ALL units through the library; a few sampled units are compared with the oracle,
# teacher-forced (the oracle is fed the library's state before the stage).

def _with_fresh_row(view: UnitView, units, kn64, vn64, H_kv):
    """The view of a cache after Eq. 2 appended (kn, vn) to every sampled unit: what the attention of a
    keepkv_decode_step call must see."""
    out = UnitView.__new__(UnitView)
    out.H = view.H
    out.seq_len = view.seq_len + 1
    out._u = {}
    for u in units:
        b, h = divmod(u, H_kv)
        n = int(view.seq_len[b])
        K, V, p, ls = (a.copy() for a in view._u[u])
        K[n], V[n], p[n], ls[n] = kn64[b, h], vn64[b, h], 1.0, -math.inf
        out._u[u] = (K, V, p, ls)
    return out


def _protocol_at_stated_shape(name, units, layer=0):
    w = W.CONFIGS[name]
    P_ = w.period
    n_cap = -(-(w.N + P_) // 64) * 64                     # as bench.py
    p = workload_params(w, n_cap=n_cap)
    cache = workload_cache(w, n_cap=n_cap, layer=layer)
    lens = cache.seq_len.cpu().numpy()
    bud = np.array([w.budget(int(n)) for n in lens], dtype=np.int32)
    nrec = np.array([w.n_recent(int(x)) for x in bud], dtype=np.int32)
    ragged = bool(np.any(bud != bud[0]))
    steady = P_ <= 128 and int(np.max(bud + P_ - w.n_sink - nrec)) <= 2048 and int(np.max(bud)) <= 16384
    budget_arg = torch.from_numpy(bud).cuda() if ragged else int(bud[0])
    nrec_arg = torch.from_numpy(nrec).cuda() if ragged else None
    p_inc = workload_params(w, n_cap=n_cap, flags=kb.FLAG_COMPRESS_STEADY if steady else 0)
    ws, st = kb.new_workspace(p), kb.new_status()
    U = w.U
    q_all, kn_all, vn_all = W.make_step_inputs(w, layer, 0, P_ + 1)
    out = torch.empty(w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(w.B, w.H_q, dtype=torch.float32, device="cuda")
    Por = oracle_params(p)

    def compress(pp, src, stage):
        dst = kb.Cache.empty(p)
        ret = torch.full((U, n_cap), -7, dtype=torch.int32, device="cuda")
        tgt = torch.full((U, n_cap), -7, dtype=torch.int32, device="cuda")
        stats = torch.zeros(U, 8, dtype=torch.int32, device="cuda")
        before = UnitView(src, units)
        kb.keepkv_compress(pp, src, dst, budget_arg, ws, st, n_recent_dev=nrec_arg, retained_idx=ret, target=tgt,
                           stats=stats)
        torch.cuda.synchronize()
        assert int(st.item()) == 0, f"{name} {stage}: status {int(st.item())}"
        assert dst.seq_len.cpu().numpy().tolist() == np.minimum(bud, src.seq_len.cpu().numpy()).tolist()
        after = UnitView(dst, units)
        ret, tgt, stats = ret.cpu().numpy(), tgt.cpu().numpy(), stats.cpu().numpy()
        for u in units:
            bb = u // w.H_kv
            # a handful of entries may sit in a group on the edge of the gamma guard; everything else is exact
            check_compress_unit(p, u, int(bud[bb]), int(nrec[bb]), before, after, ret, tgt, stats,
                                what=f"{name} {stage}", max_tolerated=8)
        return dst

    # ---- Eq. 8, first case: scores at the end of prefill from a 32-query window
    Wq = 32
    qwin = bits_to_dev(q_all[1:1 + Wq]).permute(1, 2, 0, 3).contiguous()         # [B, H_q, W, d]
    before = UnitView(cache, units)
    kb.keepkv_prefill_scores(p, cache, qwin, st)
    torch.cuda.synchronize()
    q64 = to_f64(qwin)
    for u in units:
        b, h = divmod(u, w.H_kv)
        K = before.unit(u)[0]
        qu = np.ascontiguousarray(q64[b, h * w.G:(h + 1) * w.G].transpose(1, 0, 2))
        ref = O.prefill_scores(Por, qu, K)
        check_close(to_f64(cache.lscore[b, h, :len(ref)]), ref, f"{name} prefill scores u={u}", ulps=None,
                    max_abs=1e-3, mean_rel=1e-4)
    # ---- step 0 on the whole prompt (Eq. 6 + Eq. 8)
    before = UnitView(cache, units)
    q0 = bits_to_dev(q_all[0])
    kb.keepkv_decode_attention(p, cache, q0, out, lse, True, ws, st)
    torch.cuda.synchronize()
    _check_decode(p, before, units, q0, out, cache.lscore, f"{name} step 0", lse=lse)
    # ---- first compression: prompt -> budget (general pipeline)
    cur = compress(p, cache, "first compression")
    del cache
    # ---- one period of decode steps (append folded into the attention launch, as the benchmark runs it)
    for t in range(1, P_ + 1):
        if t == P_:
            torch.cuda.synchronize()
            before = UnitView(cur, units)
        q = bits_to_dev(q_all[t])
        kb.keepkv_decode_step(p, cur, q, bits_to_dev(kn_all[t]), bits_to_dev(vn_all[t]), out, lse, True, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and cur.seq_len.cpu().numpy().tolist() == (bud + P_).tolist()
    seen = _with_fresh_row(before, units, to_f64(bits_to_dev(kn_all[P_])), to_f64(bits_to_dev(vn_all[P_])), w.H_kv)
    _check_decode(p, seen, units, q, out, cur.lscore, f"{name} last step of the period", lse=lse)
    # ---- steady-state compression: budget + P -> budget (one kernel where the benchmark uses it)
    compress(p_inc, cur, "steady-state compression")
    return steady


def test_c3_stated_shape_sampled_units():
    """Workload C3: 16 sequences x 32 heads (G = 1), 4096-entry prompts, budget 410, period 64, drifting
    queries: prompt scoring, step 0, first compression 4096 -> 410 on all 512 units, 64 decode steps, the
    steady-state compression 474 -> 410; units of the first, a middle and the last sequence checked."""
    assert _protocol_at_stated_shape("C3", [0, 5 * 32 + 17, 511]) is True


def test_c4_stated_shape_sampled_unit():
    """Workload C4 (one of its 32 layers): 2 sequences x 8 kv heads (G = 4, d = 128), 32768-entry prompts,
    budget 3277, period 256: the similarity search runs 13 column tiles in chunks over 29 491 evicted rows
    per unit, several CTAs resolve a unit, the steady-state compression takes the general pipeline."""
    assert _protocol_at_stated_shape("C4", [11], layer=3) is False


def test_c5_stated_shape_sampled_units():
    """Workload C5: 64 sequences x 8 kv heads (G = 8), ragged prompts of 4096-16384 entries, per-sequence
    budgets (10 %) and recent windows, period 128; a head of the longest and one of the shortest sequence."""
    w = W.CONFIGS["C5"]
    lens = W.seq_lens(w, 0)
    b_long, b_short = int(np.argmax(lens)), int(np.argmin(lens))
    assert _protocol_at_stated_shape("C5", [b_long * 8 + 3, b_short * 8 + 6]) is True


def test_c2_period_as_the_benchmark_launches_it():
    """Workload C2 in the launch configuration bench.py times: three layer caches of the full shape visited
    round-robin, keepkv_decode_step with KEEPKV_FLAG_CACHE_IDLE replayed from a CUDA graph, then the single-kernel
    steady-state compression.  After 24 steps the caches and outputs equal, bit for bit, those of the unflagged
    append + attention calls on twin caches; the last step of every layer is compared with the oracle on sampled
    units, and so is the compression that follows."""
    w = W.CONFIGS["C2"]
    Lr, steps = 3, 24
    p = workload_params(w)
    p_idle = workload_params(w, flags=kb.FLAG_CACHE_IDLE)
    p_inc = workload_params(w, flags=kb.FLAG_COMPRESS_STEADY)
    b = w.budget()
    units = [5, 38]
    ws, st = kb.new_workspace(p), kb.new_status()
    clone = lambda c: kb.Cache(c.K.clone(), c.V.clone(), c.votes.clone(), c.lscore.clone(), c.seq_len.clone())
    # per layer: prompt of its own seed, scored by one step, compressed to the budget
    layers = []
    for l in range(Lr):
        prompt = workload_cache(w, n_cap=p.N_cap, layer=l)
        q0 = bits_to_dev(W.make_step_inputs(w, l, 0, 1)[0][0])
        o0 = torch.empty(w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
        kb.keepkv_decode_attention(p, prompt, q0, o0, None, True, ws, st)
        dst = kb.Cache.empty(p)
        kb.keepkv_compress(p, prompt, dst, b, ws, st)
        torch.cuda.synchronize()
        layers.append(dst)
        del prompt
    twins = [clone(c) for c in layers]
    ins = [W.make_step_inputs(w, l, 1, steps + 1) for l in range(Lr)]
    q = [[bits_to_dev(ins[l][0][t]) for l in range(Lr)] for t in range(steps)]
    kn = [[bits_to_dev(ins[l][1][t]) for l in range(Lr)] for t in range(steps)]
    vn = [[bits_to_dev(ins[l][2][t]) for l in range(Lr)] for t in range(steps)]
    out = torch.zeros(steps, Lr, w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(steps, Lr, w.B, w.H_q, dtype=torch.float32, device="cuda")
    out2, lse2 = torch.zeros_like(out), torch.zeros_like(lse)

    def run(t0, t1):
        for t in range(t0, t1):
            for l in range(Lr):
                kb.keepkv_decode_step(p_idle, layers[l], q[t][l], kn[t][l], vn[t][l], out[t, l], lse[t, l], True, ws, st)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run(0, 1)
        g = torch.cuda.CUDAGraph()
        stream.synchronize()
        with torch.cuda.graph(g, stream=stream):
            run(1, steps - 1)
        g.replay()
        stream.synchronize()
        before = [UnitView(c, units) for c in layers]
        run(steps - 1, steps)
        stream.synchronize()
    for t in range(steps):
        for l in range(Lr):
            kb.keepkv_append(p, twins[l], kn[t][l], vn[t][l], st)
            kb.keepkv_decode_attention(p, twins[l], q[t][l], out2[t, l], lse2[t, l], True, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16)) and torch.equal(lse.view(torch.int32), lse2.view(torch.int32))
    n = b + steps
    for l in range(Lr):
        assert layers[l].seq_len.cpu().tolist() == [n] * w.B == twins[l].seq_len.cpu().tolist()
        assert torch.equal(layers[l].K[:, :, :n].view(torch.int16), twins[l].K[:, :, :n].view(torch.int16))
        assert torch.equal(layers[l].V[:, :, :n].view(torch.int16), twins[l].V[:, :, :n].view(torch.int16))
        assert torch.equal(layers[l].votes[:, :, :n], twins[l].votes[:, :, :n])
        assert torch.equal(layers[l].lscore[:, :, :n].view(torch.int32), twins[l].lscore[:, :, :n].view(torch.int32))
        seen = _with_fresh_row(before[l], units, to_f64(kn[steps - 1][l]), to_f64(vn[steps - 1][l]), w.H_kv)
        _check_decode(p, seen, units, q[steps - 1][l], out[steps - 1, l], layers[l].lscore, f"C2 layer {l} last step",
                      lse=lse[steps - 1, l])
    # the steady-state compression of one layer, one kernel
    src = UnitView(layers[0], units)
    dst, ret, tgt, stats = _compress(p_inc, layers[0], b)
    dview = UnitView(dst, units)
    for u in units:
        check_compress_unit(p, u, b, p.n_recent, src, dview, ret, tgt, stats, what="C2 steady compress after 24 steps",
                            max_tolerated=8)
