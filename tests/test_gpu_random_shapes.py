"""Seeded random shapes through the GPU path: the launch shape of the decode kernel (split over the whole tile
list, one cluster per unit, cluster size) and the path of the compression depend on the batch, so a sweep over
batches exercises combinations the hand-picked cases do not."""
import math

import numpy as np
import pytest
import torch

from helpers import HostCache, check_decode_unit, f32_to_dev_bf16, random_cache, to_f64
from paper_2504_09936_b200 import binding as kb

pytestmark = pytest.mark.gpu


def _clone(c):
    return kb.Cache(c.K.clone(), c.V.clone(), c.votes.clone(), c.lscore.clone(), c.seq_len.clone())


@pytest.mark.parametrize("seed", range(12))
def test_decode_random_batches(seed):
    """Random batch size, head layout and lengths (equal-ish or ragged, some empty): outputs against the oracle on
    a sample of units, keepkv_decode_step against append + decode bit for bit."""
    rng = np.random.default_rng(1000 + seed)
    d = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    H_kv = int(rng.choice([1, 2, 4, 8]))
    B = int(rng.integers(1, 41))
    n_cap = int(rng.choice([128, 256, 512]))
    if rng.random() < 0.6:      # similar lengths: the cluster path where the unit count allows it
        base = int(rng.integers(1, n_cap - 8))
        lens = [min(n_cap - 2, max(0, base + int(rng.integers(-3, 4)))) for _ in range(B)]
    else:
        lens = [int(rng.integers(0, n_cap - 1)) for _ in range(B)]
    if rng.random() < 0.3:
        lens[int(rng.integers(0, B))] = 0
    p = kb.make_params(B=B, H_q=H_kv * G, H_kv=H_kv, d=d, N_cap=n_cap, ema_alpha=0.9)
    c1 = random_cache(p, lens, seed=seed, vote_max=3, scored_frac=0.7)
    c2 = _clone(c1)
    ws, st = kb.new_workspace(p), kb.new_status()
    mk = lambda *s: f32_to_dev_bf16(rng.standard_normal(s).astype(np.float32))
    U = B * H_kv
    for step in range(2):
        q, kn, vn = mk(B, H_kv * G, d), mk(B, H_kv, d), mk(B, H_kv, d)
        o1, o2 = torch.empty_like(q), torch.empty_like(q)
        l1 = torch.empty(B, H_kv * G, dtype=torch.float32, device="cuda")
        l2 = torch.empty_like(l1)
        kb.keepkv_decode_step(p, c1, q, kn, vn, o1, l1, True, ws, st)
        kb.keepkv_append(p, c2, kn, vn, st)
        hc = HostCache(c2)
        kb.keepkv_decode_attention(p, c2, q, o2, l2, True, ws, st)
        torch.cuda.synchronize()
        what = f"seed {seed} step {step} B={B} H_kv={H_kv} G={G} d={d} lens={lens[:6]}"
        assert int(st.item()) == 0, what
        assert torch.equal(c1.seq_len, c2.seq_len), what
        assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)), what
        assert torch.equal(l1.view(torch.int32), l2.view(torch.int32)), what
        ls_after = to_f64(c2.lscore).reshape(U, -1)
        for u in sorted(set(int(x) for x in rng.integers(0, U, size=4))):
            check_decode_unit(p, u, hc, to_f64(q), to_f64(o2), to_f64(l2), ls_after, what=what)


@pytest.mark.parametrize("seed", range(10))
def test_steady_compression_random_batches(seed):
    """Random steady-state compressions (few evicted entries): the single kernel and the pipeline leave the same bits."""
    rng = np.random.default_rng(2000 + seed)
    d = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 4]))
    H_kv = int(rng.choice([1, 2, 8]))
    B = int(rng.integers(1, 25))
    budget = int(rng.integers(8, 700))
    n_ev_max = int(rng.integers(1, 129))
    lens = [budget + int(rng.integers(-5, n_ev_max + 1)) for _ in range(B)]
    lens = [max(0, x) for x in lens]
    n_cap = -(-(max(lens) + 1) // 64) * 64
    n_recent = int(rng.integers(0, max(1, budget - 4)))
    T = float(rng.choice([-math.inf, 0.0, 0.3, 0.8]))
    p = kb.make_params(B=B, H_q=H_kv * G, H_kv=H_kv, d=d, N_cap=n_cap, period=0, n_sink=int(rng.integers(0, 6)),
                       n_recent=n_recent, merge_threshold=T)
    src = random_cache(p, lens, seed=seed, vote_max=3, scored_frac=0.9)
    outs = []
    for flags in (kb.FLAG_COMPRESS_STEADY, 0):
        pf = kb.make_params(B=B, H_q=H_kv * G, H_kv=H_kv, d=d, N_cap=n_cap, period=0, n_sink=p.n_sink,
                            n_recent=n_recent, merge_threshold=T, flags=flags)
        dst = kb.Cache.empty(p)
        ws, st = kb.new_workspace(p), kb.new_status()
        U = B * H_kv
        ret = torch.full((U, n_cap), -7, dtype=torch.int32, device="cuda")
        tgt = torch.full((U, n_cap), -7, dtype=torch.int32, device="cuda")
        stats = torch.zeros(U, 8, dtype=torch.int32, device="cuda")
        kb.keepkv_compress(pf, src, dst, budget, ws, st, retained_idx=ret, target=tgt, stats=stats)
        torch.cuda.synchronize()
        assert int(st.item()) == 0, (seed, flags)
        outs.append((dst, ret.cpu().numpy(), tgt.cpu().numpy(), stats.cpu().numpy()))
    (a, ra, ta, sa), (b2, rb, tb, sb) = outs
    what = f"seed {seed} B={B} H_kv={H_kv} d={d} budget={budget} lens={lens[:6]} T={T}"
    new_len = a.seq_len.cpu().numpy()
    assert np.array_equal(new_len, b2.seq_len.cpu().numpy()), what
    assert np.array_equal(sa, sb), what
    for u in range(B * H_kv):
        bb, h = divmod(u, H_kv)
        n, L = int(new_len[bb]), lens[bb]
        assert np.array_equal(ra[u, :n], rb[u, :n]) and np.array_equal(ta[u, :L], tb[u, :L]), (what, u)
        for x, y in ((a.K, b2.K), (a.V, b2.V)):
            assert torch.equal(x[bb, h, :n].view(torch.int16), y[bb, h, :n].view(torch.int16)), (what, u)
        for x, y in ((a.votes, b2.votes), (a.lscore, b2.lscore)):
            assert torch.equal(x[bb, h, :n].view(torch.int32), y[bb, h, :n].view(torch.int32)), (what, u)
