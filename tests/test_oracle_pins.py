"""Pins for the CPU oracle: everything the paper and plain mathematics fix about
the path, checked without a GPU.  Each test names the passage it rests on.

The reference computations in this file are written independently of the oracle's
formulas wherever possible: library softmax attention, brute-force duplication,
the theorems' invariants, linear-domain closed forms, numpy sorting.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

RNG = np.random.default_rng


def _rand_unit(rng, n, d, G=1, scale=1.0):
    K = rng.standard_normal((n, d)) * scale
    V = rng.standard_normal((n, d))
    q = rng.standard_normal((G, d))
    return q, K, V


# --------------------------------------------------------------------- rounding

def test_round_bf16_matches_torch_and_ties_to_even():
    rng = RNG(1)
    x = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-30, 30, 2000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e+38, 1e-40, -1e-45]])
    x32 = x.astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = O.round_bf16(x32.astype(np.float64))
    assert np.array_equal(got, want)
    # 1 + 2^-8 is exactly half way between 1 and 1 + 2^-7: ties go to the even significand
    assert O.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert O.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2 * 2.0 ** -7
    # directly from fp64 (no double rounding through fp32)
    assert O.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 1.0 + 2.0 ** -7


# ------------------------------------------------------- Eq. 3 / Eq. 6 attention

@pytest.mark.parametrize("G,d,n", [(1, 8, 16), (4, 64, 200), (8, 128, 77)])
def test_votes_one_is_library_softmax_attention(G, d, n):
    """Eq. 6 with p = 1 is Eq. 3, i.e. textbook scaled-dot-product attention."""
    rng = RNG(2)
    q, K, V = _rand_unit(rng, n, d, G)
    P = O.Params(G=G, d=d)
    out, lse = O.decode(P, q, K, V, np.ones(n))
    tq, tK, tV = (torch.from_numpy(a) for a in (q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[None], tK[None], tV[None])[0].numpy()
    assert np.allclose(out, ref, rtol=0, atol=1e-12)
    ref_lse = torch.logsumexp(tq @ tK.T / math.sqrt(d), dim=-1).numpy()
    assert np.allclose(lse, ref_lse, atol=1e-12)


def test_votes_equal_duplicated_entries():
    """Section 3.3.1: an entry with p votes acts as p identical independent copies."""
    rng = RNG(3)
    n, d, G = 9, 8, 2
    q, K, V = _rand_unit(rng, n, d, G)
    votes = rng.integers(1, 5, n).astype(np.float64)
    P = O.Params(G=G, d=d)
    out, lse = O.decode(P, q, K, V, votes)
    rep = np.repeat(np.arange(n), votes.astype(int))
    out2, lse2 = O.decode(P, q, K[rep], V[rep], np.ones(len(rep)))
    assert np.allclose(out, out2, atol=1e-13)
    assert np.allclose(lse, lse2, atol=1e-13)


def test_decode_empty_and_single():
    P = O.Params(G=2, d=4)
    out, lse = O.decode(P, np.ones((2, 4)), np.zeros((0, 4)), np.zeros((0, 4)), np.zeros(0))
    assert np.all(out == 0) and np.all(np.isneginf(lse))
    V = np.arange(4.0)[None]
    out, _ = O.decode(P, np.ones((2, 4)), np.ones((1, 4)), V, np.array([3.0]))
    assert np.allclose(out, np.repeat(V, 2, 0))


# ----------------------------------------------------------------- Eq. 8 (EMA)

def test_ema_closed_forms():
    """Eq. 8: alpha = 0 gives s_hat = s^t; a constant score sequence gives s_hat = s exactly;
    in general S^n = alpha^(n-1) s^1 + (1-alpha) sum_k alpha^(n-k) s^k, evaluated here in the
    linear domain, which the oracle never forms."""
    rng = RNG(4)
    n, d, G = 12, 8, 1
    _, K, _ = _rand_unit(rng, n, d, G)
    qs = rng.standard_normal((6, G, d))
    s = np.stack([np.exp(qs[t, 0] @ K.T / math.sqrt(d)) for t in range(6)])   # [t, n]
    # alpha = 0
    P0 = O.Params(G=G, d=d, ema_alpha=0.0)
    ls = np.full(n, -np.inf)
    for t in range(3):
        ls = O.score_update(P0, qs[t], K, ls)
        assert np.allclose(np.exp(ls), s[t], rtol=1e-12)
    # constant sequence
    Pa = O.Params(G=G, d=d, ema_alpha=0.9)
    ls = np.full(n, -np.inf)
    for t in range(5):
        ls = O.score_update(Pa, qs[0], K, ls)
    assert np.allclose(np.exp(ls), s[0], rtol=1e-12)
    # general closed form
    a = 0.7
    Pb = O.Params(G=G, d=d, ema_alpha=a)
    ls = np.full(n, -np.inf)
    for t in range(6):
        ls = O.score_update(Pb, qs[t], K, ls)
    S = a ** 5 * s[0] + (1 - a) * sum(a ** (5 - k) * s[k] for k in range(1, 6))
    assert np.allclose(np.exp(ls), S, rtol=1e-12)


def test_gqa_score_is_group_mean_of_exponentials():
    rng = RNG(5)
    n, d, G = 10, 8, 4
    q, K, _ = _rand_unit(rng, n, d, G)
    P = O.Params(G=G, d=d, ema_alpha=0.0)
    ls = O.score_update(P, q, K, np.full(n, -np.inf))
    s = np.exp(q @ K.T / math.sqrt(d)).mean(axis=0)
    assert np.allclose(np.exp(ls), s, rtol=1e-12)


# ------------------------------------------------------------------- selection

def _select_numpy(kap, budget, n_sink, n_recent):
    n = len(kap)
    if budget >= n:
        return np.arange(n)
    n_sink = min(n_sink, budget)
    n_recent = min(n_recent, budget - n_sink)
    lo, hi = n_sink, n - n_recent
    mid = np.arange(lo, hi)
    order = np.lexsort((mid, -kap[mid].astype(np.float64)))   # by kappa descending, then index ascending
    heavy = mid[order[:budget - n_sink - n_recent]]
    return np.sort(np.concatenate([np.arange(lo), heavy, np.arange(hi, n)]))


@pytest.mark.parametrize("seed", range(6))
def test_selection_against_sorting_and_ties(seed):
    rng = RNG(100 + seed)
    n = int(rng.integers(5, 200))
    kap = rng.standard_normal(n).astype(np.float32)
    kap[rng.integers(0, n, n // 3)] = kap[rng.integers(0, n)]     # plant equal keys
    if seed % 2:
        kap[rng.integers(0, n, 3)] = -np.inf                         # never-scored entries
    for budget in (0, 1, 3, n // 4, n // 2, n - 1, n, n + 5):
        for n_sink, n_recent in ((0, 0), (4, 0), (4, 7), (2, n)):
            want = _select_numpy(kap, budget, n_sink, n_recent)
            got = O.select(kap, budget, n_sink, n_recent)
            got2 = O.select(kap, budget, n_sink, n_recent, sorted_impl=True)
            assert np.array_equal(got, want), (n, budget, n_sink, n_recent)
            assert np.array_equal(got2, want)
            assert len(got) == min(n, max(budget, 0))


def test_selection_tie_keeps_lowest_index():
    kap = np.array([0, 5, 5, 5, 1], dtype=np.float32)
    assert list(O.select(kap, 2, 0, 0)) == [1, 2]
    assert list(O.select(kap, 3, 1, 1)) == [0, 1, 4]


@pytest.mark.parametrize("seed", range(4))
def test_compress_with_caller_supplied_selection_scores(seed):
    """Section 3.4 / 4.5: any token selection may designate the retained and evicted sets.  With caller scores
    the retained set is the numpy-sorted selection on those scores; the rest of Algorithm 1 is unchanged, so
    (a) passing kappa itself as the scores reproduces the default compression exactly, and (b) the output equals
    the default compression of a cache whose lscore makes kappa equal to the scores, wherever that substitution
    does not touch the merge (no evicted entry merged: T above every cosine)."""
    rng = RNG(300 + seed)
    n, d, budget, n_sink, n_recent = int(rng.integers(40, 160)), 16, 24, 3, 9
    K = O.round_bf16(rng.standard_normal((n, d)))
    V = O.round_bf16(rng.standard_normal((n, d)))
    votes = rng.integers(1, 4, n).astype(np.float64)
    ls = rng.standard_normal(n)
    key = np.abs(rng.standard_normal(n)).cumsum()[rng.permutation(n)].astype(np.float32)   # accumulated-attention-like
    key[rng.integers(0, n, 5)] = key[rng.integers(0, n)]                                    # ties
    P = O.Params(G=1, d=d, n_sink=n_sink, n_recent=n_recent, merge_threshold=0.3)
    c = O.compress(P, budget, K, V, votes, ls, select_key=key)
    assert np.array_equal(c["ret_idx"], _select_numpy(key, budget, n_sink, n_recent))
    # (a) kappa as scores = default
    c0 = O.compress(P, budget, K, V, votes, ls)
    ck = O.compress(P, budget, K, V, votes, ls, select_key=O.kappa(votes, ls))
    for f in ("ret_idx", "target", "K", "V", "votes", "lscore"):
        assert np.array_equal(c0[f], ck[f], equal_nan=True), f
    # (b) nothing merged: the scores only pick rows
    P1 = O.Params(G=1, d=d, n_sink=n_sink, n_recent=n_recent, merge_threshold=1.5)
    c1 = O.compress(P1, budget, K, V, votes, ls, select_key=key)
    r = c1["ret_idx"]
    assert np.all(c1["target"][np.setdiff1d(np.arange(n), r)] == -1)
    assert np.array_equal(c1["K"], K[r]) and np.array_equal(c1["V"], V[r])
    assert np.array_equal(c1["votes"], votes[r]) and np.array_equal(c1["lscore"], ls[r])
    # merge targets depend only on the sets: wherever an entry was merged, it went where the matcher alone sends it
    tgt, _, _ = O.match(P, K, c["ret_idx"])
    merged = c["target"] >= 0
    assert merged.any() and np.array_equal(c["target"][merged], np.asarray(tgt)[merged])


def test_kappa_is_log_of_vote_weighted_score():
    votes = np.array([1.0, 2.0, 7.0])
    ls = np.array([0.25, -3.0, -np.inf])
    k = O.kappa(votes, ls)
    assert k.dtype == np.float32
    assert k[0] == np.float32(0.25) and np.isneginf(k[2])
    assert abs(float(k[1]) - (math.log(2.0) - 3.0)) < 1e-6


# ------------------------------------------------- Algorithm 1, similarity and arg-max steps: match

def test_match_agrees_with_fp64_cosine_away_from_ties():
    rng = RNG(7)
    n, d = 120, 32
    K = O.round_bf16(rng.standard_normal((n, d)))
    ret = np.sort(rng.choice(n, 30, replace=False)).astype(np.int32)
    P = O.Params(G=1, d=d, merge_threshold=-np.inf)
    target, umax, second = O.match(P, K, ret)
    Kn = K / np.linalg.norm(K, axis=1, keepdims=True)
    U = Kn @ Kn[ret].T
    for e in range(n):
        if e in ret:
            assert target[e] == -2
            continue
        assert abs(umax[e] - U[e].max()) < 1e-5
        srt = np.sort(U[e])
        if srt[-1] - srt[-2] > 1e-5:
            assert target[e] == int(np.argmax(U[e]))
        assert 0 <= target[e] < len(ret)


def test_match_threshold_and_tie_break_and_degenerate():
    d = 8
    e1 = np.eye(d)
    K = np.stack([e1[0], e1[0], 2 * e1[0] + 0.01 * e1[1], e1[1], np.zeros(d)])
    ret = np.array([0, 1, 3], dtype=np.int32)      # slots 0,1 hold identical keys
    P = O.Params(G=1, d=d, merge_threshold=0.8)
    target, umax, _ = O.match(P, K, ret)
    assert list(target[:4]) == [-2, -2, 0, -2]     # equal cosine: lowest slot wins
    assert target[4] == -1                         # zero key: cosine undefined, never merged
    P2 = O.Params(G=1, d=d, merge_threshold=0.9999999)
    t2, _, _ = O.match(P2, K, ret)
    assert t2[2] == -1                             # below T -> evicted without merge
    # the fixed fp32 recipe: cos(x, x) is exactly 1 for a power-of-two norm
    assert O.cosine(2 * e1[0], 4 * e1[0]) == 1.0
    # no retained entries at all
    t3, u3, _ = O.match(P, K, np.zeros(0, dtype=np.int32))
    assert np.all(t3 == -1) and np.all(np.isneginf(u3))


# --------------------------------------------------------- Eq. 7 / (A.3): merge

def _eq7_literal(pe, se, ke, ve, pc, sc, kc, vc):
    """Eq. 7 exactly as printed (exponential domain)."""
    we, wc = pe * se, pc * sc
    kr = (we * ke + wc * kc) * math.log((we + wc) / (pe + pc)) / (we * math.log(se) + wc * math.log(sc))
    vr = (we * ve + wc * vc) / (we + wc)
    return kr, vr, pe + pc


def test_pair_merge_equals_printed_equation_7():
    rng = RNG(8)
    d = 8
    for _ in range(50):
        K = rng.standard_normal((2, d)); V = rng.standard_normal((2, d))
        p = rng.integers(1, 6, 2).astype(np.float64)
        lam = rng.uniform(0.2, 3.0, 2) * rng.choice([-1, 1])      # same sign: denominator away from 0
        m = O.merge_group(d, [0, 1], K, V, p, lam)
        kr, vr, pr = _eq7_literal(p[0], math.exp(lam[0]), K[0], V[0], p[1], math.exp(lam[1]), K[1], V[1])
        assert np.allclose(m["k_r"], kr, rtol=1e-11, atol=1e-13)
        assert np.allclose(m["v_r"], vr, rtol=1e-12)
        assert m["p_r"] == pr


def test_golden_two_entry_values():
    """Hand-evaluated instances of Eq. 7 (tests/golden/zip_merge_pairs.txt)."""
    path = os.path.join(os.path.dirname(__file__), "golden", "zip_merge_pairs.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 3
    for r in rows:
        l0, l1, p0, p1, L, lbar, gamma, om0 = map(float, r)
        K = np.array([[1.0, 0.0], [0.0, 1.0]]); V = K.copy()
        m = O.merge_group(2, [0, 1], K, V, [p0, p1], [l0, l1])
        assert abs(m["lambda_r"] - L) < 2e-6
        assert abs(m["lambda_bar"] - lbar) < 2e-6
        assert abs(m["gamma"] - gamma) < 2e-6
        assert abs(m["v_r"][0] - om0) < 2e-6       # v_r = omega_0 e_0 + omega_1 e_1
        assert abs(m["k_r"][0] - gamma * om0) < 4e-6


def _lossless_case(rng, n, d, budget, votes_max, guard=False, n_sink=0, n_recent=0):
    q, K, V = _rand_unit(rng, n, d, 1)
    votes = rng.integers(1, votes_max + 1, n).astype(np.float64)
    P = O.Params(G=1, d=d, ema_alpha=0.0, merge_threshold=-np.inf, n_sink=n_sink, n_recent=n_recent,
                 gamma_min=0.0 if guard else -np.inf, gamma_max=4.0 if guard else np.inf)
    ls = O.score_update(P, q, K, np.full(n, -np.inf))       # s_hat = s^t
    o0, lse0 = O.decode(P, q, K, V, votes)
    c = O.compress(P, budget, K, V, votes, ls)
    o1, lse1 = O.decode(P, q, c["K"], c["V"], c["votes"])
    return P, q, K, V, votes, ls, c, (o0, lse0), (o1, lse1)


@pytest.mark.parametrize("seed", range(20))
def test_single_step_lossless_theorem_2(seed):
    """Theorem 2 / Eq. (A.3): with s_hat = s^t, recomputing step t on the compressed cache
    reproduces the output, for pair and many-to-one merges and any vote counts."""
    rng = RNG(200 + seed)
    n = int(rng.integers(3, 40)); d = int(rng.choice([4, 8, 16]))
    budget = int(rng.integers(1, n))
    P, q, K, V, votes, ls, c, (o0, lse0), (o1, lse1) = _lossless_case(rng, n, d, budget, 4, n_sink=seed % 3,
                                                                      n_recent=seed % 4)
    lbar_ok = np.all(np.isnan(c["gammas"]) | (np.abs(c["gammas"]) < 1e6))
    if not lbar_ok:
        pytest.skip("group with lambda_bar ~ 0: the printed formula is singular there")
    assert c["stats"]["n_merged"] == n - budget          # T = -inf: every evicted entry merges
    assert np.max(np.abs(o1 - o0)) < 1e-9                # far inside the 1e-5 this invariant is specified to
    assert abs(lse1[0] - lse0[0]) < 1e-9                 # the denominator is conserved too
    # Electoral-Votes conservation: p_r = sum of members' votes
    assert c["votes"].sum() == votes.sum()


def test_conserved_sums_per_group():
    """Eq. (A.2): sum_{K'_e} p_i s_i = p_r s_r and sum p_i s_i v_i = p_r s_r v_r for every group,
    with s_r = exp(q.k_r/sqrt(d)) evaluated on the merged key."""
    rng = RNG(9)
    n, d = 30, 8
    P, q, K, V, votes, ls, c, _, _ = _lossless_case(rng, n, d, 6, 3)
    s = np.exp(q[0] @ K.T / math.sqrt(d))
    for slot, ci in enumerate(c["ret_idx"]):
        mem = [ci] + [e for e in range(n) if c["target"][e] == slot]
        s_r = math.exp(q[0] @ c["K"][slot] / math.sqrt(d))
        p_r = c["votes"][slot]
        assert p_r == votes[mem].sum()
        assert math.isclose(p_r * s_r, (votes[mem] * s[mem]).sum(), rel_tol=1e-9)
        assert np.allclose(p_r * s_r * c["V"][slot], ((votes[mem] * s[mem])[:, None] * V[mem]).sum(0), rtol=1e-9)
        # reading R8: the merged entry's score state carries ln(sum p s_hat / sum p)
        assert math.isclose(c["lscore"][slot], math.log((votes[mem] * s[mem]).sum() / p_r), rel_tol=1e-9, abs_tol=1e-12)


def test_softmax_probabilities_instead_of_exponentials_break_losslessness():
    """Negative control for the reading s = exp(q.k/sqrt(d)) (Eq. 3): feeding normalised
    attention weights into Eq. 7 does not preserve the output."""
    rng = RNG(10)
    n, d = 12, 8
    q, K, V = _rand_unit(rng, n, d, 1)
    P = O.Params(G=1, d=d, ema_alpha=0.0, merge_threshold=-np.inf, n_sink=0, gamma_min=-np.inf, gamma_max=np.inf)
    ell = q[0] @ K.T / math.sqrt(d)
    ls_prob = ell - np.log(np.exp(ell).sum())              # ln softmax probability
    o0, _ = O.decode(P, q, K, V, np.ones(n))
    c = O.compress(P, 4, K, V, np.ones(n), ls_prob)
    o1, _ = O.decode(P, q, c["K"], c["V"], c["votes"])
    assert np.max(np.abs(o1 - o0)) > 1e-3


def test_identical_pair_lemma():
    """Lemma 1: merging identical entries keeps (k, v), sets p = 2, and stays exact for every later query."""
    rng = RNG(11)
    d = 8
    k = rng.standard_normal(d); v = rng.standard_normal(d)
    lam = 0.7
    m = O.merge_group(d, [0, 1], np.stack([k, k]), np.stack([v, v]), [1.0, 1.0], [lam, lam])
    assert np.allclose(m["k_r"], k, atol=1e-14) and np.allclose(m["v_r"], v, atol=1e-14)
    assert m["p_r"] == 2.0 and abs(m["gamma"] - 1.0) < 1e-14
    K = np.vstack([rng.standard_normal((5, d)), k, k]); V = np.vstack([rng.standard_normal((5, d)), v, v])
    P = O.Params(G=1, d=d)
    for _ in range(5):
        q = rng.standard_normal((1, d))
        o0, _ = O.decode(P, q, K, V, np.ones(7))
        o1, _ = O.decode(P, q, np.vstack([K[:5], m["k_r"]]), np.vstack([V[:5], m["v_r"]]), np.r_[np.ones(5), 2.0])
        assert np.allclose(o0, o1, atol=1e-13)


@pytest.mark.parametrize("seed", range(30))
def test_multi_step_bound_theorem_3(seed):
    """Theorem 3: with relative prediction error eps < 1 on every entry of the group and on the
    merged entry, the perturbation at a later step is below 2 eps (1+eps) gamma / (1-eps)^2."""
    rng = RNG(300 + seed)
    n, d = 12, 8
    K = rng.standard_normal((n, d)) * 0.5
    V = rng.standard_normal((n, d))
    votes = rng.integers(1, 3, n).astype(np.float64)
    q2 = rng.standard_normal((1, d))                        # the later query (step t')
    s2 = np.exp(q2[0] @ K.T / math.sqrt(d))                 # true scores at t'
    group = [int(i) for i in rng.choice(n, int(rng.integers(2, 5)), replace=False)]
    shat = s2 * (1.0 + rng.uniform(-0.3, 0.3, n))           # estimates used by the merge
    m = O.merge_group(d, group, K, V, votes, np.log(shat))
    rest = [i for i in range(n) if i not in group]
    K1 = np.vstack([K[rest], m["k_r"]]); V1 = np.vstack([V[rest], m["v_r"]]); p1 = np.r_[votes[rest], m["p_r"]]
    P = O.Params(G=1, d=d)
    o_full, _ = O.decode(P, q2, K, V, votes)
    o_cmp, _ = O.decode(P, q2, K1, V1, p1)
    theta = np.linalg.norm(o_full - o_cmp)
    s_r = math.exp(q2[0] @ m["k_r"] / math.sqrt(d)); shat_r = math.exp(m["lambda_r"])
    eps = max(np.max(np.abs(1 - shat[group] / s2[group])), abs(1 - shat_r / s_r))
    if eps >= 1.0:
        pytest.skip("prediction error outside the theorem's range")
    gam = max(np.linalg.norm(V[j] - V[i]) for j in group for i in range(n))
    assert theta < 2 * eps * (1 + eps) * gam / (1 - eps) ** 2


def test_eviction_identity_equation_4():
    """Eq. 4 / (A.1): entries that find no target above T are dropped, and the output moves to
    (o - sum_j A_j v_j) / (1 - sum_j A_j)."""
    rng = RNG(12)
    n, d = 20, 8
    q, K, V = _rand_unit(rng, n, d, 1)
    P = O.Params(G=1, d=d, ema_alpha=0.0, merge_threshold=np.inf, n_sink=0)
    ls = O.score_update(P, q, K, np.full(n, -np.inf))
    o0, _ = O.decode(P, q, K, V, np.ones(n))
    c = O.compress(P, 7, K, V, np.ones(n), ls)
    assert c["stats"]["n_merged"] == 0 and c["stats"]["n_below_T"] == n - 7
    ev = [i for i in range(n) if i not in c["ret_idx"]]
    A = np.exp(ls) / np.exp(ls).sum()
    want = (o0[0] - (A[ev, None] * V[ev]).sum(0)) / (1 - A[ev].sum())
    o1, _ = O.decode(P, q, c["K"], c["V"], c["votes"])
    assert np.allclose(o1[0], want, atol=1e-12)
    # retained rows are copied untouched, in ascending original index
    assert np.array_equal(c["K"], K[c["ret_idx"]]) and np.all(np.diff(c["ret_idx"]) > 0)
    # the kept set is the top-7 by score here (no sinks, no recent window)
    assert set(c["ret_idx"]) == set(np.argsort(-ls)[:7])


def test_attention_sag_of_convex_merging_theorem_1():
    """Theorem 1 (negative control): a convex combination of two entries receives less attention
    than the two did together, so the same check that passes for ZIP merging fails here."""
    rng = RNG(13)
    n, d = 10, 8
    q, K, V = _rand_unit(rng, n, d, 1)
    P = O.Params(G=1, d=d)
    s = np.exp(q[0] @ K.T / math.sqrt(d)); A = s / s.sum()
    e, c, w = 2, 5, 0.35
    kr = w * K[e] + (1 - w) * K[c]; vr = w * V[e] + (1 - w) * V[c]
    rest = [i for i in range(n) if i not in (e, c)]
    s_r = math.exp(q[0] @ kr / math.sqrt(d))
    A_r = s_r / (s[rest].sum() + s_r)
    assert A_r < A[e] + A[c]
    o0, _ = O.decode(P, q, K, V, np.ones(n))
    o1, _ = O.decode(P, q, np.vstack([K[rest], kr]), np.vstack([V[rest], vr]), np.ones(n - 1))
    assert np.linalg.norm(o0 - o1) > 1e-4


def test_guard_on_rescale_factor():
    """A group whose log-scores straddle zero makes the printed rescale factor negative; with the
    guard on, its members are evicted and the target is left untouched."""
    d = 4
    K = np.eye(4)[:3] + 0.0; V = np.eye(4)[:3] + 1.0
    K[1] = K[0] * 1.0001                                   # entry 1 will pick slot of entry 0
    votes = np.ones(3); ls = np.array([0.5, -2.0, 3.0])
    m = O.merge_group(d, [0, 1], K, V, votes, ls)
    assert abs(m["gamma"] - (-0.368)) < 2e-3               # L = -0.114, lambda_bar = +0.310
    P = O.Params(G=1, d=d, merge_threshold=-np.inf, n_sink=0)
    c = O.compress(P, 2, K, V, votes, ls)
    assert list(c["ret_idx"]) == [0, 2] and c["target"][1] == -1
    assert c["stats"]["n_guard_groups"] == 1 and c["stats"]["n_merged"] == 0
    assert np.array_equal(c["K"][0], K[0]) and c["votes"][0] == 1.0
    Pu = O.Params(G=1, d=d, merge_threshold=-np.inf, n_sink=0, gamma_min=-np.inf, gamma_max=np.inf)
    cu = O.compress(Pu, 2, K, V, votes, ls)
    assert cu["target"][1] == 0 and cu["votes"][0] == 2.0


def test_compress_is_ordered_copy_when_budget_not_exceeded():
    rng = RNG(14)
    n, d = 9, 4
    q, K, V = _rand_unit(rng, n, d, 1)
    P = O.Params(G=1, d=d)
    c = O.compress(P, 9, K, V, np.ones(n), np.zeros(n))
    assert np.array_equal(c["K"], K) and np.array_equal(c["V"], V) and len(c["ret_idx"]) == n
    c = O.compress(P, 50, K, V, np.ones(n), np.zeros(n))
    assert len(c["ret_idx"]) == n


def test_storage_faithful_mode_rounds_every_write():
    rng = RNG(15)
    n, d = 24, 8
    q, K, V = _rand_unit(rng, n, d, 1)
    K = O.round_bf16(K); V = O.round_bf16(V)
    P = O.Params(G=1, d=d, ema_alpha=0.0, merge_threshold=-np.inf, n_sink=0, storage_faithful=True,
                 gamma_min=-np.inf, gamma_max=np.inf)
    ls = O.score_update(P, q, K, np.full(n, -np.inf))
    assert np.array_equal(ls, ls.astype(np.float32).astype(np.float64))
    c = O.compress(P, 5, K, V, np.ones(n), ls)
    assert np.array_equal(c["K"], O.round_bf16(c["K"])) and np.array_equal(c["V"], O.round_bf16(c["V"]))
    # rounding the merged rows to bf16 costs accuracy but stays within bf16 resolution of lossless
    o0, _ = O.decode(P, q, K, V, np.ones(n))
    o1, _ = O.decode(P, q, c["K"], c["V"], c["votes"])
    assert np.max(np.abs(o1 - o0)) < 5e-2


def test_append_equation_2():
    d = 4
    K = np.zeros((5, d)); V = np.zeros((5, d)); votes = np.zeros(5); ls = np.zeros(5)
    n = O.append(K, V, votes, ls, 2, np.arange(4.0), -np.arange(4.0))
    assert n == 3 and np.array_equal(K[2], np.arange(4.0)) and np.array_equal(V[2], -np.arange(4.0))
    assert votes[2] == 1.0 and np.isneginf(ls[2]) and np.all(K[3:] == 0)


def test_batch_wrappers_match_per_unit():
    rng = RNG(16)
    U, n_cap, d, G = 3, 20, 8, 2
    P = O.Params(G=G, d=d, merge_threshold=-np.inf, n_sink=1, n_recent=2)
    K = rng.standard_normal((U, n_cap, d)); V = rng.standard_normal((U, n_cap, d))
    votes = np.ones((U, n_cap)); ls = np.full((U, n_cap), -np.inf)
    q = rng.standard_normal((U, G, d))
    lens = np.array([20, 13, 0], dtype=np.int32)
    out, lse = O.decode_batch(P, lens, q, K, V, votes, ls, True)
    for u in range(U):
        n = lens[u]
        o, l = O.decode(P, q[u], K[u, :n], V[u, :n], votes[u, :n])
        assert np.array_equal(out[u], o) and np.array_equal(lse[u], l)
        assert np.array_equal(ls[u, :n], O.score_update(P, q[u], K[u, :n], np.full(n, -np.inf)))
    r = O.compress_batch(P, lens, np.array([5, 5, 5], dtype=np.int32), K, V, votes, ls)
    for u in range(U):
        n = lens[u]
        c = O.compress(P, 5, K[u, :n], V[u, :n], votes[u, :n], ls[u, :n])
        m = r["new_lens"][u]
        assert m == len(c["ret_idx"])
        assert np.array_equal(r["K"][u, :m], c["K"]) and np.array_equal(r["votes"][u, :m], c["votes"])
        assert np.array_equal(r["ret_idx"][u, :m], c["ret_idx"]) and np.array_equal(r["target"][u, :n], c["target"])


# ------------------------------------------------------------------ Eq. 8, first case (windowed initialisation)

def _raw_scores(q_window, K, d):
    """s_i^k = mean over the group of exp(q.k/sqrt(d)), written out with numpy: [W, len]."""
    logits = np.einsum("kgd,id->kgi", q_window, K) / np.sqrt(d)
    return np.exp(logits).mean(axis=1)


@pytest.mark.parametrize("alpha,W,G", [(0.9, 8, 1), (0.5, 5, 4), (0.9, 33, 2)])
def test_windowed_init_equals_bias_corrected_recursion(alpha, W, G):
    """Eq. 8: running the recursion S <- alpha S + (1 - alpha) s over the window from S = 0 and dividing
    by 1 - alpha^n (n = steps taken) gives the windowed first case.  Entries older than the window see
    every query; the recursion is written out here in numpy, independently of the oracle."""
    rng = np.random.default_rng(int(alpha * 100) + W)
    d, n = 16, 40 + W
    K = rng.standard_normal((n, d)) * 0.7
    qw = rng.standard_normal((W, G, d))
    P = O.Params(G=G, d=d, ema_alpha=alpha)
    got = O.prefill_scores(P, qw, K)
    s = _raw_scores(qw, K, d)
    old = np.arange(n) <= n - W            # entries every query of the window can see
    S = np.zeros(n)
    for k in range(W):
        S = alpha * S + (1 - alpha) * s[k]
    want = np.log(S / (1 - alpha ** W))
    assert np.allclose(got[old], want[old], rtol=1e-12, atol=1e-12)


def test_windowed_init_respects_causality_and_constant_scores():
    """An entry inside the window is scored only by the queries at or after its position, with the weights
    renormalised (brute force per entry); identical queries give s_hat = s whatever alpha is; W = 1 is
    the first observation of the decode path."""
    rng = np.random.default_rng(7)
    d, n, W, G, alpha = 8, 12, 5, 2, 0.8
    K = rng.standard_normal((n, d))
    qw = rng.standard_normal((W, G, d))
    P = O.Params(G=G, d=d, ema_alpha=alpha)
    got = O.prefill_scores(P, qw, K)
    s = _raw_scores(qw, K, d)
    for i in range(n):
        ks = [k for k in range(W) if n - W + k >= i]
        w = np.array([alpha ** (W - 1 - k) for k in ks])
        want = np.log((w * s[ks, i]).sum() / w.sum())
        assert abs(got[i] - want) < 1e-12, i
    # constant query sequence: the estimate is the score itself
    qc = np.repeat(qw[:1], W, axis=0)
    assert np.allclose(O.prefill_scores(P, qc, K), np.log(_raw_scores(qc, K, d)[0]), atol=1e-12)
    # window of one query = first observation in the recursive path; alpha = 0 keeps only the last query
    one = O.prefill_scores(P, qw[-1:], K)
    assert np.allclose(one, O.score_update(P, qw[-1], K, np.full(n, -np.inf)), atol=1e-12)
    P0 = O.Params(G=G, d=d, ema_alpha=0.0)
    assert np.allclose(O.prefill_scores(P0, qw, K), one, atol=1e-12)
    # a prompt shorter than the window: the queries before position 0 do not exist
    short = O.prefill_scores(P, qw, K[:3])
    assert np.allclose(short, O.prefill_scores(P, qw[-3:], K[:3]), atol=1e-12)


# ------------------------------------------------ Section 3.4 / App. B Table 3: prefill merge-first policy

def _clustered_keys(rng, n, d, n_clusters, spread):
    """Keys that come in clusters of near-duplicates (cosine well above any threshold inside a cluster, near zero
    between clusters), in random order: the structure the merge-first policy exists for."""
    centers = rng.standard_normal((n_clusters, d)) * 3.0
    which = rng.integers(0, n_clusters, n)
    return centers[which] + spread * rng.standard_normal((n, d)), which


def _brute_force_merge_first(K, T):
    """The pairing rule written out with numpy in fp64: partner = most similar other entry (lowest index on
    exactly equal cosines), an entry wants to merge iff its best cosine exceeds T and the partner is earlier, and
    it is merged only if that partner does not itself want to merge."""
    n = K.shape[0]
    Kn = K / np.linalg.norm(K, axis=1, keepdims=True)
    U = Kn @ Kn.T
    np.fill_diagonal(U, -np.inf)
    partner = np.argmax(U, axis=1)
    best = U[np.arange(n), partner]
    wants = (best > T) & (partner < np.arange(n))
    member = wants & ~wants[partner]
    return partner, best, member


@pytest.mark.parametrize("seed", range(8))
def test_merge_first_pairing_rule_against_brute_force(seed):
    """Which entries are merged into which: the oracle's fixed-fp32-cosine decisions against an fp64 numpy
    restatement of the rule, on inputs whose margins are far from both the ties and the threshold."""
    T = 0.9
    for attempt in range(20):   # redraw an input with a near tie (fp32 and fp64 may legitimately order it differently)
        rng = RNG(700 + seed + 1000 * attempt)
        n, d = int(rng.integers(20, 90)), int(rng.choice([8, 16, 64]))
        K, _ = _clustered_keys(rng, n, d, n_clusters=int(rng.integers(3, 9)), spread=0.6)
        V = rng.standard_normal((n, d))
        votes = rng.integers(1, 4, n).astype(float); ls = rng.standard_normal(n) + 1.5
        partner, best, member = _brute_force_merge_first(K, T)
        Kn = K / np.linalg.norm(K, axis=1, keepdims=True)
        srt = np.sort(np.where(np.eye(n, dtype=bool), -np.inf, Kn @ Kn.T), axis=1)
        if np.min(srt[:, -1] - srt[:, -2]) >= 2e-6 and np.min(np.abs(best - T)) >= 2e-6:
            break
    else:
        raise AssertionError("no input without a near tie in 20 draws")
    P = O.Params(G=1, d=d, merge_threshold=T, gamma_min=-np.inf, gamma_max=np.inf)
    r = O.merge_similar(P, K, V, votes, ls)
    kept = np.nonzero(~member)[0]
    assert np.array_equal(r["ret_idx"], kept)
    slot_of = -np.ones(n, dtype=int); slot_of[kept] = np.arange(len(kept))
    want_target = np.where(member, slot_of[partner], -2)
    assert np.array_equal(r["target"], want_target)
    assert member.sum() > 0 and r["stats"]["n_merged"] == member.sum() and r["stats"]["n_evicted"] == member.sum()
    # no entry is both a target and a member
    assert not np.any(member[partner[member]])


def test_merge_first_chain_and_mutual_pair():
    """Hand-built cases of the rule.  Keys a, b, c at angles 0, 0.3, 0.65: b's best partner is a (cos .955 against
    .939), c's best partner is b (.939 against .796).  b merges into a; c's partner is itself merged away, so c
    stays.  A mutual pair merges the later entry into the earlier one."""
    d = 4
    def unit(theta):
        return np.array([math.cos(theta), math.sin(theta), 0.0, 0.0])
    far = np.array([0.0, 0.0, 1.0, 0.0]); far2 = np.array([0.0, 0.0, 0.0, 1.0])
    K = np.stack([unit(0.0), unit(0.3), unit(0.65), far, far2 * 2.0, far2 * 0.5])
    V = np.arange(6 * d, dtype=float).reshape(6, d)
    P = O.Params(G=1, d=d, merge_threshold=0.9, gamma_min=-np.inf, gamma_max=np.inf)
    r = O.merge_similar(P, K, V, np.ones(6), np.full(6, 1.0))
    # entry 1 -> 0 (cos .955 > T, partner earlier).  entry 2's best partner is 1 (cos .939 > T), which is merged away: 2 stays.
    # entries 4, 5 are parallel (cos 1): a mutual pair, 5 merges into 4.  entry 3 has no similar neighbour.
    assert list(r["ret_idx"]) == [0, 2, 3, 4]
    assert list(r["target"]) == [-2, 0, -2, -2, -2, 3]
    assert list(r["votes"]) == [2.0, 1.0, 1.0, 2.0]
    # equal scores: omega = 1/2 each, gamma = 1 (the merged score equals the members' common score)
    assert np.allclose(r["K"][0], 0.5 * (K[0] + K[1])) and np.allclose(r["V"][3], 0.5 * (V[4] + V[5]))
    assert np.array_equal(r["K"][1], K[2]) and np.array_equal(r["K"][2], K[3])


@pytest.mark.parametrize("seed", range(6))
def test_merge_first_is_lossless_for_the_current_query_and_conserves_votes(seed):
    """Theorem 2 applies to every group the policy forms: with s_hat = s^t (alpha = 0, G = 1) the attention output
    and its denominator are unchanged by the merge, whatever the vote counts; and since nothing is evicted, the
    votes of the cache are conserved (p_r = sum of the members' votes)."""
    rng = RNG(800 + seed)
    n, d = 60, 16
    K, _ = _clustered_keys(rng, n, d, n_clusters=5, spread=0.08)
    q = rng.standard_normal((1, d)) * 0.3
    V = rng.standard_normal((n, d))
    votes = rng.integers(1, 5, n).astype(float)
    P = O.Params(G=1, d=d, ema_alpha=0.0, merge_threshold=0.8, gamma_min=-np.inf, gamma_max=np.inf)
    ls = O.score_update(P, q, K, np.full(n, -np.inf))       # lscore = this step's logits
    o0, lse0 = O.decode(P, q, K, V, votes)
    r = O.merge_similar(P, K, V, votes, ls)
    assert r["stats"]["n_merged"] > 10
    if np.nanmax(np.abs(r["gammas"])) > 1e6:
        pytest.skip("group with lambda_bar ~ 0: the printed formula is singular there")
    o1, lse1 = O.decode(P, q, r["K"], r["V"], r["votes"])
    assert np.max(np.abs(o1 - o0)) < 1e-9 and abs(lse1[0] - lse0[0]) < 1e-9
    assert r["votes"].sum() == votes.sum()


def test_merge_first_degenerate_cases():
    """T = +inf merges nothing (an ordered copy); exact duplicates collapse onto their first occurrence with the
    key and value unchanged (Lemma 1) and the votes added; a single entry and an empty unit pass through."""
    rng = RNG(9)
    n, d = 10, 8
    K = rng.standard_normal((n, d)); V = rng.standard_normal((n, d)); votes = np.arange(1, n + 1, dtype=float)
    ls = rng.standard_normal(n)
    r = O.merge_similar(O.Params(G=1, d=d, merge_threshold=np.inf), K, V, votes, ls)
    assert np.array_equal(r["K"], K) and np.array_equal(r["votes"], votes) and list(r["target"]) == [-2] * n
    K2 = np.vstack([K, K[3], K[3], K[7]]); V2 = np.vstack([V, V[3], V[3], V[7]])
    ls2 = np.r_[ls, ls[3], ls[3], ls[7]]
    r = O.merge_similar(O.Params(G=1, d=d, merge_threshold=0.99, gamma_min=-np.inf, gamma_max=np.inf), K2, V2,
                        np.ones(n + 3), ls2)
    assert list(r["ret_idx"]) == list(range(n)) and list(r["target"][n:]) == [3, 3, 7]
    assert np.allclose(r["K"][3], K[3], atol=1e-12) and np.allclose(r["V"][7], V[7], atol=1e-12)
    assert list(r["votes"]) == [1, 1, 1, 3, 1, 1, 1, 2, 1, 1]
    one = O.merge_similar(O.Params(G=1, d=d), K[:1], V[:1], votes[:1], ls[:1])
    assert one["stats"]["n_retained"] == 1 and np.array_equal(one["K"], K[:1])
    none = O.merge_similar(O.Params(G=1, d=d), K[:0], V[:0], votes[:0], ls[:0])
    assert none["stats"]["n_retained"] == 0


def test_merge_first_then_evict_keeps_what_evict_first_loses():
    """The point of the policy (App. B, Table 3): with the same budget, merging similar entries before the
    eviction keeps the votes of near-duplicates that an eviction without merging discards.  Pure eviction is
    okv_compress with T = +inf."""
    rng = RNG(10)
    n, d, budget = 80, 16, 20
    K, which = _clustered_keys(rng, n, d, n_clusters=6, spread=0.05)
    V = rng.standard_normal((n, d)); votes = np.ones(n); ls = rng.standard_normal(n) * 0.3 + 2.0
    Pm = O.Params(G=1, d=d, n_sink=0, n_recent=0, merge_threshold=0.9)
    Pe = O.Params(G=1, d=d, n_sink=0, n_recent=0, merge_threshold=np.inf)
    first = O.merge_similar(Pm, K, V, votes, ls)
    then = O.compress(Pe, budget, first["K"], first["V"], first["votes"], first["lscore"])
    plain = O.compress(Pe, budget, K, V, votes, ls)
    assert then["stats"]["n_merged"] == 0 and plain["stats"]["n_merged"] == 0
    assert plain["votes"].sum() == budget                       # eviction alone keeps one vote per kept entry
    assert then["votes"].sum() > 2 * budget                     # merge-first kept whole clusters


def test_first_observation_initialisation_is_not_the_bias_corrected_mean_after_step_one():
    """What the EMA reading is and is not (Eq. 8).  An entry's first observed score initialises its state, which
    coincides with the bias-corrected estimate S_n / (1 - alpha^n) counted from the entry's first observation at
    n = 1.  At n = 2 the two differ: the oracle holds alpha s_1 + (1 - alpha) s_2, the corrected form would be
    (alpha s_1 + s_2) / (1 + alpha)."""
    d, alpha = 4, 0.9
    P = O.Params(G=1, d=d, ema_alpha=alpha)
    K = np.array([[1.0, 0.0, 0.0, 0.0]])
    q1 = np.array([[2.0, 0.0, 0.0, 0.0]]); q2 = np.array([[-1.0, 0.0, 0.0, 0.0]])
    s1, s2 = math.exp(2.0 / math.sqrt(d)), math.exp(-1.0 / math.sqrt(d))
    ls = O.score_update(P, q1, K, np.array([-np.inf]))
    assert math.isclose(math.exp(ls[0]), s1, rel_tol=1e-12)                      # n = 1: both readings agree
    ls = O.score_update(P, q2, K, ls)
    plain = alpha * s1 + (1 - alpha) * s2
    corrected = ((1 - alpha) * (alpha * s1 + s2)) / (1 - alpha ** 2)
    assert math.isclose(math.exp(ls[0]), plain, rel_tol=1e-12)
    assert abs(plain - corrected) / corrected > 0.05                             # ... and here they do not


# ------------------------------------------------ Algorithm 1 in place (periodic mode): position array instead of row order

def _sorted_by_pos(r):
    o = np.argsort(r["pos"])
    return r["K"][o], r["V"][o], r["votes"][o], r["lscore"][o], r["pos"][o]


@pytest.mark.parametrize("seed", range(10))
def test_inplace_compression_is_the_compression_of_the_token_ordered_cache(seed):
    """Rows in random order with their token positions: the in-place compression must keep, merge and drop exactly
    the entries that okv_compress (pinned above) keeps, merges and drops on the same cache laid out in token order
    -- the cache order is a storage matter, the method is defined on tokens.  (Random scores and keys: no ties,
    where the two tie rules -- lower row, lower position -- would differ.)"""
    rng = RNG(900 + seed)
    n, d = int(rng.integers(12, 70)), int(rng.choice([8, 16]))
    budget = int(rng.integers(3, n))
    q, K, V = _rand_unit(rng, n, d, 1)
    votes = rng.integers(1, 4, n).astype(float); ls = rng.standard_normal(n)
    P = O.Params(G=1, d=d, n_sink=int(rng.integers(0, 3)), n_recent=int(rng.integers(0, 5)),
                 merge_threshold=float(rng.choice([-np.inf, 0.0, 0.3])))
    ref = O.compress(P, budget, K, V, votes, ls)                         # rows = tokens
    perm = rng.permutation(n)                                            # row i holds token perm[i]
    got = O.compress_inplace(P, budget, K[perm], V[perm], votes[perm], ls[perm], perm)
    gK, gV, gp, gl, gpos = _sorted_by_pos(got)
    assert np.array_equal(gpos, ref["ret_idx"])                          # the same tokens survive
    assert np.array_equal(gp, ref["votes"])
    assert np.allclose(gK, ref["K"], rtol=1e-12, atol=1e-13) and np.allclose(gV, ref["V"], rtol=1e-12, atol=1e-13)
    assert np.allclose(gl, ref["lscore"], rtol=1e-12, atol=1e-13)
    for f in ("n_retained", "n_evicted", "n_merged", "n_below_T", "n_guard_groups", "n_groups", "max_group"):
        assert got["stats"][f] == ref["stats"][f], f
    # attention does not care about the order (Eq. 6 is a sum over entries)
    o_ref, lse_ref = O.decode(P, q, ref["K"], ref["V"], ref["votes"])
    o_got, lse_got = O.decode(P, q, got["K"], got["V"], got["votes"])
    assert np.allclose(o_got, o_ref, atol=1e-12) and np.allclose(lse_got, lse_ref, atol=1e-12)


def test_inplace_compression_moves_only_what_it_must():
    """'Discard (k_e, v_e), (k_c, v_c) and insert (k_r, v_r)' taken literally: a retained row that is not a merge
    target and sits below the new length keeps its bits and its row; retained rows above the new length fill the
    holes in ascending order; everything is where moved_from says."""
    rng = RNG(31)
    n, d, budget = 40, 8, 30
    _, K, V = _rand_unit(rng, n, d, 1)
    votes = np.ones(n); ls = rng.standard_normal(n)
    pos = rng.permutation(n).astype(np.int32)
    P = O.Params(G=1, d=d, n_sink=2, n_recent=6, merge_threshold=0.2, gamma_min=-np.inf, gamma_max=np.inf)
    r = O.compress_inplace(P, budget, K, V, votes, ls, pos)
    tgt = r["target"]
    kept = np.nonzero(tgt == -2)[0]
    holes = [i for i in range(budget) if tgt[i] != -2]
    movers = [i for i in kept if i >= budget]
    assert len(holes) == len(movers) and len(kept) == budget
    merged_targets = set(int(t) for t in tgt if t >= 0)
    for row in range(budget):
        src = int(r["moved_from"][row])
        if row in holes:
            assert src == movers[holes.index(row)]                       # k-th hole takes the k-th mover
        else:
            assert src == row
        assert r["pos"][row] == pos[src]
        if src not in merged_targets:                                    # untouched by the merge: the same bits
            assert np.array_equal(r["K"][row], K[src]) and np.array_equal(r["V"][row], V[src])
            assert r["votes"][row] == votes[src] and r["lscore"][row] == ls[src]
        else:
            assert r["votes"][row] == 1 + np.sum(tgt == src)             # p_r = p_c + sum of its members' votes
    assert r["stats"]["n_merged"] == np.sum(tgt >= 0) and r["stats"]["n_below_T"] == np.sum(tgt == -1)
    # a cache within its budget is left alone
    same = O.compress_inplace(P, n, K, V, votes, ls, pos)
    assert np.array_equal(same["K"], K) and np.array_equal(same["pos"], pos) and list(same["moved_from"]) == list(range(n))


def test_inplace_compression_ties_go_to_the_lower_row_and_theorem_2_holds():
    """Equal selection keys and equal cosines are decided by the lower ROW (this oracle's rule for a cache without
    order); and Theorem 2 does not care where rows sit: with s_hat = s^t the output of the step is unchanged."""
    rng = RNG(32)
    n, d = 16, 8
    q, K, V = _rand_unit(rng, n, d, 1)
    K[9] = K[3]                                                          # two identical keys: equal cosines to anything
    P = O.Params(G=1, d=d, n_sink=0, n_recent=0, ema_alpha=0.0, merge_threshold=-np.inf, gamma_min=-np.inf,
                 gamma_max=np.inf)
    ls = np.zeros(n); ls[[3, 9]] = 5.0; ls[[2, 7, 11]] = 1.0             # rows 3 and 9 kept; 2, 7, 11 tie for the third place
    pos = np.arange(n)[::-1].copy()                                      # reversed: the lower row is the LATER token
    r = O.compress_inplace(P, 3, K, V, np.ones(n), ls, pos)
    assert sorted(np.nonzero(r["target"] == -2)[0]) == [2, 3, 9]         # row 2 wins the tie, not the earlier tokens 7, 11
    # an evicted row identical in direction to rows 3 and 9 would tie: check with row 12 := 2 * K[3]
    K2 = K.copy(); K2[12] = 2.0 * K[3]
    r2 = O.compress_inplace(P, 3, K2, V, np.ones(n), ls, pos)
    assert r2["target"][12] == 3                                         # equal cosines (1.0): the lower row
    ls_t = O.score_update(P, q, K, np.full(n, -np.inf))
    o0, lse0 = O.decode(P, q, K, V, np.ones(n))
    r3 = O.compress_inplace(P, 5, K, V, np.ones(n), ls_t, pos)
    if np.nanmax(np.abs(r3["gammas"])) < 1e6:
        o1, lse1 = O.decode(P, q, r3["K"], r3["V"], r3["votes"])
        assert np.max(np.abs(o1 - o0)) < 1e-9 and abs(lse1[0] - lse0[0]) < 1e-9
