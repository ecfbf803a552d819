#!/usr/bin/env python
"""Benchmark of the KeepKV hot path on B200.

One "step" is one compression period of the steady-state decode loop of a workload
(default C2, the Llama-3-8B-shaped layer): P x (append one token, decode attention with
score update; one keepkv_decode_step launch) followed by one compression (budget + P -> budget), for every one of
`--layers` independent layer caches visited round-robin, so that no call finds its
cache in L2.  value = decode tokens/s of one layer = B * P * layers / step time.

  python bench.py [--gpus N --steps K --warmup W] [--impl reference]

N > 1 (torchrun): every rank runs its own replica of the batch (the path shards by
sequence with no collective); value is the sum over ranks over the slowest rank's time.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_09936_b200 import workloads as W  # noqa: E402

METRIC = "decode tokens/s + compress GB/s, fraction of HBM roofline"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the kernel the roofline entry times
# (keepkv_decode_step in the steady state), per workload, from an ncu capture of that kernel as it stands now;
# None where no capture of the current kernel exists
# (C2: mean of the two captured launches of the committed ncu summary of this kernel and workload)
DECODE_TRAFFIC_BYTES = {"C2": 60_450_000}
UNIT = "tokens/s"


def peaks():
    """(HBM copy rate in GB/s, sustained dense bf16 rate in TFLOP/s, where they come from)."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            m = json.load(f)
        return float(m["hbm_gbs"]), float(m.get("bf16_tflops_sustained", 1400.0)), "measured"
    except Exception:
        return 6650.0, 1400.0, "fallback"


def decode_bytes(w, entries_total):
    """Algorithmic bytes of one decode call: per entry K and V rows, votes, lscore read+write;
    plus queries and outputs."""
    return entries_total * (4 * w.d + 12) + 4 * w.B * w.H_q * w.d


def compress_bytes(w, len_, b, m):
    """Algorithmic bytes of one compression, all units: every key once, values of kept and merged
    entries, votes+lscore of every entry, and the rows written."""
    per_unit = len_ * 2 * w.d + (b + m) * 2 * w.d + len_ * 8 + b * (4 * w.d + 8)
    return w.U * per_unit


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms",
                                       "100", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- CPU oracle legs

_SAMPLE = {}


def oracle_period_time(w, n_units, n_decode, seed_layer=0):
    """Times the oracle, as it stands, on `n_units` units of the workload in its steady state:
    `n_decode` decode steps (Eq. 6 + Eq. 8) at length b + P/2 and one compression b + P -> b.
    Returns (seconds for a whole period of all U units extrapolated, threads, description, ...)."""
    import oracle as O
    b, P = w.budget(), w.period
    n_cap = b + P
    nu = min(n_units, w.U)
    key = (w.name, nu, n_decode, seed_layer)
    if key not in _SAMPLE:
        K = np.zeros((nu, n_cap, w.d)); V = np.zeros((nu, n_cap, w.d))
        for u in range(nu):
            c = W.make_unit(w, seed_layer, u, n_cap)
            K[u], V[u] = c["K"], c["V"]
        q = np.stack([W.make_queries(w, seed_layer, u, 0, n_decode + 1) for u in range(nu)], axis=1).astype(np.float64)
        _SAMPLE[key] = (K, V, q)
    K, V, q = _SAMPLE[key]
    votes = np.ones((nu, n_cap)); ls = np.full((nu, n_cap), -np.inf)
    Pm = O.Params(G=w.G, d=w.d, n_sink=w.n_sink, n_recent=w.n_recent(), storage_faithful=True, ema_alpha=0.9)
    lens_mid = np.full(nu, b + P // 2, dtype=np.int32)
    O.decode_batch(Pm, np.full(nu, n_cap, dtype=np.int32), np.ascontiguousarray(q[0]), K, V, votes, ls, True)
    t0 = time.perf_counter()
    for t in range(n_decode):
        O.decode_batch(Pm, lens_mid, np.ascontiguousarray(q[t + 1]), K, V, votes, ls, True)
    t_dec = (time.perf_counter() - t0) / n_decode
    t0 = time.perf_counter()
    O.compress_batch(Pm, np.full(nu, n_cap, dtype=np.int32), np.full(nu, b, dtype=np.int32), K, V, votes, ls)
    t_cmp = time.perf_counter() - t0
    scale = w.U / nu
    period_s = (P * t_dec + t_cmp) * scale
    desc = (f"{nu} of {w.U} units; {n_decode} of {P} decode steps at len {b + P // 2} and one compression "
            f"{b + P}->{b}, extrapolated to a whole period of all units")
    return period_s, O.num_threads(), desc, t_dec * scale, t_cmp * scale


def run_reference(args, w, rank):
    if rank != 0:
        return
    # A step is one compression period of ONE layer cache (the oracle has no cache to miss): every decode step of the
    # period is executed where that stays within a few seconds, else a stated number of them; `timed_s` is what
    # the clock really measured for one step, `ms_per_step` the period it stands for.
    n_dec = w.period if w.period * w.U * (w.budget() + w.period) * w.d * w.G <= 2.5e10 else 8
    t_all, t_meas = [], []
    for _ in range(min(args.warmup, 1)):
        oracle_period_time(w, w.U, n_dec)
    info = None
    for _ in range(args.steps):
        t0 = time.perf_counter()
        info = oracle_period_time(w, w.U, n_dec)
        t_meas.append(time.perf_counter() - t0)
        t_all.append(info[0])
    period_s = float(np.mean(t_all))
    val = w.B * w.period / period_s
    cpu = {"value": val, "unit": UNIT, "cores": info[1], "kind": "oracle", "sample": info[2],
           "timed_s": float(np.mean(t_meas)), "decode_steps_timed": n_dec, "decode_steps_per_period": w.period}
    print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": period_s * 1e3,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                      "data": "synthetic", "config": config_dict(w, args), "cpu_baseline": cpu,
                      "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                      "gpu_launches": 0}))


def config_dict(w, args):
    b, P = w.budget(), w.period
    mb = (w.U * (b + P // 2) * (4 * w.d + 12) + 4 * w.B * w.H_q * w.d) / 1e6
    return {"workload": f"{w.name}: B={w.B}, {w.H_q}q/{w.H_kv}kv heads, d={w.d}, N={w.N}, budget {b} "
                        f"({w.budget_ratio:.0%}), period {P}; steady-state compression period",
            "tokens": "layer-tokens: one token of one sequence attended in one layer cache (B * period * layers per step)",
            "layers_round_robin": args.layers,
            "l2": f"each call works on one of {args.layers} distinct layer caches visited round-robin "
                  f"({args.layers} x {mb:.0f} MB = {args.layers * mb:.0f} MB "
                  f"{'>' if args.layers * mb > 126 else '<= (NOT larger than)'} 126 MB L2)",
            "parallelism": f"replicas x{args.gpus}"}


# --------------------------------------------------------------------------- replicas (N > 1)

def slowest_rank(times, dist, device):
    """Element-wise maximum of `times` over the ranks (the path shards by sequence with no collective
    inside it, so the only exchange of a multi-GPU run is this one after the timed region)."""
    if dist is None:
        return [float(t) for t in times]
    import torch
    tt = torch.tensor([float(t) for t in times], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return [float(x) for x in tt]


def job_throughput(tokens_per_rank_step, world, steps, seconds):
    """Whole-job tokens/s: every rank processes its own replica of the batch (weak scaling)."""
    return tokens_per_rank_step * world * steps / seconds


# --------------------------------------------------------------------------- GPU leg

def run_ours(args, w, rank, world):
    import torch
    from paper_2504_09936_b200 import binding as kb

    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    kb.lib()  # fails loudly when the CUDA library is missing
    L, P, b = args.layers, w.period, w.budget()
    n_cap = -(-(w.N + P) // 64) * 64
    p = kb.make_params(B=w.B, H_q=w.H_q, H_kv=w.H_kv, d=w.d, N_cap=n_cap, period=P, n_sink=w.n_sink,
                       n_recent=w.n_recent(), ema_alpha=0.9, merge_threshold=0.8)
    dev = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    # inputs: one seeded prompt cache (per rank its own seed offset), replicated into L distinct buffers
    Kb, Vb, lens = W.make_cache(w, layer=rank, n_cap=n_cap)
    # budgets follow each sequence's own prompt length (they differ only for the ragged workload)
    bud = np.array([w.budget(int(n)) for n in lens], dtype=np.int32)
    nrec = np.array([w.n_recent(int(x)) for x in bud], dtype=np.int32)
    ragged = bool(np.any(bud != bud[0]))
    # Every compression after the first evicts exactly P entries per unit: when that is within the limits of the
    # single-kernel path, the steady-state calls say so and skip the launches of the general pipeline.
    steady = P <= 128 and int(np.max(bud + P - w.n_sink - nrec)) <= 2048 and int(np.max(bud)) <= 16384
    budget_arg = torch.from_numpy(bud).cuda() if ragged else b
    p_inc = kb.make_params(B=w.B, H_q=w.H_q, H_kv=w.H_kv, d=w.d, N_cap=n_cap, period=P, n_sink=w.n_sink,
                           n_recent=w.n_recent(), ema_alpha=0.9, merge_threshold=0.8,
                           flags=kb.FLAG_COMPRESS_STEADY if steady else 0)
    # The decode steps of the loop visit the layer caches round-robin, so with two layers or more the kernel that
    # precedes a step on the stream never writes the step's cache: the calls say so and start reading early.
    p_step = kb.make_params(B=w.B, H_q=w.H_q, H_kv=w.H_kv, d=w.d, N_cap=n_cap, period=P, n_sink=w.n_sink,
                            n_recent=w.n_recent(), ema_alpha=0.9, merge_threshold=0.8,
                            flags=kb.FLAG_CACHE_IDLE if L >= 2 else 0)
    nrec_arg = torch.from_numpy(nrec).cuda() if ragged else None
    K0, V0 = dev(Kb).view(w.B, w.H_kv, n_cap, w.d), dev(Vb).view(w.B, w.H_kv, n_cap, w.d)
    del Kb, Vb
    A = [kb.Cache(K0.clone(), V0.clone(), torch.ones(w.B, w.H_kv, n_cap, device="cuda"),
                  torch.full((w.B, w.H_kv, n_cap), -math.inf, device="cuda"), torch.from_numpy(lens).cuda())
         for _ in range(L)]
    Bc = [kb.Cache.empty(p) for _ in range(L)]
    del K0, V0
    # step inputs: step 0 scores the prompt; after it every period draws P fresh steps (a token is never appended
    # twice, which would plant exact duplicates of keys in the cache).  The graphs read the current period's
    # inputs from q_all/kn_all/vn_all[1:], refreshed from the pool by a device copy before every replay.
    n_e2e = max(2, min(args.steps, 6))
    n_pool = 2 + args.warmup + args.steps + 1 + 2 + n_e2e
    qb, knb, vnb = W.make_step_inputs(w, rank, 0, n_pool * P + 1)
    q_pool, kn_pool, vn_pool = dev(qb), dev(knb), dev(vnb)
    q_all, kn_all, vn_all = q_pool[:P + 1].clone(), kn_pool[:P + 1].clone(), vn_pool[:P + 1].clone()
    pool_next = [0]

    def load_period():
        k = pool_next[0]
        pool_next[0] += 1
        assert k < n_pool
        sl = slice(1 + k * P, 1 + (k + 1) * P)
        q_all[1:].copy_(q_pool[sl]); kn_all[1:].copy_(kn_pool[sl]); vn_all[1:].copy_(vn_pool[sl])
        return sl
    ws, st = kb.new_workspace(p), kb.new_status()
    out = torch.empty(w.B, w.H_q, w.d, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.Stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    launches = 0

    with torch.cuda.stream(stream):
        # ---- phase 0: windowed score initialisation at the end of prefill (Eq. 8, first case), one decode
        #      step on the full cache, then the first (full) compression
        Wq = 32
        qwin = q_pool[1:1 + Wq].permute(1, 2, 0, 3).contiguous()      # [B, H_q, W, d] stand-in for the last prompt queries
        for l in range(L):   # warm
            kb.keepkv_prefill_scores(p, A[l], qwin, st)
            kb.keepkv_decode_attention(p, A[l], q_all[0], out, None, False, ws, st)
        stream.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for l in range(L):
            kb.keepkv_prefill_scores(p, A[l], qwin, st)
        e1.record(); stream.synchronize()
        t_prefill_scores = e0.elapsed_time(e1) * 1e-3 / L
        e0.record()
        for l in range(L):
            kb.keepkv_decode_attention(p, A[l], q_all[0], out, None, True, ws, st)
        e1.record(); stream.synchronize()
        t_full_decode = e0.elapsed_time(e1) * 1e-3 / L
        stats = torch.zeros(L, w.U, 8, dtype=torch.int32, device="cuda")
        # ---- the prefill compression under the merge-first policy (Section 3.4), on copies of the scored prompt
        #      caches (it works in place and the phases below need the prompt as it is); Bc serves as its scratch
        n_mf = min(L, 2)
        mf = [kb.Cache(A[l].K.clone(), A[l].V.clone(), A[l].votes.clone(), A[l].lscore.clone(), A[l].seq_len.clone())
              for l in list(range(n_mf)) + [0]]
        kb.keepkv_compress_merge_first(p, mf[n_mf], Bc[0], budget_arg, ws, st, n_recent_dev=nrec_arg)   # loads the kernels
        stream.synchronize()
        e0.record()
        for l in range(n_mf):
            kb.keepkv_compress_merge_first(p, mf[l], Bc[l], budget_arg, ws, st, n_recent_dev=nrec_arg)
        e1.record(); stream.synchronize()
        t_merge_first = e0.elapsed_time(e1) * 1e-3 / n_mf
        del mf
        kb.keepkv_compress(p, A[0], Bc[0], budget_arg, ws, st, n_recent_dev=nrec_arg, stats=stats[0])   # loads the kernels
        stream.synchronize()
        e0.record()
        for l in range(L):
            kb.keepkv_compress(p, A[l], Bc[l], budget_arg, ws, st, n_recent_dev=nrec_arg, stats=stats[l])
        e1.record(); stream.synchronize()
        t_full_compress = e0.elapsed_time(e1) * 1e-3 / L
        m_full = float(stats[:, :, 2].sum().item()) / (L * w.U)

        # ---- one period as a CUDA graph, in both directions (src/dst swap after every compression)
        def period(cur, oth, stats_t=None):
            n = 0
            for t in range(P):
                for l in range(L):
                    kb.keepkv_decode_step(p_step, cur[l], q_all[t + 1], kn_all[t + 1], vn_all[t + 1], out, None, True, ws, st)
                    n += 1
            for l in range(L):
                kb.keepkv_compress(p_inc, cur[l], oth[l], budget_arg, ws, st, n_recent_dev=nrec_arg,
                                   stats=None if stats_t is None else stats_t[l])
                n += kb.last_launch_count()
            return n

        graphs = []
        per_period = 0
        load_period(); period(Bc, A)          # eager warm-up of both directions (also loads every kernel)
        load_period(); period(A, Bc)
        stream.synchronize()
        for cur, oth in ((Bc, A), (A, Bc)):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                per_period = period(cur, oth, stats)
            graphs.append(g)
        for k in range(args.warmup):
            load_period()
            graphs[k % 2].replay()
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        sampler = ClockSampler(local) if rank == 0 else None
        torch.cuda.synchronize()
        e0.record()
        for k in range(args.steps):
            load_period()
            graphs[(args.warmup + k) % 2].replay()
        e1.record()
        torch.cuda.synchronize()
        t_steps = e0.elapsed_time(e1) * 1e-3
        launches = per_period * args.steps
        clocks = sampler.stop() if sampler else None
        assert int(st.item()) == 0, "device status flag raised during the benchmark"

        # ---- dominant kernel alone: decode over the round-robin layers at mid-period length
        cur = (Bc, A)[(args.warmup + args.steps) % 2]
        oth = A if cur is Bc else Bc
        load_period()
        for t in range(P // 2):              # a real half period with fresh tokens
            for l in range(L):
                kb.keepkv_decode_step(p_step, cur[l], q_all[t + 1], kn_all[t + 1], vn_all[t + 1], out, None, True, ws, st)
        reps = 16
        gd = torch.cuda.CUDAGraph()
        stream.synchronize()
        with torch.cuda.graph(gd, stream=stream):
            for _ in range(reps):
                for l in range(L):
                    kb.keepkv_decode_step(p_step, cur[l], q_all[P // 2], kn_all[P // 2], vn_all[P // 2], out, None, True, ws, st)
        lens_keep = [c_.seq_len.clone() for c_ in cur]            # the launch the loop runs appends: put the lengths back
        gd.replay(); stream.synchronize()
        for c_, n_ in zip(cur, lens_keep):
            c_.seq_len.copy_(n_)
        e0.record(); gd.replay(); e1.record(); stream.synchronize()
        for c_, n_ in zip(cur, lens_keep):
            c_.seq_len.copy_(n_)
        t_decode = e0.elapsed_time(e1) * 1e-3 / (reps * L)
        # ---- compression alone (incremental, budget + P -> budget), as a graph of the L calls
        for t in range(P // 2, P):
            for l in range(L):
                kb.keepkv_decode_step(p_step, cur[l], q_all[t + 1], kn_all[t + 1], vn_all[t + 1], out, None, True, ws, st)
        gc = torch.cuda.CUDAGraph()
        stream.synchronize()
        with torch.cuda.graph(gc, stream=stream):
            for l in range(L):
                kb.keepkv_compress(p_inc, cur[l], oth[l], budget_arg, ws, st, n_recent_dev=nrec_arg, stats=stats[l])
        gc.replay(); stream.synchronize()
        e0.record(); gc.replay(); gc.replay(); e1.record(); stream.synchronize()
        t_inc_compress = e0.elapsed_time(e1) * 1e-3 / (2 * L)
        m_inc = float(stats[:, :, 2].sum().item()) / (L * w.U)
        # ---- the same compression in place (position array; only evicted / merged rows are touched), on copies
        t_inplace = None
        if not ragged:
            ip = [kb.Cache(c_.K.clone(), c_.V.clone(), c_.votes.clone(), c_.lscore.clone(), c_.seq_len.clone()) for c_ in cur[:min(L, 4)]]
            pos0 = torch.arange(n_cap, dtype=torch.int32, device="cuda").expand(w.B, w.H_kv, n_cap).contiguous()
            pos_l = [pos0.clone() for _ in ip]
            plen_l = [c_.seq_len.clone() for c_ in ip]
            seen_l = [c_.seq_len.clone() for c_ in ip]
            for c_, a_, b_, s_ in zip(ip, pos_l, plen_l, seen_l):     # warm (loads the kernels); then restore the lengths
                kb.keepkv_compress_inplace(p, c_, a_, b_, s_, budget_arg, ws, st)
            stream.synchronize()
            for c_, b_, src_ in zip(ip, plen_l, cur):
                c_.seq_len.copy_(src_.seq_len); b_.copy_(src_.seq_len)   # rows beyond the budget count as fresh tokens again
            e0.record()
            for c_, a_, b_, s_ in zip(ip, pos_l, plen_l, seen_l):
                kb.keepkv_compress_inplace(p, c_, a_, b_, s_, budget_arg, ws, st)
            e1.record(); stream.synchronize()
            t_inplace = e0.elapsed_time(e1) * 1e-3 / len(ip)
            del ip, pos_l
        cur, oth = oth, cur                   # the compressed caches are current now

        # ---- end to end through the host-buffer entry point: pinned inputs in, outputs back, every step
        pin = lambda t: t.cpu().pin_memory()
        qh, knh, vnh = pin(q_pool), pin(kn_pool), pin(vn_pool)
        # One decode step of all layers through the host-buffer entry point (one H2D copy each of the layers'
        # queries, keys and values from pinned memory, one launch per layer, one D2H copy of the outputs).  The
        # host lays a period's inputs out per step and layer beforehand (a serving loop would have produced them
        # there); the timed region is the steps themselves: enqueue, copies, kernels, and the wait for the
        # outputs that the next token depends on.
        # a step's queries, keys and values lie back to back, on the host and in the staging buffer on the device:
        # the entry point then moves them with one copy
        nq, nk = L * w.B * w.H_q * w.d, L * w.B * w.H_kv * w.d
        in_h = torch.empty(P, nq + 2 * nk, dtype=torch.bfloat16).pin_memory()         # one period of host inputs
        in_d = torch.empty(nq + 2 * nk, dtype=torch.bfloat16, device="cuda")
        qh_p = in_h[:, :nq].view(P, L, w.B, w.H_q, w.d)
        knh_p = in_h[:, nq:nq + nk].view(P, L, w.B, w.H_kv, w.d)
        vnh_p = in_h[:, nq + nk:].view(P, L, w.B, w.H_kv, w.d)
        oh = torch.empty(L, w.B, w.H_q, w.d, dtype=torch.bfloat16).pin_memory()
        qd, kd, vd = in_d[:nq].view(L, w.B, w.H_q, w.d), in_d[nq:nq + nk].view(L, w.B, w.H_kv, w.d), in_d[nq + nk:].view(L, w.B, w.H_kv, w.d)
        od = torch.empty_like(oh, device="cuda")

        def period_e2e(cur, oth):
            k = pool_next[0]
            pool_next[0] += 1
            assert k < n_pool
            sl = slice(1 + k * P, 1 + (k + 1) * P)
            for dst_h, src_h in ((qh_p, qh), (knh_p, knh), (vnh_p, vnh)):
                dst_h.copy_(src_h[sl].unsqueeze(1).expand_as(dst_h))
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for t in range(P):
                kb.keepkv_decode_step_host_layers(p_step, cur, qh_p[t], knh_p[t], vnh_p[t], oh, qd, kd, vd, od, True, ws, st)
                stream.synchronize()          # the next token's queries depend on this step's output
            for l in range(L):
                kb.keepkv_compress(p_inc, cur[l], oth[l], budget_arg, ws, st, n_recent_dev=nrec_arg)
            stream.synchronize()
            return time.perf_counter() - t0

        pair = [(cur, oth), (oth, cur)]
        period_e2e(*pair[0]); period_e2e(*pair[1])
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        t_e2e = sum(period_e2e(*pair[k % 2]) for k in range(n_e2e)) / n_e2e

    # ---- reduce over ranks: slowest rank's time, summed tokens
    t_steps, t_e2e = slowest_rank([t_steps, t_e2e], dist, "cuda")
    tokens_per_step = w.B * P * L * world
    value = job_throughput(w.B * P * L, world, args.steps, t_steps)
    e2e_val = job_throughput(w.B * P * L, world, 1, t_e2e)
    hbm, tens, src = peaks()
    bud64 = bud.astype(np.int64)
    entries = int((bud64 + P // 2 + 8).sum()) * w.H_kv      # the timed launches append: 16 replays from mid period
    ach = decode_bytes(w, entries) / t_decode / 1e9
    full_dec_gbs = decode_bytes(w, int(lens.astype(np.int64).sum()) * w.H_kv) / t_full_decode / 1e9

    def cbytes(len_b, m_per_unit):   # algorithmic bytes of one compression, summed over the units
        per_seq = len_b * 2 * w.d + (bud64 + m_per_unit) * 2 * w.d + len_b * 8 + bud64 * (4 * w.d + 8)
        return float(per_seq.sum()) * w.H_kv

    inc_bytes, full_bytes = cbytes(bud64 + P, m_inc), cbytes(lens.astype(np.int64), m_full)
    inc_gbs = inc_bytes / t_inc_compress / 1e9
    full_gbs = full_bytes / t_full_compress / 1e9
    gemm_flops = float((2.0 * (lens.astype(np.int64) - bud64) * bud64 * w.d).sum()) * w.H_kv
    # windowed initialisation: every key once, lscore written, the window queries
    pf_bytes = float(lens.astype(np.int64).sum()) * w.H_kv * (2 * w.d + 4) + 2.0 * w.B * w.H_q * 32 * w.d
    pf_gbs = pf_bytes / t_prefill_scores / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": t_steps / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_dict(w, args),
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_val, "unit": UNIT,
                "h2d_bytes_per_step": int(L * P * (q_all[0].numel() + 2 * kn_all[0].numel()) * 2),
                "d2h_bytes_per_step": int(L * P * out.numel() * 2), "steps": n_e2e,
                "note": "keepkv_decode_step_host_layers called once per token for all layers, stream sync after every step"},
        "roofline": {"bound": "hbm", "kernel": "decode_kernel (keepkv_decode_step, the launch the timed loop runs)",
                     "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": ach / hbm, "peak_source": src,
                     "traffic": DECODE_TRAFFIC_BYTES.get(w.name),
                     "bytes_per_launch": decode_bytes(w, entries), "us_per_launch": t_decode * 1e6},
        "roofline_compress_incremental": {
            "bound": "hbm", "kernel": "steady_compress_kernel" if steady else "compression pipeline (5 kernels)",
            "achieved": inc_gbs, "peak": hbm, "unit": "GB/s", "frac": inc_gbs / hbm, "peak_source": src, "traffic": None,
            "bytes_per_call": inc_bytes, "us_per_call": t_inc_compress * 1e6},
        "roofline_compress_full": {
            "bound": "tensor", "kernel": "nominate_kernel (similarity search of the first compression)",
            "achieved": gemm_flops / t_full_compress / 1e12, "peak": tens, "unit": "TFLOP/s",
            "frac": gemm_flops / t_full_compress / 1e12 / tens, "peak_source": src + " (sustained bf16)", "traffic": None,
            "flops_per_call": gemm_flops, "us_per_call": t_full_compress * 1e6},
        "phases": {
            "decode_steady_us": t_decode * 1e6, "decode_steady_gbs": ach, "decode_steady_frac_hbm": ach / hbm,
            "decode_full_cache_us": t_full_decode * 1e6, "decode_full_cache_gbs": full_dec_gbs,
            "decode_full_cache_frac_hbm": full_dec_gbs / hbm,
            "prefill_scores_us": t_prefill_scores * 1e6, "prefill_scores_gbs": pf_gbs,
            "prefill_scores_frac_hbm": pf_gbs / hbm,
            "compress_incremental_us": t_inc_compress * 1e6, "compress_incremental_gbs": inc_gbs,
            "compress_incremental_frac_hbm": inc_gbs / hbm, "merged_per_unit_incremental": m_inc,
            "compress_incremental_path": "single kernel (KEEPKV_FLAG_COMPRESS_STEADY)" if steady else "pipeline",
            "compress_full_us": t_full_compress * 1e6, "compress_full_gbs": full_gbs,
            "compress_full_frac_hbm": full_gbs / hbm, "merged_per_unit_full": m_full,
            "compress_full_gemm_tflops": gemm_flops / t_full_compress / 1e12,
            "compress_inplace_us": None if t_inplace is None else t_inplace * 1e6,
            "compress_merge_first_us": t_merge_first * 1e6,
            "compress_inplace_note": "keepkv_compress_inplace on the same caches: rows touched = evicted + merged, not the whole cache",
        },
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            period_s, cores, desc, _, _ = oracle_period_time(w, w.U, min(w.period, 128))
            line["cpu_baseline"] = {"value": w.B * P / period_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": desc}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2", choices=sorted(W.CONFIGS))
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    w = W.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, w, rank)
    else:
        run_ours(args, w, rank, world)


if __name__ == "__main__":
    main()
