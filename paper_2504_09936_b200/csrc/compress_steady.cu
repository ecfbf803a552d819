// keepkv_compress with KEEPKV_FLAG_COMPRESS_STEADY: Algorithm 1 in one kernel for a cache that is only one
// period over its budget.  A unit qualifies when it evicts at most kStEv entries and has at most kStCand
// entries between the sinks and the recent window; the others are reported and left alone.  The R CTAs of
// a unit (grid (R, U)) each
//   1. repeat the selection (Algorithm 1, selection step): keys of the candidates in shared memory, a radix search,
//      one ordered pass -> the kept candidates and the evicted entries as lists in shared memory;
//   2. stream their slice of the retained slots src -> dst (Algorithm 1, insertion step), 64 slots at a time.  The key rows go
//      global -> shared by cp.async into a ring of 128-byte-swizzled tiles, three tiles ahead of their use (a
//      slice that lies in the recent window does not depend on the selection and starts before it), and are
//      stored to dst from there; values pass through registers.  The key tiles are the B operand of a tcgen05.mma (M = 128 evicted keys, staged once as A operand; N = 64; fp32
//      accumulators in tensor memory, double-buffered) that one thread issues per tile (Algorithm 1, similarity step).  All eight
//      warps drain the accumulator of the previous tile with tcgen05.ld while the next product runs: a thread
//      owns one evicted row and half of the columns and keeps the row's two best cosines with their slots;
//   3. leave their two best per row in the workspace; the last CTA of the unit to arrive folds them, settles
//      arg-max and threshold (Algorithm 1, arg-max and threshold step) with the interface's exact fp32 chain wherever the tensor-core ranking is
//      closer than kRankEps, sorts the entries to merge into groups and merges them (Eq. A.3; Algorithm 1, merge step).
// Decisions, and therefore all outputs, are the same bits as the general pipeline's (compress.cu).
// Every wait on the tensor core is bounded; one that runs out raises KEEPKV_DEV_TIMEOUT and the CTA goes on
// without further products (its unit's result is then unspecified), frees its tensor memory and returns.
#include "compress.cuh"
#include "ptx.cuh"

namespace keepkv {

constexpr int kStThreads = 256;
constexpr int kStWarps = kStThreads / 32;
constexpr int kStCand = 2048;    // candidates (entries between sinks and recent window) a CTA holds keys for
constexpr int kStEv = 128;       // evicted entries per unit (rows of the product, lanes of tensor memory)
constexpr int kStRet = 16384;    // retained entries per unit
constexpr int kStN = 64;         // retained slots per tile (columns of the product)
constexpr int kStTmemCols = 128; // two accumulators of kStN columns

template <int D>
struct StSmem {
  static constexpr int kSub = D / 64;                            // 64-channel (128-byte) atoms per row
  static constexpr int kABytes = kSub * kStEv * 128;
  static constexpr int kBBytes = kSub * kStN * 128;
  static constexpr int kStages = 4;
  static constexpr int kStageBytes = kBBytes;                    // one stage: a key tile, swizzled
  static constexpr int kA = 0;                                   // evicted keys, swizzled
  static constexpr int kRing = kA + kABytes;
  static constexpr int kCinv = kRing + kStages * kStageBytes;    // f32 [4][64]   1/|k| of the keys of four tiles
  static constexpr int kEinv = kCinv + 4 * kStN * 4;             // f32 [kStEv]   1/|k_e|
  static constexpr int kXchg = kEinv + kStEv * 4;                // u32 [kStEv][4] column-half exchange
  static constexpr int kHeavy = kXchg + kStEv * 16;              // i32 [kStCand] source index of kept candidates
  static constexpr int kEv = kHeavy + kStCand * 4;               // i32 [kStEv]   source index of evicted entries
  static constexpr int kBytes = kEv + kStEv * 4;
  static constexpr int kKeys = kA;                               // u32 [kStCand] selection keys, gone before A is staged
  // scratch of the last CTA, laid over the operand tiles once the similarity search is over
  static constexpr int kKe = 0;                                  // f32 [kStWarps][D]
  static constexpr int kKc = kKe + kStWarps * D * 4;             // f32 [kStWarps][2][D]
  static constexpr int kQ = kKc + kStWarps * 2 * D * 4;          // i32 [7][kStEv]
  static constexpr int kSkey = kQ + 7 * kStEv * 4;               // u32 [kStEv]
  static constexpr int kGhead = kSkey + kStEv * 4;               // i32 [kStEv + 1]
  static_assert(kGhead + (kStEv + 1) * 4 <= kCinv, "tail scratch must fit the operand tiles");
  static_assert(kStCand * 4 <= kABytes, "selection keys must fit the A tile");
};

template <int D>
__global__ void __launch_bounds__(kStThreads, 2)
steady_compress_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *budget_dev, int budget_scalar,
                       const int32_t *n_recent_dev, int32_t *ret_idx, int32_t *target, UnitInfo *unit_info, float4 *nom_v,
                       int32_t *nom_si, int C_max, int *counters, keepkv_stats *stats, int32_t *status_dev,
                       const float *__restrict__ select_key) {
  using SL = StSmem<D>;
  constexpr int KSTEPS = D / 16;          // k-steps of the similarity product
  constexpr int CH = D / 8;               // 16-byte chunks of a row
  constexpr int RP = kStThreads / CH;     // rows the CTA moves per pass (one chunk per thread)
  constexpr int NP = kStN / RP;           // passes per 64-slot tile
  constexpr uint32_t IDESC = umma_idesc_bf16(kStEv, kStN);
  extern __shared__ __align__(1024) uint8_t st_smem_raw[];
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_sel[3];
  __shared__ int s_last, s_nq;
  __shared__ __align__(8) uint64_t bars[3];   // t_full[2], drain
  __shared__ uint32_t s_tmem;
  __shared__ volatile int s_abort;
  uint8_t *st_smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(st_smem_raw) + 1023) & ~(uintptr_t)1023);
  float *cinv = reinterpret_cast<float *>(st_smem + SL::kCinv);
  float *einv = reinterpret_cast<float *>(st_smem + SL::kEinv);
  uint32_t *xchg = reinterpret_cast<uint32_t *>(st_smem + SL::kXchg);
  uint32_t *keys = reinterpret_cast<uint32_t *>(st_smem + SL::kKeys);
  int *heavy = reinterpret_cast<int *>(st_smem + SL::kHeavy);
  int *ev = reinterpret_cast<int *>(st_smem + SL::kEv);
  const uint32_t bar_t_full = smem_u32(&bars[0]), bar_drain = smem_u32(&bars[2]);

  const int u = blockIdx.y, r = blockIdx.x, R = gridDim.x, b = u / p.H_kv, h = u % p.H_kv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_trigger();
  // ---- the sets of Algorithm 1, selection step, exactly as the general selection defines them
  const int len = max(0, min(src.seq_len[b], p.N_cap));
  int budget = budget_dev ? budget_dev[b] : budget_scalar;
  budget = max(0, min(budget, p.N_cap));
  int n_sink = p.n_sink, n_recent = n_recent_dev ? max(0, n_recent_dev[b]) : p.n_recent;
  int lo, hi, n_heavy;
  if (budget >= len) {
    lo = hi = len;
    n_heavy = 0;
  } else {
    n_sink = min(n_sink, budget);
    n_recent = min(n_recent, budget - n_sink);
    lo = n_sink;
    hi = len - n_recent;
    n_heavy = budget - n_sink - n_recent;
  }
  const int m_cand = hi - lo, n_ret = min(len, budget), n_ev = len - n_ret;
  if (m_cand > kStCand || n_ev > kStEv || n_ret > kStRet) {
    if (r == 0 && tid == 0) atomicOr(status_dev, KEEPKV_DEV_NOT_STEADY);   // the promise does not hold here
    return;
  }
  const size_t base = (size_t)u * p.N_cap;
  if (tid == 0) {
    mbar_init(bar_t_full, 1);
    mbar_init(bar_t_full + 8, 1);
    mbar_init(bar_drain, 1);
    s_abort = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&s_tmem), kStTmemCols);
    tmem_relinquish();
  }
  const uint8_t *kS = reinterpret_cast<const uint8_t *>(src.K) + base * (2 * D);
  const uint8_t *vS = reinterpret_cast<const uint8_t *>(src.V) + base * (2 * D);
  uint8_t *kD = reinterpret_cast<uint8_t *>(dst.K) + base * (2 * D);
  uint8_t *vD = reinterpret_cast<uint8_t *>(dst.V) + base * (2 * D);
  const uint32_t sbase = smem_u32(st_smem);
  // byte offset of 16-byte chunk c of row `row` inside a swizzled tile of `rows` rows
  auto swz = [](int rows, int row, int c) { return (c >> 3) * (rows * 128) + row * 128 + (((c & 7) ^ (row & 7)) << 4); };
  // source index of retained slot s: sinks, kept candidates (known once the selection is done), recent window
  auto ret = [&](int s) { return s < lo ? s : (s < lo + n_heavy ? heavy[s - lo] : hi + (s - lo - n_heavy)); };

  // ---- this CTA's slice of the retained slots, in 64-slot tiles, and the ring that feeds it
  constexpr int S = SL::kStages;
  const int n_tiles = (n_ret + kStN - 1) / kStN;
  const int t0 = (int)((long long)n_tiles * r / R), t1 = (int)((long long)n_tiles * (r + 1) / R);
  const int crow = tid / CH, cch = tid % CH;   // the row (of every pass) and the 16-byte chunk this thread moves
  // The keys of tile t into their stage by cp.async, three tiles ahead of the product; values (with votes and
  // score estimates) pass through registers, one tile ahead.  A commit per call, also for a tile past the
  // slice, keeps the group count uniform.
  auto issue_keys = [&](int t) {
    if (t < t1) {
      const uint32_t st = sbase + SL::kRing + ((t - t0) % S) * SL::kStageBytes;
#pragma unroll
      for (int j = 0; j < NP; ++j) {
        const int rw = j * RP + crow, s = t * kStN + rw;
        const bool ok = s < n_ret;
        cp_async_16(st + swz(kStN, rw, cch), kS + (ok ? (size_t)ret(s) * (2 * D) + cch * 16 : 0), ok);
      }
    }
    cp_async_commit();
  };
  uint4 vr[NP];
  float sv[NP];   // votes (chunk 1) or score estimate (chunk 2) of the row
  int srow[NP];
  auto load_values = [&](int t) {
#pragma unroll
    for (int j = 0; j < NP; ++j) {
      const int s = t * kStN + j * RP + crow;
      srow[j] = (t < t1 && s < n_ret) ? ret(s) : -1;
      vr[j] = make_uint4(0u, 0u, 0u, 0u);
      sv[j] = 0.f;
      if (srow[j] >= 0) {
        vr[j] = *reinterpret_cast<const uint4 *>(vS + (size_t)srow[j] * (2 * D) + cch * 16);
        if (cch == 1) sv[j] = src.votes[base + srow[j]];
        if (cch == 2) sv[j] = src.lscore[base + srow[j]];
      }
    }
  };
  // A slice that starts in the recent window does not depend on the selection: its first tiles are requested now.
  const bool early = t0 * kStN >= lo + n_heavy;
  if (early) { issue_keys(t0); issue_keys(t0 + 1); issue_keys(t0 + 2); load_values(t0); }

  // ---- selection (Algorithm 1, selection step)
  for (int i = tid; i < m_cand; i += kStThreads)   // the caller's scores where given, else kappa = ln p + lscore
    keys[i] = select_key ? ordered_key(select_key[base + lo + i])
                         : kappa_key(src.votes[base + lo + i], src.lscore[base + lo + i]);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  uint32_t kth = 0u;
  int n_tie = 0, tot_ties = 0;
  if (n_heavy > 0) block_radix_select(keys, m_cand, n_heavy, hist, s_sel, kth, n_tie, tot_ties);
  {
    // one ordered pass over the candidates: a thread owns 8 consecutive ones (kStCand = 8 * kStThreads)
    static_assert(kStCand == 8 * kStThreads, "one sweep covers all candidates");
    const bool rank_ties = n_heavy > 0 && n_tie < tot_ties;
    const int i0 = tid * 8;
    bool keepf[8], tief[8];
    int n_t = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int i = i0 + j;
      const bool valid = i < m_cand && n_heavy > 0;
      const uint32_t k = valid ? keys[i] : 0u;
      tief[j] = valid && k == kth;
      keepf[j] = valid && k > kth;
      n_t += tief[j] ? 1 : 0;
    }
    if (n_heavy > 0) {
      int tie_rank = 0, tot_tie = 0;
      if (rank_ties) tie_rank = block_excl_sum(n_t, warp_tot, tot_tie, kStWarps);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (tief[j]) { keepf[j] = !rank_ties || tie_rank < n_tie; ++tie_rank; }
    }
    int n_k = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) n_k += keepf[j] ? 1 : 0;
    int tot_keep;
    int slot = block_excl_sum(n_k, warp_tot, tot_keep, kStWarps);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int i = i0 + j;
      if (i < m_cand) {
        if (keepf[j]) heavy[slot++] = lo + i;
        else ev[i - slot] = lo + i;
      }
    }
  }
  __syncthreads();   // the lists are complete; nobody reads the selection keys any more
  if (!early) { issue_keys(t0); issue_keys(t0 + 1); issue_keys(t0 + 2); load_values(t0); }

  const int quarter = warp & 3, half = warp >> 2;   // drain: 32 lanes of tensor memory, 32 of a tile's 64 columns
  const int row = quarter * 32 + lane;              // the evicted entry this thread tracks
  const bool live = quarter * 32 < n_ev;            // the warp's rows exist
  Top2 top, topb;   // two lists over alternate columns: two independent dependency chains
  top.init(0.f);
  topb.init(0.f);
  {
    // The copy (Algorithm 1, insertion step) of tile t, whose keys have landed in their stage and whose values are in vr, with the
    // per-slot records and the inverse norms the product ranks with.
    auto copy_tile = [&](int t) {
      const uint8_t *st = st_smem + SL::kRing + ((t - t0) % S) * SL::kStageBytes;
      float *ci = cinv + ((t - t0) & 3) * kStN;
#pragma unroll
      for (int j = 0; j < NP; ++j) {
        const int rw = j * RP + crow, s = t * kStN + rw;
        const uint4 kr = *reinterpret_cast<const uint4 *>(st + swz(kStN, rw, cch));
        float ss = 0.f;
        const uint32_t w[4] = {kr.x, kr.y, kr.z, kr.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) { ss = fmaf(bf16_lo(w[c]), bf16_lo(w[c]), ss); ss = fmaf(bf16_hi(w[c]), bf16_hi(w[c]), ss); }
#pragma unroll
        for (int o = 1; o < CH; o <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (cch == 0) ci[rw] = rsqrtf(ss);   // rows past the slice: 1/0 = inf, their products 0 * inf never rank
        if (srow[j] >= 0) {
          *reinterpret_cast<uint4 *>(kD + (size_t)s * (2 * D) + cch * 16) = kr;
          *reinterpret_cast<uint4 *>(vD + (size_t)s * (2 * D) + cch * 16) = vr[j];
          if (cch == 0) { ret_idx[base + s] = srow[j]; target[base + srow[j]] = -2; }
          if (cch == 1) dst.votes[base + s] = sv[j];
          if (cch == 2) dst.lscore[base + s] = sv[j];
        }
      }
    };
    {
      // ---- A operand: the evicted keys, sixteen lanes per row, with their inverse norms
      constexpr int REPS = kStEv / 16;
      const int ch = tid & 15, rsub = tid >> 4;
      uint4 val[REPS];
#pragma unroll
      for (int rep = 0; rep < REPS; ++rep) {
        const int rw = rep * 16 + rsub;
        val[rep] = make_uint4(0u, 0u, 0u, 0u);
        if (ch < CH && rw < n_ev) val[rep] = *reinterpret_cast<const uint4 *>(kS + (size_t)ev[rw] * (2 * D) + ch * 16);
      }
#pragma unroll
      for (int rep = 0; rep < REPS; ++rep) {
        const int rw = rep * 16 + rsub;
        float ss = 0.f;
        const uint32_t w[4] = {val[rep].x, val[rep].y, val[rep].z, val[rep].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) { ss = fmaf(bf16_lo(w[c]), bf16_lo(w[c]), ss); ss = fmaf(bf16_hi(w[c]), bf16_hi(w[c]), ss); }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        ss += __shfl_xor_sync(0xffffffffu, ss, 4);
        ss += __shfl_xor_sync(0xffffffffu, ss, 8);
        if (ch < CH) *reinterpret_cast<uint4 *>(st_smem + SL::kA + swz(kStEv, rw, ch)) = val[rep];
        if (ch == 0) einv[rw] = rsqrtf(ss);
      }
    }
    if (t0 < t1) {
      cp_async_wait<2>();
      __syncthreads();
      copy_tile(t0);
      load_values(t0 + 1);
      // values are compared before the division by |k_e|: the closeness margin scales with it
      top.init(2.f * kRankEps / einv[row]);
      topb.init(top.thr);
    }
    // Drains the accumulator of tile i (relative to t0): 32 columns of this thread's row.
    auto drain = [&](int i) {
      tc_fence_after();
      uint32_t acc[32];
      tmem_ld_32x32(tmem + ((uint32_t)(quarter * 32) << 16) + (i & 1) * kStN + half * 32, acc);
      tmem_ld_wait();
      const float *ci = cinv + (i & 3) * kStN + half * 32;
      const int c0 = (t0 + i) * kStN + half * 32;
      if (i == 0) {   // cold lists: insert everything
#pragma unroll
        for (int k = 0; k < 32; k += 4)
          offer4<false>(top, topb, __uint_as_float(acc[k]), __uint_as_float(acc[k + 1]), __uint_as_float(acc[k + 2]),
                        __uint_as_float(acc[k + 3]), *reinterpret_cast<const float4 *>(ci + k), c0 + k);
        top.cut = fmaxf(top.best, topb.best) - top.thr;
      } else {
#pragma unroll
        for (int k = 0; k < 32; k += 4)
          offer4<true>(top, topb, __uint_as_float(acc[k]), __uint_as_float(acc[k + 1]), __uint_as_float(acc[k + 2]),
                       __uint_as_float(acc[k + 3]), *reinterpret_cast<const float4 *>(ci + k), c0 + k);
      }
    };
    // Waits (bounded) until the product of tile i has completed.
    auto wait_product = [&](int i) {
      int ok = 1;
      if (lane == 0) ok = s_abort ? 0 : (int)mbar_wait(bar_t_full + 8 * (i & 1), (i >> 1) & 1);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) s_abort = 1;
      return ok != 0;
    };
    for (int t = t0; t < t1; ++t) {
      const int i = t - t0;
      cp_async_wait<1>();          // the keys of tiles <= t + 1 have landed (this thread's copies)
      fence_proxy_async_smem();    // ... and are visible to the tensor core, like the A tile
      tc_fence_before();
      __syncthreads();             // everyone's; and everyone has finished the previous iteration
      tc_fence_after();
      if (tid == 0 && !s_abort) {
        const uint32_t a_base = sbase + SL::kA, b_base = sbase + SL::kRing + (i % S) * SL::kStageBytes;
#pragma unroll
        for (int k = 0; k < KSTEPS; ++k) {
          const uint64_t ad = umma_desc_sw128(a_base + (k >> 2) * (kStEv * 128) + (k & 3) * 32);
          const uint64_t bd = umma_desc_sw128(b_base + (k >> 2) * (kStN * 128) + (k & 3) * 32);
          umma_bf16(tmem + (i & 1) * kStN, ad, bd, IDESC, k > 0 ? 1u : 0u);
        }
        umma_commit(bar_t_full + 8 * (i & 1));
      }
      // the previous product has completed: its stage can be refilled and its accumulator drained
      const bool prev = i > 0 && wait_product(i - 1);
      issue_keys(t + 3);   // into the stage of tile t - 1
      if (t + 1 < t1) {
        copy_tile(t + 1);
        load_values(t + 2);
      }
      if (prev && live) drain(i - 1);
    }
    cp_async_wait<0>();
    if (t0 < t1 && wait_product(t1 - t0 - 1) && live) drain(t1 - t0 - 1);
  }
  // ---- tensor memory is no longer needed
  __syncthreads();
  if (s_abort && tid == 0) {
    atomicOr(status_dev, KEEPKV_DEV_TIMEOUT);
    umma_commit(bar_drain);
    mbar_wait(bar_drain, 0);   // products still in flight get a bounded chance to retire
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kStTmemCols);
  }
  // ---- per evicted row: the two lists and the two column halves folded (equal values -> lower slot),
  // scaled by the row's own inverse norm
  top.insert_any(topb.best, topb.bi);
  top.insert_any(topb.second, topb.si);
  if (half == 1) {
    xchg[row * 4] = __float_as_uint(top.best); xchg[row * 4 + 1] = (uint32_t)top.bi;
    xchg[row * 4 + 2] = __float_as_uint(top.second); xchg[row * 4 + 3] = (uint32_t)top.si;
  }
  __syncthreads();
  const bool valid = tid < n_ev;   // threads 0..127 are the first column half of rows 0..127
  Top2 mine;
  mine.init(0.f);
  if (valid) {
    mine = top;
    mine.insert_any(__uint_as_float(xchg[row * 4]), (int)xchg[row * 4 + 1]);
    mine.insert_any(__uint_as_float(xchg[row * 4 + 2]), (int)xchg[row * 4 + 3]);
    mine.best *= einv[row];
    mine.second *= einv[row];
  }
  if (R > 1) {
    if (valid) {
      nom_v[(base + tid) * C_max + r] = make_float4(mine.best, mine.second, 0.f, __int_as_float(mine.bi));
      nom_si[(base + tid) * C_max + r] = mine.si;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      s_last = atomicAdd(&counters[u], 1) == R - 1;
      if (s_last) counters[u] = 0;   // ready for the next call
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (valid) {
      mine.init(0.f);
      for (int c = 0; c < R; ++c) {   // chunks hold ascending slots: strict comparisons keep the lower slot on ties
        const float4 v = __ldcg(&nom_v[(base + tid) * C_max + c]);
        mine.insert(v.x, __float_as_int(v.w));
        mine.insert(v.y, __ldcg(&nom_si[(base + tid) * C_max + c]));
      }
    }
  }

  // ---- Algorithm 1, arg-max and threshold step: arg-max and threshold; the interface's exact arithmetic where the ranking is too close to call
  float *ke_s = reinterpret_cast<float *>(st_smem + SL::kKe), *kc_s = reinterpret_cast<float *>(st_smem + SL::kKc);
  int *qs = reinterpret_cast<int *>(st_smem + SL::kQ);
  int *q_tid = qs, *q_e = qs + kStEv, *q_kind = qs + 2 * kStEv, *q_a = qs + 3 * kStEv, *q_b = qs + 4 * kStEv,
      *res_slot = qs + 5 * kStEv, *res_merge = qs + 6 * kStEv;
  uint32_t *skey = reinterpret_cast<uint32_t *>(st_smem + SL::kSkey);
  int *ghead = reinterpret_cast<int *>(st_smem + SL::kGhead);
  const __nv_bfloat16 *sK = reinterpret_cast<const __nv_bfloat16 *>(src.K) + base * D;
  const float T = p.merge_threshold;
  int e = 0, slot = -1, kind = 0;
  bool merge = false;
  if (valid) {
    e = ev[tid];
    if (mine.bi >= 0) {
      slot = mine.bi;
      if (!(mine.best - mine.second > kRankEps)) kind = mine.si >= 0 ? 1 : 2;
      else if (!(fabsf(mine.best - T) > kRankEps)) kind = 2;
      else merge = mine.best > T;
    }
  }
  if (tid == 0) s_nq = 0;
  __syncthreads();   // every warp has left the similarity product: the key rows' memory is free
  if (kind) {
    const int qi = atomicAdd(&s_nq, 1);
    q_tid[qi] = tid; q_e[qi] = e; q_kind[qi] = kind; q_a[qi] = mine.bi; q_b[qi] = mine.si;
  }
  __syncthreads();
  for (int qi = warp; qi < s_nq; qi += kStWarps) {
    const int ee = q_e[qi], kd = q_kind[qi], ca = q_a[qi], cb = kd == 1 ? q_b[qi] : q_a[qi];
    float u0, u1;
    exact_cosines<D>(sK + (size_t)ee * D, sK + (size_t)ret(ca) * D, sK + (size_t)ret(cb) * D, ke_s + warp * D,
                     kc_s + warp * 2 * D, u0, u1);
    int win = ca;
    float wu = u0;
    if (kd == 1 && (u1 > u0 || (u1 == u0 && cb < ca))) { win = cb; wu = u1; }
    if (lane == 0) { res_slot[q_tid[qi]] = win; res_merge[q_tid[qi]] = wu > T; }
  }
  __syncthreads();
  if (kind) { slot = res_slot[tid]; merge = res_merge[tid] != 0; }

  // ---- groups: the entries to merge sorted by (slot, position)
  int M;
  const int off = block_excl_count(merge, warp_tot, M, kStWarps);
  if (valid) target[base + e] = merge ? slot : -1;
  if (merge) skey[off] = ((uint32_t)slot << 16) | (uint32_t)tid;
  __syncthreads();
  uint32_t mk = 0xFFFFFFFFu;
  int rank = 0;
  if (tid < M) {
    mk = skey[tid];
    for (int j = 0; j < M; ++j) rank += skey[j] < mk ? 1 : 0;
  }
  __syncthreads();
  if (tid < M) skey[rank] = mk;
  __syncthreads();
  const bool head = tid < M && (tid == 0 || (skey[tid] >> 16) != (skey[tid - 1] >> 16));
  int n_groups;
  const int pos = block_excl_count(head, warp_tot, n_groups, kStWarps);
  if (head) ghead[pos] = tid;
  if (tid == 0) {
    ghead[n_groups] = M;
    keepkv_stats st;
    st.n_retained = n_ret; st.n_evicted = n_ev; st.n_merged = 0; st.n_below_T = n_ev - M;
    st.n_guard_groups = 0; st.n_groups = 0; st.max_group = 0; st.reserved = 0;
    stats[u] = st;
    if (h == 0) dst.seq_len[b] = n_ret;
  }
  __syncthreads();
  // ---- Algorithm 1, merge step: one warp per group
  for (int gi = warp; gi < n_groups; gi += kStWarps) {
    const int beg = ghead[gi], n = ghead[gi + 1] - beg;
    const int c = (int)(skey[beg] >> 16);
    merge_group<D>(p, src, dst, c, ret(c), [&](int t) { return ev[skey[beg + t] & 0xFFFFu]; }, n, target + base, base,
                   stats + u);
  }
}

template <int D>
static void launch_steady_t(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                            const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                            int32_t *ret_idx, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                            int32_t *status_dev, const float *select_key, LaunchCtx &ctx) {
  using SL = StSmem<D>;
  const int U = p.B * p.H_kv;
  constexpr size_t smem_bytes = (size_t)SL::kBytes + 1024;   // slack to align the swizzled tiles
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(steady_compress_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    attr_done_dev[dev & 63] = true;
  }
  // CTAs per unit: what two resident CTAs per SM can hold at once, at most one per column chunk of the workspace
  int R = 2 * sm_count() / U;
  R = R < 1 ? 1 : (R > L.nom_chunks ? L.nom_chunks : R);
  launch_pdl(steady_compress_kernel<D>, dim3(R, U), dim3(kStThreads), smem_bytes, ctx.stream, p, src, dst,
             budget_dev, budget_scalar, n_recent_dev, ret_idx, target, reinterpret_cast<UnitInfo *>(ws + L.unit_info),
             reinterpret_cast<float4 *>(ws + L.nom_v), reinterpret_cast<int32_t *>(ws + L.nom_si), L.nom_chunks,
             reinterpret_cast<int *>(ws + L.counters), stats, status_dev, select_key);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_compress_steady(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                            const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                            int32_t *ret_idx, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                            int32_t *status_dev, const float *select_key, LaunchCtx &ctx) {
  if (p.d == 128)
    launch_steady_t<128>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L, status_dev,
                         select_key, ctx);
  else
    launch_steady_t<64>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L, status_dev,
                        select_key, ctx);
}

}  // namespace keepkv
