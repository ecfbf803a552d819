// keepkv_compress: Algorithm 1 of the paper, out of place, one (sequence, kv-head) unit at a time.
//   select   -> retained / evicted sets from the key kappa = ln p + lscore       (Algorithm 1, selection step)
//   compact  -> retained rows copied to dst in ascending source order            (Algorithm 1, insertion step)
//   nominate -> two best cosines of every evicted key over the retained keys,
//               on the tensor cores (nominate.cu)                                (Algorithm 1, similarity step)
//   resolve  -> arg-max and threshold of Algorithm 1, decided in the interface's fixed fp32
//               arithmetic wherever the tensor-core ranking is too close to call; members
//               of each retained slot sorted into groups                         (many-to-one, App. A.2)
//   merge    -> Eq. A.3 with the EMA estimate as score                           (Algorithm 1, merge step)
#include "compress.cuh"

namespace keepkv {

constexpr int kWarpSelectMax = 2048;   // candidate sets up to this size are searched by one warp, without block barriers

// ------------------------------------------------------------------ select
// One CTA per unit.  The keys of the whole unit live in shared memory; the heavy-hitter threshold
// is found by a 4-pass radix select over the candidates [lo, hi), and one ordered pass writes the
// retained list, the evicted list and the per-entry marks.
__global__ void __launch_bounds__(1024)
select_kernel(keepkv_params p, keepkv_cache src, int32_t *dst_seq_len, const int32_t *budget_dev, int budget_scalar,
              const int32_t *n_recent_dev, int32_t *ret_idx, int32_t *target, int32_t *ev_idx, UnitInfo *unit_info,
              keepkv_stats *stats, const float *__restrict__ select_key, const int32_t *__restrict__ unit_len,
              int32_t *pos, const int32_t *pos_len, const int32_t *n_seen, int32_t *status_dev) {
  extern __shared__ uint32_t keys[];
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_kr, s_cnt;
  const int u = blockIdx.x, b = u / p.H_kv, h = u % p.H_kv, tid = threadIdx.x;
  pdl_wait();
  pdl_trigger();
  // (unit_len: the heads of a sequence differ in length -- only between the two passes of the merge-first compression)
  const int len = max(0, min(unit_len ? unit_len[u] : src.seq_len[b], p.N_cap));
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
  const size_t base = (size_t)u * p.N_cap;
  // Short units need few threads, and every barrier below costs by the warp: the surplus warps leave.
  const int nthr = min((int)blockDim.x, max(128, ((len + 3) / 4 + 31) & ~31)), nw = nthr >> 5;
  if (tid >= nthr) return;
  if (pos) {
    // A cache that is not in token order (in-place compression): sinks and recent window are told by the token
    // position of a row, not by the row.  Rows from pos_len[b] on are the tokens appended since the last call, in
    // order: they get their positions here.  A sink or recent row takes key 0, below every real key, so that the
    // search over all rows ranks the candidates only; what the row order decides elsewhere (equal keys), it
    // decides here too.
    const int first_fresh = max(0, min(pos_len[b], len)), n_total = n_seen[b] + (len - first_fresh);
    const bool all = budget >= len;
    int n_fixed = 0;
    for (int i = tid; i < len; i += nthr) {
      int ps = pos[base + i];
      if (i >= first_fresh) { ps = n_seen[b] + (i - first_fresh); pos[base + i] = ps; }
      const bool fixed = all || ps < n_sink || ps >= n_total - n_recent;
      n_fixed += (!all && fixed) ? 1 : 0;
      keys[i] = fixed ? 0u : kappa_key(src.votes[base + i], src.lscore[base + i]);
    }
    int tot;
    block_excl_sum(n_fixed, warp_tot, tot, nw);
    // the n_sink first and the n_recent last tokens must all be present (they are, if the windows never grew faster
    // than the cache): otherwise positions and ranks disagree and the unit is reported, its result unspecified
    if (!all && tot != n_sink + n_recent && tid == 0) atomicOr(status_dev, KEEPKV_DEV_POSITIONS);
    lo = 0;
    hi = len;
  } else {
    for (int i = tid; i < len; i += nthr) {
      // the caller's scores where given, else kappa = ln p + lscore
      keys[i] = select_key ? ordered_key(select_key[base + i]) : kappa_key(src.votes[base + i], src.lscore[base + i]);
    }
  }
  __syncthreads();

  uint32_t kth = 0;
  int n_tie = 0, tot_ties = 0;
  const int m_cand = hi - lo;
  if (n_heavy > 0 && m_cand <= kWarpSelectMax) {
    // few candidates (every steady-state compression): warp 0 alone finds the threshold, so the four
    // digit passes cost no block barrier
    if (tid < 32) {
      uint32_t k_ = 0;
      int nt_ = 0, tt_ = 0;
      warp_radix_select(keys, lo, hi, n_heavy, hist, k_, nt_, tt_);
      if (tid == 0) { s_prefix = k_; s_kr = nt_; s_cnt = tt_; }
    }
    __syncthreads();
    kth = s_prefix;
    n_tie = s_kr;
    tot_ties = s_cnt;
  } else if (n_heavy > 0) {
    uint32_t prefix = 0, mask = 0;
    int kr = n_heavy;
    const int lane = tid & 31;
    for (int pass = 3; pass >= 0; --pass) {
      for (int i = tid; i < 256; i += nthr) hist[i] = 0;
      __syncthreads();
      for (int start = lo; start < hi; start += nthr) {
        const int i = start + tid;
        const uint32_t k = i < hi ? keys[i] : 0u;
        const bool in = i < hi && (k & mask) == prefix;
        // one shared-memory atomic per distinct bin of the warp (the leading bytes of most keys coincide)
        const int bin = in ? (int)((k >> (8 * pass)) & 255u) : -1 - lane;
        const unsigned peers = __match_any_sync(0xffffffffu, bin);
        if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
      }
      __syncthreads();
      if (tid < 32) {
        // bins are scanned from the top: lane l owns bins 8l..8l+7
        int c[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = hist[8 * lane + j]; sum += c[j]; }
        int x = sum;   // becomes the count in bins of lanes >= lane
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_down_sync(0xffffffffu, x, o);
          if (lane + o < 32) x += y;
        }
        const int above = x - sum;
        if (above < kr && x >= kr) {
          int cum = above, bin = 0, cnt = 0;
          bool found = false;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (!found) {
              if (cum + c[j] >= kr) { bin = j; cnt = c[j]; found = true; }
              else cum += c[j];
            }
          }
          s_prefix = prefix | ((uint32_t)(8 * lane + bin) << (8 * pass));
          s_kr = kr - cum;
          s_cnt = cnt;
        }
      }
      __syncthreads();   // s_prefix is not written again before the second barrier of the next pass
      prefix = s_prefix;
      kr = s_kr;
      mask |= 0xFFu << (8 * pass);
    }
    kth = prefix;        // the n_heavy-th largest key
    n_tie = kr;          // how many entries equal to it are taken, lowest index first
    tot_ties = s_cnt;    // how many entries equal to it exist (the last pass counted full keys)
  }

  // One ordered pass writes both lists: every thread owns a run of consecutive entries, so one block
  // scan per sweep gives the slots.  The rank among keys equal to the threshold is needed only if
  // some of them lose.
  const bool rank_ties = n_heavy > 0 && n_tie < tot_ties;
  auto valid_key = [&](int i) { return i < len ? keys[i] : 0u; };
  constexpr int RUN = 4;
  int base_tie = 0, base_keep = 0;
  for (int start = 0; start < len; start += nthr * RUN) {
    const int i0 = start + tid * RUN;
    bool keepf[RUN], tief[RUN];
    int n_t = 0;
#pragma unroll
    for (int r = 0; r < RUN; ++r) {
      const int i = i0 + r;
      const uint32_t k = valid_key(i);
      const bool valid = i < len, in_mid = valid && i >= lo && i < hi && !(pos && k == 0u);
      tief[r] = false;
      if (!in_mid) {
        keepf[r] = valid;
      } else {
        tief[r] = n_heavy > 0 && k == kth;
        keepf[r] = n_heavy > 0 && k > kth;   // ties are added below
        n_t += tief[r] ? 1 : 0;
      }
    }
    if (n_heavy > 0) {
      int tie_rank = base_tie, tot_tie = 0;
      if (rank_ties) tie_rank += block_excl_sum(n_t, warp_tot, tot_tie, nw);
#pragma unroll
      for (int r = 0; r < RUN; ++r)
        if (tief[r]) { keepf[r] = !rank_ties || tie_rank < n_tie; ++tie_rank; }
      base_tie += tot_tie;
    }
    int n_k = 0;
#pragma unroll
    for (int r = 0; r < RUN; ++r) n_k += keepf[r] ? 1 : 0;
    int tot_keep;
    int slot = base_keep + block_excl_sum(n_k, warp_tot, tot_keep, nw);
#pragma unroll
    for (int r = 0; r < RUN; ++r) {
      const int i = i0 + r;
      if (i < len) {
        if (keepf[r]) {
          ret_idx[base + slot] = i;
          target[base + i] = -2;
          ++slot;
        } else {
          ev_idx[base + (i - slot)] = i;
          target[base + i] = -1;
        }
      }
    }
    base_keep += tot_keep;
  }
  if (tid == 0) {
    UnitInfo ui{len, base_keep, len - base_keep, 0, 0, 0, base_keep, 0};   // (pad0: the retained count once more, for the in-place path)
    unit_info[u] = ui;
    if (h == 0 && dst_seq_len) dst_seq_len[b] = base_keep;   // (in place: the length changes when the rows have moved)
    keepkv_stats st;
    st.n_retained = base_keep; st.n_evicted = len - base_keep; st.n_merged = 0;
    st.n_below_T = len - base_keep;   // resolve_kernel replaces this once targets are known
    st.n_guard_groups = 0; st.n_groups = 0; st.max_group = 0; st.reserved = 0;
    stats[u] = st;
  }
}

// ------------------------------------------------------------------ compact
// grid (up to 32, U), 256 threads, 64 slots per CTA and sweep.  Sixteen lanes move one retained row (a 16-byte piece of
// K and of V each); a warp has eight rows in flight.  The same lanes tree-sum the squared key for
// the inverse norm the similarity search ranks with.
template <int D>
__global__ void __launch_bounds__(256)
compact_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *__restrict__ ret_idx,
               const UnitInfo *__restrict__ unit_info, float *__restrict__ inv_norm) {
  constexpr int CH = D / 8;       // 16-byte chunks per row
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.y, n_ret = unit_info[u].n_ret;
  for (int s0 = blockIdx.x * 64; s0 < n_ret; s0 += gridDim.x * 64) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, ch = lane & 15, sub = lane >> 4;
  const size_t base = (size_t)u * p.N_cap;
  const uint4 *sK = reinterpret_cast<const uint4 *>(src.K), *sV = reinterpret_cast<const uint4 *>(src.V);
  uint4 *dK = reinterpret_cast<uint4 *>(dst.K), *dV = reinterpret_cast<uint4 *>(dst.V);
  int slot[4], si[4];
  uint4 kv[4], vv[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    slot[r] = s0 + warp * 8 + r * 2 + sub;
    si[r] = slot[r] < n_ret ? ret_idx[base + slot[r]] : -1;
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    kv[r] = make_uint4(0, 0, 0, 0);
    vv[r] = kv[r];
    if (si[r] >= 0 && ch < CH) {
      kv[r] = sK[(base + si[r]) * CH + ch];
      vv[r] = sV[(base + si[r]) * CH + ch];
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    if (si[r] >= 0 && ch < CH) {
      dK[(base + slot[r]) * CH + ch] = kv[r];
      dV[(base + slot[r]) * CH + ch] = vv[r];
    }
    float ss = 0.f;
    const uint32_t w[4] = {kv[r].x, kv[r].y, kv[r].z, kv[r].w};
#pragma unroll
    for (int q = 0; q < 4; ++q) { const float a = bf16_lo(w[q]), b = bf16_hi(w[q]); ss = fmaf(a, a, ss); ss = fmaf(b, b, ss); }
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
    ss += __shfl_xor_sync(0xffffffffu, ss, 8);
    if (si[r] >= 0 && ch == 0) {
      inv_norm[base + slot[r]] = rsqrtf(ss);
      dst.votes[base + slot[r]] = src.votes[base + si[r]];
      dst.lscore[base + slot[r]] = src.lscore[base + si[r]];
    }
  }
  }
}

// ------------------------------------------------------------------ resolve + group
// grid (R, U).  The tensor-core search left, per evicted entry, the largest cosines over the retained
// keys (best and second, with their slots).  Its values differ from the interface's
// fp32 chain only by accumulation order (far below kRankEps), so:
//   best - second > eps              the arg-max is settled; otherwise both candidates are re-evaluated
//                                    with the exact chain and the larger wins (equal -> lower slot);
//   |best - T|    <= eps             the threshold test uses the exact chain of the winner.
// (Three distinct cosines within the accumulation error of each other, the one case this cannot
// settle, would need a coincidence of order 1e-8 per row; exact duplicates are handled, because equal
// keys give equal values and the lower slot stays in front.)
// Rows that need the exact chain are queued and shared out over the warps of the CTA (coalesced row
// loads into shared memory, the sequential chains on three lanes).  The last CTA of a unit to finish
// sorts the entries to merge by (slot, position), which makes every group contiguous and ascending.
constexpr int kMergeInline = 32;   // units with at most this many groups are merged by resolve_kernel itself
constexpr int kResolveThreads = 512;
constexpr int kResolveWarps = kResolveThreads / 32;

// Sorts the M entries to merge of unit u by (slot, position) -- which makes every group contiguous and ascending --,
// publishes the sorted members and the start of every group, and merges the groups itself when there are few.
// Called by a whole CTA of kResolveThreads threads.  keys: where the M keys are now (key_smem when `single`, else gk).
template <int D>
__device__ __forceinline__ void group_and_merge(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                                                int u, size_t base, int n_ev, int M, bool single, uint32_t *key_smem,
                                                int smem_keys, uint32_t *gk, const int32_t *__restrict__ ret_idx,
                                                const int32_t *__restrict__ ev_idx, int32_t *target, int32_t *grp_head,
                                                UnitInfo *unit_info, keepkv_stats *stats, int *warp_tot) {
  const int tid = threadIdx.x, warp = tid >> 5;
  int Mp = 1;
  while (Mp < M) Mp <<= 1;
  uint32_t *keys = (single || Mp <= smem_keys) ? key_smem : gk;
  if (keys != gk && !single)
    for (int i = tid; i < M; i += kResolveThreads) keys[i] = __ldcg(&gk[i]);
  for (int i = M + tid; i < Mp; i += kResolveThreads) keys[i] = 0xFFFFFFFFu;
  __syncthreads();
  if (Mp <= kResolveThreads && keys == key_smem) {
    // few keys (all distinct): every thread finds the rank of its key by counting, one barrier
    uint32_t mine = 0xFFFFFFFFu;
    int rank = 0;
    if (tid < M) {
      mine = keys[tid];
      for (int j = 0; j < M; ++j) rank += keys[j] < mine ? 1 : 0;
    }
    __syncthreads();
    if (tid < M) keys[rank] = mine;
    __syncthreads();
  } else {
    // bitonic sort, ascending
    for (int k = 2; k <= Mp; k <<= 1) {
      for (int jj = k >> 1; jj > 0; jj >>= 1) {
        for (int i = tid; i < Mp; i += kResolveThreads) {
          const int ixj = i ^ jj;
          if (ixj > i) {
            const uint32_t a = keys[i], b = keys[ixj];
            if ((a > b) == ((i & k) == 0)) { keys[i] = b; keys[ixj] = a; }
          }
        }
        __syncthreads();
      }
    }
  }
  // publish the sorted members and the start of every group
  int n_groups = 0;
  for (int i0 = 0; i0 < M; i0 += kResolveThreads) {
    const int i = i0 + tid;
    const bool head = i < M && (i == 0 || (keys[i] >> 16) != (keys[i - 1] >> 16));
    int tot;
    const int pos = n_groups + block_excl_count(head, warp_tot, tot);
    if (head) grp_head[base + pos] = i;
    if (i < M && keys != gk) gk[i] = keys[i];
    n_groups += tot;
  }
  if (tid == 0) {
    grp_head[base + n_groups] = M;
    unit_info[u].n_groups = n_groups <= kMergeInline ? 0 : n_groups;
    stats[u].n_below_T = n_ev - M;
  }
  if (n_groups <= kMergeInline) {
    // few groups (every steady-state compression): merge them here, one warp per group
    __syncthreads();   // the keys and group starts written above are visible to the whole CTA
    for (int g = warp; g < n_groups; g += kResolveWarps) {
      const int beg = grp_head[base + g], n = grp_head[base + g + 1] - beg;
      const int c = (int)(gk[beg] >> 16);
      merge_group<D>(p, src, dst, c, ret_idx[base + c], [&](int t) { return ev_idx[base + (gk[beg + t] & 0xFFFFu)]; }, n,
                     target + base, base, stats + u);
    }
  }
}


template <int D>
__global__ void __launch_bounds__(kResolveThreads)
resolve_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *__restrict__ ev_idx,
               UnitInfo *unit_info, const float4 *__restrict__ nom_v, const int32_t *__restrict__ nom_si,
               const int32_t *__restrict__ sched, int C_max, const int32_t *__restrict__ ret_idx, int32_t *target,
               uint32_t *grp_key, int key_stride, int32_t *grp_head, keepkv_stats *stats, int smem_keys, int decide_only) {
  extern __shared__ uint32_t key_smem[];
  __shared__ float ke_s[kResolveWarps][D];
  __shared__ float kc_s[kResolveWarps][2][D];
  __shared__ int warp_tot[32];
  __shared__ int s_nq[2], s_base, s_last;
  __shared__ int q_tid[kResolveThreads], q_e[kResolveThreads], q_kind[kResolveThreads], q_a[kResolveThreads],
      q_b[kResolveThreads];
  __shared__ int res_slot[kResolveThreads], res_merge[kResolveThreads];
  const int u = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_trigger();
  const UnitInfo ui = unit_info[u];
  const size_t base = (size_t)u * p.N_cap;
  const __nv_bfloat16 *sK = reinterpret_cast<const __nv_bfloat16 *>(src.K) + base * D;
  const __nv_bfloat16 *dK = reinterpret_cast<const __nv_bfloat16 *>(dst.K) + base * D;
  uint32_t *gk = grp_key + (size_t)u * key_stride;
  const int C = sched[0];
  const float T = p.merge_threshold;
  // CTAs of the unit that have rows; the others leave at once.  A unit whose rows fit one pass of one CTA
  // (every steady-state compression) needs no exchange through global memory.
  const int n_cta = min((int)gridDim.x, (ui.n_ev + kResolveThreads - 1) / kResolveThreads);
  if ((int)blockIdx.x >= n_cta) return;
  const bool single = ui.n_ev <= kResolveThreads && !decide_only;
  if (tid == 0) { s_nq[0] = s_nq[1] = 0; s_base = 0; }
  __syncthreads();

  int pass = 0;
  for (int j0 = blockIdx.x * kResolveThreads; j0 < ui.n_ev; j0 += gridDim.x * kResolveThreads, ++pass) {
    const int j = j0 + tid;
    const bool valid = j < ui.n_ev;
    int e = 0, slot = -1, kind = 0, bi = -1, si = -1;
    bool merge = false;
    if (valid) {
      e = ev_idx[base + j];
      float best = -CUDART_INF_F, second = -CUDART_INF_F;
      for (int c = 0; c < C; ++c) {   // chunks hold ascending slots: strict comparisons keep the lower slot on ties
        const float4 v = nom_v[(base + j) * C_max + c];
        const int vi[2] = {__float_as_int(v.w), nom_si[(base + j) * C_max + c]};
        const float vv[2] = {v.x, v.y};
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const bool p1 = vv[t] > best, p2 = vv[t] > second;
          second = p1 ? best : fmaxf(second, vv[t]);
          si = p1 ? bi : (p2 ? vi[t] : si);
          bi = p1 ? vi[t] : bi;
          best = fmaxf(best, vv[t]);
        }
      }
      if (bi >= 0) {
        slot = bi;
        if (!(best - second > kRankEps)) kind = si >= 0 ? 1 : 2;
        else if (!(fabsf(best - T) > kRankEps)) kind = 2;
        else merge = best > T;
      }
    }
    // ---- rows that need the interface's exact arithmetic, shared out over the warps
    const int par = pass & 1;
    if (kind) {
      const int q = atomicAdd(&s_nq[par], 1);
      q_tid[q] = tid; q_e[q] = e; q_kind[q] = kind; q_a[q] = bi; q_b[q] = si;
    }
    __syncthreads();
    const int nq = s_nq[par];
    if (tid == 0) s_nq[par ^ 1] = 0;   // the next pass counts in the other word
    for (int q = warp; q < nq; q += kResolveWarps) {
      const int ee = q_e[q], kd = q_kind[q], ca = q_a[q], cb = kd == 1 ? q_b[q] : q_a[q];
      float u0, u1;
      exact_cosines<D>(sK + (size_t)ee * D, dK + (size_t)ca * D, dK + (size_t)cb * D, ke_s[warp], &kc_s[warp][0][0], u0, u1);
      int win = ca;
      float wu = u0;
      if (kd == 1 && (u1 > u0 || (u1 == u0 && cb < ca))) { win = cb; wu = u1; }
      if (lane == 0) { res_slot[q_tid[q]] = win; res_merge[q_tid[q]] = win >= 0 && wu > T; }
    }
    __syncthreads();
    if (kind) { slot = res_slot[tid]; merge = res_merge[tid] != 0; }
    if (decide_only) {   // the caller pairs the entries itself (merge-first policy): the partner above T, or -1
      if (valid) target[base + e] = merge ? slot : -1;
      continue;
    }
    // ---- record the decision; entries to merge go to the unit's key list (any order: it is sorted below)
    int tot;
    const int off = block_excl_count(merge, warp_tot, tot);
    if (single) {   // this CTA holds all rows of the unit: its keys never leave shared memory
      if (valid) {
        target[base + e] = merge ? slot : -1;
        if (merge) key_smem[off] = ((uint32_t)slot << 16) | (uint32_t)j;
      }
      if (tid == 0) s_base = tot;
      __syncthreads();
      continue;
    }
    if (tid == 0) s_base = tot ? atomicAdd(&unit_info[u].n_keys, tot) : 0;
    __syncthreads();
    if (valid) {
      target[base + e] = merge ? slot : -1;
      if (merge) gk[s_base + off] = ((uint32_t)slot << 16) | (uint32_t)j;
    }
  }
  if (decide_only) return;
  int M;
  if (single) {
    M = s_base;
  } else {
    // ---- the last CTA of the unit to arrive groups the entries
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&unit_info[u].ticket, 1) == n_cta - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    M = *reinterpret_cast<volatile int *>(&unit_info[u].n_keys);
  }
  group_and_merge<D>(p, src, dst, u, base, ui.n_ev, M, single, key_smem, smem_keys, gk, ret_idx, ev_idx, target, grp_head,
                     unit_info, stats, warp_tot);
}

// ------------------------------------------------------------------ merge
// Units with many groups (the first compression of a long prompt): warps of several CTAs share them.
// Units with few groups were already merged by resolve_kernel, which left n_groups = 0 here.
template <int D>
__global__ void __launch_bounds__(256)
merge_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *__restrict__ ret_idx,
             const int32_t *__restrict__ ev_idx, int32_t *target, const UnitInfo *__restrict__ unit_info,
             const uint32_t *__restrict__ grp_key, int key_stride, const int32_t *__restrict__ grp_head,
             keepkv_stats *stats) {
  const int u = blockIdx.y;
  pdl_wait();
  pdl_trigger();
  const UnitInfo ui = unit_info[u];
  const size_t base = (size_t)u * p.N_cap;
  const uint32_t *gk = grp_key + (size_t)u * key_stride;
  for (int g = blockIdx.x * 8 + (threadIdx.x >> 5); g < ui.n_groups; g += gridDim.x * 8) {
    const int beg = grp_head[base + g], n = grp_head[base + g + 1] - beg;
    const int c = (int)(gk[beg] >> 16);
    merge_group<D>(p, src, dst, c, ret_idx[base + c], [&](int t) { return ev_idx[base + (gk[beg + t] & 0xFFFFu)]; }, n,
                   target + base, base, stats + u);
  }
}

// ------------------------------------------------------------------ host side
template <int D>
static void launch_compress_t(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                              const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                              int32_t *ret_idx, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                              int32_t *status_dev, const float *select_key, LaunchCtx &ctx) {
  const int U = p.B * p.H_kv;
  UnitInfo *ui = reinterpret_cast<UnitInfo *>(ws + L.unit_info);
  int32_t *sched = reinterpret_cast<int32_t *>(ws + L.sched);
  int32_t *ev_idx = reinterpret_cast<int32_t *>(ws + L.ev_idx);
  float *inv_norm = reinterpret_cast<float *>(ws + L.inv_norm);
  float4 *nom_v = reinterpret_cast<float4 *>(ws + L.nom_v);
  int32_t *nom_si = reinterpret_cast<int32_t *>(ws + L.nom_si);
  uint32_t *grp_key = reinterpret_cast<uint32_t *>(ws + L.grp_key);
  int32_t *grp_head = reinterpret_cast<int32_t *>(ws + L.grp_head);
  const int ret_bound = budget_dev ? p.N_cap : (budget_scalar < p.N_cap ? budget_scalar : p.N_cap);

  const size_t sel_smem = (size_t)p.N_cap * sizeof(uint32_t);
  const int smem_keys = L.key_stride < 32768 ? L.key_stride : 32768;
  static bool attr_done_dev[64] = {};   // opt-in to large dynamic shared memory once per device
  int dev = 0;
  cudaGetDevice(&dev);
  bool &attr_done = attr_done_dev[dev & 63];
  if (!attr_done) {
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4);
    cudaFuncSetAttribute(resolve_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    attr_done = true;
  }
  if (p.flags & KEEPKV_FLAG_COMPRESS_STEADY) {   // the caller vouches for every unit: one kernel does it all
    launch_compress_steady(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L, status_dev,
                           select_key, ctx);
    return;
  }
  launch_pdl(select_kernel, dim3(U), dim3(512), sel_smem, ctx.stream, p, src, dst.seq_len, budget_dev, budget_scalar,
             n_recent_dev, ret_idx, target, ev_idx, ui, stats, select_key, (const int32_t *)nullptr, (int32_t *)nullptr,
             (const int32_t *)nullptr, (const int32_t *)nullptr, status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
  if (ret_bound <= 0) return;   // nothing is kept: every entry is dropped, which select has recorded
  const int cgx = (ret_bound + 63) / 64 < 32 ? (ret_bound + 63) / 64 : 32;   // the retained count is only known on the device
  launch_pdl(compact_kernel<D>, dim3(cgx, U), dim3(256), 0, ctx.stream, p, src, dst, ret_idx, ui,
             inv_norm);
  KEEPKV_CHECK_LAUNCH(ctx);
  // T = +inf: no cosine can exceed it, nothing merges -- the eviction strategy alone (what follows a merge-first pass)
  if (isinf(p.merge_threshold) && p.merge_threshold > 0.f) return;
  launch_nominate(p, src, dst, ev_idx, ui, inv_norm, sched, nom_v, nom_si, L.nom_chunks, status_dev, ctx);
  launch_pdl(resolve_kernel<D>, dim3(L.nom_chunks, U), dim3(kResolveThreads), (size_t)smem_keys * 4, ctx.stream,
      p, src, dst, ev_idx, ui, nom_v, nom_si, sched, L.nom_chunks, ret_idx, target, grp_key, L.key_stride, grp_head,
      stats, smem_keys, 0);
  KEEPKV_CHECK_LAUNCH(ctx);
  int gx = 4096 / U;
  gx = gx < 1 ? 1 : (gx > 32 ? 32 : gx);
  launch_pdl(merge_kernel<D>, dim3(gx, U), dim3(256), 0, ctx.stream, p, src, dst, ret_idx, ev_idx, target, ui, grp_key,
             L.key_stride, grp_head, stats);
  KEEPKV_CHECK_LAUNCH(ctx);
}


// ------------------------------------------------------------------ prefill merge-first policy (Section 3.4; App. B, Table 3)
// keepkv_merge_similar: before any eviction, every entry whose most similar OTHER key exceeds T is merged into that
// entry, provided the partner is earlier in the cache and is not itself merged away (the earlier of two entries is
// the target; no entry is both target and member).  The similarity search is the compression's own
// (nominate_kernel + resolve_kernel) with rows and columns both running over all entries of the unit and the
// diagonal masked; what is new is the pairing rule, which needs every entry's partner before any entry can be
// placed:
//   mf_prepare  -> inverse norms of all keys, the identity row list, the unit's sizes
//   nominate    -> two best cosines per entry over all other entries
//   resolve     -> partner above T per entry, exact where the ranking is close       (decide_only)
//   mf_mark     -> members, kept entries and their slots, targets, the key list of the groups
//   compact     -> kept rows to dst
//   group       -> keys sorted into groups, few groups merged at once
//   merge       -> Eq. A.3 for units with many groups
template <int D>
__global__ void __launch_bounds__(256)
mf_prepare_kernel(keepkv_params p, keepkv_cache src, int32_t *ev_idx, UnitInfo *unit_info, float *__restrict__ inv_norm) {
  constexpr int CH = D / 8;
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.y, b = u / p.H_kv;
  const int len = max(0, min(src.seq_len[b], p.N_cap));
  const size_t base = (size_t)u * p.N_cap;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    UnitInfo ui{len, len, len, 0, 0, 0, 0, 0};
    unit_info[u] = ui;
  }
  const uint4 *sK = reinterpret_cast<const uint4 *>(src.K);
  const int lane = threadIdx.x & 31, ch = lane & 15, sub = lane >> 4, warp = threadIdx.x >> 5;
  for (int r0 = blockIdx.x * 16; r0 < len; r0 += gridDim.x * 16) {   // sixteen lanes per row, two rows per warp
    const int i = r0 + warp * 2 + sub;
    uint4 kv = make_uint4(0, 0, 0, 0);
    if (i < len && ch < CH) kv = sK[(base + i) * CH + ch];
    float ss = 0.f;
    const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) { const float a = bf16_lo(w[q]), bb = bf16_hi(w[q]); ss = fmaf(a, a, ss); ss = fmaf(bb, bb, ss); }
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
    ss += __shfl_xor_sync(0xffffffffu, ss, 8);
    if (i < len && ch == 0) { inv_norm[base + i] = rsqrtf(ss); ev_idx[base + i] = i; }
  }
}

// One CTA per unit.  partner[e] (in `target`): the entry e would merge into, or -1.  Writes the kept list (ret_idx),
// the member list (ev_idx), target[e] = slot of the partner for a member / -2 for a kept entry, the group keys
// (slot << 16 | position among the members), sizes and the initial statistics.  slot_of: scratch [N] per unit.
__global__ void __launch_bounds__(1024)
mf_mark_kernel(keepkv_params p, int32_t *unit_len, int32_t *ret_idx, int32_t *target, int32_t *ev_idx, int32_t *slot_of,
               uint32_t *grp_key, int key_stride, UnitInfo *unit_info, keepkv_stats *stats) {
  __shared__ int warp_tot[32];
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.x, tid = threadIdx.x, nthr = blockDim.x, nw = nthr >> 5;
  const int len = unit_info[u].len;
  const size_t base = (size_t)u * p.N_cap;
  int32_t *tg = target + base;
  uint32_t *gk = grp_key + (size_t)u * key_stride;
  auto wants = [&](int e) { const int t = tg[e]; return t >= 0 && t < e; };
  // pass 1: kept entries and their slots (a thread owns a run of consecutive entries)
  constexpr int RUN = 4;
  int n_keep = 0;
  for (int start = 0; start < len; start += nthr * RUN) {
    const int i0 = start + tid * RUN;
    bool mem[RUN];
    int n_k = 0;
#pragma unroll
    for (int r = 0; r < RUN; ++r) {
      const int e = i0 + r;
      mem[r] = e < len && wants(e) && !wants(tg[e]);   // its partner stays: e is a member
      n_k += (e < len && !mem[r]) ? 1 : 0;
    }
    int tot;
    int slot = n_keep + block_excl_sum(n_k, warp_tot, tot, nw);
#pragma unroll
    for (int r = 0; r < RUN; ++r) {
      const int e = i0 + r;
      if (e < len) {
        if (mem[r]) {
          ev_idx[base + (e - slot)] = e;
          slot_of[base + e] = -1 - (e - slot);   // a member: its position among the members
        } else {
          ret_idx[base + slot] = e;
          slot_of[base + e] = slot;
          ++slot;
        }
      }
    }
    n_keep += tot;
  }
  __syncthreads();   // (block scope: the global writes above are visible to the whole CTA)
  // pass 2: members look up the slot of their partner (partners are read before any target is overwritten:
  // a member's partner is a kept entry, and kept entries' targets are rewritten to -2 only after the barrier below)
  for (int e = tid; e < len; e += nthr) {
    const int so = slot_of[base + e];
    if (so < 0) {
      const int pos = -1 - so, slot = slot_of[base + tg[e]];
      gk[pos] = ((uint32_t)slot << 16) | (uint32_t)pos;
      slot_of[base + e] = -0x40000000 + slot;   // remembered for the rewrite below
    }
  }
  __syncthreads();
  for (int e = tid; e < len; e += nthr) {
    const int so = slot_of[base + e];
    tg[e] = so < 0 ? so + 0x40000000 : -2;
  }
  if (tid == 0) {
    const int n_ev = len - n_keep;
    UnitInfo ui{len, n_keep, n_ev, 0, n_ev, 0, 0, 0};   // n_keys: every member is an entry to merge
    unit_info[u] = ui;
    unit_len[u] = n_keep;
    keepkv_stats st;
    st.n_retained = n_keep; st.n_evicted = n_ev; st.n_merged = 0; st.n_below_T = 0;
    st.n_guard_groups = 0; st.n_groups = 0; st.max_group = 0; st.reserved = 0;
    stats[u] = st;
  }
}

// One CTA per unit: the unit's key list (in global memory) sorted into groups; few groups are merged here.
template <int D>
__global__ void __launch_bounds__(kResolveThreads)
group_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *__restrict__ ret_idx,
             const int32_t *__restrict__ ev_idx, int32_t *target, UnitInfo *unit_info, uint32_t *grp_key, int key_stride,
             int32_t *grp_head, keepkv_stats *stats, int smem_keys) {
  extern __shared__ uint32_t key_smem[];
  __shared__ int warp_tot[32];
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.x;
  const UnitInfo ui = unit_info[u];
  const size_t base = (size_t)u * p.N_cap;
  group_and_merge<D>(p, src, dst, u, base, ui.n_ev, ui.n_keys, false, key_smem, smem_keys, grp_key + (size_t)u * key_stride,
                     ret_idx, ev_idx, target, grp_head, unit_info, stats, warp_tot);
}

// Budget of each sequence for the eviction pass: the caller's, capped by the sequence's shortest merged head (the
// heads of a sequence share one seq_len, so they must all end at the same length).
__global__ void mf_budget_kernel(keepkv_params p, const int32_t *budget_dev, int budget_scalar, const int32_t *unit_len,
                                 int32_t *eff_budget) {
  pdl_wait();
  pdl_trigger();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.B) return;
  int m = p.N_cap;
  for (int h = 0; h < p.H_kv; ++h) m = min(m, unit_len[b * p.H_kv + h]);
  const int budget = max(0, min(budget_dev ? budget_dev[b] : budget_scalar, p.N_cap));
  eff_budget[b] = min(budget, m);
}

// What the caller sees of the two passes: the prompt index of every row of the result, and one record of statistics.
__global__ void mf_compose_kernel(keepkv_params p, const int32_t *seq_len, const int32_t *__restrict__ ret1,
                                  const int32_t *__restrict__ ret2, int32_t *ret_out, const keepkv_stats *st1,
                                  const UnitInfo *unit_info, const int32_t *prompt_len, keepkv_stats *stats_out) {
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.y, b = u / p.H_kv;
  const size_t base = (size_t)u * p.N_cap;
  const int n = seq_len[b];
  if (ret_out)
    for (int s = blockIdx.x * blockDim.x + threadIdx.x; s < n; s += gridDim.x * blockDim.x)
      ret_out[base + s] = ret1[base + ret2[base + s]];
  if (stats_out && blockIdx.x == 0 && threadIdx.x == 0) {
    keepkv_stats st = st1[u];
    st.n_evicted = st.n_retained + st.n_evicted - n;   // of the prompt's entries (kept + merged away in the merge pass)
    st.n_retained = n;
    st.n_below_T = 0;
    stats_out[u] = st;
  }
}

template <int D>
static void launch_compress_merge_first_t(const keepkv_params &p, const keepkv_cache &cache, const keepkv_cache &scratch,
                                          const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                                          int32_t *ret_idx_out, keepkv_stats *stats_out, char *ws, const WsLayout &L,
                                          int32_t *status_dev, LaunchCtx &ctx) {
  const int U = p.B * p.H_kv;
  UnitInfo *ui = reinterpret_cast<UnitInfo *>(ws + L.unit_info);
  int32_t *sched = reinterpret_cast<int32_t *>(ws + L.sched);
  int32_t *ret1 = reinterpret_cast<int32_t *>(ws + L.ret_idx);      // kept entries of the merge pass
  int32_t *target = reinterpret_cast<int32_t *>(ws + L.target);
  int32_t *ev_idx = reinterpret_cast<int32_t *>(ws + L.ev_idx);
  float *inv_norm = reinterpret_cast<float *>(ws + L.inv_norm);
  float4 *nom_v = reinterpret_cast<float4 *>(ws + L.nom_v);
  int32_t *nom_si = reinterpret_cast<int32_t *>(ws + L.nom_si);
  uint32_t *grp_key = reinterpret_cast<uint32_t *>(ws + L.grp_key);
  int32_t *grp_head = reinterpret_cast<int32_t *>(ws + L.grp_head);
  keepkv_stats *st1 = reinterpret_cast<keepkv_stats *>(ws + L.stats2);
  keepkv_stats *st2 = reinterpret_cast<keepkv_stats *>(ws + L.stats);
  int32_t *unit_len = reinterpret_cast<int32_t *>(ws + L.unit_len);
  int32_t *eff_budget = reinterpret_cast<int32_t *>(ws + L.eff_budget);
  const int smem_keys = L.key_stride < 32768 ? L.key_stride : 32768;
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4);
    cudaFuncSetAttribute(resolve_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    cudaFuncSetAttribute(group_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    attr_done_dev[dev & 63] = true;
  }
  // ---- pass 1: similar entries merged with each other, cache -> scratch (every head keeps its own length for now)
  int gx = 2 * sm_count() / U;
  gx = gx < 1 ? 1 : (gx > 32 ? 32 : gx);
  launch_pdl(mf_prepare_kernel<D>, dim3(gx, U), dim3(256), 0, ctx.stream, p, cache, ev_idx, ui, inv_norm);
  KEEPKV_CHECK_LAUNCH(ctx);
  // rows and columns are the same keys: the "retained" operand of the search is the prompt itself
  launch_nominate(p, cache, cache, ev_idx, ui, inv_norm, sched, nom_v, nom_si, L.nom_chunks, status_dev, ctx, 1);
  launch_pdl(resolve_kernel<D>, dim3(L.nom_chunks, U), dim3(kResolveThreads), (size_t)smem_keys * 4, ctx.stream,
      p, cache, cache, ev_idx, ui, nom_v, nom_si, sched, L.nom_chunks, ret1, target, grp_key, L.key_stride, grp_head,
      st1, smem_keys, 1);
  KEEPKV_CHECK_LAUNCH(ctx);
  launch_pdl(mf_mark_kernel, dim3(U), dim3(1024), 0, ctx.stream, p, unit_len, ret1, target, ev_idx, grp_head, grp_key,
             L.key_stride, ui, st1);
  KEEPKV_CHECK_LAUNCH(ctx);
  const int cgx = (p.N_cap + 63) / 64 < 32 ? (p.N_cap + 63) / 64 : 32;
  launch_pdl(compact_kernel<D>, dim3(cgx, U), dim3(256), 0, ctx.stream, p, cache, scratch, ret1, ui, inv_norm);
  KEEPKV_CHECK_LAUNCH(ctx);
  launch_pdl(group_kernel<D>, dim3(U), dim3(kResolveThreads), (size_t)smem_keys * 4, ctx.stream, p, cache, scratch, ret1,
             ev_idx, target, ui, grp_key, L.key_stride, grp_head, st1, smem_keys);
  KEEPKV_CHECK_LAUNCH(ctx);
  int mgx = 4096 / U;
  mgx = mgx < 1 ? 1 : (mgx > 32 ? 32 : mgx);
  launch_pdl(merge_kernel<D>, dim3(mgx, U), dim3(256), 0, ctx.stream, p, cache, scratch, ret1, ev_idx, target, ui, grp_key,
             L.key_stride, grp_head, st1);
  KEEPKV_CHECK_LAUNCH(ctx);
  // ---- pass 2: the eviction strategy alone, scratch -> cache
  launch_pdl(mf_budget_kernel, dim3((p.B + 127) / 128), dim3(128), 0, ctx.stream, p, budget_dev, budget_scalar, unit_len,
             eff_budget);
  KEEPKV_CHECK_LAUNCH(ctx);
  int32_t *ret2 = grp_head;   // (free again: the groups are merged)
  launch_pdl(select_kernel, dim3(U), dim3(512), (size_t)p.N_cap * sizeof(uint32_t), ctx.stream, p, scratch, cache.seq_len,
             (const int32_t *)eff_budget, 0, n_recent_dev, ret2, target, ev_idx, ui, st2, (const float *)nullptr,
             (const int32_t *)unit_len, (int32_t *)nullptr, (const int32_t *)nullptr, (const int32_t *)nullptr, status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
  launch_pdl(compact_kernel<D>, dim3(cgx, U), dim3(256), 0, ctx.stream, p, scratch, cache, ret2, ui, inv_norm);
  KEEPKV_CHECK_LAUNCH(ctx);
  if (ret_idx_out || stats_out) {
    launch_pdl(mf_compose_kernel, dim3(4, U), dim3(256), 0, ctx.stream, p, cache.seq_len, ret1, ret2, ret_idx_out, st1, ui,
               unit_len, stats_out);
    KEEPKV_CHECK_LAUNCH(ctx);
  }
}

void launch_compress_merge_first(const keepkv_params &p, const keepkv_cache &cache, const keepkv_cache &scratch,
                                 const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                                 int32_t *ret_idx_out, keepkv_stats *stats_out, char *ws, const WsLayout &L,
                                 int32_t *status_dev, LaunchCtx &ctx) {
  if (p.d == 128)
    launch_compress_merge_first_t<128>(p, cache, scratch, budget_dev, budget_scalar, n_recent_dev, ret_idx_out, stats_out, ws,
                                       L, status_dev, ctx);
  else
    launch_compress_merge_first_t<64>(p, cache, scratch, budget_dev, budget_scalar, n_recent_dev, ret_idx_out, stats_out, ws,
                                      L, status_dev, ctx);
}


// ------------------------------------------------------------------ Algorithm 1 in place (periodic mode, Section 1)
// keepkv_compress_inplace: "discard (k_e, v_e), (k_c, v_c) and insert (k_r, v_r)" taken literally.  Retained entries
// stay where they are, a merged entry overwrites its target's row, and only the retained rows beyond the new
// length move (into the rows of evicted entries below it), so a compression touches O(evicted + merged) rows
// instead of rewriting the cache.  The cache is then no longer in token order: a position array tells sinks and
// recent window (select_kernel in position mode).  The similarity search runs over the cache as it lies: its
// columns are all rows of the unit, and the rows that are not retained are taken out by a NaN in place of their
// inverse norm (a NaN never passes the strict comparisons of the search).
//   select (positions) -> ip_prepare (norms, sizes) -> nominate -> resolve (+ few merges) -> merge -> ip_move
template <int D>
__global__ void __launch_bounds__(256)
ip_prepare_kernel(keepkv_params p, keepkv_cache c, const int32_t *__restrict__ target, int32_t *ident, UnitInfo *unit_info,
                  float *__restrict__ inv_norm) {
  constexpr int CH = D / 8;
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.y;
  const int len = unit_info[u].len;
  const size_t base = (size_t)u * p.N_cap;
  const uint4 *sK = reinterpret_cast<const uint4 *>(c.K);
  const int lane = threadIdx.x & 31, ch = lane & 15, sub = lane >> 4, warp = threadIdx.x >> 5;
  for (int r0 = blockIdx.x * 16; r0 < len; r0 += gridDim.x * 16) {   // sixteen lanes per row, two rows per warp
    const int i = r0 + warp * 2 + sub;
    const bool kept = i < len && target[base + i] == -2;
    uint4 kv = make_uint4(0, 0, 0, 0);
    if (kept && ch < CH) kv = sK[(base + i) * CH + ch];
    float ss = 0.f;
    const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) { const float a = bf16_lo(w[q]), bb = bf16_hi(w[q]); ss = fmaf(a, a, ss); ss = fmaf(bb, bb, ss); }
    ss += __shfl_xor_sync(0xffffffffu, ss, 1);
    ss += __shfl_xor_sync(0xffffffffu, ss, 2);
    ss += __shfl_xor_sync(0xffffffffu, ss, 4);
    ss += __shfl_xor_sync(0xffffffffu, ss, 8);
    if (i < len && ch == 0) {
      inv_norm[base + i] = kept ? rsqrtf(ss) : __int_as_float(0x7fffffff);   // a row that is not retained is no column
      ident[base + i] = i;   // the slot of a target is its row
    }
  }
}

// The search's column count is the unit's length (all rows lie in the operand); the rest of the record stays.
__global__ void ip_columns_kernel(UnitInfo *unit_info, int U, int all_rows) {
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u < U) unit_info[u].n_ret = all_rows ? unit_info[u].len : unit_info[u].pad0;
}

// One CTA per unit: the retained rows at or above the new length move into the evicted rows below it, both in
// ascending order (ev_idx is ascending: the holes are its head; kept is ascending: the movers are its tail).  Then
// the new lengths are published.
template <int D>
__global__ void __launch_bounds__(256)
ip_move_kernel(keepkv_params p, keepkv_cache c, int32_t *pos, int32_t *pos_len, int32_t *n_seen,
               const int32_t *__restrict__ kept, const int32_t *__restrict__ ev_idx, const UnitInfo *__restrict__ unit_info,
               int32_t *moved_from) {
  constexpr int CH = D / 8;
  __shared__ int s_holes;
  pdl_wait();
  pdl_trigger();
  const int u = blockIdx.x, b = u / p.H_kv, h = u % p.H_kv, tid = threadIdx.x;
  const UnitInfo ui = unit_info[u];
  const int n_ret = ui.pad0, n_ev = ui.n_ev;   // pad0: the number of retained rows (n_ret holds the column count of the search)
  const size_t base = (size_t)u * p.N_cap;
  if (tid == 0) {   // holes = evicted rows below n_ret: a prefix of the ascending list
    int lo = 0, hi = n_ev;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (ev_idx[base + mid] < n_ret) lo = mid + 1; else hi = mid; }
    s_holes = lo;
  }
  __syncthreads();
  const int n_holes = s_holes;
  if (moved_from)
    for (int r = tid; r < n_ret; r += blockDim.x) moved_from[base + r] = r;
  __syncthreads();
  uint4 *K = reinterpret_cast<uint4 *>(c.K), *V = reinterpret_cast<uint4 *>(c.V);
  for (int idx = tid; idx < n_holes * 2 * CH; idx += blockDim.x) {   // a row pair (K, V) is 2 * CH pieces of 16 bytes
    const int k = idx / (2 * CH), piece = idx % (2 * CH);
    const int to = ev_idx[base + k], from = kept[base + (n_ret - n_holes + k)];
    uint4 *A = piece < CH ? K : V;
    const int ch = piece < CH ? piece : piece - CH;
    A[(base + to) * CH + ch] = A[(base + from) * CH + ch];
  }
  for (int k = tid; k < n_holes; k += blockDim.x) {
    const int to = ev_idx[base + k], from = kept[base + (n_ret - n_holes + k)];
    c.votes[base + to] = c.votes[base + from];
    c.lscore[base + to] = c.lscore[base + from];
    pos[base + to] = pos[base + from];
    if (moved_from) moved_from[base + to] = from;
  }
  if (h == 0 && tid == 0) {
    const int len = ui.len, first_fresh = max(0, min(pos_len[b], len));
    c.seq_len[b] = n_ret;
    n_seen[b] += len - first_fresh;
    pos_len[b] = n_ret;
  }
}

template <int D>
static void launch_compress_inplace_t(const keepkv_params &p, const keepkv_cache &c, int32_t *pos, int32_t *pos_len,
                                      int32_t *n_seen, const int32_t *budget_dev, int32_t budget_scalar,
                                      const int32_t *n_recent_dev, int32_t *moved_from, int32_t *target, keepkv_stats *stats,
                                      char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx) {
  const int U = p.B * p.H_kv;
  UnitInfo *ui = reinterpret_cast<UnitInfo *>(ws + L.unit_info);
  int32_t *sched = reinterpret_cast<int32_t *>(ws + L.sched);
  int32_t *ident = reinterpret_cast<int32_t *>(ws + L.ret_idx);    // slot -> row: the identity here
  int32_t *kept = reinterpret_cast<int32_t *>(ws + L.kept);        // retained rows, ascending
  int32_t *ev_idx = reinterpret_cast<int32_t *>(ws + L.ev_idx);
  float *inv_norm = reinterpret_cast<float *>(ws + L.inv_norm);
  float4 *nom_v = reinterpret_cast<float4 *>(ws + L.nom_v);
  int32_t *nom_si = reinterpret_cast<int32_t *>(ws + L.nom_si);
  uint32_t *grp_key = reinterpret_cast<uint32_t *>(ws + L.grp_key);
  int32_t *grp_head = reinterpret_cast<int32_t *>(ws + L.grp_head);
  const int smem_keys = L.key_stride < 32768 ? L.key_stride : 32768;
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4);
    cudaFuncSetAttribute(resolve_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 * 4);
    attr_done_dev[dev & 63] = true;
  }
  launch_pdl(select_kernel, dim3(U), dim3(512), (size_t)p.N_cap * sizeof(uint32_t), ctx.stream, p, c, (int32_t *)nullptr,
             budget_dev, budget_scalar, n_recent_dev, kept, target, ev_idx, ui, stats, (const float *)nullptr,
             (const int32_t *)nullptr, pos, (const int32_t *)pos_len, (const int32_t *)n_seen, status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
  int gx = 2 * sm_count() / U;
  gx = gx < 1 ? 1 : (gx > 32 ? 32 : gx);
  launch_pdl(ip_prepare_kernel<D>, dim3(gx, U), dim3(256), 0, ctx.stream, p, c, (const int32_t *)target, ident, ui, inv_norm);
  KEEPKV_CHECK_LAUNCH(ctx);
  const bool merges = !(isinf(p.merge_threshold) && p.merge_threshold > 0.f);
  if (merges) {
    launch_pdl(ip_columns_kernel, dim3((U + 127) / 128), dim3(128), 0, ctx.stream, ui, U, 1);
    KEEPKV_CHECK_LAUNCH(ctx);
    launch_nominate(p, c, c, ev_idx, ui, inv_norm, sched, nom_v, nom_si, L.nom_chunks, status_dev, ctx);
    launch_pdl(resolve_kernel<D>, dim3(L.nom_chunks, U), dim3(kResolveThreads), (size_t)smem_keys * 4, ctx.stream,
        p, c, c, ev_idx, ui, nom_v, nom_si, sched, L.nom_chunks, ident, target, grp_key, L.key_stride, grp_head,
        stats, smem_keys, 0);
    KEEPKV_CHECK_LAUNCH(ctx);
    int mgx = 4096 / U;
    mgx = mgx < 1 ? 1 : (mgx > 32 ? 32 : mgx);
    launch_pdl(merge_kernel<D>, dim3(mgx, U), dim3(256), 0, ctx.stream, p, c, c, ident, ev_idx, target, ui, grp_key,
               L.key_stride, grp_head, stats);
    KEEPKV_CHECK_LAUNCH(ctx);
  }
  launch_pdl(ip_move_kernel<D>, dim3(U), dim3(256), 0, ctx.stream, p, c, pos, pos_len, n_seen, (const int32_t *)kept,
             (const int32_t *)ev_idx, (const UnitInfo *)ui, moved_from);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_compress_inplace(const keepkv_params &p, const keepkv_cache &c, int32_t *pos, int32_t *pos_len, int32_t *n_seen,
                             const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                             int32_t *moved_from, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                             int32_t *status_dev, LaunchCtx &ctx) {
  if (p.d == 128)
    launch_compress_inplace_t<128>(p, c, pos, pos_len, n_seen, budget_dev, budget_scalar, n_recent_dev, moved_from, target,
                                   stats, ws, L, status_dev, ctx);
  else
    launch_compress_inplace_t<64>(p, c, pos, pos_len, n_seen, budget_dev, budget_scalar, n_recent_dev, moved_from, target,
                                  stats, ws, L, status_dev, ctx);
}

void launch_compress(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                     const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev, int32_t *ret_idx,
                     int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L, int32_t *status_dev,
                     LaunchCtx &ctx, const float *select_key) {
  if (p.d == 128)
    launch_compress_t<128>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L,
                           status_dev, select_key, ctx);
  else
    launch_compress_t<64>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L,
                          status_dev, select_key, ctx);
}

}  // namespace keepkv
