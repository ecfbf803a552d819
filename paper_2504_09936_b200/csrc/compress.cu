// keepkv_compress: Algorithm 1 of the paper, out of place, one (sequence, kv-head) unit at a time.
//   select  -> retained / evicted sets from the key kappa = ln p + lscore        (lines 2-3)
//   compact -> retained rows copied to dst in ascending source order             (line 11)
//   match   -> cosine arg-max of every evicted key over the retained keys        (lines 4-5)
//   group   -> members of each retained slot, ascending                          (many-to-one, App. A.2)
//   merge   -> Eq. A.3 with the EMA estimate as score                            (lines 7-10)
#include "common.cuh"

namespace keepkv {

struct UnitInfo { int len, n_ret, n_ev, budget; };

// ------------------------------------------------------------------ block scan of 0/1 flags
// Exclusive prefix count of `flag` over the block in thread order; total returned through `total`.
__device__ __forceinline__ int block_excl_count(bool flag, int *warp_tot, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  const int in_warp = __popc(bal & ((1u << lane) - 1u));
  __syncthreads();  // warp_tot may still be read from the previous call
  if (lane == 0) warp_tot[warp] = __popc(bal);
  __syncthreads();
  int off = 0, tot = 0;
  for (int w = 0; w < nw; ++w) {
    const int t = warp_tot[w];
    if (w < warp) off += t;
    tot += t;
  }
  total = tot;
  return off + in_warp;
}

// Exclusive prefix sum of small non-negative ints over the block (thread order).
__device__ __forceinline__ int block_excl_sum(int v, int *warp_tot, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = x;
  __syncthreads();
  int off = 0, tot = 0;
  for (int w = 0; w < nw; ++w) {
    const int t = warp_tot[w];
    if (w < warp) off += t;
    tot += t;
  }
  total = tot;
  return off + x - v;
}

// Order-preserving map of an fp32 value to u32 (-0 folded onto +0 so equal floats give equal keys).
__device__ __forceinline__ uint32_t ordered_key(float x) {
  x += 0.0f;
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ------------------------------------------------------------------ select
// One CTA per unit.  The keys of the whole unit live in shared memory; the heavy-hitter threshold
// is found by a 4-pass radix select over the candidates [lo, hi), and one ordered pass writes the
// retained list, the evicted list and the per-entry marks.
__global__ void __launch_bounds__(1024)
select_kernel(keepkv_params p, keepkv_cache src, int32_t *dst_seq_len, const int32_t *budget_dev, int budget_scalar,
              const int32_t *n_recent_dev, int32_t *ret_idx, int32_t *target, int32_t *ev_idx, UnitInfo *unit_info,
              keepkv_stats *stats) {
  extern __shared__ uint32_t keys[];
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_kr;
  const int u = blockIdx.x, b = u / p.H_kv, h = u % p.H_kv, tid = threadIdx.x;
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
  const size_t base = (size_t)u * p.N_cap;
  for (int i = tid; i < len; i += blockDim.x) {
    const float pv = src.votes[base + i], ls = src.lscore[base + i];
    // kappa = ln p + lscore in fp64, rounded once to fp32 (p = 1 needs no logarithm)
    const float kappa = (pv == 1.0f) ? ls : (float)(log((double)pv) + (double)ls);
    keys[i] = ordered_key(kappa);
  }
  __syncthreads();

  uint32_t kth = 0;
  int n_tie = 0;
  if (n_heavy > 0) {
    uint32_t prefix = 0, mask = 0;
    int kr = n_heavy;
    for (int pass = 3; pass >= 0; --pass) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int i = lo + tid; i < hi; i += blockDim.x) {
        const uint32_t k = keys[i];
        if ((k & mask) == prefix) atomicAdd(&hist[(k >> (8 * pass)) & 255u], 1);
      }
      __syncthreads();
      if (tid == 0) {
        int cum = 0, bin = 255;
        for (; bin > 0; --bin) {
          if (cum + hist[bin] >= kr) break;
          cum += hist[bin];
        }
        s_prefix = prefix | ((uint32_t)bin << (8 * pass));
        s_kr = kr - cum;
      }
      __syncthreads();
      prefix = s_prefix;
      kr = s_kr;
      mask |= 0xFFu << (8 * pass);
      __syncthreads();
    }
    kth = prefix;   // the n_heavy-th largest key
    n_tie = kr;     // how many entries equal to it are taken, lowest index first
  }

  int base_tie = 0, base_keep = 0;
  for (int start = 0; start < len; start += blockDim.x) {
    const int i = start + tid;
    const bool valid = i < len;
    const uint32_t k = valid ? keys[i] : 0u;
    const bool in_mid = valid && i >= lo && i < hi;
    const bool is_tie = in_mid && n_heavy > 0 && k == kth;
    int tot_tie, tot_keep;
    const int tie_rank = base_tie + block_excl_count(is_tie, warp_tot, tot_tie);
    const bool keep = valid && (!in_mid || (n_heavy > 0 && (k > kth || (is_tie && tie_rank < n_tie))));
    const int slot = base_keep + block_excl_count(keep, warp_tot, tot_keep);
    if (valid) {
      if (keep) {
        ret_idx[base + slot] = i;
        target[base + i] = -2;
      } else {
        ev_idx[base + (i - slot)] = i;
        target[base + i] = -1;
      }
    }
    base_tie += tot_tie;
    base_keep += tot_keep;
  }
  if (tid == 0) {
    UnitInfo ui{len, base_keep, len - base_keep, budget};
    unit_info[u] = ui;
    if (h == 0) dst_seq_len[b] = base_keep;
    keepkv_stats st;
    st.n_retained = base_keep; st.n_evicted = len - base_keep; st.n_merged = 0; st.n_below_T = 0;
    st.n_guard_groups = 0; st.n_groups = 0; st.max_group = 0; st.reserved = 0;
    stats[u] = st;
  }
}

// ------------------------------------------------------------------ compact
// grid (ceil(bound/32), U), 256 threads: 32 retained rows per CTA.  A warp moves a K row with its
// lower half and the V row with its upper half; afterwards 32 threads run the fp32 norm chain.
template <int D>
__global__ void __launch_bounds__(256)
compact_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *ret_idx, const UnitInfo *unit_info,
               float *dst_norm) {
  constexpr int CH = D / 8;       // 16-byte chunks per row
  constexpr int RS = D + 8;       // padded row stride (bf16 elements) in shared memory
  __shared__ __align__(16) __nv_bfloat16 Ks[32 * RS];
  const int u = blockIdx.y, s0 = blockIdx.x * 32;
  const int n_ret = unit_info[u].n_ret;
  if (s0 >= n_ret) return;
  const size_t base = (size_t)u * p.N_cap;
  const uint4 *sK = reinterpret_cast<const uint4 *>(src.K), *sV = reinterpret_cast<const uint4 *>(src.V);
  uint4 *dK = reinterpret_cast<uint4 *>(dst.K), *dV = reinterpret_cast<uint4 *>(dst.V);
  for (int idx = threadIdx.x; idx < 32 * CH * 2; idx += blockDim.x) {
    const int r = idx / (2 * CH), rem = idx % (2 * CH), isv = rem / CH, j = rem % CH;
    const int slot = s0 + r;
    if (slot >= n_ret) continue;
    const int si = ret_idx[base + slot];
    if (isv) {
      dV[(base + slot) * CH + j] = sV[(base + si) * CH + j];
    } else {
      const uint4 v = sK[(base + si) * CH + j];
      dK[(base + slot) * CH + j] = v;
      *reinterpret_cast<uint4 *>(&Ks[r * RS + j * 8]) = v;
    }
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    const int slot = s0 + threadIdx.x;
    if (slot < n_ret) {
      const int si = ret_idx[base + slot];
      float acc = 0.f;
      for (int j = 0; j < D; ++j) {
        const float x = __bfloat162float(Ks[threadIdx.x * RS + j]);
        acc = fmaf(x, x, acc);
      }
      dst_norm[base + slot] = sqrtf(acc);
      dst.votes[base + slot] = src.votes[base + si];
      dst.lscore[base + slot] = src.lscore[base + si];
    }
  }
}

// ------------------------------------------------------------------ match (exact fp32 chain)
// grid (ceil(N_cap/64), U), 256 threads as 16x16; each thread owns a 4x4 block of the
// 64 evicted x 64 retained cosine tile.  Every dot product is accumulated by fused multiply-add
// from 0 over channels 0..D-1 in order, which is the arithmetic the interface fixes for the
// cosine, so the arg-max taken here is final.
template <int D>
__global__ void __launch_bounds__(256)
match_exact_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *ev_idx,
                   const UnitInfo *unit_info, const float *dst_norm, int32_t *target, float *umax,
                   keepkv_stats *stats) {
  constexpr int LD = 68;
  extern __shared__ float smf[];
  float *As = smf;                 // [D][LD]  evicted keys, channel-major
  float *Bs = smf + D * LD;        // [D][LD]  retained keys, channel-major
  __shared__ float na[64], nb[64];
  __shared__ float red_v[64][17];
  __shared__ int red_i[64][17];
  __shared__ int s_below;
  const int u = blockIdx.y, r0 = blockIdx.x * 64;
  const UnitInfo ui = unit_info[u];
  if (r0 >= ui.n_ev) return;
  const size_t base = (size_t)u * p.N_cap;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const __nv_bfloat16 *sK = reinterpret_cast<const __nv_bfloat16 *>(src.K) + base * D;
  const __nv_bfloat16 *dK = reinterpret_cast<const __nv_bfloat16 *>(dst.K) + base * D;
  if (tid == 0) s_below = 0;
  for (int idx = tid; idx < 64 * (D / 2); idx += 256) {
    const int r = idx / (D / 2), jj = idx % (D / 2);
    uint32_t v = 0;
    if (r0 + r < ui.n_ev) v = *reinterpret_cast<const uint32_t *>(sK + (size_t)ev_idx[base + r0 + r] * D + 2 * jj);
    As[(2 * jj) * LD + r] = bf16_lo(v);
    As[(2 * jj + 1) * LD + r] = bf16_hi(v);
  }
  __syncthreads();
  if (tid < 64) {
    float acc = 0.f;
    for (int j = 0; j < D; ++j) acc = fmaf(As[j * LD + tid], As[j * LD + tid], acc);
    na[tid] = sqrtf(acc);
  }
  float best[4];
  int bi[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { best[r] = -CUDART_INF_F; bi[r] = -1; }

  for (int c0 = 0; c0 < ui.n_ret; c0 += 64) {
    __syncthreads();
    for (int idx = tid; idx < 64 * (D / 2); idx += 256) {
      const int c = idx / (D / 2), jj = idx % (D / 2);
      uint32_t v = 0;
      if (c0 + c < ui.n_ret) v = *reinterpret_cast<const uint32_t *>(dK + (size_t)(c0 + c) * D + 2 * jj);
      Bs[(2 * jj) * LD + c] = bf16_lo(v);
      Bs[(2 * jj + 1) * LD + c] = bf16_hi(v);
    }
    if (tid < 64) nb[tid] = (c0 + tid < ui.n_ret) ? dst_norm[base + c0 + tid] : 1.f;
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[r][c] = 0.f;
#pragma unroll 4
    for (int j = 0; j < D; ++j) {
      const float4 a = *reinterpret_cast<const float4 *>(&As[j * LD + ty * 4]);
      const float4 bb = *reinterpret_cast<const float4 *>(&Bs[j * LD + tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = c0 + tx * 4 + c;
        if (col < ui.n_ret) {
          const float uu = acc[r][c] / (na[ty * 4 + r] * nb[tx * 4 + c]);
          if (uu > best[r]) { best[r] = uu; bi[r] = col; }
        }
      }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) { red_v[ty * 4 + r][tx] = best[r]; red_i[ty * 4 + r][tx] = bi[r]; }
  __syncthreads();
  if (tid < 64 && r0 + tid < ui.n_ev) {
    float bv = -CUDART_INF_F;
    int bx = -1;
    for (int t = 0; t < 16; ++t) {
      const float v = red_v[tid][t];
      const int ix = red_i[tid][t];
      if (ix >= 0 && (v > bv || (v == bv && ix < bx) || bx < 0)) { bv = v; bx = ix; }
    }
    const int e = ev_idx[base + r0 + tid];
    const bool merge = bx >= 0 && bv > p.merge_threshold;
    target[base + e] = merge ? bx : -1;
    umax[base + e] = bv;
    if (!merge) atomicAdd(&s_below, 1);
  }
  __syncthreads();
  if (tid == 0 && s_below) atomicAdd(&stats[u].n_below_T, s_below);
}

// ------------------------------------------------------------------ group
// One CTA per unit: count members per slot, scan, then one warp fills the CSR lists walking the
// evicted entries in ascending order, so that every member list is ascending and the result
// does not depend on scheduling.
__global__ void __launch_bounds__(256)
group_kernel(keepkv_params p, const int32_t *ev_idx, const int32_t *target, const UnitInfo *unit_info,
             int32_t *grp_ptr, int32_t *grp_fill, int32_t *grp_mem) {
  __shared__ int warp_tot[32];
  const int u = blockIdx.x, tid = threadIdx.x;
  const UnitInfo ui = unit_info[u];
  const size_t base = (size_t)u * p.N_cap;
  int32_t *ptr = grp_ptr + (size_t)u * (p.N_cap + 1);
  volatile int32_t *fill = grp_fill + base;
  int32_t *mem = grp_mem + base;
  for (int c = tid; c <= ui.n_ret; c += blockDim.x) ptr[c] = 0;
  __syncthreads();
  for (int j = tid; j < ui.n_ev; j += blockDim.x) {
    const int c = target[base + ev_idx[base + j]];
    if (c >= 0) atomicAdd(&ptr[c], 1);
  }
  __syncthreads();
  int run = 0;
  for (int start = 0; start < ui.n_ret; start += blockDim.x) {
    const int c = start + tid;
    const int v = c < ui.n_ret ? ptr[c] : 0;
    int tot;
    const int ex = run + block_excl_sum(v, warp_tot, tot);
    if (c < ui.n_ret) { ptr[c] = ex; fill[c] = ex; }
    run += tot;
  }
  if (tid == 0) ptr[ui.n_ret] = run;
  __syncthreads();
  if (tid < 32) {
    const int lane = tid;
    for (int j0 = 0; j0 < ui.n_ev; j0 += 32) {
      const int j = j0 + lane;
      int e = -1, c = -1;
      if (j < ui.n_ev) { e = ev_idx[base + j]; c = target[base + e]; }
      const int keyc = c >= 0 ? c : -1 - lane;  // inactive lanes match nobody
      const unsigned grp = __match_any_sync(0xffffffffu, keyc);
      if (c >= 0) {
        const int rank = __popc(grp & ((1u << lane) - 1u));
        const int pos = fill[c] + rank;
        mem[pos] = e;
      }
      __syncwarp();
      if (c >= 0 && (grp >> lane) == 1u) fill[c] = fill[c] + __popc(grp);  // highest lane of the group
      __syncwarp();
    }
  }
}

// ------------------------------------------------------------------ merge
// One warp per retained slot that has members.  With a_i = ln p_i + lscore_i over the group
// K'_e (target first, then members ascending):  omega = softmax(a),  v_r = sum omega_i v_i,
// k_r = gamma * sum omega_i k_i,  gamma = L / lambda_bar,  L = LSE(a) - ln(sum p),
// lambda_bar = sum omega_i lscore_i,  p_r = sum p,  lscore_r = L   (Eq. A.3 in logarithms).
template <int D>
__global__ void __launch_bounds__(128)
merge_kernel(keepkv_params p, keepkv_cache src, keepkv_cache dst, const int32_t *ret_idx, int32_t *target,
             const UnitInfo *unit_info, const int32_t *grp_ptr, const int32_t *grp_mem, keepkv_stats *stats) {
  constexpr int EPL = D / 32;
  const int u = blockIdx.y, lane = threadIdx.x & 31;
  const int c = blockIdx.x * 4 + (threadIdx.x >> 5);
  const UnitInfo ui = unit_info[u];
  if (c >= ui.n_ret || ui.n_ev == 0) return;
  const size_t base = (size_t)u * p.N_cap;
  const int32_t *ptr = grp_ptr + (size_t)u * (p.N_cap + 1);
  const int beg = ptr[c], n = ptr[c + 1] - beg;
  if (n == 0) return;
  const int32_t *mem = grp_mem + base + beg;
  const int ci = ret_idx[base + c];
  const float *votes = src.votes + base, *ls = src.lscore + base;

  const float a_c = logf(votes[ci]) + ls[ci];
  float M = a_c;
  for (int t = lane; t < n; t += 32) { const int e = mem[t]; M = fmaxf(M, logf(votes[e]) + ls[e]); }
  M = warp_max(M);
  float Z = 0.f, Ps = 0.f;
  if (lane == 0) { Z = expf(a_c - M); Ps = votes[ci]; }
  for (int t = lane; t < n; t += 32) { const int e = mem[t]; Z += expf(logf(votes[e]) + ls[e] - M); Ps += votes[e]; }
  Z = warp_sum(Z);
  Ps = warp_sum(Ps);
  const float Lam = M + logf(Z);
  const float L = Lam - logf(Ps);

  const __nv_bfloat16 *sK = reinterpret_cast<const __nv_bfloat16 *>(src.K) + base * D;
  const __nv_bfloat16 *sV = reinterpret_cast<const __nv_bfloat16 *>(src.V) + base * D;
  float ka[EPL], va[EPL], lbar = 0.f;
#pragma unroll
  for (int e = 0; e < EPL; ++e) { ka[e] = 0.f; va[e] = 0.f; }
  for (int t = -1; t < n; ++t) {
    const int i = t < 0 ? ci : mem[t];
    const float lsi = ls[i];
    const float om = expf(logf(votes[i]) + lsi - Lam);
    lbar = fmaf(om, lsi, lbar);
    if constexpr (EPL == 4) {
      const uint2 kk = *reinterpret_cast<const uint2 *>(sK + (size_t)i * D + lane * 4);
      const uint2 vv = *reinterpret_cast<const uint2 *>(sV + (size_t)i * D + lane * 4);
      ka[0] = fmaf(om, bf16_lo(kk.x), ka[0]); ka[1] = fmaf(om, bf16_hi(kk.x), ka[1]);
      ka[2] = fmaf(om, bf16_lo(kk.y), ka[2]); ka[3] = fmaf(om, bf16_hi(kk.y), ka[3]);
      va[0] = fmaf(om, bf16_lo(vv.x), va[0]); va[1] = fmaf(om, bf16_hi(vv.x), va[1]);
      va[2] = fmaf(om, bf16_lo(vv.y), va[2]); va[3] = fmaf(om, bf16_hi(vv.y), va[3]);
    } else {
      const uint32_t kk = *reinterpret_cast<const uint32_t *>(sK + (size_t)i * D + lane * 2);
      const uint32_t vv = *reinterpret_cast<const uint32_t *>(sV + (size_t)i * D + lane * 2);
      ka[0] = fmaf(om, bf16_lo(kk), ka[0]); ka[1] = fmaf(om, bf16_hi(kk), ka[1]);
      va[0] = fmaf(om, bf16_lo(vv), va[0]); va[1] = fmaf(om, bf16_hi(vv), va[1]);
    }
  }
  const float gamma = L / lbar;
  const bool ok = gamma > p.gamma_min && gamma <= p.gamma_max && fabsf(lbar) >= 1e-6f;
  if (!ok) {
    // guard: the members are dropped after all and the target keeps the row copied by compaction
    for (int t = lane; t < n; t += 32) target[base + mem[t]] = -1;
    if (lane == 0) { atomicAdd(&stats[u].n_guard_groups, 1); atomicAdd(&stats[u].n_groups, 1); }
    return;
  }
  __nv_bfloat16 *dK = reinterpret_cast<__nv_bfloat16 *>(dst.K) + (base + c) * D;
  __nv_bfloat16 *dV = reinterpret_cast<__nv_bfloat16 *>(dst.V) + (base + c) * D;
  if constexpr (EPL == 4) {
    uint2 ko, vo;
    ko.x = pack_bf16(gamma * ka[0], gamma * ka[1]); ko.y = pack_bf16(gamma * ka[2], gamma * ka[3]);
    vo.x = pack_bf16(va[0], va[1]); vo.y = pack_bf16(va[2], va[3]);
    *reinterpret_cast<uint2 *>(dK + lane * 4) = ko;
    *reinterpret_cast<uint2 *>(dV + lane * 4) = vo;
  } else {
    *reinterpret_cast<uint32_t *>(dK + lane * 2) = pack_bf16(gamma * ka[0], gamma * ka[1]);
    *reinterpret_cast<uint32_t *>(dV + lane * 2) = pack_bf16(va[0], va[1]);
  }
  if (lane == 0) {
    dst.votes[base + c] = Ps;
    dst.lscore[base + c] = L;
    atomicAdd(&stats[u].n_merged, n);
    atomicAdd(&stats[u].n_groups, 1);
    atomicMax(&stats[u].max_group, n);
  }
}

// ------------------------------------------------------------------ host side
template <int D>
static void launch_compress_t(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                              const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                              int32_t *ret_idx, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                              LaunchCtx &ctx) {
  const int U = p.B * p.H_kv;
  UnitInfo *ui = reinterpret_cast<UnitInfo *>(ws + L.unit_info);
  int32_t *ev_idx = reinterpret_cast<int32_t *>(ws + L.ev_idx);
  float *dst_norm = reinterpret_cast<float *>(ws + L.dst_norm);
  float *umax = reinterpret_cast<float *>(ws + L.umax);
  int32_t *grp_ptr = reinterpret_cast<int32_t *>(ws + L.grp_ptr);
  int32_t *grp_fill = reinterpret_cast<int32_t *>(ws + L.grp_fill);
  int32_t *grp_mem = reinterpret_cast<int32_t *>(ws + L.grp_mem);
  const int ret_bound = budget_dev ? p.N_cap : (budget_scalar < p.N_cap ? budget_scalar : p.N_cap);

  const size_t sel_smem = (size_t)p.N_cap * sizeof(uint32_t);
  static bool attr_done_dev[64] = {};   // opt-in to large dynamic shared memory once per device
  int dev = 0;
  cudaGetDevice(&dev);
  bool &attr_done = attr_done_dev[dev & 63];
  if (!attr_done) {
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 49152 * 4);
    cudaFuncSetAttribute(match_exact_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 64 * 68 * 4);
    cudaFuncSetAttribute(match_exact_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 128 * 68 * 4);
    attr_done = true;
  }
  select_kernel<<<U, 1024, sel_smem, ctx.stream>>>(p, src, dst.seq_len, budget_dev, budget_scalar, n_recent_dev,
                                                   ret_idx, target, ev_idx, ui, stats);
  KEEPKV_CHECK_LAUNCH(ctx);
  if (ret_bound > 0) {
    compact_kernel<D><<<dim3((ret_bound + 31) / 32, U), 256, 0, ctx.stream>>>(p, src, dst, ret_idx, ui, dst_norm);
    KEEPKV_CHECK_LAUNCH(ctx);
  }
  match_exact_kernel<D><<<dim3(p.N_cap / 64, U), 256, 2 * D * 68 * 4, ctx.stream>>>(p, src, dst, ev_idx, ui, dst_norm,
                                                                                    target, umax, stats);
  KEEPKV_CHECK_LAUNCH(ctx);
  if (ret_bound > 0) {
    group_kernel<<<U, 256, 0, ctx.stream>>>(p, ev_idx, target, ui, grp_ptr, grp_fill, grp_mem);
    KEEPKV_CHECK_LAUNCH(ctx);
    merge_kernel<D><<<dim3((ret_bound + 3) / 4, U), 128, 0, ctx.stream>>>(p, src, dst, ret_idx, target, ui, grp_ptr,
                                                                          grp_mem, stats);
    KEEPKV_CHECK_LAUNCH(ctx);
  }
}

void launch_compress(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                     const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev, int32_t *ret_idx,
                     int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L, int32_t *status_dev,
                     LaunchCtx &ctx) {
  (void)status_dev;
  if (p.d == 128)
    launch_compress_t<128>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L, ctx);
  else
    launch_compress_t<64>(p, src, dst, budget_dev, budget_scalar, n_recent_dev, ret_idx, target, stats, ws, L, ctx);
}

}  // namespace keepkv
