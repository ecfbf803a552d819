// Device helpers shared by the kernels of keepkv_compress (compress.cu: the general pipeline;
// compress_steady.cu: the single-kernel path of a steady-state compression).
#pragma once
#include "common.cuh"

namespace keepkv {

constexpr float kRankEps = 1e-4f;   // tensor-core cosines closer than this are re-evaluated in the interface's fp32 chain

// ------------------------------------------------------------------ block scans
// Exclusive prefix count of `flag` over the first nw warps of the block in thread order (the other
// warps have left the kernel); total returned through `total`.
__device__ __forceinline__ int block_excl_count(bool flag, int *warp_tot, int &total, int nw) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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
__device__ __forceinline__ int block_excl_count(bool flag, int *warp_tot, int &total) {
  return block_excl_count(flag, warp_tot, total, (int)(blockDim.x >> 5));
}

// Exclusive prefix sum of small non-negative ints over the block (thread order).
__device__ __forceinline__ int block_excl_sum(int v, int *warp_tot, int &total, int nw) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
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

// ------------------------------------------------------------------ selection key
// Order-preserving map of an fp32 value to u32 (-0 folded onto +0 so equal floats give equal keys).
__device__ __forceinline__ uint32_t ordered_key(float x) {
  x += 0.0f;
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
// kappa = ln p + lscore in fp64, rounded once to fp32 (p = 1 needs no logarithm)
__device__ __forceinline__ uint32_t kappa_key(float pv, float ls) {
  const float kappa = (pv == 1.0f) ? ls : (float)(log((double)pv) + (double)ls);
  return ordered_key(kappa);
}

// One warp finds the kr-th largest of keys[lo..hi) by four 8-bit digit passes (hist: 256 ints of shared
// memory owned by the warp).  Returns, in every lane: kth = that key, n_tie = how many entries equal to it
// belong to the kr largest (lowest index first), tot_ties = how many entries equal to it exist.
__device__ __forceinline__ void warp_radix_select(const uint32_t *keys, int lo, int hi, int kr, int *hist, uint32_t &kth,
                                                  int &n_tie, int &tot_ties) {
  const int lane = threadIdx.x & 31;
  uint32_t prefix = 0, mask = 0;
  int cnt_last = 0;
  for (int pass = 3; pass >= 0; --pass) {
#pragma unroll
    for (int j = 0; j < 8; ++j) hist[8 * lane + j] = 0;
    __syncwarp();
    for (int i = lo + lane; i < hi; i += 32) {
      const uint32_t k = keys[i];
      if ((k & mask) == prefix) atomicAdd(&hist[(k >> (8 * pass)) & 255u], 1);
    }
    __syncwarp();
    int c[8], sum = 0;   // bins are scanned from the top: lane l owns bins 8l..8l+7
#pragma unroll
    for (int j = 0; j < 8; ++j) { c[j] = hist[8 * lane + j]; sum += c[j]; }
    int x = sum;   // becomes the count in bins of lanes >= lane
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_down_sync(0xffffffffu, x, o);
      if (lane + o < 32) x += y;
    }
    const int above = x - sum;
    const bool here = above < kr && x >= kr;
    int cum = above, bin = 0, cnt = 0;
    bool found = false;
#pragma unroll
    for (int j = 7; j >= 0; --j) {
      if (!found) {
        if (cum + c[j] >= kr) { bin = j; cnt = c[j]; found = true; }
        else cum += c[j];
      }
    }
    const int src_lane = __ffs(__ballot_sync(0xffffffffu, here)) - 1;
    prefix |= (uint32_t)__shfl_sync(0xffffffffu, 8 * lane + bin, src_lane) << (8 * pass);
    kr = __shfl_sync(0xffffffffu, kr - cum, src_lane);
    cnt_last = __shfl_sync(0xffffffffu, cnt, src_lane);
    mask |= 0xFFu << (8 * pass);
    __syncwarp();
  }
  kth = prefix;
  n_tie = kr;
  tot_ties = cnt_last;
}

// The same search by a whole block of 256 threads (one histogram bin per thread); three barriers per digit.
// sh: three words of shared memory.  Results in every thread.
__device__ __forceinline__ void block_radix_select(const uint32_t *keys, int n, int kr, int *hist, uint32_t *sh,
                                                   uint32_t &kth, int &n_tie, int &tot_ties) {
  const int tid = threadIdx.x, lane = tid & 31;
  uint32_t prefix = 0, mask = 0;
  for (int pass = 3; pass >= 0; --pass) {
    hist[tid] = 0;
    __syncthreads();
    for (int start = 0; start < n; start += 256) {
      const int i = start + tid;
      const uint32_t k = i < n ? keys[i] : 0u;
      const bool in = i < n && (k & mask) == prefix;
      // one shared-memory atomic per distinct bin among the warp's keys that are still in the race (the leading
      // bytes of most keys coincide; in the later passes few keys are left)
      const unsigned racing = __ballot_sync(0xffffffffu, in);
      if (in) {
        const int bin = (int)((k >> (8 * pass)) & 255u);
        const unsigned peers = __match_any_sync(racing, bin);
        if (lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
      }
    }
    __syncthreads();
    if (tid < 32) {
      int c[8], sum = 0;   // bins are scanned from the top: lane l owns bins 8l..8l+7
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
        sh[0] = prefix | ((uint32_t)(8 * lane + bin) << (8 * pass));
        sh[1] = (uint32_t)(kr - cum);
        sh[2] = (uint32_t)cnt;
      }
    }
    __syncthreads();   // sh is not written again before the second barrier of the next pass
    prefix = sh[0];
    kr = (int)sh[1];
    mask |= 0xFFu << (8 * pass);
  }
  kth = prefix;
  n_tie = kr;
  tot_ties = (int)sh[2];
}

// ------------------------------------------------------------------ tensor-core ranking: top two of a row
// Running top two of one row.  Only values within `thr` of the running best are looked at: the
// final best can only be larger, so every value within thr of the FINAL best has been inserted, and
// (best, second) are exact among those -- which is all the caller's closeness tests use.
// A warp holds 32 rows, and the drain is bound by the ALU pipe (compares and selects), so a group of
// four columns is either skipped by the whole warp -- four fused multiply-adds give v - cut and the
// sign bits are AND-ed -- or updated by the whole warp with selects only (no divergent branch).
struct Top2 {
  float best, second, cut, thr;
  int bi, si;
  __device__ __forceinline__ void init(float thr_) {
    best = second = cut = -CUDART_INF_F;
    thr = thr_;
    bi = si = -1;
  }
  // Comparisons are strict, so among equal values the one seen first (the lower slot) stays in
  // front, and a NaN (a zero-norm key) is never taken.
  __device__ __forceinline__ void insert(float v, int idx) {
    const bool p1 = v > best, p2 = v > second;
    second = p1 ? best : fmaxf(second, v);
    si = p1 ? bi : (p2 ? idx : si);
    bi = p1 ? idx : bi;
    best = fmaxf(best, v);
  }
  // Insert for candidates that arrive out of slot order (the other tracker of the thread): equal values
  // go to the lower slot, as if the columns had been scanned in order.
  __device__ __forceinline__ void insert_any(float v, int idx) {
    const bool p1 = v > best || (v == best && idx < bi), p2 = v > second || (v == second && idx < si);
    second = p1 ? best : (p2 ? v : second);
    si = p1 ? bi : (p2 ? idx : si);
    bi = p1 ? idx : bi;
    best = p1 ? v : best;
  }
};

// Two trackers per thread, one for the even and one for the odd columns, so that the select chains of
// neighbouring columns do not wait on each other.  Both share one cut (kept in ta.cut), taken from the larger of
// their two bests: the row's final best is at least that, so a value below the cut cannot be within thr of it,
// whichever list it would have gone to; what the two lists hold together still contains the row's two largest
// values within thr of its best.  (A cut from the smaller best lets through everything between the two bests,
// and with 32 rows per warp the warp-wide skip then hardly ever fires.)
// a_i: accumulators, w_i: inverse norms of the four columns idx..idx+3.
// TEST = false (the first tile of an item, where nearly every group holds a new candidate for some row):
// all four columns are inserted without the skip test, so nothing but the select chains is on the
// critical path.
template <bool TEST>
__device__ __forceinline__ void offer4(Top2 &ta, Top2 &tb, float a0, float a1, float a2, float a3, const float4 w,
                                       int idx) {
  if (TEST) {
    const float ncut = -ta.cut;
    const uint32_t s = __float_as_uint(fmaf(a0, w.x, ncut)) & __float_as_uint(fmaf(a1, w.y, ncut)) &
                       __float_as_uint(fmaf(a2, w.z, ncut)) & __float_as_uint(fmaf(a3, w.w, ncut));
    if (!__any_sync(0xffffffffu, (int)s >= 0)) return;   // no lane has a value that is not below its cut
  }
  ta.insert(a0 * w.x, idx); tb.insert(a1 * w.y, idx + 1); ta.insert(a2 * w.z, idx + 2); tb.insert(a3 * w.w, idx + 3);
  if (TEST) ta.cut = fmaxf(ta.best, tb.best) - ta.thr;
}

// ------------------------------------------------------------------ the interface's cosine
// One warp evaluates cos(k_e, k_a) and cos(k_e, k_b) in the fixed fp32 arithmetic of the interface:
// dot and squared norms by fused multiply-add from 0 over channels 0..D-1, then dot/(sqrtf(n_e)*sqrtf(n_c)).
// ke_s [D] and kc_s [2][D] are the warp's staging rows in shared memory.  Results in every lane.
template <int D>
__device__ __forceinline__ void exact_cosines(const __nv_bfloat16 *ke, const __nv_bfloat16 *ka, const __nv_bfloat16 *kb,
                                              float *ke_s, float *kc_s, float &ua, float &ub) {
  const int lane = threadIdx.x & 31;
  __syncwarp();
  for (int c = lane; c < D; c += 32) {
    ke_s[c] = __bfloat162float(ke[c]);
    kc_s[c] = __bfloat162float(ka[c]);
    kc_s[D + c] = __bfloat162float(kb[c]);
  }
  __syncwarp();
  // lanes 0 and 1: dot and |k_c|^2 of one candidate each; lane 2: |k_e|^2
  const float *x = ke_s, *y = lane == 2 ? ke_s : kc_s + (lane & 1) * D;
  float dot = 0.f, nn = 0.f;
  if (lane < 3)
    for (int c = 0; c < D; ++c) { dot = fmaf(x[c], y[c], dot); nn = fmaf(y[c], y[c], nn); }
  const float ne = __shfl_sync(0xffffffffu, nn, 2);
  const float uu = dot / (sqrtf(ne) * sqrtf(nn));
  ua = __shfl_sync(0xffffffffu, uu, 0);
  ub = __shfl_sync(0xffffffffu, uu, 1);
}

// ------------------------------------------------------------------ merge
// One warp per group.  With a_i = ln p_i + lscore_i over the group K'_e (target first, then members
// ascending):  omega = softmax(a),  v_r = sum omega_i v_i,  k_r = gamma * sum omega_i k_i,
// gamma = L / lambda_bar,  L = LSE(a) - ln(sum p),  lambda_bar = sum omega_i lscore_i,  p_r = sum p,
// lscore_r = L   (Eq. A.3 in logarithms).  c: the target's slot in dst, ci: its source index,
// member(t): source index of the t-th member (ascending), target_u: the unit's per-entry targets.
template <int D, typename MemberFn>
__device__ __forceinline__ void merge_group(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                                            int c, int ci, MemberFn member, int n, int32_t *target_u, size_t base,
                                            keepkv_stats *st) {
  constexpr int EPL = D / 32;
  const int lane = threadIdx.x & 31;
  const float *votes = src.votes + base, *ls = src.lscore + base;
  const __nv_bfloat16 *sK = reinterpret_cast<const __nv_bfloat16 *>(src.K) + base * D;
  const __nv_bfloat16 *sV = reinterpret_cast<const __nv_bfloat16 *>(src.V) + base * D;

  // The group's scalars are evaluated in fp64: L = LSE(a) - ln(sum p) and lambda_bar cancel to almost nothing
  // when the members' log-scores sit near zero, and gamma = L / lambda_bar then carries whatever relative error
  // they have into every channel of the merged key (an fp32 L of 1e-5 is off by a percent).  A handful of
  // double-precision logarithms per group cost nothing next to the rows it loads; the row sums stay fp32.
  float ka[EPL], va[EPL];
  double lbar = 0.0, L, Ps;
#pragma unroll
  for (int e = 0; e < EPL; ++e) { ka[e] = 0.f; va[e] = 0.f; }
  auto accumulate = [&](int i, float om) {
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
  };
  auto wsum_d = [](double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
  };
  auto wmax_d = [](double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
  };
  const double NEG_INF = -CUDART_INF;
  if (n < 32) {
    // the usual case: lane 0 holds the target, lane t the t-th member, so that their votes and scores are
    // fetched together and the row loads of the accumulation do not wait on one another
    const int idx = lane == 0 ? ci : (lane <= n ? member(lane - 1) : -1);
    const float pv = idx >= 0 ? votes[idx] : 0.f, lsv = idx >= 0 ? ls[idx] : 0.f;
    // fp32 first: with |L| and |lambda_bar| away from zero its error (about 1e-6 absolute) is far below bf16
    // resolution in gamma; only a group near the cancellation is evaluated again in fp64 (a warp-uniform choice)
    float om;
    {
      const float a = idx >= 0 ? logf(pv) + lsv : -CUDART_INF_F;
      const float M = warp_max(a);
      const float Z = warp_sum(idx >= 0 ? expf(a - M) : 0.f);
      const float Psf = warp_sum(pv);
      const float Lam = M + logf(Z);
      const float Lf = Lam - logf(Psf);
      om = idx >= 0 ? expf(a - Lam) : 0.f;
      const float lbf = warp_sum(om * lsv);
      Ps = (double)Psf; L = (double)Lf; lbar = (double)lbf;
    }
    if (!(fabs(L) >= 0.25 && fabs(lbar) >= 0.25)) {
      const double a = idx >= 0 ? log((double)pv) + (double)lsv : NEG_INF;
      const double M = wmax_d(a);
      const double Z = wsum_d(idx >= 0 ? exp(a - M) : 0.0);
      Ps = wsum_d((double)pv);
      const double Lam = M + log(Z);
      L = Lam - log(Ps);
      const double omd = idx >= 0 ? exp(a - Lam) : 0.0;
      lbar = wsum_d(omd * (double)lsv);
      om = (float)omd;
    }
#pragma unroll 4
    for (int t = 0; t <= n; ++t) accumulate(__shfl_sync(0xffffffffu, idx, t), __shfl_sync(0xffffffffu, om, t));
  } else {
    const double a_c = log((double)votes[ci]) + (double)ls[ci];
    double M = a_c;
    for (int t = lane; t < n; t += 32) { const int e = member(t); M = fmax(M, log((double)votes[e]) + (double)ls[e]); }
    M = wmax_d(M);
    double Z = 0.0;
    Ps = 0.0;
    if (lane == 0) { Z = exp(a_c - M); Ps = (double)votes[ci]; }
    for (int t = lane; t < n; t += 32) {
      const int e = member(t);
      Z += exp(log((double)votes[e]) + (double)ls[e] - M);
      Ps += (double)votes[e];
    }
    Z = wsum_d(Z);
    Ps = wsum_d(Ps);
    const double Lam = M + log(Z);
    L = Lam - log(Ps);
    // every lane walks all members (the rows are spread over the lanes by channel), so lambda_bar is summed per lane
    for (int t = -1; t < n; ++t) {
      const int i = t < 0 ? ci : member(t);
      const double lsi = (double)ls[i];
      const double omd = exp(log((double)votes[i]) + lsi - Lam);
      lbar += omd * lsi;
      accumulate(i, (float)omd);
    }
  }
  const double gamma_d = L / lbar;
  const float gamma = (float)gamma_d;
  const bool ok = gamma_d > (double)p.gamma_min && gamma_d <= (double)p.gamma_max && fabs(lbar) >= 1e-6;
  if (!ok) {
    // guard: the members are dropped after all and the target keeps the row copied by compaction
    for (int t = lane; t < n; t += 32) target_u[member(t)] = -1;
    if (lane == 0) { atomicAdd(&st->n_guard_groups, 1); atomicAdd(&st->n_groups, 1); }
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
    dst.votes[base + c] = (float)Ps;
    dst.lscore[base + c] = (float)L;
    atomicAdd(&st->n_merged, n);
    atomicAdd(&st->n_groups, 1);
    atomicMax(&st->max_group, n);
  }
}

// the single-kernel path of a steady-state compression (compress_steady.cu)
void launch_compress_steady(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                            const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                            int32_t *ret_idx, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                            int32_t *status_dev, const float *select_key, LaunchCtx &ctx);

}  // namespace keepkv
