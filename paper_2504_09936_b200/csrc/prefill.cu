// keepkv_prefill_scores: the score estimate every entry starts decoding with (Eq. 8, first case): a
// bias-corrected exponentially weighted mean of the entry's scores under the last W prompt queries.
//
// Per (sequence, kv-head) unit this is a (len x d) . (d x G*W) contraction followed by a weighted
// log-sum-exp along the G*W query columns, bound by the one pass over the keys.  The keys are the A
// operand of a tcgen05.mma (128 entries = 128 tensor-memory lanes per tile), the unit's G*W window
// queries the B operand (head g, query k in column g*32 + k), so every drain thread owns one entry and
// reduces its columns in registers, without shuffles.  One persistent CTA per SM walks a contiguous
// range of the global list of 128-entry tiles:
//   warp 0     TMA producer: the unit's window queries (one box of W rows per head) when the unit
//              changes, key tiles into a 3-stage ring;
//   warp 1     one thread issues the MMAs into one of two accumulators and commits to the barriers;
//   warps 2-17 drain (four warps per 32 entries, heads g = w, w + 4 of the group for the w-th of them, combined
//              through shared memory): per entry a running max / sum of 2^(x + log2 weight - max) over the
//              visible queries (a prompt is causal: query k, at position len - W + k, scores only entries
//              at or before it), then lscore = ln(sum / sum of the visible weights / G).  The logarithms
//              of the window weights are kernel parameters, i.e. constant-bank operands of the multiply-add
//              that scales the logit, so they cost neither registers nor instructions.
// Every wait is bounded; one that runs out raises KEEPKV_DEV_TIMEOUT and the CTA winds down.
#include "common.cuh"
#include "ptx.cuh"

namespace keepkv {

constexpr int kPfM = 128;        // entries per tile
constexpr int kPfDrainWarps = 16; // four per 32-lane quarter of tensor memory
constexpr int kPfThreads = 32 * (2 + kPfDrainWarps);   // producer, MMA issuer, drain warps
constexpr int kPfWmax = 32;      // window queries per head (columns reserved per head)
constexpr float kPfLog2e = 1.4426950408889634f;
constexpr float kPfLn2 = 0.6931471805599453f;

template <int D, int G>
struct PfSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kNB = G * kPfWmax;                   // columns of the accumulator
  // Producer, MMA issuer and drain hand a tile over in about a microsecond whatever its size, so up to G = 4 (where
  // four accumulators fit the 512 columns of tensor memory) a hand-over is a pair of 128-entry tiles.
  static constexpr int kTP = G <= 4 ? 2 : 1;                // 128-entry tiles per hand-over
  static constexpr int kRows = kPfM * kTP;                  // entries per hand-over
  static constexpr int kStages = kTP == 2 ? 2 : 3;          // key ring
  static constexpr int kABytes = kSub * kRows * 128;
  static constexpr int kBBytes = kSub * kNB * 128;
  static constexpr int kA = 0;
  static constexpr int kB = kStages * kABytes;
  static constexpr int kWt = kB + kBBytes;                  // f32 [32] weights, f32 [33] their suffix sums (as ln)
  static constexpr int kXchg = kWt + 512;                   // float2 [3 hand-overs in flight][kRows entries][4 warps]: (max, sum)
  static constexpr int kBytes = kXchg + 3 * kRows * 4 * 8;
};

// Position in the global tile list: sequence, kv head, tile of the unit; next() moves to the next tile.
__device__ __forceinline__ float pf_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// log2 of the window weights alpha^(W-1-k), -inf for k >= W (and, with alpha = 0, for all but the last query)
// w: the weights themselves and whether the drain may use them as multipliers (every one of the 32 a normal fp32
// number: a full window and an alpha that is not tiny)
struct PfLogWeights { float c[kPfWmax]; float w[kPfWmax]; int mult; };

struct PfWalker {
  int b, h, tile, len, tb, rows;   // rows: entries per tile of the list (a hand-over)
  __device__ __forceinline__ void load(const keepkv_params &p, const int32_t *seq_len) {
    len = max(0, min(seq_len[b], p.N_cap));
    tb = (len + rows - 1) / rows;
  }
  __device__ __forceinline__ void next(const keepkv_params &p, const int32_t *seq_len, bool more) {
    if (++tile == tb && more) {
      tile = 0;
      if (++h == p.H_kv) {
        h = 0;
        do { ++b; load(p, seq_len); } while (tb == 0);
      }
    }
  }
};

template <int D, int G>
__global__ void __launch_bounds__(kPfThreads, 1)
prefill_scores_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapQ,
                      keepkv_params p, keepkv_cache c, int W, const PfLogWeights lw, int32_t *status_dev) {
  using SL = PfSmem<D, G>;
  constexpr int KSTEPS = D / 16, NB = SL::kNB, TP = SL::kTP, ROWS = SL::kRows, kPfStages = SL::kStages;
  constexpr uint32_t IDESC = umma_idesc_bf16(kPfM, NB);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[2 * 3 + 7];   // a_full[S], a_empty[S], b_full, b_empty, t_full[2], t_empty[2], drain
  __shared__ uint32_t s_tmem;
  __shared__ int s_scan[kPfThreads / 32];
  __shared__ int s_start[4];
  __shared__ volatile int s_abort;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar_a_full = smem_u32(&bars[0]), bar_a_empty = smem_u32(&bars[kPfStages]);
  const uint32_t bar_b_full = smem_u32(&bars[2 * kPfStages]), bar_b_empty = smem_u32(&bars[2 * kPfStages + 1]);
  const uint32_t bar_t_full = smem_u32(&bars[2 * kPfStages + 2]), bar_t_empty = smem_u32(&bars[2 * kPfStages + 4]);
  const uint32_t bar_drain = smem_u32(&bars[2 * kPfStages + 6]);
  float *wt = reinterpret_cast<float *>(smem + SL::kWt);   // wt[k], k < 32
  float *lnwsuf = wt + 32;                                  // ln sum_{k' >= k} wt[k'], k <= 32

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, grid = gridDim.x;

  if (tid == 0) {
    for (int i = 0; i < kPfStages; ++i) { mbar_init(bar_a_full + 8 * i, 1); mbar_init(bar_a_empty + 8 * i, 1); }
    mbar_init(bar_b_full, 1);
    mbar_init(bar_b_empty, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(bar_t_full + 8 * i, 1); mbar_init(bar_t_empty + 8 * i, kPfDrainWarps); }
    mbar_init(bar_drain, 1);
    s_abort = 0;
    s_start[0] = p.B;
    mbar_fence_init();
    prefetch_tensormap(&mapK);
    prefetch_tensormap(&mapQ);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&s_tmem), 512);
    tmem_relinquish();
  }
  // rows of the query tile that no copy writes (k >= W) must hold finite numbers: zero the tile once
  for (int i = tid; i < SL::kBBytes / 16; i += kPfThreads)
    *reinterpret_cast<uint4 *>(smem + SL::kB + i * 16) = make_uint4(0, 0, 0, 0);
  if (tid < 32) {
    // weights alpha^(W-1-k) of the window's queries (alpha = 0: the last query only) and the logarithms of
    // their suffix sums (the weight an entry first seen by query k has accumulated)
    const float wk = tid < W ? (p.ema_alpha > 0.f ? expf((float)(W - 1 - tid) * logf(p.ema_alpha)) : (tid == W - 1 ? 1.f : 0.f))
                             : 0.f;
    wt[tid] = wk;
    float suf = wk;   // inclusive suffix sum over lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float y = __shfl_down_sync(0xffffffffu, suf, o);
      if (lane + o < 32) suf += y;
    }
    lnwsuf[tid] = logf(suf);
    if (tid == 0) lnwsuf[32] = -CUDART_INF_F;
  }
  fence_proxy_async_smem();
  pdl_wait();
  pdl_trigger();

  // ---- the tile list: every thread sums a block of consecutive sequences, a block scan gives the offsets
  auto tiles_of = [&](int b) { return (max(0, min(c.seq_len[b], p.N_cap)) + ROWS - 1) / ROWS; };
  const int per = (p.B + kPfThreads - 1) / kPfThreads;
  const int b_lo = min(p.B, tid * per), b_hi = min(p.B, b_lo + per);
  int mine = 0;
  for (int b = b_lo; b < b_hi; ++b) mine += tiles_of(b);
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_scan[warp] = incl;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  int before = incl - mine, total_b = 0;
  for (int w = 0; w < kPfThreads / 32; ++w) {
    if (w < warp) before += s_scan[w];
    total_b += s_scan[w];
  }
  const long long T = (long long)total_b * p.H_kv;
  const int chunk = (int)((T + grid - 1) / grid);
  const long long g0 = min(T, (long long)cta * chunk), g1 = min(T, g0 + chunk);
  const int ntiles = (int)(g1 - g0);
  if (ntiles > 0 && (long long)before * p.H_kv <= g0 && g0 < (long long)(before + mine) * p.H_kv) {
    long long at = (long long)before * p.H_kv;
    for (int b = b_lo; b < b_hi; ++b) {
      const int tb = tiles_of(b);
      const long long span = (long long)tb * p.H_kv;
      if (g0 < at + span) {
        const int r = (int)(g0 - at);
        s_start[0] = b; s_start[1] = r / tb; s_start[2] = r % tb;
        break;
      }
      at += span;
    }
  }
  __syncthreads();
  const uint32_t tmem = s_tmem;
  PfWalker wk;
  wk.b = s_start[0]; wk.h = s_start[1]; wk.tile = s_start[2]; wk.len = 0; wk.tb = 1; wk.rows = ROWS;
  if (ntiles > 0) wk.load(p, c.seq_len);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int n_units = 0;
      for (int it = 0; it < ntiles && !s_abort; ++it) {
        const int u = wk.b * p.H_kv + wk.h;
        if (it == 0 || wk.tile == 0) {   // the unit's window queries: W rows per head into columns g*32 ..
          if (n_units > 0 && !mbar_wait(bar_b_empty, (n_units - 1) & 1)) { s_abort = 1; break; }
          ++n_units;
          mbar_expect_tx(bar_b_full, (uint32_t)(G * SL::kSub * W * 128));
#pragma unroll
          for (int g = 0; g < G; ++g)
#pragma unroll
            for (int sub = 0; sub < SL::kSub; ++sub)
              tma_load_2d(sbase + SL::kB + sub * (NB * 128) + g * kPfWmax * 128, &mapQ, sub * 64,
                          (wk.b * p.H_q + wk.h * G + g) * W, bar_b_full);
        }
        const int s = it % kPfStages;
        if (!mbar_wait(bar_a_empty + 8 * s, ((it / kPfStages) & 1) ^ 1)) { s_abort = 1; break; }
        mbar_expect_tx(bar_a_full + 8 * s, SL::kABytes);
#pragma unroll
        for (int sub = 0; sub < SL::kSub; ++sub)
          tma_load_2d(sbase + SL::kA + s * SL::kABytes + sub * (ROWS * 128), &mapK, sub * 64,
                      u * p.N_cap + wk.tile * ROWS, bar_a_full + 8 * s);
        wk.next(p, c.seq_len, it + 1 < ntiles);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int n_units = 0;
      for (int it = 0; it < ntiles && !s_abort; ++it) {
        if (it == 0 || wk.tile == 0) {
          if (!mbar_wait(bar_b_full, n_units & 1)) { s_abort = 1; break; }
          ++n_units;
        }
        const int s = it % kPfStages, a = it & 1;
        if (!mbar_wait(bar_a_full + 8 * s, (it / kPfStages) & 1) ||
            !mbar_wait(bar_t_empty + 8 * a, ((it >> 1) & 1) ^ 1)) { s_abort = 1; break; }
        tc_fence_after();
        const uint32_t a_base = sbase + SL::kA + s * SL::kABytes, b_base = sbase + SL::kB;
#pragma unroll
        for (int hf = 0; hf < TP; ++hf) {   // the 128-entry tiles of the hand-over, each into its own columns
#pragma unroll
          for (int k = 0; k < KSTEPS; ++k) {
            const uint64_t ad = umma_desc_sw128(a_base + (k >> 2) * (ROWS * 128) + hf * (kPfM * 128) + (k & 3) * 32);
            const uint64_t bd = umma_desc_sw128(b_base + (k >> 2) * (NB * 128) + (k & 3) * 32);
            umma_bf16(tmem + (a * TP + hf) * NB, ad, bd, IDESC, k > 0 ? 1u : 0u);
          }
        }
        umma_commit(bar_a_empty + 8 * s);
        umma_commit(bar_t_full + 8 * a);
        const bool unit_ends = wk.tile == wk.tb - 1 || it == ntiles - 1;
        if (unit_ends) umma_commit(bar_b_empty);   // the query tile may be replaced once these MMAs have read it
        wk.next(p, c.seq_len, it + 1 < ntiles);
      }
      umma_commit(bar_drain);
      mbar_wait(bar_drain, 0);   // every MMA issued above has retired (bounded)
    }
  } else {
    // ------------------------------------------------------------ drain: one entry per thread
    const int quarter = warp & 3, hq = (warp - 2) >> 2;         // this warp takes heads hq, hq + 4 of the group
    const int g_last = hq < G ? hq + ((G - 1 - hq) / 4) * 4 : -1;   // its last head (none: it only keeps in step)
    const float scale2 = p.sm_scale * kPfLog2e;
    const float ln_G = logf((float)G);
    float2 *xchg = reinterpret_cast<float2 *>(smem + SL::kXchg);
    // A wait that runs out (here or in another warp) ends the warp's work but not its walk: it goes through the
    // rest of the tiles without waiting and without reading the accumulators, and meets the warps of its quarter at
    // their barrier on every tile.
    bool dead = false;
    for (int it = 0; it < ntiles; ++it) {
      const int a = it & 1;
      if (!dead) {
        int ok = 0;
        if (lane == 0) ok = !s_abort && mbar_wait(bar_t_full + 8 * a, (it >> 1) & 1);
        if (!__shfl_sync(0xffffffffu, ok, 0)) { s_abort = 1; dead = true; }
      }
      tc_fence_after();
      const int row = quarter * 32 + lane;
      float mH[TP], SH[TP];   // (max, sum) of this thread's entry in each 128-entry tile of the hand-over
      if (g_last < 0 || dead) {   // no head for this warp (or no data any more): the accumulator is not its business
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_t_empty + 8 * a);
      }
#pragma unroll
      for (int hf = 0; hf < TP; ++hf) {
      const int i = wk.tile * ROWS + hf * kPfM + row;             // this thread's entry
      const int klo = min(32, max(0, i - wk.len + W));            // first window query that sees it
      const bool full = wk.tile * ROWS + hf * kPfM + kPfM - 1 - wk.len + W <= 0;   // every query sees the whole tile
      const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (a * TP + hf) * NB;
      float m = -CUDART_INF_F, S = 0.f;
#pragma unroll 1
      for (int g = dead ? G : hq; g < G; g += 4) {
        uint32_t r[32];
        tmem_ld_32x32(taddr + g * 32, r);
        tmem_ld_wait();
        if (g == g_last && hf == TP - 1) {   // this warp's part of the accumulators is in registers: hand them back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_t_empty + 8 * a);
        }
        // y_k = log2 of (weight_k * score_k); queries k >= W carry weight 0 (log2 = -inf).  Two copies of the
        // loop, chosen per tile: only the last tiles of a unit hold entries that some window queries do not see.
        if (full && lw.mult) {
          // Every query sees every entry of the tile and every weight is an ordinary number: the reference of the
          // exponentials is the largest raw logit (at most the window's weight range above the true maximum) and
          // the weight multiplies the exponential inside the sum: max, multiply-add, ex2, multiply-add per score.
          float r0 = fmaxf(__uint_as_float(r[0]), __uint_as_float(r[1])), r1 = fmaxf(__uint_as_float(r[2]), __uint_as_float(r[3]));
#pragma unroll
          for (int k = 4; k < 32; k += 4) {
            r0 = fmaxf(r0, fmaxf(__uint_as_float(r[k]), __uint_as_float(r[k + 1])));
            r1 = fmaxf(r1, fmaxf(__uint_as_float(r[k + 2]), __uint_as_float(r[k + 3])));
          }
          const float m_new = fmaxf(m, fmaxf(r0, r1) * scale2);
          S *= pf_ex2(m - m_new);   // m = -inf: S is 0 and stays 0 (the logits are finite, so m_new is)
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
          for (int k = 0; k < 32; k += 4) {
            a0 = fmaf(lw.w[k], pf_ex2(fmaf(__uint_as_float(r[k]), scale2, -m_new)), a0);
            a1 = fmaf(lw.w[k + 1], pf_ex2(fmaf(__uint_as_float(r[k + 1]), scale2, -m_new)), a1);
            a2 = fmaf(lw.w[k + 2], pf_ex2(fmaf(__uint_as_float(r[k + 2]), scale2, -m_new)), a2);
            a3 = fmaf(lw.w[k + 3], pf_ex2(fmaf(__uint_as_float(r[k + 3]), scale2, -m_new)), a3);
          }
          S += (a0 + a1) + (a2 + a3);
          m = m_new;
          continue;
        }
        float y[32], mc = -CUDART_INF_F, mc2 = -CUDART_INF_F;
        if (full) {
#pragma unroll
          for (int k = 0; k < 32; k += 2) {
            y[k] = fmaf(__uint_as_float(r[k]), scale2, lw.c[k]);
            y[k + 1] = fmaf(__uint_as_float(r[k + 1]), scale2, lw.c[k + 1]);
            mc = fmaxf(mc, y[k]);
            mc2 = fmaxf(mc2, y[k + 1]);
          }
        } else {
#pragma unroll
          for (int k = 0; k < 32; k += 2) {
            y[k] = k >= klo ? fmaf(__uint_as_float(r[k]), scale2, lw.c[k]) : -CUDART_INF_F;
            y[k + 1] = k + 1 >= klo ? fmaf(__uint_as_float(r[k + 1]), scale2, lw.c[k + 1]) : -CUDART_INF_F;
            mc = fmaxf(mc, y[k]);
            mc2 = fmaxf(mc2, y[k + 1]);
          }
        }
        const float m_new = fmaxf(m, fmaxf(mc, mc2));
        if (m_new > -CUDART_INF_F) {
          S *= pf_ex2(m - m_new);   // m = -inf: S is 0 and stays 0
          float add0 = 0.f, add1 = 0.f;
#pragma unroll
          for (int k = 0; k < 32; k += 2) {
            add0 += pf_ex2(y[k] - m_new);
            add1 += pf_ex2(y[k + 1] - m_new);
          }
          S += add0 + add1;
          m = m_new;
        }
      }
      mH[hf] = m; SH[hf] = S;
      }
      if (G > 1) {
        // The warps of a quarter do not wait for each other: those of heads 1-3 leave their (max, sum) and arrive,
        // only the warp of head 0 waits for them.  They can be two tiles ahead of it at most (the accumulator of
        // tile t + 3 is not written before the head-0 warp has read tile t + 1, hence combined tile t), so the
        // exchange area and the barrier rotate over three tiles.  (The same hand-over through mbarriers, with or
        // without the finishing role rotating over the four warps, measured 8-11 us slower on the C2 prompt.)
        const int x3 = it % 3;
        float2 *x2 = xchg + (x3 * ROWS + row) * 4;   // the entry of tile hf: x2 + hf * 128 * 4
        if (hq > 0) {
          if (hq < G) {
#pragma unroll
            for (int hf = 0; hf < TP; ++hf) x2[hf * kPfM * 4 + hq] = make_float2(mH[hf], SH[hf]);
          }
          __threadfence_block();
          if (dead)   // no longer paced by the accumulators: stay in step with the head-0 warp instead
            asm volatile("bar.sync %0, 128;" ::"r"(1 + quarter + 4 * x3) : "memory");
          else
            asm volatile("bar.arrive %0, 128;" ::"r"(1 + quarter + 4 * x3) : "memory");
        } else {
          asm volatile("bar.sync %0, 128;" ::"r"(1 + quarter + 4 * x3) : "memory");
        }
        if (hq == 0) {
#pragma unroll
          for (int hf = 0; hf < TP; ++hf) {
            float m = mH[hf], S = SH[hf];
#pragma unroll
            for (int w = 1; w < (G < 4 ? G : 4); ++w) {
              const float2 o = x2[hf * kPfM * 4 + w];
              const float mm = fmaxf(m, o.x);
              if (mm > -CUDART_INF_F) S = S * pf_ex2(m - mm) + o.y * pf_ex2(o.x - mm);
              m = mm;
            }
            mH[hf] = m; SH[hf] = S;
          }
        }
      }
      if (hq == 0 && !dead) {
#pragma unroll
        for (int hf = 0; hf < TP; ++hf) {
          const int i = wk.tile * ROWS + hf * kPfM + row;
          const int klo = min(32, max(0, i - wk.len + W));
          if (i < wk.len)
            c.lscore[((size_t)(wk.b * p.H_kv + wk.h)) * p.N_cap + i] =
                (mH[hf] + log2f(SH[hf])) * kPfLn2 - lnwsuf[klo] - ln_G;
        }
      }
      wk.next(p, c.seq_len, it + 1 < ntiles);
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (s_abort) {
    if (tid == 0) {
      atomicOr(status_dev, KEEPKV_DEV_TIMEOUT);
      for (int i = 0; i < kPfStages; ++i) { mbar_wait(bar_a_full + 8 * i, 0); mbar_wait(bar_a_full + 8 * i, 1); }
      mbar_wait(bar_b_full, 0); mbar_wait(bar_b_full, 1);
    }
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

template <int D, int G>
static void launch_prefill_t(const keepkv_params &p, const keepkv_cache &c, const void *q_window, int W,
                             int32_t *status_dev, LaunchCtx &ctx) {
  using SL = PfSmem<D, G>;
  constexpr size_t smem_bytes = (size_t)SL::kBytes + 1024;
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(prefill_scores_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    attr_done_dev[dev & 63] = true;
  }
  CUtensorMap mapK, mapQ;
  if (!make_bf16_rows_map(&mapK, c.K, (uint64_t)p.B * p.H_kv * p.N_cap, D, SL::kRows) ||
      !make_bf16_rows_map(&mapQ, const_cast<void *>(q_window), (uint64_t)p.B * p.H_q * W, D, W)) {
    if (ctx.err == cudaSuccess) ctx.err = cudaErrorInvalidValue;
    return;
  }
  PfLogWeights lw;
  for (int k = 0; k < kPfWmax; ++k) {
    if (k >= W) lw.c[k] = -INFINITY;
    else if (p.ema_alpha > 0.f) lw.c[k] = (float)(W - 1 - k) * log2f(p.ema_alpha);
    else lw.c[k] = k == W - 1 ? 0.f : -INFINITY;
    lw.w[k] = exp2f(lw.c[k]);
  }
  lw.mult = (W == kPfWmax && lw.c[0] >= -60.f && p.sm_scale > 0.f) ? 1 : 0;
  launch_pdl(prefill_scores_kernel<D, G>, dim3(sm_count()), dim3(kPfThreads), smem_bytes, ctx.stream, mapK, mapQ, p, c,
             W, lw, status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_prefill_scores(const keepkv_params &p, const keepkv_cache &c, const void *q_window, int W,
                           int32_t *status_dev, LaunchCtx &ctx) {
  const int G = p.H_q / p.H_kv;
#define KEEPKV_DISPATCH(DD, GG) \
  if (p.d == DD && G == GG) return launch_prefill_t<DD, GG>(p, c, q_window, W, status_dev, ctx);
  KEEPKV_DISPATCH(128, 1) KEEPKV_DISPATCH(128, 2) KEEPKV_DISPATCH(128, 4) KEEPKV_DISPATCH(128, 8)
  KEEPKV_DISPATCH(64, 1) KEEPKV_DISPATCH(64, 2) KEEPKV_DISPATCH(64, 4) KEEPKV_DISPATCH(64, 8)
#undef KEEPKV_DISPATCH
}

}  // namespace keepkv
