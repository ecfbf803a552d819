// keepkv_decode_attention: Electoral-Votes attention (Eq. 6) over the cache, with the per-entry
// score estimate of Eq. 8 advanced in the same pass.
//
// Work is the list of all 64-entry tiles of all (sequence, kv-head) units, in unit order.  A
// persistent grid (two CTAs per SM) cuts the list into equal contiguous ranges, so ragged batches
// and any number of units load every SM alike; a unit whose tiles fall into several ranges is
// finished by the last of those CTAs to arrive (one ticket per unit), in a fixed order, so results
// are bit-reproducible.
//
// With a moderate number of units (two dozen to one per SM) the grid is launched as clusters of S <= 8 CTAs, one
// cluster per unit, S * units <= two CTAs per SM.  If the units are about equally long -- every steady-state
// step -- a cluster splits its unit's tiles evenly, and the S partial results meet in distributed shared
// memory instead of global memory: each CTA leaves its partial in its own shared memory, a cluster barrier,
// each CTA folds 1/S of the outputs from its peers' memories (in rank order), a second barrier.  Ragged
// batches fall back to the equal ranges over the whole list, whatever the launch shape.
//
// One CTA = 4 warps.  Thread 0 also walks the range as producer: per tile it issues TMA loads of the
// K and V tiles (128-byte swizzled boxes), bulk copies of the tile's votes and lscore, and a small
// descriptor, into a ring of shared-memory stages guarded by full/empty mbarriers, two tiles ahead
// of the arithmetic.  The two warp pairs take alternate tiles; a warp owns 32 entries of its tile:
// the G query heads of the unit are the
// rows of an m16n8k16 bf16 MMA (rows >= G are zero), so K is read once for all heads; logits come
// out in fp32; the vote weight enters as + log2 p_i before the online softmax
// (p_i e^{l_i} = 2^{l_i log2 e + log2 p_i}), and the probabilities go back into the tensor core
// split into a bf16 head (A rows 0-7) and a bf16 remainder (A rows 8-15), so that P.V keeps
// fp32-level accuracy in one MMA.  The Eq. 8 update is done one entry per lane, from the logits the
// warp exchanges through shared memory.
//
// keepkv_decode_step runs the same kernel with the step's new token (Eq. 2) folded in: lengths count the fresh
// entry from the start; the warp that owns its row patches it into the tile it has just received (and stores
// it to the cache), so that the attention sees it.  The new lengths are published when nobody reads the old
// ones any more: every CTA copies the lengths into shared memory first and then signs off on a counter, and
// the last one to sign off writes them (batches beyond kSeqCache sequences: the last CTA to finish does).
#include <mutex>

#include "common.cuh"
#include "ptx.cuh"

namespace keepkv {

constexpr int kDecConsumers = 4;                  // warps per CTA
constexpr int kDecThreads = 32 * kDecConsumers;   // 128 threads leave each of them up to 255 registers at two CTAs per SM
constexpr int kSeqCache = 256;                    // sequence lengths a CTA keeps in shared memory
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Descriptor the producer leaves with every tile.
struct TileDesc {
  int u;          // unit
  int tile;       // tile index inside the unit
  int len;        // valid entries of the unit
  int flags;      // bit 0: first tile of this CTA's segment of the unit, bit 1: last tile of the segment
  int c_first;    // first CTA that holds a segment of the unit
  int nparts;     // CTAs that hold a segment of the unit
  int u_next;     // unit of the next tile of this CTA's range when this tile ends its unit, else -1
  int fresh;      // row inside the tile of the entry this call appends, -1 if the tile does not hold it
};

template <int D>
struct DecSmem {
  static constexpr int kSub = D / 64;
  static constexpr int kSubBytes = kTile * 128;
  static constexpr int kK = 0;
  static constexpr int kV = kSub * kSubBytes;
  static constexpr int kVotes = 2 * kSub * kSubBytes;
  static constexpr int kLscore = kVotes + kTile * 4;
  static constexpr int kTxBytes = kLscore + kTile * 4;                 // what the async copies deliver
  static constexpr int kDesc = kTxBytes;
  static constexpr int kStride = (kDesc + 32 + 1023) / 1024 * 1024;    // sub-tiles need 1024-byte alignment
  static constexpr int kStages = D == 128 ? 3 : 6;
  // Per consumer warp one region that serves two purposes at different times: while the warp works on
  // a tile, the logits it exchanges (f32 [8 heads][32 entries]) and the log2 votes (f32 [32]); while a
  // segment is combined, the warp's numerators (f32 [4 heads][D]).  A warp writes its numerators only
  // after its own tile work, and the others read them only between the barriers of the combine.
  static constexpr int kWarpRegion = (4 * D * 4 > 8 * 32 * 4 + 32 * 4) ? 4 * D * 4 : 8 * 32 * 4 + 32 * 4;
  static constexpr int kComb = kStages * kStride;
  static constexpr int kML = kComb + kDecConsumers * kWarpRegion;      // f32 [4 warps][8][2]
  static constexpr int kBytes = kML + kDecConsumers * 8 * 2 * 4;
};

// Byte offset of 16-byte chunk `chunk` (0..D/8-1) of tile row `row` inside a swizzled K or V tile.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * (kTile * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Bounded wait with a caller-chosen number of polls.
__device__ __forceinline__ bool mbar_wait_n(uint32_t bar, uint32_t parity, int limit) {
  for (int it = 0; it < limit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}

// One partial result of a unit: running maxima (base-2 exponents), sums and numerators of its G heads.
template <int D, int G>
struct PartRec {
  float m[8], l[8];
  float acc[G * D];
};

// kEarly: the variant for KEEPKV_FLAG_CACHE_IDLE (a compile-time choice: as a run-time branch the same code lost the
// gain and 0.4 us more, measured).
template <int D, int G, bool kEarly>
__global__ void __launch_bounds__(kDecThreads, 2)
decode_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, keepkv_params p,
              keepkv_cache c, const __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ out,
              float *__restrict__ lse, int update_scores, int *counters, PartRec<D, G> *pool, int32_t *status_dev,
              const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new, int spin_limit, int withhold) {
  using SL = DecSmem<D>;
  constexpr int S = SL::kStages;
  constexpr int KS = D / 16;   // k-steps of the QK^T product
  constexpr int NT = D / 8;    // 8-channel n-tiles of the PV product
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[S], empty_bar[S];
  __shared__ int s_scan[8], s_tbmax[4];
  __shared__ int s_start[4];   // b, h, tile of the first tile of this CTA's range
  __shared__ volatile int s_abort;
  __shared__ volatile int s_issued, s_stop;   // tiles the producer has handed over; first tile that never will be
  __shared__ int s_last, s_finisher;
  __shared__ int s_seq[kSeqCache];   // the lengths as they were when the kernel started

  // dynamic shared memory is only guaranteed 16-byte aligned: round up to the swizzle atom
  // (the offset is added to the array itself, so that the compiler still knows every derived pointer as shared memory)
  uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const uint32_t smem_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, grid = gridDim.x;
  const int U = p.B * p.H_kv;

  if (tid == 0) {
    for (int i = 0; i < S; ++i) { mbar_init(smem_u32(&full_bar[i]), 1); mbar_init(smem_u32(&empty_bar[i]), kDecConsumers); }
    s_abort = 0;
    s_issued = 0;
    s_stop = 0x7fffffff;
    s_start[0] = p.B;
    mbar_fence_init();
    fence_proxy_async_smem();
    prefetch_tensormap(&mapK);
    prefetch_tensormap(&mapV);
  }
  // With KEEPKV_FLAG_CACHE_IDLE the preceding kernel of the stream does not write this cache: the lengths and the
  // first tiles are then requested before the wait for that kernel, behind whose tail they arrive.  Everything else
  // (queries, the token to append, the workspace, every write) stays behind the wait.
  constexpr bool early = kEarly;
  if (!early) {
    pdl_wait();      // everything above ran while the previous kernel of the stream was finishing
    pdl_trigger();
  }

  // ---- the tile list: every thread sums a block of consecutive sequences, a block scan gives the offsets
  // entries of sequence b this call attends to: with a token to append, the fresh entry counts
  const bool cached = p.B <= kSeqCache;   // then every thread copies the lengths of its block of sequences below
  auto old_len = [&](int b) { return cached ? s_seq[b] : c.seq_len[b]; };
  auto len_of = [&](int b) {
    int n = old_len(b);
    if (k_new && n >= 0 && n < p.N_cap) ++n;
    return max(0, min(n, p.N_cap));
  };
  auto tiles_of = [&](int b) { return (len_of(b) + kTile - 1) / kTile; };
  const int per = (p.B + kDecThreads - 1) / kDecThreads;
  const int b_lo = min(p.B, tid * per), b_hi = min(p.B, b_lo + per);
  int mine = 0, tb_max = 0;
  for (int b = b_lo; b < b_hi; ++b) {
    if (cached) s_seq[b] = c.seq_len[b];   // read back by this thread here, by the others after the barrier below
    const int tb = tiles_of(b);
    mine += tb;
    tb_max = max(tb_max, tb);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) tb_max = max(tb_max, __shfl_xor_sync(0xffffffffu, tb_max, o));
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) { s_scan[warp] = incl; s_tbmax[warp] = tb_max; }
  __syncthreads();
  int before = incl - mine, total_b = 0;
  for (int w = 0; w < kDecConsumers; ++w) {
    if (w < warp) before += s_scan[w];
    total_b += s_scan[w];
  }
  const long long T = (long long)total_b * p.H_kv;
  // Equal ranges of `chunk` tiles per CTA.  When every unit has the same number of tiles and a range holds more than
  // one unit, the range is rounded up to whole units (if that costs at most an eighth more tiles per CTA): no unit is
  // then cut between two CTAs, and none of them needs the partial results and the ticket.
  int chunk = (int)((T + grid - 1) / grid);
  // one cluster per unit, if the launch has them and no sequence is much longer than the average
  const int csize = (int)cluster_nctarank(), crank = (int)cluster_ctarank();
  tb_max = max(max(s_tbmax[0], s_tbmax[1]), max(s_tbmax[2], s_tbmax[3]));
  if (tb_max > 0 && (long long)tb_max * p.B == total_b && chunk > tb_max) {
    const int up = (chunk + tb_max - 1) / tb_max * tb_max;
    if (up * 8 <= chunk * 9) chunk = up;
  }
  const bool aligned = csize > 1 && grid == U * csize && total_b > 0 && (long long)tb_max * p.B * 4 <= 5LL * total_b;
  long long g0 = min(T, (long long)cta * chunk), g1 = min(T, g0 + chunk);
  int tb_unit = 0;   // aligned: tiles of this cluster's unit
  if (aligned) {
    const int ub = (cta / csize) / p.H_kv;
    tb_unit = tiles_of(ub);
    const int t_lo = (int)((long long)crank * tb_unit / csize), t_hi = (int)((long long)(crank + 1) * tb_unit / csize);
    g0 = t_lo;   // only the tile count matters below
    g1 = t_hi;
    if (tid == 0 && t_hi > t_lo) { s_start[0] = ub; s_start[1] = (cta / csize) % p.H_kv; s_start[2] = t_lo; }
  }
  const int ntiles = (int)(g1 - g0);
  if (!aligned && ntiles > 0 && (long long)before * p.H_kv <= g0 && g0 < (long long)(before + mine) * p.H_kv) {
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
  // ------------------------------------------------------------ producer state (thread 0)
  int pb = 0, ph = 0, ptile = 0, plen = 0, ptb = 1, pit = 0;
  if (tid == 0 && ntiles > 0) {
    pb = s_start[0]; ph = s_start[1]; ptile = s_start[2];
    plen = len_of(pb);
    ptb = (plen + kTile - 1) / kTile;
  }
  // Issues the copies of tile `pit` of the range (thread 0 only); false if the stage never came free.
  auto issue_tile = [&]() -> bool {
    const int it = pit, stage = it % S;
    if (!mbar_wait_n(smem_u32(&empty_bar[stage]), ((it / S) & 1) ^ 1, spin_limit)) return false;
    const long long cur = g0 + it;
    const int u = pb * p.H_kv + ph;
    const long long us = cur - ptile, ue = us + ptb;
    TileDesc d;
    d.u = u; d.tile = ptile; d.len = plen;
    d.flags = ((it == 0 || ptile == 0) ? 1 : 0) | ((it == ntiles - 1 || ptile == ptb - 1) ? 2 : 0);
    if (aligned) {   // every CTA of the cluster holds a partial (possibly empty) unless the unit is a single tile
      d.c_first = 0;
      d.nparts = ptb == 1 ? 1 : csize;
    } else if (T < 0x7fffffffLL) {   // (64-bit divisions cost this one thread hundreds of cycles per tile)
      d.c_first = (int)us / chunk;
      d.nparts = ((int)ue - 1) / chunk - d.c_first + 1;
    } else {
      d.c_first = (int)(us / chunk);
      d.nparts = (int)((ue - 1) / chunk) - d.c_first + 1;
    }
    d.u_next = -1;
    d.fresh = -1;
    if (k_new) {
      const int old = old_len(pb);   // the fresh entry goes to row `old` of the unit
      if (old >= 0 && old < p.N_cap && old / kTile == ptile) d.fresh = old % kTile;
    }
    const size_t ubase = (size_t)u * p.N_cap;
    const int row = (int)ubase + ptile * kTile;
    const int this_tile = ptile;
    // next tile of the list (units without entries have no tiles)
    if (++ptile == ptb && it + 1 < ntiles) {
      ptile = 0;
      if (++ph == p.H_kv) {
        ph = 0;
        do {
          ++pb;
          plen = len_of(pb);
          ptb = (plen + kTile - 1) / kTile;
        } while (ptb == 0);
      }
      d.u_next = pb * p.H_kv + ph;
    }
    uint8_t *st = smem + stage * SL::kStride;
    *reinterpret_cast<TileDesc *>(st + SL::kDesc) = d;
    const uint32_t bar = smem_u32(&full_bar[stage]);
    const uint32_t dst = smem_base + stage * SL::kStride;
    if (it == withhold) {   // test hook: the tile is announced, its copies are never issued
      ++pit;
      __threadfence_block();
      s_issued = pit;
      return true;
    }
    mbar_expect_tx(bar, SL::kTxBytes);
    tma_load_3d(dst + SL::kK, &mapK, 0, row, 0, bar);   // both 64-channel halves of the tile in one copy
    tma_load_3d(dst + SL::kV, &mapV, 0, row, 0, bar);
    bulk_load_1d(dst + SL::kVotes, c.votes + ubase + (size_t)this_tile * kTile, kTile * 4, bar);
    bulk_load_1d(dst + SL::kLscore, c.lscore + ubase + (size_t)this_tile * kTile, kTile * 4, bar);
    ++pit;
    __threadfence_block();
    s_issued = pit;   // the descriptor of every tile below pit is in place
    return true;
  };
  // One cluster per unit: tile `it` of this CTA is tile a_tlo + it of the cluster's unit, so its descriptor needs
  // none of the walk over sequences and heads above (about 400 cycles per tile of this one thread).
  const int a_u = aligned ? cta / csize : 0;
  const int a_len = aligned ? len_of(a_u / p.H_kv) : 0;
  const int a_tlo = aligned ? (int)g0 : 0;
  int a_fresh_tile = -1, a_fresh_row = -1;
  if (aligned && k_new) {
    const int old = old_len(a_u / p.H_kv);
    if (old >= 0 && old < p.N_cap) { a_fresh_tile = old / kTile; a_fresh_row = old % kTile; }
  }
  auto issue_aligned = [&]() -> bool {
    const int it = pit, stage = it % S;
    if (!mbar_wait_n(smem_u32(&empty_bar[stage]), ((it / S) & 1) ^ 1, spin_limit)) return false;
    const int tile = a_tlo + it;
    TileDesc d;
    d.u = a_u; d.tile = tile; d.len = a_len;
    d.flags = (it == 0 ? 1 : 0) | (it == ntiles - 1 ? 2 : 0);
    d.c_first = 0;
    d.nparts = tb_unit == 1 ? 1 : csize;
    d.u_next = -1;
    d.fresh = tile == a_fresh_tile ? a_fresh_row : -1;
    *reinterpret_cast<TileDesc *>(smem + stage * SL::kStride + SL::kDesc) = d;
    if (it != withhold) {   // (test hook: the tile is announced, its copies are never issued)
      const uint32_t bar = smem_u32(&full_bar[stage]);
      const uint32_t dst = smem_base + stage * SL::kStride;
      const size_t ubase = (size_t)a_u * p.N_cap;
      const int row = (int)ubase + tile * kTile;
      mbar_expect_tx(bar, SL::kTxBytes);
      tma_load_3d(dst + SL::kK, &mapK, 0, row, 0, bar);
      tma_load_3d(dst + SL::kV, &mapV, 0, row, 0, bar);
      bulk_load_1d(dst + SL::kVotes, c.votes + ubase + (size_t)tile * kTile, kTile * 4, bar);
      bulk_load_1d(dst + SL::kLscore, c.lscore + ubase + (size_t)tile * kTile, kTile * 4, bar);
    }
    ++pit;
    __threadfence_block();
    s_issued = pit;
    return true;
  };
  auto issue_next = [&]() -> bool { return aligned ? issue_aligned() : issue_tile(); };
  if (tid == 0) {
    const int first = early ? S : S - 1;   // nothing else to do before the wait: fill the whole ring
    while (pit < ntiles && pit < first)
      if (!issue_next()) { s_stop = pit; s_abort = 1; break; }
  }
  if (early) {
    pdl_wait();
    pdl_trigger();   // only now: the next launch may run ahead of this one, never of this one's predecessor
  }
  if (k_new && cached && tid == kDecThreads - 1) {
    // every CTA signs off once it holds its copy of the lengths; the last one publishes the new ones (this thread
    // is not the producer: its wait for the counter hides behind the first tile's flight)
    if (atomicAdd(&counters[U], 1) == grid - 1) {
      counters[U] = 0;   // ready for the next call
      for (int b = 0; b < p.B; ++b) {
        const int n = s_seq[b];
        if (n >= 0 && n < p.N_cap) c.seq_len[b] = n + 1;
        else atomicOr(status_dev, KEEPKV_DEV_APPEND_FULL);
      }
    }
  }


  {
    // ------------------------------------------------------------ the arithmetic
    const int g = lane >> 2, qd = lane & 3;   // MMA row (query head) and position inside the quad
    const int pair = warp >> 1;               // the two warp pairs take alternate tiles
    const int r0 = (warp & 1) * 32;           // this warp's 32 rows inside a tile
    const int ctid = tid;                     // 0..127
    constexpr int WR = SL::kWarpRegion / 4;   // floats per warp region
    float *comb = reinterpret_cast<float *>(smem + SL::kComb);
    float *cml = reinterpret_cast<float *>(smem + SL::kML);
    float *sc_w = comb + warp * WR;
    float *lp_w = sc_w + 8 * 32;

    // sequences without entries: output 0, lse = -inf
    for (int u = cta; u < U; u += grid) {
      const int b = u / p.H_kv, h = u % p.H_kv;
      if (len_of(b) <= 0) {
        for (int idx = ctid; idx < G * D; idx += 32 * kDecConsumers)
          out[((size_t)b * p.H_q + h * G) * D + idx] = __float2bfloat16_rn(0.f);
        if (lse && ctid < G) lse[(size_t)b * p.H_q + h * G + ctid] = -CUDART_INF_F;
      }
    }

    const float ln_alpha = p.ema_alpha > 0.f ? __logf(p.ema_alpha) : -CUDART_INF_F;
    const float ln_1ma = log1pf(-p.ema_alpha);
    const float ln_G = __logf((float)G);

    // Q fragments (A operand of QK^T): row g = query head, rows >= G and rows 8-15 are zero.  They are
    // fetched ahead of the segment that uses them: before the first tile arrives, and while the
    // previous segment is being combined.
    uint32_t qa[KS][2];
    auto load_q = [&](int u) {
      const int b = u / p.H_kv, h = u % p.H_kv;
      const __nv_bfloat16 *qrow = q + ((size_t)b * p.H_q + h * G + (g < G ? g : 0)) * D;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qa[ks][0] = g < G ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + qd * 2) : 0u;
        qa[ks][1] = g < G ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + 8 + qd * 2) : 0u;
      }
    };
    if (ntiles > 0) load_q(s_start[0] * p.H_kv + s_start[1]);
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
    float m_run = -CUDART_INF_F, l_run = 0.f;   // running max (base-2 exponent) and per-thread partial sum of head g
    bool dead = false;                          // a bounded wait ran out: no more waiting, no more arithmetic

    for (int it = 0; it < ntiles; ++it) {
      const int stage = it % S;
      // keep the ring S-1 tiles ahead: the stage of tile it-1 is free once all four warps have left it
      if (tid == 0 && pit < ntiles && pit <= it + S - 1 && s_stop > pit)
        if (!issue_next()) { s_stop = pit; s_abort = 1; }
      __syncwarp();
      if (!dead) {
        int ok = 0;
        if (lane == 0) ok = !s_abort && mbar_wait_n(smem_u32(&full_bar[stage]), (it / S) & 1, spin_limit);
        if (!__shfl_sync(0xffffffffu, ok, 0)) { s_abort = 1; dead = true; }
      }
      if (dead) {
        // A wait ran out (here or in another warp): the kernel's result is lost, but its barriers are not.  The warp
        // walks the rest of its range without waiting for data and without arithmetic, so that it still meets the
        // others at every barrier of the combines; it only makes sure that the descriptor it acts on exists, and
        // all four warps stop at the same tile if the producer gave up.
        int go = 1;
        if (lane == 0) {
          int polls = 0;
          while (s_issued <= it && s_stop > it && polls < spin_limit) { ++polls; __nanosleep(64); }
          go = s_issued > it;
        }
        if (!__shfl_sync(0xffffffffu, go, 0)) break;
      }
      const uint32_t st = smem_base + stage * SL::kStride;
      const uint8_t *stp = smem + stage * SL::kStride;
      const TileDesc d = *reinterpret_cast<const TileDesc *>(stp + SL::kDesc);
      const int b = d.u / p.H_kv, h = d.u % p.H_kv;

      const int i_base = d.tile * kTile + r0;     // first entry of this warp's slice
      const int n_valid = d.len - i_base;         // entries of the slice that exist (may be <= 0 or >= 32)
      const bool mine = (it & 1) == pair && !dead;
      const bool patch = mine && d.fresh >= r0 && d.fresh < r0 + 32;
      if (patch) {
        // Eq. 2 inside this call: the row of the fresh entry arrived with whatever the cache held; this warp,
        // the only one to read it, overwrites it in the tile and in the cache (one vote, no score history)
        constexpr int CH = D / 8;
        const size_t e = (size_t)d.u * p.N_cap + d.tile * kTile + d.fresh;
        const int half = lane >> 4, ch = lane & 15;
        if (ch < CH) {
          const uint4 val = (half ? v_new : k_new)[(size_t)d.u * CH + ch];
          *reinterpret_cast<uint4 *>(smem + stage * SL::kStride + (half ? SL::kV : SL::kK) + swz(d.fresh, ch)) = val;
          reinterpret_cast<uint4 *>(half ? c.V : c.K)[e * CH + ch] = val;
        }
        if (lane == 0) {
          reinterpret_cast<float *>(smem + stage * SL::kStride + SL::kVotes)[d.fresh] = 1.0f;
          reinterpret_cast<float *>(smem + stage * SL::kStride + SL::kLscore)[d.fresh] = -CUDART_INF_F;
          c.votes[e] = 1.0f;
          if (!update_scores) c.lscore[e] = -CUDART_INF_F;   // otherwise Eq. 8 below writes the first observation
        }
        __syncwarp();
      }
      if (mine && n_valid > 0) {
        const bool ragged = n_valid < 32;
        if (ragged) {
          // rows past the sequence hold unspecified bits; zero their V so that 0 * garbage cannot turn
          // into NaN inside the tensor core
          for (int idx = lane; idx < 32 * (D / 8); idx += 32) {
            const int r = idx / (D / 8), ch = idx % (D / 8);
            if (r >= n_valid)
              *reinterpret_cast<uint4 *>(smem + stage * SL::kStride + SL::kV + swz(r0 + r, ch)) = make_uint4(0, 0, 0, 0);
          }
          __syncwarp();
        }

        // ---- logits: S[head][entry] for the 32 entries, four independent n-tiles of 8
        float sc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
        for (int kk = 0; kk < KS / 2; ++kk) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int row = r0 + j * 8 + (lane & 7);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(st + SL::kK + swz(row, kk * 4 + (lane >> 3)), b0, b1, b2, b3);
            mma_bf16(sc[j], qa[2 * kk][0], 0u, qa[2 * kk][1], 0u, b0, b1);
            mma_bf16(sc[j], qa[2 * kk + 1][0], 0u, qa[2 * kk + 1][1], 0u, b2, b3);
          }
        }
        // this thread holds head g, entries e(j,t) = 8 j + 2 qd + t of the slice, in natural-log units
        float x[4][2];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          x[j][0] = sc[j][0] * p.sm_scale;
          x[j][1] = sc[j][1] * p.sm_scale;
          if (g < G) *reinterpret_cast<float2 *>(sc_w + g * 32 + j * 8 + qd * 2) = make_float2(x[j][0], x[j][1]);
        }
        __syncwarp();

        // ---- one lane per entry: log2 of the vote; Eq. 8 with the kv head's score = mean over its G heads of e^{l}
        {
          const int e = lane;
          const float pv = reinterpret_cast<const float *>(stp + SL::kVotes)[r0 + e];
          if (update_scores) {
            float mx = sc_w[e];
#pragma unroll
            for (int gg = 1; gg < G; ++gg) mx = fmaxf(mx, sc_w[gg * 32 + e]);
            float sigma = mx;
            if (G > 1) {
              float se = 0.f;
#pragma unroll
              for (int gg = 0; gg < G; ++gg) se += ex2f((sc_w[gg * 32 + e] - mx) * kLog2e);
              sigma = mx + lg2f(se) * kLn2 - ln_G;
            }
            const float old = reinterpret_cast<const float *>(stp + SL::kLscore)[r0 + e];
            float r = sigma;
            if (old > -CUDART_INF_F && p.ema_alpha > 0.f) {
              const float a = ln_alpha + old, bb = ln_1ma + sigma;
              const float hi = fmaxf(a, bb), lo = fminf(a, bb);
              r = hi + lg2f(1.f + ex2f((lo - hi) * kLog2e)) * kLn2;
            }
            if (e < n_valid) c.lscore[(size_t)d.u * p.N_cap + i_base + e] = r;
          }
          lp_w[e] = e < n_valid ? lg2f(pv) : -CUDART_INF_F;
        }
        __syncwarp();

        // ---- Eq. 6: weights p_i e^{l_i} = 2^{x log2e + log2 p} through an online softmax
        float mloc = -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 lp = *reinterpret_cast<const float2 *>(lp_w + j * 8 + qd * 2);
          x[j][0] = fmaf(x[j][0], kLog2e, lp.x);   // -inf for entries past the sequence
          x[j][1] = fmaf(x[j][1], kLog2e, lp.y);
          if (ragged) {   // garbage logits of missing entries may be NaN or +inf
            if (j * 8 + qd * 2 >= n_valid) x[j][0] = -CUDART_INF_F;
            if (j * 8 + qd * 2 + 1 >= n_valid) x[j][1] = -CUDART_INF_F;
          }
          mloc = fmaxf(mloc, fmaxf(x[j][0], x[j][1]));
        }
        mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, 1));
        mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, 2));
        const float m_new = fmaxf(m_run, mloc);
        const bool grow = m_new > m_run;
        if (__any_sync(0xffffffffu, grow)) {
          const float scale = grow ? ex2f(m_run - m_new) : 1.f;   // m_run = -inf gives 0; o and l are 0 then anyway
          l_run *= scale;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            o[nt][0] *= scale; o[nt][1] *= scale; o[nt][2] *= scale; o[nt][3] *= scale;
          }
          m_run = m_new;
        }
        // A fragments of P for the two 16-entry k-steps: a0/a2 = bf16 head (rows 0-7), a1/a3 = bf16
        // remainder (rows 8-15)
        uint32_t pa[2][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float p0 = m_run > -CUDART_INF_F ? ex2f(x[j][0] - m_run) : 0.f;
          const float p1 = m_run > -CUDART_INF_F ? ex2f(x[j][1] - m_run) : 0.f;
          l_run += p0 + p1;
          const uint32_t hi2 = pack_bf16(p0, p1);
          pa[j >> 1][2 * (j & 1)] = hi2;
          pa[j >> 1][2 * (j & 1) + 1] = pack_bf16(p0 - bf16_lo(hi2), p1 - bf16_hi(hi2));
        }
        // ---- O += P V   (rows 0-7 collect the head part, rows 8-15 the remainder part)
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
          const int vrow = r0 + ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
          for (int np = 0; np < NT / 2; ++np) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(st + SL::kV + swz(vrow, np * 2 + (lane >> 4)), b0, b1, b2, b3);
            mma_bf16(o[2 * np], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b0, b1);
            mma_bf16(o[2 * np + 1], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b2, b3);
          }
        }
        if (ragged || patch) fence_proxy_async_smem();   // the rows written here precede the next TMA write
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&empty_bar[stage]));   // this warp is done with the stage

      if (d.flags & 2) {
        // ---- end of this CTA's segment of the unit: combine the four warps
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
        l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
        if (g < G && qd == 0) { cml[(warp * 8 + g) * 2] = m_run; cml[(warp * 8 + g) * 2 + 1] = l_run; }
        const bool whole = d.nparts == 1;
        PartRec<D, G> *rec = pool + (size_t)cta * 2 + (d.c_first == cta ? 1 : 0);
        float osum[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          osum[nt][0] = o[nt][0] + o[nt][2]; osum[nt][1] = o[nt][1] + o[nt][3];
          o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
        }
        if (d.u_next >= 0) load_q(d.u_next);   // in flight while this segment is combined
        m_run = -CUDART_INF_F;
        l_run = 0.f;
        constexpr int ROUNDS = (G + 3) / 4, RG = G < 4 ? G : 4;
#pragma unroll
        for (int rd = 0; rd < ROUNDS; ++rd) {
          if (g < G && (g >> 2) == rd) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
              *reinterpret_cast<float2 *>(&comb[(size_t)warp * WR + (g & 3) * D + nt * 8 + qd * 2]) =
                  make_float2(osum[nt][0], osum[nt][1]);
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
          for (int idx = ctid; idx < RG * D; idx += 32 * kDecConsumers) {
            const int gl = idx / D, j = idx % D, gg = rd * 4 + gl;
            float M = cml[gg * 2];
#pragma unroll
            for (int w = 1; w < kDecConsumers; ++w) M = fmaxf(M, cml[(w * 8 + gg) * 2]);
            float Ls = 0.f, a = 0.f;
            if (M > -CUDART_INF_F) {
#pragma unroll
              for (int w = 0; w < kDecConsumers; ++w) {
                const float f = ex2f(cml[(w * 8 + gg) * 2] - M);
                Ls += f * cml[(w * 8 + gg) * 2 + 1];
                a += f * comb[(size_t)w * WR + gl * D + j];
              }
            }
            if (whole) {
              const size_t qo = (size_t)b * p.H_q + h * G + gg;
              out[qo * D + j] = __float2bfloat16_rn(Ls > 0.f ? a / Ls : 0.f);
              if (lse && j == 0) lse[qo] = Ls > 0.f ? (M + lg2f(Ls)) * kLn2 : -CUDART_INF_F;
            } else if (aligned) {   // this CTA's partial stays in its shared memory (the ring is idle by now)
              float *xr = reinterpret_cast<float *>(smem);
              xr[16 + gg * D + j] = a;
              if (j == 0) { xr[gg] = M; xr[8 + gg] = Ls; }
            } else {
              rec->acc[gg * D + j] = a;
              if (j == 0) { rec->m[gg] = M; rec->l[gg] = Ls; }
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        if (!whole && !aligned) {
          // ---- the last CTA of the unit to arrive merges the partials, in CTA order
          __threadfence();
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (ctid == 0) {
            const int ticket = atomicAdd(&counters[d.u], 1);
            s_last = (ticket == d.nparts - 1);
            if (s_last) counters[d.u] = 0;   // ready for the next call
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (s_last) {
            __threadfence();
            // comb[part][head] = (m_k, scale factor 2^{m_k - M}); cml[head] = M
            constexpr int kMaxParts = kDecConsumers * WR / (2 * G);
            const int np_ = d.nparts;
            auto part = [&](int k) { return pool + (size_t)(d.c_first + k) * 2 + (k == 0 ? 1 : 0); };
            constexpr int NI = (G * D + 32 * kDecConsumers - 1) / (32 * kDecConsumers);   // outputs per thread
            constexpr int KF = NI <= 4 ? 8 : 4;   // parts the register path holds
            if (np_ <= KF) {
              // few parts (the usual case): everything in registers, one round trip to L2
              float pm[KF][NI], pl[KF][NI], pa_[KF][NI];
#pragma unroll
              for (int k = 0; k < KF; ++k) {
                const PartRec<D, G> *r = part(k < np_ ? k : 0);
#pragma unroll
                for (int i = 0; i < NI; ++i) {
                  const int idx = min(ctid + i * 32 * kDecConsumers, G * D - 1);
                  pm[k][i] = k < np_ ? __ldcg(&r->m[idx / D]) : -CUDART_INF_F;
                  pl[k][i] = __ldcg(&r->l[idx / D]);
                  pa_[k][i] = __ldcg(&r->acc[idx]);
                }
              }
#pragma unroll
              for (int i = 0; i < NI; ++i) {
                const int idx = ctid + i * 32 * kDecConsumers;
                float M = pm[0][i];
#pragma unroll
                for (int k = 1; k < KF; ++k) M = fmaxf(M, pm[k][i]);
                float Ls = 0.f, a = 0.f;
#pragma unroll
                for (int k = 0; k < KF; ++k) {
                  const float f = pm[k][i] > -CUDART_INF_F ? ex2f(pm[k][i] - M) : 0.f;
                  Ls = fmaf(f, pl[k][i], Ls);
                  a = fmaf(f, pa_[k][i], a);
                }
                if (idx < G * D) {
                  const int gg = idx / D, j = idx % D;
                  const size_t qo = (size_t)b * p.H_q + h * G + gg;
                  out[qo * D + j] = __float2bfloat16_rn(Ls > 0.f ? a / Ls : 0.f);
                  if (lse && j == 0) lse[qo] = Ls > 0.f ? (M + lg2f(Ls)) * kLn2 : -CUDART_INF_F;
                }
              }
            } else if (np_ <= kMaxParts) {
              for (int idx = ctid; idx < np_ * G; idx += 32 * kDecConsumers)
                comb[idx * 2] = __ldcg(&part(idx / G)->m[idx % G]);
              asm volatile("bar.sync 1, 128;" ::: "memory");
              for (int idx = ctid; idx < np_ * G; idx += 32 * kDecConsumers) {
                const int gg = idx % G;
                float M = -CUDART_INF_F;
                for (int k = 0; k < np_; ++k) M = fmaxf(M, comb[(k * G + gg) * 2]);
                comb[idx * 2 + 1] = M > -CUDART_INF_F ? ex2f(comb[idx * 2] - M) : 0.f;
                if (idx < G) cml[gg] = M;
              }
              asm volatile("bar.sync 1, 128;" ::: "memory");
              // every thread owns NI outputs; the parts are the outer loop so that all loads of a part
              // are in flight together
              float Ls[NI], a[NI];
#pragma unroll
              for (int i = 0; i < NI; ++i) Ls[i] = a[i] = 0.f;
#pragma unroll 2
              for (int k = 0; k < np_; ++k) {
                const PartRec<D, G> *r = part(k);
#pragma unroll
                for (int i = 0; i < NI; ++i) {
                  const int idx = ctid + i * 32 * kDecConsumers;
                  if (idx < G * D) {
                    const int gg = idx / D;
                    const float f = comb[(k * G + gg) * 2 + 1];
                    Ls[i] = fmaf(f, __ldcg(&r->l[gg]), Ls[i]);
                    a[i] = fmaf(f, __ldcg(&r->acc[idx]), a[i]);
                  }
                }
              }
#pragma unroll
              for (int i = 0; i < NI; ++i) {
                const int idx = ctid + i * 32 * kDecConsumers;
                if (idx < G * D) {
                  const int gg = idx / D, j = idx % D;
                  const size_t qo = (size_t)b * p.H_q + h * G + gg;
                  out[qo * D + j] = __float2bfloat16_rn(Ls[i] > 0.f ? a[i] / Ls[i] : 0.f);
                  if (lse && j == 0) lse[qo] = Ls[i] > 0.f ? (cml[gg] + lg2f(Ls[i])) * kLn2 : -CUDART_INF_F;
                }
              }
            } else {
              for (int idx = ctid; idx < G * D; idx += 32 * kDecConsumers) {
                const int gg = idx / D, j = idx % D;
                float M = -CUDART_INF_F;
                for (int k = 0; k < np_; ++k) M = fmaxf(M, __ldcg(&part(k)->m[gg]));
                float Ls = 0.f, a = 0.f;
                if (M > -CUDART_INF_F) {
                  for (int k = 0; k < np_; ++k) {
                    const float f = ex2f(__ldcg(&part(k)->m[gg]) - M);
                    Ls = fmaf(f, __ldcg(&part(k)->l[gg]), Ls);
                    a = fmaf(f, __ldcg(&part(k)->acc[gg * D + j]), a);
                  }
                }
                const size_t qo = (size_t)b * p.H_q + h * G + gg;
                out[qo * D + j] = __float2bfloat16_rn(Ls > 0.f ? a / Ls : 0.f);
                if (lse && j == 0) lse[qo] = Ls > 0.f ? (M + lg2f(Ls)) * kLn2 : -CUDART_INF_F;
              }
            }
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");   // s_last is reused by the next segment
        }
      }
    }
  }

  __syncthreads();
  if (aligned && tb_unit > 1) {
    // ---- the cluster folds its unit's partials through distributed shared memory: [m[8], l[8], acc[G*D]] per CTA
    float *xr = reinterpret_cast<float *>(smem);
    if (ntiles == 0 && tid < 8) { xr[tid] = -CUDART_INF_F; xr[8 + tid] = 0.f; }   // no tiles here: an empty partial
    cluster_sync_all();
    const int u = cta / csize, b = u / p.H_kv, h = u % p.H_kv;
    const int per_cta = G * D / csize;   // outputs this CTA folds
    const uint32_t xr_addr = smem_u32(xr);
    for (int k = tid; k < per_cta; k += kDecThreads) {
      const int idx = crank * per_cta + k, gg = idx / D, j = idx % D;
      float pm[8], pl[8], pa_[8];
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        pm[r] = -CUDART_INF_F; pl[r] = 0.f; pa_[r] = 0.f;
        if (r < csize) {
          const uint32_t ra = mapa_shared(xr_addr, (uint32_t)r);
          pm[r] = ld_shared_cluster_f32(ra + gg * 4);
          pl[r] = ld_shared_cluster_f32(ra + (8 + gg) * 4);
          pa_[r] = ld_shared_cluster_f32(ra + (16 + idx) * 4);
        }
      }
      float M = pm[0];
#pragma unroll
      for (int r = 1; r < 8; ++r) M = fmaxf(M, pm[r]);
      float Ls = 0.f, a = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        // a CTA without tiles published m = -inf and nothing else: its numerators are whatever its shared
        // memory held (0 * NaN would poison the sum), so an empty partial is skipped, not weighted by zero
        if (pm[r] > -CUDART_INF_F) {
          const float f = ex2f(pm[r] - M);
          Ls = fmaf(f, pl[r], Ls);
          a = fmaf(f, pa_[r], a);
        }
      }
      const size_t qo = (size_t)b * p.H_q + h * G + gg;
      out[qo * D + j] = __float2bfloat16_rn(Ls > 0.f ? a / Ls : 0.f);
      if (lse && j == 0) lse[qo] = Ls > 0.f ? (M + lg2f(Ls)) * kLn2 : -CUDART_INF_F;
    }
    cluster_sync_all();   // nobody leaves while a peer still reads its shared memory
  }
  if (k_new && !cached) {
    // the new lengths are published by the last CTA to get here: every CTA has read the old ones for the last time
    if (tid == 0) {
      __threadfence();
      s_finisher = atomicAdd(&counters[U], 1) == grid - 1;
      if (s_finisher) counters[U] = 0;   // ready for the next call
    }
    __syncthreads();
    if (s_finisher) {
      for (int b = tid; b < p.B; b += kDecThreads) {
        const int n = c.seq_len[b];
        if (n >= 0 && n < p.N_cap) c.seq_len[b] = n + 1;
        else atomicOr(status_dev, KEEPKV_DEV_APPEND_FULL);
      }
    }
  }
  if (s_abort) {
    // give copies still in flight a bounded chance to land before the CTA's shared memory goes away
    if (tid == 0) {
      atomicOr(status_dev, KEEPKV_DEV_TIMEOUT);
      for (int i = 0; i < S; ++i) { mbar_wait_n(smem_u32(&full_bar[i]), 0, spin_limit); mbar_wait_n(smem_u32(&full_bar[i]), 1, spin_limit); }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------- host side
// What a test may change: the number of polls of a bounded wait, and one position of every CTA's tile range
// that the producer announces without issuing its copies, so that the consumers' wait for it runs out with
// nothing in flight (keepkv_debug_decode in the header).
static int g_dbg_spin = kSpinLimit;
static int g_dbg_withhold = -1;
void decode_debug(int spin_limit, int withhold) {
  g_dbg_spin = spin_limit > 0 ? spin_limit : kSpinLimit;
  g_dbg_withhold = withhold;
}

// Tensor maps are a function of (base pointer, rows, D): a serving loop calls with the same few caches over and
// over, so the encoded maps are kept in a small table instead of being rebuilt by the driver on every launch.
struct MapKey { const void *base; uint64_t rows; int D; };
static bool cached_rows_map(CUtensorMap *out, void *base, uint64_t rows, int D) {
  constexpr int N = 64;
  static MapKey keys[N];
  static CUtensorMap maps[N];
  static int used = 0, next = 0;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < used; ++i)
    if (keys[i].base == base && keys[i].rows == rows && keys[i].D == D) { *out = maps[i]; return true; }
  if (!make_bf16_halves_map(out, base, rows, D, kTile)) return false;
  const int slot = used < N ? used++ : (next++ % N);
  keys[slot] = MapKey{base, rows, D};
  maps[slot] = *out;
  return true;
}
template <int D, int G, bool E>
static void launch_t(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                     int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, const void *k_new,
                     const void *v_new, LaunchCtx &ctx) {
  using SL = DecSmem<D>;
  constexpr size_t smem_bytes = (size_t)SL::kBytes + 1024;
  static_assert(sizeof(PartRec<D, G>) == (16 + G * D) * 4, "partial record layout");
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(decode_kernel<D, G, E>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    attr_done_dev[dev & 63] = true;
  }
  CUtensorMap mapK, mapV;
  const uint64_t rows = (uint64_t)p.B * p.H_kv * p.N_cap;
  if (!cached_rows_map(&mapK, c.K, rows, D) || !cached_rows_map(&mapV, c.V, rows, D)) {
    if (ctx.err == cudaSuccess) ctx.err = cudaErrorInvalidValue;
    return;
  }
  // two CTAs per SM, never more than tiles could exist or than the partial pool holds
  const long long max_tiles = (long long)p.B * p.H_kv * (p.N_cap / kTile);   // N_cap % 64 == 0: at least one
  long long grid = 2LL * sm_count();
  if (grid > kDecMaxCtas) grid = kDecMaxCtas;
  // Two dozen units to one per SM: one cluster per unit, with as many CTAs per cluster (8, 4 or 2) as two per SM
  // allow -- provided all clusters are resident at once and at least 0.6 of the CTA slots are used (16 units
  // x 8 = 128 CTAs ran 17.3 us where the equal ranges over the whole list took 15.9 us).  The idle-cache variant
  // takes clusters from 0.2 of the slots on: the slots a small launch leaves free are where the next launch's CTAs
  // start reading (16 units x 8: 13.3 us against 15.4 us; 8 short units x 8: 8.1 against 11.8 us).
  const int U = p.B * p.H_kv;
  int cs = 1;
  if (2 * U <= grid && p.N_cap / kTile >= 2) {
    static int max_clusters_dev[64][4] = {};   // per device and log2(cluster size); 0 = not asked yet, -1 = none
    for (int c = 8; c > 1 && cs == 1; c >>= 1) {
      if ((long long)U * c > grid || (E ? 5LL * U * c < 1 * grid : 5LL * U * c < 3 * grid)) continue;
      if (c == 8 && 4LL * U * c > 3 * grid) continue;   // 32 clusters of 8 are all resident, yet ran 16.7 us against 14.2 us
      const int li = c == 8 ? 3 : (c == 4 ? 2 : 1);
      int &mc = max_clusters_dev[dev & 63][li];
      if (mc == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(U * c));
        cfg.blockDim = dim3(kDecThreads);
        cfg.dynamicSmemBytes = smem_bytes;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)c;
        at[0].val.clusterDim.y = 1;
        at[0].val.clusterDim.z = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, decode_kernel<D, G, E>, &cfg) != cudaSuccess) { n = 0; cudaGetLastError(); }
        mc = n > 0 ? n : -1;
      }
      if (U <= mc) cs = c;
    }
  }
  if (cs > 1) {
    launch_pdl_cluster(decode_kernel<D, G, E>, dim3((unsigned)(U * cs)), dim3(kDecThreads), smem_bytes, ctx.stream, cs,
        mapK, mapV, p, c, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out), lse,
        update_scores, reinterpret_cast<int *>(ws + L.counters), reinterpret_cast<PartRec<D, G> *>(ws + L.part_pool),
        status_dev, reinterpret_cast<const uint4 *>(k_new), reinterpret_cast<const uint4 *>(v_new), g_dbg_spin, g_dbg_withhold);
    KEEPKV_CHECK_LAUNCH(ctx);
    return;
  }
  if (grid > max_tiles) grid = max_tiles;
  launch_pdl(decode_kernel<D, G, E>, dim3((unsigned)grid), dim3(kDecThreads), smem_bytes, ctx.stream,
      mapK, mapV, p, c, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out), lse,
      update_scores, reinterpret_cast<int *>(ws + L.counters), reinterpret_cast<PartRec<D, G> *>(ws + L.part_pool),
      status_dev, reinterpret_cast<const uint4 *>(k_new), reinterpret_cast<const uint4 *>(v_new), g_dbg_spin, g_dbg_withhold);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_decode(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                   int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx, const void *k_new,
                   const void *v_new) {
  const int G = p.H_q / p.H_kv;
  const bool early = (p.flags & KEEPKV_FLAG_CACHE_IDLE) != 0;
#define KEEPKV_DISPATCH(DD, GG) \
  if (p.d == DD && G == GG) \
    return early ? launch_t<DD, GG, true>(p, c, q, out, lse, update_scores, ws, L, status_dev, k_new, v_new, ctx) \
                 : launch_t<DD, GG, false>(p, c, q, out, lse, update_scores, ws, L, status_dev, k_new, v_new, ctx);
  KEEPKV_DISPATCH(128, 1) KEEPKV_DISPATCH(128, 2) KEEPKV_DISPATCH(128, 4) KEEPKV_DISPATCH(128, 8)
  KEEPKV_DISPATCH(64, 1) KEEPKV_DISPATCH(64, 2) KEEPKV_DISPATCH(64, 4) KEEPKV_DISPATCH(64, 8)
#undef KEEPKV_DISPATCH
}

}  // namespace keepkv

extern "C" int keepkv_debug_decode(int spin_limit, int withhold_tile) {
  keepkv::decode_debug(spin_limit, withhold_tile);
  return KEEPKV_OK;
}
