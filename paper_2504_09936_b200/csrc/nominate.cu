// Similarity search of keepkv_compress (Algorithm 1, similarity step: U = cosineSimilarity(K_e, K_c)) on the
// 5th-generation tensor cores.  The cosine matrix is never stored: for every evicted key the kernel
// keeps the two largest cosines over the retained keys and their slots, which is all the arg-max
// of Algorithm 1 needs.  The values found here only *rank* candidates; wherever the
// ranking is closer than the accumulation error allows, the caller re-evaluates the candidates in
// the fixed fp32 arithmetic the interface defines (see resolve_kernel in compress.cu).
//
// Work item = (unit, 128 evicted rows, one chunk of 256-column tiles of the unit's retained keys).
// A persistent grid of one CTA per SM walks the items.  Inside a CTA:
//   warp 0      TMA producer: retained-key tiles (256 rows x D, 128-byte swizzle) from the compacted
//               dst cache into a 2-stage ring;
//   warp 1      one thread issues tcgen05.mma (M=128, N=256, K=16, bf16 -> fp32) into one of two
//               256-column accumulators in tensor memory and commits to the ring / accumulator barriers;
//   warps 2-17  gather the 128 evicted rows from the src cache into the swizzled A tile, then drain the
//               accumulators with tcgen05.ld: four warps per 32-lane quarter, each 64 of a tile's 256 columns
//               (the drain is a latency chain per warp: with two warps per quarter the issue slots were a third
//               full), scaling by the retained keys' inverse norms and tracking the row's top two.
// Every wait is bounded; a wait that runs out raises KEEPKV_DEV_TIMEOUT, the CTA stops issuing work,
// drains what is in flight, frees its tensor memory and returns.
#include <type_traits>

#include "compress.cuh"
#include "ptx.cuh"

namespace keepkv {

constexpr int kNomM = 128;        // evicted rows per item (tensor-memory lanes)
constexpr int kNomN = 256;        // retained columns per tile
constexpr int kNomStages = 2;     // B ring
constexpr int kNomDrainWarps = 16; // four per 32-lane quarter of tensor memory, each a quarter of a tile's columns
constexpr int kNomThreads = 32 * (2 + kNomDrainWarps);

template <int D>
struct NomSmem {
  static constexpr int kSub = D / 64;                     // 64-channel (128-byte) K atoms per row
  static constexpr int kABytes = kSub * kNomM * 128;
  static constexpr int kBBytes = kSub * kNomN * 128;
  static constexpr int kA = 0;
  static constexpr int kB = 2 * kABytes;                  // two A tiles: the next item is gathered while this one is drained
  static constexpr int kInv = kB + kNomStages * kBBytes;  // f32 [16 warps][64]   inverse norms of the warp's columns
  static constexpr int kRowInv = kInv + 16 * 64 * 4;      // f32 [2][128]         inverse norms of the staged rows
  static constexpr int kXchg = kRowInv + 2 * 128 * 4;     // u32 [2][128][3][3]   exchange between the column quarters
  static constexpr int kPrefix = kXchg + 2 * 128 * 9 * 4; // i32 [kMaxUnits + 1]  row-tile prefix over units
  static constexpr int kBytes = kPrefix + (kMaxUnits + 1) * 4;
};

struct NomItem { int u, m_tile, chunk, t0, t1, n_ev, n_ret; };

__device__ __forceinline__ NomItem nom_item(int item, int C, const int *prefix, int U, const UnitInfo *unit_info) {
  NomItem it;
  const int mg = item / C;
  it.chunk = item % C;
  int lo = 0, hi = U;   // largest u with prefix[u] <= mg
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (prefix[mid] <= mg) lo = mid; else hi = mid;
  }
  it.u = lo;
  it.m_tile = mg - prefix[lo];
  const UnitInfo ui = unit_info[lo];
  it.n_ev = ui.n_ev;
  it.n_ret = ui.n_ret;
  const int T = (ui.n_ret + kNomN - 1) / kNomN;
  it.t0 = (int)((long long)it.chunk * T / C);
  it.t1 = (int)((long long)(it.chunk + 1) * T / C);
  return it;
}

template <int D>
__global__ void __launch_bounds__(kNomThreads, 1)
nominate_kernel(const __grid_constant__ CUtensorMap mapB, keepkv_params p, const __nv_bfloat16 *__restrict__ srcK,
                const int32_t *__restrict__ ev_idx, const UnitInfo *__restrict__ unit_info,
                const float *__restrict__ inv_norm, int32_t *sched, float4 *__restrict__ nom_v,
                int32_t *__restrict__ nom_si, int C_max, int32_t *status_dev, int self_mask) {
  using SL = NomSmem<D>;
  constexpr int KSTEPS = D / 16;
  constexpr uint32_t IDESC = umma_idesc_bf16(kNomM, kNomN);
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bars[11];   // a_ready[2], b_full[2], b_empty[2], t_full[2], t_empty[2], drain
  __shared__ uint32_t s_tmem;
  __shared__ int s_wtot[kNomThreads / 32];
  __shared__ volatile int s_abort;

  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar_a_ready = smem_u32(&bars[0]);
  const uint32_t bar_b_full = smem_u32(&bars[2]), bar_b_empty = smem_u32(&bars[4]);
  const uint32_t bar_t_full = smem_u32(&bars[6]), bar_t_empty = smem_u32(&bars[8]);
  const uint32_t bar_drain = smem_u32(&bars[10]);
  int *prefix = reinterpret_cast<int *>(smem + SL::kPrefix);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int U = p.B * p.H_kv;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_a_ready + 8 * i, kNomDrainWarps);
      mbar_init(bar_b_full + 8 * i, 1);
      mbar_init(bar_b_empty + 8 * i, 1);
      mbar_init(bar_t_full + 8 * i, 1);
      mbar_init(bar_t_empty + 8 * i, kNomDrainWarps);
    }
    mbar_init(bar_drain, 1);
    s_abort = 0;
    mbar_fence_init();
    fence_proxy_async_smem();
    prefetch_tensormap(&mapB);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&s_tmem), 512);
    tmem_relinquish();
  }
  pdl_wait();      // barrier set-up and tensor-memory allocation overlap the previous kernel's tail
  pdl_trigger();
  {   // exclusive prefix of 128-row tiles over the units: one unit per thread and pass
    int run = 0;
    for (int u0 = 0; u0 < U; u0 += kNomThreads) {
      const int u = u0 + tid;
      const int t = u < U ? (unit_info[u].n_ev + kNomM - 1) / kNomM : 0;
      int x = t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
      }
      if (lane == 31) s_wtot[warp] = x;
      __syncthreads();
      int off = 0, tot = 0;
#pragma unroll
      for (int w = 0; w < kNomThreads / 32; ++w) {
        const int v = s_wtot[w];
        off += w < warp ? v : 0;
        tot += v;
      }
      if (u < U) prefix[u] = run + off + x - t;
      run += tot;
      __syncthreads();
    }
    if (tid == 0) prefix[U] = run;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  const uint32_t tmem = s_tmem;
  const int total_m = prefix[U];
  // few row tiles: split every row's columns into chunks so that all SMs get one item (a second wave
  // of items would cost more in fixed latency than the shorter items save)
  int C = total_m > 0 ? (int)gridDim.x / total_m : 1;
  C = max(1, min(C, C_max));
  const int n_items = total_m * C;
  if (blockIdx.x == 0 && tid == 0) sched[0] = C;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int ring = 0;
      for (int item = blockIdx.x; item < n_items && !s_abort; item += gridDim.x) {
        const NomItem it = nom_item(item, C, prefix, U, unit_info);
        for (int t = it.t0; t < it.t1; ++t, ++ring) {
          const int s = ring & 1;
          if (!mbar_wait(bar_b_empty + 8 * s, ((ring >> 1) & 1) ^ 1)) { s_abort = 1; break; }
          mbar_expect_tx(bar_b_full + 8 * s, SL::kBBytes);
          const uint32_t dst = sbase + SL::kB + s * SL::kBBytes;
          const int row = it.u * p.N_cap + t * kNomN;
#pragma unroll
          for (int sub = 0; sub < SL::kSub; ++sub)
            tma_load_2d(dst + sub * (kNomN * 128), &mapB, sub * 64, row, bar_b_full + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int ring = 0, acc = 0, n_done = 0;
      for (int item = blockIdx.x; item < n_items && !s_abort; item += gridDim.x) {
        const NomItem it = nom_item(item, C, prefix, U, unit_info);
        if (it.t0 == it.t1) continue;
        const int abuf = n_done & 1;
        if (!mbar_wait(bar_a_ready + 8 * abuf, (n_done >> 1) & 1)) { s_abort = 1; break; }
        ++n_done;
        tc_fence_after();
        for (int t = it.t0; t < it.t1; ++t, ++ring, ++acc) {
          const int s = ring & 1, a = acc & 1;
          if (!mbar_wait(bar_b_full + 8 * s, (ring >> 1) & 1) ||
              !mbar_wait(bar_t_empty + 8 * a, ((acc >> 1) & 1) ^ 1)) { s_abort = 1; break; }
          tc_fence_after();
          const uint32_t a_base = sbase + SL::kA + abuf * SL::kABytes, b_base = sbase + SL::kB + s * SL::kBBytes;
#pragma unroll
          for (int k = 0; k < KSTEPS; ++k) {
            const uint64_t ad = umma_desc_sw128(a_base + (k >> 2) * (kNomM * 128) + (k & 3) * 32);
            const uint64_t bd = umma_desc_sw128(b_base + (k >> 2) * (kNomN * 128) + (k & 3) * 32);
            umma_bf16(tmem + a * kNomN, ad, bd, IDESC, k > 0 ? 1u : 0u);
          }
          umma_commit(bar_b_empty + 8 * s);   // the stage may be refilled once these MMAs have read it
          umma_commit(bar_t_full + 8 * a);    // the accumulator is complete
        }
      }
      umma_commit(bar_drain);
      mbar_wait(bar_drain, 0);   // every MMA issued above has retired (bounded)
    }
  } else {
    // ------------------------------------------------------------ A staging + accumulator drain
    const int ew = warp - 2, quarter = warp & 3, cq = ew >> 2;   // cq: which 64 columns of a tile
    const int row = quarter * 32 + lane;                        // tensor-memory lane = row of the item
    float *inv_w = reinterpret_cast<float *>(smem + SL::kInv) + ew * 64;
    float *rowinv = reinterpret_cast<float *>(smem + SL::kRowInv);
    uint32_t *xchg = reinterpret_cast<uint32_t *>(smem + SL::kXchg);
    const size_t n_total = (size_t)U * p.N_cap;
    int acc = 0, n_done = 0;
    bool dead = false, staged = false;
    // Gathers the 128 evicted rows of an item into swizzled A tile `abuf`, sixteen lanes per row (32 rows per round), and
    // leaves the rows' inverse norms in rowinv[abuf].
    auto stage_rows = [&](const NomItem &si, int abuf) {
      constexpr int REPS = kNomM / 32;
      const size_t sbase_u = (size_t)si.u * p.N_cap;
      const int sm0 = si.m_tile * kNomM;
      const int ch = lane & 15, rsub = ew * 2 + (lane >> 4);
      int esrc[REPS];
      uint4 val[REPS];
#pragma unroll
      for (int rep = 0; rep < REPS; ++rep) {
        const int r = rep * 32 + rsub;
        esrc[rep] = (ch < D / 8 && sm0 + r < si.n_ev) ? ev_idx[sbase_u + sm0 + r] : -1;
      }
#pragma unroll
      for (int rep = 0; rep < REPS; ++rep) {
        val[rep] = make_uint4(0, 0, 0, 0);
        if (esrc[rep] >= 0) val[rep] = *reinterpret_cast<const uint4 *>(srcK + (sbase_u + esrc[rep]) * D + ch * 8);
      }
#pragma unroll
      for (int rep = 0; rep < REPS; ++rep) {
        const int r = rep * 32 + rsub;
        float ss = 0.f;
        const uint32_t w[4] = {val[rep].x, val[rep].y, val[rep].z, val[rep].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) { const float a = bf16_lo(w[q]), b = bf16_hi(w[q]); ss = fmaf(a, a, ss); ss = fmaf(b, b, ss); }
        ss += __shfl_xor_sync(0xffffffffu, ss, 1);
        ss += __shfl_xor_sync(0xffffffffu, ss, 2);
        ss += __shfl_xor_sync(0xffffffffu, ss, 4);
        ss += __shfl_xor_sync(0xffffffffu, ss, 8);
        if (ch < D / 8)
          *reinterpret_cast<uint4 *>(smem + SL::kA + abuf * SL::kABytes + (ch >> 3) * (kNomM * 128) + r * 128 +
                                     (((ch & 7) ^ (r & 7)) << 4)) = val[rep];
        if (ch == 0) rowinv[abuf * 128 + r] = rsqrtf(ss);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_a_ready + 8 * abuf);
    };
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
      const NomItem it = nom_item(item, C, prefix, U, unit_info);
      const size_t ubase = (size_t)it.u * p.N_cap;
      const int m0 = it.m_tile * kNomM;
      const int buf = n_done & 1;
      Top2 top, topb;   // two trackers over alternate groups of four columns: two independent dependency chains
      top.init(0.f);
      if (it.t0 == it.t1) {   // a chunk without tiles (fewer tiles than chunks): publish an empty result
        if (cq == 0 && m0 + row < it.n_ev) {
          const size_t o = (ubase + m0 + row) * C_max + it.chunk;
          nom_v[o] = make_float4(top.best, top.second, 0.f, __int_as_float(-1));
          nom_si[o] = -1;
        }
        continue;
      }
      dead = __any_sync(0xffffffffu, dead || s_abort != 0);
      {
        if (!staged) {   // the first item of this CTA; every later one was gathered while its predecessor was drained
          stage_rows(it, buf);
          staged = true;
        }
        // rowinv of this item is visible to every warp, and nobody still reads the other buffer's
        // rowinv (the previous item's results have been published)
        asm volatile("bar.sync 1, 512;" ::: "memory");
        // gather the next item's rows into the other A tile now, so that its MMAs can start while this
        // item is drained (the MMAs that last read that tile belong to the item before this one: retired)
        {
          int nx = item + gridDim.x;
          NomItem nit;
          for (; nx < n_items; nx += gridDim.x) {
            nit = nom_item(nx, C, prefix, U, unit_info);
            if (nit.t0 < nit.t1) break;
          }
          if (nx < n_items) stage_rows(nit, buf ^ 1);
        }
        // values are compared before the division by |k_e|: the closeness margin scales with it
        top.init(2.f * kRankEps / rowinv[buf * 128 + row]);
        topb.init(top.thr);

        for (int t = it.t0; t < it.t1; ++t, ++acc) {
          const int a = acc & 1;
          const int c0 = t * kNomN + cq * 64;
          {
            const size_t g = ubase + c0 + 4 * lane;
            float4 iv = make_float4(0.f, 0.f, 0.f, 0.f);
            if (lane < 16 && g + 3 < n_total) iv = *reinterpret_cast<const float4 *>(inv_norm + g);
            __syncwarp();
            if (lane < 16) *reinterpret_cast<float4 *>(inv_w + 4 * lane) = iv;
            __syncwarp();
          }
          if (!dead) {
            int ok = 1;
            if (lane == 0) ok = mbar_wait(bar_t_full + 8 * a, (acc >> 1) & 1);
            if (!__shfl_sync(0xffffffffu, ok, 0)) { dead = true; s_abort = 1; }
          }
          // nothing to track if this warp's 32 rows lie past the evicted entries or its columns past the
          // retained ones: release the accumulator without reading it
          const bool live = m0 + quarter * 32 < it.n_ev && c0 < it.n_ret;
          if (!dead && !live) {
            tc_fence_before();
            if (lane == 0) mbar_arrive(bar_t_empty + 8 * a);
          }
          if (!dead && live) {
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + a * kNomN + cq * 64;
            const int n_valid = it.n_ret - c0;   // columns of this quarter that exist
            // rows and columns are the same entries (self_mask): the column of the row's own key does not count
            const int diag = self_mask ? m0 + row - c0 : -1;
            const bool crosses = self_mask && m0 + quarter * 32 < c0 + 64 && c0 <= m0 + quarter * 32 + 31;
#pragma unroll 1
            for (int jg = 0; jg < 2; ++jg) {   // 32 columns at a time: the register budget of 18 warps
              uint32_t r0[32];
              tmem_ld_32x32(taddr + jg * 32, r0);
              tmem_ld_wait();
              if (jg == 1) {   // everything this warp needs from the accumulator is in registers
                tc_fence_before();
                if (lane == 0) mbar_arrive(bar_t_empty + 8 * a);
              }
              const int cb = jg * 32;
              const bool ragged = n_valid < cb + 32 || crosses;   // columns past n_ret hold other rows' data
              // `masked` is a compile-time flag: only the last tile of a row of tiles has columns to mask, and a
              // run-time test inside the unrolled loop would be turned into selects that every group pays for
              auto drain32 = [&](auto test, auto masked, const uint32_t (&r)[32], int off) {
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                  float4 iv = *reinterpret_cast<const float4 *>(inv_w + off + i);
                  float a0 = __uint_as_float(r[i]), a1 = __uint_as_float(r[i + 1]);
                  float a2 = __uint_as_float(r[i + 2]), a3 = __uint_as_float(r[i + 3]);
                  if (decltype(masked)::value) {   // a masked column contributes -inf
                    if (off + i >= n_valid || off + i == diag) { a0 = -CUDART_INF_F; iv.x = 1.f; }
                    if (off + i + 1 >= n_valid || off + i + 1 == diag) { a1 = -CUDART_INF_F; iv.y = 1.f; }
                    if (off + i + 2 >= n_valid || off + i + 2 == diag) { a2 = -CUDART_INF_F; iv.z = 1.f; }
                    if (off + i + 3 >= n_valid || off + i + 3 == diag) { a3 = -CUDART_INF_F; iv.w = 1.f; }
                  }
                  offer4<decltype(test)::value>(top, topb, a0, a1, a2, a3, iv, c0 + off + i);
                }
              };
              const bool cold = t == it.t0;   // cold lists: insert everything
              if (cold && ragged) {
                drain32(std::false_type{}, std::true_type{}, r0, cb);
              } else if (cold) {
                drain32(std::false_type{}, std::false_type{}, r0, cb);
              } else if (ragged) {
                drain32(std::true_type{}, std::true_type{}, r0, cb);
              } else {
                drain32(std::true_type{}, std::false_type{}, r0, cb);
              }
              if (cold && jg == 1) top.cut = fmaxf(top.best, topb.best) - top.thr;
            }
          }
        }
        ++n_done;
      }
      top.insert_any(topb.best, topb.bi);
      top.insert_any(topb.second, topb.si);
      // ---- combine the two column halves of each row and publish the chunk's result
      uint32_t *x = xchg + (size_t)(buf * 128 + row) * 9;
      if (cq > 0) {   // slots are below 65535 (N_cap <= 49152); -1 = none
        uint32_t *xw = x + (cq - 1) * 3;
        xw[0] = __float_as_uint(top.best);
        xw[1] = __float_as_uint(top.second);
        xw[2] = (uint32_t)(top.bi + 1) | ((uint32_t)(top.si + 1) << 16);
      }
      asm volatile("bar.sync 1, 512;" ::: "memory");
      if (cq == 0) {
#pragma unroll
        for (int w = 0; w < 3; ++w) {   // ascending columns: a later quarter holds higher slots, ties keep the earlier one
          const uint32_t *xw = x + w * 3;
          const uint32_t sl = xw[2];
          top.insert(__uint_as_float(xw[0]), (int)(sl & 0xffffu) - 1);
          top.insert(__uint_as_float(xw[1]), (int)(sl >> 16) - 1);
        }
        if (m0 + row < it.n_ev) {
          const float ri = rowinv[buf * 128 + row];
          const size_t o = (ubase + m0 + row) * C_max + it.chunk;
          nom_v[o] = make_float4(top.best * ri, top.second * ri, 0.f, __int_as_float(top.bi));
          nom_si[o] = top.si;
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (s_abort) {
    if (tid == 0) {
      atomicOr(status_dev, KEEPKV_DEV_TIMEOUT);
      // copies still in flight get a bounded chance to land before the shared memory goes away
      for (int i = 0; i < 2; ++i) { mbar_wait(bar_b_full + 8 * i, 0); mbar_wait(bar_b_full + 8 * i, 1); }
    }
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

template <int D>
static void launch_nominate_t(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                              const int32_t *ev_idx, const UnitInfo *unit_info, const float *inv_norm, int32_t *sched,
                              float4 *nom_v, int32_t *nom_si, int nom_chunks, int32_t *status_dev, LaunchCtx &ctx,
                              int self_mask) {
  using SL = NomSmem<D>;
  constexpr size_t smem_bytes = (size_t)SL::kBytes + 1024;
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(nominate_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    attr_done_dev[dev & 63] = true;
  }
  CUtensorMap mapB;
  if (!make_bf16_rows_map(&mapB, dst.K, (uint64_t)p.B * p.H_kv * p.N_cap, D, kNomN)) {
    if (ctx.err == cudaSuccess) ctx.err = cudaErrorInvalidValue;
    return;
  }
  launch_pdl(nominate_kernel<D>, dim3(sm_count()), dim3(kNomThreads), smem_bytes, ctx.stream,
      mapB, p, reinterpret_cast<const __nv_bfloat16 *>(src.K), ev_idx, unit_info, inv_norm, sched, nom_v, nom_si,
      nom_chunks, status_dev, self_mask);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_nominate(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst, const int32_t *ev_idx,
                     const UnitInfo *unit_info, const float *inv_norm, int32_t *sched, float4 *nom_v, int32_t *nom_si,
                     int nom_chunks, int32_t *status_dev, LaunchCtx &ctx, int self_mask) {
  if (p.d == 128)
    launch_nominate_t<128>(p, src, dst, ev_idx, unit_info, inv_norm, sched, nom_v, nom_si, nom_chunks, status_dev, ctx, self_mask);
  else
    launch_nominate_t<64>(p, src, dst, ev_idx, unit_info, inv_norm, sched, nom_v, nom_si, nom_chunks, status_dev, ctx, self_mask);
}

}  // namespace keepkv
