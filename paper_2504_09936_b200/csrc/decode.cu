// keepkv_decode_attention: Electoral-Votes attention (Eq. 6) over the cache, split along the
// entry axis (split-KV), with the per-entry score estimate of Eq. 8 advanced in the same pass.
//
// One CTA = 4 warps works through a contiguous range of 64-entry tiles of one (sequence, kv-head)
// unit.  K/V tiles arrive by TMA (128-byte swizzled boxes) into a 3-stage shared-memory ring,
// votes and lscore of the tile by bulk copies on the same mbarrier.  Each warp owns 16 entries
// of a tile: the G query heads of the unit are the rows of an m16n8k16 bf16 MMA (rows >= G are
// zero), so K is read once for all heads; logits come out in fp32, the vote weight enters as
// + ln p_i before the online softmax (p_i e^{l_i} = e^{l_i + ln p_i}), and the probabilities go
// back into the tensor core split into a bf16 head (A rows 0-7) and a bf16 remainder (A rows
// 8-15) so that P.V keeps fp32-level accuracy in one MMA.
#include <cuda.h>

#include "common.cuh"

namespace keepkv {

constexpr int kDecWarps = 4;
constexpr int kStages = 3;
constexpr int kSpinLimit = 1 << 20;

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (each poll itself blocks for a short hardware interval).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Split s of a unit covers tiles [t0, t1).
__device__ __forceinline__ void split_tiles(int len, int S, int s, int &t0, int &t1) {
  const int tiles = (len + kTile - 1) / kTile;
  const int per = (tiles + S - 1) / S;
  t0 = min(tiles, s * per);
  t1 = min(tiles, t0 + per);
}

// Shared-memory layout of one stage: K tile, V tile (each D/64 swizzled sub-tiles of 64 rows x 128 B),
// then the tile's votes and lscore.
template <int D>
struct StageLayout {
  static constexpr int kSub = D / 64;
  static constexpr int kSubBytes = kTile * 128;
  static constexpr int kK = 0;
  static constexpr int kV = kSub * kSubBytes;
  static constexpr int kVotes = 2 * kSub * kSubBytes;
  static constexpr int kLscore = kVotes + kTile * 4;
  static constexpr int kBytes = kLscore + kTile * 4;                 // what one stage receives
  static constexpr int kStride = (kBytes + 1023) / 1024 * 1024;      // sub-tiles need 1024-byte alignment
};

// Byte offset of 16-byte chunk `chunk` (0..D/8-1) of tile row `row` inside a swizzled K or V tile.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * (kTile * 128) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// Merge the S partial results of a unit: o = sum_s e^{m_s - M} acc_s / sum_s e^{m_s - M} l_s.
template <int D, int G>
__device__ void combine_splits(const keepkv_params &p, int u, int S, const float *part_ml, const float *part_acc,
                               __nv_bfloat16 *out, float *lse) {
  const int b = u / p.H_kv, h = u % p.H_kv;
  for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
    const int g = idx / D, j = idx % D;
    float M = -CUDART_INF_F;
    for (int s = 0; s < S; ++s) M = fmaxf(M, part_ml[(((size_t)u * S + s) * G + g) * 2]);
    float Lsum = 0.f, acc = 0.f;
    if (M > -CUDART_INF_F) {
      for (int s = 0; s < S; ++s) {
        const size_t o = ((size_t)u * S + s) * G + g;
        const float w = __expf(part_ml[o * 2] - M);
        Lsum += w * part_ml[o * 2 + 1];
        acc += w * part_acc[o * D + j];
      }
    }
    const size_t qo = ((size_t)b * p.H_q + h * G + g);
    out[qo * D + j] = __float2bfloat16_rn(Lsum > 0.f ? acc / Lsum : 0.f);
    if (lse && j == 0) lse[qo] = Lsum > 0.f ? M + logf(Lsum) : -CUDART_INF_F;
  }
}

template <int D, int G>
__global__ void __launch_bounds__(kDecWarps * 32, 2)
decode_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV, keepkv_params p,
              keepkv_cache c, const __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ out,
              float *__restrict__ lse, int update_scores, int *counters, float *part_ml, float *part_acc,
              int32_t *status_dev) {
  using SL = StageLayout<D>;
  constexpr int KS = D / 16;   // k-steps of the QK^T product
  constexpr int NT = D / 8;    // 8-channel n-tiles of the PV product
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[kStages];
  __shared__ int s_abort, s_last;

  // dynamic shared memory is only guaranteed 16-byte aligned: round up to the swizzle atom
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t smem_base = smem_u32(smem);

  const int u = blockIdx.y, s = blockIdx.x, S = gridDim.x;
  const int b = u / p.H_kv, h = u % p.H_kv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, qd = lane & 3;   // MMA row (query head) and position inside the quad
  const int len = max(0, min(c.seq_len[b], p.N_cap));
  int t0, t1;
  split_tiles(len, S, s, t0, t1);
  const int ntiles = t1 - t0;
  const size_t ubase = (size_t)u * p.N_cap;

  if (tid == 0) {
    for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(&full_bar[i]), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  auto issue = [&](int stage, int tile) {
    const uint32_t bar = smem_u32(&full_bar[stage]);
    const uint32_t dst = smem_base + stage * SL::kStride;
    const int row = (int)(ubase) + tile * kTile;
    mbar_expect_tx(bar, SL::kBytes);
#pragma unroll
    for (int sub = 0; sub < SL::kSub; ++sub) {
      tma_load_2d(dst + SL::kK + sub * SL::kSubBytes, &mapK, sub * 64, row, bar);
      tma_load_2d(dst + SL::kV + sub * SL::kSubBytes, &mapV, sub * 64, row, bar);
    }
    bulk_load_1d(dst + SL::kVotes, c.votes + ubase + (size_t)tile * kTile, kTile * 4, bar);
    bulk_load_1d(dst + SL::kLscore, c.lscore + ubase + (size_t)tile * kTile, kTile * 4, bar);
  };
  if (tid == 0) {
    for (int i = 0; i < kStages && i < ntiles; ++i) issue(i, t0 + i);
  }

  // Q fragments (A operand of QK^T): row g = query head, rows >= G and rows 8-15 are zero.
  uint32_t qa[KS][2];
  {
    const __nv_bfloat16 *qrow = q + ((size_t)b * p.H_q + h * G + (g < G ? g : 0)) * D;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = g < G ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + qd * 2) : 0u;
      qa[ks][1] = g < G ? *reinterpret_cast<const uint32_t *>(qrow + ks * 16 + 8 + qd * 2) : 0u;
    }
  }
  const float ln_alpha = p.ema_alpha > 0.f ? __logf(p.ema_alpha) : -CUDART_INF_F;
  const float ln_1ma = log1pf(-p.ema_alpha);
  const float ln_G = __logf((float)G);
  float *lscore_g = c.lscore + ubase;

  float o[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
  float m_run = -CUDART_INF_F, l_run = 0.f;   // running max and (per-thread partial) sum of head g

  const int r0 = warp * 16;                   // this warp's rows inside a tile
  for (int it = 0; it < ntiles; ++it) {
    const int stage = it % kStages;
    const uint32_t parity = (it / kStages) & 1;
    if (!mbar_wait(smem_u32(&full_bar[stage]), parity)) {
      s_abort = 1;
      atomicOr(status_dev, KEEPKV_DEV_TIMEOUT);
    }
    const uint32_t st = smem_base + stage * SL::kStride;
    const uint8_t *stp = smem + stage * SL::kStride;
    const int i_base = (t0 + it) * kTile + r0;    // first entry of this warp's slice
    const int n_valid = len - i_base;              // entries of the slice that exist (may be <= 0 or >= 16)

    if (n_valid < 16) {
      // ragged tail: rows past the sequence hold unspecified bits; zero their V so that 0 * garbage
      // cannot turn into NaN inside the tensor core
      for (int idx = lane; idx < 16 * (D / 8); idx += 32) {
        const int r = idx / (D / 8), ch = idx % (D / 8);
        if (r >= n_valid) *reinterpret_cast<uint4 *>(smem + stage * SL::kStride + SL::kV + swz(r0 + r, ch)) = make_uint4(0, 0, 0, 0);
      }
      __syncwarp();
    }

    // ---- logits: S[head][entry] for the 16 entries, two n-tiles of 8
    float sc[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.f;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int row = r0 + j * 8 + (lane & 7);
#pragma unroll
      for (int kk = 0; kk < KS / 2; ++kk) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(st + SL::kK + swz(row, kk * 4 + (lane >> 3)), b0, b1, b2, b3);
        mma_bf16(sc[j], qa[2 * kk][0], 0u, qa[2 * kk][1], 0u, b0, b1);
        mma_bf16(sc[j], qa[2 * kk + 1][0], 0u, qa[2 * kk + 1][1], 0u, b2, b3);
      }
    }
    // this thread holds head g, entries e(j,t) = i_base + 8 j + 2 qd + t
    float x[2][2];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int t = 0; t < 2; ++t) x[j][t] = sc[j][t] * p.sm_scale;

    // ---- Eq. 8: score of the kv head = mean over its G heads of e^{l}; kept as a logarithm
    if (update_scores) {
      const float *ls_s = reinterpret_cast<const float *>(stp + SL::kLscore) + r0;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float sig[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          const float v = g < G ? x[j][t] : -CUDART_INF_F;
          float mx = v;
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          float se = __expf(v - mx);
          se += __shfl_xor_sync(0xffffffffu, se, 4);
          se += __shfl_xor_sync(0xffffffffu, se, 8);
          se += __shfl_xor_sync(0xffffffffu, se, 16);
          sig[t] = mx + __logf(se) - ln_G;
        }
        if (g == 0) {
          const int e = j * 8 + qd * 2;
          float r[2];
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const float old = ls_s[e + t];
            r[t] = sig[t];
            if (old > -CUDART_INF_F && p.ema_alpha > 0.f) {
              const float a = ln_alpha + old, bb = ln_1ma + sig[t];
              const float mm = fmaxf(a, bb);
              r[t] = mm + __logf(__expf(a - mm) + __expf(bb - mm));
            }
          }
          if (e + 1 < n_valid)
            *reinterpret_cast<float2 *>(lscore_g + i_base + e) = make_float2(r[0], r[1]);
          else if (e < n_valid)
            lscore_g[i_base + e] = r[0];
        }
      }
    }

    // ---- Eq. 6: weights p_i e^{l_i} through an online softmax over x + ln p
    const float *vt_s = reinterpret_cast<const float *>(stp + SL::kVotes) + r0;
    float mloc = -CUDART_INF_F;
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int e = j * 8 + qd * 2 + t;
        x[j][t] = e < n_valid ? x[j][t] + __logf(vt_s[e]) : -CUDART_INF_F;
        mloc = fmaxf(mloc, x[j][t]);
      }
    mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, 1));
    mloc = fmaxf(mloc, __shfl_xor_sync(0xffffffffu, mloc, 2));
    const float m_new = fmaxf(m_run, mloc);
    const bool grow = m_new > m_run;
    if (__any_sync(0xffffffffu, grow)) {
      const float scale = grow ? __expf(m_run - m_new) : 1.f;   // m_run = -inf gives 0, o and l are 0 then anyway
      l_run *= scale;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        o[nt][0] *= scale; o[nt][1] *= scale; o[nt][2] *= scale; o[nt][3] *= scale;
      }
      m_run = m_new;
    }
    uint32_t pa[4];   // A fragment of P: a0/a2 = bf16 head (rows 0-7), a1/a3 = bf16 remainder (rows 8-15)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float pr[2], hi[2];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        pr[t] = m_run > -CUDART_INF_F ? __expf(x[j][t] - m_run) : 0.f;
        l_run += pr[t];
        hi[t] = __bfloat162float(__float2bfloat16_rn(pr[t]));
      }
      pa[2 * j] = pack_bf16(hi[0], hi[1]);
      pa[2 * j + 1] = pack_bf16(pr[0] - hi[0], pr[1] - hi[1]);
    }
    // ---- O += P V   (rows 0-7 collect the head part, rows 8-15 the remainder part)
    {
      const int vrow = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(st + SL::kV + swz(vrow, np * 2 + (lane >> 4)), b0, b1, b2, b3);
        mma_bf16(o[2 * np], pa[0], pa[1], pa[2], pa[3], b0, b1);
        mma_bf16(o[2 * np + 1], pa[0], pa[1], pa[2], pa[3], b2, b3);
      }
    }
    __syncthreads();   // every warp is done with this stage
    if (s_abort) break;
    if (tid == 0 && it + kStages < ntiles) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      issue(stage, t0 + it + kStages);
    }
  }
  if (s_abort) {
    // give copies still in flight a bounded chance to land before the CTA's shared memory goes away
    __syncthreads();
    if (tid == 0)
      for (int i = 0; i < kStages; ++i) { mbar_wait(smem_u32(&full_bar[i]), 0); mbar_wait(smem_u32(&full_bar[i]), 1); }
    __syncthreads();
  }

  // ---- combine the four warps of this CTA (stage memory is free now)
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  float *cm = reinterpret_cast<float *>(smem);            // [warps][8]
  float *cl = cm + kDecWarps * 8;                          // [warps][8]
  float *co = cl + kDecWarps * 8;                          // [warps][G][D]
  if (g < G) {
    if (qd == 0) { cm[warp * 8 + g] = m_run; cl[warp * 8 + g] = l_run; }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float2 v = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
      *reinterpret_cast<float2 *>(&co[((size_t)warp * G + g) * D + nt * 8 + qd * 2]) = v;
    }
  }
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += blockDim.x) {
    const int gg = idx / D, j = idx % D;
    float M = cm[gg];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) M = fmaxf(M, cm[w * 8 + gg]);
    float Ls = 0.f, a = 0.f;
    if (M > -CUDART_INF_F) {
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) {
        const float f = __expf(cm[w * 8 + gg] - M);
        Ls += f * cl[w * 8 + gg];
        a += f * co[((size_t)w * G + gg) * D + j];
      }
    }
    const size_t oo = ((size_t)u * S + s) * G + gg;
    part_acc[oo * D + j] = a;
    if (j == 0) { part_ml[oo * 2] = M; part_ml[oo * 2 + 1] = Ls; }
  }
  // ---- the last CTA of the unit to arrive merges the partials
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&counters[u], 1);
    s_last = (ticket == S - 1);
    if (s_last) counters[u] = 0;   // ready for the next call
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    combine_splits<D, G>(p, u, S, part_ml, part_acc, out, lse);
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Tensor map over a [rows, D] bf16 matrix with boxes of 64 rows x 64 channels, 128-byte swizzle;
// rows past the end read as zero.
static bool make_map(CUtensorMap *map, void *base, uint64_t rows, int D) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)D * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)kTile};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int G>
static void launch_t(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                     int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx) {
  using SL = StageLayout<D>;
  constexpr size_t smem_bytes = (size_t)kStages * SL::kStride + 1024;
  static bool attr_done_dev[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done_dev[dev & 63]) {
    cudaFuncSetAttribute(decode_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
    attr_done_dev[dev & 63] = true;
  }
  CUtensorMap mapK, mapV;
  const uint64_t rows = (uint64_t)p.B * p.H_kv * p.N_cap;
  if (!make_map(&mapK, c.K, rows, D) || !make_map(&mapV, c.V, rows, D)) {
    if (ctx.err == cudaSuccess) ctx.err = cudaErrorInvalidValue;
    return;
  }
  const int S = choose_splits(p, L.max_splits);
  dim3 grid(S, p.B * p.H_kv);
  decode_kernel<D, G><<<grid, kDecWarps * 32, smem_bytes, ctx.stream>>>(
      mapK, mapV, p, c, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out), lse,
      update_scores, reinterpret_cast<int *>(ws + L.counters), reinterpret_cast<float *>(ws + L.part_ml),
      reinterpret_cast<float *>(ws + L.part_acc), status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_decode(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                   int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx) {
  const int G = p.H_q / p.H_kv;
#define KEEPKV_DISPATCH(DD, GG) \
  if (p.d == DD && G == GG) return launch_t<DD, GG>(p, c, q, out, lse, update_scores, ws, L, status_dev, ctx);
  KEEPKV_DISPATCH(128, 1) KEEPKV_DISPATCH(128, 2) KEEPKV_DISPATCH(128, 4) KEEPKV_DISPATCH(128, 8)
  KEEPKV_DISPATCH(64, 1) KEEPKV_DISPATCH(64, 2) KEEPKV_DISPATCH(64, 4) KEEPKV_DISPATCH(64, 8)
#undef KEEPKV_DISPATCH
}

}  // namespace keepkv
