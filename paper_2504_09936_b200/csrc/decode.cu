// keepkv_decode_attention: Electoral-Votes attention (Eq. 6) over the cache, split along the
// entry axis, with the per-entry score estimate of Eq. 8 advanced in the same pass.
#include "common.cuh"

namespace keepkv {

constexpr int kDecWarps = 4;

// Split s of unit u covers tiles [t0, t1) of kTile entries.
__device__ __forceinline__ void split_range(int len, int S, int s, int &i0, int &i1) {
  const int tiles = (len + kTile - 1) / kTile;
  const int per = (tiles + S - 1) / S;
  const int t0 = min(tiles, s * per), t1 = min(tiles, t0 + per);
  i0 = t0 * kTile;
  i1 = min(len, t1 * kTile);
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

// grid (S, U).  Each warp walks entries i0+w, i0+w+4, ...; the 32 lanes split the d channels.
template <int D, int G>
__global__ void __launch_bounds__(kDecWarps * 32)
decode_kernel(keepkv_params p, keepkv_cache c, const __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ out,
              float *__restrict__ lse, int update_scores, int *counters, float *part_ml, float *part_acc) {
  constexpr int EPL = D / 32;  // channels per lane
  const int u = blockIdx.y, s = blockIdx.x, S = gridDim.x;
  const int b = u / p.H_kv, h = u % p.H_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int len = min(c.seq_len[b], p.N_cap);
  int i0, i1;
  split_range(len, S, s, i0, i1);

  float qf[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      qf[g][e] = __bfloat162float(q[((size_t)b * p.H_q + h * G + g) * D + lane * EPL + e]);

  const __nv_bfloat16 *K = reinterpret_cast<const __nv_bfloat16 *>(c.K) + (size_t)u * p.N_cap * D;
  const __nv_bfloat16 *V = reinterpret_cast<const __nv_bfloat16 *>(c.V) + (size_t)u * p.N_cap * D;
  const float *votes = c.votes + (size_t)u * p.N_cap;
  float *lscore = c.lscore + (size_t)u * p.N_cap;
  const float ln_alpha = p.ema_alpha > 0.f ? logf(p.ema_alpha) : -CUDART_INF_F;
  const float ln_1ma = log1pf(-p.ema_alpha);
  const float ln_G = logf((float)G);

  float m[G], l[G], acc[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -CUDART_INF_F;
    l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
  }

  for (int i = i0 + warp; i < i1; i += kDecWarps) {
    float kf[EPL], vf[EPL];
    if constexpr (EPL == 4) {
      const uint2 kk = *reinterpret_cast<const uint2 *>(K + (size_t)i * D + lane * 4);
      const uint2 vv = *reinterpret_cast<const uint2 *>(V + (size_t)i * D + lane * 4);
      kf[0] = bf16_lo(kk.x); kf[1] = bf16_hi(kk.x); kf[2] = bf16_lo(kk.y); kf[3] = bf16_hi(kk.y);
      vf[0] = bf16_lo(vv.x); vf[1] = bf16_hi(vv.x); vf[2] = bf16_lo(vv.y); vf[3] = bf16_hi(vv.y);
    } else {
      const uint32_t kk = *reinterpret_cast<const uint32_t *>(K + (size_t)i * D + lane * 2);
      const uint32_t vv = *reinterpret_cast<const uint32_t *>(V + (size_t)i * D + lane * 2);
      kf[0] = bf16_lo(kk); kf[1] = bf16_hi(kk);
      vf[0] = bf16_lo(vv); vf[1] = bf16_hi(vv);
    }
    const float lnp = __logf(votes[i]);
    float x[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float dsum = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) dsum = fmaf(qf[g][e], kf[e], dsum);
      x[g] = warp_sum(dsum) * p.sm_scale;  // logit l_{g,i}
    }
    if (update_scores && lane == 0) {
      float mx = x[0];
#pragma unroll
      for (int g = 1; g < G; ++g) mx = fmaxf(mx, x[g]);
      float se = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) se += __expf(x[g] - mx);
      const float sigma = mx + logf(se) - ln_G;  // ln of the group-mean score
      const float old = lscore[i];
      float r = sigma;
      if (old > -CUDART_INF_F && p.ema_alpha > 0.f) {
        const float a = ln_alpha + old, bb = ln_1ma + sigma;
        const float mm = fmaxf(a, bb);
        r = mm + logf(__expf(a - mm) + __expf(bb - mm));
      }
      lscore[i] = r;
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float xv = x[g] + lnp;  // ln(p_i s_i)
      const float mn = fmaxf(m[g], xv);
      const float sc = __expf(m[g] - mn), w = __expf(xv - mn);
      l[g] = l[g] * sc + w;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(acc[g][e], sc, w * vf[e]);
      m[g] = mn;
    }
  }

  // combine the four warps of this CTA
  __shared__ float sm_m[kDecWarps][G], sm_l[kDecWarps][G], sm_acc[kDecWarps][G][D];
  __shared__ int sm_last;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    if (lane == 0) { sm_m[warp][g] = m[g]; sm_l[warp][g] = l[g]; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_acc[warp][g][lane * EPL + e] = acc[g][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
    const int g = idx / D, j = idx % D;
    float M = sm_m[0][g];
#pragma unroll
    for (int w = 1; w < kDecWarps; ++w) M = fmaxf(M, sm_m[w][g]);
    float Ls = 0.f, a = 0.f;
    if (M > -CUDART_INF_F) {
#pragma unroll
      for (int w = 0; w < kDecWarps; ++w) {
        const float f = __expf(sm_m[w][g] - M);
        Ls += f * sm_l[w][g];
        a += f * sm_acc[w][g][j];
      }
    }
    const size_t o = ((size_t)u * S + s) * G + g;
    part_acc[o * D + j] = a;
    if (j == 0) { part_ml[o * 2] = M; part_ml[o * 2 + 1] = Ls; }
  }
  // the last CTA of the unit to arrive merges the partials
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int ticket = atomicAdd(&counters[u], 1);
    sm_last = (ticket == S - 1);
    if (sm_last) counters[u] = 0;  // ready for the next call
  }
  __syncthreads();
  if (sm_last) {
    __threadfence();
    combine_splits<D, G>(p, u, S, part_ml, part_acc, out, lse);
  }
}

template <int D, int G>
static void launch_t(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                     int update_scores, char *ws, const WsLayout &L, LaunchCtx &ctx) {
  const int S = choose_splits(p, L.max_splits);
  dim3 grid(S, p.B * p.H_kv);
  decode_kernel<D, G><<<grid, kDecWarps * 32, 0, ctx.stream>>>(
      p, c, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out), lse, update_scores,
      reinterpret_cast<int *>(ws + L.counters), reinterpret_cast<float *>(ws + L.part_ml),
      reinterpret_cast<float *>(ws + L.part_acc));
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_decode(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                   int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx) {
  (void)status_dev;
  const int G = p.H_q / p.H_kv;
#define KEEPKV_DISPATCH(DD, GG) \
  if (p.d == DD && G == GG) return launch_t<DD, GG>(p, c, q, out, lse, update_scores, ws, L, ctx);
  KEEPKV_DISPATCH(128, 1) KEEPKV_DISPATCH(128, 2) KEEPKV_DISPATCH(128, 4) KEEPKV_DISPATCH(128, 8)
  KEEPKV_DISPATCH(64, 1) KEEPKV_DISPATCH(64, 2) KEEPKV_DISPATCH(64, 4) KEEPKV_DISPATCH(64, 8)
#undef KEEPKV_DISPATCH
}

}  // namespace keepkv
