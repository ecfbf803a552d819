// C ABI of libkeepkv: argument validation, workspace layout, and dispatch to the kernels.
#include <math.h>
#include <string.h>

#include "common.cuh"

namespace keepkv {

static thread_local int g_last_cuda_error = 0;
static thread_local int g_last_launches = 0;

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WsLayout ws_layout(const keepkv_params &p) {
  WsLayout L;
  const size_t U = (size_t)p.B * p.H_kv, N = (size_t)p.N_cap, G = (size_t)(p.H_q / p.H_kv);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.counters = take((U + 1) * 4);
  L.part_pool = take((size_t)kDecMaxCtas * 2 * (16 + G * (size_t)p.d) * 4);
  L.decode_bytes = off;
  L.counter_bytes = (U + 1) * 4;
  L.unit_info = take(U * sizeof(UnitInfo));
  L.sched = take(4 * 4);
  size_t C = (2 * 148 + U - 1) / U;
  if (C < 1) C = 1;
  if (C > (size_t)kNomChunksMax) C = kNomChunksMax;
  L.nom_chunks = (int)C;
  size_t Np2 = 1;
  while (Np2 < N) Np2 <<= 1;
  L.key_stride = (int)Np2;
  L.ret_idx = take(U * N * 4);
  L.target = take(U * N * 4);
  L.ev_idx = take(U * N * 4);
  L.inv_norm = take(U * N * 4);
  L.nom_v = take(U * N * C * 16);
  L.nom_si = take(U * N * C * 4);
  L.grp_key = take(U * Np2 * 4);
  L.grp_head = take(U * N * 4);
  L.stats = take(U * sizeof(keepkv_stats));
  L.stats2 = take(U * sizeof(keepkv_stats));
  L.unit_len = take(U * 4);
  L.eff_budget = take((size_t)p.B * 4);
  L.kept = take(U * N * 4);
  L.total = off;
  return L;
}

static int validate(const keepkv_params *p) {
  if (!p) return KEEPKV_ERR_INVALID_ARG;
  if (p->B <= 0 || p->H_q <= 0 || p->H_kv <= 0 || p->N_cap <= 0) return KEEPKV_ERR_INVALID_ARG;
  if ((p->flags & ~(KEEPKV_FLAG_COMPRESS_STEADY | KEEPKV_FLAG_CACHE_IDLE)) || p->reserved[0] || p->reserved[1]) return KEEPKV_ERR_INVALID_ARG;
  if (p->H_q % p->H_kv) return KEEPKV_ERR_UNSUPPORTED;
  const int G = p->H_q / p->H_kv;
  if (!(G == 1 || G == 2 || G == 4 || G == 8)) return KEEPKV_ERR_UNSUPPORTED;
  if (!(p->d == 64 || p->d == 128)) return KEEPKV_ERR_UNSUPPORTED;
  if (p->N_cap % 64) return KEEPKV_ERR_UNSUPPORTED;
  if (p->N_cap > 49152) return KEEPKV_ERR_UNSUPPORTED;  // selection keeps one key per entry in shared memory
  if (p->n_sink < 0 || p->n_recent < 0 || p->period < 0) return KEEPKV_ERR_INVALID_ARG;
  if (!(p->ema_alpha >= 0.0f && p->ema_alpha < 1.0f)) return KEEPKV_ERR_INVALID_ARG;
  if (!(p->sm_scale > 0.0f) || isnan(p->merge_threshold) || isnan(p->gamma_min) || isnan(p->gamma_max))
    return KEEPKV_ERR_INVALID_ARG;
  return KEEPKV_OK;
}

static bool aligned(const void *ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) == 0; }

int sm_count() {
  static int n[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  dev &= 63;
  if (!n[dev]) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    n[dev] = v;
  }
  return n[dev];
}

static int validate_cache(const keepkv_cache *c) {
  if (!c || !c->K || !c->V || !c->votes || !c->lscore || !c->seq_len) return KEEPKV_ERR_INVALID_ARG;
  if (!aligned(c->K, 16) || !aligned(c->V, 16) || !aligned(c->votes, 16) || !aligned(c->lscore, 16))
    return KEEPKV_ERR_INVALID_ARG;
  return KEEPKV_OK;
}

static int finish(LaunchCtx &ctx) {
  g_last_launches = ctx.launches;
  if (ctx.err != cudaSuccess) {
    g_last_cuda_error = (int)ctx.err;
    return KEEPKV_ERR_CUDA;
  }
  return KEEPKV_OK;
}

int finish_call(LaunchCtx &ctx) { return finish(ctx); }

}  // namespace keepkv

using namespace keepkv;

extern "C" {

int keepkv_workspace_bytes(const keepkv_params *p, size_t *bytes) {
  int rc = validate(p);
  if (rc) return rc;
  if (!bytes) return KEEPKV_ERR_INVALID_ARG;
  *bytes = ws_layout(*p).total;
  return KEEPKV_OK;
}

int keepkv_workspace_init(const keepkv_params *p, void *ws, size_t ws_bytes, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if (!ws || !aligned(ws, 256)) return KEEPKV_ERR_INVALID_ARG;
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  ctx.err = cudaMemsetAsync((char *)ws + L.counters, 0, L.counter_bytes, ctx.stream);
  return finish(ctx);
}

int keepkv_append(const keepkv_params *p, const keepkv_cache *cache, const void *k_new, const void *v_new,
                  int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!k_new || !v_new || !status_dev || !aligned(k_new, 16) || !aligned(v_new, 16)) return KEEPKV_ERR_INVALID_ARG;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  launch_append(*p, *cache, k_new, v_new, status_dev, ctx);
  return finish(ctx);
}

int keepkv_decode_attention(const keepkv_params *p, const keepkv_cache *cache, const void *q, void *out,
                            float *lse_or_null, int update_scores, void *ws, size_t ws_bytes, int32_t *status_dev,
                            void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!q || !out || !ws || !status_dev || !aligned(q, 16) || !aligned(out, 16) || !aligned(ws, 256))
    return KEEPKV_ERR_INVALID_ARG;
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  launch_decode(*p, *cache, q, out, lse_or_null, update_scores, (char *)ws, L, status_dev, ctx);
  return finish(ctx);
}

int keepkv_decode_step(const keepkv_params *p, const keepkv_cache *cache, const void *q, const void *k_new,
                       const void *v_new, void *out, float *lse_or_null, int update_scores, void *ws, size_t ws_bytes,
                       int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!q || !k_new || !v_new || !out || !ws || !status_dev || !aligned(q, 16) || !aligned(k_new, 16) ||
      !aligned(v_new, 16) || !aligned(out, 16) || !aligned(ws, 256))
    return KEEPKV_ERR_INVALID_ARG;
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  launch_decode(*p, *cache, q, out, lse_or_null, update_scores, (char *)ws, L, status_dev, ctx, k_new, v_new);
  return finish(ctx);
}

int keepkv_prefill_scores(const keepkv_params *p, const keepkv_cache *cache, const void *q_window, int32_t W,
                          int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!q_window || !status_dev || !aligned(q_window, 16)) return KEEPKV_ERR_INVALID_ARG;
  if (W < 1) return KEEPKV_ERR_INVALID_ARG;
  if (W > 32) return KEEPKV_ERR_UNSUPPORTED;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  launch_prefill_scores(*p, *cache, q_window, W, status_dev, ctx);
  return finish(ctx);
}

int keepkv_compress(const keepkv_params *p, const keepkv_cache *src, const keepkv_cache *dst,
                    const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                    int32_t *retained_idx_or_null, int32_t *target_or_null, keepkv_stats *stats_or_null, void *ws,
                    size_t ws_bytes, int32_t *status_dev, void *stream) {
  return keepkv_compress_scored(p, src, dst, nullptr, budget_dev, budget_scalar, n_recent_dev, retained_idx_or_null,
                                target_or_null, stats_or_null, ws, ws_bytes, status_dev, stream);
}

int keepkv_compress_scored(const keepkv_params *p, const keepkv_cache *src, const keepkv_cache *dst,
                           const float *select_score_or_null, const int32_t *budget_dev, int32_t budget_scalar,
                           const int32_t *n_recent_dev, int32_t *retained_idx_or_null, int32_t *target_or_null,
                           keepkv_stats *stats_or_null, void *ws, size_t ws_bytes, int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(src))) return rc;
  if ((rc = validate_cache(dst))) return rc;
  if (src->K == dst->K || src->V == dst->V || src->votes == dst->votes || src->lscore == dst->lscore ||
      src->seq_len == dst->seq_len)
    return KEEPKV_ERR_INVALID_ARG;
  if (!ws || !status_dev || !aligned(ws, 256)) return KEEPKV_ERR_INVALID_ARG;
  if ((long long)p->B * p->H_kv > kMaxUnits) return KEEPKV_ERR_UNSUPPORTED;
  if (!budget_dev) {
    if (budget_scalar < 0) return KEEPKV_ERR_INVALID_ARG;
    if ((p->flags & KEEPKV_FLAG_COMPRESS_STEADY) && budget_scalar == 0) return KEEPKV_ERR_INVALID_ARG;
    if (budget_scalar > p->N_cap || (long long)budget_scalar + p->period > p->N_cap) return KEEPKV_ERR_CAPACITY;
  }
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  char *w = (char *)ws;
  launch_compress(*p, *src, *dst, budget_dev, budget_scalar, n_recent_dev,
                  retained_idx_or_null ? retained_idx_or_null : (int32_t *)(w + L.ret_idx),
                  target_or_null ? target_or_null : (int32_t *)(w + L.target),
                  stats_or_null ? stats_or_null : (keepkv_stats *)(w + L.stats), w, L, status_dev, ctx,
                  select_score_or_null);
  return finish(ctx);
}

int keepkv_compress_inplace(const keepkv_params *p, const keepkv_cache *cache, int32_t *pos, int32_t *pos_len,
                            int32_t *n_seen, const int32_t *budget_dev, int32_t budget_scalar,
                            const int32_t *n_recent_dev, int32_t *moved_from_or_null, int32_t *target_or_null,
                            keepkv_stats *stats_or_null, void *ws, size_t ws_bytes, int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!pos || !pos_len || !n_seen || !ws || !status_dev || !aligned(ws, 256)) return KEEPKV_ERR_INVALID_ARG;
  if ((long long)p->B * p->H_kv > kMaxUnits) return KEEPKV_ERR_UNSUPPORTED;
  if (p->flags & KEEPKV_FLAG_COMPRESS_STEADY) return KEEPKV_ERR_INVALID_ARG;
  if (!budget_dev) {
    if (budget_scalar < 0) return KEEPKV_ERR_INVALID_ARG;
    if (budget_scalar > p->N_cap || (long long)budget_scalar + p->period > p->N_cap) return KEEPKV_ERR_CAPACITY;
  }
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  char *w = (char *)ws;
  launch_compress_inplace(*p, *cache, pos, pos_len, n_seen, budget_dev, budget_scalar, n_recent_dev, moved_from_or_null,
                          target_or_null ? target_or_null : (int32_t *)(w + L.target),
                          stats_or_null ? stats_or_null : (keepkv_stats *)(w + L.stats), w, L, status_dev, ctx);
  return finish(ctx);
}

int keepkv_compress_merge_first(const keepkv_params *p, const keepkv_cache *cache, const keepkv_cache *scratch,
                                const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                                int32_t *retained_idx_or_null, keepkv_stats *stats_or_null, void *ws, size_t ws_bytes,
                                int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if ((rc = validate_cache(scratch))) return rc;
  if (cache->K == scratch->K || cache->V == scratch->V || cache->votes == scratch->votes ||
      cache->lscore == scratch->lscore || cache->seq_len == scratch->seq_len)
    return KEEPKV_ERR_INVALID_ARG;
  if (!ws || !status_dev || !aligned(ws, 256)) return KEEPKV_ERR_INVALID_ARG;
  if ((long long)p->B * p->H_kv > kMaxUnits) return KEEPKV_ERR_UNSUPPORTED;
  if (p->flags & KEEPKV_FLAG_COMPRESS_STEADY) return KEEPKV_ERR_INVALID_ARG;   // a prompt is not a steady-state cache
  if (!budget_dev) {
    if (budget_scalar < 0) return KEEPKV_ERR_INVALID_ARG;
    if (budget_scalar > p->N_cap || (long long)budget_scalar + p->period > p->N_cap) return KEEPKV_ERR_CAPACITY;
  }
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  launch_compress_merge_first(*p, *cache, *scratch, budget_dev, budget_scalar, n_recent_dev, retained_idx_or_null,
                              stats_or_null, (char *)ws, L, status_dev, ctx);
  return finish(ctx);
}

int keepkv_decode_step_host(const keepkv_params *p, const keepkv_cache *cache, const void *q_host,
                            const void *k_new_host, const void *v_new_host, void *out_host, void *q_dev,
                            void *k_new_dev, void *v_new_dev, void *out_dev, int update_scores, void *ws,
                            size_t ws_bytes, int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(cache))) return rc;
  if (!q_host || !k_new_host || !v_new_host || !out_host || !q_dev || !k_new_dev || !v_new_dev || !out_dev || !ws ||
      !status_dev)
    return KEEPKV_ERR_INVALID_ARG;
  if (!aligned(q_dev, 16) || !aligned(k_new_dev, 16) || !aligned(v_new_dev, 16) || !aligned(out_dev, 16) ||
      !aligned(ws, 256))
    return KEEPKV_ERR_INVALID_ARG;
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  const size_t qb = (size_t)p->B * p->H_q * p->d * 2, kb = (size_t)p->B * p->H_kv * p->d * 2;
  auto cp = [&](void *dstp, const void *srcp, size_t n, cudaMemcpyKind kind) {
    cudaError_t e = cudaMemcpyAsync(dstp, srcp, n, kind, ctx.stream);
    if (e != cudaSuccess && ctx.err == cudaSuccess) ctx.err = e;
  };
  cp(q_dev, q_host, qb, cudaMemcpyHostToDevice);
  cp(k_new_dev, k_new_host, kb, cudaMemcpyHostToDevice);
  cp(v_new_dev, v_new_host, kb, cudaMemcpyHostToDevice);
  if (ctx.err == cudaSuccess)
    launch_decode(*p, *cache, q_dev, out_dev, nullptr, update_scores, (char *)ws, L, status_dev, ctx, k_new_dev, v_new_dev);
  if (ctx.err == cudaSuccess) cp(out_host, out_dev, qb, cudaMemcpyDeviceToHost);
  return finish(ctx);
}

int keepkv_decode_step_host_layers(const keepkv_params *p, const keepkv_cache *caches_host, int32_t n_layers,
                                   const void *q_host, const void *k_new_host, const void *v_new_host, void *out_host,
                                   void *q_dev, void *k_new_dev, void *v_new_dev, void *out_dev, int update_scores,
                                   void *ws, size_t ws_bytes, int32_t *status_dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if (!caches_host || n_layers <= 0) return KEEPKV_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if ((rc = validate_cache(&caches_host[l]))) return rc;
  if (!q_host || !k_new_host || !v_new_host || !out_host || !q_dev || !k_new_dev || !v_new_dev || !out_dev || !ws ||
      !status_dev)
    return KEEPKV_ERR_INVALID_ARG;
  if (!aligned(q_dev, 16) || !aligned(k_new_dev, 16) || !aligned(v_new_dev, 16) || !aligned(out_dev, 16) ||
      !aligned(ws, 256))
    return KEEPKV_ERR_INVALID_ARG;
  WsLayout L = ws_layout(*p);
  if (ws_bytes < L.total) return KEEPKV_ERR_WORKSPACE;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  const size_t qb = (size_t)p->B * p->H_q * p->d * 2, kb = (size_t)p->B * p->H_kv * p->d * 2;
  auto cp = [&](void *dstp, const void *srcp, size_t n, cudaMemcpyKind kind) {
    cudaError_t e = cudaMemcpyAsync(dstp, srcp, n, kind, ctx.stream);
    if (e != cudaSuccess && ctx.err == cudaSuccess) ctx.err = e;
  };
  const size_t qn = qb * n_layers, kn = kb * n_layers;
  const bool packed = (const char *)k_new_host == (const char *)q_host + qn && (const char *)v_new_host == (const char *)k_new_host + kn &&
                      (char *)k_new_dev == (char *)q_dev + qn && (char *)v_new_dev == (char *)k_new_dev + kn;
  if (packed) {   // queries, keys and values lie back to back on both sides: one copy instead of three
    cp(q_dev, q_host, qn + 2 * kn, cudaMemcpyHostToDevice);
  } else {
    cp(q_dev, q_host, qn, cudaMemcpyHostToDevice);
    cp(k_new_dev, k_new_host, kn, cudaMemcpyHostToDevice);
    cp(v_new_dev, v_new_host, kn, cudaMemcpyHostToDevice);
  }
  for (int l = 0; l < n_layers && ctx.err == cudaSuccess; ++l) {
    launch_decode(*p, caches_host[l], (const char *)q_dev + qb * l, (char *)out_dev + qb * l, nullptr, update_scores,
                  (char *)ws, L, status_dev, ctx, (const char *)k_new_dev + kb * l, (const char *)v_new_dev + kb * l);
  }
  if (ctx.err == cudaSuccess) cp(out_host, out_dev, qb * n_layers, cudaMemcpyDeviceToHost);
  return finish(ctx);
}

int keepkv_complete_append_host(const keepkv_params *p, void *K_host, void *V_host, int32_t *seq_len_host,
                                const void *k_new_host, const void *v_new_host) {
  int rc = validate(p);
  if (rc) return rc;
  if (!K_host || !V_host || !seq_len_host || !k_new_host || !v_new_host) return KEEPKV_ERR_INVALID_ARG;
  for (int b = 0; b < p->B; ++b)
    if (seq_len_host[b] < 0 || seq_len_host[b] >= p->N_cap) return KEEPKV_ERR_CAPACITY;   // nothing is written
  const size_t row = (size_t)p->d * 2;
  for (int b = 0; b < p->B; ++b) {
    for (int h = 0; h < p->H_kv; ++h) {
      const size_t u = (size_t)b * p->H_kv + h, at = (u * p->N_cap + seq_len_host[b]) * row;
      memcpy((char *)K_host + at, (const char *)k_new_host + u * row, row);
      memcpy((char *)V_host + at, (const char *)v_new_host + u * row, row);
    }
    seq_len_host[b] += 1;
  }
  return KEEPKV_OK;
}

int keepkv_complete_load_host(const keepkv_params *p, const void *K_host, const void *V_host,
                              const int32_t *seq_len_host, const keepkv_cache *dev, void *stream) {
  int rc = validate(p);
  if (rc) return rc;
  if ((rc = validate_cache(dev))) return rc;
  if (!K_host || !V_host || !seq_len_host) return KEEPKV_ERR_INVALID_ARG;
  for (int b = 0; b < p->B; ++b)
    if (seq_len_host[b] < 0 || seq_len_host[b] > p->N_cap) return KEEPKV_ERR_CAPACITY;
  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  const size_t row = (size_t)p->d * 2, pitch = (size_t)p->N_cap * row;
  auto cp = [&](cudaError_t e) { if (e != cudaSuccess && ctx.err == cudaSuccess) ctx.err = e; };
  for (int b = 0; b < p->B; ++b) {   // the H_kv units of a sequence have the same length: one pitched copy per array
    if (seq_len_host[b] == 0) continue;
    const size_t off = (size_t)b * p->H_kv * pitch, width = (size_t)seq_len_host[b] * row;
    cp(cudaMemcpy2DAsync((char *)dev->K + off, pitch, (const char *)K_host + off, pitch, width, p->H_kv,
                         cudaMemcpyHostToDevice, ctx.stream));
    cp(cudaMemcpy2DAsync((char *)dev->V + off, pitch, (const char *)V_host + off, pitch, width, p->H_kv,
                         cudaMemcpyHostToDevice, ctx.stream));
  }
  cp(cudaMemcpyAsync(dev->seq_len, seq_len_host, (size_t)p->B * 4, cudaMemcpyHostToDevice, ctx.stream));
  if (ctx.err == cudaSuccess) launch_fresh_state(*p, *dev, ctx);
  return finish(ctx);
}

const char *keepkv_status_string(int status) {
  switch (status) {
    case KEEPKV_OK: return "KEEPKV_OK";
    case KEEPKV_ERR_INVALID_ARG: return "KEEPKV_ERR_INVALID_ARG";
    case KEEPKV_ERR_UNSUPPORTED: return "KEEPKV_ERR_UNSUPPORTED";
    case KEEPKV_ERR_CAPACITY: return "KEEPKV_ERR_CAPACITY";
    case KEEPKV_ERR_WORKSPACE: return "KEEPKV_ERR_WORKSPACE";
    case KEEPKV_ERR_CUDA: return "KEEPKV_ERR_CUDA";
    default: return "KEEPKV_UNKNOWN_STATUS";
  }
}

int keepkv_last_cuda_error(void) { return g_last_cuda_error; }
int keepkv_last_launch_count(void) { return g_last_launches; }

}  // extern "C"
