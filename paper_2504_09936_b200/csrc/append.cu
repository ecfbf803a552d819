// keepkv_append: Eq. 2 of the paper -- the cache grows by one (k_t, v_t) row per sequence.
#include "common.cuh"

namespace keepkv {

// One CTA per sequence: all kv heads of a sequence share seq_len[b], so the CTA that owns the
// sequence reads it once, writes every head's row, and only then publishes the new length.
__global__ void __launch_bounds__(128) append_kernel(keepkv_params p, keepkv_cache c, const uint4 *__restrict__ k_new,
                                                     const uint4 *__restrict__ v_new, int32_t *status_dev) {
  const int b = blockIdx.x;
  pdl_wait();
  pdl_trigger();
  const int pos = c.seq_len[b];
  if (pos < 0 || pos >= p.N_cap) {   // full, or a length that is not one: skipped and reported, never written
    if (threadIdx.x == 0) atomicOr(status_dev, KEEPKV_DEV_APPEND_FULL);
    return;
  }
  const int chunks = p.d / 8;  // 16-byte pieces per row
  uint4 *K = reinterpret_cast<uint4 *>(c.K), *V = reinterpret_cast<uint4 *>(c.V);
  for (int i = threadIdx.x; i < p.H_kv * chunks; i += blockDim.x) {
    const int h = i / chunks, j = i % chunks;
    const size_t u = (size_t)b * p.H_kv + h;
    const size_t row = (u * p.N_cap + pos) * chunks + j;
    K[row] = k_new[u * chunks + j];
    V[row] = v_new[u * chunks + j];
  }
  for (int h = threadIdx.x; h < p.H_kv; h += blockDim.x) {
    const size_t e = ((size_t)b * p.H_kv + h) * p.N_cap + pos;
    c.votes[e] = 1.0f;                // a fresh entry holds one vote
    c.lscore[e] = -CUDART_INF_F;      // and has no score history
  }
  __syncthreads();
  if (threadIdx.x == 0) c.seq_len[b] = pos + 1;
}

// Fresh state of a cache whose rows were just loaded: one vote per entry, no score history.
__global__ void fresh_state_kernel(keepkv_params p, keepkv_cache c) {
  const int u = blockIdx.y, b = u / p.H_kv;
  const int len = max(0, min(c.seq_len[b], p.N_cap));
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < len; i += gridDim.x * blockDim.x) {
    c.votes[(size_t)u * p.N_cap + i] = 1.0f;
    c.lscore[(size_t)u * p.N_cap + i] = -CUDART_INF_F;
  }
}

void launch_fresh_state(const keepkv_params &p, const keepkv_cache &c, LaunchCtx &ctx) {
  fresh_state_kernel<<<dim3(8, p.B * p.H_kv), 256, 0, ctx.stream>>>(p, c);
  KEEPKV_CHECK_LAUNCH(ctx);
}

void launch_append(const keepkv_params &p, const keepkv_cache &c, const void *k_new, const void *v_new,
                   int32_t *status_dev, LaunchCtx &ctx) {
  launch_pdl(append_kernel, dim3(p.B), dim3(128), 0, ctx.stream, p, c, reinterpret_cast<const uint4 *>(k_new),
             reinterpret_cast<const uint4 *>(v_new), status_dev);
  KEEPKV_CHECK_LAUNCH(ctx);
}

}  // namespace keepkv
