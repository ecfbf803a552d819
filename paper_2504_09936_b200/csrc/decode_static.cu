// keepkv_decode_attention_static: the decode attention of keepkv_decode_attention for callers that
// cannot hand the library a workspace, because they cannot allocate device memory at the point
// where they call it (a plug-in running inside another runtime's memory pool, a replayed
// inference loop whose buffers were all fixed at start-up, a host that forbids cudaMalloc after
// initialisation).  The split-KV scratch lives in a fixed array inside the library image.
#include <mutex>

#include "common.cuh"

namespace keepkv {

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[KEEPKV_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address has to be asked for, once per device, while that device is current.
static unsigned char *static_scratch_ptr(cudaError_t &err) {
  static std::mutex mu;
  static unsigned char *ptrs[64] = {};
  int dev = 0;
  err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) { err = cudaErrorInvalidDevice; return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  if (!ptrs[dev]) {
    void *ptr = nullptr;
    err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (err != cudaSuccess) return nullptr;
    ptrs[dev] = static_cast<unsigned char *>(ptr);
  }
  return ptrs[dev];
}

}  // namespace keepkv

using namespace keepkv;

extern "C" int keepkv_decode_attention_static(const keepkv_params *p, const keepkv_cache *cache, const void *q,
                                              void *out, float *lse_or_null, int update_scores, int32_t *status_dev,
                                              void *stream) {
  size_t total = 0;
  int rc = keepkv_workspace_bytes(p, &total);   // validates the shape
  if (rc) return rc;
  if (!cache || !cache->K || !cache->V || !cache->votes || !cache->lscore || !cache->seq_len || !q || !out ||
      !status_dev)
    return KEEPKV_ERR_INVALID_ARG;
  auto misaligned = [](const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; };
  if (misaligned(cache->K) || misaligned(cache->V) || misaligned(cache->votes) || misaligned(cache->lscore) ||
      misaligned(q) || misaligned(out))
    return KEEPKV_ERR_INVALID_ARG;
  // The decode arrays are the first ones of the workspace layout; the compression arrays that follow are not needed.
  const WsLayout L = ws_layout(*p);
  const size_t need = L.decode_bytes;
  if (need > (size_t)KEEPKV_STATIC_SCRATCH_BYTES) return KEEPKV_ERR_WORKSPACE;

  LaunchCtx ctx{(cudaStream_t)stream, 0, cudaSuccess};
  unsigned char *scratch = static_scratch_ptr(ctx.err);
  if (scratch && ctx.err == cudaSuccess) {
    // the arrival counters must start at zero whatever the previous call left behind
    ctx.err = cudaMemsetAsync(scratch + L.counters, 0, L.counter_bytes, ctx.stream);
  }
  if (ctx.err == cudaSuccess)
    launch_decode(*p, *cache, q, out, lse_or_null, update_scores, reinterpret_cast<char *>(scratch), L, status_dev,
                  ctx);
  return finish_call(ctx);
}
