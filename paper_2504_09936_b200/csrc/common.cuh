// Internal declarations shared by the translation units of libkeepkv (not installed).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include <utility>

#include "keepkv.h"

namespace keepkv {

constexpr int kTile = 64;          // entries per K/V tile of the decode kernel
constexpr int kDecMaxCtas = 512;    // upper bound on the persistent decode grid (sizes the partial pool)

constexpr int kMaxUnits = 4096;    // B * H_kv that keepkv_compress accepts (per-unit tables live in shared memory)
constexpr int kNomChunksMax = 8;   // upper bound on the column chunks a row's similarity search is split into

// n_keys / ticket: entries to merge appended so far and resolve CTAs finished (select_kernel zeroes them)
struct UnitInfo { int len, n_ret, n_ev, n_groups, n_keys, ticket, pad0, pad1; };

// Byte offsets of the arrays kept in the caller's workspace.  U = B*H_kv, N = N_cap.
struct WsLayout {
  size_t counters;    // i32 [U + 1]        split-KV arrival counters per unit, finished CTAs of a step (zero between calls)
  size_t part_pool;   // f32 [kDecMaxCtas,2,16+G*d]  partial results of units cut across CTAs (two per CTA)
  size_t unit_info;   // UnitInfo [U]       len, n_ret, n_ev, n_groups of the running compression
  size_t sched;       // i32 [4]            column-chunk count the nomination kernel settled on
  size_t ret_idx;     // i32 [U,N]          source index of each retained slot, ascending
  size_t target;      // i32 [U,N]          per source entry: slot, -1 dropped, -2 retained
  size_t ev_idx;      // i32 [U,N]          source indices of evicted entries, ascending
  size_t inv_norm;    // f32 [U,N]          1/|k| of each retained key (tree-summed; only ranks candidates)
  size_t nom_v;       // float4 [U,N,C]     per evicted row and column chunk: best, second cosine, unused, best slot
  size_t nom_si;      // i32 [U,N,C]        slot of the second-best cosine
  size_t grp_key;     // u32 [U,Npow2]      (slot << 16 | evicted position) of merged entries, sorted
  size_t grp_head;    // i32 [U,N]          position in grp_key where each group starts
  size_t stats;       // keepkv_stats [U]   used when the caller passes no stats array
  size_t stats2;      // keepkv_stats [U]   merge-first: statistics of the merge pass
  size_t unit_len;    // i32 [U]            merge-first: entries of each unit after the merge pass
  size_t eff_budget;  // i32 [B]            merge-first: budget of each sequence, capped by its shortest head
  size_t kept;        // i32 [U,N]          in place: the retained rows, ascending
  size_t total;
  size_t decode_bytes;   // the leading part that keepkv_decode_attention uses (counters and partials)
  size_t counter_bytes;  // size of the counters array
  int nom_chunks;        // C: column chunks reserved per evicted row
  int key_stride;        // Npow2: N rounded up to a power of two
};

WsLayout ws_layout(const keepkv_params &p);

struct LaunchCtx {
  cudaStream_t stream;
  int launches;
  cudaError_t err;
};

// records the launch count / CUDA error of a finished call and maps them to a keepkv_status
int finish_call(LaunchCtx &ctx);

// launchers (each returns cudaSuccess or the launch error and bumps ctx.launches)
void launch_append(const keepkv_params &p, const keepkv_cache &c, const void *k_new, const void *v_new,
                   int32_t *status_dev, LaunchCtx &ctx);
void launch_fresh_state(const keepkv_params &p, const keepkv_cache &c, LaunchCtx &ctx);
// k_new / v_new: the step's token to append inside the same launch (keepkv_decode_step), or null
void launch_decode(const keepkv_params &p, const keepkv_cache &c, const void *q, void *out, float *lse,
                   int update_scores, char *ws, const WsLayout &L, int32_t *status_dev, LaunchCtx &ctx,
                   const void *k_new = nullptr, const void *v_new = nullptr);
void launch_compress(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst,
                     const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev, int32_t *ret_idx,
                     int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L, int32_t *status_dev,
                     LaunchCtx &ctx, const float *select_key = nullptr);
// tcgen05 similarity search: for every evicted key the two largest cosines over the retained keys
void launch_nominate(const keepkv_params &p, const keepkv_cache &src, const keepkv_cache &dst, const int32_t *ev_idx,
                     const UnitInfo *unit_info, const float *inv_norm, int32_t *sched, float4 *nom_v, int32_t *nom_si,
                     int nom_chunks, int32_t *status_dev, LaunchCtx &ctx, int self_mask = 0);
// Algorithm 1 in place on a cache with a position array (compress.cu)
void launch_compress_inplace(const keepkv_params &p, const keepkv_cache &c, int32_t *pos, int32_t *pos_len, int32_t *n_seen,
                             const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                             int32_t *moved_from, int32_t *target, keepkv_stats *stats, char *ws, const WsLayout &L,
                             int32_t *status_dev, LaunchCtx &ctx);
// Section 3.4, prefill merge-first policy (compress.cu): cache -> scratch (merge) -> cache (eviction)
void launch_compress_merge_first(const keepkv_params &p, const keepkv_cache &cache, const keepkv_cache &scratch,
                                 const int32_t *budget_dev, int32_t budget_scalar, const int32_t *n_recent_dev,
                                 int32_t *ret_idx_out, keepkv_stats *stats_out, char *ws, const WsLayout &L,
                                 int32_t *status_dev, LaunchCtx &ctx);
void launch_prefill_scores(const keepkv_params &p, const keepkv_cache &c, const void *q_window, int W,
                           int32_t *status_dev, LaunchCtx &ctx);
int sm_count();

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in
// the stream is still draining, and runs its preamble (barrier set-up, tensor-map prefetch, tensor
// memory allocation) there.  Every kernel of this library calls pdl_wait() before it touches global
// memory, which blocks until the predecessor has completed and its writes are visible, so stream
// order is preserved; pdl_trigger() lets the successor start its own preamble early.
template <typename... KArgs, typename... Args>
inline void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                       Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}
// The same with the grid cut into thread-block clusters of `cluster_x` consecutive CTAs.
template <typename... KArgs, typename... Args>
inline void launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                               unsigned cluster_x, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

#define KEEPKV_CHECK_LAUNCH(ctx)                        \
  do {                                                  \
    cudaError_t e__ = cudaGetLastError();               \
    (ctx).launches++;                                   \
    if (e__ != cudaSuccess && (ctx).err == cudaSuccess) \
      (ctx).err = e__;                                  \
  } while (0)

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

}  // namespace keepkv
