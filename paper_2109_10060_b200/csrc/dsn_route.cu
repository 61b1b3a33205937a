// Stable grouping of samples by path index: histogram, exclusive scan, stable permutation.
// Integer work, bit-exact and deterministic.  One CTA of 1024 threads handles any B: the batch
// is walked in chunks of 1024 samples; inside a chunk every warp ranks its 32 samples with
// __match_any_sync, per-warp per-path counts are scanned across the 32 warps, and a running
// per-path base carries the order from chunk to chunk.
#include "dsn_internal.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__global__ void __launch_bounds__(kThreads, 1)
route_kernel(const int32_t* __restrict__ idx, int B, int T, int32_t* __restrict__ counts,
             int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
             int32_t* status) {
  __shared__ int32_t s_warp_cnt[kWarps][DSN_MAX_SLICES];  // per-warp count of each path in this chunk
  __shared__ int32_t s_run[DSN_MAX_SLICES];               // samples of each path seen in earlier chunks
  __shared__ int32_t s_off[DSN_MAX_SLICES + 1];
  __shared__ int32_t s_bad;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (tid < DSN_MAX_SLICES) s_run[tid] = 0;
  if (tid == 0) s_bad = 0;
  __syncthreads();

  // pass 1: histogram
  int bad_local = 0;
  for (int base = 0; base < B; base += kThreads) {
    const int i = base + tid;
    int key = -1;
    if (i < B) {
      key = idx[i];
      if (key < 0 || key >= T) { key = -1; ++bad_local; }
    }
    if (key >= 0) atomicAdd(&s_run[key], 1);   // integer adds commute: the counts are exact
  }
  if (bad_local) atomicAdd(&s_bad, bad_local);
  __syncthreads();

  if (tid == 0) {
    int acc = 0;
    for (int t = 0; t < T; ++t) {
      s_off[t] = acc;
      acc += s_run[t];
    }
    s_off[T] = acc;
    if (s_bad) {
      dsn_set_status(status, DSN_ERR_BAD_INDEX, s_bad);
      if (status) atomicAdd(status + 3, s_bad);
    }
  }
  __syncthreads();
  if (tid < T) counts[tid] = s_run[tid];
  if (tid <= T) offsets[tid] = s_off[tid];
  const int placed = s_off[T];
  for (int p = placed + tid; p < B; p += kThreads) perm[p] = -1;
  __syncthreads();
  if (tid < DSN_MAX_SLICES) s_run[tid] = 0;
  __syncthreads();

  // pass 2: stable positions
  for (int base = 0; base < B; base += kThreads) {
    const int i = base + tid;
    int key = -1;
    if (i < B) {
      key = idx[i];
      if (key < 0 || key >= T) key = -1;
    }
    for (int t = lane; t < T; t += 32) s_warp_cnt[warp][t] = 0;
    __syncwarp();
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
    if (key >= 0 && rank_in_warp == 0) s_warp_cnt[warp][key] = __popc(peers);
    __syncthreads();
    // exclusive scan over warps, one thread per path
    if (tid < T) {
      int acc = s_run[tid];
      for (int w = 0; w < kWarps; ++w) {
        const int c = s_warp_cnt[w][tid];
        s_warp_cnt[w][tid] = acc;
        acc += c;
      }
      s_run[tid] = acc;
    }
    __syncthreads();
    if (key >= 0) {
      const int p = s_off[key] + s_warp_cnt[warp][key] + rank_in_warp;
      perm[p] = i;
      inv_perm[i] = p;
    } else if (i < B) {
      inv_perm[i] = -1;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t dsn_launch_route(const int32_t* idx, int B, int T, int32_t* counts, int32_t* offsets,
                             int32_t* perm, int32_t* inv_perm, int32_t* status, cudaStream_t s) {
  return dsn_launch(route_kernel, dim3(1), dim3(kThreads), 0, s, 1, idx, B, T, counts, offsets, perm, inv_perm, status);
}
