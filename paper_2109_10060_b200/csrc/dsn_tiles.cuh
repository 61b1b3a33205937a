// Tile schedule over ragged groups, built inside each kernel from the device-resident group
// offsets (group sizes never travel to the host).  Groups are walked from the last (widest path)
// to the first so that the most expensive tiles are handed out first.
#pragma once
#include <stdint.h>

// s_prefix[j] = number of tiles in the j first groups of the reversed order (j = 0..G);
// ntiles_of(g) gives the tile count of group g.  All threads of the CTA must call this.
template <typename F>
__device__ __forceinline__ void dsn_build_tile_prefix(int G, int32_t* s_prefix, F ntiles_of) {
  for (int j = threadIdx.x; j < G; j += blockDim.x) s_prefix[j + 1] = ntiles_of(G - 1 - j);
  if (threadIdx.x == 0) s_prefix[0] = 0;
  __syncthreads();
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    int carry = 0;
    for (int base = 0; base < G; base += 32) {
      const int j = base + lane;
      int v = j < G ? s_prefix[j + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      if (j < G) s_prefix[j + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
}

// position j in the reversed order whose tile range contains `tile` (tile < s_prefix[G])
__device__ __forceinline__ int dsn_find_tile_slot(const int32_t* s_prefix, int G, int tile) {
  int lo = 0, hi = G;  // s_prefix[lo] <= tile < s_prefix[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_prefix[mid] <= tile) lo = mid; else hi = mid;
  }
  return lo;
}
