// Row movement between input order and grouped order, and zero-fill of the unused output tail.
// HBM-bound copies: one CTA per grouped position p (one sample), 16-byte accesses whenever the
// slice width, leading dimensions and base pointers allow, otherwise element-wise.
#include "dsn_internal.cuh"

namespace {

constexpr int kThreads = 256;

// group that owns grouped position p: largest g with offsets[g] <= p (empty groups skipped)
__device__ __forceinline__ int find_group(const int32_t* __restrict__ offsets, int G, int p) {
  int lo = 0, hi = G;  // invariant: offsets[lo] <= p < offsets[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (offsets[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

struct RowJob {
  int valid;
  int slice;
  int sample;
};

__device__ __forceinline__ RowJob locate(int p, int G, const int32_t* offsets, const int32_t* perm,
                                         const int32_t* group_slice) {
  __shared__ RowJob job;
  if (threadIdx.x == 0) {
    RowJob j;
    j.valid = p < offsets[G];
    if (j.valid) {
      const int g = find_group(offsets, G, p);
      j.slice = group_slice ? group_slice[g] : g;
      j.sample = perm[p];
      if (j.sample < 0) j.valid = 0;
    } else {
      j.slice = 0;
      j.sample = 0;
    }
    job = j;
  }
  __syncthreads();
  return job;
}

__global__ void __launch_bounds__(kThreads)
permute_rows_kernel(SliceTable st, int elem_bytes, int R, const char* __restrict__ src, int64_t ld_src,
                    char* __restrict__ dst, int64_t ld_dst, int to_grouped, int G,
                    const int32_t* __restrict__ offsets, const int32_t* __restrict__ perm,
                    const int32_t* __restrict__ group_slice) {
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int p = blockIdx.x;
  const RowJob j = locate(p, G, offsets, perm, group_slice);
  if (!j.valid) return;
  const int64_t row_bytes = (int64_t)st.k_in[j.slice] * elem_bytes;
  const int64_t sb = ld_src * elem_bytes, db = ld_dst * elem_bytes;
  const char* s = src + (int64_t)(to_grouped ? j.sample : p) * R * sb;
  char* d = dst + (int64_t)(to_grouped ? p : j.sample) * R * db;
  const bool vec = (row_bytes % 16 == 0) && (sb % 16 == 0) && (db % 16 == 0) &&
                   ((reinterpret_cast<uintptr_t>(s) & 15) == 0) && ((reinterpret_cast<uintptr_t>(d) & 15) == 0);
  if (vec) {
    const int nv = (int)(row_bytes >> 4);
    const int64_t total = (int64_t)R * nv;
    for (int64_t e = threadIdx.x; e < total; e += kThreads) {
      const int r = (int)(e / nv), v = (int)(e - (int64_t)r * nv);
      reinterpret_cast<uint4*>(d + r * db)[v] = __ldg(reinterpret_cast<const uint4*>(s + r * sb) + v);
    }
  } else {
    const int64_t total = (int64_t)R * row_bytes;
    for (int64_t e = threadIdx.x; e < total; e += kThreads) {
      const int r = (int)(e / row_bytes);
      const int64_t c = e - (int64_t)r * row_bytes;
      d[r * db + c] = s[r * sb + c];
    }
  }
}

__global__ void __launch_bounds__(kThreads)
zero_tail_kernel(SliceTable st, int elem_bytes, int R, int C_out, char* __restrict__ y, int64_t ldy,
                 int y_input_order, int G, const int32_t* __restrict__ offsets,
                 const int32_t* __restrict__ perm, const int32_t* __restrict__ group_slice) {
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int p = blockIdx.x;
  const RowJob j = locate(p, G, offsets, perm, group_slice);
  if (!j.valid) return;
  const int64_t first = (int64_t)st.k_out[j.slice] * elem_bytes, last = (int64_t)C_out * elem_bytes;
  if (first >= last) return;
  const int64_t yb = ldy * elem_bytes, span = last - first;
  char* d = y + (int64_t)(y_input_order ? j.sample : p) * R * yb + first;
  for (int64_t e = threadIdx.x; e < (int64_t)R * span; e += kThreads) {
    const int r = (int)(e / span);
    d[r * yb + (e - (int64_t)r * span)] = 0;
  }
}

}  // namespace

cudaError_t dsn_launch_permute_rows(const SliceTable& st, int elem_bytes, int R, const void* src,
                                    int64_t ld_src, void* dst, int64_t ld_dst, int to_grouped, int B, int G,
                                    const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                    cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  return dsn_launch(permute_rows_kernel, dim3(B), dim3(kThreads), 0, s, 1, st, elem_bytes, R,
                    static_cast<const char*>(src), ld_src, static_cast<char*>(dst), ld_dst, to_grouped, G, offsets, perm,
                    group_slice);
}

cudaError_t dsn_launch_zero_tail(const SliceTable& st, int elem_bytes, int R, int C_out, void* y, int64_t ldy,
                                 int y_input_order, int B, int G, const int32_t* offsets, const int32_t* perm,
                                 const int32_t* group_slice, cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  return dsn_launch(zero_tail_kernel, dim3(B), dim3(kThreads), 0, s, 1, st, elem_bytes, R, C_out, static_cast<char*>(y),
                    ldy, y_input_order, G, offsets, perm, group_slice);
}
