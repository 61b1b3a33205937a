// fp32 sliced linear layer on plain FMA units (no TF32): y = x[:, :k_in] * W[:k_out, :k_in]^T per
// group.  Classic shared-memory tiling: 64x64 output tile, K step 16, 256 threads with a 4x4
// register block each.  Persistent CTAs walk the ragged tile list built from the group offsets.
#include "dsn_internal.cuh"
#include "dsn_tiles.cuh"

namespace {

constexpr int BM = 64, BN = 64, BK = 16, kThreads = 256;

__device__ __forceinline__ float apply_act(float v, int act) {
  if (act == DSN_ACT_RELU) return fmaxf(v, 0.f);
  if (act == DSN_ACT_GELU) return 0.5f * v * (1.f + erff(v * 0.70710678118654752f));
  return v;
}

__global__ void __launch_bounds__(kThreads)
linear_f32_kernel(SliceTable st, int R, const float* __restrict__ x, int64_t ldx, const float* __restrict__ W,
                  int64_t ldw, float* __restrict__ y, int64_t ldy, const float* __restrict__ bias,
                  const float* __restrict__ bn_scale, const float* __restrict__ bn_shift, int bn_ld,
                  const float* __restrict__ residual, int act,
                  int x_input_order, int y_input_order, int G, const int32_t* __restrict__ offsets,
                  const int32_t* __restrict__ perm, const int32_t* __restrict__ group_slice) {
  extern __shared__ int32_t s_prefix[];  // [G+1]
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];

  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  auto ntiles_of = [&](int g) {
    const int rows = (offsets[g + 1] - offsets[g]) * R;
    const int sl = group_slice ? group_slice[g] : g;
    return ((rows + BM - 1) / BM) * ((st.k_out[sl] + BN - 1) / BN);
  };
  dsn_build_tile_prefix(G, s_prefix, ntiles_of);
  const int total = s_prefix[G];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  for (int tile = blockIdx.x; tile < total; tile += gridDim.x) {
    const int j = dsn_find_tile_slot(s_prefix, G, tile);
    const int g = G - 1 - j;
    const int sl = group_slice ? group_slice[g] : g;
    const int ki = st.k_in[sl], ko = st.k_out[sl];
    const int p0 = offsets[g], rows_g = (offsets[g + 1] - p0) * R;
    const int ntn = (ko + BN - 1) / BN;
    const int local = tile - s_prefix[j];
    const int row0 = (local / ntn) * BM, n0 = (local % ntn) * BN;

    // rows this thread loads (4 of them) and the W rows it loads
    const float* xrow[4];
    const float* wrow[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = (tid >> 4) + 16 * i;
      const int gr = row0 + r;
      if (gr < rows_g) {
        const int p = p0 + gr / R, rr = gr % R;
        const int smp = x_input_order ? perm[p] : p;
        xrow[i] = x + ((int64_t)smp * R + rr) * ldx;
      } else {
        xrow[i] = nullptr;
      }
      wrow[i] = (n0 + r < ko) ? W + (int64_t)(n0 + r) * ldw : nullptr;
    }
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    for (int k0 = 0; k0 < ki; k0 += BK) {
      const int kk = tid & 15;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = (tid >> 4) + 16 * i;
        const bool kin = k0 + kk < ki;
        As[kk][r] = (xrow[i] && kin) ? xrow[i][k0 + kk] : 0.f;
        Bs[kk][r] = (wrow[i] && kin) ? wrow[i][k0 + kk] : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          a[i] = As[k][ty * 4 + i];
          b[i] = Bs[k][tx * 4 + i];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int q = 0; q < 4; ++q) acc[i][q] = fmaf(a[i], b[q], acc[i][q]);
      }
      __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gr = row0 + ty * 4 + i;
      if (gr >= rows_g) continue;
      const int p = p0 + gr / R, rr = gr % R;
      const int smp = y_input_order ? perm[p] : p;
      float* yr = y + ((int64_t)smp * R + rr) * ldy;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int n = n0 + tx * 4 + q;
        if (n < ko) {
          float v = acc[i][q] + (bias ? bias[n] : 0.f);
          if (bn_scale) v = fmaf(v, bn_scale[(int64_t)sl * bn_ld + n], bn_shift[(int64_t)sl * bn_ld + n]);
          if (residual) v += residual[((int64_t)smp * R + rr) * ldy + n];
          yr[n] = apply_act(v, act);
        }
      }
    }
  }
}

}  // namespace

cudaError_t dsn_launch_linear_f32(const SliceTable& st, int T, int R, const float* x, int64_t ldx,
                                  const float* W, int64_t ldw, float* y, int64_t ldy, const float* bias,
                                  const float* bn_scale, const float* bn_shift, int bn_ld, const float* residual, int act, int x_input_order, int y_input_order, int B, int G,
                                  const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                  int sm_count, cudaStream_t s) {
  (void)T;
  if (B == 0) return cudaSuccess;
  int max_ko = 1;
  for (int t = 0; t < DSN_MAX_SLICES; ++t) max_ko = st.k_out[t] > max_ko ? st.k_out[t] : max_ko;
  const int64_t bound = ((int64_t)B * R / BM + G) * ((max_ko + BN - 1) / BN);
  int64_t grid = bound < (int64_t)sm_count * 4 ? bound : (int64_t)sm_count * 4;
  if (grid < 1) grid = 1;
  return dsn_launch(linear_f32_kernel, dim3((unsigned)grid), dim3(kThreads), sizeof(int32_t) * (G + 1), s, 1, st, R, x,
                    ldx, W, ldw, y, ldy, bias, bn_scale, bn_shift, bn_ld, residual, act, x_input_order, y_input_order, G, offsets, perm,
                    group_slice);
}
