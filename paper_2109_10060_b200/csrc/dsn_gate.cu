// Gate routing head (Sec. 3.5): average pooling over the R positions of each sample, a two-layer
// MLP (ReLU between), and the index of the first maximum score.
//
// Kernel 1 (HBM-bound): grid (splits, B), 512 threads.  A CTA streams a contiguous band of rows of
// one sample: consecutive threads read consecutive 16 bytes of a row, the CTA's row groups walk
// different rows, four loads are in flight per thread; fp32 accumulation in registers, one
// shared-memory reduction across the row groups, column sums to partial[b][split][c].  No atomics,
// so sums are reproducible run to run.
// Kernel 2 (L2-bound, plain FMA): grid (B/4, C_mlp/16).  A CTA folds the partial sums of 4 samples
// (scaled by 1/R) into shared memory and computes 16 hidden units for them, one warp per two
// units with 16-byte weight loads and a shuffle reduction; ReLU; hid[b][j] to scratch.
// Kernel 3 (tiny): one warp per sample evaluates the T scores and takes the arg-max with a strict
// '>' scan in ascending path order (ties keep the lowest index).
#include "dsn_internal.cuh"

namespace {

constexpr int kSB = 4;             // samples per CTA in the hidden-layer kernel
constexpr int kJB = 16;            // hidden units per CTA in the hidden-layer kernel
constexpr int kPoolThreads = 512;
constexpr int kMlpThreads = 256;

// 16-byte read-only load that the compiler keeps in program order, so that a run of them stays
// in flight together instead of being interleaved with the arithmetic that consumes them
__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void add8(float (&acc)[8], const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    acc[2 * j] += __uint_as_float(w[j] << 16);
    acc[2 * j + 1] += __uint_as_float(w[j] & 0xffff0000u);
  }
}

// bf16 input, c_valid % 8 == 0, ldx % 8 == 0, x 16-byte aligned.  CT = column threads (power of two).
__global__ void __launch_bounds__(kPoolThreads)
pool_bf16_vec_kernel(const __nv_bfloat16* __restrict__ x, int R, int64_t ldx, int c_valid, int splits, int CT,
                     float* __restrict__ partial) {
  __shared__ float red[kPoolThreads * 8];
  const int b = blockIdx.y, sp = blockIdx.x;
  const int r0 = (int)(((int64_t)R * sp) / splits), r1 = (int)(((int64_t)R * (sp + 1)) / splits);
  const int nvec = c_valid >> 3;
  const int tx = threadIdx.x & (CT - 1), ty = threadIdx.x / CT, RG = kPoolThreads / CT;
  const __nv_bfloat16* xb = x + (int64_t)b * R * ldx;
  float* out = partial + ((int64_t)b * splits + sp) * c_valid;
  const int64_t stride = ldx >> 3;  // row pitch in uint4
  for (int v0 = 0; v0 < nvec; v0 += CT) {
    const int v = v0 + tx;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (v < nvec) {
      const uint4* col = reinterpret_cast<const uint4*>(xb) + v;
      int r = r0 + ty;
      for (; r + 7 * RG < r1; r += 8 * RG) {  // eight independent loads in flight per thread
        uint4 a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) a[u] = ld_stream16(col + (int64_t)(r + u * RG) * stride);
#pragma unroll
        for (int u = 0; u < 8; ++u) add8(acc, a[u]);
      }
      for (; r + 3 * RG < r1; r += 4 * RG) {
        const uint4 a0 = ld_stream16(col + (int64_t)r * stride), a1 = ld_stream16(col + (int64_t)(r + RG) * stride),
                    a2 = ld_stream16(col + (int64_t)(r + 2 * RG) * stride), a3 = ld_stream16(col + (int64_t)(r + 3 * RG) * stride);
        add8(acc, a0); add8(acc, a1); add8(acc, a2); add8(acc, a3);
      }
      for (; r < r1; r += RG) add8(acc, __ldg(col + (int64_t)r * stride));
    }
    float4* mine = reinterpret_cast<float4*>(red + (size_t)threadIdx.x * 8);
    mine[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    mine[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    __syncthreads();
    // one thread per (column vector, half): sum over the row groups in a fixed order
    if (threadIdx.x < 2 * CT) {
      const int cx = threadIdx.x >> 1, half = threadIdx.x & 1;
      if (v0 + cx < nvec) {
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int g = 0; g < RG; ++g) {
          const float4 t = reinterpret_cast<const float4*>(red + (size_t)(g * CT + cx) * 8)[half];
          sum.x += t.x; sum.y += t.y; sum.z += t.z; sum.w += t.w;
        }
        reinterpret_cast<float4*>(out + 8 * (v0 + cx))[half] = sum;
      }
    }
    __syncthreads();
  }
}

// any dtype / any width: one channel per thread
template <typename Tin>
__global__ void __launch_bounds__(128)
pool_scalar_kernel(const Tin* __restrict__ x, int R, int64_t ldx, int c_valid, int splits,
                   float* __restrict__ partial) {
  const int b = blockIdx.y, sp = blockIdx.x;
  const int r0 = (int)(((int64_t)R * sp) / splits), r1 = (int)(((int64_t)R * (sp + 1)) / splits);
  const Tin* xb = x + (int64_t)b * R * ldx;
  float* out = partial + ((int64_t)b * splits + sp) * c_valid;
  for (int c = threadIdx.x; c < c_valid; c += 128) {
    float acc = 0.f;
    for (int r = r0; r < r1; ++r) acc += (float)xb[(int64_t)r * ldx + c];
    out[c] = acc;
  }
}

__global__ void __launch_bounds__(kMlpThreads)
gate_hidden_kernel(const float* __restrict__ partial, int splits, int B, int R, int C_full, int c_valid, int C_mlp,
                   const float* __restrict__ W1, const float* __restrict__ b1, float* __restrict__ hid) {
  extern __shared__ __align__(16) float pooled[];  // [kSB][c_valid]
  const int b0 = blockIdx.x * kSB, j0 = blockIdx.y * kJB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float inv_r = 1.0f / (float)R;
  if (c_valid % 4 == 0) {  // partial rows are 16-byte aligned: fold with 16-byte loads, splits in flight together
    const int n4 = c_valid >> 2;
    for (int e = tid; e < kSB * n4; e += kMlpThreads) {
      const int s = e / n4, c4 = e - s * n4;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (b0 + s < B) {
        const float4* p = reinterpret_cast<const float4*>(partial + ((int64_t)(b0 + s) * splits) * c_valid) + c4;
#pragma unroll 8
        for (int sp = 0; sp < splits; ++sp) {
          const float4 t = p[(int64_t)sp * n4];
          acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
      }
      reinterpret_cast<float4*>(pooled + s * c_valid)[c4] = make_float4(acc.x * inv_r, acc.y * inv_r, acc.z * inv_r, acc.w * inv_r);
    }
  } else {
    for (int e = tid; e < kSB * c_valid; e += kMlpThreads) {
      const int s = e / c_valid, c = e - s * c_valid;
      float acc = 0.f;
      if (b0 + s < B) {
        const float* p = partial + ((int64_t)(b0 + s) * splits) * c_valid + c;
        for (int sp = 0; sp < splits; ++sp) acc += p[(int64_t)sp * c_valid];
      }
      pooled[e] = acc * inv_r;
    }
  }
  __syncthreads();
  const bool vec = (c_valid % 4 == 0) && (C_full % 4 == 0) && ((reinterpret_cast<uintptr_t>(W1) & 15) == 0);
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int j = j0 + 2 * warp + u;
    if (j >= C_mlp) break;  // warp-uniform
    float acc[kSB];
#pragma unroll
    for (int s = 0; s < kSB; ++s) acc[s] = 0.f;
    const float* w = W1 + (int64_t)j * C_full;
    if (vec) {
      const float4* w4 = reinterpret_cast<const float4*>(w);
      const int n4 = c_valid >> 2;
#pragma unroll 8
      for (int c = lane; c < n4; c += 32) {
        const float4 wv = __ldg(w4 + c);
#pragma unroll
        for (int s = 0; s < kSB; ++s) {
          const float4 pv = reinterpret_cast<const float4*>(pooled + s * c_valid)[c];
          acc[s] = fmaf(wv.x, pv.x, acc[s]);
          acc[s] = fmaf(wv.y, pv.y, acc[s]);
          acc[s] = fmaf(wv.z, pv.z, acc[s]);
          acc[s] = fmaf(wv.w, pv.w, acc[s]);
        }
      }
    } else {
      for (int c = lane; c < c_valid; c += 32) {
        const float wv = __ldg(w + c);
#pragma unroll
        for (int s = 0; s < kSB; ++s) acc[s] = fmaf(wv, pooled[s * c_valid + c], acc[s]);
      }
    }
#pragma unroll
    for (int s = 0; s < kSB; ++s) {
      float v = acc[s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && b0 + s < B) hid[(int64_t)(b0 + s) * C_mlp + j] = fmaxf(v + (b1 ? b1[j] : 0.f), 0.f);
    }
  }
}

__global__ void __launch_bounds__(kMlpThreads)
gate_score_kernel(const float* __restrict__ hid, int B, int C_mlp, int T, const float* __restrict__ W2,
                  const float* __restrict__ b2, int32_t* __restrict__ idx_out, float* __restrict__ logits_out,
                  int32_t* status, int w2_in_smem) {
  extern __shared__ __align__(16) float w2s[];  // [T][C_mlp] when it fits
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (w2_in_smem) {  // one round of loads by the whole CTA instead of T dependent first touches per warp
    for (int e = threadIdx.x; e < T * C_mlp; e += kMlpThreads) w2s[e] = __ldg(W2 + e);
    __syncthreads();
  }
  const int b = blockIdx.x * (kMlpThreads / 32) + warp;
  if (b >= B) return;
  const float* h = hid + (int64_t)b * C_mlp;
  const float* wbase = w2_in_smem ? w2s : W2;
  int best = 0, nonfinite = 0;
  float best_v = 0.f;
  for (int t = 0; t < T; ++t) {
    const float* w = wbase + (int64_t)t * C_mlp;
    float v = 0.f;
    for (int j = lane; j < C_mlp; j += 32) v = fmaf(w[j], h[j], v);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    v += b2 ? b2[t] : 0.f;
    if (!isfinite(v)) ++nonfinite;
    if (t == 0) {
      best_v = v;
    } else if (v > best_v) {  // strict: ties keep the lower index
      best = t;
      best_v = v;
    }
    if (lane == 0 && logits_out) logits_out[(int64_t)b * T + t] = v;
  }
  if (lane == 0) {
    idx_out[b] = best;
    if (nonfinite) {
      dsn_set_status(status, DSN_ERR_NONFINITE, b);
      if (status) atomicAdd(status + 2, nonfinite);
    }
  }
}

}  // namespace

int dsn_gate_splits(const dsn_gate_desc& g, int sm_count) {
  // at most four 512-thread CTAs per SM (one resident wave), at least 8 rows per CTA
  int want = (4 * sm_count) / g.B;
  int max_by_rows = g.R / 8 > 0 ? g.R / 8 : 1;
  int s = want < max_by_rows ? want : max_by_rows;
  if (s < 1) s = 1;
  if (s > 64) s = 64;
  return s;
}

// scratch = partial[B][splits][c_valid] followed by hid[B][C_mlp] (floats)
cudaError_t dsn_launch_gate(const dsn_gate_desc& g, const void* x, int32_t* idx_out, float* logits_out,
                            float* partial, int splits, int32_t* status, cudaStream_t s) {
  dim3 grid(splits, g.B);
  float* hid = partial + (size_t)g.B * splits * g.c_valid;
  const bool vec = g.dtype == DSN_BF16 && (g.c_valid % 8 == 0) && (g.ldx % 8 == 0) &&
                   ((reinterpret_cast<uintptr_t>(x) & 15) == 0);
  if (vec) {
    const int nvec = g.c_valid / 8;
    int CT = 8;
    while (CT < nvec && CT < 128) CT <<= 1;
    pool_bf16_vec_kernel<<<grid, kPoolThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(x), g.R, g.ldx,
                                                        g.c_valid, splits, CT, partial);
  } else if (g.dtype == DSN_BF16) {
    pool_scalar_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(static_cast<const __nv_bfloat16*>(x), g.R, g.ldx,
                                                           g.c_valid, splits, partial);
  } else {
    pool_scalar_kernel<float><<<grid, 128, 0, s>>>(static_cast<const float*>(x), g.R, g.ldx, g.c_valid, splits,
                                                   partial);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = sizeof(float) * (size_t)kSB * g.c_valid;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(gate_hidden_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 hgrid((g.B + kSB - 1) / kSB, (g.C_mlp + kJB - 1) / kJB);
  gate_hidden_kernel<<<hgrid, kMlpThreads, smem, s>>>(partial, splits, g.B, g.R, g.C_full, g.c_valid, g.C_mlp, g.W1,
                                                      g.b1, hid);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int per_cta = kMlpThreads / 32;
  const size_t w2_bytes = sizeof(float) * (size_t)g.T * g.C_mlp;
  const int w2_in_smem = w2_bytes <= 40 * 1024;
  gate_score_kernel<<<(g.B + per_cta - 1) / per_cta, kMlpThreads, w2_in_smem ? w2_bytes : 0, s>>>(
      hid, g.B, g.C_mlp, g.T, g.W2, g.b2, idx_out, logits_out, status, w2_in_smem);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// dsn_gate_static: the gate for callers that cannot allocate device memory.
//
// The pooling partial sums normally live in a workspace the caller allocates.  Some callers have no
// allocator to ask: code running inside a region where cudaMalloc is forbidden or would stall the
// device (a latency-critical serving loop that must never touch the allocator, a plug-in that is
// handed only its input and output buffers, a process whose memory pool has been handed out in
// full).  For them the same kernels run with their scratch in a fixed array that is part of the
// loaded library image: 4 MiB per GPU that loads the library, held until the process exits.
// ------------------------------------------------------------------------------------------------
#define DSN_GATE_STATIC_MAX_FLOATS (1u << 20)

static __device__ __align__(256) float g_gate_static_scratch[DSN_GATE_STATIC_MAX_FLOATS];

namespace {
constexpr int kMaxDevices = 64;
float* g_static_scratch_ptr[kMaxDevices];  // device address of the array, per device, 0 = not looked up yet

// The array's name is only a host-side handle; kernels need its device address, which is looked up
// once per device while that device is current.
int static_scratch_address(int device, float** out) {
  if (device < 0 || device >= kMaxDevices) return DSN_ERR_INVALID_ARG;
  int current = -1;
  if (cudaGetDevice(&current) != cudaSuccess) return DSN_ERR_CUDA;
  if (current != device) return DSN_ERR_INVALID_ARG;
  if (!g_static_scratch_ptr[device]) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_gate_static_scratch) != cudaSuccess || !ptr)
      return DSN_ERR_CUDA;
    g_static_scratch_ptr[device] = ptr;
  }
  *out = g_static_scratch_ptr[device];
  return DSN_OK;
}
}  // namespace

extern "C" int dsn_gate_static(dsn_ctx* ctx, const dsn_gate_desc* g, const void* x, int32_t* idx_out,
                               float* logits_out, void* stream) {
  if (!ctx || !g || !x || !idx_out || !g->W1 || !g->W2) return DSN_ERR_INVALID_ARG;
  if (g->dtype != DSN_BF16 && g->dtype != DSN_F32) return DSN_ERR_INVALID_ARG;
  if (g->B < 0 || g->R < 1 || g->C_full < 1 || g->c_valid < 1 || g->c_valid > g->C_full || g->C_mlp < 1 ||
      g->T < 1 || g->T > DSN_MAX_SLICES || g->ldx < g->c_valid)
    return DSN_ERR_INVALID_ARG;
  if ((size_t)4 * kSB * (size_t)g->c_valid > 200 * 1024) return DSN_ERR_UNSUPPORTED;
  if (g->B == 0) return DSN_OK;
  const int splits = dsn_gate_splits(*g, ctx->sm_count);
  const size_t need = (size_t)g->B * splits * g->c_valid + (size_t)g->B * g->C_mlp;
  if (need > DSN_GATE_STATIC_MAX_FLOATS) return DSN_ERR_WORKSPACE;  // batch too large for the fixed scratch
  float* scratch = nullptr;
  const int e = static_scratch_address(ctx->device, &scratch);
  if (e != DSN_OK) return e;
  // every scratch value a later kernel reads is overwritten by an earlier one of the same call, so
  // nothing needs clearing
  if (dsn_launch_gate(*g, x, idx_out, logits_out, scratch, splits, ctx->d_status,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}
