// Gate routing head (Sec. 3.5): average pooling over the R positions of each sample, a two-layer
// MLP (ReLU between), and the index of the first maximum score.
//
// Kernel 1 (HBM-bound): grid (splits, B).  A CTA streams a contiguous band of rows of one sample
// with 16-byte loads (consecutive threads read consecutive 16 bytes of a row) and accumulates in
// fp32 registers; its column sums go to partial[b][split][c].  No atomics, so sums are
// reproducible run to run.
// Kernel 2 (tiny, plain FMA): a CTA owns kSB samples; it folds the partial sums, scales by 1/R,
// and evaluates both FC layers with one warp per output unit (lanes stride the reduction,
// shuffle reduce), then one thread per sample takes the arg-max with a strict '>' scan.
#include "dsn_internal.cuh"

namespace {

constexpr int kSB = 4;            // samples per CTA in the MLP kernel
constexpr int kPoolThreads = 128;
constexpr int kMlpThreads = 256;

__device__ __forceinline__ void add8(float (&acc)[8], const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    acc[2 * j] += __uint_as_float(w[j] << 16);
    acc[2 * j + 1] += __uint_as_float(w[j] & 0xffff0000u);
  }
}

// bf16 input, c_valid % 8 == 0, ldx % 8 == 0, x 16-byte aligned
__global__ void __launch_bounds__(kPoolThreads)
pool_bf16_vec_kernel(const __nv_bfloat16* __restrict__ x, int R, int64_t ldx, int c_valid, int splits,
                     float* __restrict__ partial) {
  const int b = blockIdx.y, sp = blockIdx.x;
  const int r0 = (int)(((int64_t)R * sp) / splits), r1 = (int)(((int64_t)R * (sp + 1)) / splits);
  const int nvec = c_valid >> 3;
  const __nv_bfloat16* xb = x + (int64_t)b * R * ldx;
  float* out = partial + ((int64_t)b * splits + sp) * c_valid;
  for (int v = threadIdx.x; v < nvec; v += kPoolThreads) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const uint4* col = reinterpret_cast<const uint4*>(xb + (int64_t)r0 * ldx) + v;
    const int64_t stride = ldx >> 3;  // in uint4
    int r = r0;
    for (; r + 4 <= r1; r += 4) {     // four independent loads in flight per thread
      const uint4 a0 = __ldg(col), a1 = __ldg(col + stride), a2 = __ldg(col + 2 * stride),
                  a3 = __ldg(col + 3 * stride);
      add8(acc, a0); add8(acc, a1); add8(acc, a2); add8(acc, a3);
      col += 4 * stride;
    }
    for (; r < r1; ++r) {
      add8(acc, __ldg(col));
      col += stride;
    }
    float4* o = reinterpret_cast<float4*>(out + 8 * v);
    o[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    o[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
}

// any dtype / any width: one channel per thread
template <typename Tin>
__global__ void __launch_bounds__(kPoolThreads)
pool_scalar_kernel(const Tin* __restrict__ x, int R, int64_t ldx, int c_valid, int splits,
                   float* __restrict__ partial) {
  const int b = blockIdx.y, sp = blockIdx.x;
  const int r0 = (int)(((int64_t)R * sp) / splits), r1 = (int)(((int64_t)R * (sp + 1)) / splits);
  const Tin* xb = x + (int64_t)b * R * ldx;
  float* out = partial + ((int64_t)b * splits + sp) * c_valid;
  for (int c = threadIdx.x; c < c_valid; c += kPoolThreads) {
    float acc = 0.f;
    for (int r = r0; r < r1; ++r) acc += (float)xb[(int64_t)r * ldx + c];
    out[c] = acc;
  }
}

__global__ void __launch_bounds__(kMlpThreads)
gate_mlp_kernel(const float* __restrict__ partial, int splits, int B, int R, int C_full, int c_valid, int C_mlp,
                int T, const float* __restrict__ W1, const float* __restrict__ b1,
                const float* __restrict__ W2, const float* __restrict__ b2, int32_t* __restrict__ idx_out,
                float* __restrict__ logits_out, int32_t* status) {
  extern __shared__ float smem[];
  float* pooled = smem;                        // [kSB][c_valid]
  float* hid = pooled + kSB * c_valid;         // [kSB][C_mlp]
  float* logit = hid + kSB * C_mlp;            // [kSB][T]
  const int b0 = blockIdx.x * kSB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kMlpThreads / 32;
  const float inv_r = 1.0f / (float)R;

  for (int e = tid; e < kSB * c_valid; e += kMlpThreads) {
    const int s = e / c_valid, c = e - s * c_valid;
    float acc = 0.f;
    if (b0 + s < B) {
      const float* p = partial + ((int64_t)(b0 + s) * splits) * c_valid + c;
      for (int sp = 0; sp < splits; ++sp) acc += p[(int64_t)sp * c_valid];
    }
    pooled[e] = acc * inv_r;
  }
  __syncthreads();

  for (int j = warp; j < C_mlp; j += nwarp) {
    float acc[kSB];
#pragma unroll
    for (int s = 0; s < kSB; ++s) acc[s] = 0.f;
    const float* w = W1 + (int64_t)j * C_full;
    for (int c = lane; c < c_valid; c += 32) {
      const float wv = __ldg(w + c);
#pragma unroll
      for (int s = 0; s < kSB; ++s) acc[s] = fmaf(wv, pooled[s * c_valid + c], acc[s]);
    }
#pragma unroll
    for (int s = 0; s < kSB; ++s) {
      float v = acc[s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) hid[s * C_mlp + j] = fmaxf(v + (b1 ? b1[j] : 0.f), 0.f);
    }
  }
  __syncthreads();

  for (int t = warp; t < T; t += nwarp) {
    float acc[kSB];
#pragma unroll
    for (int s = 0; s < kSB; ++s) acc[s] = 0.f;
    const float* w = W2 + (int64_t)t * C_mlp;
    for (int j = lane; j < C_mlp; j += 32) {
      const float wv = __ldg(w + j);
#pragma unroll
      for (int s = 0; s < kSB; ++s) acc[s] = fmaf(wv, hid[s * C_mlp + j], acc[s]);
    }
#pragma unroll
    for (int s = 0; s < kSB; ++s) {
      float v = acc[s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) logit[s * T + t] = v + (b2 ? b2[t] : 0.f);
    }
  }
  __syncthreads();

  if (tid < kSB && b0 + tid < B) {
    const float* l = logit + tid * T;
    int best = 0, nonfinite = 0;
    for (int t = 0; t < T; ++t) {
      if (!isfinite(l[t])) ++nonfinite;
      if (t > 0 && l[t] > l[best]) best = t;
      if (logits_out) logits_out[(int64_t)(b0 + tid) * T + t] = l[t];
    }
    idx_out[b0 + tid] = best;
    if (nonfinite) {
      dsn_set_status(status, DSN_ERR_NONFINITE, b0 + tid);
      if (status) atomicAdd(status + 2, nonfinite);
    }
  }
}

}  // namespace

int dsn_gate_splits(const dsn_gate_desc& g, int sm_count) {
  // enough CTAs to fill the machine about four times over, at least 8 rows per CTA
  int want = (4 * sm_count + g.B - 1) / g.B;
  int max_by_rows = g.R / 8 > 0 ? g.R / 8 : 1;
  int s = want < max_by_rows ? want : max_by_rows;
  if (s < 1) s = 1;
  if (s > 64) s = 64;
  return s;
}

cudaError_t dsn_launch_gate(const dsn_gate_desc& g, const void* x, int32_t* idx_out, float* logits_out,
                            float* partial, int splits, int32_t* status, cudaStream_t s) {
  dim3 grid(splits, g.B);
  const bool vec = g.dtype == DSN_BF16 && (g.c_valid % 8 == 0) && (g.ldx % 8 == 0) &&
                   ((reinterpret_cast<uintptr_t>(x) & 15) == 0);
  if (vec) {
    pool_bf16_vec_kernel<<<grid, kPoolThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(x), g.R, g.ldx,
                                                        g.c_valid, splits, partial);
  } else if (g.dtype == DSN_BF16) {
    pool_scalar_kernel<__nv_bfloat16><<<grid, kPoolThreads, 0, s>>>(static_cast<const __nv_bfloat16*>(x), g.R,
                                                                    g.ldx, g.c_valid, splits, partial);
  } else {
    pool_scalar_kernel<float><<<grid, kPoolThreads, 0, s>>>(static_cast<const float*>(x), g.R, g.ldx, g.c_valid,
                                                            splits, partial);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = sizeof(float) * (size_t)kSB * (g.c_valid + g.C_mlp + g.T);
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(gate_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  gate_mlp_kernel<<<(g.B + kSB - 1) / kSB, kMlpThreads, smem, s>>>(partial, splits, g.B, g.R, g.C_full, g.c_valid,
                                                                  g.C_mlp, g.T, g.W1, g.b1, g.W2, g.b2, idx_out,
                                                                  logits_out, status);
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
  if ((size_t)4 * kSB * ((size_t)g->c_valid + g->C_mlp + g->T) > 200 * 1024) return DSN_ERR_UNSUPPORTED;
  if (g->B == 0) return DSN_OK;
  const int splits = dsn_gate_splits(*g, ctx->sm_count);
  const size_t need = (size_t)g->B * splits * g->c_valid;
  if (need > DSN_GATE_STATIC_MAX_FLOATS) return DSN_ERR_WORKSPACE;  // batch too large for the fixed scratch
  float* scratch = nullptr;
  const int e = static_scratch_address(ctx->device, &scratch);
  if (e != DSN_OK) return e;
  // every partial sum the second kernel reads is overwritten by the first one, so nothing needs clearing
  if (dsn_launch_gate(*g, x, idx_out, logits_out, scratch, splits, ctx->d_status,
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}
