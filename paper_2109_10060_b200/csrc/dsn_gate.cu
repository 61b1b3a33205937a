// Gate routing head (Sec. 3.5): average pooling over the R positions of each sample, a two-layer
// MLP (ReLU between), and the index of the first maximum score.
//
// Kernel 1 (HBM-bound): grid (splits, B), 512 threads.  A CTA streams a contiguous band of rows of
// one sample: consecutive threads read consecutive 16 bytes of a row, the CTA's row groups walk
// different rows, four loads are in flight per thread; fp32 accumulation in registers, one
// shared-memory reduction across the row groups, column sums to partial[b][split][c].  No atomics,
// so sums are reproducible run to run.
// Kernel 2 (latency-bound, plain FMA): grid (B/4 or B/8, C_mlp/16).  A CTA folds the partial sums of its
// samples (scaled by 1/R) into shared memory and computes 16 hidden units for them, one warp per
// two units, all weight loads of a 512-channel panel in flight at once; ReLU; hid[b][j] to scratch.
// Kernel 3 (tiny): one warp per sample, 32 / T lanes per path; arg-max by a strict '>' scan in
// ascending path order (ties keep the lowest index).
// Kernels 2 and 3 load their weights before they wait for the kernel ahead of them in the stream.
#include "dsn_internal.cuh"

namespace {

constexpr int kSBSmall = 4;        // samples per CTA in the hidden-layer kernel
constexpr int kSBLarge = 8;        // ... for large batches, where re-reading W1 per CTA would bound the kernel
constexpr int kSBLargeMinBatch = 512;  // batches from this size on take kSBLarge (measured: at B = 256 the larger form is slower)
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
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
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
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
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

// 16-byte load kept in program order (see ld_stream16) but allowed to stay in L1/L2
__device__ __forceinline__ float4 ld_ordered16(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// Hidden layer for kSB samples x kJB units per CTA.  The kernel is a chain of load latencies, so every
// load that can be issued early is: the loop over the input channels runs in panels of 512; a warp
// issues the 16-byte loads of its two weight rows for a panel (4 + 4 per lane) in one round, and those of
// the first panel BEFORE the wait for the pooling kernel (the weights are parameters, nothing in the stream
// writes them); the CTA then folds the pooling partial sums of the panel into shared memory (thread t owns
// 16-byte column t % 128 of every other sample; the loads of two samples x four splits are in flight
// together and nothing is divided); the FMAs run out of registers and shared memory.
constexpr int kPanel = 512;
template <int kSB>
__global__ void __launch_bounds__(kMlpThreads, 2)
gate_hidden_kernel(const float* __restrict__ partial, int splits, int B, int R, int C_full, int c_valid, int C_mlp,
                   const float* __restrict__ W1, const float* __restrict__ b1, float* __restrict__ hid) {
  __shared__ __align__(16) float pooled[kSB][kPanel];
  const int b0 = blockIdx.x * kSB, j0 = blockIdx.y * kJB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float inv_r = 1.0f / (float)R;
  const bool vec = (c_valid % 4 == 0) && (C_full % 4 == 0) && ((reinterpret_cast<uintptr_t>(W1) & 15) == 0);
  const int ja = j0 + 2 * warp, jb = ja + 1;
  float4 wa[4], wb[4];
  auto load_weights = [&](int cbase, int cw) {
    const float4* pa = reinterpret_cast<const float4*>(W1 + (int64_t)(ja < C_mlp ? ja : 0) * C_full + cbase);
    const float4* pb = reinterpret_cast<const float4*>(W1 + (int64_t)(jb < C_mlp ? jb : 0) * C_full + cbase);
    const int n4 = cw >> 2;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = lane + 32 * i;
      wa[i] = c < n4 ? ld_ordered16(pa + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      wb[i] = c < n4 ? ld_ordered16(pb + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  if (vec) load_weights(0, c_valid < kPanel ? c_valid : kPanel);
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  float acc[2][kSB];
#pragma unroll
  for (int u = 0; u < 2; ++u)
#pragma unroll
    for (int s = 0; s < kSB; ++s) acc[u][s] = 0.f;

  for (int cbase = 0; cbase < c_valid; cbase += kPanel) {
    const int cw = c_valid - cbase < kPanel ? c_valid - cbase : kPanel;  // panel width
    if (vec && cbase > 0) load_weights(cbase, cw);
    // fold the partial sums of this panel
    if (c_valid % 4 == 0) {
      const int n4 = cw >> 2, row4 = c_valid >> 2;
      const int c4 = tid & (kPanel / 4 - 1), s0 = tid / (kPanel / 4);  // kMlpThreads / (kPanel / 4) = 2 samples per round
      if (c4 < n4) {
#pragma unroll
        for (int u0 = 0; u0 < kSB / 2; u0 += 2) {  // two samples of this thread per round
          const int smp0 = b0 + s0 + 2 * u0, smp1 = smp0 + 2;
          const bool in0 = smp0 < B, in1 = smp1 < B;
          const float4* p0 = reinterpret_cast<const float4*>(partial + ((int64_t)(in0 ? smp0 : 0) * splits) * c_valid + cbase) + c4;
          const float4* p1 = reinterpret_cast<const float4*>(partial + ((int64_t)(in1 ? smp1 : 0) * splits) * c_valid + cbase) + c4;
          float4 sa = make_float4(0.f, 0.f, 0.f, 0.f), sb = sa;
          int sp = 0;
          for (; sp + 4 <= splits; sp += 4) {  // eight independent loads in flight
            float4 ta[4], tb[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) { ta[q] = __ldg(p0 + (int64_t)(sp + q) * row4); tb[q] = __ldg(p1 + (int64_t)(sp + q) * row4); }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              sa.x += ta[q].x; sa.y += ta[q].y; sa.z += ta[q].z; sa.w += ta[q].w;
              sb.x += tb[q].x; sb.y += tb[q].y; sb.z += tb[q].z; sb.w += tb[q].w;
            }
          }
          for (; sp < splits; ++sp) {
            const float4 ta = __ldg(p0 + (int64_t)sp * row4), tb = __ldg(p1 + (int64_t)sp * row4);
            sa.x += ta.x; sa.y += ta.y; sa.z += ta.z; sa.w += ta.w;
            sb.x += tb.x; sb.y += tb.y; sb.z += tb.z; sb.w += tb.w;
          }
          const float fa = in0 ? inv_r : 0.f, fb = in1 ? inv_r : 0.f;  // samples past the batch: zeros
          reinterpret_cast<float4*>(pooled[s0 + 2 * u0])[c4] = make_float4(sa.x * fa, sa.y * fa, sa.z * fa, sa.w * fa);
          reinterpret_cast<float4*>(pooled[s0 + 2 * u0 + 2])[c4] = make_float4(sb.x * fb, sb.y * fb, sb.z * fb, sb.w * fb);
        }
      }
    } else {
      for (int e = tid; e < kSB * cw; e += kMlpThreads) {
        const int s = e / cw, c = e - s * cw;
        float sum = 0.f;
        if (b0 + s < B) {
          const float* p = partial + ((int64_t)(b0 + s) * splits) * c_valid + cbase + c;
          for (int sp = 0; sp < splits; ++sp) sum += p[(int64_t)sp * c_valid];
        }
        pooled[s][c] = sum * inv_r;
      }
    }
    __syncthreads();
    if (vec) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int c = lane + 32 * i;
        if (c < (cw >> 2)) {
#pragma unroll
          for (int s = 0; s < kSB; ++s) {
            const float4 pv = reinterpret_cast<const float4*>(pooled[s])[c];
            acc[0][s] = fmaf(wa[i].x, pv.x, acc[0][s]); acc[0][s] = fmaf(wa[i].y, pv.y, acc[0][s]);
            acc[0][s] = fmaf(wa[i].z, pv.z, acc[0][s]); acc[0][s] = fmaf(wa[i].w, pv.w, acc[0][s]);
            acc[1][s] = fmaf(wb[i].x, pv.x, acc[1][s]); acc[1][s] = fmaf(wb[i].y, pv.y, acc[1][s]);
            acc[1][s] = fmaf(wb[i].z, pv.z, acc[1][s]); acc[1][s] = fmaf(wb[i].w, pv.w, acc[1][s]);
          }
        }
      }
    } else {
      for (int c = lane; c < cw; c += 32) {
        const float va = ja < C_mlp ? __ldg(W1 + (int64_t)ja * C_full + cbase + c) : 0.f;
        const float vb = jb < C_mlp ? __ldg(W1 + (int64_t)jb * C_full + cbase + c) : 0.f;
#pragma unroll
        for (int s = 0; s < kSB; ++s) {
          acc[0][s] = fmaf(va, pooled[s][c], acc[0][s]);
          acc[1][s] = fmaf(vb, pooled[s][c], acc[1][s]);
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int j = ja + u;
#pragma unroll
    for (int s = 0; s < kSB; ++s) {
      float v = acc[u][s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && j < C_mlp && b0 + s < B) hid[(int64_t)(b0 + s) * C_mlp + j] = fmaxf(v + (b1 ? b1[j] : 0.f), 0.f);
    }
  }
}

// Scores and arg-max: one warp per sample.  W2 ([T][C_mlp]) is staged in shared memory BEFORE the wait for
// the hidden-layer kernel (a parameter, written by nothing in the stream), the sample's hidden vector after
// it.  P = 32 / T (rounded down to a power of two, at least 1) lanes share the dot product of one path, each
// over every P-th hidden unit, and add their parts up in a fixed butterfly; the row pitch of W2 in shared
// memory is chosen so that the 32 lanes of a step hit 32 different banks.  Lane 0 then scans the T scores in
// ascending order with a strict '>' so that ties keep the lowest index.
__global__ void __launch_bounds__(kMlpThreads)
gate_score_kernel(const float* __restrict__ hid, int B, int C_mlp, int T, const float* __restrict__ W2,
                  const float* __restrict__ b2, int32_t* __restrict__ idx_out, float* __restrict__ logits_out,
                  int32_t* status) {
  extern __shared__ __align__(16) float sm[];
  int P = 1;
  while (2 * P * T <= 32) P <<= 1;
  const int pitch = C_mlp + ((P - C_mlp) & 31);      // pitch % 32 == P % 32: path t, part q -> bank (t P + q) % 32
  float* w2s = sm;                                   // [T][pitch]
  float* hs = w2s + (size_t)T * pitch;               // [warps][C_mlp]
  float* sc = hs + (size_t)(kMlpThreads / 32) * C_mlp;  // [warps][DSN_MAX_SLICES]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x * (kMlpThreads / 32) + warp;
  for (int t = warp; t < T; t += kMlpThreads / 32)
    for (int j = lane; j < C_mlp; j += 32) w2s[t * pitch + j] = __ldg(W2 + (int64_t)t * C_mlp + j);
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (b < B)
    for (int j = lane; j < C_mlp; j += 32) hs[warp * C_mlp + j] = hid[(int64_t)b * C_mlp + j];
  __syncthreads();
  if (b >= B) return;
  const float* h = hs + warp * C_mlp;
  const int part = lane & (P - 1), per_round = 32 / P;
  for (int t0 = 0; t0 < T; t0 += per_round) {
    const int t = t0 + lane / P;
    const float* w = w2s + (t < T ? t : 0) * pitch;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    int j = part;
    for (; j + 3 * P < C_mlp; j += 4 * P) {
      a0 = fmaf(w[j], h[j], a0); a1 = fmaf(w[j + P], h[j + P], a1);
      a2 = fmaf(w[j + 2 * P], h[j + 2 * P], a2); a3 = fmaf(w[j + 3 * P], h[j + 3 * P], a3);
    }
    for (; j < C_mlp; j += P) a0 = fmaf(w[j], h[j], a0);
    float v = (a0 + a1) + (a2 + a3);
    for (int o = P >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (part == 0 && t < T) {
      v += b2 ? b2[t] : 0.f;
      sc[warp * DSN_MAX_SLICES + t] = v;
      if (logits_out) logits_out[(int64_t)b * T + t] = v;
    }
  }
  __syncwarp();
  if (lane == 0) {
    const float* l = sc + warp * DSN_MAX_SLICES;
    int best = 0, nonfinite = 0;
    for (int t = 0; t < T; ++t) {
      if (!isfinite(l[t])) ++nonfinite;
      if (t > 0 && l[t] > l[best]) best = t;
    }
    idx_out[b] = best;
    if (nonfinite) {
      dsn_set_status(status, DSN_ERR_NONFINITE, b);
      if (status) atomicAdd(status + 2, nonfinite);
    }
  }
}

// Attention head (Sec. 3.5): scale[b][c] = 1 + tanh(b3[c] + sum_j W3[c][j] * hid[b][j]).  A CTA owns
// kSBSmall samples x 64 channels; their hidden vectors sit in shared memory, a warp walks 8 channels
// with its lanes across the C_mlp products (16-byte loads of the W3 row when C_mlp % 4 == 0).
__global__ void __launch_bounds__(kMlpThreads)
gate_attention_kernel(const float* __restrict__ hid, int B, int C_mlp, int C_full, int c_valid,
                      const float* __restrict__ W3, const float* __restrict__ b3, float* __restrict__ scale_out) {
  extern __shared__ __align__(16) float hs[];  // [kSBSmall][C_mlp]
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int b0 = blockIdx.x * kSBSmall, c0 = blockIdx.y * 64;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < kSBSmall * C_mlp; e += kMlpThreads) {
    const int s = e / C_mlp, j = e - s * C_mlp;
    hs[e] = (b0 + s < B) ? hid[(int64_t)(b0 + s) * C_mlp + j] : 0.f;
  }
  __syncthreads();
  const bool vec = (C_mlp % 4 == 0) && ((reinterpret_cast<uintptr_t>(W3) & 15) == 0);
  for (int u = 0; u < 8; ++u) {
    const int c = c0 + warp * 8 + u;
    if (c >= c_valid) break;  // warp-uniform
    float acc[kSBSmall];
#pragma unroll
    for (int s = 0; s < kSBSmall; ++s) acc[s] = 0.f;
    const float* w = W3 + (int64_t)c * C_mlp;
    if (vec) {
      for (int j4 = lane; j4 < (C_mlp >> 2); j4 += 32) {
        const float4 wv = __ldg(reinterpret_cast<const float4*>(w) + j4);
#pragma unroll
        for (int s = 0; s < kSBSmall; ++s) {
          const float4 hv = reinterpret_cast<const float4*>(hs + s * C_mlp)[j4];
          acc[s] = fmaf(wv.x, hv.x, acc[s]); acc[s] = fmaf(wv.y, hv.y, acc[s]);
          acc[s] = fmaf(wv.z, hv.z, acc[s]); acc[s] = fmaf(wv.w, hv.w, acc[s]);
        }
      }
    } else {
      for (int j = lane; j < C_mlp; j += 32) {
        const float wv = __ldg(w + j);
#pragma unroll
        for (int s = 0; s < kSBSmall; ++s) acc[s] = fmaf(wv, hs[s * C_mlp + j], acc[s]);
      }
    }
#pragma unroll
    for (int s = 0; s < kSBSmall; ++s) {
      float v = acc[s];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && b0 + s < B) scale_out[(int64_t)(b0 + s) * c_valid + c] = 1.f + tanhf(v + (b3 ? b3[c] : 0.f));
    }
  }
  (void)C_full;
}

// y = x * scale[sample][channel]; one CTA per (row band, sample); grouped output when perm is given.
template <typename Tio>
__global__ void __launch_bounds__(256)
scale_channels_kernel(const Tio* __restrict__ x, int64_t ldx, const float* __restrict__ scale, Tio* __restrict__ y,
                      int64_t ldy, int R, int c_valid, int bands, const int32_t* __restrict__ perm) {
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int pos = blockIdx.y, band = blockIdx.x;
  const int smp = perm ? perm[pos] : pos;   // output position pos holds sample smp
  if (smp < 0) return;
  const int r0 = (int)(((int64_t)R * band) / bands), r1 = (int)(((int64_t)R * (band + 1)) / bands);
  const Tio* xs = x + (int64_t)smp * R * ldx;
  Tio* ys = y + (int64_t)pos * R * ldy;
  const float* sc = scale + (int64_t)smp * c_valid;
  const int64_t total = (int64_t)(r1 - r0) * c_valid;
  for (int64_t e = threadIdx.x; e < total; e += 256) {
    const int r = r0 + (int)(e / c_valid), c = (int)(e % c_valid);
    ys[(int64_t)r * ldy + c] = (Tio)((float)xs[(int64_t)r * ldx + c] * __ldg(sc + c));
  }
}

// bf16, c_valid % 8 == 0, 16-byte aligned rows: eight channels per thread
__global__ void __launch_bounds__(256)
scale_channels_bf16_vec_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, const float* __restrict__ scale,
                               __nv_bfloat16* __restrict__ y, int64_t ldy, int R, int c_valid, int bands,
                               const int32_t* __restrict__ perm) {
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int pos = blockIdx.y, band = blockIdx.x;
  const int smp = perm ? perm[pos] : pos;
  if (smp < 0) return;
  const int r0 = (int)(((int64_t)R * band) / bands), r1 = (int)(((int64_t)R * (band + 1)) / bands);
  const int nvec = c_valid >> 3;
  const uint4* xs = reinterpret_cast<const uint4*>(x + (int64_t)smp * R * ldx);
  uint4* ys = reinterpret_cast<uint4*>(y + (int64_t)pos * R * ldy);
  const float* sc = scale + (int64_t)smp * c_valid;
  const int64_t total = (int64_t)(r1 - r0) * nvec, sx = ldx >> 3, sy = ldy >> 3;
  for (int64_t e = threadIdx.x; e < total; e += 256) {
    const int r = r0 + (int)(e / nvec), v = (int)(e % nvec);
    const uint4 in = __ldg(xs + (int64_t)r * sx + v);
    const float4 s0 = __ldg(reinterpret_cast<const float4*>(sc) + 2 * v), s1 = __ldg(reinterpret_cast<const float4*>(sc) + 2 * v + 1);
    const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = __uint_as_float(w[j] << 16) * sv[2 * j], b = __uint_as_float(w[j] & 0xffff0000u) * sv[2 * j + 1];
      __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
      o[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    ys[(int64_t)r * sy + v] = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// a_t = gamma / sigma_t, b_t = beta - gamma * mu_t / sigma_t
__global__ void resbn_fold_kernel(int n, int C, const float* __restrict__ gamma, const float* __restrict__ beta,
                                  const float* __restrict__ mu, const float* __restrict__ sigma,
                                  float* __restrict__ scale_out, float* __restrict__ shift_out) {
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  const int c = e % C;
  const float a = gamma[c] / sigma[e];
  scale_out[e] = a;
  shift_out[e] = fmaf(-a, mu[e], beta[c]);
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
    dsn_launch(pool_bf16_vec_kernel, grid, dim3(kPoolThreads), 0, s, 1, static_cast<const __nv_bfloat16*>(x), g.R,
               g.ldx, g.c_valid, splits, CT, partial);
  } else if (g.dtype == DSN_BF16) {
    dsn_launch(pool_scalar_kernel<__nv_bfloat16>, grid, dim3(128), 0, s, 1, static_cast<const __nv_bfloat16*>(x), g.R,
               g.ldx, g.c_valid, splits, partial);
  } else {
    dsn_launch(pool_scalar_kernel<float>, grid, dim3(128), 0, s, 1, static_cast<const float*>(x), g.R, g.ldx, g.c_valid,
               splits, partial);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (g.B >= kSBLargeMinBatch) {
    dim3 hgrid((g.B + kSBLarge - 1) / kSBLarge, (g.C_mlp + kJB - 1) / kJB);
    dsn_launch(gate_hidden_kernel<kSBLarge>, hgrid, dim3(kMlpThreads), 0, s, 1, (const float*)partial, splits, g.B, g.R,
               g.C_full, g.c_valid, g.C_mlp, g.W1, g.b1, hid);
  } else {
    dim3 hgrid((g.B + kSBSmall - 1) / kSBSmall, (g.C_mlp + kJB - 1) / kJB);
    dsn_launch(gate_hidden_kernel<kSBSmall>, hgrid, dim3(kMlpThreads), 0, s, 1, (const float*)partial, splits, g.B, g.R,
               g.C_full, g.c_valid, g.C_mlp, g.W1, g.b1, hid);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int per_cta = kMlpThreads / 32;
  const size_t smem = sizeof(float) * ((size_t)g.T * (g.C_mlp + 32) + (size_t)per_cta * g.C_mlp +
                                       (size_t)per_cta * DSN_MAX_SLICES);
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(gate_score_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dsn_launch(gate_score_kernel, dim3((g.B + per_cta - 1) / per_cta), dim3(kMlpThreads), smem, s, 1, (const float*)hid,
             g.B, g.C_mlp, g.T, g.W2, g.b2, idx_out, logits_out, status);
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
  if ((size_t)4 * ((size_t)g->T * (g->C_mlp + 32) + 8 * (size_t)g->C_mlp + 8 * DSN_MAX_SLICES) > 200 * 1024)
    return DSN_ERR_UNSUPPORTED;
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

cudaError_t dsn_launch_gate_attention(const dsn_gate_desc& g, const float* hid, const float* W3, const float* b3,
                                      float* scale_out, cudaStream_t s) {
  dim3 grid((g.B + kSBSmall - 1) / kSBSmall, (g.c_valid + 63) / 64);
  return dsn_launch(gate_attention_kernel, grid, dim3(kMlpThreads), sizeof(float) * kSBSmall * g.C_mlp, s, 1, hid, g.B,
                    g.C_mlp, g.C_full, g.c_valid, W3, b3, scale_out);
}

cudaError_t dsn_launch_scale_channels(int elem_bytes, int B, int R, int c_valid, const void* x, int64_t ldx,
                                      const float* scale, void* y, int64_t ldy, const int32_t* perm_or_null,
                                      cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  int bands = R / 16 > 0 ? R / 16 : 1;
  if (bands > 16) bands = 16;
  dim3 grid(bands, B);
  const bool vec = elem_bytes == 2 && c_valid % 8 == 0 && ldx % 8 == 0 && ldy % 8 == 0 &&
                   ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(scale)) & 15) == 0;
  if (vec)
    return dsn_launch(scale_channels_bf16_vec_kernel, grid, dim3(256), 0, s, 1, static_cast<const __nv_bfloat16*>(x), ldx,
                      scale, static_cast<__nv_bfloat16*>(y), ldy, R, c_valid, bands, perm_or_null);
  if (elem_bytes == 2)
    return dsn_launch(scale_channels_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, 1, static_cast<const __nv_bfloat16*>(x),
                      ldx, scale, static_cast<__nv_bfloat16*>(y), ldy, R, c_valid, bands, perm_or_null);
  return dsn_launch(scale_channels_kernel<float>, grid, dim3(256), 0, s, 1, static_cast<const float*>(x), ldx, scale,
                    static_cast<float*>(y), ldy, R, c_valid, bands, perm_or_null);
}

cudaError_t dsn_launch_resbn_fold(int n, int C, const float* gamma, const float* beta, const float* mu,
                                  const float* sigma, float* scale_out, float* shift_out, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  return dsn_launch(resbn_fold_kernel, dim3((n + 255) / 256), dim3(256), 0, s, 1, n, C, gamma, beta, mu, sigma, scale_out,
                    shift_out);
}
