// Slice-able depthwise convolution (MobileNet DSConv's first half), channels last, bf16 storage with
// fp32 arithmetic.  HBM-bound: a thread owns 8 consecutive channels (16 bytes) of one output pixel and
// walks the k x k taps of its sample's kernel size (the centred part of the K x K filter); neighbouring
// threads read neighbouring 16-byte pieces of a pixel, so every load and store is coalesced, and the
// re-reads of overlapping windows are served by L1/L2.  Filter layout [K][K][C] (channels last).
// A sample of path t uses channels < c[t] and kernel size ksize[t]; the rest is neither read nor written.
#include "dsn_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kPx = 3;   // output pixels of a row per thread on the 3 x 3 path (measured on the 14 x 14 x 640 block: 4 pixels and
                         // two CTAs per SM 72 us, 4 and three 62 us, 2 and four 59 us, 3 and four 58 us)

struct DwParams {
  int16_t c[DSN_MAX_SLICES];
  int8_t ksize[DSN_MAX_SLICES];
  int32_t H, W, Ho, Wo, K, stride, C, T, G, bands;
  int32_t x_input_order, y_input_order, act;
  const int32_t* offsets;
  const int32_t* perm;
  const int32_t* group_slice;
  const __nv_bfloat16* x;
  int64_t ldx;
  const __nv_bfloat16* w;
  const float* bias;
  const float* bn_scale;
  const float* bn_shift;
  __nv_bfloat16* y;
  int64_t ldy;
};

__device__ __forceinline__ float act_apply(float v, int act) {
  if (act == DSN_ACT_RELU) return fmaxf(v, 0.f);
  if (act == DSN_ACT_GELU) return 0.5f * v * (1.f + erff(v * 0.70710678118654752f));
  return v;
}

__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
// eight bf16 (16 bytes) -> four packed fp32 pairs
__device__ __forceinline__ void widen8(const uint4& v, uint64_t (&o)[4]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) o[j] = pack2(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xffff0000u));
}

// 3 x 3 fast path: a thread owns 8 channels of kPx neighbouring output pixels of one output row.  Per filter row it
// requests the 3 + (kPx - 1) * STRIDE input vectors the windows cover and the row's three filter vectors in one round,
// widens each once and feeds every window it belongs to (a sliding window in registers): a third of the loads and of
// the widening work of one pixel per thread, and packed fp32 FMAs (two channels per instruction).
template <int STRIDE>
__device__ __forceinline__ void depthwise3x3_rows(const DwParams& p, const __nv_bfloat16* xs, __nv_bfloat16* ys, int ct,
                                                  const float* sc, const float* sh, int row0, int row1) {
  constexpr int NCOL = 3 + (kPx - 1) * STRIDE;
  const int nvec = ct >> 3, quads = (p.Wo + kPx - 1) / kPx;
  const int k0 = (p.K - 3) >> 1;
  const int64_t total = (int64_t)(row1 - row0) * quads * nvec;
  for (int64_t e = threadIdx.x; e < total; e += kThreads) {
    const int v = (int)(e % nvec);
    const int qi = (int)(e / nvec);
    const int oy = row0 + qi / quads, ox0 = kPx * (qi % quads);
    const int c0 = 8 * v;
    const int npx = p.Wo - ox0 < kPx ? p.Wo - ox0 : kPx;
    uint64_t acc[kPx][4];
#pragma unroll
    for (int px = 0; px < kPx; ++px)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[px][j] = 0ull;
    const int ix0 = ox0 * STRIDE - 1;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int iy = oy * STRIDE - 1 + r;
      if (iy < 0 || iy >= p.H) continue;   // the padding rows contribute nothing
      uint4 xv[NCOL], wv[3];
#pragma unroll
      for (int j = 0; j < NCOL; ++j) {
        const int ix = ix0 + j;
        const bool need = ix >= 0 && ix < p.W && j <= (npx - 1) * STRIDE + 2;
        xv[j] = need ? __ldg(reinterpret_cast<const uint4*>(xs + ((int64_t)iy * p.W + ix) * p.ldx + c0)) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int t = 0; t < 3; ++t)
        wv[t] = __ldg(reinterpret_cast<const uint4*>(p.w + ((int64_t)(k0 + r) * p.K + (k0 + t)) * p.C + c0));
      uint64_t wf[3][4];
#pragma unroll
      for (int t = 0; t < 3; ++t) widen8(wv[t], wf[t]);
#pragma unroll
      for (int j = 0; j < NCOL; ++j) {
        uint64_t xf[4];
        widen8(xv[j], xf);
#pragma unroll
        for (int px = 0; px < kPx; ++px) {
          const int t = j - px * STRIDE;   // which tap of window px this input column is
          if (t >= 0 && t < 3) {
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[px][q] = ffma2(xf[q], wf[t][q], acc[px][q]);
          }
        }
      }
    }
#pragma unroll
    for (int px = 0; px < kPx; ++px) {
      if (px < npx) {
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float a, b;
          unpack2(acc[px][j], a, b);
          const int ca = c0 + 2 * j, cb = ca + 1;
          if (p.bias) { a += p.bias[ca]; b += p.bias[cb]; }
          if (sc) { a = fmaf(a, sc[ca], sh[ca]); b = fmaf(b, sc[cb], sh[cb]); }
          __nv_bfloat162 h = __floats2bfloat162_rn(act_apply(a, p.act), act_apply(b, p.act));
          o[j] = *reinterpret_cast<uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(ys + ((int64_t)oy * p.Wo + ox0 + px) * p.ldy + c0) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads, 4) depthwise_kernel(const __grid_constant__ DwParams p) {
  __shared__ int s_info[3];  // slice, sample, valid
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  const int pos = blockIdx.y, band = blockIdx.x;
  // The group of this position: thread g tests group g (one round of loads instead of a binary search's chain of
  // dependent ones), another thread fetches the sample index at the same time.
  if (threadIdx.x < 3) s_info[threadIdx.x] = 0;
  __syncthreads();
  for (int g = threadIdx.x; g < p.G; g += kThreads) {
    const int lo = p.offsets[g], hi = p.offsets[g + 1];
    if (lo <= pos && pos < hi) {
      const int sl = p.group_slice ? p.group_slice[g] : g;
      s_info[0] = sl;
      s_info[2] = (sl >= 0 && sl < p.T) ? 1 : 0;
    }
  }
  if (threadIdx.x == kThreads - 1) s_info[1] = p.perm[pos];
  __syncthreads();
  if (s_info[1] < 0) return;
  if (!s_info[2]) return;
  const int sl = s_info[0], smp = s_info[1];
  const int ct = p.c[sl], k = p.ksize[sl];
  const int k0 = (p.K - k) >> 1, pad = (k - 1) >> 1;
  const __nv_bfloat16* xs = p.x + (int64_t)(p.x_input_order ? smp : pos) * p.H * p.W * p.ldx;
  __nv_bfloat16* ys = p.y + (int64_t)(p.y_input_order ? smp : pos) * p.Ho * p.Wo * p.ldy;
  const float* sc = p.bn_scale ? p.bn_scale + (int64_t)sl * p.C : nullptr;
  const float* sh = p.bn_scale ? p.bn_shift + (int64_t)sl * p.C : nullptr;
  const int nvec = (ct + 7) >> 3;
  const int pix0 = (int)(((int64_t)p.Ho * p.Wo * band) / p.bands), pix1 = (int)(((int64_t)p.Ho * p.Wo * (band + 1)) / p.bands);
  const bool vec_ok = (p.ldx % 8 == 0) && (p.ldy % 8 == 0) && (p.C % 8 == 0) &&
                      ((reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.y) | reinterpret_cast<uintptr_t>(p.w)) & 15) == 0;
  if (k == 3 && vec_ok && (ct & 7) == 0) {   // whole output rows per band
    const int row0 = (int)(((int64_t)p.Ho * band) / p.bands), row1 = (int)(((int64_t)p.Ho * (band + 1)) / p.bands);
    if (p.stride == 1) depthwise3x3_rows<1>(p, xs, ys, ct, sc, sh, row0, row1);
    else depthwise3x3_rows<2>(p, xs, ys, ct, sc, sh, row0, row1);
    return;
  }
  for (int64_t e = threadIdx.x; e < (int64_t)(pix1 - pix0) * nvec; e += kThreads) {
    const int pix = pix0 + (int)(e / nvec), v = (int)(e % nvec);
    const int yy = pix / p.Wo, xx = pix - yy * p.Wo;
    const int c0 = v * 8;
    const int nch = ct - c0 < 8 ? ct - c0 : 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (k == 3 && vec_ok && nch == 8) {
      // 3 x 3: all nine input vectors and filter vectors are requested before the first one is used, so the
      // thread waits for memory once per output, not once per tap; out-of-image taps read as zeros
      const int iy0 = yy * p.stride - 1, ix0 = xx * p.stride - 1;
      uint4 xv[9], wv[9];
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) {
        const int iy = iy0 + tap / 3, ix = ix0 + tap % 3;
        xv[tap] = (iy >= 0 && iy < p.H && ix >= 0 && ix < p.W)
                      ? __ldg(reinterpret_cast<const uint4*>(xs + ((int64_t)iy * p.W + ix) * p.ldx + c0))
                      : make_uint4(0u, 0u, 0u, 0u);
        wv[tap] = __ldg(reinterpret_cast<const uint4*>(p.w + ((int64_t)(k0 + tap / 3) * p.K + (k0 + tap % 3)) * p.C + c0));
      }
#pragma unroll
      for (int tap = 0; tap < 9; ++tap) {
        const uint32_t xa[4] = {xv[tap].x, xv[tap].y, xv[tap].z, xv[tap].w}, wa[4] = {wv[tap].x, wv[tap].y, wv[tap].z, wv[tap].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] = fmaf(__uint_as_float(xa[j] << 16), __uint_as_float(wa[j] << 16), acc[2 * j]);
          acc[2 * j + 1] = fmaf(__uint_as_float(xa[j] & 0xffff0000u), __uint_as_float(wa[j] & 0xffff0000u), acc[2 * j + 1]);
        }
      }
    } else
    for (int r = 0; r < k; ++r) {
      const int iy = yy * p.stride + r - pad;
      if (iy < 0 || iy >= p.H) continue;
      for (int s = 0; s < k; ++s) {
        const int ix = xx * p.stride + s - pad;
        if (ix < 0 || ix >= p.W) continue;
        const __nv_bfloat16* xp = xs + ((int64_t)iy * p.W + ix) * p.ldx + c0;
        const __nv_bfloat16* wp = p.w + ((int64_t)(k0 + r) * p.K + (k0 + s)) * p.C + c0;
        if (vec_ok && nch == 8) {
          const uint4 xv = __ldg(reinterpret_cast<const uint4*>(xp)), wv = __ldg(reinterpret_cast<const uint4*>(wp));
          const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w}, wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            acc[2 * j] = fmaf(__uint_as_float(xa[j] << 16), __uint_as_float(wa[j] << 16), acc[2 * j]);
            acc[2 * j + 1] = fmaf(__uint_as_float(xa[j] & 0xffff0000u), __uint_as_float(wa[j] & 0xffff0000u), acc[2 * j + 1]);
          }
        } else {
          for (int j = 0; j < nch; ++j) acc[j] = fmaf(__bfloat162float(xp[j]), __bfloat162float(wp[j]), acc[j]);
        }
      }
    }
    __nv_bfloat16* yp = ys + (int64_t)pix * p.ldy + c0;
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float a = acc[2 * j], b = acc[2 * j + 1];
      const int ca = c0 + 2 * j, cb = ca + 1;
      if (p.bias) { if (ca < ct) a += p.bias[ca]; if (cb < ct) b += p.bias[cb]; }
      if (sc) { if (ca < ct) a = fmaf(a, sc[ca], sh[ca]); if (cb < ct) b = fmaf(b, sc[cb], sh[cb]); }
      __nv_bfloat162 h = __floats2bfloat162_rn(act_apply(a, p.act), act_apply(b, p.act));
      o[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    if (vec_ok && nch == 8) {
      *reinterpret_cast<uint4*>(yp) = make_uint4(o[0], o[1], o[2], o[3]);
    } else {
      for (int j = 0; j < nch; ++j)
        reinterpret_cast<uint16_t*>(yp)[j] = (j & 1) ? (uint16_t)(o[j >> 1] >> 16) : (uint16_t)(o[j >> 1] & 0xffffu);
    }
  }
}

}  // namespace

cudaError_t dsn_launch_depthwise(const int32_t* c, const int32_t* ksize, int T, int H, int W, int K, int stride, int C,
                                 int B, int G, const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                 int x_input_order, int y_input_order, const void* x, int64_t ldx, const void* w,
                                 const float* bias, const float* bn_scale, const float* bn_shift, int act, void* y,
                                 int64_t ldy, cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  DwParams p;
  memset(&p, 0, sizeof(p));
  for (int t = 0; t < T; ++t) {
    p.c[t] = (int16_t)c[t];
    p.ksize[t] = (int8_t)ksize[t];
  }
  p.H = H; p.W = W; p.K = K; p.stride = stride; p.C = C; p.T = T; p.G = G;
  p.Ho = (H - 1) / stride + 1; p.Wo = (W - 1) / stride + 1;
  // about eight (pixel, 8-channel) outputs per thread: many small CTAs fill the SMs more evenly than few long-running
  // ones, but every CTA pays its group lookup (measured on 14 x 14 x 640, 256 samples: 3 bands 61 us, 7 bands 55 us,
  // 14 bands 58 us)
  int bands = (int)(((int64_t)p.Ho * p.Wo * ((C + 7) / 8)) / (8 * kThreads));
  if (bands < 1) bands = 1;
  if (bands > p.Ho) bands = p.Ho;   // bands are whole output rows on the 3 x 3 fast path
  if (bands > 64) bands = 64;
  p.bands = bands;
  p.x_input_order = x_input_order; p.y_input_order = y_input_order; p.act = act;
  p.offsets = offsets; p.perm = perm; p.group_slice = group_slice;
  p.x = static_cast<const __nv_bfloat16*>(x); p.ldx = ldx;
  p.w = static_cast<const __nv_bfloat16*>(w);
  p.bias = bias; p.bn_scale = bn_scale; p.bn_shift = bn_shift;
  p.y = static_cast<__nv_bfloat16*>(y); p.ldy = ldy;
  return dsn_launch(depthwise_kernel, dim3(bands, B), dim3(kThreads), 0, s, 1, p);
}
