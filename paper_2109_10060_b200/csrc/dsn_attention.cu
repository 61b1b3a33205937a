// Slimmable self-attention core (Sec. 3.4): for a sample routed to a path with h heads,
//   A_a = Softmax(Q_a K_a^T / sqrt(D_h)) V_a,  a < h,   out = Concat(A_0 .. A_{h-1}).
//
// Input is the output of the fused, head-major QKV layer: row r of a sample holds [head][q|k|v][64];
// the output row holds [head][64] and feeds the sliced projection (k_in = h * 64).  Heads >= h of a
// sample are neither read nor written.
//
// One CTA (128 threads) per (sample, head), N <= 256 tokens, D_h = 64:
//   K [256 keys][64] and Q [128 queries][64] arrive by TMA (K-major, 128-byte swizzle);
//   V is transposed by the threads into V^T [64][256 keys] in the same swizzled K-major layout
//   (keys >= N are written as zeros);
//   S = Q K^T: tcgen05.mma M = 128, N = keys rounded to 16, K = 64, fp32 in TMEM;
//   every thread owns one query row: two passes over its S row in TMEM (row maximum; exponentials,
//   row sum, P as bf16 into a swizzled K-major shared-memory tile, keys >= N as zeros);
//   O = P V: tcgen05.mma M = 128, N = 64, K = keys rounded to 16; the row is scaled by 1 / sum,
//   rounded to bf16 and stored as one 128-byte line.
// The two 128-query halves of the sample run one after the other.  Waits are bounded as in the GEMM.
#include "dsn_gemm_device.cuh"

namespace {

using namespace dsn_gemm;

constexpr int kAttThreads = 128;
constexpr uint32_t kQBytes = 128 * 128;       // 128 queries x 64 bf16
constexpr uint32_t kKBytes = 256 * 128;       // 256 keys x 64 bf16
constexpr uint32_t kVtBytes = 4 * 64 * 128;   // 4 key chunks x 64 (d) rows x 64 keys bf16
constexpr uint32_t kPBytes = 4 * 128 * 128;   // 4 key chunks x 128 queries x 64 keys bf16

struct AttParams {
  CUtensorMap map;        // qkv seen as [rows][3H][64], box 128 rows x 1 x 64
  int8_t heads[DSN_MAX_SLICES];
  int32_t N, H, B, G, T;
  int32_t grouped;        // 1: position p holds its data at row block p; 0: at row block perm[p]
  const int32_t* offsets;
  const int32_t* perm;
  const int32_t* group_slice;
  const __nv_bfloat16* qkv;
  int64_t ld_qkv;
  __nv_bfloat16* out;
  int64_t ld_out;
  int32_t* status;
};

__device__ __forceinline__ int find_group_of(const int32_t* __restrict__ offsets, int G, int p) {
  int lo = 0, hi = G;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (offsets[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kAttThreads, 1) attention_kernel(const __grid_constant__ AttParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  // layout: control 1 KB | Q 16 KB | K 32 KB | V^T 32 KB | P 64 KB
  const uint32_t bar_load = base, bar_mma = base + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 20);
  int32_t* s_info = reinterpret_cast<int32_t*>(smem + 24);  // [0] heads of this sample, [1] row block
  const uint32_t q_s = base + 1024, k_s = q_s + kQBytes, vt_s = k_s + kKBytes, p_s = vt_s + kVtBytes;
  uint8_t* vt_ptr = smem + 1024 + kQBytes + kKBytes;
  uint8_t* p_ptr = vt_ptr + kVtBytes;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int head = blockIdx.x, pos = blockIdx.y;

  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (tid == 0) {
    int h = 0, blk = 0;
    if (pos < p.offsets[p.G]) {
      const int g = find_group_of(p.offsets, p.G, pos);
      const int sl = p.group_slice ? p.group_slice[g] : g;
      if (sl >= 0 && sl < p.T) h = p.heads[sl];
      blk = p.grouped ? pos : p.perm[pos];
      if (blk < 0) h = 0;
    }
    s_info[0] = h;
    s_info[1] = blk;
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (head >= s_info[0]) return;  // this sample's path has fewer heads (uniform over the CTA)
  const int N = p.N;
  const int64_t row0 = (int64_t)s_info[1] * N;
  const int npad = (N + 15) & ~15;  // keys rounded to the MMA's K step / N granule

  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  if (tid == 0) {  // K (two boxes of 128 keys) and the first 128 queries
    mbar_expect_tx(bar_load, kKBytes + kQBytes);
    tma_load_3d(k_s, &p.map, 0, head * 3 + 1, (int)row0, bar_load);
    tma_load_3d(k_s + 128 * 128, &p.map, 0, head * 3 + 1, (int)row0 + 128, bar_load);
    tma_load_3d(q_s, &p.map, 0, head * 3 + 0, (int)row0, bar_load);
  }
  // V^T: element (d, key) -> chunk key/64, row d, 16-byte piece (key%64)/8 XOR (d & 7), slot key % 8
  {
    const __nv_bfloat16* vsrc = p.qkv + row0 * p.ld_qkv + (int64_t)(head * 3 + 2) * 64;
    for (int e = tid; e < 256 * 8; e += kAttThreads) {  // (key, group of 8 d)
      const int key = e >> 3, d8 = e & 7;
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      if (key < N) val = __ldg(reinterpret_cast<const uint4*>(vsrc + (int64_t)key * p.ld_qkv) + d8);
      const uint32_t w[4] = {val.x, val.y, val.z, val.w};
      const int kc = key >> 6, kk = key & 63;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int d = d8 * 8 + i;
        const uint16_t bits = (i & 1) ? (uint16_t)(w[i >> 1] >> 16) : (uint16_t)(w[i >> 1] & 0xffffu);
        *reinterpret_cast<uint16_t*>(vt_ptr + kc * 8192 + d * 128 + (((kk >> 3) ^ (d & 7)) << 4) + (kk & 7) * 2) = bits;
      }
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 256;
  const uint32_t idesc_s = make_idesc(128, npad), idesc_o = make_idesc(128, 64);
  const float sl2 = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
  bool ok = true;
  uint32_t load_phase = 0, mma_phase = 0;

  for (int half = 0; half < 2 && ok; ++half) {
    if (half * 128 >= N) break;
    if (half == 1) {  // second 128 queries into the same buffer (the S MMA that read it has completed)
      if (tid == 0) {
        mbar_expect_tx(bar_load, kQBytes);
        tma_load_3d(q_s, &p.map, 0, head * 3 + 0, (int)row0 + 128, bar_load);
      }
    }
    // ---- S = Q K^T
    if (tid == 0) {
      if (mbar_wait(bar_load, load_phase, abort_flag, p.status, 21)) {
        tc_fence_after();
        const uint64_t dq = make_smem_desc(q_s), dk = make_smem_desc(k_s);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) umma_bf16(tmem_S, dq + 2u * ks, dk + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
        umma_commit(bar_mma);
      }
    }
    load_phase ^= 1u;
    ok = __syncthreads_and(mbar_wait(bar_mma, mma_phase, abort_flag, p.status, 22) ? 1 : 0) != 0;
    mma_phase ^= 1u;
    if (!ok) break;
    tc_fence_after();

    // ---- softmax of this thread's query row; P (bf16) into the swizzled K-major tile
    const int m = warp * 32 + lane;  // accumulator row = TMEM lane
    const uint32_t trow = tmem_S + ((uint32_t)(warp * 32) << 16);
    float mx = -INFINITY;
    for (int c0 = 0; c0 < npad; c0 += 32) {
      uint32_t v[32];
      tmem_ld_32x32(trow + c0, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (c0 + i < N) mx = fmaxf(mx, __uint_as_float(v[i]));
    }
    float sum = 0.f;
    for (int c0 = 0; c0 < npad; c0 += 32) {
      uint32_t v[32];
      tmem_ld_32x32(trow + c0, v);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = 8 * j + 2 * e;
          float a = 0.f, b = 0.f;
          if (c0 + c < N) a = exp2f((__uint_as_float(v[c]) - mx) * sl2);
          if (c0 + c + 1 < N) b = exp2f((__uint_as_float(v[c + 1]) - mx) * sl2);
          __nv_bfloat162 hb = __floats2bfloat162_rn(a, b);
          // the row sum uses the rounded probabilities, the values the second MMA multiplies
          sum += __low2float(hb) + __high2float(hb);
          w[e] = *reinterpret_cast<uint32_t*>(&hb);
        }
        const int key = c0 + 8 * j;
        if (key < npad)
          *reinterpret_cast<uint4*>(p_ptr + (key >> 6) * 16384 + m * 128 + ((((key & 63) >> 3) ^ (m & 7)) << 4)) =
              make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();

    // ---- O = P V
    if (tid == 0) {
      tc_fence_after();
      for (int ks = 0; ks < npad / 16; ++ks) {
        const uint64_t dp = make_smem_desc(p_s + (ks >> 2) * 16384) + 2u * (ks & 3);
        const uint64_t dv = make_smem_desc(vt_s + (ks >> 2) * 8192) + 2u * (ks & 3);
        umma_bf16(tmem_O, dp, dv, idesc_o, ks > 0 ? 1u : 0u);
      }
      umma_commit(bar_mma);
    }
    ok = __syncthreads_and(mbar_wait(bar_mma, mma_phase, abort_flag, p.status, 23) ? 1 : 0) != 0;
    mma_phase ^= 1u;
    if (!ok) break;
    tc_fence_after();
    {
      const uint32_t orow = tmem_O + ((uint32_t)(warp * 32) << 16);
      const int q = half * 128 + m;
      const float inv = 1.f / sum;
      __nv_bfloat16* dst = p.out + (row0 + q) * p.ld_out + (int64_t)head * 64;
#pragma unroll
      for (int c0 = 0; c0 < 64; c0 += 32) {
        uint32_t v[32];
        tmem_ld_32x32(orow + c0, v);
        tmem_ld_wait();
        if (q < N) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 hb = __floats2bfloat162_rn(__uint_as_float(v[8 * j + 2 * e]) * inv,
                                                        __uint_as_float(v[8 * j + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<uint32_t*>(&hb);
            }
            *reinterpret_cast<uint4*>(dst + c0 + 8 * j) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
    tc_fence_before();
    __syncthreads();  // TMEM rows and the P tile are free for the next half
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

struct dsn_attention_launch {
  AttParams p;
};

cudaError_t dsn_launch_attention(const CUtensorMap& map, const int32_t* heads, int T, int N, int H, int B, int G,
                                 int grouped, const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                 const void* qkv, int64_t ld_qkv, void* out, int64_t ld_out, int32_t* status,
                                 cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  AttParams p;
  memset(&p, 0, sizeof(p));
  p.map = map;
  for (int t = 0; t < T; ++t) p.heads[t] = (int8_t)heads[t];
  p.N = N; p.H = H; p.B = B; p.G = G; p.T = T; p.grouped = grouped;
  p.offsets = offsets; p.perm = perm; p.group_slice = group_slice;
  p.qkv = static_cast<const __nv_bfloat16*>(qkv); p.ld_qkv = ld_qkv;
  p.out = static_cast<__nv_bfloat16*>(out); p.ld_out = ld_out;
  p.status = status;
  const size_t smem = 1024 + 1024 + kQBytes + kKBytes + kVtBytes + kPBytes;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  return dsn_launch(attention_kernel, dim3(H, B), dim3(kAttThreads), smem, s, 1, p);
}
