// Slimmable self-attention core (Sec. 3.4): for a sample routed to a path with h heads,
//   A_a = Softmax(Q_a K_a^T / sqrt(D_h)) V_a,  a < h,   out = Concat(A_0 .. A_{h-1}).
//
// Input is the output of the fused, head-major QKV layer: row r of a sample holds [head][q|k|v][64];
// the output row holds [head][64] and feeds the sliced projection (k_in = h * 64).  Heads >= h of a
// sample are neither read nor written.
//
// One work item = (sample, head, half of the queries), N <= 256 tokens, D_h = 64, worked by one CTA of
// 256 threads; two CTAs fit on an SM (about 99 KB of shared memory and 256 TMEM columns each), so one
// CTA's loads and barriers hide behind the other's arithmetic.  Two CTAs per SM walk the list of items
// that exist (heads a path does not have are not in it) and fetch the next item's tiles while the
// current output leaves; with more groups than the item table holds, one CTA per item of the dense grid.
// Per item:
//   Q [128 queries][64], K [256 keys][64] and V [256 keys][64] arrive by TMA (128-byte rows,
//   128-byte swizzle).  K is the K-major B operand of S = Q K^T; V, whose rows are keys and whose
//   64 contiguous elements are the head dimension, is the MN-major B operand of O = P V, so it is
//   used as loaded (its rows >= N are cleared: they belong to the next sample);
//   S = Q K^T: tcgen05.mma M = 128, N = keys rounded to 16, K = 64, fp32 in TMEM;
//   two threads share one query row (warps w and w + 4 own the same TMEM lanes and half of the keys
//   each): a first pass over their part of the S row, read from TMEM 16 keys at a time into two alternating register blocks, gives the row
//   maximum; a second pass the exponentials, the row sum and P as bf16 in a swizzled K-major
//   shared-memory tile that reuses the space of K and Q (keys >= N: zeros);
//   O = P V: tcgen05.mma M = 128, N = 64, K = keys rounded to 16, into the TMEM columns S has left;
//   the row is scaled by 1 / sum, rounded to bf16 and stored (each of the two threads writes 64 bytes
//   of the 128-byte line).
// Waits are bounded as in the GEMM.
#include <stdlib.h>
#include <string.h>

#include "dsn_gemm_device.cuh"
#include "dsn_attention.cuh"

namespace {

using namespace dsn_gemm;

constexpr int kAttThreads = 256;
constexpr uint32_t kQBytes = 128 * 128;       // 128 queries x 64 bf16
constexpr uint32_t kKBytes = 256 * 128;       // 256 keys x 64 bf16
constexpr uint32_t kVBytes = 256 * 128;       // 256 keys x 64 bf16
constexpr uint32_t kPBytes = 4 * 128 * 128;   // 4 key chunks x 128 queries x 64 keys bf16 (over K, Q and 16 KB more)
constexpr uint32_t kAttTmemCols = 256;

__device__ __forceinline__ int find_group_of(const int32_t* __restrict__ offsets, int G, int p) {
  int lo = 0, hi = G;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (offsets[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

// MN-major operand descriptor: rows of the tile are K indices (128 bytes = 64 contiguous M/N elements
// each), 8-row groups 1024 bytes apart, 128-byte swizzle; one K = 16 step is 16 rows = 2048 bytes.
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}


// One work item = (sample position, head, half of the queries).  kPersist = false: one CTA per item of
// the dense grid (head, position, half); items of heads the sample's path does not have return at once.
// kPersist = true (G <= kAttTableGroups): a fixed grid of CTAs walks the list of existing items
// (group by group: position, half, head fastest) with a stride of gridDim.x.  Each CTA builds the
// per-group item prefix once, so that finding an item needs no global load, allocates TMEM and
// initialises its barriers once, and issues the loads of its next item as soon as the P V product of
// the current one has finished with shared memory, i.e. under the read-out and store of O.
template <bool kPersist>
__global__ void __launch_bounds__(kAttThreads, 2) attention_kernel(const __grid_constant__ AttParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  // layout: control 3 KB (barriers, row maxima, row sums, item table) | V 32 KB | K 32 KB | Q 16 KB | 16 KB;
  // P (64 KB) overlays K, Q and the last 16 KB once S has been computed
  const uint32_t bar_load = base, bar_mma = base + 8;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 20);
  int32_t* s_heads = reinterpret_cast<int32_t*>(smem + 24);
  float* s_max = reinterpret_cast<float*>(smem + 64);     // [2 parts][128 rows] row maxima
  float* s_sum = reinterpret_cast<float*>(smem + 1088);   // [2 parts][128 rows] row sums
  int32_t* s_pre = reinterpret_cast<int32_t*>(smem + 2112);  // [G + 1] items before group g
  int32_t* s_off = s_pre + kAttTableGroups + 1;              // [G] first position of group g
  int32_t* s_h = s_off + kAttTableGroups;                    // [G] heads of group g's path
  const uint32_t v_s = base + 3072, k_s = v_s + kVBytes, q_s = k_s + kKBytes, p_s = k_s;
  uint8_t* v_ptr = smem + 3072;
  uint8_t* p_ptr = v_ptr + kVBytes;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.N;
  const int halves = N > 128 ? 2 : 1;

  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  int head, half, blk;       // the current item
  int it = 0, total = 0;     // persistent form: its index in the item list, and the length of the list
  const int stride = kPersist ? (int)gridDim.x : 1;
  // item `i` of the list -> (head, half, row block); false when the sample is not part of the batch
  auto decode = [&](int i, int& hd, int& hf, int& bk) {
    int g = 0;
    while (s_pre[g + 1] <= i) ++g;  // i < s_pre[G]: ends; empty groups are stepped over
    const int local = i - s_pre[g], hg = s_h[g];
    const int r = local / hg;
    hd = local - r * hg;
    hf = halves == 2 ? (r & 1) : 0;
    const int pos = s_off[g] + (halves == 2 ? (r >> 1) : r);
    bk = p.grouped ? pos : p.perm[pos];
    return bk >= 0;
  };
  if (kPersist) {
    for (int g = tid; g < p.G; g += kAttThreads) {
      const int lo = p.offsets[g], hi = p.offsets[g + 1];
      const int sl = p.group_slice ? p.group_slice[g] : g;
      const int hh = (sl >= 0 && sl < p.T) ? p.heads[sl] : 0;
      s_off[g] = lo;
      s_h[g] = hh;
      s_pre[g + 1] = (hi - lo) * hh * halves;
    }
    __syncthreads();
    if (tid == 0) {
      int acc = 0;
      s_pre[0] = 0;
      for (int g = 0; g < p.G; ++g) {
        acc += s_pre[g + 1];
        s_pre[g + 1] = acc;
      }
    }
    __syncthreads();
    total = s_pre[p.G];
    it = blockIdx.x;
    while (it < total && !decode(it, head, half, blk)) it += stride;
    if (it >= total) return;  // nothing for this CTA (uniform)
  } else {
    head = blockIdx.x;
    half = blockIdx.z;
    const int pos = blockIdx.y;
    if (half * 128 >= N) return;
    // The group of this position is the one with offsets[g] <= pos < offsets[g+1] (empty groups never match).
    // Thread g tests group g and fetches that group's head count at the same time, so the lookup costs two
    // dependent loads instead of a chain of four; the owner leaves the count in shared memory and the
    // barrier tells everybody whether there was an owner.
    blk = p.grouped ? pos : p.perm[pos];
    int owner = 0;
    for (int g = tid; g < p.G; g += kAttThreads) {
      const int lo = p.offsets[g], hi = p.offsets[g + 1];
      const int sl = p.group_slice ? p.group_slice[g] : g;
      const int hh = (sl >= 0 && sl < p.T) ? p.heads[sl] : 0;
      if (lo <= pos && pos < hi) {
        owner = 1;
        *s_heads = hh;
      }
    }
    const int heads_here = (__syncthreads_or(owner) && blk >= 0) ? *s_heads : 0;
    if (head >= heads_here) return;  // this sample's path has fewer heads (uniform over the CTA)
  }
  const int npad = (N + 15) & ~15;
  const int kboxes = npad > 128 ? 2 : 1;
  auto issue_loads = [&](int hd, int hf, int bk) {  // by one elected lane
    mbar_expect_tx(bar_load, (uint32_t)kboxes * 2u * 16384u + kQBytes);
    for (int b2 = 0; b2 < kboxes; ++b2) {
      tma_load_4d(k_s + b2 * 16384, &p.map, 0, hd * 3 + 1, 128 * b2, bk, bar_load);
      tma_load_4d(v_s + b2 * 16384, &p.map, 0, hd * 3 + 2, 128 * b2, bk, bar_load);
    }
    tma_load_4d(q_s, &p.map, 0, hd * 3 + 0, 128 * hf, bk, bar_load);
  };

  if (warp == 1) {  // not the warp that issues the loads: the allocation may have to wait for the SM's other CTA
    tmem_alloc(smem_u32(tmem_slot), kAttTmemCols);
    tmem_relinquish();
  }
  if (warp == 0 && elect_one()) issue_loads(head, half, blk);  // operands stay in uniform registers
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t idesc_s = make_idesc(128, npad);
  const uint32_t idesc_o = make_idesc(128, 64) | (1u << 16);  // B operand MN-major
  const float sl2 = 0.125f * 1.4426950408889634f;             // 1/sqrt(64) * log2(e)
  const int part = warp >> 2;                 // which half of the keys this thread owns
  const int m = (warp & 3) * 32 + lane;       // query row within the half = TMEM lane
  const int cols_per = npad >> 1;             // keys per part, a multiple of 8
  const int cbeg = part * cols_per;
  const uint32_t trow = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);

  for (uint32_t n_done = 0;; ++n_done) {
    // the item after this one (persistent form); its row block may need one load from the permutation
    int head_n = 0, half_n = 0, blk_n = 0, it_n = total;
    if (kPersist) {
      it_n = it + stride;
      while (it_n < total && !decode(it_n, head_n, half_n, blk_n)) it_n += stride;
    }
    const int64_t row0 = (int64_t)blk * N;
    // a warp whose 32 query rows all lie beyond N has no row to normalise: it only keeps the barriers
    const bool rows_live = half * 128 + (warp & 3) * 32 < N;

    bool ok = __syncthreads_and(mbar_wait(bar_load, n_done & 1u, abort_flag, p.status, 21) ? 1 : 0) != 0;
    if (ok) {
      // V rows >= N belong to the next sample (or to nobody): clear them so that 0 * garbage cannot appear
      for (int e = tid; e < (npad - N) * 8; e += kAttThreads)
        *reinterpret_cast<uint4*>(v_ptr + (N + (e >> 3)) * 128 + (e & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
      // (these rows are first read by the P V product, behind the barrier that follows the softmax)
      if (warp == 0 && elect_one()) {
        tc_fence_after();
        const uint64_t dq = make_smem_desc(q_s), dk = make_smem_desc(k_s);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) umma_bf16(tmem_base, dq + 2u * ks, dk + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
        umma_commit(bar_mma);
      }
      ok = __syncthreads_and(mbar_wait(bar_mma, 0, abort_flag, p.status, 22) ? 1 : 0) != 0;
    }
    if (!ok) break;

    tc_fence_after();
    // ---- pass 1 over this thread's part of the S row: the maximum.  The scores are read from TMEM one
    // 16-key block at a time and not kept: 104 scores per thread would not fit the register budget of two
    // CTAs per SM, and a second read of TMEM (pass 2) is cheaper than spilling them.
    // Keys >= N (next sample's rows, or padding) count as -inf; only the block that straddles N pays for the test.
    float mx = -INFINITY;
    const int nblk = (cols_per + 15) >> 4;  // blocks of 16 keys; two register blocks alternate (see pass 2)
    auto max_block = [&](const uint32_t (&v)[16], int c) {
      const int kb = cbeg + 16 * c;                                  // first key of the block
      const int nk = cols_per - 16 * c < 16 ? cols_per - 16 * c : 16;  // keys of this part in the block (multiple of 8)
      if (kb + nk > N) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (i < nk && kb + i < N) mx = fmaxf(mx, __uint_as_float(v[i]));
      } else if (nk == 16) {
#pragma unroll
        for (int i = 0; i < 16; i += 2) mx = fmaxf(mx, fmaxf(__uint_as_float(v[i]), __uint_as_float(v[i + 1])));
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (i < nk) mx = fmaxf(mx, __uint_as_float(v[i]));
      }
    };
    if (rows_live) {
      uint32_t va[16], vb[16];
      tmem_ld_32x16(trow + cbeg, va);
      tmem_ld_wait();
#pragma unroll 1
      for (int c = 0; c < nblk; c += 2) {
        if (c + 1 < nblk) tmem_ld_32x16(trow + cbeg + 16 * (c + 1), vb);
        max_block(va, c);
        tmem_ld_wait();
        if (c + 1 < nblk) {
          if (c + 2 < nblk) tmem_ld_32x16(trow + cbeg + 16 * (c + 2), va);
          max_block(vb, c + 1);
          tmem_ld_wait();
        }
      }
    }
    s_max[part * 128 + m] = mx;
    __syncthreads();
    mx = fmaxf(s_max[m], s_max[128 + m]);
    const float mxs = mx * sl2;
    float sum = 0.f;
    // ---- pass 2: exp2(s * c - max * c), one FMA and one special-function instruction per key, probabilities
    // rounded to bf16 into the swizzled P tile (which overlays K and Q: S has been computed, and pass 1 of
    // every thread is over).  Rows of a warp that is not live keep whatever the tile held: a row of P only
    // reaches the same row of O, which is not stored.
    // 16 keys at a time, two register blocks alternating: the TMEM load of the next block is in flight
    // while the exponentials of this one are computed.
    auto exp_block = [&](uint32_t (&v)[16], int c) {
      const int kb = cbeg + 16 * c;
      if (kb + 16 > N) {
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (kb + i >= N) v[i] = 0xff800000u;  // -inf: probability 0
      }
#pragma unroll
      for (int jv = 0; jv < 2; ++jv) {
        const int j0 = 16 * c + 8 * jv;       // first of 8 keys, relative to the part
        if (j0 < cols_per) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float a, b;
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(a) : "f"(fmaf(__uint_as_float(v[8 * jv + 2 * e]), sl2, -mxs)));
            asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(b) : "f"(fmaf(__uint_as_float(v[8 * jv + 2 * e + 1]), sl2, -mxs)));
            sum += a + b;
            __nv_bfloat162 hb = __floats2bfloat162_rn(a, b);
            w[e] = *reinterpret_cast<uint32_t*>(&hb);
          }
          const int key = cbeg + j0;
          *reinterpret_cast<uint4*>(p_ptr + (key >> 6) * 16384 + m * 128 + ((((key & 63) >> 3) ^ (m & 7)) << 4)) =
              make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    };
    if (rows_live) {
      uint32_t va[16], vb[16];
      tmem_ld_32x16(trow + cbeg, va);
      tmem_ld_wait();
#pragma unroll 1
      for (int c = 0; c < nblk; c += 2) {
        if (c + 1 < nblk) tmem_ld_32x16(trow + cbeg + 16 * (c + 1), vb);
        exp_block(va, c);
        tmem_ld_wait();
        if (c + 1 < nblk) {
          if (c + 2 < nblk) tmem_ld_32x16(trow + cbeg + 16 * (c + 2), va);
          exp_block(vb, c + 1);
          tmem_ld_wait();
        }
      }
    }
    tc_fence_before();  // the PV product writes its accumulator over the columns just read
    s_sum[part * 128 + m] = sum;
    fence_async_smem();
    __syncthreads();
    sum = s_sum[m] + s_sum[128 + m];

    // ---- O = P V, into the columns S occupied
    if (warp == 0 && elect_one()) {
      tc_fence_after();
      for (int ks = 0; ks < npad / 16; ++ks) {
        const uint64_t dp = make_smem_desc(p_s + (ks >> 2) * 16384) + 2u * (ks & 3);
        const uint64_t dv = make_smem_desc_mn(v_s + ks * 2048);
        umma_bf16(tmem_base, dp, dv, idesc_o, ks > 0 ? 1u : 0u);
      }
      umma_commit(bar_mma);
    }
    ok = __syncthreads_and(mbar_wait(bar_mma, 1, abort_flag, p.status, 23) ? 1 : 0) != 0;
    if (!ok) break;
    // the tensor core has finished with P and V: the next item's tiles may land while O leaves
    if (kPersist && it_n < total && warp == 0 && elect_one()) issue_loads(head_n, half_n, blk_n);
    tc_fence_after();
    {
      const uint32_t orow = trow + 32 * part;
      const int q = half * 128 + m;
      const float inv = 1.f / sum;
      __nv_bfloat16* dst = p.out + (row0 + q) * p.ld_out + (int64_t)head * 64 + 32 * part;
      if (rows_live) {
        uint32_t o[32];
        tmem_ld_32x32(orow, o);
        tmem_ld_wait();
        if (q < N) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              __nv_bfloat162 hb = __floats2bfloat162_rn(__uint_as_float(o[8 * j + 2 * e]) * inv,
                                                        __uint_as_float(o[8 * j + 2 * e + 1]) * inv);
              w[e] = *reinterpret_cast<uint32_t*>(&hb);
            }
            *reinterpret_cast<uint4*>(dst + 8 * j) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
    if (!kPersist || it_n >= total) break;
    tc_fence_before();  // O has been read: the next item's S may overwrite it once every thread has passed the load barrier
    it = it_n; head = head_n; half = half_n; blk = blk_n;
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kAttTmemCols);
  }
}

}  // namespace

// 0 (default): the warp-specialised form where it applies; DSN_ATTENTION=items keeps the form with one
// (sample, head, query half) item per CTA pass everywhere (for comparisons).
static int dsn_attention_form() {
  static int form = -1;
  if (form < 0) {
    const char* e = getenv("DSN_ATTENTION");
    form = (e && strcmp(e, "items") == 0) ? 1 : 0;
  }
  return form;
}

cudaError_t dsn_launch_attention(const CUtensorMap& map, const CUtensorMap& map_out, const int32_t* heads, int T, int N, int H, int B, int G,
                                 int grouped, const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                 const void* qkv, int64_t ld_qkv, void* out, int64_t ld_out, int32_t* status,
                                 cudaStream_t s) {
  if (B == 0) return cudaSuccess;
  AttParams p;
  memset(&p, 0, sizeof(p));
  p.map = map;
  p.map_out = map_out;
  for (int t = 0; t < T; ++t) p.heads[t] = (int8_t)heads[t];
  p.N = N; p.H = H; p.B = B; p.G = G; p.T = T; p.grouped = grouped;
  p.offsets = offsets; p.perm = perm; p.group_slice = group_slice;
  p.qkv = static_cast<const __nv_bfloat16*>(qkv); p.ld_qkv = ld_qkv;
  p.out = static_cast<__nv_bfloat16*>(out); p.ld_out = ld_out;
  p.status = status;
  const size_t smem = 1024 + 3072 + kVBytes + kPBytes;  // P overlays K, Q and 16 KB more
  static size_t configured[2][DSN_MAX_DEVICES] = {};
  cudaError_t e = dsn_ensure_dynamic_smem(attention_kernel<false>, smem, configured[0]);
  if (e == cudaSuccess) e = dsn_ensure_dynamic_smem(attention_kernel<true>, smem, configured[1]);
  int dev = 0, sms = 0;
  if (e == cudaSuccess) e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const int resident = 2 * sms;  // CTAs the persistent form keeps in flight: two per SM
  const int halves = N > 128 ? 2 : 1;
  if (G <= kAttTableGroups && dsn_attention_form() == 0) return dsn_launch_attention_ws(p, sms, s);
  if (G <= kAttTableGroups) {
    const long long dense = (long long)H * B * halves;
    return dsn_launch(attention_kernel<true>, dim3((unsigned)(dense < resident ? dense : resident)), dim3(kAttThreads), smem, s,
                      1, p);
  }
  return dsn_launch(attention_kernel<false>, dim3(H, B, halves), dim3(kAttThreads), smem, s, 1, p);
}
