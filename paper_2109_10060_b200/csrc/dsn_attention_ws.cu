// Slimmable self-attention core (Sec. 3.4), warp-specialised form:
//   A_a = Softmax(Q_a K_a^T / sqrt(D_h)) V_a,  a < h heads of the sample's path,  out = Concat(A_0 .. A_{h-1}).
//
// One work item = (sample, head): all N <= 256 queries against all N keys, D_h = 64.  One persistent CTA per
// SM walks the items that exist (heads a path does not have are not in the list) with the stride of the grid.
// Roles (320 threads):
//   warp 0      loader: Q (2 x 128 rows), K and V (256 rows each) of the item after the current one by TMA into
//               the other of two operand stages (96 KB each); every tile is fetched exactly once.  The tensor
//               map sees the samples as a dimension of their own, so rows >= N arrive as zeros.
//   warp 1      tensor-core issue: S_h = Q_h K^T (M = 128, N = keys rounded to 16, K = 64) and O_h = P_h V
//               (M = 128, N = 64, K = keys) for the two query halves h, in the order
//               PV_0(i), QK_0(i+1), PV_1(i), QK_1(i+1): the softmax of one half runs under the products of the other.
//   warps 2-5   softmax of half 0, warps 6-9 of half 1: one thread per query row (= TMEM lane), no exchange between
//               threads.  Pass 1 reads the row of S from TMEM for its maximum, pass 2 reads it again, takes exp2 of
//               the scaled difference, sums, and writes the probabilities as bf16 back into TMEM over columns of S
//               already read.  P is the A operand of the second product straight from TMEM, so it never passes
//               through shared memory.  O_h lands in columns of S_h that are dead by then; it is read (which frees
//               the region for the next item's S), scaled by 1 / sum, rounded to bf16, staged per warp in the
//               item's Q tiles (dead since S was computed) and leaves by one TMA store per warp.
// TMEM: 512 columns = two 256-column regions; in region h: S_h in columns 0..npad-1, P_h over columns 0..npad/2-1,
// O_h in columns 192..255.  Every wait is bounded (see dsn_gemm_device.cuh).
#include "dsn_gemm_device.cuh"
#include "dsn_attention.cuh"

namespace {

using namespace dsn_gemm;

constexpr int kWsThreads = 320;   // loader warp, issue warp, 8 softmax warps
constexpr uint32_t kTileBytes = 128 * 128;           // 128 rows x 64 bf16
constexpr uint32_t kStageBytes = 6 * kTileBytes;     // Q0 Q1 | K (2 tiles) | V (2 tiles)
constexpr uint32_t kWsCtrlBytes = 1024;  // barriers and item table
constexpr uint32_t kRegionCols = 256, kOCol = 192;

__device__ __forceinline__ void tmem_alloc_512(uint32_t slot_smem) { tmem_alloc(slot_smem, 512); }

// D[tmem] (+)= A[tmem] * B[smem]: A rows are TMEM lanes, its K elements packed two bf16 per 32-bit column.
__device__ __forceinline__ void umma_bf16_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const uint32_t (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, int c0, int c1, int c2, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 2^t for two non-positive arguments without the special-function unit (one warp gets at most one
// special-function instruction every 16 cycles issued, so half of the exponentials are computed here, on the
// FMA pipe, two per instruction): t = n + f with n = round(t) taken from the mantissa of t + 1.5 * 2^23 and
// f in [-1/2, 1/2]; 2^f by a cubic (own minimax fit, relative error 7.5e-5, a thirtieth of a bfloat16
// rounding step); 2^n by adding n to the exponent field.  Arguments below -126 (and -inf) give 2^-126.
__device__ __forceinline__ void exp2_pair_fma(uint64_t t2, float& x0, float& x1) {
  float t0, t1;
  unpack2(t2, t0, t1);
  t2 = pack2(fmaxf(t0, -126.f), fmaxf(t1, -126.f));
  const uint64_t magic = pack2(12582912.f, 12582912.f), nmagic = pack2(-12582912.f, -12582912.f);
  const uint64_t r2 = fadd2(t2, magic);
  const uint64_t n2 = fadd2(r2, nmagic);
  const uint64_t f2 = ffma2(n2, pack2(-1.f, -1.f), t2);
  uint64_t p2 = ffma2(pack2(0.0551716685f, 0.0551716685f), f2, pack2(0.2426111251f, 0.2426111251f));
  p2 = ffma2(p2, f2, pack2(0.6932609677f, 0.6932609677f));
  p2 = ffma2(p2, f2, pack2(0.9999280572f, 0.9999280572f));
  float r0, r1, p0, p1;
  unpack2(r2, r0, r1);
  unpack2(p2, p0, p1);
  x0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(r0) << 23));
  x1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(r1) << 23));
}
// MN-major B operand (V as loaded: rows are keys, 64 contiguous head-dimension elements per 128-byte row).
__device__ __forceinline__ uint64_t make_smem_desc_mn_ws(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// The list of items: group by group, inside a group position by position, head fastest.
struct ItemWalk {
  const int32_t* s_pre;  // [G + 1] items before group g
  const int32_t* s_off;  // [G] first position of group g
  const int32_t* s_h;    // [G] heads of group g's path
  int g;                 // group of the last decoded item (items are visited in ascending order)
  __device__ __forceinline__ void decode(int i, int& head, int& pos) {
    while (s_pre[g + 1] <= i) ++g;  // i < s_pre[G]: ends; empty groups are stepped over
    const int local = i - s_pre[g], hg = s_h[g];
    const int r = local / hg;
    head = local - r * hg;
    pos = s_off[g] + r;
  }
};

__global__ void __launch_bounds__(kWsThreads, 1) attention_ws_kernel(const __grid_constant__ AttParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  // control block: barriers, TMEM slot, abort flag, item table; then two operand stages
  const uint32_t bar_kv_full = base, bar_kv_empty = base + 16;              // [2] each
  const uint32_t bar_s_full = base + 32, bar_p_full = base + 48, bar_o_full = base + 64, bar_s_empty = base + 80;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 112);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 116);
  int32_t* s_pre = reinterpret_cast<int32_t*>(smem + 128);
  int32_t* s_off = s_pre + kAttTableGroups + 1;
  int32_t* s_h = s_off + kAttTableGroups;
  const uint32_t stage0 = base + kWsCtrlBytes;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int N = p.N;
  const int halves = N > 128 ? 2 : 1;
  const int npad = (N + 15) & ~15;

  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_kv_full + 8 * i, 1);
      mbar_init(bar_kv_empty + 8 * i, 1 + 4 * halves);  // the issue warp (operands read) + every softmax warp (its staging tile read)
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_p_full + 8 * i, 4);   // one arrival per softmax warp of the half
      mbar_init(bar_o_full + 8 * i, 1);
      mbar_init(bar_s_empty + 8 * i, 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int g = tid; g < p.G; g += kWsThreads) {
    const int lo = p.offsets[g], hi = p.offsets[g + 1];
    const int sl = p.group_slice ? p.group_slice[g] : g;
    const int hh = (sl >= 0 && sl < p.T) ? p.heads[sl] : 0;
    s_off[g] = lo;
    s_h[g] = hh;
    s_pre[g + 1] = (hi - lo) * hh;
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
  if (warp == 1) {
    tmem_alloc_512(smem_u32(tmem_slot));
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = s_pre[p.G];
  const int stride = (int)gridDim.x;
  ItemWalk walk{s_pre, s_off, s_h, 0};

  if (warp == 0) {
    // ------------------------------------------------------------------------------ loader
    uint32_t n = 0;
    for (int it = blockIdx.x; it < total; it += stride, ++n) {
      int head, pos;
      walk.decode(it, head, pos);
      int blk = p.grouped ? pos : p.perm[pos];
      if (blk < 0) blk = 0;  // a sample outside the batch: its item is walked by every role, its output not stored
      const uint32_t s = n & 1u;
      if (n >= 2 && !mbar_wait(bar_kv_empty + 8 * s, ((n >> 1) - 1u) & 1u, abort_flag, p.status, 31)) break;
      if (elect_one()) {
        const uint32_t st = stage0 + s * kStageBytes;
        const uint32_t full = bar_kv_full + 8 * s;
        mbar_expect_tx(full, (uint32_t)(3 * halves) * kTileBytes);
        for (int b2 = 0; b2 < halves; ++b2) {
          tma_load_4d(st + (2 + b2) * kTileBytes, &p.map, 0, head * 3 + 1, 128 * b2, blk, full);  // K
          tma_load_4d(st + b2 * kTileBytes, &p.map, 0, head * 3 + 0, 128 * b2, blk, full);        // Q
          tma_load_4d(st + (4 + b2) * kTileBytes, &p.map, 0, head * 3 + 2, 128 * b2, blk, full);  // V
        }
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------------------ tensor-core issue
    const uint32_t idesc_s = make_idesc(128, npad);
    const uint32_t idesc_o = make_idesc(128, 64) | (1u << 16);  // B operand MN-major
    auto issue_qk = [&](uint32_t st, int h) {  // S_h = Q_h K^T
      const uint64_t dq = make_smem_desc(st + h * kTileBytes), dk = make_smem_desc(st + 2 * kTileBytes);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16(tmem_base + h * kRegionCols, dq + 2u * ks, dk + 2u * ks, idesc_s, ks > 0 ? 1u : 0u);
      umma_commit(bar_s_full + 8 * h);
    };
    auto issue_pv = [&](uint32_t st, int h) {  // O_h = P_h V, P_h read from TMEM
      const uint32_t region = tmem_base + h * kRegionCols;
      for (int ks = 0; ks < npad / 16; ++ks)
        umma_bf16_a_tmem(region + kOCol, region + 8u * ks, make_smem_desc_mn_ws(st + 4 * kTileBytes + ks * 2048), idesc_o,
                         ks > 0 ? 1u : 0u);
      umma_commit(bar_o_full + 8 * h);
    };
    bool ok = true;
    uint32_t n = 0;
    // The two halves run half a period apart: while one is in its exponentials (special-function unit) the
    // other is in its maximum pass, waits for its products or moves O out.  The offset is set up once, by
    // issuing S_1 of the first item only when P_0 of that item is complete, and the fixed issue order
    // PV_0(n), QK_0(n+1), PV_1(n), QK_1(n+1) keeps it.
    if ((int)blockIdx.x < total) {
      ok = mbar_wait(bar_kv_full, 0, abort_flag, p.status, 32);
      if (ok && elect_one()) {
        tc_fence_after();
        issue_qk(stage0, 0);
      }
      __syncwarp();
    }
    for (int it = blockIdx.x; ok && it < total; it += stride, ++n) {
      const uint32_t s = n & 1u, sn = s ^ 1u;
      const uint32_t st = stage0 + s * kStageBytes, stn = stage0 + sn * kStageBytes;
      const bool more = it + stride < total;
      for (int h = 0; h < halves && ok; ++h) {
        ok = mbar_wait(bar_p_full + 8 * h, n & 1u, abort_flag, p.status, 33);
        if (!ok) break;
        if (elect_one()) {
          tc_fence_after();
          issue_pv(st, h);
          if (h == halves - 1) umma_commit(bar_kv_empty + 8 * s);  // every product of the item has read its operands
          if (n == 0 && h == 0 && halves == 2) issue_qk(st, 1);    // the delayed start of the second half
        }
        __syncwarp();
        if (more) {  // S_h of the next item, once O_h of this one has been read out
          if (h == 0) ok = mbar_wait(bar_kv_full + 8 * sn, ((n + 1u) >> 1) & 1u, abort_flag, p.status, 34);
          ok = ok && mbar_wait(bar_s_empty + 8 * h, n & 1u, abort_flag, p.status, 35);
          if (!ok) break;
          if (elect_one()) {
            tc_fence_after();
            issue_qk(stn, h);
          }
          __syncwarp();
        }
      }
    }
  } else {
    // ------------------------------------------------------------------------------ softmax, one thread per query row
    const int h = (warp - 2) >> 2;              // query half of this warp group
    const int quarter = warp & 3;               // TMEM lanes this warp may touch: 32 * (warp % 4) ...
    const bool warp_live = h * 128 + quarter * 32 < N;   // some row of this warp exists
    const uint32_t region = tmem_base + h * kRegionCols + ((uint32_t)(quarter * 32) << 16);
    const float sl2 = 0.125f * 1.4426950408889634f;      // 1/sqrt(64) * log2(e)
    const int nb32 = (npad + 31) >> 5;          // blocks of 32 keys in the row (the last may be half valid)
    uint32_t n = 0;
    if (h < halves) {
      int head = 0, blk = 0;   // the current item, decoded one item ahead (under the wait for the second product)
      if ((int)blockIdx.x < total) {
        int pos;
        walk.decode(blockIdx.x, head, pos);
        blk = p.grouped ? pos : p.perm[pos];
      }
      bool store_pending = false;   // lane 0: a TMA store of the previous item may still be reading its staging tile
      for (int it = blockIdx.x; it < total; it += stride, ++n) {
        const uint32_t s = n & 1u;
        // the previous item's store has read its staging tile by the time S of this item is ready (or shortly after): that
        // stage goes back to the loader before the maximum pass, which then has all of this item to refill it
        if (lane == 0 && store_pending) {
          bulk_wait_read0();
          mbar_arrive(bar_kv_empty + 8 * (s ^ 1u));
          store_pending = false;
        }
        if (!mbar_wait(bar_s_full + 8 * h, n & 1u, abort_flag, p.status, 36)) break;
        tc_fence_after();
        float sum = 0.f;
        if (warp_live) {
          // pass 1: the row maximum; keys >= N (zero rows of K, stale columns beyond the padded row) do not count.
          // Two register blocks of 32 scores, both loads in flight before the wait.
          uint32_t va[32], vb[32];
          float mx0 = -INFINITY, mx1 = -INFINITY;
          {
            auto max_block = [&](const uint32_t (&v)[32], int key0) {
              if (key0 + 32 > N) {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                  if (key0 + i < N) mx0 = fmaxf(mx0, __uint_as_float(v[i]));
              } else {
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                  mx0 = fmax3(mx0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                  mx1 = fmax3(mx1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                }
              }
            };
#pragma unroll 1
            for (int c = 0; c < nb32; c += 2) {
              tmem_ld_32x32(region + 32 * c, va);
              if (c + 1 < nb32) tmem_ld_32x32(region + 32 * (c + 1), vb);
              tmem_ld_wait();
              max_block(va, 32 * c);
              if (c + 1 < nb32) max_block(vb, 32 * (c + 1));
            }
          }
          // pass 2: exp2(s * c - max * c); probabilities rounded to bf16 and written over columns of S this thread
          // has already read (P block c: 16 columns at 16 c).  Two keys per instruction where the hardware has a
          // packed fp32 form (scale-and-subtract, row sum); of the exponentials every other pair is one
          // special-function instruction per key, the rest runs on the FMA pipe.  Two register blocks: the next
          // block's load is in flight under the arithmetic.
          const float mxs = fmaxf(mx0, mx1) * sl2;
          const uint64_t sl2_2 = pack2(sl2, sl2), nmx_2 = pack2(-mxs, -mxs);
          uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
          auto exp_block = [&](uint32_t (&v)[32], int c) {
            if (32 * c + 32 > N) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (32 * c + i >= N) v[i] = 0xff800000u;  // -inf: probability 0
            }
#pragma unroll
            for (int half_b = 0; half_b < 2; ++half_b) {
              if (32 * c + 16 * half_b < npad) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  float x0, x1;
                  const uint64_t t2 = ffma2(pack2(__uint_as_float(v[16 * half_b + 2 * e]), __uint_as_float(v[16 * half_b + 2 * e + 1])), sl2_2, nmx_2);
                  if (e & 1) {
                    exp2_pair_fma(t2, x0, x1);   // every other pair on the FMA pipe
                  } else {
                    float t0, t1;
                    unpack2(t2, t0, t1);
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(x0) : "f"(t0));
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(x1) : "f"(t1));
                  }
                  if (e & 2) sum_b = fadd2(sum_b, pack2(x0, x1)); else sum_a = fadd2(sum_a, pack2(x0, x1));
                  __nv_bfloat162 hb = __floats2bfloat162_rn(x0, x1);
                  w[e] = *reinterpret_cast<uint32_t*>(&hb);
                }
                tmem_st_32x8(region + (uint32_t)(16 * c + 8 * half_b), w);
              }
            }
          };
          tmem_ld_32x32(region, va);
          tmem_ld_wait();
#pragma unroll 1
          for (int c = 0; c < nb32; c += 2) {
            if (c + 1 < nb32) tmem_ld_32x32(region + 32 * (c + 1), vb);
            exp_block(va, c);
            tmem_ld_wait();
            if (c + 2 < nb32) tmem_ld_32x32(region + 32 * (c + 2), va);
            if (c + 1 < nb32) exp_block(vb, c + 1);
            tmem_ld_wait();
          }
          {
            float s0, s1, s2, s3;
            unpack2(sum_a, s0, s1);
            unpack2(sum_b, s2, s3);
            sum = (s0 + s1) + (s2 + s3);
          }
          tmem_st_wait();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_p_full + 8 * h);
        // under the wait for O_h = P_h V: the item after this one is looked up
        const int head_cur = head, blk_cur = blk;
        if (it + stride < total) {
          int pos;
          walk.decode(it + stride, head, pos);
          blk = p.grouped ? pos : p.perm[pos];
        }
        if (!mbar_wait(bar_o_full + 8 * h, n & 1u, abort_flag, p.status, 37)) break;
        tc_fence_after();
        // The row leaves through a 32-row x 128-byte swizzled staging tile per warp and one TMA store (rows >= N are
        // clipped by the map).  The tiles of the eight softmax warps fill the item's two Q tiles, which nothing reads
        // once both S products are complete.  TMEM is handed back before the conversion starts.
        uint8_t* stg = smem + kWsCtrlBytes + s * kStageBytes + (uint32_t)(h * 4 + quarter) * 4096u;
        if (warp_live) {
          const float inv = 1.f / sum;
          uint32_t o[32], o2[32];
          tmem_ld_32x32(region + kOCol, o);
          tmem_ld_32x32(region + kOCol + 32, o2);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_s_empty + 8 * h);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float f0 = __uint_as_float(j < 4 ? o[8 * j + 2 * e] : o2[8 * (j - 4) + 2 * e]) * inv;
              const float f1 = __uint_as_float(j < 4 ? o[8 * j + 2 * e + 1] : o2[8 * (j - 4) + 2 * e + 1]) * inv;
              __nv_bfloat162 hb = __floats2bfloat162_rn(f0, f1);
              w[e] = *reinterpret_cast<uint32_t*>(&hb);
            }
            *reinterpret_cast<uint4*>(stg + lane * 128 + ((j ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {   // always the same thread: bulk groups belong to the thread that committed them
            if (blk_cur >= 0) tma_store_3d(&p.map_out, head_cur * 64, h * 128 + quarter * 32, blk_cur, smem_u32(stg));
            bulk_commit();
            store_pending = true;   // the stage is handed back to the loader during the next item (see below)
          }
          __syncwarp();
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar_s_empty + 8 * h);
            mbar_arrive(bar_kv_empty + 8 * s);
          }
        }
      }
    }
  }
  if (warp >= 2 && lane == 0) bulk_wait0();  // the last stores have left shared memory for good before the CTA ends


  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

size_t dsn_attention_ws_smem_bytes() { return 1024 + kWsCtrlBytes + 2 * (size_t)kStageBytes; }

cudaError_t dsn_launch_attention_ws(const AttParams& p, int sm_count, cudaStream_t s) {
  static size_t configured[DSN_MAX_DEVICES] = {};
  const size_t smem = dsn_attention_ws_smem_bytes();
  cudaError_t e = dsn_ensure_dynamic_smem(attention_ws_kernel, smem, configured);
  if (e != cudaSuccess) return e;
  const long long dense = (long long)p.H * p.B;
  return dsn_launch(attention_ws_kernel, dim3((unsigned)(dense < sm_count ? dense : sm_count)), dim3(kWsThreads), smem, s, 1, p);
}
