// Device-side building blocks shared by the grouped-GEMM kernels (one CTA per tile, and CTA pairs):
// PTX wrappers for mbarriers, TMA, tcgen05 and TMEM, descriptor encoders, the activation functions
// and the epilogue of one tile.  Included by the kernel translation units only.
#pragma once
#include "dsn_internal.cuh"
#include "dsn_tiles.cuh"

namespace dsn_gemm {

#ifndef DSN_EPI_WARPS
#define DSN_EPI_WARPS 8
#endif
constexpr int kEpiWarps = DSN_EPI_WARPS;        // a multiple of 4: kEpiWarps / 4 warps share each TMEM lane quarter
constexpr int kThreads = 64 + 32 * kEpiWarps;   // TMA warp, MMA warp, epilogue warps
constexpr int BM = DSN_GEMM_BM;
constexpr int BK = DSN_GEMM_BK;
constexpr uint32_t kABytes = BM * BK * 2;  // 16 KB: 128 rows of 128 bytes
constexpr uint32_t kCtrlBytes = 1024;
constexpr int kMaxStages = 8;
constexpr uint32_t kStageOutBytes = kEpiWarps * 32 * 128;  // epilogue staging: 32 rows x 128 bytes per warp
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s: the default limit of a bounded wait

// ---------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Limit of a bounded wait: the context's setting (microseconds, in the status block) or the default.
__device__ __forceinline__ uint64_t wait_limit_ns(const int32_t* status) {
  const uint32_t us = status ? *reinterpret_cast<const volatile uint32_t*>(status + DSN_STATUS_WAIT_US) : 0u;
  return us ? (uint64_t)us * 1000ull : kWaitLimitNs;
}

// True in exactly one lane of a converged warp.  Guarding the TMA / tcgen05 issue of a warp-uniform
// loop with it (rather than with lane == 0) lets the operands of those instructions stay in uniform
// registers: measured 289 instead of 510 cycles per stage of four tcgen05.mma plus a commit.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}

// Bounded wait.  Returns false when the CTA is aborting (this or another thread ran out of time).
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                            int32_t* status, int where) {
  const uint64_t t0 = globaltimer_ns();
  const uint64_t limit = wait_limit_ns(status);
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 31u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit) {
        *abort_flag = 1;
        dsn_set_status(status, DSN_ERR_TIMEOUT, where);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          int32_t* status, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, where);
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int c0, int c1, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(src)
               : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(src)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// make shared-memory writes of this thread visible to the async (TMA) proxy
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, fp32 accumulate
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the mbarrier receives one arrival once every tcgen05.mma issued so far by this thread is done
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (the layout TMA writes with CU_TENSOR_MAP_SWIZZLE_128B).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);       // start address, 16-byte units
  d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M x N tile.
__device__ __forceinline__ uint32_t make_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Packed fp32 pairs (two lanes per 64-bit register) and the three-input maximum.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t p, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(p)); }
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// erf(z) ~= tanh(c1 z + c3 z^3 + c5 z^5): coefficients fitted by least squares so that the GELU built
// on it stays within 3e-5 (absolute) of the exact erf form for every x; evaluated with the hardware
// tanh (relative error <= 2^-11), i.e. one special-function instruction per element instead of the
// two (reciprocal, exponential) a rational erf needs, which kept the epilogue behind the main loop.
// The total deviation from exact GELU stays below 1e-3 absolute at |x| = 4, a quarter of a bfloat16
// ulp of the output there.
__device__ __forceinline__ float erf_fast(float z) {
  const float z2 = z * z;
  const float u = z * fmaf(z2, fmaf(z2, -0.0020293f, 0.1047942f), 1.12777659f);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return t;
}

// The same GELU for two values at once with packed fp32 arithmetic (two lanes per instruction): the epilogue is bound
// by instruction issue, not by a pipe, and this form needs 6 packed instructions and 2 tanh for a pair where the
// scalar form needs 16 and 2 (measured: cfg3 fc1 57.4 -> 53.5 us, cfg5 fc1 on the narrowest path 203 -> 188 us).  0.5 v (1 + t) is evaluated as h + h t with h = v / 2.
__device__ __forceinline__ void gelu_pair(float a, float b, float& ra, float& rb) {
  // erf(v / sqrt 2) ~= tanh(v (k1 + k3 v^2 + k5 v^4)) with the 1 / sqrt 2 folded into the coefficients of erf_fast
  const uint64_t zero2 = pack2(0.f, 0.f);
  const uint64_t v2 = pack2(a, b);
  const uint64_t z2 = ffma2(v2, v2, zero2);
  uint64_t q = ffma2(z2, pack2(-0.00035873294f, -0.00035873294f), pack2(0.037050344f, 0.037050344f));
  q = ffma2(z2, q, pack2(0.79745847f, 0.79745847f));
  float u0, u1, t0, t1;
  unpack2(ffma2(v2, q, zero2), u0, u1);
  asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(u0));
  asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(u1));
  const uint64_t h2 = ffma2(v2, pack2(0.5f, 0.5f), zero2);
  unpack2(ffma2(h2, pack2(t0, t1), h2), ra, rb);
}

// The activation (and whether any per-column affine term exists) is a template parameter so that the
// per-element loop holds no trace of the other variants: an if-converted erf or a few unused loads per
// element are enough to put the epilogue behind the main loop.
template <int ACT>
__device__ __forceinline__ float apply_act(float v) {
  if (ACT == DSN_ACT_RELU) return fmaxf(v, 0.f);
  if (ACT == DSN_ACT_GELU) return 0.5f * v * (1.f + erf_fast(v * 0.70710678118654752f));
  return v;
}

// The 1..7 last columns of a row whose width is no multiple of 8 (packed bf16 pairs in `w`): one 8-, one 4- and one
// 2-byte store when the piece starts on an 8-byte boundary (it does whenever the row does), else 2-byte stores.
__device__ __forceinline__ void store_row_tail(__nv_bfloat16* dst, const uint32_t (&w)[4], int n) {
  if ((reinterpret_cast<uintptr_t>(dst) & 7u) == 0) {
    int off = 0;
    if (n & 4) { *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]); off = 4; }
    if (n & 2) { *reinterpret_cast<uint32_t*>(dst + off) = w[off >> 1]; off += 2; }
    if (n & 1) reinterpret_cast<uint16_t*>(dst)[off] = (uint16_t)(w[off >> 1] & 0xffffu);
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (e < n) reinterpret_cast<uint16_t*>(dst)[e] = (e & 1) ? (uint16_t)(w[e >> 1] >> 16) : (uint16_t)(w[e >> 1] & 0xffffu);
  }
}

// 32 accumulator columns of this thread's row (TMEM address `taddr`; columns cb .. cb + 31 of the tile) ->
// bias, per-path Re-SBN, skip features, activation -> 16 packed bf16 pairs.
template <int ACT, bool AFF, bool RES>
__device__ __forceinline__ void epilogue_half(uint32_t taddr, int cb, int ncols, const float* brow, const float* sc_row,
                                              const float* sh_row, const __nv_bfloat16* res_row, uint32_t (&out)[16]) {
  // the skip features of this row's 32 columns: four 16-byte loads in flight at once, issued ahead of
  // the TMEM load (a ragged or unaligned piece takes scalar loads)
  uint4 rres[4];
  bool rvec = false;
  if (RES && res_row) {
    const __nv_bfloat16* rp = res_row + cb;
    rvec = cb + 32 <= ncols && (reinterpret_cast<uintptr_t>(rp) & 15u) == 0;
    if (rvec) {
#pragma unroll
      for (int i = 0; i < 4; ++i) rres[i] = __ldg(reinterpret_cast<const uint4*>(rp) + i);
    }
  }
  uint32_t v[32];
  tmem_ld_32x32(taddr, v);
  tmem_ld_wait();
#pragma unroll
  for (int jj = 0; jj < 4; ++jj) {
    const uint4 rv = rvec ? rres[jj] : make_uint4(0u, 0u, 0u, 0u);
    const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c = 8 * jj + 2 * e;
      float a = __uint_as_float(v[c]), b = __uint_as_float(v[c + 1]);
      if (AFF) {  // bias, the per-path Re-SBN scale and shift of this tile's columns, the skip features of this row
        if (cb + c < ncols) {
          if (brow) a += __ldg(brow + cb + c);
          if (sc_row) a = fmaf(a, __ldg(sc_row + cb + c), __ldg(sh_row + cb + c));
          if (RES && rvec) a += __uint_as_float(rw[e] << 16);
          else if (RES && res_row) a += __bfloat162float(res_row[cb + c]);
        }
        if (cb + c + 1 < ncols) {
          if (brow) b += __ldg(brow + cb + c + 1);
          if (sc_row) b = fmaf(b, __ldg(sc_row + cb + c + 1), __ldg(sh_row + cb + c + 1));
          if (RES && rvec) b += __uint_as_float(rw[e] & 0xffff0000u);
          else if (RES && res_row) b += __bfloat162float(res_row[cb + c + 1]);
        }
      }
      if (ACT == DSN_ACT_GELU) gelu_pair(a, b, a, b);
      else { a = apply_act<ACT>(a); b = apply_act<ACT>(b); }
      __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
      out[4 * jj + e] = *reinterpret_cast<uint32_t*>(&h);
    }
  }
}

// Epilogue of one tile for one warp: accumulator rows (one per lane) -> bias, activation, bf16 ->
// 32 x 128-byte swizzled staging tile -> global memory.  The warp takes the 64-column chunks
// `first`, `first + kEpiWarps / 4`, ...  `yrow` is this lane's output row (nullptr when the row is not part of the
// result).  With `contig` the 32 rows are consecutive output rows starting at
// `base_row` and each chunk leaves as one TMA store (columns clipped by the map); otherwise eight
// lanes store one 128-byte piece of a row each.
template <int ACT, bool AFF, bool RES = false>
__device__ __forceinline__ void epilogue_tile(uint32_t taddr, int ncols, int n0, int first, const float* brow,
                                              const float* sc_row, const float* sh_row, const __nv_bfloat16* res_row, uint8_t* stage_w, __nv_bfloat16* yrow, int lane, bool contig,
                                              const CUtensorMap* mapY, int base_row) {
  for (int c0 = 64 * first; c0 < ncols; c0 += 16 * kEpiWarps) {
    // an earlier TMA store of this warp (this tile or the one before) must have finished reading the
    // staging tile before it is overwritten; free when nothing is outstanding
    if (elect_one()) bulk_wait_read0();
    __syncwarp();
    // phase 1: this thread's row, 64 columns -> bf16 -> its 128-byte row of the staging tile
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      if (c0 + 32 * half < ncols) {  // warp-uniform
        uint32_t w[16];
        epilogue_half<ACT, AFF, RES>(taddr + c0 + 32 * half, c0 + 32 * half, ncols, brow, sc_row, sh_row, res_row, w);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = 4 * half + jj;
          *reinterpret_cast<uint4*>(stage_w + lane * 128 + ((j ^ (lane & 7)) << 4)) =
              make_uint4(w[4 * jj], w[4 * jj + 1], w[4 * jj + 2], w[4 * jj + 3]);
        }
      }
    }
    if (contig) {
      // The store's tensor map ends at the slice width rounded DOWN to 8 columns (a TMA store clips at 16-byte
      // granularity); a width that is no multiple of 8 leaves 1..7 columns, which every lane writes for its own row.
      fence_async_smem();
      __syncwarp();
      if (elect_one()) {
        tma_store_2d(mapY, n0 + c0, base_row, smem_u32(stage_w));
        bulk_commit();
      }
      const int col8 = ncols & ~7, tail_n = ncols & 7;
      if (tail_n != 0 && col8 >= c0 && col8 < c0 + 64) {
        const int j = (col8 - c0) >> 3;
        const uint4 val = *reinterpret_cast<const uint4*>(stage_w + lane * 128 + ((j ^ (lane & 7)) << 4));
        const uint32_t w[4] = {val.x, val.y, val.z, val.w};
        store_row_tail(yrow + col8, w, tail_n);
      }
      continue;
    }
    __syncwarp();
    // phase 2: eight lanes per row, 16 bytes each: contiguous 128-byte pieces of output rows.  Lane l
    // stores row 4*i + l/8 of the warp's 32 rows in step i; the row pointers come from their owners.
    __nv_bfloat16* rp[8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
      rp[i] = reinterpret_cast<__nv_bfloat16*>(
          __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(yrow), 4 * i + (lane >> 3)));
    const int j = lane & 7, col = c0 + 8 * j;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = 4 * i + (lane >> 3);
      if (rp[i] != nullptr && col < ncols) {
        const uint4 val = *reinterpret_cast<const uint4*>(stage_w + row * 128 + ((j ^ (row & 7)) << 4));
        if (col + 8 <= ncols) {
          *reinterpret_cast<uint4*>(rp[i] + col) = val;
        } else {  // slice width not a multiple of 8: the 1..7 columns left leave as one 8-, one 4- and one 2-byte store
          // (the piece starts on a 16-byte boundary of the row whenever the row itself does; an odd start falls back to 2-byte stores)
          const uint32_t w[4] = {val.x, val.y, val.z, val.w};
          store_row_tail(rp[i] + col, w, ncols - col);
        }
      }
    }
    __syncwarp();
  }
}

}  // namespace dsn_gemm
