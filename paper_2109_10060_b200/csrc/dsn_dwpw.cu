// Depthwise-separable block of the slice-able MobileNet (Sec. 3.3: group convolution whose group count follows
// the elastic width, kernel-size slicing; routing-space table of DS-MBNet): depthwise k x k on the c_t leading
// channels (+ bias, per-path affine, activation, rounded to bf16) fused with the pointwise 1x1 layer
//   Y[rows of g, :k_out] = act( D[rows of g, :c_t] * W[:k_out, :c_t]^T + bias ),   D = depthwise(X)
// so that the c_t-wide tensor between the two never goes to global memory.
//
// The pointwise part is the ragged grouped GEMM of dsn_gemm_bf16.cu (one persistent CTA per SM, tcgen05 MMA with
// M = 128, TMEM accumulators, weights by TMA).  Its A operand, however, is not loaded: four producer warps
// compute it.  For a stage (128 output pixels x 64 channels) eight lanes share a pixel, each owning 8 channels
// (16 bytes): they read the k x k window of the input in place (channels last, so a warp's load covers whole
// 128-byte lines; neighbouring windows are served by L1), accumulate in fp32, apply the depthwise epilogue,
// round to bf16 (the value the unfused path would have stored) and write the 16 bytes into the swizzled K-major
// tile the tensor core reads.  Because the rows are produced, not loaded, M rows are the group's output pixels in
// grouped order with no regard to sample boundaries, whatever the order of the input: no padding rows and no
// gather pass.  An n-tile is 256 columns wide; wider slices run the reduction once per n-tile (the depthwise
// arithmetic is a few percent of the pointwise tile's).
//
// Roles (448 threads): warp 0 weight loads (TMA), warp 1 MMA issue, warps 2-9 epilogue (dsn_gemm_device.cuh),
// warps 10-13 depthwise producers.  Every wait is bounded.
#include "dsn_gemm_device.cuh"
#include "dsn_tiles.cuh"

namespace {

using namespace dsn_gemm;

constexpr int kProdWarps = 4;
constexpr int kDwThreads = kThreads + 32 * kProdWarps;

struct TileInfo {
  int map, ki, ko, n0, slice;
  int row0, rows_end;
};

__device__ __forceinline__ TileInfo decode_tile(const DwPwParams& q, const int32_t* s_prefix, int tile) {
  const GemmParams& p = q.g;
  TileInfo t;
  const int j = dsn_find_tile_slot(s_prefix, p.G, tile);
  const int grp = p.G - 1 - j;
  const int sl = s_prefix[2 * p.G + 2 + grp];
  t.slice = sl;
  t.map = p.map_id[sl];
  t.ki = p.k_in[sl];
  t.ko = p.k_out[sl];
  const int p0 = s_prefix[p.G + 1 + grp];
  const int p_end = s_prefix[p.G + 2 + grp];
  const int ntn = (t.ko + p.g.BN - 1) / p.g.BN;
  const int local = tile - s_prefix[j];
  const int nt = local % ntn, mt = local / ntn;
  t.n0 = nt * p.g.BN;
  t.row0 = p0 * p.g.R + mt * BM;
  t.rows_end = p_end * p.g.R;
  return t;
}

template <int ACT>
__device__ __forceinline__ uint4 dw_finish(const float (&acc)[8], const float* bias, const float* sc, const float* sh, int c0) {
  uint32_t o[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float a = acc[2 * j], b = acc[2 * j + 1];
    if (bias) { a += __ldg(bias + c0 + 2 * j); b += __ldg(bias + c0 + 2 * j + 1); }
    if (sc) {
      a = fmaf(a, __ldg(sc + c0 + 2 * j), __ldg(sh + c0 + 2 * j));
      b = fmaf(b, __ldg(sc + c0 + 2 * j + 1), __ldg(sh + c0 + 2 * j + 1));
    }
    __nv_bfloat162 h = __floats2bfloat162_rn(apply_act<ACT>(a), apply_act<ACT>(b));
    o[j] = *reinterpret_cast<uint32_t*>(&h);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

__global__ void __launch_bounds__(kDwThreads, 1) dwpw_kernel(const __grid_constant__ DwPwParams q) {
  extern __shared__ uint8_t smem_raw[];
  const GemmParams& p = q.g;
  const GemmGeom& g = p.g;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);

  const uint32_t bar_full = base;                       // [kMaxStages]: weights landed (1 arrival + bytes) and A written (kProdWarps arrivals)
  const uint32_t bar_empty = base + 8 * kMaxStages;     // [kMaxStages]
  const uint32_t bar_tfull = base + 16 * kMaxStages;    // [2]
  const uint32_t bar_tempty = bar_tfull + 16;           // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16 * kMaxStages + 32);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 16 * kMaxStages + 36);

  const int stages = g.stages;
  const uint32_t b_bytes = (uint32_t)g.BN * BK * 2;
  const uint32_t stage_bytes = kABytes + b_bytes;
  const uint32_t tiles_base = base + kCtrlBytes;
  uint8_t* out_stage = smem + kCtrlBytes + (size_t)stages * stage_bytes;
  int32_t* s_prefix = reinterpret_cast<int32_t*>(out_stage + kStageOutBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tmem_cols = 2u * (uint32_t)g.BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8 * s, 1 + kProdWarps);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish();
  }
  auto ntiles_of = [&](int grp) {
    const int sl = p.group_slice ? p.group_slice[grp] : grp;
    if (sl < 0 || sl >= p.T || p.map_id[sl] == 0xFF) return 0;
    const int cnt = p.offsets[grp + 1] - p.offsets[grp];
    if (cnt <= 0) return 0;
    return ((cnt * g.R + BM - 1) / BM) * ((p.k_out[sl] + g.BN - 1) / g.BN);
  };
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  for (int j = threadIdx.x; j <= p.G; j += blockDim.x) s_prefix[p.G + 1 + j] = p.offsets[j];
  for (int j = threadIdx.x; j < p.G; j += blockDim.x) {
    const int sl = p.group_slice ? p.group_slice[j] : j;
    s_prefix[2 * p.G + 2 + j] = (sl >= 0 && sl < p.T) ? sl : 0;
  }
  dsn_build_tile_prefix(p.G, s_prefix, ntiles_of);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = s_prefix[p.G];

  if (warp == 0) {
    // ------------------------------------------------------------------ weight loads
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
      const TileInfo t = decode_tile(q, s_prefix, tile);
      const CUtensorMap* mB = &p.mapB[t.map];
      const int nkc = (t.ki + BK - 1) / BK;
      for (int kc = 0; kc < nkc; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, 41));
        if (!ok) break;
        if (elect_one()) {
          const uint32_t full = bar_full + 8 * stage;
          mbar_expect_tx(full, b_bytes);
          tma_load_3d(tiles_base + stage * stage_bytes + kABytes, mB, kc * BK, 0, t.n0, full);
        }
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) {
      for (int s = 0; s < stages; ++s) {  // let copies already issued land before the CTA gives up its shared memory
        const uint64_t t0 = globaltimer_ns();
        const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
        while (!mbar_try_wait(bar_full + 8 * s, par) && globaltimer_ns() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    int stage = 0;
    uint32_t phase = 0;
    int it = 0;
    bool ok = true;
    const uint64_t da0 = make_smem_desc(tiles_base), db0 = make_smem_desc(tiles_base + kABytes);
    const uint64_t dstep = (uint64_t)(stage_bytes >> 4);
    uint64_t da = da0, db = db0;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x, ++it) {
      const TileInfo t = decode_tile(q, s_prefix, tile);
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, p.status, 42));
      if (!ok) break;
      tc_fence_after();
      int n_inst = t.ko - t.n0;
      n_inst = n_inst > g.BN ? g.BN : ((n_inst + 15) & ~15);
      const uint32_t idesc = make_idesc(BM, n_inst);
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * g.BN);
      const int nkc = (t.ki + BK - 1) / BK;
      const int tail_ks = ((t.ki & (BK - 1)) + 15) >> 4;
      uint32_t accumulate = 0;
      for (int kc = nkc; kc > 0; --kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status, 43));
        if (!ok) break;
        tc_fence_after();
        const int nks = (kc == 1 && tail_ks != 0) ? tail_ks : BK / 16;
        if (elect_one()) {
          umma_bf16(d_tmem, da, db, idesc, accumulate);
          if (nks > 1) umma_bf16(d_tmem, da + 2u, db + 2u, idesc, 1u);
          if (nks > 2) umma_bf16(d_tmem, da + 4u, db + 4u, idesc, 1u);
          if (nks > 3) umma_bf16(d_tmem, da + 6u, db + 6u, idesc, 1u);
          umma_commit(bar_empty + 8 * stage);
        }
        accumulate = 1;
        da += dstep;
        db += dstep;
        if (++stage == stages) { stage = 0; phase ^= 1u; da = da0; db = db0; }
      }
      if (ok && elect_one()) umma_commit(bar_tfull + 8 * acc);
    }
  } else if (warp < 2 + kEpiWarps) {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int qd = warp & 3;
    const int first = (warp - 2) >> 2;
    const int m = qd * 32 + lane;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x, ++it) {
      const TileInfo t = decode_tile(q, s_prefix, tile);
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      const int gr = t.row0 + m;
      const bool valid = gr < t.rows_end;
      int64_t out_row = gr;
      if (valid && g.y_input_order) {
        const int pp = gr / g.R;
        out_row = (int64_t)p.perm[pp] * g.R + (gr - pp * g.R);
      }
      __nv_bfloat16* yrow = valid ? p.y + out_row * p.ldy + t.n0 : nullptr;
      const float* brow = p.bias ? p.bias + t.n0 : nullptr;
      const float* sc_row = p.bn_scale ? p.bn_scale + (int64_t)t.slice * p.bn_ld + t.n0 : nullptr;
      const float* sh_row = p.bn_scale ? p.bn_shift + (int64_t)t.slice * p.bn_ld + t.n0 : nullptr;
      int ncols = t.ko - t.n0;
      ncols = ncols > g.BN ? g.BN : ncols;
      const long long base_row = __shfl_sync(0xffffffffu, (long long)out_row, 0);
      const bool contig = __all_sync(0xffffffffu, valid && out_row == base_row + lane) && t.ko >= 8;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, p.status, 44));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)(acc * g.BN);
      uint8_t* stage_w = out_stage + (warp - 2) * (32 * 128);
      const CUtensorMap* mY = &p.mapY[t.map];
      const int variant = p.act * 2 + ((brow || sc_row) ? 1 : 0);
      switch (variant) {
        case 0: epilogue_tile<DSN_ACT_NONE, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 1: epilogue_tile<DSN_ACT_NONE, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 2: epilogue_tile<DSN_ACT_RELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 3: epilogue_tile<DSN_ACT_RELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 4: epilogue_tile<DSN_ACT_GELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        default: epilogue_tile<DSN_ACT_GELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, nullptr, stage_w, yrow, lane, contig, mY, (int)base_row); break;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
    }
    if (elect_one()) bulk_wait0();
  } else {
    // ------------------------------------------------------------------ depthwise producers (warps 10..13)
    const int pw = warp - 2 - kEpiWarps;     // 0..3
    const int cg = lane & 7;                 // channel group of 8 within the 64-channel chunk
    const int rsub = lane >> 3;              // 4 rows per warp pass
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    const int Ro = g.R, Wo = q.Wo, K = q.K, stride = q.stride, H = q.H, W = q.W;
    constexpr int kPasses = BM / (4 * kProdWarps);   // rows of the tile this thread produces
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
      const TileInfo t = decode_tile(q, s_prefix, tile);
      const int k = q.ksize[t.slice];
      const int k0 = (K - k) >> 1, pad = (k - 1) >> 1;
      const float* sc = q.dw_bn_scale ? q.dw_bn_scale + (int64_t)t.slice * q.C : nullptr;
      const float* sh = q.dw_bn_scale ? q.dw_bn_shift + (int64_t)t.slice * q.C : nullptr;
      const int nkc = (t.ki + BK - 1) / BK;
      // this thread's rows of the tile: input sample and the window's origin, looked up once per tile
      const __nv_bfloat16* xrow[kPasses];
      int yx[kPasses];   // (iy0 + 8) << 16 | (ix0 + 8): origin of the window in the input, biased to stay positive
#pragma unroll
      for (int pass = 0; pass < kPasses; ++pass) {
        const int gr = t.row0 + pass * (4 * kProdWarps) + pw * 4 + rsub;
        xrow[pass] = nullptr;
        yx[pass] = 0;
        if (gr < t.rows_end) {
          const int pp = gr / Ro, pix = gr - pp * Ro;
          const int oy = pix / Wo, ox = pix - oy * Wo;
          const int smp = g.a_input_order ? p.perm[pp] : pp;
          xrow[pass] = q.x + (int64_t)smp * H * W * q.ldx;
          yx[pass] = ((oy * stride - pad + 8) << 16) | (ox * stride - pad + 8);
        }
      }
      for (int kc = 0; kc < nkc; ++kc) {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, 45));
        if (!ok) break;
        uint8_t* a_tile = smem + kCtrlBytes + (size_t)stage * stage_bytes;
        const int c0 = kc * BK + cg * 8;
        const bool ch_ok = c0 < t.ki;  // widths are multiples of 8: a group of 8 channels is inside the slice or outside
        if (k == 3) {
          // 3 x 3: the nine filter vectors of this channel group stay in registers for the whole stage; the nine
          // input vectors of a row are fetched in one round (out-of-image taps read as zeros = the padding)
          uint4 wv[9];
#pragma unroll
          for (int tap = 0; tap < 9; ++tap)
            wv[tap] = ch_ok ? __ldg(reinterpret_cast<const uint4*>(q.w + ((int64_t)(k0 + tap / 3) * K + (k0 + tap % 3)) * q.C + c0))
                            : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
          for (int pass = 0; pass < kPasses; ++pass) {
            const int m = pass * (4 * kProdWarps) + pw * 4 + rsub;
            uint4 outv = make_uint4(0u, 0u, 0u, 0u);
            if (ch_ok && xrow[pass]) {
              const int iy0 = (yx[pass] >> 16) - 8, ix0 = (yx[pass] & 0xffff) - 8;
              uint4 xv[9];
#pragma unroll
              for (int tap = 0; tap < 9; ++tap) {
                const int iy = iy0 + tap / 3, ix = ix0 + tap % 3;
                xv[tap] = (iy >= 0 && iy < H && ix >= 0 && ix < W)
                              ? __ldg(reinterpret_cast<const uint4*>(xrow[pass] + ((int64_t)iy * W + ix) * q.ldx + c0))
                              : make_uint4(0u, 0u, 0u, 0u);
              }
              float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
              for (int tap = 0; tap < 9; ++tap) {
                const uint32_t xa[4] = {xv[tap].x, xv[tap].y, xv[tap].z, xv[tap].w};
                const uint32_t wa[4] = {wv[tap].x, wv[tap].y, wv[tap].z, wv[tap].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  acc[2 * j] = fmaf(__uint_as_float(xa[j] << 16), __uint_as_float(wa[j] << 16), acc[2 * j]);
                  acc[2 * j + 1] = fmaf(__uint_as_float(xa[j] & 0xffff0000u), __uint_as_float(wa[j] & 0xffff0000u), acc[2 * j + 1]);
                }
              }
              if (q.dw_act == DSN_ACT_RELU) outv = dw_finish<DSN_ACT_RELU>(acc, q.dw_bias, sc, sh, c0);
              else if (q.dw_act == DSN_ACT_GELU) outv = dw_finish<DSN_ACT_GELU>(acc, q.dw_bias, sc, sh, c0);
              else outv = dw_finish<DSN_ACT_NONE>(acc, q.dw_bias, sc, sh, c0);
            }
            *reinterpret_cast<uint4*>(a_tile + m * 128 + ((cg ^ (m & 7)) << 4)) = outv;
          }
        } else {
          // other kernel sizes: tap by tap (the pass loop is unrolled so that the per-row data stay in registers)
#pragma unroll
          for (int pass = 0; pass < kPasses; ++pass) {
            const int m = pass * (4 * kProdWarps) + pw * 4 + rsub;
            uint4 outv = make_uint4(0u, 0u, 0u, 0u);
            if (ch_ok && xrow[pass]) {
              const int iy0 = (yx[pass] >> 16) - 8, ix0 = (yx[pass] & 0xffff) - 8;
              float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
              for (int r = 0; r < k; ++r) {
                const int iy = iy0 + r;
                if (iy < 0 || iy >= H) continue;
                for (int s2 = 0; s2 < k; ++s2) {
                  const int ix = ix0 + s2;
                  if (ix < 0 || ix >= W) continue;
                  const uint4 xv = __ldg(reinterpret_cast<const uint4*>(xrow[pass] + ((int64_t)iy * W + ix) * q.ldx + c0));
                  const uint4 wv = __ldg(reinterpret_cast<const uint4*>(q.w + ((int64_t)(k0 + r) * K + (k0 + s2)) * q.C + c0));
                  const uint32_t xa[4] = {xv.x, xv.y, xv.z, xv.w}, wa[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    acc[2 * j] = fmaf(__uint_as_float(xa[j] << 16), __uint_as_float(wa[j] << 16), acc[2 * j]);
                    acc[2 * j + 1] = fmaf(__uint_as_float(xa[j] & 0xffff0000u), __uint_as_float(wa[j] & 0xffff0000u), acc[2 * j + 1]);
                  }
                }
              }
              if (q.dw_act == DSN_ACT_RELU) outv = dw_finish<DSN_ACT_RELU>(acc, q.dw_bias, sc, sh, c0);
              else if (q.dw_act == DSN_ACT_GELU) outv = dw_finish<DSN_ACT_GELU>(acc, q.dw_bias, sc, sh, c0);
              else outv = dw_finish<DSN_ACT_NONE>(acc, q.dw_bias, sc, sh, c0);
            }
            *reinterpret_cast<uint4*>(a_tile + m * 128 + ((cg ^ (m & 7)) << 4)) = outv;
          }
        }
        fence_async_smem();   // the tile is read by the tensor core (async proxy)
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_full + 8 * stage);
        if (++stage == stages) { stage = 0; phase ^= 1u; }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

}  // namespace

size_t dsn_dwpw_smem_bytes(int BN, int stages, int G) {
  return 1024 + kCtrlBytes + (size_t)stages * (kABytes + (size_t)BN * BK * 2) + kStageOutBytes +
         sizeof(int32_t) * (3 * (size_t)G + 3);
}

cudaError_t dsn_launch_dwpw(const DwPwParams& q, int sm_count, size_t smem_bytes, cudaStream_t s) {
  static size_t configured[DSN_MAX_DEVICES] = {};
  cudaError_t e = dsn_ensure_dynamic_smem(dwpw_kernel, smem_bytes, configured);
  if (e != cudaSuccess) return e;
  return dsn_launch(dwpw_kernel, dim3(sm_count), dim3(kDwThreads), smem_bytes, s, 1, q);
}
