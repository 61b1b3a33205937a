// Ragged grouped sliced GEMM, bf16 operands, fp32 accumulation, for sm_100a.
//
//   for every group g (samples routed to one path, slice (k_in, k_out)):
//       Y[rows of g, :k_out] = act( X[rows of g, :k_in] * W[:k_out, :k_in]^T + bias )
//
// The same kernel covers linear layers, 1x1 convolutions and 3x3 convolutions as implicit GEMM
// over channels-last activations: the reduction runs over (tap, channel chunk) and the activation
// tile of tap (r, s) is the output tile's pixel rectangle shifted by (r - pad, s - pad); the TMA
// unit zero-fills what falls outside the image, which is the convolution's zero padding.
//
// Operands are read in place.  Every distinct slice (k_in, k_out) has its own pair of tensor maps
// whose extents are the slice's (k_in channels; k_out weight rows) but whose strides are those of
// the full tensors, so everything beyond the slice arrives in shared memory as zeros: it is never
// fetched from L2 and never multiplied.
//
// Structure of a CTA (persistent, one per SM, 320 threads):
//   warp 0      walks the tile schedule (warp-uniform loop), one elected lane issues the TMA loads into a ring of stages
//   warp 1      same form, one elected lane issues tcgen05.mma (M = 128, N = 16..256, K = 16) into a TMEM accumulator;
//               two accumulator buffers let the epilogue of tile i overlap the main loop of tile i+1
//   warps 2..9  epilogue, two warps per TMEM lane quarter taking alternate 64-column chunks:
//               tcgen05.ld (one accumulator row per thread), bias / activation, bf16 rounding into a
//               32-row x 128-byte swizzled staging tile, then one TMA store of that tile when the
//               warp's 32 rows are consecutive rows of the output (the tensor map clips the columns
//               at k_out); otherwise stores in which eight lanes write one contiguous 128-byte
//               piece of an output row (group tails, sample boundaries of scattered output)
// Every mbarrier wait is bounded; on a timeout the CTA records DSN_ERR_TIMEOUT, stops issuing
// work, lets its copies land, frees its TMEM and returns.
#include "dsn_gemm_device.cuh"

namespace {

using namespace dsn_gemm;

// ---------------------------------------------------------------------------------- tile decode
struct TileInfo {
  int map, ki, ko, n0, slice;
  int p_end;            // one past the group's last grouped position
  int row0, rows_end;   // flat: first grouped row of the tile, one past the group's last row
  int b0, x0, y0;       // per-image tiling: first position, pixel origin
};

__device__ __forceinline__ TileInfo decode_tile(const GemmParams& p, const int32_t* s_prefix, int tile) {
  TileInfo t;
  const GemmGeom& g = p.g;
  const int j = dsn_find_tile_slot(s_prefix, p.G, tile);
  const int grp = p.G - 1 - j;
  const int sl = s_prefix[2 * p.G + 2 + grp];  // group -> slice, cached in shared memory
  t.slice = sl;
  t.map = p.map_id[sl];
  t.ki = p.k_in[sl];
  t.ko = p.k_out[sl];
  const int p0 = s_prefix[p.G + 1 + grp];      // group offsets, cached in shared memory
  t.p_end = s_prefix[p.G + 2 + grp];
  const int ntn = (t.ko + g.BN - 1) / g.BN;
  const int local = tile - s_prefix[j];
  const int nt = local % ntn, mt = local / ntn;
  t.n0 = nt * g.BN;
  if (g.flat) {
    t.row0 = p0 * g.R + mt * BM;
    t.rows_end = t.p_end * g.R;
    t.b0 = t.x0 = t.y0 = 0;
  } else {
    const int per_img = g.tiles_x * g.tiles_y;
    const int ib = mt / per_img, rem = mt - ib * per_img;
    const int ty = rem / g.tiles_x, tx = rem - ty * g.tiles_x;
    t.b0 = p0 + ib * g.nb;
    t.y0 = ty * g.bh;
    t.x0 = tx * g.bw;
    t.row0 = t.rows_end = 0;
  }
  return t;
}

// ---------------------------------------------------------------------------------- kernel
// kRes: the layer has skip features (residual add before the activation).  The form without them holds no
// trace of that code: its registers and code size weighed on every other epilogue variant.
template <bool kRes>
__global__ void __launch_bounds__(kThreads, 1) gemm_bf16_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const GemmGeom& g = p.g;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);

  // control block
  const uint32_t bar_full = base;                       // [kMaxStages]
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
  const uint32_t tmem_cols = 2u * (uint32_t)g.BN;  // 128, 256 or 512: a power of two >= 32

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
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
    const int mt = g.flat ? (cnt * g.R + BM - 1) / BM : ((cnt + g.nb - 1) / g.nb) * g.tiles_x * g.tiles_y;
    return mt * ((p.k_out[sl] + g.BN - 1) / g.BN);
  };
  // barriers and TMEM are set up; everything below reads what earlier kernels wrote
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  // s_prefix[0..G]: tile prefix; [G+1 .. 2G+1]: group offsets; [2G+2 .. 3G+1]: slice of each group
  for (int j = threadIdx.x; j <= p.G; j += blockDim.x) s_prefix[p.G + 1 + j] = p.offsets[j];
  for (int j = threadIdx.x; j < p.G; j += blockDim.x) {
    const int sl = p.group_slice ? p.group_slice[j] : j;
    s_prefix[2 * p.G + 2 + j] = (sl >= 0 && sl < p.T) ? sl : 0;
  }
  dsn_build_tile_prefix(p.G, s_prefix, ntiles_of);  // contains __syncthreads
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = s_prefix[p.G];

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The whole warp walks the schedule (warp-uniform loop), one elected lane issues the copies.
    int stage = 0;
    uint32_t phase = 0;
    const uint32_t a_box_bytes = g.flat ? kABytes : (uint32_t)(g.bw * g.bh * g.nb) * BK * 2;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x) {
      const TileInfo t = decode_tile(p, s_prefix, tile);
      const CUtensorMap* mA = &p.mapA[t.map];
      const CUtensorMap* mB = &p.mapB[t.map];
      const int nkc = (t.ki + BK - 1) / BK;
      int bsel = t.b0;
      if (g.a_input_order) bsel = p.perm[t.b0];
      for (int tap = 0; ok && tap < g.taps; ++tap) {
        const int r = tap / g.KW, sx = tap - r * g.KW;
        const int cx = g.flat ? t.row0 : t.x0 + sx - g.pad, cy = g.flat ? 0 : t.y0 + r - g.pad, cb = g.flat ? 0 : bsel;
        for (int kc = 0; kc < nkc; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, 1));
          if (!ok) break;
          if (elect_one()) {
            const uint32_t full = bar_full + 8 * stage;
            mbar_expect_tx(full, a_box_bytes + b_bytes);
            const uint32_t sa = tiles_base + stage * stage_bytes;
            tma_load_4d(sa, mA, kc * BK, cx, cy, cb, full);
            tma_load_3d(sa + kABytes, mB, kc * BK, tap, t.n0, full);
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
    if (!ok && lane == 0) {
      // let copies already issued land before the CTA gives up its shared memory
      for (int s = 0; s < stages; ++s) {
        const uint64_t t0 = globaltimer_ns();
        const uint32_t par = (s < stage) ? phase : (phase ^ 1u);
        while (!mbar_try_wait(bar_full + 8 * s, par) && globaltimer_ns() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // Warp-uniform loop, one elected lane issues: running descriptors, four unrolled K steps.
    int stage = 0;
    uint32_t phase = 0;
    int it = 0;
    bool ok = true;
    const uint64_t da0 = make_smem_desc(tiles_base), db0 = make_smem_desc(tiles_base + kABytes);
    const uint64_t dstep = (uint64_t)(stage_bytes >> 4);
    uint64_t da = da0, db = db0;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x, ++it) {
      const TileInfo t = decode_tile(p, s_prefix, tile);
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, p.status, 2));
      if (!ok) break;
      tc_fence_after();
      int n_inst = t.ko - t.n0;
      n_inst = n_inst > g.BN ? g.BN : ((n_inst + 15) & ~15);
      const uint32_t idesc = make_idesc(BM, n_inst);
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * g.BN);
      const int nkc = (t.ki + BK - 1) / BK;
      const int tail_ks = ((t.ki & (BK - 1)) + 15) >> 4;  // K steps of a partial last chunk (0: none)
      uint32_t accumulate = 0;
      for (int tap = 0; ok && tap < g.taps; ++tap) {
        for (int kc = nkc; kc > 0; --kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status, 3));
          if (!ok) break;
          tc_fence_after();
          const int nks = (kc == 1 && tail_ks != 0) ? tail_ks : BK / 16;
          if (elect_one()) {
            umma_bf16(d_tmem, da, db, idesc, accumulate);  // +32 bytes per K step
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
      }
      if (ok && elect_one()) umma_commit(bar_tfull + 8 * acc);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int q = warp & 3;          // TMEM lane quarter this warp may read
    const int first = (warp - 2) >> 2;  // which alternate 64-column chunks this warp takes
    const int m = q * 32 + lane;     // accumulator row of this thread
    int it = 0;
    bool ok = true;
    const int box_rows = g.bw * g.bh * g.nb, img_rows = g.bw * g.bh;
    for (int tile = blockIdx.x; ok && tile < total; tile += gridDim.x, ++it) {
      const TileInfo t = decode_tile(p, s_prefix, tile);
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;

      bool valid;
      int64_t out_row;
      if (g.flat) {
        const int gr = t.row0 + m;
        valid = gr < t.rows_end;
        out_row = gr;
        if (valid && g.y_input_order) {
          const int pp = gr / g.R;
          out_row = (int64_t)p.perm[pp] * g.R + (gr - pp * g.R);
        }
      } else {
        const int bi = m / img_rows, rem = m - bi * img_rows;
        const int yy = t.y0 + rem / g.bw, xx = t.x0 + rem % g.bw;
        const int pp = t.b0 + bi;
        valid = m < box_rows && yy < g.H && xx < g.W && pp < t.p_end;
        out_row = 0;
        if (valid) {
          const int smp = g.y_input_order ? p.perm[pp] : pp;
          out_row = (int64_t)smp * g.R + yy * g.W + xx;
        }
      }
      __nv_bfloat16* yrow = valid ? p.y + out_row * p.ldy + t.n0 : nullptr;
      const float* brow = p.bias ? p.bias + t.n0 : nullptr;
      const float* sc_row = p.bn_scale ? p.bn_scale + (int64_t)t.slice * p.bn_ld + t.n0 : nullptr;
      const float* sh_row = p.bn_scale ? p.bn_shift + (int64_t)t.slice * p.bn_ld + t.n0 : nullptr;
      const __nv_bfloat16* res_row = (kRes && valid) ? p.residual + out_row * p.ldy + t.n0 : nullptr;
      int ncols = t.ko - t.n0;
      ncols = ncols > g.BN ? g.BN : ncols;
      const long long base_row = __shfl_sync(0xffffffffu, (long long)out_row, 0);
      // (a slice width that is no multiple of 8 columns = 16 bytes keeps the element-wise path: the
      // store was seen to clip the row at 16-byte granularity and would touch columns >= k_out)
      const bool contig = __all_sync(0xffffffffu, valid && out_row == base_row + lane) && t.ko >= 8;

      // every lane waits, then the warp takes one decision so that tcgen05.ld stays warp-wide
      ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, p.status, 4));
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * g.BN);
      uint8_t* stage_w = out_stage + (warp - 2) * (32 * 128);
      const CUtensorMap* mY = &p.mapY[t.map];
      if constexpr (kRes) {
        switch (p.act) {
          case DSN_ACT_NONE: epilogue_tile<DSN_ACT_NONE, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case DSN_ACT_RELU: epilogue_tile<DSN_ACT_RELU, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          default: epilogue_tile<DSN_ACT_GELU, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        }
      } else {
        const int variant = p.act * 2 + ((brow || sc_row) ? 1 : 0);
        switch (variant) {
          case 0: epilogue_tile<DSN_ACT_NONE, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 1: epilogue_tile<DSN_ACT_NONE, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 2: epilogue_tile<DSN_ACT_RELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 3: epilogue_tile<DSN_ACT_RELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 4: epilogue_tile<DSN_ACT_GELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          default: epilogue_tile<DSN_ACT_GELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
    }
    if (elect_one()) bulk_wait0();  // this warp's TMA stores (issued by the elected lane) are complete before the CTA retires
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
}

}  // namespace

size_t dsn_gemm_smem_bytes(int BN, int stages, int G) {
  return 1024 /* alignment slack */ + kCtrlBytes + (size_t)stages * (kABytes + (size_t)BN * BK * 2) + kStageOutBytes +
         sizeof(int32_t) * (3 * (size_t)G + 3);
}

cudaError_t dsn_launch_gemm_bf16(const GemmParams& p, int sm_count, size_t smem_bytes, cudaStream_t s) {
  static size_t configured[2][DSN_MAX_DEVICES] = {};
  const int res = p.residual ? 1 : 0;
  void (*kernel)(GemmParams) = res ? gemm_bf16_kernel<true> : gemm_bf16_kernel<false>;
  {
    cudaError_t e = dsn_ensure_dynamic_smem(kernel, smem_bytes, configured[res]);
    if (e != cudaSuccess) return e;
  }
  return dsn_launch(kernel, dim3(sm_count), dim3(kThreads), smem_bytes, s, 1, p);
}
