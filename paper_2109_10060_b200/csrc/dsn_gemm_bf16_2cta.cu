// Ragged grouped sliced GEMM on CTA pairs (tcgen05 cta_group::2), bf16 operands, fp32 accumulation.
//
// Same contract as the one-CTA kernel, different tile ownership: a cluster of two CTAs (two SMs)
// computes a 256-row x BN-column tile.  Each CTA loads its own 128 activation rows and HALF of the
// weight tile (BN/2 rows), the even CTA's MMA thread issues tcgen05.mma.cta_group::2 with M = 256,
// and the tensor cores of both SMs read both halves of the weight tile.  Per SM the operand traffic
// from L2 into shared memory drops from 16 KB + 32 KB to 16 KB + 16 KB per 128x256x64 block of
// work, which is what bounds the one-CTA kernel on wide layers.  No multicast loads are used: every
// CTA fetches its own bytes.
//
// Barriers (every CTA has the same shared-memory layout):
//   full[s]    even CTA only.  One arrival (its producer's expect_tx for the bytes of BOTH CTAs);
//              the TMA loads of both CTAs complete their bytes on it.
//   empty[s]   both CTAs.  The even CTA's tcgen05.commit (multicast to both) frees the stage.
//   tfull[a]   both CTAs.  The same multicast commit tells both epilogues that accumulator a is done.
//   tempty[a]  even CTA only, 2 x 8 arrivals: the epilogue warps of both CTAs (remote arrive).
// Every wait is bounded; on a timeout the CTA flags DSN_ERR_TIMEOUT and leaves its loops.
#include <cuda_runtime.h>

#include "dsn_gemm_pair_device.cuh"

namespace {

using namespace dsn_gemm;

// kRes: the layer has skip features (residual add before the activation).  The form without them holds no
// trace of that code: its registers and code size weighed on every other epilogue variant.
// kLean (only without kRes): no bias, no per-path affine, no GELU: the epilogue holds the plain and the ReLU
// variant only.
template <bool kRes, bool kLean>
__global__ void __launch_bounds__(kThreads, 1) gemm_bf16_pair_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const GemmGeom& g = p.g;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);

  const uint32_t bar_full = base;
  const uint32_t bar_empty = base + 8 * kMaxStages;
  const uint32_t bar_tfull = base + 16 * kMaxStages;
  const uint32_t bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16 * kMaxStages + 32);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 16 * kMaxStages + 36);

  const int stages = g.stages;
  const uint32_t bh_bytes = (uint32_t)(g.BN / 2) * BK * 2;  // this CTA's half of the weight tile
  const uint32_t stage_bytes = kABytes + bh_bytes;
  const uint32_t tiles_base = base + kCtrlBytes;
  uint8_t* out_stage = smem + kCtrlBytes + (size_t)stages * stage_bytes;
  int32_t* s_prefix = reinterpret_cast<int32_t*>(out_stage + kStageOutBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const uint32_t tmem_cols = 2u * (uint32_t)g.BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 2 * kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish_pair();
  }

  auto ntiles_of = [&](int grp) {
    const int sl = p.group_slice ? p.group_slice[grp] : grp;
    if (sl < 0 || sl >= p.T || p.map_id[sl] == 0xFF) return 0;
    const int cnt = p.offsets[grp + 1] - p.offsets[grp];
    if (cnt <= 0) return 0;
    const int mt = g.flat ? (cnt * g.R + BM - 1) / BM : ((cnt + g.nb - 1) / g.nb) * g.tiles_x * g.tiles_y;
    return ((mt + 1) / 2) * ((p.k_out[sl] + g.BN - 1) / g.BN);
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
  dsn_build_tile_prefix(p.G, s_prefix, ntiles_of);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything can arrive on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = s_prefix[p.G];
  PairCursor cursor;  // every role walks its own tile sequence

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    // The whole warp walks the schedule (addresses, coordinates and the loop itself stay
    // warp-uniform, which keeps the per-stage instruction count low); one elected lane issues.
    int stage = 0;
    uint32_t phase = 0;
    const uint32_t a_box_bytes = g.flat ? kABytes : (uint32_t)(g.bw * g.bh * g.nb) * BK * 2;
    const uint32_t tx_bytes = 2u * (a_box_bytes + bh_bytes);
    bool ok = true;
    for (int tile = pair; ok && tile < total; tile += npairs) {
      const PairTile t = decode_pair_tile(p, s_prefix, tile, rank, cursor);
      const CUtensorMap* mA = &p.mapA[t.map];
      const CUtensorMap* mB = &p.mapB[t.map];
      const int nkc = (t.ki + BK - 1) / BK;
      const int ncols = t.ncols;
      const int n_inst = (ncols + 31) & ~31;
      const int brow0 = t.n0 + rank * (n_inst >> 1);  // first weight row of this CTA's half
      int bsel = t.b0;
      if (g.a_input_order) bsel = t.b0 < t.p_end ? p.perm[t.b0] : p.B;  // past the group: out of range, zeros
      for (int tap = 0; ok && tap < g.taps; ++tap) {
        const int r = tap / g.KW, sx = tap - r * g.KW;
        const int cx = g.flat ? t.row0 : t.x0 + sx - g.pad, cy = g.flat ? 0 : t.y0 + r - g.pad, cb = g.flat ? 0 : bsel;
        for (int kc = 0; kc < nkc; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, 11));
          if (!ok) break;
          if (elect_one()) {
            const uint32_t full_lead = leader_addr(bar_full + 8 * stage);  // the even CTA's barrier
            if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, tx_bytes);
            const uint32_t sa = tiles_base + stage * stage_bytes;
            tma_load_4d_pair(sa, mA, kc * BK, cx, cy, cb, full_lead);
            tma_load_3d_pair(sa + kABytes, mB, kc * BK, tap, brow0, full_lead);
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    // Warp-uniform loop, one elected lane issues.  The issuing warp is the critical resource of a tile with
    // wide N (four instructions of 128 tensor-pipe cycles per stage), so the per-stage path is
    // kept short: running descriptors, four unrolled K steps, a separate short loop for a partial
    // last chunk.
    if (rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      const uint64_t da0 = make_smem_desc(tiles_base), db0 = make_smem_desc(tiles_base + kABytes);
      const uint64_t dstep = (uint64_t)(stage_bytes >> 4);
      uint64_t da = da0, db = db0;
      for (int tile = pair; ok && tile < total; tile += npairs, ++it) {
        const PairTile t = decode_pair_tile(p, s_prefix, tile, 0, cursor);
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, p.status, 12));
        if (!ok) break;
        tc_fence_after();
        const int ncols = t.ncols;
        const int n_inst = (ncols + 31) & ~31;
        const uint32_t idesc = make_idesc(2 * BM, n_inst);
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * g.BN);
        const int nkc = (t.ki + BK - 1) / BK;
        const int tail_ks = ((t.ki & (BK - 1)) + 15) >> 4;  // K steps of a partial last chunk (0: none)
        uint32_t accumulate = 0;
        for (int tap = 0; ok && tap < g.taps; ++tap) {
          for (int kc = nkc; kc > 0; --kc) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status, 13));
            if (!ok) break;
            tc_fence_after();
            const int nks = (kc == 1 && tail_ks != 0) ? tail_ks : BK / 16;
            if (elect_one()) {
              umma_bf16_pair(d_tmem, da, db, idesc, accumulate);  // +32 bytes per K step
              if (nks > 1) umma_bf16_pair(d_tmem, da + 2u, db + 2u, idesc, 1u);
              if (nks > 2) umma_bf16_pair(d_tmem, da + 4u, db + 4u, idesc, 1u);
              if (nks > 3) umma_bf16_pair(d_tmem, da + 6u, db + 6u, idesc, 1u);
              umma_commit_pair(bar_empty + 8 * stage);
            }
            accumulate = 1;
            da += dstep;
            db += dstep;
            if (++stage == stages) { stage = 0; phase ^= 1u; da = da0; db = db0; }
          }
        }
        if (ok && elect_one()) umma_commit_pair(bar_tfull + 8 * acc);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;
    const int first = (warp - 2) >> 2;
    const int m = q * 32 + lane;
    int it = 0;
    bool ok = true;
    const int box_rows = g.bw * g.bh * g.nb, img_rows = g.bw * g.bh;
    // this thread's place in a per-image tile does not change from tile to tile
    const int row_bi = g.flat ? 0 : m / img_rows, row_rem = g.flat ? 0 : m - row_bi * img_rows;
    const int row_j = g.flat ? 0 : row_rem / g.bw, row_x = g.flat ? 0 : row_rem - row_j * g.bw;
    for (int tile = pair; ok && tile < total; tile += npairs, ++it) {
      const PairTile t = decode_pair_tile(p, s_prefix, tile, rank, cursor);
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
        const int yy = t.y0 + row_j, xx = t.x0 + row_x;
        const int pp = t.b0 + row_bi;
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
      const int ncols = t.ncols;
      const long long base_row = __shfl_sync(0xffffffffu, (long long)out_row, 0);
      const bool contig = __all_sync(0xffffffffu, valid && out_row == base_row + lane) && t.ko >= 8;

      ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, p.status, 14));
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
          case 1: if constexpr (!kLean) epilogue_tile<DSN_ACT_NONE, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 2: epilogue_tile<DSN_ACT_RELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 3: if constexpr (!kLean) epilogue_tile<DSN_ACT_RELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          case 4: if constexpr (!kLean) epilogue_tile<DSN_ACT_GELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
          default: if constexpr (!kLean) epilogue_tile<DSN_ACT_GELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_addr(bar_tempty + 8 * acc));  // the even CTA's MMA thread waits on it
    }
    if (elect_one()) bulk_wait0();  // the lane that issued this warp's TMA stores
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA retires while its partner may still read its memory or signal its barriers
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, tmem_cols);
  }
}

}  // namespace

size_t dsn_gemm_pair_smem_bytes(int BN, int stages, int G) {
  return 1024 + kCtrlBytes + (size_t)stages * (kABytes + (size_t)(BN / 2) * BK * 2) + kStageOutBytes +
         sizeof(int32_t) * (3 * (size_t)G + 3);
}

// Largest number of CTA pairs that can be resident at once for this shared-memory size (0: no pair fits).
int dsn_gemm_pair_max_clusters(size_t smem_bytes) {
  if (cudaFuncSetAttribute(gemm_bf16_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) !=
      cudaSuccess)
    return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gemm_bf16_pair_kernel<false, false>, &cfg) != cudaSuccess) return 0;
  return n;
}

cudaError_t dsn_launch_gemm_bf16_pair(const GemmParams& p, int clusters, size_t smem_bytes, cudaStream_t s) {
  static size_t configured[3][DSN_MAX_DEVICES] = {};
  const bool lean = !p.residual && !p.bias && !p.bn_scale && p.act != DSN_ACT_GELU;
  const int form = p.residual ? 2 : (lean ? 1 : 0);
  void (*kernel)(GemmParams) = form == 2 ? gemm_bf16_pair_kernel<true, false>
                               : form == 1 ? gemm_bf16_pair_kernel<false, true> : gemm_bf16_pair_kernel<false, false>;
  {
    cudaError_t e = dsn_ensure_dynamic_smem(kernel, smem_bytes, configured[form]);
    if (e != cudaSuccess) return e;
  }
  return dsn_launch(kernel, dim3(2 * clusters), dim3(kThreads), smem_bytes, s, 2, p);
}
