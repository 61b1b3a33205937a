// 3x3 sliced convolution (stride 1, zero padding 1) on CTA pairs with the input tile staged ONCE.
//
// The tap-shifted form of the pair GEMM loads the activation tile nine times per 64-channel chunk
// (one TMA box per tap).  Here one TMA box per chunk brings the tile WITH its one-pixel halo
// ((bh + 2) image rows x (W + 2) pixels, out-of-image pixels zero-filled = the padding) into shared
// memory, and the nine taps are nine views of that block: row m of the MMA's A operand for tap
// (r, s) is halo pixel m + r (W + 2) + s, i.e. the same 128-byte rows read through a descriptor whose
// start address is moved by (r (W + 2) + s) x 128 bytes.  The 128-byte swizzle is a function of the
// shared-memory address bits for TMA and MMA alike, so a view that starts at any 128-byte row of a
// 1024-byte-aligned block reads the layout TMA wrote; the descriptor's base-offset field stays 0
// (checked on the device: with the row phase in that field the sums come out wrong).
// M rows are numbered over the padded width: m = j (W + 2) + x; the two rows per image row with
// x >= W compute nothing that is stored.  Weights stream through a ring of (tap, chunk) boxes as
// before; the activation blocks have a ring of their own (2 to 6 slots, as many as fit).
//
// Same contract, roles and accumulators as dsn_gemm_bf16_2cta.cu.  Added barriers:
//   afull[a]   even CTA only: the activation boxes of both CTAs have landed
//   aempty[a]  both CTAs: the MMAs of all nine taps that read the slot are done (multicast commit)
//
// Schedule.  A pair works on ONE contiguous range of the tile sequence (groups from the widest path down), the
// ranges cut so that every pair gets the same estimated tensor time (tensor instructions of a tile x their cycles,
// plus a fixed amount per tile).  Consecutive tiles of a range mostly share their slice, and when the weights of a
// (slice, n-tile) fit the ring whole they are loaded once and stay until a tile needs others: the issuing warp
// hands their slots back (commit on `empty`) only then.
//
// Epilogue.  With rows numbered over the padded width a warp's 32 rows are not 32 consecutive output rows (two
// padding positions per image row), so a store per warp cannot be one box.  The four warps of a column group
// therefore stage the CTA's 128 rows of a 64-column chunk in one shared block, and one TMA store over
// (channel, x, y, sample) writes it: the padding positions and the rows below the image lie outside the tensor
// and are clipped by the store.  Per group:
//   swritten   4 arrivals: each warp has written its 32 rows of the block
//   sfree      1 arrival: the store of the chunk before has finished reading the block
#include <cuda_runtime.h>

#include "dsn_gemm_pair_device.cuh"

namespace {

using namespace dsn_gemm;

// A run: the tiles of one group, which share everything but their place (sample, image rows).  The roles walk
// their tiles run by run: what depends on the slice is worked out once per run, and the place of a tile follows
// from the place of the tile before by adding a fixed step (no division per tile).
struct HaloRun {
  int lo, hi;              // tiles [lo, hi) of the schedule
  int slice, map, ki, ko;  // the group's slice, its tensor maps, its widths
  int p0, p_end;           // the group's positions of the grouped order
};
__device__ __forceinline__ HaloRun halo_find_run(const GemmParams& p, const int32_t* s_prefix, int tile) {
  HaloRun r;
  const int j = dsn_find_tile_slot(s_prefix, p.G, tile);
  const int grp = p.G - 1 - j;
  r.lo = s_prefix[j];
  r.hi = s_prefix[j + 1];
  r.slice = s_prefix[2 * p.G + 2 + grp];
  r.map = p.map_id[r.slice];
  r.ki = p.k_in[r.slice];
  r.ko = p.k_out[r.slice];
  r.p0 = s_prefix[p.G + 1 + grp];
  r.p_end = s_prefix[p.G + 2 + grp];
  return r;
}
// Place of an m-tile inside its group: image `ib` of the group, band `ty` of the image (bands per image: nty).
struct HaloPos { int ib, ty; };
__device__ __forceinline__ HaloPos halo_pos(int mt, int nty) {
  HaloPos q;
  q.ib = mt / nty;
  q.ty = mt - q.ib * nty;
  return q;
}
__device__ __forceinline__ void halo_advance(HaloPos& q, const HaloPos& step, int nty) {
  q.ib += step.ib;
  q.ty += step.ty;
  if (q.ty >= nty) { q.ty -= nty; ++q.ib; }
}

// What a thread of the epilogue knows about the tile at hand.
struct HaloEpi {
  uint32_t taddr;              // this thread's TMEM lane, first column of the accumulator
  int ncols, n0, ko;           // columns of this n-tile, its first column, the slice's width
  const float *brow, *sc_row, *sh_row;
  const __nv_bfloat16* res_row;
  __nv_bfloat16* yrow;         // this thread's output row (nullptr: padding position, not stored)
  const CUtensorMap* mapY;     // (channel, x, y, sample), box 64 x (W + 2) x bh x 1
  int y0, smp;                 // first image row of the tile, output sample (-1: none)
};

// One tile through the epilogue of a column group: chunks chunk0, chunk0 + chunk_step, ... of 64 columns.
// `cn` counts the chunks this group has staged (barrier phases), `pending` says that the issuing warp still has to
// hand the block back.  Returns false when the CTA is aborting.
template <int ACT, bool AFF, bool RES>
__device__ __forceinline__ bool halo_epilogue_tile(const HaloEpi& e, int chunk0, int chunk_step, int q, int lane, uint8_t* stage_g,
                                                   uint32_t bar_sw, uint32_t bar_sf, uint32_t& cn, bool& pending,
                                                   volatile uint32_t* abort_flag, int32_t* status) {
  const int m = q * 32 + lane;
  uint8_t* stage_row = stage_g + m * 128;
  for (int c0 = 64 * chunk0; c0 < e.ncols; c0 += 64 * chunk_step, ++cn) {
    if (q == 0 && pending) {  // the issuing warp: the store of the chunk before has read the block
      if (lane == 0) {
        bulk_wait_read0();
        mbar_arrive(bar_sf);
      }
      pending = false;
      __syncwarp();
    }
    if (cn > 0 && !__all_sync(0xffffffffu, mbar_wait(bar_sf, (cn - 1u) & 1u, abort_flag, status, 44))) return false;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      if (c0 + 32 * half < e.ncols) {  // warp-uniform
        uint32_t w[16];
        epilogue_half<ACT, AFF, RES>(e.taddr + c0 + 32 * half, c0 + 32 * half, e.ncols, e.brow, e.sc_row, e.sh_row, e.res_row, w);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = 4 * half + jj;
          *reinterpret_cast<uint4*>(stage_row + ((j ^ (lane & 7)) << 4)) = make_uint4(w[4 * jj], w[4 * jj + 1], w[4 * jj + 2], w[4 * jj + 3]);
        }
      }
    }
    // the store's tensor ends at the slice width rounded down to 8 columns: the 1..7 columns beyond leave here
    const int col8 = e.ncols & ~7, tail_n = e.ncols & 7;
    if (tail_n != 0 && col8 >= c0 && col8 < c0 + 64 && e.yrow) {
      const int j = (col8 - c0) >> 3;
      const uint4 val = *reinterpret_cast<const uint4*>(stage_row + ((j ^ (lane & 7)) << 4));
      const uint32_t w[4] = {val.x, val.y, val.z, val.w};
      store_row_tail(e.yrow + col8, w, tail_n);
    }
    fence_async_smem();
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_sw);
    if (q == 0) {
      if (!__all_sync(0xffffffffu, mbar_wait(bar_sw, cn & 1u, abort_flag, status, 45))) return false;
      if (lane == 0) {
        if (e.ko >= 8 && e.smp >= 0) tma_store_4d(e.mapY, e.n0 + c0, 0, e.y0, e.smp, smem_u32(stage_g));
        bulk_commit();
      }
      pending = true;
      __syncwarp();
    }
  }
  return true;
}

// kRes: the layer has skip features (residual add before the activation).  The form without them holds no
// trace of that code: its registers and code size weighed on every other epilogue variant.
// kLean (only without kRes): no bias, no per-path affine, no GELU: the epilogue holds the plain and the ReLU
// variant only.
template <bool kRes, bool kLean>
__global__ void __launch_bounds__(kThreads, 1) gemm_bf16_halo_kernel(const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const GemmGeom& g = p.g;
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);

  const uint32_t bar_full = base;
  const uint32_t bar_empty = base + 8 * kMaxStages;
  const uint32_t bar_tfull = base + 16 * kMaxStages + 48 + 16 * kMaxStages;  // [8]
  const uint32_t bar_tempty = bar_tfull + 64;                                // [8]
  // accumulators: as many n-tile-wide buffers as TMEM's 512 columns hold (2, 4 or 8).  With narrow
  // slices the main loop and the epilogue of a tile are both short, and what a tile costs is the
  // hand-over between them; more buffers keep more tiles in flight.
  const int acc_log2 = g.BN == 256 ? 1 : (g.BN == 128 ? 2 : 3);
  const int nacc = 1 << acc_log2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16 * kMaxStages + 32);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 16 * kMaxStages + 36);

  const uint32_t bar_afull = base + 16 * kMaxStages + 48;   // [kMaxStages]
  const uint32_t bar_aempty = bar_afull + 8 * kMaxStages;  // [kMaxStages]
  const uint32_t bar_stage = base + kCtrlBytes - 16 * (kEpiWarps / 4);  // per column group: swritten, sfree
  const int aslots = g.a_slots;                            // depth of the activation ring
  const int stages = g.stages;                             // depth of the weight ring
  const uint32_t bh_bytes = (uint32_t)(g.BN / 2) * BK * 2;  // this CTA's half of the weight tile of one tap
  // Narrow n-tiles put all nine taps of a chunk into ONE ring slot (one wait and one commit per 36
  // instructions: with N <= 128 an instruction is too short to hide a barrier round per tap); the
  // 16 KB boxes of 256-wide tiles keep a slot per tap.
  const int tps = g.tps;                                    // taps per ring slot: 9 or 1
  const uint32_t slot_b = (uint32_t)tps * bh_bytes;
  const uint32_t a_slot = dsn_halo_slot_bytes(g.bw, g.bh);  // one activation block with halo (+ overrun rows)
  const uint32_t a_base = base + kCtrlBytes;
  const uint32_t b_base = a_base + (uint32_t)aslots * a_slot;
  uint8_t* out_stage = smem + kCtrlBytes + (size_t)aslots * a_slot + (size_t)stages * slot_b;
  int32_t* s_prefix = reinterpret_cast<int32_t*>(out_stage + kStageOutBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const uint32_t tmem_cols = 512u;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < nacc; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, g.BN == 64 ? 2 * 4 : 2 * kEpiWarps);  // 64-wide n-tiles: one column group (four warps in each CTA) per tile
    }
    for (int a = 0; a < aslots; ++a) {
      mbar_init(bar_afull + 8 * a, 1);
      mbar_init(bar_aempty + 8 * a, 1);
    }
    for (int f = 0; f < kEpiWarps / 4; ++f) {
      mbar_init(bar_stage + 16 * f, 4);      // swritten
      mbar_init(bar_stage + 16 * f + 8, 1);  // sfree
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
  // s_prefix[0..G]: tile prefix; [G+1 .. 2G+1]: group offsets; [2G+2 .. 3G+1]: slice of each group; [3G+3 .. 4G+3]: cost prefix
  for (int j = threadIdx.x; j <= p.G; j += blockDim.x) s_prefix[p.G + 1 + j] = p.offsets[j];
  for (int j = threadIdx.x; j < p.G; j += blockDim.x) {
    const int sl = p.group_slice ? p.group_slice[j] : j;
    s_prefix[2 * p.G + 2 + j] = (sl >= 0 && sl < p.T) ? sl : 0;
  }
  dsn_build_tile_prefix(p.G, s_prefix, ntiles_of);
  // estimated time of a group's tiles, in units of 16 cycles.  Measured on this kernel: about 1000 cycles of fixed
  // work per tile in the issuing warp, and per tensor instruction N / 2 cycles but never less than about 40
  int32_t* s_cost = s_prefix + 3 * p.G + 3;
  auto tile_cost = [&](int sl) {
    const int nw = p.k_out[sl] < g.BN ? p.k_out[sl] : g.BN;
    const int n_inst = (nw + 31) & ~31;
    const int cyc = n_inst / 2 > 40 ? n_inst / 2 : 40;
    // a tile of several chunks fills the activation ring alone: part of the next tile's load is then exposed
    const int exposed = (p.k_in[sl] > BK && aslots < 4) ? 1200 : 0;
    return (9 * ((p.k_in[sl] + 15) >> 4) * cyc + 1000 + exposed) >> 4;
  };
  auto cost_of = [&](int grp) {
    const int n = ntiles_of(grp);
    return n ? n * tile_cost(p.group_slice ? p.group_slice[grp] : grp) : 0;
  };
  dsn_build_tile_prefix(p.G, s_cost, cost_of);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything can arrive on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int total = s_prefix[p.G];
  // first tile of pair k: where the running cost reaches k / npairs of the whole
  auto range_start = [&](int k) {
    if (k <= 0 || total == 0) return 0;
    if (k >= npairs) return total;
    const int32_t target = (int32_t)(((int64_t)s_cost[p.G] * k) / npairs);
    const int j = dsn_find_tile_slot(s_cost, p.G, target);
    const int n = s_prefix[j + 1] - s_prefix[j];
    return s_prefix[j] + (int)(((int64_t)(target - s_cost[j]) * n) / (s_cost[j + 1] - s_cost[j]));
  };
  // g.ranges: a contiguous range per pair; otherwise tile pair, pair + npairs, ... (every pair sees every group)
  const int tile_begin = g.ranges ? range_start(pair) : pair, tile_end = g.ranges ? range_start(pair + 1) : total;
  const int sched = g.ranges ? 1 : npairs;  // distance between two tiles of this pair

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    // The whole warp walks the schedule (addresses, coordinates and the loop itself stay
    // warp-uniform, which keeps the per-stage instruction count low); one elected lane issues.
    int stage = 0, aslot = 0;
    uint32_t phase = 0, aphase = 0;
    const uint32_t a_box_bytes = (uint32_t)(g.bw * (g.bh + 2)) * BK * 2;  // (W + 2) x (bh + 2) pixels
    int res_key = -1;  // the slice whose weights the ring holds whole (-1: none)
    bool ok = true;
    const HaloPos step = halo_pos(2 * sched, g.tiles_y);
    int tile = tile_begin;
    while (ok && tile < tile_end) {
      const HaloRun r = halo_find_run(p, s_prefix, tile);
      const int run_end = r.hi < tile_end ? r.hi : tile_end;
      const CUtensorMap* mA = &p.mapA[r.map];
      const CUtensorMap* mB = &p.mapB[r.map];
      const int nkc = (r.ki + BK - 1) / BK;
      const int n_inst = ((r.ko < g.BN ? r.ko : g.BN) + 31) & ~31;
      const int brow0 = rank * (n_inst >> 1);  // first weight row of this CTA's half (a slice is one n-tile here)
      bool reuse = r.slice == res_key;         // the weights are in the ring already
      if (!reuse) res_key = nkc * (9 / tps) <= stages ? r.slice : -1;
      const bool keep = res_key >= 0;
      // the sample a tile reads: looked up (a global load) one tile ahead
      auto sample_of = [&](const HaloPos& q) {
        const int b0 = r.p0 + q.ib;
        if (!g.a_input_order) return b0;
        return b0 < r.p_end ? __ldg(p.perm + b0) : p.B;  // past the group: out of range, zeros
      };
      HaloPos pos = halo_pos(2 * (tile - r.lo) + rank, g.tiles_y);
      int bsel = sample_of(pos);
      for (; ok && tile < run_end; tile += sched) {
        HaloPos pos_next = pos;
        halo_advance(pos_next, step, g.tiles_y);
        const int bsel_next = tile + sched < run_end ? sample_of(pos_next) : 0;
        const int y0 = pos.ty * g.bh;
        for (int kc = 0; ok && kc < nkc; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_aempty + 8 * aslot, aphase ^ 1u, abort_flag, p.status, 41));
          if (!ok) break;
          if (elect_one()) {
            const uint32_t lead = leader_addr(bar_afull + 8 * aslot);
            if (rank == 0) mbar_expect_tx(bar_afull + 8 * aslot, 2u * a_box_bytes);
            tma_load_4d_pair(a_base + aslot * a_slot, mA, kc * BK, -1, y0 - 1, bsel, lead);  // halo: starts one pixel out
          }
          if (++aslot == aslots) { aslot = 0; aphase ^= 1u; }
          for (int tap0 = 0; !reuse && tap0 < 9; tap0 += tps) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, p.status, 42));
            if (!ok) break;
            if (elect_one()) {
              const uint32_t lead = leader_addr(bar_full + 8 * stage);
              if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2u * slot_b);
              for (int u = 0; u < tps; ++u)
                tma_load_3d_pair(b_base + stage * slot_b + u * bh_bytes, mB, kc * BK, tap0 + u, brow0, lead);
            }
            if (++stage == stages) { stage = 0; phase ^= 1u; }
          }
        }
        reuse = keep;  // kept weights serve the rest of the run
        pos = pos_next;
        bsel = bsel_next;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    // Warp-uniform loop, one elected lane issues.  The issuing warp is the critical resource of a tile with
    // wide N (four instructions of 128 tensor-pipe cycles per stage), so the per-stage path is
    // kept short: running descriptors, four unrolled K steps, a separate short loop for a partial
    // last chunk.
    if (rank == 0) {
      int stage = 0, aslot = 0;
      uint32_t phase = 0, aphase = 0;
      int it = 0;
      bool ok = true;
      const uint64_t db0 = make_smem_desc(b_base);
      const uint64_t dbstep = (uint64_t)(slot_b >> 4), dbtap = (uint64_t)(bh_bytes >> 4);
      const uint64_t darow = (uint64_t)(g.bw * 8);  // one image row of the padded block, in 16-byte units
      int res_key = -1, res_stage = 0, res_n = 0;  // weights kept in the ring: their slice, first slot, slots
      int tile = tile_begin;
      while (ok && tile < tile_end) {
        const HaloRun r = halo_find_run(p, s_prefix, tile);
        const int run_end = r.hi < tile_end ? r.hi : tile_end;
        const int n_inst = ((r.ko < g.BN ? r.ko : g.BN) + 31) & ~31;
        const uint32_t idesc = make_idesc(2 * BM, n_inst);
        const int nkc = (r.ki + BK - 1) / BK;
        const int tail_ks = ((r.ki & (BK - 1)) + 15) >> 4;  // K steps of a partial last chunk (0: none)
        bool reuse = r.slice == res_key;
        if (!reuse) {
          if (res_key >= 0 && elect_one()) {  // other weights are needed: the kept slots go back to the producer
            for (int k = 0; k < res_n; ++k) {
              const int sl = res_stage + k;
              umma_commit_pair(bar_empty + 8 * (sl >= stages ? sl - stages : sl));
            }
          }
          res_n = nkc * (9 / tps);
          res_key = res_n <= stages ? r.slice : -1;
          res_stage = stage;
        }
        const bool keep = res_key >= 0;
        for (; ok && tile < run_end; tile += sched, ++it) {
          const int acc = it & (nacc - 1);
          const uint32_t acc_phase = (uint32_t)(it >> acc_log2) & 1u;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, p.status, 12));
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(acc * g.BN);
          int ws = reuse ? res_stage : stage;  // the slot read next
          uint32_t accumulate = 0;
          for (int kc = nkc; ok && kc > 0; --kc) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_afull + 8 * aslot, aphase, abort_flag, p.status, 43));
            if (!ok) break;
            const int nks = (kc == 1 && tail_ks != 0) ? tail_ks : BK / 16;
            const uint32_t a_addr = a_base + aslot * a_slot;
            const uint64_t da0 = make_smem_desc(a_addr);
            for (int tap0 = 0; tap0 < 9; tap0 += tps) {
              if (!reuse) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status, 13));
                if (!ok) break;
                tc_fence_after();
              }
              const uint64_t db = db0 + (uint64_t)ws * dbstep;
              // a tap's view of the block: same rows, start moved by whole 128-byte rows (8 descriptor units each)
              if (tps == 9) {
                if (elect_one()) {
#pragma unroll
                  for (int u = 0; u < 9; ++u) {
                    const uint64_t da = da0 + (uint64_t)(u / 3) * darow + (uint64_t)(8 * (u % 3)), dbt = db + (uint64_t)u * dbtap;
                    umma_bf16_pair(d_tmem, da, dbt, idesc, u == 0 ? accumulate : 1u);  // +32 bytes per K step
                    if (nks > 1) umma_bf16_pair(d_tmem, da + 2u, dbt + 2u, idesc, 1u);
                    if (nks > 2) umma_bf16_pair(d_tmem, da + 4u, dbt + 4u, idesc, 1u);
                    if (nks > 3) umma_bf16_pair(d_tmem, da + 6u, dbt + 6u, idesc, 1u);
                  }
                  if (!keep) umma_commit_pair(bar_empty + 8 * stage);
                }
              } else {
                const int tr = tap0 / 3, sx = tap0 - 3 * tr;
                const uint64_t da = da0 + (uint64_t)tr * darow + (uint64_t)(8 * sx);
                if (elect_one()) {
                  umma_bf16_pair(d_tmem, da, db, idesc, accumulate);
                  if (nks > 1) umma_bf16_pair(d_tmem, da + 2u, db + 2u, idesc, 1u);
                  if (nks > 2) umma_bf16_pair(d_tmem, da + 4u, db + 4u, idesc, 1u);
                  if (nks > 3) umma_bf16_pair(d_tmem, da + 6u, db + 6u, idesc, 1u);
                  if (!keep) umma_commit_pair(bar_empty + 8 * stage);
                }
              }
              accumulate = 1;
              if (++ws == stages) ws = 0;
              if (!reuse && ++stage == stages) { stage = 0; phase ^= 1u; }
            }
            if (ok && elect_one()) umma_commit_pair(bar_aempty + 8 * aslot);  // all nine taps have read the block
            if (++aslot == aslots) { aslot = 0; aphase ^= 1u; }
          }
          if (ok && elect_one()) umma_commit_pair(bar_tfull + 8 * acc);
          reuse = keep;  // kept weights serve the rest of the run
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;
    const int first = (warp - 2) >> 2;
    const int m = q * 32 + lane;
    uint8_t* stage_g = out_stage + first * (4 * 32 * 128);  // this column group's block: 128 rows of 128 bytes
    const uint32_t bar_sw = bar_stage + 16 * first, bar_sf = bar_sw + 8;
    uint32_t cn = 0;
    bool pending = false;
    bool ok = true;
    // this thread's place in the tile (rows run over the padded width) does not change from tile to tile
    const int row_j = m / g.bw, row_x = m - row_j * g.bw;
    // 64-wide n-tiles are a single chunk: the two column groups take every other tile instead of every other chunk
    const bool alternate = g.BN == 64;
    const int chunk0 = alternate ? 0 : first, chunk_step = alternate ? 1 : kEpiWarps / 4;
    const int it_step = alternate ? kEpiWarps / 4 : 1, tile_step = it_step * sched;
    const HaloPos step = halo_pos(2 * tile_step, g.tiles_y);
    int tile = tile_begin + (alternate ? first * sched : 0), it = alternate ? first : 0;
    while (ok && tile < tile_end) {
      const HaloRun r = halo_find_run(p, s_prefix, tile);
      const int run_end = r.hi < tile_end ? r.hi : tile_end;
      HaloEpi e;
      e.ncols = r.ko < g.BN ? r.ko : g.BN;  // a slice is one n-tile here
      e.n0 = 0;
      e.ko = r.ko;
      e.brow = p.bias;
      e.sc_row = p.bn_scale ? p.bn_scale + (int64_t)r.slice * p.bn_ld : nullptr;
      e.sh_row = p.bn_scale ? p.bn_shift + (int64_t)r.slice * p.bn_ld : nullptr;
      e.mapY = &p.mapY[r.map];
      // the sample a tile writes: looked up (a global load) one tile ahead
      auto sample_of = [&](const HaloPos& q) {
        const int b0 = r.p0 + q.ib;
        if (b0 >= r.p_end) return -1;
        return g.y_input_order ? __ldg(p.perm + b0) : b0;
      };
      HaloPos pos = halo_pos(2 * (tile - r.lo) + rank, g.tiles_y);
      int smp = sample_of(pos);
      for (; ok && tile < run_end; tile += tile_step, it += it_step) {
        HaloPos pos_next = pos;
        halo_advance(pos_next, step, g.tiles_y);
        const int smp_next = tile + tile_step < run_end ? sample_of(pos_next) : -1;
        const int acc = it & (nacc - 1);
        const uint32_t acc_phase = (uint32_t)(it >> acc_log2) & 1u;
        e.y0 = pos.ty * g.bh;
        e.smp = smp;
        const int yy = e.y0 + row_j;
        const bool valid = smp >= 0 && row_j < g.bh && yy < g.H && row_x < g.W;
        const int64_t out_row = valid ? (int64_t)smp * g.R + yy * g.W + row_x : 0;
        e.res_row = (kRes && valid) ? p.residual + out_row * p.ldy : nullptr;
        e.yrow = valid ? p.y + out_row * p.ldy : nullptr;

        ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, p.status, 14));
        if (!ok) break;
        tc_fence_after();
        e.taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * g.BN);
#define DSN_HALO_EPI(ACT, AFF, RES) \
  ok = halo_epilogue_tile<ACT, AFF, RES>(e, chunk0, chunk_step, q, lane, stage_g, bar_sw, bar_sf, cn, pending, abort_flag, p.status)
        if constexpr (kRes) {
          switch (p.act) {
            case DSN_ACT_NONE: DSN_HALO_EPI(DSN_ACT_NONE, true, true); break;
            case DSN_ACT_RELU: DSN_HALO_EPI(DSN_ACT_RELU, true, true); break;
            default: DSN_HALO_EPI(DSN_ACT_GELU, true, true); break;
          }
        } else {
          const int variant = p.act * 2 + ((e.brow || e.sc_row) ? 1 : 0);
          switch (variant) {
            case 0: DSN_HALO_EPI(DSN_ACT_NONE, false, false); break;
            case 1: if constexpr (!kLean) DSN_HALO_EPI(DSN_ACT_NONE, true, false); break;
            case 2: DSN_HALO_EPI(DSN_ACT_RELU, false, false); break;
            case 3: if constexpr (!kLean) DSN_HALO_EPI(DSN_ACT_RELU, true, false); break;
            case 4: if constexpr (!kLean) DSN_HALO_EPI(DSN_ACT_GELU, false, false); break;
            default: if constexpr (!kLean) DSN_HALO_EPI(DSN_ACT_GELU, true, false); break;
          }
        }
#undef DSN_HALO_EPI
        if (!ok) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_addr(bar_tempty + 8 * acc));  // the even CTA's MMA thread waits on it
        pos = pos_next;
        smp = smp_next;
      }
    }
    if (q == 0 && lane == 0) bulk_wait0();  // the lane that issued this group's TMA stores
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

size_t dsn_gemm_halo_smem_bytes(int BN, int stages, int tps, int a_slots, int G, int wp, int bh) {
  return 1024 + kCtrlBytes + (size_t)a_slots * dsn_halo_slot_bytes(wp, bh) + (size_t)stages * tps * ((size_t)(BN / 2) * BK * 2) +
         kStageOutBytes + sizeof(int32_t) * (4 * (size_t)G + 4);
}

cudaError_t dsn_launch_gemm_bf16_halo(const GemmParams& p, int clusters, size_t smem_bytes, cudaStream_t s) {
  static size_t configured[3][DSN_MAX_DEVICES] = {};
  const bool lean = !p.residual && !p.bias && !p.bn_scale && p.act != DSN_ACT_GELU;
  const int form = p.residual ? 2 : (lean ? 1 : 0);
  void (*kernel)(GemmParams) = form == 2 ? gemm_bf16_halo_kernel<true, false>
                               : form == 1 ? gemm_bf16_halo_kernel<false, true> : gemm_bf16_halo_kernel<false, false>;
  {
    cudaError_t e = dsn_ensure_dynamic_smem(kernel, smem_bytes, configured[form]);
    if (e != cudaSuccess) return e;
  }
  return dsn_launch(kernel, dim3(2 * clusters), dim3(kThreads), smem_bytes, s, 2, p);
}
