// A chain of sliced layers (e.g. the bottleneck 1x1 -> 3x3 -> 1x1) in ONE launch on CTA pairs.
//
// Small batches leave every layer of the chain with one or two tiles per CTA pair; run as separate
// launches, each layer then pays its own set-up, its own ramp and its own tail.  Here a pair owns
// whole samples: for a sample it runs the tiles of layer 0, then of layer 1, ... with the
// intermediates in global memory (they stay in L2) in grouped order.  Nothing else has to wait: the
// only dependency is per sample (a 3x3 tile needs every pixel of the sample from the layer before),
// and it is tracked inside the pair.  Two samples are interleaved so that the epilogue of one
// overlaps the main loop of the other:
//
//     A.L0  B.L0  A.L1  B.L1  A.L2 ...  B.L2 ...       (A, B: the pair's two samples of this round)
//
// Per-sample semantics make this legal (Eq. dyn_net, Sec. 3.1: every input runs the sub-network its
// own gate picks; one gate decision holds for all layers of a block, Sec. 5).
//
// Roles, barriers and the tile kernels' contracts are those of the pair GEMM (dsn_gemm_bf16_2cta.cu):
// TMA producer warp and epilogue warps in both CTAs, MMA issue in the even CTA, 2 accumulators in
// TMEM.  Added here: done[slot], a counter in each CTA's shared memory that the epilogue warps of
// BOTH CTAs bump (release, cluster scope) once the stores of a tile of a non-final layer are
// complete; the producers read it (acquire) before the first load of the sample's next layer.
// All waits are bounded.
//
// Last layer fed from tensor memory (kFuse forms).  When the last layer is a 1x1 / linear layer whose input is the
// whole output tile of the layer before (one pair tile per sample, at most 256 channels), that output never leaves
// the SM: the epilogue of the layer before converts its accumulator rows to bf16 (bias, affine, activation as
// usual) and writes them, two values per 32-bit column, over the first columns of the SAME accumulator region
// (tcgen05.st; a thread only overwrites columns it has read), and the last layer's products take their A operand
// from there (tcgen05.mma with A in tensor memory), so only its weights are loaded.  Its own accumulators are 128
// columns wide and live in the upper halves of the two regions, which the epilogue of the layer before has read
// by then.  ares[slot]: the 2 x 4 converting warps -> the issuing warp, the sample's rows are in place.
#include "dsn_gemm_pair_device.cuh"

namespace {

using namespace dsn_gemm;

struct ChainTile {
  int map, ki, ko, n0, slice;
  int p_end, b0, x0, y0;
};

__device__ __forceinline__ uint32_t ld_acquire_cluster(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.acquire.cluster.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
// +1 on the counter at this shared-window address (own CTA or the partner), release at cluster scope
__device__ __forceinline__ void red_release_cluster_add(uint32_t cluster_addr) {
  asm volatile("red.release.cluster.shared::cluster.add.u32 [%0], %1;" ::"r"(cluster_addr), "r"(1u) : "memory");
}
__device__ __forceinline__ uint32_t cta_addr_in_cluster(uint32_t local_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(cta_rank));
  return r;
}
// orders accesses to global memory through the generic proxy (plain loads / stores) and through the async proxy (TMA)
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem]^T over the pair: every CTA supplies its 128 rows of A from its own tensor memory
__device__ __forceinline__ void umma_bf16_pair_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                      uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// One warp converts its 32 accumulator rows of a whole tile (n_inst columns at `taddr`) and writes them back as
// packed bf16 pairs over columns 0 .. n_inst / 2 - 1 of the same region: block c (32 columns) is read before the 16
// columns at 16 c are written, which lie inside blocks this warp has already read.
template <int ACT, bool AFF, bool RES>
__device__ __forceinline__ void convert_tile_in_tmem(uint32_t taddr, int n_inst, int ko, const float* brow,
                                                     const float* sc_row, const float* sh_row,
                                                     const __nv_bfloat16* res_row) {
  for (int c0 = 0; c0 < n_inst; c0 += 32) {
    uint32_t w[16];
    epilogue_half<ACT, AFF, RES>(taddr + c0, c0, ko, brow, sc_row, sh_row, res_row, w);
    tmem_st_32x16(taddr + (c0 >> 1), w);
  }
  tmem_st_wait();
}

// Bounded wait until the counter reaches `target`.
static __device__ __noinline__ bool wait_counter(uint32_t addr, uint32_t target, volatile uint32_t* abort_flag,
                                                 int32_t* status, int where) {
  const uint64_t t0 = globaltimer_ns();
  const uint64_t limit = wait_limit_ns(status);
  uint32_t spins = 0;
  while ((int32_t)(ld_acquire_cluster(addr) - target) < 0) {
    if ((++spins & 31u) == 0) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit) {
        *abort_flag = 1;
        dsn_set_status(status, DSN_ERR_TIMEOUT, where);
        return false;
      }
    }
  }
  return true;
}

// group of grouped position `pos` (pos < offsets[G]): the last group whose first position is <= pos
// and that is not empty
__device__ __forceinline__ int group_of(const int32_t* s_off, int G, int pos) {
  int lo = 0, hi = G;  // s_off[lo] <= pos < s_off[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_off[mid] <= pos) lo = mid; else hi = mid;
  }
  return lo;
}

// Walks the pair's task list in execution order; every role calls it with its own body.
// body(layer, slot, tile, it, first_of_layer, tiles_before) -> false to stop.
template <typename F>
__device__ __forceinline__ void chain_walk(const DsnChainParams& cp, const int32_t* s_off, int pair, int npairs,
                                           int rank, F&& body) {
  const int G = cp.L[0].G;
  const int n_valid = s_off[G];
  int it = 0;
  // Samples are handed out widest path first, in rounds of 2 * npairs: the pair takes rank
  // `pair` of the round and, from the other end, rank 2 * npairs - 1 - pair (a wide sample is
  // teamed with a narrow one).
  for (int c = 0; c + pair < n_valid; c += 2 * npairs) {
    const int rank_of_slot[2] = {c + pair, c + 2 * npairs - 1 - pair};
    const int nslots = (rank_of_slot[1] < n_valid) ? 2 : 1;
    for (int l = 0; l < cp.n_layers; ++l) {
      const GemmParams& P = cp.L[l];
      const GemmGeom& g = P.g;
      const int per_img = g.tiles_x * g.tiles_y;
      const int mpairs = (per_img + 1) >> 1;
      for (int slot = 0; slot < nslots; ++slot) {
        const int pos = n_valid - 1 - rank_of_slot[slot];
        const int sl = group_of(s_off, G, pos);  // groups made by dsn_route: group index = path index
        ChainTile t;
        t.slice = sl;
        t.map = P.map_id[sl];
        t.ki = P.k_in[sl];
        t.ko = P.k_out[sl];
        t.p_end = pos + 1;
        const int ntn = (t.ko + g.BN - 1) / g.BN;
        const int ntiles = mpairs * ntn;
        for (int local = 0; local < ntiles; ++local, ++it) {
          const int nt = local % ntn, mt = 2 * (local / ntn) + rank;
          t.n0 = nt * g.BN;
          if (mt < per_img) {
            const int ty = mt / g.tiles_x, tx = mt - ty * g.tiles_x;
            t.b0 = pos;
            t.y0 = ty * g.bh;
            t.x0 = tx * g.bw;
          } else {  // the odd m-tile past the sample's last one: no valid rows
            t.b0 = pos + 1;
            t.y0 = t.x0 = 0;
          }
          if (!body(l, slot, t, it, local == 0, ntiles)) return;
        }
      }
    }
  }
}

// kAff: some layer of the block has a bias or a per-path affine; kGelu: some layer ends in GELU.  A form
// without one of them holds none of that code: the kernel is sensitive to its own size (each of the two cuts
// took about 1 us off the bottleneck step).
template <bool kAff, bool kGelu, bool kRes = false, bool kFuse = false>
__global__ void __launch_bounds__(kThreads, 1) gemm_bf16_chain_kernel(const __grid_constant__ DsnChainParams cp) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);

  const uint32_t bar_full = base;
  const uint32_t bar_empty = base + 8 * kMaxStages;
  const uint32_t bar_tfull = base + 16 * kMaxStages;
  const uint32_t bar_tempty = bar_tfull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 16 * kMaxStages + 32);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + 16 * kMaxStages + 36);
  uint32_t* done_cnt = reinterpret_cast<uint32_t*>(smem + 16 * kMaxStages + 40);  // [2]
  const uint32_t done_addr = base + 16 * kMaxStages + 40;
  const uint32_t bar_ares = base + 16 * kMaxStages + 48;  // [2]
  const int fuse_from = kFuse ? cp.n_layers - 2 : -2;     // the layer whose output stays in tensor memory

  const int stages = cp.stages;
  const uint32_t bh_bytes = (uint32_t)(cp.bn_max / 2) * BK * 2;  // this CTA's half of the widest weight tile
  const uint32_t stage_bytes = kABytes + bh_bytes;
  const uint32_t tiles_base = base + kCtrlBytes;
  uint8_t* out_stage = smem + kCtrlBytes + (size_t)stages * stage_bytes;
  int32_t* s_off = reinterpret_cast<int32_t*>(out_stage + kStageOutBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const uint32_t tmem_cols = 2u * (uint32_t)cp.bn_max;
  int32_t* status = cp.L[0].status;
  const int G = cp.L[0].G;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 2 * kEpiWarps);
      mbar_init(bar_ares + 8 * a, 2 * 4);  // one converting warp per lane quarter in each CTA
    }
    *abort_flag = 0;
    done_cnt[0] = done_cnt[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish_pair();
  }
  // barriers and TMEM are set up; everything below reads what earlier kernels wrote
  dsn_grid_dependency_wait();
  dsn_grid_launch_dependents();
  for (int j = threadIdx.x; j <= G; j += blockDim.x) s_off[j] = cp.L[0].offsets[j];
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the partner's barriers and counters are initialised before anything can arrive on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    int stage = 0;
    uint32_t phase = 0;
    uint32_t target[2] = {0u, 0u};  // epilogue-warp arrivals after which the slot's next layer may load
    bool ok = true;
    chain_walk(cp, s_off, pair, npairs, rank,
               [&](int l, int slot, const ChainTile& t, int, bool first_of_layer, int ntiles) {
      const GemmParams& P = cp.L[l];
      const GemmGeom& g = P.g;
      const bool a_in_tmem = kFuse && l == fuse_from + 1;  // this layer's activations are not loaded
      if (first_of_layer) {
        if (l > 0 && !a_in_tmem) {
          // every tile of the layer before, of this sample, has been stored by both CTAs
          ok = __all_sync(0xffffffffu, wait_counter(done_addr + 4 * slot, target[slot], abort_flag, status, 31));
          if (!ok) return false;
          fence_proxy_async_all();  // the loads below read through the async proxy
        }
        if (l + 1 < cp.n_layers && l != fuse_from) target[slot] += 2u * kEpiWarps * (uint32_t)ntiles;
      }
      const CUtensorMap* mA = &P.mapA[t.map];
      const CUtensorMap* mB = &P.mapB[t.map];
      const uint32_t a_box_bytes = a_in_tmem ? 0u : (uint32_t)(g.bw * g.bh) * BK * 2;
      const uint32_t tx_bytes = 2u * (a_box_bytes + (uint32_t)(g.BN / 2) * BK * 2);
      const int nkc = (t.ki + BK - 1) / BK;
      int ncols = t.ko - t.n0;
      ncols = ncols > g.BN ? g.BN : ncols;
      const int n_inst = (ncols + 31) & ~31;
      const int brow0 = t.n0 + rank * (n_inst >> 1);
      int bsel = P.B;  // past the sample: out of range, zeros
      if (t.b0 < t.p_end) bsel = g.a_input_order ? P.perm[t.b0] : t.b0;
      for (int tap = 0; tap < g.taps; ++tap) {
        const int r = tap / g.KW, sx = tap - r * g.KW;
        const int cx = t.x0 + sx - g.pad, cy = t.y0 + r - g.pad;
        for (int kc = 0; kc < nkc; ++kc) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1u, abort_flag, status, 32));
          if (!ok) return false;
          if (elect_one()) {
            const uint32_t full_lead = leader_addr(bar_full + 8 * stage);
            if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, tx_bytes);
            const uint32_t sa = tiles_base + stage * stage_bytes;
            if (!a_in_tmem) tma_load_4d_pair(sa, mA, kc * BK, cx, cy, bsel, full_lead);
            tma_load_3d_pair(sa + kABytes, mB, kc * BK, tap, brow0, full_lead);
          }
          if (++stage == stages) { stage = 0; phase ^= 1u; }
        }
      }
      return true;
    });
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    if (rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t da0 = make_smem_desc(tiles_base), db0 = make_smem_desc(tiles_base + kABytes);
      const uint64_t dstep = (uint64_t)(stage_bytes >> 4);
      uint64_t da = da0, db = db0;
      uint32_t ares_t0 = 0u, ares_t1 = 0u;   // where the rows of the sample of slot 0 / 1 sit in tensor memory
      uint32_t ares_ph0 = 0u, ares_ph1 = 0u;
      chain_walk(cp, s_off, pair, npairs, 0, [&](int l, int slot, const ChainTile& t, int it, bool first_of_layer, int) {
        const GemmGeom& g = cp.L[l].g;
        const int acc = it & 1;
        const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
        const bool a_in_tmem = kFuse && l == fuse_from + 1;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1u, abort_flag, status, 33));
        if (!ok) return false;
        if (kFuse && l == fuse_from) {
          if (slot) ares_t1 = tmem_base + (uint32_t)(acc * cp.bn_max); else ares_t0 = tmem_base + (uint32_t)(acc * cp.bn_max);
        }
        if (a_in_tmem && first_of_layer) {  // the converted rows of the layer before are in place in both CTAs
          ok = __all_sync(0xffffffffu, mbar_wait(bar_ares + 8 * slot, slot ? ares_ph1 : ares_ph0, abort_flag, status, 36));
          if (!ok) return false;
          if (slot) ares_ph1 ^= 1u; else ares_ph0 ^= 1u;
        }
        tc_fence_after();
        int ncols = t.ko - t.n0;
        ncols = ncols > g.BN ? g.BN : ncols;
        const int n_inst = (ncols + 31) & ~31;
        const uint32_t idesc = make_idesc(2 * BM, n_inst);
        // accumulators of a layer fed from tensor memory: the upper half of the region (the lower holds a sample's rows)
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * cp.bn_max) + (a_in_tmem ? (uint32_t)(cp.bn_max >> 1) : 0u);
        const int nkc = (t.ki + BK - 1) / BK;
        const int tail_ks = ((t.ki & (BK - 1)) + 15) >> 4;
        uint32_t accumulate = 0;
        for (int tap = 0; tap < g.taps; ++tap) {
          for (int kc = nkc; kc > 0; --kc) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * stage, phase, abort_flag, status, 34));
            if (!ok) return false;
            tc_fence_after();
            const int nks = (kc == 1 && tail_ks != 0) ? tail_ks : BK / 16;
            if (a_in_tmem) {
              if (elect_one()) {
                const uint32_t a0 = (slot ? ares_t1 : ares_t0) + (uint32_t)(32 * (nkc - kc));  // 64 bf16 = 32 columns per chunk
                umma_bf16_pair_a_tmem(d_tmem, a0, db, idesc, accumulate);
                if (nks > 1) umma_bf16_pair_a_tmem(d_tmem, a0 + 8u, db + 2u, idesc, 1u);
                if (nks > 2) umma_bf16_pair_a_tmem(d_tmem, a0 + 16u, db + 4u, idesc, 1u);
                if (nks > 3) umma_bf16_pair_a_tmem(d_tmem, a0 + 24u, db + 6u, idesc, 1u);
                umma_commit_pair(bar_empty + 8 * stage);
              }
            } else if (elect_one()) {
              umma_bf16_pair(d_tmem, da, db, idesc, accumulate);
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
        if (elect_one()) umma_commit_pair(bar_tfull + 8 * acc);
        return true;
      });
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    const int q = warp & 3;
    const int first = (warp - 2) >> 2;
    const int m = q * 32 + lane;
    bool ok = true;
    int pending_slot = -1;  // slot whose counter still has to hear about this warp's last tile
    uint8_t* stage_w = out_stage + (warp - 2) * (32 * 128);
    const uint32_t done_mine = cta_addr_in_cluster(done_addr, (uint32_t)rank);
    const uint32_t done_peer = cta_addr_in_cluster(done_addr, (uint32_t)(rank ^ 1));
    // The sample's next layer reads the rows a tile of a non-final layer wrote: its TMA stores must be
    // complete and its plain stores ordered before reads of the async proxy; then one arrival on the
    // slot's counter in both CTAs.  Completion takes a few microseconds, so the warp does not wait for
    // it after the tile: it releases the accumulator, and signals when it comes back for its next tile
    // (where it would wait for the main loop anyway) or leaves.
    auto signal_pending = [&]() {
      if (pending_slot < 0) return;
      if (elect_one()) bulk_wait0();   // this warp's TMA stores have been written
      fence_proxy_async_all();         // plain stores of the ragged path, ordered before reads of the async proxy
      __syncwarp();                    // ... and before lane 0's release below
      if (lane == 0) {
        red_release_cluster_add(done_mine + 4 * pending_slot);
        red_release_cluster_add(done_peer + 4 * pending_slot);
      }
      pending_slot = -1;
    };
    chain_walk(cp, s_off, pair, npairs, rank, [&](int l, int slot, const ChainTile& t, int it, bool, int) {
      const GemmParams& P = cp.L[l];
      const GemmGeom& g = P.g;
      const int acc = it & 1;
      const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
      signal_pending();
      const int box_rows = g.bw * g.bh;
      const int yy = t.y0 + m / g.bw, xx = t.x0 + m % g.bw;
      const int pp = t.b0;
      const bool valid = m < box_rows && yy < g.H && xx < g.W && pp < t.p_end;
      int64_t out_row = 0;
      if (valid) {
        const int smp = g.y_input_order ? P.perm[pp] : pp;
        out_row = (int64_t)smp * g.R + yy * g.W + xx;
      }
      __nv_bfloat16* yrow = valid ? P.y + out_row * P.ldy + t.n0 : nullptr;
      const float* brow = (kAff && P.bias) ? P.bias + t.n0 : nullptr;
      const float* sc_row = (kAff && P.bn_scale) ? P.bn_scale + (int64_t)t.slice * P.bn_ld + t.n0 : nullptr;
      const float* sh_row = (kAff && P.bn_scale) ? P.bn_shift + (int64_t)t.slice * P.bn_ld + t.n0 : nullptr;
      // skip features (only the forms compiled for them carry the code): laid out like the layer's own output
      const __nv_bfloat16* res_row = (kRes && P.residual && valid) ? P.residual + out_row * P.ldy + t.n0 : nullptr;
      int ncols = t.ko - t.n0;
      ncols = ncols > g.BN ? g.BN : ncols;
      const long long base_row = __shfl_sync(0xffffffffu, (long long)out_row, 0);
      // TMA stores only where nobody waits for them: their completion (needed before the sample's next
      // layer may read the rows) takes several microseconds, plain stores followed by a release do not
      const bool contig = l + 1 == cp.n_layers && __all_sync(0xffffffffu, valid && out_row == base_row + lane) && t.ko >= 8;
      const bool any_valid = __any_sync(0xffffffffu, valid);

      ok = __all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, abort_flag, status, 35));
      if (!ok) return false;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * cp.bn_max) +
                             ((kFuse && l == fuse_from + 1) ? (uint32_t)(cp.bn_max >> 1) : 0u);
      const CUtensorMap* mY = &P.mapY[t.map];
      int variant = any_valid ? P.act * 2 + ((brow || sc_row) ? 1 : 0) : -1;
      if (kRes && any_valid && P.residual) variant = 6 + P.act;
      if (kFuse && l == fuse_from) {
        // The rows stay on the SM as the next layer's A operand: the first warp of each lane quarter converts the whole
        // tile in place (nothing is stored to global memory), then tells the issuing warp.
        if (first == 0) {
          const int n_inst = (ncols + 31) & ~31;
          switch (variant) {
            case 0: convert_tile_in_tmem<DSN_ACT_NONE, false, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 1: if constexpr (kAff) convert_tile_in_tmem<DSN_ACT_NONE, true, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 2: convert_tile_in_tmem<DSN_ACT_RELU, false, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 3: if constexpr (kAff) convert_tile_in_tmem<DSN_ACT_RELU, true, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 4: if constexpr (kGelu) convert_tile_in_tmem<DSN_ACT_GELU, false, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 5: if constexpr (kAff && kGelu) convert_tile_in_tmem<DSN_ACT_GELU, true, false>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 6: if constexpr (kRes) convert_tile_in_tmem<DSN_ACT_NONE, true, true>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 7: if constexpr (kRes) convert_tile_in_tmem<DSN_ACT_RELU, true, true>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            case 8: if constexpr (kRes && kGelu) convert_tile_in_tmem<DSN_ACT_GELU, true, true>(taddr, n_inst, ncols, brow, sc_row, sh_row, res_row); break;
            default: break;  // none of this warp's rows belongs to the sample: its rows of the operand are never used
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(leader_addr(bar_ares + 8 * slot));
        }
      } else
      switch (variant) {
        case -1: break;  // none of this warp's 32 rows belongs to the sample
        case 0: epilogue_tile<DSN_ACT_NONE, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 1: if constexpr (kAff) epilogue_tile<DSN_ACT_NONE, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 2: epilogue_tile<DSN_ACT_RELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 3: if constexpr (kAff) epilogue_tile<DSN_ACT_RELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 4: if constexpr (kGelu) epilogue_tile<DSN_ACT_GELU, false>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 5: if constexpr (kAff && kGelu) epilogue_tile<DSN_ACT_GELU, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 6: if constexpr (kRes) epilogue_tile<DSN_ACT_NONE, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 7: if constexpr (kRes) epilogue_tile<DSN_ACT_RELU, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        case 8: if constexpr (kRes && kGelu) epilogue_tile<DSN_ACT_GELU, true, true>(taddr, ncols, t.n0, first, brow, sc_row, sh_row, res_row, stage_w, yrow, lane, contig, mY, (int)base_row); break;
        default: break;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_addr(bar_tempty + 8 * acc));  // the accumulator is free again
      if (l + 1 < cp.n_layers && l != fuse_from) pending_slot = slot;
      return true;
    });
    signal_pending();
    if (elect_one()) bulk_wait0();
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

size_t dsn_gemm_chain_smem_bytes(int bn_max, int stages, int G) {
  return 1024 + kCtrlBytes + (size_t)stages * (kABytes + (size_t)(bn_max / 2) * BK * 2) + kStageOutBytes +
         sizeof(int32_t) * ((size_t)G + 1);
}

cudaError_t dsn_launch_gemm_bf16_chain(const DsnChainParams& cp, int clusters, size_t smem_bytes, cudaStream_t s) {
  static size_t configured[12][DSN_MAX_DEVICES] = {};
  int aff = 0, gelu = 0, res = 0;
  for (int l = 0; l < cp.n_layers; ++l) {
    aff |= (cp.L[l].bias || cp.L[l].bn_scale) ? 1 : 0;
    gelu |= cp.L[l].act == DSN_ACT_GELU ? 1 : 0;
    res |= cp.L[l].residual ? 1 : 0;
  }
  // a block with skip features (the residual tail of a DS-ResNet block, Sec. 5) takes the forms that carry that code;
  // fuse_tail: the forms whose last layer reads its activations from tensor memory
  void (*kernel)(DsnChainParams);
  if (cp.fuse_tail) {
    kernel = res ? (gelu ? gemm_bf16_chain_kernel<true, true, true, true> : gemm_bf16_chain_kernel<true, false, true, true>)
             : aff ? (gelu ? gemm_bf16_chain_kernel<true, true, false, true> : gemm_bf16_chain_kernel<true, false, false, true>)
                   : (gelu ? gemm_bf16_chain_kernel<false, true, false, true> : gemm_bf16_chain_kernel<false, false, false, true>);
  } else {
    kernel = res ? (gelu ? gemm_bf16_chain_kernel<true, true, true> : gemm_bf16_chain_kernel<true, false, true>)
             : aff ? (gelu ? gemm_bf16_chain_kernel<true, true> : gemm_bf16_chain_kernel<true, false>)
                   : (gelu ? gemm_bf16_chain_kernel<false, true> : gemm_bf16_chain_kernel<false, false>);
  }
  const int form = (res ? 4 + gelu : 2 * aff + gelu) + (cp.fuse_tail ? 6 : 0);
  {
    cudaError_t e = dsn_ensure_dynamic_smem(kernel, smem_bytes, configured[form]);
    if (e != cudaSuccess) return e;
  }
  return dsn_launch(kernel, dim3(2 * clusters), dim3(kThreads), smem_bytes, s, 2, cp);
}
