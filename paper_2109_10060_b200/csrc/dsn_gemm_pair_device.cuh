// PTX wrappers for kernels that run as CTA pairs (clusters of two CTAs, tcgen05 cta_group::2):
// cluster addressing and barriers, pair TMA loads (no multicast: every CTA fetches its own bytes),
// pair MMA and commit.  Included by the pair GEMM kernels only.
#pragma once
#include "dsn_gemm_device.cuh"
#include "dsn_tiles.cuh"

namespace dsn_gemm {

// shared-window address of the same location in the pair's even CTA (cluster rank 0)
__device__ __forceinline__ uint32_t leader_addr(uint32_t local_addr) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(0));
  return r;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2,
                                                 uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one arrival on the barrier at this offset in BOTH CTAs once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask)
               : "memory");
}

struct PairTile {
  int map, ki, ko, n0, ncols, slice;   // the tile's columns: n0 .. n0 + ncols - 1 of the slice
  int p_end;
  int row0, rows_end;
  int b0, x0, y0;
};

// What a role remembers between two tiles: tiles come in increasing order, so the group found for one
// tile usually still holds for the next and its data need not be looked up again.
struct PairCursor {
  int lo = 0, hi = 0;   // tiles [lo, hi) belong to the cached group (hi = 0: nothing cached)
  int slice, map, ki, ko, p0, p_end, ntn;
  int nq, nr;           // n-tile widths in units of 64 columns: the first nr n-tiles hold nq + 1 units, the others nq
};

// Tile `tile` of the pair schedule as seen by CTA `rank`: the pair owns m-tiles 2*mtp and 2*mtp+1 of
// one (group, n-tile); an m-tile past the group's last one yields only invalid rows.
__device__ __forceinline__ PairTile decode_pair_tile(const GemmParams& p, const int32_t* s_prefix, int tile, int rank,
                                                     PairCursor& c) {
  PairTile t;
  const GemmGeom& g = p.g;
  if (tile >= c.hi) {
    const int j = dsn_find_tile_slot(s_prefix, p.G, tile);
    const int grp = p.G - 1 - j;
    c.lo = s_prefix[j];
    c.hi = s_prefix[j + 1];
    c.slice = s_prefix[2 * p.G + 2 + grp];  // group -> slice, cached in shared memory
    c.map = p.map_id[c.slice];
    c.ki = p.k_in[c.slice];
    c.ko = p.k_out[c.slice];
    c.p0 = s_prefix[p.G + 1 + grp];         // group offsets, cached in shared memory
    c.p_end = s_prefix[p.G + 2 + grp];
    c.ntn = (c.ko + g.BN - 1) / g.BN;
    // The slice's columns are dealt out evenly over its n-tiles in units of 64, the epilogue's store width (256 + 64
    // columns would otherwise end in a tile whose tensor instructions run at the 59-cycle floor and that loads
    // its activations all the same); only a slice's last tile can end inside a unit, where the store's map clips
    const int units = (c.ko + 63) >> 6;
    c.nq = units / c.ntn;
    c.nr = units - c.nq * c.ntn;
  }
  t.slice = c.slice;
  t.map = c.map;
  t.ki = c.ki;
  t.ko = c.ko;
  t.p_end = c.p_end;
  const int local = tile - c.lo;
  int nt = 0, mtp = local;
  if (c.ntn > 1) {
    mtp = local / c.ntn;
    nt = local - mtp * c.ntn;
  }
  const int mt = 2 * mtp + rank;
  t.n0 = 64 * (nt * c.nq + (nt < c.nr ? nt : c.nr));
  t.ncols = 64 * (c.nq + (nt < c.nr ? 1 : 0));
  if (t.ncols > t.ko - t.n0) t.ncols = t.ko - t.n0;
  if (g.flat) {
    t.row0 = c.p0 * g.R + mt * BM;
    t.rows_end = c.p_end * g.R;
    t.b0 = t.x0 = t.y0 = 0;
  } else {
    const int per_img = g.tiles_x * g.tiles_y;
    int ib = 0, rem = mt;
    if (mt >= per_img) {
      ib = mt / per_img;
      rem = mt - ib * per_img;
    }
    int ty = rem, tx = 0;
    if (g.tiles_x > 1) {
      ty = rem / g.tiles_x;
      tx = rem - ty * g.tiles_x;
    }
    t.b0 = c.p0 + ib * g.nb;
    t.y0 = ty * g.bh;
    t.x0 = tx * g.bw;
    t.row0 = t.rows_end = 0;
  }
  return t;
}

}  // namespace dsn_gemm
