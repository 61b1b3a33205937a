// C ABI of libdsn: context, argument validation, tensor-map construction, kernel selection and
// the chained dsn_layer_forward.  Every compute step runs in this library's own CUDA kernels;
// there is no host or library fallback.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "dsn_internal.cuh"

int dsn_pdl_enabled() {
  static int enabled = -1;
  if (enabled < 0) {
    const char* e = getenv("DSN_PDL");
    enabled = (e && e[0] == '0') ? 0 : 1;
  }
  return enabled;
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Every entry point runs on the context's device: launches, attribute settings and symbol look-ups all act
// on the calling thread's current device.
int check_ctx(const dsn_ctx* ctx) {
  if (!ctx) return DSN_ERR_INVALID_ARG;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return DSN_ERR_CUDA;
  return cur == ctx->device ? DSN_OK : DSN_ERR_INVALID_ARG;
}

// Launch counters and the optional call log (DSN_LOG=1: one line per launch family on stderr).
void count_launch(dsn_ctx* ctx, uint64_t dsn_stats::*field, uint64_t n = 1) {
  ctx->stats.*field += n;
  ctx->stats.launches += n;
}
void log_call(const dsn_ctx* ctx, const char* what, long long B, long long T) {
  if (ctx && ctx->log) fprintf(stderr, "[dsn] %s B=%lld T=%lld launches so far %llu\n", what, B, T, (unsigned long long)ctx->stats.launches);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

// bf16 tensor map of rank `rank` (3 or 4); dims/strides innermost first, strides[0] implied.
int encode_map(dsn_ctx* ctx, CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
               const uint64_t* strides_bytes /* rank-1 */, const uint32_t* box) {
  dsn_map_slot* slot = nullptr;
  dsn_map_key key;
  if (ctx->map_cache) {
    memset(&key, 0, sizeof(key));
    key.base = base;
    key.rank = (uint32_t)rank;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides_bytes[i];
    uint64_t h = 1469598103934665603ull;  // FNV-1a over the key
    const unsigned char* kb = reinterpret_cast<const unsigned char*>(&key);
    for (size_t i = 0; i < sizeof(key); ++i) h = (h ^ kb[i]) * 1099511628211ull;
    // four probes from the hashed slot; a miss takes the first free probe, else replaces the hashed slot
    for (int probe = 0; probe < 4; ++probe) {
      dsn_map_slot* cand = &ctx->map_cache[(h + (uint64_t)probe) % DSN_MAP_CACHE_SLOTS];
      if (cand->used && memcmp(&cand->key, &key, sizeof(key)) == 0) {
        *out = cand->map;
        ++ctx->map_hits;
        return DSN_OK;
      }
      if (!cand->used && !slot) slot = cand;
    }
    if (!slot) slot = &ctx->map_cache[h % DSN_MAP_CACHE_SLOTS];
    ++ctx->map_misses;
  }
  cuuint64_t gd[4], gs[3];
  cuuint32_t bx[4], es[4];
  for (int i = 0; i < rank; ++i) {
    gd[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
    if (box[i] == 0 || box[i] > 256 || dims[i] == 0) return DSN_ERR_INVALID_ARG;
  }
  for (int i = 0; i + 1 < rank; ++i) {
    gs[i] = strides_bytes[i];
    if (gs[i] % 16 != 0 || gs[i] == 0) return DSN_ERR_ALIGNMENT;
  }
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, bx, es,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return DSN_ERR_CUDA;
  if (slot) {
    slot->key = key;
    slot->map = *out;
    slot->used = 1;
  }
  return DSN_OK;
}

// One sliced layer in the form the kernels take.
struct LayerCall {
  int dtype;
  int H, W, K, pad;      // linear: H = 1, W = R, K = 1
  int C_in, C_out;
  int64_t ldx, ldy;      // elements between rows (pixels)
  int64_t w_row, w_tap;  // elements between output rows / taps of the weight
  int T;
  const int32_t *k_in, *k_out;
  const void* Wt;
  const float* bias;
  const float *bn_scale, *bn_shift;
  const void* residual;
  int act, in_order, out_order, tail;
  const dsn_attention_desc* att;  // non-null: this chain element is the attention core, not a sliced layer
  const dsn_depthwise_desc* dw;   // non-null: this chain element is a slice-able depthwise convolution
  int R_in;                       // rows per sample it reads (differs from H * W, the rows it writes, for a strided depthwise element)
};

int check_slices(int T, const int32_t* k_in, const int32_t* k_out, int C_in, int C_out) {
  if (T < 1 || T > DSN_MAX_SLICES || !k_in || !k_out) return DSN_ERR_INVALID_ARG;
  for (int t = 0; t < T; ++t)
    if (k_in[t] < 1 || k_in[t] > C_in || k_out[t] < 1 || k_out[t] > C_out) return DSN_ERR_INVALID_ARG;
  return DSN_OK;
}

int check_routing(const dsn_routing* r, int T) {
  if (!r || r->B < 0 || r->G < 1 || r->G > DSN_MAX_GROUPS) return DSN_ERR_INVALID_ARG;
  if (!r->offsets || !r->perm) return DSN_ERR_INVALID_ARG;
  if (!r->group_slice && r->G > T) return DSN_ERR_INVALID_ARG;
  return DSN_OK;
}

int validate_call(const LayerCall& c, const dsn_routing* r, const void* x, const void* y) {
  if (!x || !y || !c.Wt) return DSN_ERR_INVALID_ARG;
  if ((c.bn_scale == nullptr) != (c.bn_shift == nullptr)) return DSN_ERR_INVALID_ARG;
  if (c.residual && c.residual == y) return DSN_ERR_INVALID_ARG;
  if (c.residual && c.dtype == DSN_BF16 && !aligned16(c.residual)) return DSN_ERR_ALIGNMENT;
  if (c.dtype != DSN_BF16 && c.dtype != DSN_F32) return DSN_ERR_INVALID_ARG;
  if (c.H < 1 || c.W < 1 || c.C_in < 1 || c.C_out < 1 || c.C_in > 32767 || c.C_out > 32767) return DSN_ERR_INVALID_ARG;
  if (c.act < DSN_ACT_NONE || c.act > DSN_ACT_GELU) return DSN_ERR_INVALID_ARG;
  if ((c.in_order != DSN_INPUT_ORDER && c.in_order != DSN_GROUPED) ||
      (c.out_order != DSN_INPUT_ORDER && c.out_order != DSN_GROUPED) ||
      (c.tail != DSN_TAIL_UNTOUCHED && c.tail != DSN_TAIL_ZERO))
    return DSN_ERR_INVALID_ARG;
  if (c.ldx < c.C_in || c.ldy < c.C_out || c.w_row < (int64_t)c.C_in * c.K * c.K) return DSN_ERR_INVALID_ARG;
  int e = check_slices(c.T, c.k_in, c.k_out, c.C_in, c.C_out);
  if (e) return e;
  e = check_routing(r, c.T);
  if (e) return e;
  if ((int64_t)r->B * c.H * c.W > 0x7fffffffLL) return DSN_ERR_INVALID_ARG;
  if (c.dtype == DSN_BF16) {
    if (!aligned16(x) || !aligned16(y) || !aligned16(c.Wt)) return DSN_ERR_ALIGNMENT;
    if (c.ldx % 8 || c.ldy % 8 || c.w_row % 8 || c.w_tap % 8) return DSN_ERR_ALIGNMENT;
    if (!(c.K == 1 && c.pad == 0) && !(c.K == 3 && c.pad == 1)) return DSN_ERR_UNSUPPORTED;
  } else {
    if (c.K != 1) return DSN_ERR_UNSUPPORTED;
  }
  return DSN_OK;
}

void fill_slice_table(SliceTable& st, const LayerCall& c) {
  memset(&st, 0, sizeof(st));
  for (int t = 0; t < c.T; ++t) {
    st.k_in[t] = c.k_in[t];
    st.k_out[t] = c.k_out[t];
  }
}

// Tile geometry for the bf16 kernel.  `per_sample`: no tile spans two samples (chained layers).
void choose_geometry(const LayerCall& c, GemmGeom& g, bool per_sample = false, bool halo = false) {
  memset(&g, 0, sizeof(g));
  g.H = c.H;
  g.W = c.W;
  g.R = c.H * c.W;
  g.taps = c.K * c.K;
  g.KW = c.K;
  g.pad = c.pad;
  g.a_input_order = c.in_order == DSN_INPUT_ORDER;
  g.y_input_order = c.out_order == DSN_INPUT_ORDER;
  int max_ko = 1;
  for (int t = 0; t < c.T; ++t) max_ko = c.k_out[t] > max_ko ? c.k_out[t] : max_ko;
  g.BN = max_ko > 128 ? 256 : (max_ko > 64 ? 128 : 64);
  g.stages = g.BN == 256 ? 4 : (g.BN == 128 ? 6 : 8);
  if (c.K == 1 && !g.a_input_order && !per_sample) {
    g.flat = 1;  // grouped rows are contiguous: tile them without regard to sample boundaries
    g.bw = DSN_GEMM_BM;
    g.bh = g.nb = g.tiles_x = g.tiles_y = 1;
    return;
  }
  if (halo) {  // 3x3: M rows run over the padded width, whole image rows per tile
    g.halo = 1;
    g.bw = g.W + 2;
    g.bh = DSN_GEMM_BM / g.bw;
    if (g.bh > g.H) g.bh = g.H;
    const int bands = (g.H + g.bh - 1) / g.bh;
    g.bh = (g.H + bands - 1) / bands;
    g.nb = 1;
    g.tiles_x = 1;
    g.tiles_y = bands;
    return;
  }
  if (c.K == 1) {  // input order: a sample's R rows form one "image" of height 1
    g.H = 1;
    g.W = g.R;
  }
  g.bw = g.W < DSN_GEMM_BM ? g.W : DSN_GEMM_BM;
  g.bh = DSN_GEMM_BM / g.bw;
  if (g.bh > g.H) g.bh = g.H;
  if (g.bh > 1) {  // balance the row bands of an image
    const int bands = (g.H + g.bh - 1) / g.bh;
    g.bh = (g.H + bands - 1) / bands;
  }
  g.nb = 1;
  if (!g.a_input_order && !per_sample && g.bh == g.H && g.bw == g.W) {
    g.nb = DSN_GEMM_BM / (g.bw * g.bh);
    if (g.nb < 1) g.nb = 1;
  }
  g.tiles_x = (g.W + g.bw - 1) / g.bw;
  g.tiles_y = (g.H + g.bh - 1) / g.bh;
}

// Everything of the kernel parameters except the tensor maps.
void fill_gemm_params(dsn_ctx* ctx, const LayerCall& c, const dsn_routing* r, void* y, bool per_sample, GemmParams& p,
                      bool halo = false) {
  memset(&p, 0, sizeof(p));
  choose_geometry(c, p.g, per_sample, halo);
  p.B = r->B;
  p.G = r->G;
  p.T = c.T;
  p.offsets = r->offsets;
  p.perm = r->perm;
  p.group_slice = r->group_slice;
  p.y = static_cast<__nv_bfloat16*>(y);
  p.ldy = c.ldy;
  p.bias = c.bias;
  p.bn_scale = c.bn_scale;
  p.bn_shift = c.bn_shift;
  p.bn_ld = c.C_out;
  p.residual = static_cast<const __nv_bfloat16*>(c.residual);
  p.act = c.act;
  p.status = ctx->d_status;
  for (int t = 0; t < c.T; ++t) {
    p.k_in[t] = (int16_t)c.k_in[t];
    p.k_out[t] = (int16_t)c.k_out[t];
  }
}

// Tensor maps for the next DSN_GEMM_MAX_MAPS distinct slices (k_in, k_out) not yet done; one map
// triple per distinct slice.  `remaining` counts the paths still without a map afterwards.
int fill_gemm_maps(dsn_ctx* ctx, const LayerCall& c, const dsn_routing* r, const void* x, void* y, GemmParams& p,
                   int* done, int& remaining) {
  const GemmGeom& g = p.g;
  int nmaps = 0;
  int map_k[DSN_GEMM_MAX_MAPS], map_n[DSN_GEMM_MAX_MAPS];
  memset(p.map_id, 0xFF, sizeof(p.map_id));
  for (int t = 0; t < c.T; ++t) {
    if (done[t]) continue;
    int id = -1;
    for (int m = 0; m < nmaps; ++m)
      if (map_k[m] == c.k_in[t] && map_n[m] == c.k_out[t]) id = m;
    if (id < 0) {
      if (nmaps == DSN_GEMM_MAX_MAPS) continue;  // next launch
      id = nmaps++;
      map_k[id] = c.k_in[t];
      map_n[id] = c.k_out[t];
    }
    p.map_id[t] = (uint8_t)id;
    done[t] = 1;
    --remaining;
  }
  for (int m = 0; m < nmaps; ++m) {
    const uint64_t kv = (uint64_t)map_k[m];
    int e;
    if (g.flat) {
      const uint64_t rows = (uint64_t)r->B * g.R;
      const uint64_t dims[4] = {kv, rows, 1, 1};
      const uint64_t str[3] = {(uint64_t)c.ldx * 2, (uint64_t)c.ldx * 2 * rows, (uint64_t)c.ldx * 2 * rows};
      const uint32_t box[4] = {DSN_GEMM_BK, DSN_GEMM_BM, 1, 1};
      e = encode_map(ctx, &p.mapA[m], x, 4, dims, str, box);
    } else {
      const uint64_t dims[4] = {kv, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)r->B};
      const uint64_t str[3] = {(uint64_t)c.ldx * 2, (uint64_t)c.ldx * 2 * g.W, (uint64_t)c.ldx * 2 * g.W * g.H};
      const uint32_t box[4] = {DSN_GEMM_BK, (uint32_t)g.bw, (uint32_t)(g.bh + (g.halo ? 2 : 0)), (uint32_t)g.nb};
      e = encode_map(ctx, &p.mapA[m], x, 4, dims, str, box);
    }
    if (e) return e;
    const uint64_t wd[3] = {kv, (uint64_t)g.taps, (uint64_t)map_n[m]};  // rows beyond k_out: zeros, not fetched
    const uint64_t ws[2] = {(uint64_t)c.w_tap * 2, (uint64_t)c.w_row * 2};
    const uint32_t wb[3] = {DSN_GEMM_BK, 1, (uint32_t)(g.pair ? g.BN / 2 : g.BN)};
    e = encode_map(ctx, &p.mapB[m], c.Wt, 3, wd, ws, wb);
    if (e) return e;
    // columns clipped at k_out rounded down to 8 (the store clips at 16-byte granularity; the epilogue writes the 1..7
    // columns beyond with plain stores); widths below 8 never use the map
    const uint64_t yn = (uint64_t)(map_n[m] >= 8 ? (map_n[m] & ~7) : 8);
    if (g.halo) {
      // the staged-tile kernel stores a CTA's whole block at once: (channel, x, y, sample) with the block's padded
      // extent as the box; what lies beyond the image's width and height is clipped by the store
      const uint64_t yd[4] = {yn, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)r->B};
      const uint64_t ys[3] = {(uint64_t)c.ldy * 2, (uint64_t)c.ldy * 2 * g.W, (uint64_t)c.ldy * 2 * g.W * g.H};
      const uint32_t yb[4] = {64, (uint32_t)g.bw, (uint32_t)g.bh, 1};
      e = encode_map(ctx, &p.mapY[m], y, 4, yd, ys, yb);
    } else {
      const uint64_t yd[2] = {yn, (uint64_t)r->B * g.R};
      const uint64_t ys[1] = {(uint64_t)c.ldy * 2};
      const uint32_t yb[2] = {64, 32};
      e = encode_map(ctx, &p.mapY[m], y, 2, yd, ys, yb);
    }
    if (e) return e;
  }
  return DSN_OK;
}

// resident CTA pairs for this n-tile width (0: no pair can be resident, use one CTA per tile)
int pair_clusters_for(dsn_ctx* ctx, int BN) {
  if (ctx->gemm_mode != 0) return 0;
  const int bn_slot = BN == 256 ? 2 : (BN == 128 ? 1 : 0);
  if (ctx->pair_clusters[bn_slot] < 0) ctx->pair_clusters[bn_slot] = dsn_gemm_pair_max_clusters(227 * 1024);
  int clusters = ctx->pair_clusters[bn_slot];
  if (clusters > ctx->sm_count / 2) clusters = ctx->sm_count / 2;
  return clusters;
}

int run_bf16(dsn_ctx* ctx, const LayerCall& c, const dsn_routing* r, const void* x, void* y, cudaStream_t s) {
  GemmParams p;
  // 3x3 layers with slices up to 128 wide on images of at least 12 pixels a side stage the input tile once,
  // with its halo; smaller images (7x7) keep one load per tap, which packs two whole images into a tile
  bool halo = ctx->conv_halo && ctx->gemm_mode == 0 && c.K == 3 && c.pad == 1 && c.W >= 12 && c.W + 2 <= DSN_GEMM_BM;
  if (halo) {  // measured: a gain for n-tiles up to 128 wide (1.2-1.5x), none for 256-wide ones (tensor bound either way)
    int max_ko = 1;
    for (int t = 0; t < c.T; ++t) max_ko = c.k_out[t] > max_ko ? c.k_out[t] : max_ko;
    halo = max_ko <= 128;
  }
  fill_gemm_params(ctx, c, r, y, false, p, halo);
  const GemmGeom& g = p.g;
  if (halo) {
    const int clusters_h = pair_clusters_for(ctx, g.BN);
    if (clusters_h > 0) {
      p.g.pair = 1;
      // Weight ring: a slot holds all nine taps of a chunk where that fits twice (36 KB slots for 64-wide
      // n-tiles, 72 KB for 128-wide ones), otherwise one tap; two such slots hold the whole weights of slices up
      // to 128 channels in, which then stay resident from tile to tile.  The activation ring gets 2 to 4 blocks of
      // what is left.  Wide images have large blocks: the choice is made on the actual sizes.
      const size_t limit = 227 * 1024;
      bool fits = false;
      for (int tps = (g.BN == 256 ? 1 : 9); !fits; tps = 1) {
        p.g.tps = tps;
        p.g.stages = tps == 9 ? 2 : (g.BN == 256 ? 6 : 8);
        p.g.a_slots = 4;
        while (p.g.a_slots > 2 && dsn_gemm_halo_smem_bytes(g.BN, g.stages, tps, p.g.a_slots, r->G, g.bw, g.bh) > limit) --p.g.a_slots;
        while (p.g.stages > 2 && dsn_gemm_halo_smem_bytes(g.BN, p.g.stages, tps, g.a_slots, r->G, g.bw, g.bh) > limit) --p.g.stages;
        fits = dsn_gemm_halo_smem_bytes(g.BN, g.stages, tps, g.a_slots, r->G, g.bw, g.bh) <= limit;
        if (tps == 1) break;
      }
      if (!fits) return DSN_ERR_UNSUPPORTED;  // cannot happen for W + 2 <= 128: two blocks and two boxes always fit
      // Schedule: every pair gets one contiguous range of the tile sequence, cut by estimated time (few changes of
      // slice per pair, so the weights stay in the ring); the strided order is kept for comparisons.
      p.g.ranges = ctx->halo_sched != 1;
      const size_t smem_h = dsn_gemm_halo_smem_bytes(g.BN, g.stages, g.tps, g.a_slots, r->G, g.bw, g.bh);
      int done_h[DSN_MAX_SLICES];
      memset(done_h, 0, sizeof(done_h));
      int remaining_h = c.T;
      while (remaining_h > 0) {
        const int e = fill_gemm_maps(ctx, c, r, x, y, p, done_h, remaining_h);
        if (e) return e;
        count_launch(ctx, &dsn_stats::launches_gemm_halo);
        if (dsn_launch_gemm_bf16_halo(p, clusters_h, smem_h, s) != cudaSuccess) return DSN_ERR_CUDA;
      }
      return DSN_OK;
    }
    fill_gemm_params(ctx, c, r, y, false, p, false);  // no pair can be resident: the one-CTA kernel, one load per tap
  }
  // CTA pairs (two SMs per 256-row tile) halve the weight traffic per SM; fall back to one CTA per
  // tile when no pair can be resident
  const int clusters = pair_clusters_for(ctx, g.BN);
  size_t smem = 0;
  if (clusters > 0) {
    p.g.pair = 1;
    p.g.stages = g.BN == 256 ? 6 : 8;
    while (p.g.stages > 2 && dsn_gemm_pair_smem_bytes(g.BN, p.g.stages, r->G) > 227 * 1024) --p.g.stages;
    smem = dsn_gemm_pair_smem_bytes(g.BN, g.stages, r->G);
  } else {
    p.g.pair = 0;
    p.g.stages = g.BN == 256 ? 4 : (g.BN == 128 ? 6 : 8);
    while (p.g.stages > 2 && dsn_gemm_smem_bytes(g.BN, p.g.stages, r->G) > 227 * 1024) --p.g.stages;
    smem = dsn_gemm_smem_bytes(g.BN, g.stages, r->G);
  }
  int done[DSN_MAX_SLICES];
  memset(done, 0, sizeof(done));
  int remaining = c.T;
  while (remaining > 0) {
    const int e = fill_gemm_maps(ctx, c, r, x, y, p, done, remaining);
    if (e) return e;
    if (g.pair) {
      if (count_launch(ctx, &dsn_stats::launches_gemm_pair), dsn_launch_gemm_bf16_pair(p, clusters, smem, s) != cudaSuccess) return DSN_ERR_CUDA;
    } else if (count_launch(ctx, &dsn_stats::launches_gemm_one_cta), dsn_launch_gemm_bf16(p, ctx->sm_count, smem, s) != cudaSuccess) {
      return DSN_ERR_CUDA;
    }
  }
  return DSN_OK;
}

// A chain of bf16 sliced layers whose batch is small enough that every CTA pair owns at most two
// samples runs as ONE launch (per-sample tiles, intermediates in grouped order): separate launches
// would each pay their own set-up, ramp and tail for one or two tiles per pair.
// Returns 1 when the chain was launched, 0 when the caller should run the layers one by one, < 0 on error.
int try_run_chain(dsn_ctx* ctx, const LayerCall* calls, int n, const dsn_routing* r, const void* const* in,
                  void* const* out, cudaStream_t s) {
  if (!ctx->chain_mode || ctx->gemm_mode != 0 || n < 2 || n > DSN_CHAIN_MAX_LAYERS) return 0;
  if (r->group_slice || r->B < 1) return 0;
  int bn_max = 64;
  for (int j = 0; j < n; ++j) {
    const LayerCall& c = calls[j];
    if (c.att || c.dw || c.dtype != DSN_BF16 || c.tail != DSN_TAIL_UNTOUCHED) return 0;
    // a sample must fill most of ONE 256-row pair tile: with more rows per sample the single-layer launches
    // (tiles across sample boundaries, halo form of the 3x3 layer) are faster (measured at 28x28 and 56x56)
    if (c.H * c.W < 150 || c.H * c.W > 256) return 0;
    int distinct = 0, seen_k[DSN_MAX_SLICES], seen_n[DSN_MAX_SLICES];
    for (int t = 0; t < c.T; ++t) {
      bool dup = false;
      for (int u = 0; u < distinct; ++u) dup = dup || (seen_k[u] == c.k_in[t] && seen_n[u] == c.k_out[t]);
      if (!dup) { seen_k[distinct] = c.k_in[t]; seen_n[distinct] = c.k_out[t]; ++distinct; }
    }
    if (distinct > DSN_GEMM_MAX_MAPS) return 0;
  }
  DsnChainParams cp;  // about 20 KB of kernel parameters
  for (int j = 0; j < n; ++j) {
    fill_gemm_params(ctx, calls[j], r, out[j], true, cp.L[j]);
    cp.L[j].g.pair = 1;
    if (cp.L[j].g.BN > bn_max) bn_max = cp.L[j].g.BN;
  }
  // The last layer can take its activations from tensor memory when it is a 1x1 / linear layer, the layer before
  // produces a sample in ONE pair tile (so a tile of that layer is all the last layer needs of the sample) and at
  // most 256 channels (128 tensor-memory columns of packed pairs beside two 128-column accumulators per region).
  // The last layer then walks the tiles of the layer before (same pixel rectangles, same rows) with 128-wide n-tiles.
  cp.fuse_tail = 0;
  if (ctx->chain_fuse) {
    const LayerCall& last = calls[n - 1];
    const GemmGeom& gp = cp.L[n - 2].g;
    bool ok = last.K == 1 && gp.tiles_x * gp.tiles_y <= 2 && gp.nb == 1 && !gp.flat;
    for (int t = 0; ok && t < last.T; ++t) ok = calls[n - 2].k_out[t] <= 256 && last.k_in[t] <= calls[n - 2].k_out[t];
    if (ok) {
      GemmGeom& gl = cp.L[n - 1].g;
      const int y_order = gl.y_input_order;
      int max_ko = 1;
      for (int t = 0; t < last.T; ++t) max_ko = last.k_out[t] > max_ko ? last.k_out[t] : max_ko;
      gl = gp;
      gl.taps = 1;
      gl.KW = 1;
      gl.pad = 0;
      gl.a_input_order = 0;
      gl.y_input_order = y_order;
      gl.BN = max_ko > 64 ? 128 : 64;
      cp.fuse_tail = 1;
      bn_max = 256;  // two regions of 256 columns: rows of a sample below, an accumulator of the last layer above
    }
  }
  const int clusters = pair_clusters_for(ctx, bn_max);
  if (clusters <= 0 || r->B > 2 * clusters) return 0;
  int stages = bn_max == 256 ? 6 : 8;
  while (stages > 2 && dsn_gemm_chain_smem_bytes(bn_max, stages, r->G) > 227 * 1024) --stages;
  for (int j = 0; j < n; ++j) {
    int done[DSN_MAX_SLICES];
    memset(done, 0, sizeof(done));
    int remaining = calls[j].T;
    cp.L[j].g.stages = stages;
    const int e = fill_gemm_maps(ctx, calls[j], r, in[j], out[j], cp.L[j], done, remaining);
    if (e) return e;
    if (remaining != 0) return 0;
  }
  cp.n_layers = n;
  cp.stages = stages;
  cp.bn_max = bn_max;
  count_launch(ctx, &dsn_stats::launches_gemm_chain);
  if (cp.fuse_tail) ++ctx->stats.launches_gemm_chain_tmem;
  if (dsn_launch_gemm_bf16_chain(cp, clusters, dsn_gemm_chain_smem_bytes(bn_max, stages, r->G), s) != cudaSuccess)
    return DSN_ERR_CUDA;
  return 1;
}

// Can the depthwise element `d` and the sliced layer `c` that follows it run as one kernel?
bool dwpw_fusable(const LayerCall& d, const LayerCall& c, const void* x) {
  if (!d.dw || c.att || c.dw || c.dtype != DSN_BF16 || c.K != 1 || c.residual || c.tail != DSN_TAIL_UNTOUCHED) return false;
  const dsn_depthwise_desc* w = d.dw;
  if (w->C % 8 || d.ldx % 8 || !aligned16(x) || !aligned16(w->W)) return false;
  for (int t = 0; t < c.T; ++t)
    if (w->c[t] % 8 || c.k_in[t] != w->c[t]) return false;
  return true;
}

// depthwise element `d` (input x, order d.in_order) + pointwise layer `c` (output y) as one launch per 16 distinct slices
int run_dwpw(dsn_ctx* ctx, const LayerCall& d, const LayerCall& c, const dsn_routing* r, const void* x, void* y,
             cudaStream_t s) {
  if (r->B == 0) return DSN_OK;
  DwPwParams q;
  memset(&q, 0, sizeof(q));
  LayerCall cc = c;
  cc.in_order = DSN_GROUPED;
  fill_gemm_params(ctx, cc, r, y, false, q.g);
  GemmGeom& g = q.g.g;
  g.flat = 1;  // M rows are the group's output pixels, whatever the order of the block input
  g.bw = DSN_GEMM_BM;
  g.bh = g.nb = g.tiles_x = g.tiles_y = 1;
  g.R = c.H * c.W;
  g.a_input_order = d.in_order == DSN_INPUT_ORDER;
  g.pair = 0;
  g.stages = g.BN == 256 ? 4 : (g.BN == 128 ? 6 : 8);
  while (g.stages > 2 && dsn_dwpw_smem_bytes(g.BN, g.stages, r->G) > 227 * 1024) --g.stages;
  const dsn_depthwise_desc* w = d.dw;
  q.x = static_cast<const __nv_bfloat16*>(x);
  q.ldx = d.ldx;
  q.w = static_cast<const __nv_bfloat16*>(w->W);
  q.dw_bias = w->bias; q.dw_bn_scale = w->bn_scale; q.dw_bn_shift = w->bn_shift; q.dw_act = w->act;
  q.H = w->H; q.W = w->W_; q.Wo = c.W; q.K = w->K; q.stride = w->stride; q.C = w->C;
  for (int t = 0; t < w->T; ++t) q.ksize[t] = (int8_t)w->ksize[t];
  int done[DSN_MAX_SLICES];
  memset(done, 0, sizeof(done));
  int remaining = c.T;
  const size_t smem = dsn_dwpw_smem_bytes(g.BN, g.stages, r->G);
  while (remaining > 0) {
    const int e = fill_gemm_maps(ctx, cc, r, y /* stands in for the activation map, which this kernel does not use */, y,
                                 q.g, done, remaining);
    if (e) return e;
    count_launch(ctx, &dsn_stats::launches_dwpw);
    if (dsn_launch_dwpw(q, ctx->sm_count, smem, s) != cudaSuccess) return DSN_ERR_CUDA;
  }
  return DSN_OK;
}

int run_layer(dsn_ctx* ctx, const LayerCall& c, const dsn_routing* r, const void* x, void* y, cudaStream_t s) {
  int e = check_ctx(ctx);
  if (e) return e;
  ++ctx->stats.calls;
  log_call(ctx, c.K == 1 ? "sliced layer (1x1 / linear)" : "sliced layer (3x3)", r ? r->B : -1, c.T);
  e = validate_call(c, r, x, y);
  if (e) return e;
  if (r->B == 0) return DSN_OK;
  SliceTable st;
  fill_slice_table(st, c);
  if (c.dtype == DSN_BF16) {
    e = run_bf16(ctx, c, r, x, y, s);
    if (e) return e;
  } else {
    count_launch(ctx, &dsn_stats::launches_linear_f32);
    if (dsn_launch_linear_f32(st, c.T, c.H * c.W, static_cast<const float*>(x), c.ldx,
                              static_cast<const float*>(c.Wt), c.w_row, static_cast<float*>(y), c.ldy, c.bias, c.bn_scale, c.bn_shift,
                              c.C_out, static_cast<const float*>(c.residual), c.act,
                              c.in_order == DSN_INPUT_ORDER, c.out_order == DSN_INPUT_ORDER, r->B, r->G, r->offsets,
                              r->perm, r->group_slice, ctx->sm_count, s) != cudaSuccess)
      return DSN_ERR_CUDA;
  }
  if (c.tail == DSN_TAIL_ZERO) {
    count_launch(ctx, &dsn_stats::launches_copy);
    if (dsn_launch_zero_tail(st, c.dtype == DSN_BF16 ? 2 : 4, c.H * c.W, c.C_out, y, c.ldy,
                             c.out_order == DSN_INPUT_ORDER, r->B, r->G, r->offsets, r->perm, r->group_slice,
                             s) != cudaSuccess)
      return DSN_ERR_CUDA;
  }
  return DSN_OK;
}

LayerCall from_linear(const dsn_linear_desc* d) {
  LayerCall c;
  c.dtype = d->dtype;
  c.H = 1; c.W = d->R; c.K = 1; c.pad = 0;
  c.C_in = d->C_in; c.C_out = d->C_out;
  c.ldx = d->ldx; c.ldy = d->ldy;
  c.w_row = d->ldw; c.w_tap = d->ldw;
  c.T = d->T; c.k_in = d->k_in; c.k_out = d->k_out;
  c.Wt = d->W; c.bias = d->bias; c.bn_scale = d->bn_scale; c.bn_shift = d->bn_shift; c.residual = d->residual; c.att = nullptr;
  c.dw = nullptr; c.R_in = d->R;
  c.act = d->act; c.in_order = d->in_order; c.out_order = d->out_order; c.tail = d->tail;
  return c;
}

LayerCall from_conv(const dsn_conv_desc* d) {
  LayerCall c;
  c.dtype = d->dtype;
  c.H = d->H; c.W = d->W_; c.K = d->K; c.pad = d->pad;
  c.C_in = d->C_in; c.C_out = d->C_out;
  c.ldx = d->ldx; c.ldy = d->ldy;
  c.w_row = (int64_t)d->K * d->K * d->C_in; c.w_tap = d->C_in;
  c.T = d->T; c.k_in = d->k_in; c.k_out = d->k_out;
  c.Wt = d->W; c.bias = d->bias; c.bn_scale = d->bn_scale; c.bn_shift = d->bn_shift; c.residual = d->residual; c.att = nullptr;
  c.dw = nullptr; c.R_in = d->H * d->W_;
  c.act = d->act; c.in_order = d->in_order; c.out_order = d->out_order; c.tail = d->tail;
  return c;
}

int check_depthwise(const dsn_depthwise_desc* d) {
  if (!d || !d->W || !d->c || !d->ksize) return DSN_ERR_INVALID_ARG;
  if (d->dtype != DSN_BF16) return DSN_ERR_UNSUPPORTED;
  if (d->H < 1 || d->W_ < 1 || d->C < 1 || d->C > 32767 || d->K < 1 || d->K > 7 || d->K % 2 == 0) return DSN_ERR_INVALID_ARG;
  if (d->stride != 1 && d->stride != 2) return DSN_ERR_UNSUPPORTED;
  if (d->ldx < d->C || d->ldy < d->C || d->T < 1 || d->T > DSN_MAX_SLICES) return DSN_ERR_INVALID_ARG;
  if (d->act < DSN_ACT_NONE || d->act > DSN_ACT_GELU) return DSN_ERR_INVALID_ARG;
  if ((d->bn_scale == nullptr) != (d->bn_shift == nullptr)) return DSN_ERR_INVALID_ARG;
  for (int t = 0; t < d->T; ++t)
    if (d->c[t] < 1 || d->c[t] > d->C || d->ksize[t] < 1 || d->ksize[t] > d->K || d->ksize[t] % 2 == 0)
      return DSN_ERR_INVALID_ARG;
  return DSN_OK;
}

// Host-side checks of an attention element (pointers may be null when only the descriptor is checked).
int check_attention(const dsn_attention_desc* d, const dsn_routing* r, const void* qkv, const void* out) {
  if (!d || !d->heads) return DSN_ERR_INVALID_ARG;
  if (d->dtype != DSN_BF16 || d->D_h != 64 || d->N > 256) return DSN_ERR_UNSUPPORTED;
  if (d->N < 1 || d->H < 1 || d->H > 64 || d->T < 1 || d->T > DSN_MAX_SLICES) return DSN_ERR_INVALID_ARG;
  if (d->ld_qkv < (int64_t)3 * d->H * d->D_h || d->ld_out < (int64_t)d->H * d->D_h) return DSN_ERR_INVALID_ARG;
  if (d->order != DSN_INPUT_ORDER && d->order != DSN_GROUPED) return DSN_ERR_INVALID_ARG;
  for (int t = 0; t < d->T; ++t)
    if (d->heads[t] < 1 || d->heads[t] > d->H) return DSN_ERR_INVALID_ARG;
  int e = check_routing(r, d->T);
  if (e) return e;
  if ((qkv && !aligned16(qkv)) || (out && !aligned16(out)) || d->ld_qkv % 8 || d->ld_out % 8) return DSN_ERR_ALIGNMENT;
  if ((int64_t)r->B * d->N > 0x7fffffffLL) return DSN_ERR_INVALID_ARG;
  return DSN_OK;
}

int check_gate(const dsn_gate_desc* g) {
  if (!g || !g->W1 || !g->W2) return DSN_ERR_INVALID_ARG;
  if (g->dtype != DSN_BF16 && g->dtype != DSN_F32) return DSN_ERR_INVALID_ARG;
  if (g->B < 0 || g->R < 1 || g->C_full < 1 || g->c_valid < 1 || g->c_valid > g->C_full || g->C_mlp < 1 ||
      g->T < 1 || g->T > DSN_MAX_SLICES || g->ldx < g->c_valid)
    return DSN_ERR_INVALID_ARG;
  if ((size_t)4 * ((size_t)g->T * (g->C_mlp + 32) + 8 * (size_t)g->C_mlp + 8 * DSN_MAX_SLICES) > 200 * 1024)
    return DSN_ERR_UNSUPPORTED;  // score kernel stages W2 in shared memory
  return DSN_OK;
}

// workspace carving for dsn_layer_forward
struct LayerPlan {
  size_t off_idx, off_counts, off_offsets, off_perm, off_inv, off_gate, off_buf[2], off_gather, total;
  size_t elem;
  bool gather_first;
};

int layer_call_of(const dsn_layer_desc* L, int j, LayerCall& c) {
  if (!L->layer[j]) return DSN_ERR_INVALID_ARG;
  if (L->kind[j] == DSN_LAYER_LINEAR) c = from_linear(static_cast<const dsn_linear_desc*>(L->layer[j]));
  else if (L->kind[j] == DSN_LAYER_CONV) c = from_conv(static_cast<const dsn_conv_desc*>(L->layer[j]));
  else if (L->kind[j] == DSN_LAYER_ATTENTION) {
    // between two sliced layers only: it reads and writes grouped intermediates
    if (j == 0 || j + 1 == L->n_layers) return DSN_ERR_INVALID_ARG;
    const dsn_attention_desc* a = static_cast<const dsn_attention_desc*>(L->layer[j]);
    if (!a->heads || a->T < 1 || a->T > DSN_MAX_SLICES || a->D_h < 1 || a->H < 1) return DSN_ERR_INVALID_ARG;
    memset(&c, 0, sizeof(c));
    c.att = a;
    c.R_in = a->N;
    c.dtype = a->dtype;
    c.H = 1; c.W = a->N; c.K = 1;
    c.C_in = 3 * a->H * a->D_h;
    c.C_out = a->H * a->D_h;
    c.T = a->T;
  } else if (L->kind[j] == DSN_LAYER_DEPTHWISE) {
    // never the last element: the block's output comes from a sliced layer
    if (j + 1 == L->n_layers) return DSN_ERR_INVALID_ARG;
    const dsn_depthwise_desc* d = static_cast<const dsn_depthwise_desc*>(L->layer[j]);
    const int e = check_depthwise(d);
    if (e) return e;
    memset(&c, 0, sizeof(c));
    c.dw = d;
    c.dtype = d->dtype;
    c.H = (d->H - 1) / d->stride + 1; c.W = (d->W_ - 1) / d->stride + 1; c.K = 1;   // the rows it writes
    c.R_in = d->H * d->W_;
    c.C_in = d->C; c.C_out = d->C;
    c.T = d->T;
    c.k_in = d->c; c.k_out = d->c;
    c.ldx = d->ldx; c.ldy = d->C;
  } else return DSN_ERR_INVALID_ARG;
  return DSN_OK;
}

int plan_layer(const dsn_layer_desc* L, LayerPlan& pl) {
  if (!L || L->B < 0 || L->T < 1 || L->T > DSN_MAX_SLICES || L->n_layers < 1 || L->n_layers > DSN_MAX_CHAIN)
    return DSN_ERR_INVALID_ARG;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t B = (size_t)L->B;
  pl.off_idx = take(4 * B);
  pl.off_counts = take(4 * (size_t)L->T);
  pl.off_offsets = take(4 * ((size_t)L->T + 1));
  pl.off_perm = take(4 * B);
  pl.off_inv = take(4 * B);
  pl.off_gate = take(L->gate ? dsn_gate_workspace_bytes(L->gate) : 0);
  size_t need[2] = {0, 0};
  LayerCall first;
  int e = layer_call_of(L, 0, first);
  if (e) return e;
  pl.elem = first.dtype == DSN_BF16 ? 2 : 4;
  int prev_out = 0, prev_R = 0;
  int prev_k_out[DSN_MAX_SLICES] = {0};
  for (int j = 0; j < L->n_layers; ++j) {
    LayerCall c;
    e = layer_call_of(L, j, c);
    if (e) return e;
    if (c.T != L->T || c.dtype != first.dtype) return DSN_ERR_INVALID_ARG;
    if (!c.att && (!c.k_in || !c.k_out)) return DSN_ERR_INVALID_ARG;
    if (j > 0 && (c.C_in != prev_out || c.R_in != prev_R)) return DSN_ERR_INVALID_ARG;
    // every layer of the block inherits the one decision (Sec. 5): a path may read no more columns of an
    // intermediate than the layer before wrote for that path (the columns beyond hold stale workspace bytes)
    for (int t = 0; t < L->T; ++t) {
      const int need_in = c.att ? 3 * c.att->heads[t] * c.att->D_h : c.k_in[t];
      if (j > 0 && need_in > prev_k_out[t]) return DSN_ERR_INVALID_ARG;
      prev_k_out[t] = c.att ? c.att->heads[t] * c.att->D_h : c.k_out[t];
    }
    prev_out = c.C_out;
    prev_R = c.H * c.W;
    if (j + 1 < L->n_layers) {
      const size_t bytes = B * (size_t)prev_R * (size_t)c.C_out * pl.elem;
      if (bytes > need[j & 1]) need[j & 1] = bytes;
    }
  }
  pl.off_buf[0] = take(need[0]);
  pl.off_buf[1] = take(need[1]);
  // a physical gather pays when a sample has too few rows to fill a 128-row tile on its own
  pl.gather_first = first.dtype == DSN_BF16 && first.H * first.W <= 64 && !first.dw;
  pl.off_gather = take(pl.gather_first ? B * (size_t)(first.H * first.W) * (size_t)first.C_in * pl.elem : 0);
  pl.total = off;
  return DSN_OK;
}

}  // namespace

// ================================================================================== C ABI
extern "C" {

const char* dsn_strerror(int code) {
  switch (code) {
    case DSN_OK: return "ok";
    case DSN_ERR_INVALID_ARG: return "invalid argument";
    case DSN_ERR_ALIGNMENT: return "pointer or leading dimension not aligned as required";
    case DSN_ERR_WORKSPACE: return "workspace missing or too small";
    case DSN_ERR_UNSUPPORTED: return "unsupported combination";
    case DSN_ERR_BAD_INDEX: return "routing index out of range";
    case DSN_ERR_CUDA: return "CUDA call failed";
    case DSN_ERR_TIMEOUT: return "bounded device wait ran out";
    case DSN_ERR_NONFINITE: return "non-finite gate score";
    default: return "unknown dsn status";
  }
}

int dsn_create(dsn_ctx** out, int device) {
  if (!out) return DSN_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return DSN_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return DSN_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return DSN_ERR_CUDA;
  if (prop.major != 10) return DSN_ERR_UNSUPPORTED;  // the kernels are sm_100a only
  dsn_ctx* c = static_cast<dsn_ctx*>(calloc(1, sizeof(dsn_ctx)));
  if (!c) return DSN_ERR_INVALID_ARG;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->pair_clusters[0] = c->pair_clusters[1] = c->pair_clusters[2] = -1;
  {
    const char* m = getenv("DSN_GEMM_MODE");  // "1cta" forces one CTA per tile (for comparisons)
    c->gemm_mode = (m && strcmp(m, "1cta") == 0) ? 1 : 0;
    const char* cv = getenv("DSN_CONV3X3");  // "taps": 3x3 layers load the tile once per tap (for comparisons)
    c->conv_halo = (cv && strcmp(cv, "taps") == 0) ? 0 : 1;
    const char* hs = getenv("DSN_HALO_SCHED");
    c->halo_sched = (hs && strcmp(hs, "strided") == 0) ? 1 : ((hs && strcmp(hs, "ranges") == 0) ? 2 : 0);
    const char* lg = getenv("DSN_LOG");  // "1": one line per entry-point call on stderr
    c->log = (lg && lg[0] == '1') ? 1 : 0;
    const char* mc = getenv("DSN_MAP_CACHE");  // "0": encode every tensor map anew on every call (for comparisons)
    if (!(mc && mc[0] == '0')) c->map_cache = static_cast<dsn_map_slot*>(calloc(DSN_MAP_CACHE_SLOTS, sizeof(dsn_map_slot)));
    const char* dp = getenv("DSN_DWPW");  // "fused": a depthwise element and the 1x1 layer after it run as one kernel
    c->dwpw_fused = (dp && strcmp(dp, "fused") == 0) ? 1 : 0;
    const char* ch = getenv("DSN_CHAIN");  // "0": one launch per layer even for small batches (for comparisons)
    c->chain_mode = (ch && ch[0] == '0') ? 0 : 1;
    // "1": in a chained launch the last 1x1 layer reads the layer before from tensor memory (measured slower on the
    // bottleneck block: the last layer then runs on 128-wide n-tiles; off by default)
    const char* cf = getenv("DSN_CHAIN_FUSE");
    c->chain_fuse = (cf && cf[0] == '1') ? 1 : 0;
  }
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !c->encode_tiled) {
    free(c);
    return DSN_ERR_CUDA;
  }
  if (cudaMalloc(&c->d_status, sizeof(int32_t) * DSN_STATUS_WORDS) != cudaSuccess ||
      cudaMemset(c->d_status, 0, sizeof(int32_t) * DSN_STATUS_WORDS) != cudaSuccess) {
    free(c);
    return DSN_ERR_CUDA;
  }
  *out = c;
  return DSN_OK;
}

int dsn_destroy(dsn_ctx* ctx) {
  if (!ctx) return DSN_ERR_INVALID_ARG;
  cudaFree(ctx->d_status);
  free(ctx->map_cache);
  free(ctx);
  return DSN_OK;
}

int dsn_get_status(dsn_ctx* ctx, void* stream, int32_t* code, int32_t* detail) {
  if (int e = check_ctx(ctx)) return e;
  int32_t h[DSN_STATUS_REPORT_WORDS];
  cudaStream_t s = as_stream(stream);
  if (cudaMemcpyAsync(h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return DSN_ERR_CUDA;
  if (cudaMemsetAsync(ctx->d_status, 0, sizeof(h), s) != cudaSuccess) return DSN_ERR_CUDA;  // the report words only
  if (cudaStreamSynchronize(s) != cudaSuccess) return DSN_ERR_CUDA;
  if (code) *code = h[0];
  if (detail) *detail = h[1];
  return DSN_OK;
}

int dsn_set_wait_limit(dsn_ctx* ctx, uint32_t microseconds, void* stream) {
  if (int e = check_ctx(ctx)) return e;
  cudaStream_t s = as_stream(stream);
  // the source of an asynchronous copy must stay valid until the copy has run: wait for an earlier one first
  if (cudaStreamSynchronize(s) != cudaSuccess) return DSN_ERR_CUDA;
  ctx->wait_limit_us = microseconds;
  if (cudaMemcpyAsync(ctx->d_status + DSN_STATUS_WAIT_US, &ctx->wait_limit_us, sizeof(uint32_t), cudaMemcpyHostToDevice,
                      s) != cudaSuccess)
    return DSN_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_map_cache_stats(dsn_ctx* ctx, uint64_t* hits, uint64_t* misses) {
  if (!ctx) return DSN_ERR_INVALID_ARG;
  if (hits) *hits = ctx->map_hits;
  if (misses) *misses = ctx->map_misses;
  return DSN_OK;
}

int dsn_get_stats(dsn_ctx* ctx, dsn_stats* out) {
  if (!ctx || !out) return DSN_ERR_INVALID_ARG;
  ctx->stats.map_hits = ctx->map_hits;
  ctx->stats.map_misses = ctx->map_misses;
  *out = ctx->stats;
  return DSN_OK;
}

int dsn_selftest_bounded_wait(dsn_ctx* ctx, void* stream) {
  if (int e = check_ctx(ctx)) return e;
  return dsn_launch_selftest_wait(ctx->d_status, as_stream(stream)) == cudaSuccess ? DSN_OK : DSN_ERR_CUDA;
}

int dsn_widths_from_ratios(int32_t C, const double* ratios, int32_t T, int32_t granule, int32_t* widths_out) {
  if (C < 1 || !ratios || !widths_out || T < 1 || granule < 0) return DSN_ERR_INVALID_ARG;
  int g = granule;
  if (g == 0) {
    g = C / 32 < 8 ? C / 32 : 8;
    if (g < 1) g = 1;
  }
  for (int t = 0; t < T; ++t) {
    if (!(ratios[t] > 0.0) || ratios[t] > 1.0) return DSN_ERR_INVALID_ARG;
    long k = (long)g * (long)floor(ratios[t] * C / g + 0.5 + 1e-9);
    if (k < g) k = g;
    if (k > C) k = C;
    widths_out[t] = (int32_t)k;
  }
  return DSN_OK;
}

int64_t dsn_executed_macs(const int32_t* counts, int32_t T, int32_t R, const int32_t* k_in, const int32_t* k_out,
                          int32_t K) {
  if (!counts || !k_in || !k_out || T < 1) return -1;
  int64_t total = 0;
  for (int t = 0; t < T; ++t) total += (int64_t)counts[t] * R * k_in[t] * k_out[t] * K * K;
  return total;
}

size_t dsn_gate_workspace_bytes(const dsn_gate_desc* g) {
  if (check_gate(g)) return 0;
  // the split count depends on the SM count; size for the largest count the launcher can pick
  int splits = g->R / 8 > 0 ? g->R / 8 : 1;
  if (splits > 64) splits = 64;
  return align_up(((size_t)g->B * splits * g->c_valid + (size_t)g->B * g->C_mlp) * sizeof(float), 256) + 256;
}

int dsn_gate(dsn_ctx* ctx, const dsn_gate_desc* g, const void* x, int32_t* idx_out, float* logits_out,
             void* workspace, size_t ws_bytes, void* stream) {
  if (!x || !idx_out) return DSN_ERR_INVALID_ARG;
  int e = check_ctx(ctx);
  if (e) return e;
  e = check_gate(g);
  if (e) return e;
  if (g->B == 0) return DSN_OK;
  const int splits = dsn_gate_splits(*g, ctx->sm_count);
  const size_t need = ((size_t)g->B * splits * g->c_valid + (size_t)g->B * g->C_mlp) * sizeof(float);
  if (!workspace || ws_bytes < need) return DSN_ERR_WORKSPACE;
  if (!aligned16(workspace)) return DSN_ERR_ALIGNMENT;
  count_launch(ctx, &dsn_stats::launches_gate, 3);  // pool, hidden layer, scores
  if (dsn_launch_gate(*g, x, idx_out, logits_out, static_cast<float*>(workspace), splits, ctx->d_status,
                      as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_gate_attention(dsn_ctx* ctx, const dsn_gate_desc* g, const float* W3, const float* b3, const void* x,
                       int32_t* idx_out, float* logits_out, float* scale_out, void* workspace, size_t ws_bytes,
                       void* stream) {
  if (!W3 || !scale_out) return DSN_ERR_INVALID_ARG;
  int e = dsn_gate(ctx, g, x, idx_out, logits_out, workspace, ws_bytes, stream);
  if (e) return e;
  if (g->B == 0) return DSN_OK;
  if ((size_t)4 * 4 * g->C_mlp > 48 * 1024) return DSN_ERR_UNSUPPORTED;
  const int splits = dsn_gate_splits(*g, ctx->sm_count);
  const float* hid = static_cast<const float*>(workspace) + (size_t)g->B * splits * g->c_valid;
  count_launch(ctx, &dsn_stats::launches_gate);
  if (dsn_launch_gate_attention(*g, hid, W3, b3, scale_out, as_stream(stream)) != cudaSuccess) return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_scale_channels(dsn_ctx* ctx, const dsn_routing* r, int32_t to_grouped, int32_t dtype, int32_t B, int32_t R,
                       int32_t c_valid, const void* x, int64_t ldx, const float* scale, void* y, int64_t ldy,
                       void* stream) {
  if (!x || !y || !scale || B < 0 || R < 1 || c_valid < 1 || ldx < c_valid || ldy < c_valid)
    return DSN_ERR_INVALID_ARG;
  if (int e = check_ctx(ctx)) return e;
  if (dtype != DSN_BF16 && dtype != DSN_F32) return DSN_ERR_INVALID_ARG;
  const int32_t* perm = nullptr;
  if (to_grouped) {
    if (!r || !r->perm || r->B != B) return DSN_ERR_INVALID_ARG;
    if (x == y) return DSN_ERR_INVALID_ARG;  // a permutation cannot run in place
    perm = r->perm;
  }
  count_launch(ctx, &dsn_stats::launches_copy);
  if (dsn_launch_scale_channels(dtype == DSN_BF16 ? 2 : 4, B, R, c_valid, x, ldx, scale, y, ldy, perm,
                                as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_resbn_fold(dsn_ctx* ctx, int32_t T, int32_t C, const float* gamma, const float* beta, const float* mu,
                   const float* sigma, float* scale_out, float* shift_out, void* stream) {
  if (T < 1 || T > DSN_MAX_SLICES || C < 1 || !gamma || !beta || !mu || !sigma || !scale_out || !shift_out)
    return DSN_ERR_INVALID_ARG;
  if (int e = check_ctx(ctx)) return e;
  count_launch(ctx, &dsn_stats::launches_copy);
  if (dsn_launch_resbn_fold(T * C, C, gamma, beta, mu, sigma, scale_out, shift_out, as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_route(dsn_ctx* ctx, const int32_t* idx, int32_t B, int32_t T, dsn_routing* out, void* stream) {
  if (!idx || !out || B < 0 || T < 1 || T > DSN_MAX_SLICES) return DSN_ERR_INVALID_ARG;
  if (int e = check_ctx(ctx)) return e;
  if (!out->counts || !out->offsets || !out->perm || !out->inv_perm) return DSN_ERR_INVALID_ARG;
  out->B = B;
  out->G = T;
  out->group_slice = nullptr;
  count_launch(ctx, &dsn_stats::launches_route);
  if (dsn_launch_route(idx, B, T, out->counts, out->offsets, out->perm, out->inv_perm, ctx->d_status,
                       as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_permute_rows(dsn_ctx* ctx, const dsn_routing* r, int32_t dtype, int32_t R, int32_t T, const int32_t* k,
                     const void* src, int64_t ld_src, void* dst, int64_t ld_dst, int32_t to_grouped, void* stream) {
  if (!src || !dst || !k || R < 1 || T < 1 || T > DSN_MAX_SLICES) return DSN_ERR_INVALID_ARG;
  if (dtype != DSN_BF16 && dtype != DSN_F32) return DSN_ERR_INVALID_ARG;
  int e = check_ctx(ctx);
  if (e) return e;
  e = check_routing(r, T);
  if (e) return e;
  SliceTable st;
  memset(&st, 0, sizeof(st));
  for (int t = 0; t < T; ++t) {
    if (k[t] < 1 || k[t] > ld_src || k[t] > ld_dst) return DSN_ERR_INVALID_ARG;
    st.k_in[t] = k[t];
  }
  count_launch(ctx, &dsn_stats::launches_copy);
  if (dsn_launch_permute_rows(st, dtype == DSN_BF16 ? 2 : 4, R, src, ld_src, dst, ld_dst, to_grouped ? 1 : 0, r->B,
                              r->G, r->offsets, r->perm, r->group_slice, as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

size_t dsn_linear_workspace_bytes(const dsn_linear_desc* d, int32_t B) {
  (void)d; (void)B;
  return 0;  // the tile schedule is rebuilt inside the kernel from the group offsets
}
size_t dsn_conv_workspace_bytes(const dsn_conv_desc* d, int32_t B) {
  (void)d; (void)B;
  return 0;
}

int dsn_sliced_linear(dsn_ctx* ctx, const dsn_linear_desc* d, const dsn_routing* r, const void* x, void* y,
                      void* workspace, size_t ws_bytes, void* stream) {
  (void)workspace; (void)ws_bytes;
  if (!d || d->R < 1) return DSN_ERR_INVALID_ARG;
  return run_layer(ctx, from_linear(d), r, x, y, as_stream(stream));
}

int dsn_sliced_conv(dsn_ctx* ctx, const dsn_conv_desc* d, const dsn_routing* r, const void* x, void* y,
                    void* workspace, size_t ws_bytes, void* stream) {
  (void)workspace; (void)ws_bytes;
  if (!d) return DSN_ERR_INVALID_ARG;
  if (d->dtype != DSN_BF16) return DSN_ERR_UNSUPPORTED;
  return run_layer(ctx, from_conv(d), r, x, y, as_stream(stream));
}

int dsn_sliced_depthwise(dsn_ctx* ctx, const dsn_depthwise_desc* d, const dsn_routing* r, const void* x, void* y,
                         void* stream) {
  if (!x || !y) return DSN_ERR_INVALID_ARG;
  if (int e0 = check_ctx(ctx)) return e0;
  if (int e1 = check_depthwise(d)) return e1;
  int e = check_routing(r, d->T);
  if (e) return e;
  count_launch(ctx, &dsn_stats::launches_depthwise);
  if (dsn_launch_depthwise(d->c, d->ksize, d->T, d->H, d->W_, d->K, d->stride, d->C, r->B, r->G, r->offsets, r->perm,
                           r->group_slice, d->in_order == DSN_INPUT_ORDER, d->out_order == DSN_INPUT_ORDER, x, d->ldx,
                           d->W, d->bias, d->bn_scale, d->bn_shift, d->act, y, d->ldy, as_stream(stream)) != cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

int dsn_sliced_attention(dsn_ctx* ctx, const dsn_attention_desc* d, const dsn_routing* r, const void* qkv, void* out,
                         void* stream) {
  if (!qkv || !out) return DSN_ERR_INVALID_ARG;
  int e = check_ctx(ctx);
  if (e) return e;
  e = check_attention(d, r, qkv, out);
  if (e) return e;
  if (r->B == 0) return DSN_OK;
  CUtensorMap map;
  // samples are a dimension of their own: a box that runs past the sample's last row reads zeros there
  const uint64_t dims[4] = {64, (uint64_t)3 * d->H, (uint64_t)d->N, (uint64_t)r->B};
  const uint64_t str[3] = {128, (uint64_t)d->ld_qkv * 2, (uint64_t)d->ld_qkv * 2 * (uint64_t)d->N};
  const uint32_t box[4] = {64, 1, 128, 1};
  e = encode_map(ctx, &map, qkv, 4, dims, str, box);
  if (e) return e;
  CUtensorMap map_out;
  const uint64_t od[3] = {(uint64_t)d->H * 64, (uint64_t)d->N, (uint64_t)r->B};
  const uint64_t os[2] = {(uint64_t)d->ld_out * 2, (uint64_t)d->ld_out * 2 * (uint64_t)d->N};
  const uint32_t ob[3] = {64, 32, 1};
  e = encode_map(ctx, &map_out, out, 3, od, os, ob);
  if (e) return e;
  count_launch(ctx, &dsn_stats::launches_attention);
  if (dsn_launch_attention(map, map_out, d->heads, d->T, d->N, d->H, r->B, r->G, d->order == DSN_GROUPED, r->offsets, r->perm,
                           r->group_slice, qkv, d->ld_qkv, out, d->ld_out, ctx->d_status, as_stream(stream)) !=
      cudaSuccess)
    return DSN_ERR_CUDA;
  return DSN_OK;
}

size_t dsn_layer_workspace_bytes(const dsn_layer_desc* L) {
  LayerPlan pl;
  if (plan_layer(L, pl)) return 0;
  return pl.total + 256;
}

int dsn_layer_forward(dsn_ctx* ctx, const dsn_layer_desc* L, const void* x, const int32_t* idx_in, void* y,
                      dsn_routing* r_out, int32_t* idx_out, void* workspace, size_t ws_bytes, void* stream) {
  if (!L || !x || !y) return DSN_ERR_INVALID_ARG;
  int e = check_ctx(ctx);
  if (e) return e;
  ++ctx->stats.calls;
  log_call(ctx, "dsn_layer_forward", L->B, L->T);
  LayerPlan pl;
  e = plan_layer(L, pl);
  if (e) return e;
  if (!L->gate && !idx_in) return DSN_ERR_INVALID_ARG;
  if (L->gate && (L->gate->B != L->B || L->gate->T != L->T)) return DSN_ERR_INVALID_ARG;
  if (!workspace || ws_bytes < pl.total) return DSN_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSN_ERR_ALIGNMENT;
  char* ws = static_cast<char*>(workspace);
  cudaStream_t s = as_stream(stream);

  // validate every layer before the first launch
  LayerCall calls[DSN_MAX_CHAIN];
  dsn_routing r;
  r.B = L->B;
  r.G = L->T;
  r.counts = reinterpret_cast<int32_t*>(ws + pl.off_counts);
  r.offsets = reinterpret_cast<int32_t*>(ws + pl.off_offsets);
  r.perm = reinterpret_cast<int32_t*>(ws + pl.off_perm);
  r.inv_perm = reinterpret_cast<int32_t*>(ws + pl.off_inv);
  r.group_slice = nullptr;
  for (int j = 0; j < L->n_layers; ++j) {
    LayerCall& c = calls[j];
    layer_call_of(L, j, c);
    const bool first = j == 0, last = j + 1 == L->n_layers;
    c.in_order = (first && !pl.gather_first) ? DSN_INPUT_ORDER : DSN_GROUPED;
    c.out_order = last ? DSN_INPUT_ORDER : DSN_GROUPED;
    if (first && pl.gather_first) c.ldx = c.C_in;
    if (!first) c.ldx = calls[j - 1].C_out;
    if (!last) c.ldy = c.C_out;
    const void* in = first ? (pl.gather_first ? (const void*)(ws + pl.off_gather) : x)
                           : (const void*)(ws + pl.off_buf[(j - 1) & 1]);
    void* out = last ? y : (void*)(ws + pl.off_buf[j & 1]);
    if (c.dw) {
      e = (!aligned16(in) || c.ldx % 8) ? DSN_ERR_ALIGNMENT : check_routing(&r, c.T);
    } else if (!c.att) {
      e = validate_call(c, &r, in, out);
    } else {  // the attention core between two layers: dense grouped intermediates
      dsn_attention_desc a = *c.att;
      a.ld_qkv = c.C_in;
      a.ld_out = c.C_out;
      a.order = DSN_GROUPED;
      e = check_attention(&a, &r, in, out);
    }
    if (e) return e;
  }

  const int32_t* idx = idx_in;
  if (L->gate) {
    int32_t* gi = idx_out ? idx_out : reinterpret_cast<int32_t*>(ws + pl.off_idx);
    e = dsn_gate(ctx, L->gate, x, gi, nullptr, ws + pl.off_gate, dsn_gate_workspace_bytes(L->gate), stream);
    if (e) return e;
    idx = gi;
  } else if (idx_out && L->B > 0) {
    if (cudaMemcpyAsync(idx_out, idx_in, 4 * (size_t)L->B, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
      return DSN_ERR_CUDA;
  }
  e = dsn_route(ctx, idx, L->B, L->T, &r, stream);
  if (e) return e;
  if (r_out) *r_out = r;

  if (pl.gather_first) {
    const LayerCall& c0 = calls[0];
    const dsn_linear_desc* dl = L->kind[0] == DSN_LAYER_LINEAR ? static_cast<const dsn_linear_desc*>(L->layer[0]) : nullptr;
    const int64_t ld_src = dl ? dl->ldx : static_cast<const dsn_conv_desc*>(L->layer[0])->ldx;
    e = dsn_permute_rows(ctx, &r, c0.dtype, c0.H * c0.W, c0.T, c0.k_in, x, ld_src, ws + pl.off_gather, c0.C_in, 1,
                         stream);
    if (e) return e;
  }
  if (!pl.gather_first && L->B > 0) {
    const void* ins[DSN_MAX_CHAIN];
    void* outs[DSN_MAX_CHAIN];
    for (int j = 0; j < L->n_layers; ++j) {
      ins[j] = j == 0 ? x : (const void*)(ws + pl.off_buf[(j - 1) & 1]);
      outs[j] = j + 1 == L->n_layers ? y : (void*)(ws + pl.off_buf[j & 1]);
    }
    e = try_run_chain(ctx, calls, L->n_layers, &r, ins, outs, s);
    if (e < 0) return e;
    if (e == 1) return DSN_OK;
  }
  for (int j = 0; j < L->n_layers; ++j) {
    const bool first = j == 0, last = j + 1 == L->n_layers;
    const void* in = first ? (pl.gather_first ? (const void*)(ws + pl.off_gather) : x)
                           : (const void*)(ws + pl.off_buf[(j - 1) & 1]);
    void* out = last ? y : (void*)(ws + pl.off_buf[j & 1]);
    if (calls[j].dw) {
      if (L->B > 0 && ctx->dwpw_fused && dwpw_fusable(calls[j], calls[j + 1], in)) {
        // the separable block as one kernel: the depthwise result goes from registers to the tensor core's operand tile
        void* out2 = j + 2 == L->n_layers ? y : (void*)(ws + pl.off_buf[(j + 1) & 1]);
        e = run_dwpw(ctx, calls[j], calls[j + 1], &r, in, out2, s);
        ++j;
      } else {
        dsn_depthwise_desc d2 = *calls[j].dw;
        d2.in_order = calls[j].in_order;
        d2.out_order = DSN_GROUPED;
        d2.ldx = calls[j].ldx;
        d2.ldy = calls[j].C_out;
        e = dsn_sliced_depthwise(ctx, &d2, &r, in, out, stream);
      }
    } else if (calls[j].att) {
      dsn_attention_desc a = *calls[j].att;
      a.ld_qkv = calls[j].C_in;   // dense grouped intermediates
      a.ld_out = calls[j].C_out;
      a.order = DSN_GROUPED;
      e = dsn_sliced_attention(ctx, &a, &r, in, out, stream);
    } else {
      e = run_layer(ctx, calls[j], &r, in, out, s);
    }
    if (e) return e;
  }
  return DSN_OK;
}

}  // extern "C"
