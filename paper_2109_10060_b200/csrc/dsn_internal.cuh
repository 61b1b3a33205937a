// Internal declarations shared by the translation units of libdsn (never installed).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dsn.h"

// Device status word: [0] = first condition code, [1] = detail, [2] = count of non-finite gate
// scores, [3] = count of out-of-range routing indices.  These four are read and cleared by dsn_get_status();
// word [4] holds the limit of the kernels' bounded waits in microseconds (0 = the 2 s default).
#define DSN_STATUS_WORDS 8
#define DSN_STATUS_REPORT_WORDS 4
#define DSN_STATUS_WAIT_US 4

// Tensor-map cache: encoding a map on the host costs about a microsecond and a layer needs up to three per distinct
// slice, on every call.  Maps depend only on (base pointer, extents, strides, box), so a context keeps the ones it
// has built in a small direct-mapped table; serving loops that call with the same buffers hit it every time.
#define DSN_MAP_CACHE_SLOTS 512
struct dsn_map_key {
  const void* base;
  uint64_t dims[4];
  uint64_t strides[3];
  uint32_t box[4];
  uint32_t rank;
};
struct dsn_map_slot {
  dsn_map_key key;
  CUtensorMap map;
  int used;
};

struct dsn_ctx {
  int device;
  int sm_count;
  int32_t* d_status;   // DSN_STATUS_WORDS ints
  void* encode_tiled;  // cuTensorMapEncodeTiled entry point
  int gemm_mode;       // 0 = CTA pairs where possible (default), 1 = one CTA per tile (DSN_GEMM_MODE=1cta)
  int halo_sched;      // staged 3x3 tiles: 1 = dealt out round-robin (DSN_HALO_SCHED=strided), else one time-balanced range per pair
  int conv_halo;       // 1 = 3x3 layers stage the input tile once with its halo (default), 0 = one load per tap (DSN_CONV3X3=taps)
  int chain_mode;      // 1 = small-batch chains of sliced layers run as one launch (default), 0 = one launch per layer (DSN_CHAIN=0)
  int chain_fuse;      // 1 = in a chained launch the last 1x1 layer reads the layer before from tensor memory (DSN_CHAIN_FUSE=1; default 0: measured slower)
  int dwpw_fused;      // 1 = depthwise + following 1x1 layer as one kernel (DSN_DWPW=fused); default 0: measured slower than the
                       //     two launches, because four producer warps on plain ALUs cannot keep up with the tensor core
  int pair_clusters[3];  // resident CTA pairs for BN = 64, 128, 256 (-1 = not queried yet)
  dsn_map_slot* map_cache;   // DSN_MAP_CACHE_SLOTS slots (host memory), or nullptr when the cache is off (DSN_MAP_CACHE=0)
  uint64_t map_hits, map_misses;
  dsn_stats stats;           // launch counters (dsn_get_stats)
  int log;                   // 1: DSN_LOG=1
  uint32_t wait_limit_us;  // staging copy of the wait limit (source of the asynchronous copy into the status block)
};

// Launches a one-CTA kernel that waits on a barrier nobody arrives at (the self-test of the bounded waits).
cudaError_t dsn_launch_selftest_wait(int32_t* status, cudaStream_t s);

// Programmatic dependent launch: a kernel may be scheduled while its predecessor in the stream is
// still draining.  Every kernel of this library therefore calls dsn_grid_dependency_wait() before its
// first access to global memory (it returns once the predecessor grid has completed and its writes
// are visible; the predecessors of that grid completed before it passed its own wait), and
// dsn_grid_launch_dependents() right after, which lets the next kernel's CTAs start their set-up on
// SMs that this grid has already left.
__device__ __forceinline__ void dsn_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dsn_grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

int dsn_pdl_enabled();  // 1 unless the environment says DSN_PDL=0

template <typename... KArgs, typename... Args>
inline cudaError_t dsn_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              int cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (dsn_pdl_enabled()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = (unsigned)n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The dynamic shared-memory limit of a kernel is a per-device attribute: it is raised once per (kernel form,
// device), with the launching thread's current device (the context's device: every entry point checks that).
#define DSN_MAX_DEVICES 64
template <typename K>
inline cudaError_t dsn_ensure_dynamic_smem(K kernel, size_t bytes, size_t* per_device /* [DSN_MAX_DEVICES] */) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= DSN_MAX_DEVICES) return cudaErrorInvalidDevice;
  if (bytes > per_device[dev]) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    per_device[dev] = bytes;
  }
  return cudaSuccess;
}

__device__ __forceinline__ void dsn_set_status(int32_t* status, int code, int detail) {
  if (status && atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// ----------------------------------------------------------------------------------------------
// Grouped GEMM parameters (bf16, tcgen05).  One launch covers every group whose slice has a
// tensor-map pair in this launch (map_id != 0xFF); one pair per distinct (k_in, k_out).
// ----------------------------------------------------------------------------------------------
#define DSN_GEMM_MAX_MAPS 16
#define DSN_GEMM_BM 128
#define DSN_GEMM_BK 64

struct GemmGeom {
  // activation tensor seen as [Bdim][H][W][C]; a linear layer is H = 1 (rows along W)
  int32_t H, W;            // "image" extents of one sample (input-order / per-image tiling)
  int32_t R;               // rows per sample = H*W
  int32_t taps, KW, pad;   // taps = K*K
  int32_t bw, bh, nb;      // A box = bw x bh pixels x nb images  (bw*bh*nb <= 128)
  int32_t tiles_x, tiles_y;
  int32_t flat;            // 1: grouped rows tiled without regard to sample boundaries
  int32_t a_input_order;   // A read by sample index perm[p] (needs nb == 1, flat == 0)
  int32_t y_input_order;   // rows scattered to sample perm[p]
  int32_t BN;              // n-tile (64, 128, 256) = rows of the weight box
  int32_t stages;
  int32_t pair;            // 1: tiles are owned by CTA pairs (256 rows), weight box holds BN/2 rows
  int32_t a_slots;         // halo form: depth of the activation ring
  int32_t tps;             // halo form: taps per weight-ring slot (9: all taps of a chunk in one slot, 1: a slot per tap)
  int32_t halo;            // 1: 3x3 layer with the input tile staged once with its halo: bw = W + 2 is the M-row
                           //    pitch, the activation box holds (W + 2) x (bh + 2) pixels, taps are descriptor shifts
  int32_t ranges;          // halo form: 1 = every pair works on one contiguous, cost-balanced range of the tile sequence
};

// Shared-memory bytes of one activation block of the halo form: the box itself, and at least the rows
// the last tap's view of 128 M rows reaches (128 + 2 (W + 2) + 2), rounded to the swizzle period.
__host__ __device__ inline uint32_t dsn_halo_slot_bytes(int wp, int bh) {
  const int box = wp * (bh + 2), reach = 128 + 2 * wp + 2;
  const uint32_t rows = (uint32_t)(box > reach ? box : reach);
  return (rows * 128u + 1023u) & ~1023u;
}

struct GemmParams {
  CUtensorMap mapA[DSN_GEMM_MAX_MAPS];
  CUtensorMap mapB[DSN_GEMM_MAX_MAPS];
  CUtensorMap mapY[DSN_GEMM_MAX_MAPS];  // output rows x k_out columns, 64 x 32 box, for the epilogue's TMA stores (staged 3x3 tiles: channel, x, y, sample)
  int16_t k_in[DSN_MAX_SLICES];
  int16_t k_out[DSN_MAX_SLICES];
  uint8_t map_id[DSN_MAX_SLICES];
  GemmGeom g;
  int32_t B, G, T;
  const int32_t* offsets;
  const int32_t* perm;
  const int32_t* group_slice;
  __nv_bfloat16* y;
  int64_t ldy;
  const float* bias;
  const float* bn_scale;  // [T][bn_ld] per-path affine of Re-SBN, or nullptr
  const float* bn_shift;
  int32_t bn_ld;
  const __nv_bfloat16* residual;  // laid out like y (same rows, same leading dimension), or nullptr
  int32_t act;
  int32_t* status;
};

// Depthwise k x k fused into the pointwise GEMM that follows it: `g` describes the pointwise layer (flat tiling over
// the grouped output pixels, R = Ho * Wo rows per sample; mapA is unused), the rest the depthwise producer.
struct DwPwParams {
  GemmParams g;
  const __nv_bfloat16* x;   // block input [sample][H][W][ldx], order given by g.g.a_input_order
  int64_t ldx;
  const __nv_bfloat16* w;   // depthwise filter [K][K][C]
  const float* dw_bias;
  const float* dw_bn_scale; // [T][C] or nullptr
  const float* dw_bn_shift;
  int32_t dw_act;
  int32_t H, W, Wo, K, stride, C;
  int8_t ksize[DSN_MAX_SLICES];
};
size_t dsn_dwpw_smem_bytes(int BN, int stages, int G);
cudaError_t dsn_launch_dwpw(const DwPwParams& q, int sm_count, size_t smem_bytes, cudaStream_t s);

// A chain of up to three sliced layers run by one launch (every layer tiled per sample, CTA pairs).
#define DSN_CHAIN_MAX_LAYERS 3
struct DsnChainParams {
  GemmParams L[DSN_CHAIN_MAX_LAYERS];
  int32_t n_layers;
  int32_t stages;   // depth of the operand ring
  int32_t bn_max;   // widest n-tile of the layers: accumulator stride in TMEM, weight half-box of a ring slot
  int32_t fuse_tail;  // 1: the output of layer n_layers - 2 stays in tensor memory as the A operand of the last layer
};

// launchers implemented in the .cu files
size_t dsn_gemm_chain_smem_bytes(int bn_max, int stages, int G);
cudaError_t dsn_launch_gemm_bf16_chain(const DsnChainParams& cp, int clusters, size_t smem_bytes, cudaStream_t s);
size_t dsn_gemm_halo_smem_bytes(int BN, int stages, int tps, int a_slots, int G, int wp, int bh);
cudaError_t dsn_launch_gemm_bf16_halo(const GemmParams& p, int clusters, size_t smem_bytes, cudaStream_t s);
cudaError_t dsn_launch_gemm_bf16(const GemmParams& p, int sm_count, size_t smem_bytes, cudaStream_t s);
size_t dsn_gemm_smem_bytes(int BN, int stages, int G);
cudaError_t dsn_launch_gemm_bf16_pair(const GemmParams& p, int clusters, size_t smem_bytes, cudaStream_t s);
size_t dsn_gemm_pair_smem_bytes(int BN, int stages, int G);
int dsn_gemm_pair_max_clusters(size_t smem_bytes);

cudaError_t dsn_launch_gate(const dsn_gate_desc& g, const void* x, int32_t* idx_out, float* logits_out,
                            float* partial, int splits, int32_t* status, cudaStream_t s);
int dsn_gate_splits(const dsn_gate_desc& g, int sm_count);
// attention head: hid = partial + B*splits*c_valid (written by dsn_launch_gate on the same stream)
cudaError_t dsn_launch_gate_attention(const dsn_gate_desc& g, const float* hid, const float* W3, const float* b3,
                                      float* scale_out, cudaStream_t s);
cudaError_t dsn_launch_scale_channels(int elem_bytes, int B, int R, int c_valid, const void* x, int64_t ldx,
                                      const float* scale, void* y, int64_t ldy, const int32_t* perm_or_null,
                                      cudaStream_t s);
cudaError_t dsn_launch_resbn_fold(int n, int C, const float* gamma, const float* beta, const float* mu,
                                  const float* sigma, float* scale_out, float* shift_out, cudaStream_t s);

cudaError_t dsn_launch_route(const int32_t* idx, int B, int T, int32_t* counts, int32_t* offsets,
                             int32_t* perm, int32_t* inv_perm, int32_t* status, cudaStream_t s);

cudaError_t dsn_launch_attention(const CUtensorMap& map, const CUtensorMap& map_out, const int32_t* heads, int T, int N, int H, int B, int G,
                                 int grouped, const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                 const void* qkv, int64_t ld_qkv, void* out, int64_t ld_out, int32_t* status,
                                 cudaStream_t s);

cudaError_t dsn_launch_depthwise(const int32_t* c, const int32_t* ksize, int T, int H, int W, int K, int stride, int C,
                                 int B, int G, const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                 int x_input_order, int y_input_order, const void* x, int64_t ldx, const void* w,
                                 const float* bias, const float* bn_scale, const float* bn_shift, int act, void* y,
                                 int64_t ldy, cudaStream_t s);

struct SliceTable {
  int32_t k_in[DSN_MAX_SLICES];
  int32_t k_out[DSN_MAX_SLICES];
};

cudaError_t dsn_launch_linear_f32(const SliceTable& st, int T, int R, const float* x, int64_t ldx,
                                  const float* W, int64_t ldw, float* y, int64_t ldy, const float* bias,
                                  const float* bn_scale, const float* bn_shift, int bn_ld, const float* residual, int act, int x_input_order, int y_input_order, int B, int G,
                                  const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                  int sm_count, cudaStream_t s);

cudaError_t dsn_launch_permute_rows(const SliceTable& st, int elem_bytes, int R, const void* src,
                                    int64_t ld_src, void* dst, int64_t ld_dst, int to_grouped, int B, int G,
                                    const int32_t* offsets, const int32_t* perm, const int32_t* group_slice,
                                    cudaStream_t s);

// Zero columns k_out[t] .. C_out-1 of every row (dsn_tail = ZERO).
cudaError_t dsn_launch_zero_tail(const SliceTable& st, int elem_bytes, int R, int C_out, void* y, int64_t ldy,
                                 int y_input_order, int B, int G, const int32_t* offsets, const int32_t* perm,
                                 const int32_t* group_slice, cudaStream_t s);
