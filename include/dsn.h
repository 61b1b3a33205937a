/*
 * dsn.h -- C ABI of the dynamic-weight-slicing inference library (NVIDIA B200, sm_100a).
 *
 * The library runs the batched inference path of DS-Net++ ("Dynamic Weight Slicing"):
 * a per-sample gate picks one of T paths, samples are grouped by path, every group runs a
 * dense contraction against the leading slice W[:k_out, :k_in] of the statically stored
 * full weight, and results return in input order.
 *
 * Conventions
 *   - Every function returns DSN_OK (0) or a negative dsn_status code.  No exceptions, no abort.
 *   - "device" pointers are CUDA device memory of the context's GPU; "host" pointers are
 *     ordinary host memory.  The caller owns every buffer; the library owns only dsn_ctx.
 *     No entry point allocates memory per call unless its comment says so.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *     Errors the host can detect are returned at once and nothing is launched.  Conditions only
 *     the device can detect (routing index out of range, a bounded wait that ran out, non-finite
 *     gate scores) are recorded in a device status word read by dsn_get_status().
 *   - Weights are stored [out][in] (linear) or [out][KH][KW][in] (convolution, "OHWI"),
 *     row-major, and are never modified, copied or repacked.  Activations are [B][R][C]
 *     (tokens) or [B][H][W][C] (channels last); R = H*W.
 *   - Paths are numbered 0..T-1 (the paper numbers them 1..|t|, smallest first).
 */
#ifndef DSN_H
#define DSN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dsn_ctx dsn_ctx;

enum dsn_status {
  DSN_OK = 0,
  DSN_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, k > C, T out of range ...   */
  DSN_ERR_ALIGNMENT = -2,   /* a pointer or leading dimension breaks the stated alignment  */
  DSN_ERR_WORKSPACE = -3,   /* workspace missing or smaller than dsn_*_workspace_bytes      */
  DSN_ERR_UNSUPPORTED = -4, /* a combination this build has no kernel for                  */
  DSN_ERR_BAD_INDEX = -5,   /* (device) a routing index outside [0, T)                     */
  DSN_ERR_CUDA = -6,        /* a CUDA runtime / driver call failed                         */
  DSN_ERR_TIMEOUT = -7,     /* (device) a bounded wait inside a kernel ran out             */
  DSN_ERR_NONFINITE = -8    /* (device) a gate score was NaN or infinite                   */
};

enum dsn_dtype { DSN_F32 = 0, DSN_BF16 = 1 };
/* DSN_ACT_GELU: x/2 (1 + erf(x / sqrt 2)) with erf evaluated as tanh of a fitted odd quintic on the hardware
 * tanh: within 3e-5 (absolute) of the erf form from the fit, below 1e-3 absolute overall at |x| = 4, i.e. a
 * fraction of a bfloat16 rounding step of the output. */
enum dsn_act { DSN_ACT_NONE = 0, DSN_ACT_RELU = 1, DSN_ACT_GELU = 2 };
enum dsn_order { DSN_INPUT_ORDER = 0, DSN_GROUPED = 1 };
enum dsn_tail { DSN_TAIL_UNTOUCHED = 0, DSN_TAIL_ZERO = 1 };
enum dsn_layer_kind { DSN_LAYER_LINEAR = 0, DSN_LAYER_CONV = 1, DSN_LAYER_ATTENTION = 2, DSN_LAYER_DEPTHWISE = 3 };

#define DSN_MAX_SLICES 64   /* largest T                                               */
#define DSN_MAX_GROUPS 4096 /* largest G of a caller-built group list                  */
#define DSN_MAX_CHAIN 6     /* layers per dsn_layer_forward call (a ViT block: QKV, attention, proj, fc1, fc2) */

/* Batch grouping (not in the paper, which defines only per-sample behaviour, Eq. (dyn_net):
 * every input runs the path its own gate picks).  Grouped position p holds sample perm[p];
 * group g occupies positions offsets[g] .. offsets[g+1]-1 and uses slice group_slice[g]
 * (slice g when group_slice is NULL).  dsn_route() fills it with G = T; a caller may instead
 * build any list of G <= DSN_MAX_GROUPS groups, several of which may share a slice.
 * All five arrays are device memory. */
typedef struct dsn_routing {
  int32_t B;                  /* samples                                                 */
  int32_t G;                  /* groups                                                  */
  int32_t* counts;            /* [G]                                                     */
  int32_t* offsets;           /* [G+1], exclusive prefix sum of counts                   */
  int32_t* perm;              /* [B]                                                     */
  int32_t* inv_perm;          /* [B], inv_perm[perm[p]] = p                              */
  const int32_t* group_slice; /* [G] or NULL                                             */
} dsn_routing;

/* Gate routing head (Sec. 3.5): X_E = mean over the R positions; scores = W2 ReLU(W1 X_E);
 * index = first position of the maximum score. */
typedef struct dsn_gate_desc {
  int32_t dtype;   /* dtype of x: DSN_BF16 or DSN_F32                                    */
  int32_t B, R;    /* samples, positions per sample                                      */
  int32_t C_full;  /* columns of W1                                                      */
  int32_t c_valid; /* leading channels of x that are read (elastic input), <= C_full     */
  int32_t C_mlp;   /* hidden width                                                       */
  int32_t T;       /* number of paths, 1..DSN_MAX_SLICES                                 */
  int64_t ldx;     /* elements between consecutive positions of x, >= c_valid            */
  const float* W1; /* device [C_mlp][C_full] fp32                                        */
  const float* b1; /* device [C_mlp] or NULL                                             */
  const float* W2; /* device [T][C_mlp] fp32                                             */
  const float* b2; /* device [T] or NULL                                                 */
} dsn_gate_desc;

/* Sliced linear layer (Eq. (weight_slicing); ViT forms in Sec. 3.4):
 * y[i][r][o] = act(bias[o] + sum_{c < k_in[t]} x[i][r][c] * W[o][c]),  o < k_out[t],  t = path of i. */
typedef struct dsn_linear_desc {
  int32_t dtype;        /* DSN_BF16 (x, W, y bf16; fp32 accumulate) or DSN_F32 (all fp32, plain FMA) */
  int32_t R;            /* rows per sample                                               */
  int32_t C_in, C_out;  /* full extents                                                  */
  int64_t ldx, ldw, ldy;/* elements between rows of x, W, y.  bf16: multiples of 8       */
  int32_t T;
  const int32_t* k_in;  /* host [T], 1..C_in                                             */
  const int32_t* k_out; /* host [T], 1..C_out                                            */
  const void* W;        /* device [C_out][ldw]; bf16: 16-byte aligned                    */
  const float* bias;    /* device [C_out] fp32 or NULL                                   */
  const float* bn_scale;/* device [T][C_out] fp32 or NULL: per-path affine a_t of Re-SBN (dsn_resbn_fold) */
  const float* bn_shift;/* device [T][C_out] fp32 (required with bn_scale): b_t          */
  const void* residual; /* device, same dtype, order and leading dimension as y, or NULL: the skip features of a
                           residual block (Sec. 5, DS-ResNet), added before the activation; may not alias y */
  int32_t act;          /* dsn_act; order of operations: contraction, + bias, * a_t + b_t, + residual, activation */
  int32_t in_order;     /* dsn_order of x: INPUT_ORDER [B][R][ldx] by sample, or GROUPED by position */
  int32_t out_order;    /* dsn_order of y                                                */
  int32_t tail;         /* dsn_tail: columns >= k_out[t] left untouched, or zero-filled up to C_out */
} dsn_linear_desc;

/* Slice-able convolution, filter-number / input-channel slicing (Sec. 3.3):
 * y = W[:k_out, :k_in] * x, cross-correlation, zero padding, stride 1, K = 2*pad+1 in {1, 3}. */
typedef struct dsn_conv_desc {
  int32_t dtype;        /* DSN_BF16 only                                                 */
  int32_t H, W_;        /* spatial size (output = input size)                            */
  int32_t K, pad;       /* kernel size 1 (pad 0) or 3 (pad 1)                            */
  int32_t C_in, C_out;
  int64_t ldx, ldy;     /* elements between pixels of x, y; multiples of 8               */
  int32_t T;
  const int32_t* k_in;  /* host [T]                                                      */
  const int32_t* k_out; /* host [T]                                                      */
  const void* W;        /* device [C_out][K][K][C_in] bf16, dense, 16-byte aligned, C_in % 8 == 0 */
  const float* bias;
  const float* bn_scale;/* as in dsn_linear_desc                                         */
  const float* bn_shift;
  const void* residual; /* as in dsn_linear_desc                                         */
  int32_t act;
  int32_t in_order, out_order, tail;
} dsn_conv_desc;

/* Slice-able depthwise convolution (Sec. 3.3: group convolution whose group count follows the elastic
 * input width; kernel-size slicing = the centred k x k part of the K x K filter; the padding follows
 * the kernel size so that every k gives the same output size).  x [B][H][W][ldx], y [B][Ho][Wo][ldy]
 * channels last with Ho = (H-1)/stride + 1; filter [K][K][C] bf16 (channels last), K odd <= 7.
 * A sample of path t uses channels < c[t] and kernel size ksize[t]. */
typedef struct dsn_depthwise_desc {
  int32_t dtype;         /* DSN_BF16                                                     */
  int32_t H, W_;         /* input size                                                   */
  int32_t K;             /* stored kernel size (odd, <= 7)                               */
  int32_t stride;        /* 1 or 2                                                       */
  int32_t C;             /* full channel count                                           */
  int64_t ldx, ldy;      /* elements between pixels of x, y (>= C)                       */
  int32_t T;
  const int32_t* c;      /* host [T] channels of each path, 1..C                         */
  const int32_t* ksize;  /* host [T] kernel size of each path, odd, <= K                 */
  const void* W;         /* device [K][K][C] bf16                                        */
  const float* bias;     /* device [C] or NULL                                           */
  const float* bn_scale; /* device [T][C] or NULL (dsn_resbn_fold)                       */
  const float* bn_shift;
  int32_t act;
  int32_t in_order, out_order;
} dsn_depthwise_desc;

/* Slimmable self-attention core (Sec. 3.4): A_a = Softmax(Q_a K_a^T / sqrt(D_h)) V_a for the h heads of
 * the sample's path, concatenated.  qkv rows are laid out [head][q|k|v][D_h] (the output of the sliced
 * QKV layer with the head-major fused weight), out rows [head][D_h]; heads >= h are neither read nor
 * written.  qkv and out are both in `order` (all rows of a sample are contiguous either way). */
typedef struct dsn_attention_desc {
  int32_t dtype;        /* DSN_BF16                                                      */
  int32_t N;            /* tokens per sample, 1..256                                     */
  int32_t H, D_h;       /* full head count; head dimension (64)                          */
  int64_t ld_qkv;       /* elements between rows of qkv, >= 3*H*D_h, multiple of 8       */
  int64_t ld_out;       /* elements between rows of out, >= H*D_h, multiple of 8         */
  int32_t T;
  const int32_t* heads; /* host [T]: head count of each path, 1..H                       */
  int32_t order;        /* dsn_order of qkv and out                                      */
} dsn_attention_desc;

/* One dynamic block: optional gate, routing, then up to DSN_MAX_CHAIN layers that all inherit
 * the block's routing (Sec. 5, "inherit the control signal").  Layer j reads layer j-1's output;
 * layer 0 reads x in input order, the last layer writes y in input order; intermediate
 * activations live in the workspace in grouped order. */
typedef struct dsn_layer_desc {
  const dsn_gate_desc* gate;        /* NULL: gate bypassed, idx_in supplies the path of every sample */
  int32_t B;
  int32_t T;
  int32_t n_layers;                 /* 1..DSN_MAX_CHAIN                                  */
  int32_t kind[DSN_MAX_CHAIN];      /* dsn_layer_kind                                    */
  const void* layer[DSN_MAX_CHAIN]; /* dsn_linear_desc*, dsn_conv_desc*, dsn_depthwise_desc* (not as the last element) or
                                       (between two layers) dsn_attention_desc*; order and leading-dimension fields of
                                       chained elements are ignored.  A depthwise element followed by a 1x1 layer whose
                                       k_in equals the depthwise widths (the DS-MBNet separable block, Sec. 3.3) can run
                                       as ONE kernel in which the depthwise result feeds the tensor core from shared
                                       memory and never reaches global memory (DSN_DWPW=fused; bf16, widths and row
                                       pitches multiples of 8); by default the two run one after the other through the
                                       workspace, which is the faster form on this GPU */
} dsn_layer_desc;

/* ---- context ------------------------------------------------------------------------- */
/* Creates a context on CUDA device `device` (allocates a few hundred bytes of device memory
 * for the status word; the only allocation the library ever makes).
 * Environment switches, read here, that select between kernels computing the same results (for
 * comparisons and as fallbacks): DSN_GEMM_MODE=1cta (one CTA per tile instead of CTA pairs),
 * DSN_CHAIN=0 (dsn_layer_forward: one launch per layer even for small batches), DSN_CONV3X3=taps
 * (3x3 layers: one activation load per tap instead of one tile with its halo), DSN_HALO_SCHED=strided
 * (staged 3x3 kernel: tiles dealt out round-robin instead of one time-balanced range per CTA pair), DSN_ATTENTION=items (the
 * attention core with one (sample, head, query half) per CTA pass instead of the warp-specialised form),
 * DSN_DWPW=fused (depthwise + following 1x1 layer as one kernel), DSN_CHAIN_FUSE=1 (chained launch: the last 1x1 layer
 * takes the output of the layer before from tensor memory instead of global memory), DSN_PDL=0 (no programmatic
 * dependent launch).
 * Every later call must be made with `device` as the calling thread's current CUDA device (else
 * DSN_ERR_INVALID_ARG): launches and kernel attributes act on the current device. */
int dsn_create(dsn_ctx** ctx, int device);
int dsn_destroy(dsn_ctx* ctx);
const char* dsn_strerror(int code);
/* Waits for `stream`, returns the first device-detected condition since the last call
 * (code = DSN_OK if none; detail = a count or position) and clears it. */
int dsn_get_status(dsn_ctx* ctx, void* stream, int32_t* code, int32_t* detail);

/* Limit of the bounded waits inside the kernels (every wait on a barrier or counter gives up after this
 * long, records DSN_ERR_TIMEOUT with a position code and lets the kernel return; the context stays usable).
 * microseconds = 0 restores the default of 2 s.  Synchronises `stream`.  (Failure detection; the paper has
 * no counterpart.) */
int dsn_set_wait_limit(dsn_ctx* ctx, uint32_t microseconds, void* stream);
/* Self-test of that mechanism: launches one small kernel that waits, with the library's own wait routine,
 * on a barrier nothing arrives at.  It returns after the wait limit; dsn_get_status() then reports
 * DSN_ERR_TIMEOUT (detail 9001).  Nothing faults and later calls run normally. */
int dsn_selftest_bounded_wait(dsn_ctx* ctx, void* stream);

/* The context keeps the TMA tensor maps it has encoded (keyed by base pointer, extents, strides and box; 512 slots,
 * host memory), so that repeated calls on the same buffers and slices skip the encoding (about a microsecond per
 * map, up to three maps per distinct slice and layer).  A map describes addresses and geometry only, so a hit stays
 * valid for as long as the caller's buffer does.  DSN_MAP_CACHE=0 at dsn_create turns the cache off.
 * Returns the hit and miss counts since the context was created. */
int dsn_map_cache_stats(dsn_ctx* ctx, uint64_t* hits, uint64_t* misses);

/* What a context has launched since it was created (host-side counters; kernels of this library only).  With
 * DSN_LOG=1 in the environment at dsn_create, every sliced-layer and dsn_layer_forward call also writes one line to
 * stderr. */
typedef struct dsn_stats {
  uint64_t calls;                 /* sliced-layer and dsn_layer_forward calls                              */
  uint64_t launches;              /* kernels launched, all families                                        */
  uint64_t launches_gemm_pair;    /* grouped GEMM on CTA pairs                                             */
  uint64_t launches_gemm_halo;    /* 3x3 layers, halo form                                                 */
  uint64_t launches_gemm_chain;   /* a block's layers as one launch                                        */
  uint64_t launches_gemm_one_cta; /* grouped GEMM, one CTA per tile                                        */
  uint64_t launches_linear_f32;
  uint64_t launches_attention;
  uint64_t launches_depthwise;
  uint64_t launches_dwpw;         /* depthwise + pointwise as one kernel                                   */
  uint64_t launches_gate;         /* pooling, hidden layer, scores (3 per gate), attention head            */
  uint64_t launches_route;
  uint64_t launches_copy;         /* gather / scatter, zero fill, channel scaling, Re-SBN folding          */
  uint64_t map_hits, map_misses;  /* tensor-map cache                                                      */
  uint64_t launches_gemm_chain_tmem; /* of launches_gemm_chain: last layer fed from tensor memory          */
} dsn_stats;
int dsn_get_stats(dsn_ctx* ctx, dsn_stats* out);

/* Ratio list -> channel counts (host only).  granule g = 0 picks g = min(8, C/32);
 * k = g*floor(r*C/g + 1/2) clamped to [g, C].  The paper lists channel counts, not a rounding
 * rule; this rule reproduces its DS-MBNet list 224..640 step 32 from ratios 0.35..1.0. */
int dsn_widths_from_ratios(int32_t C, const double* ratios, int32_t T, int32_t granule,
                           int32_t* widths_out /* host [T] */);

/* Multiply-adds the sliced layer executes for a routing histogram (Sec. 4.3, MAdds on the fly):
 * sum_t counts[t] * R * k_in[t] * k_out[t] * K*K.  Host arrays. */
int64_t dsn_executed_macs(const int32_t* counts, int32_t T, int32_t R, const int32_t* k_in,
                          const int32_t* k_out, int32_t K);

/* ---- gate (Sec. 3.5) ------------------------------------------------------------------ */
size_t dsn_gate_workspace_bytes(const dsn_gate_desc* g);
/* x: device [B][R][ldx].  idx_out: device [B].  logits_out: device [B][T] fp32 or NULL.
 * workspace: device, 16-byte aligned, >= dsn_gate_workspace_bytes (partial sums of the pooling). */
int dsn_gate(dsn_ctx* ctx, const dsn_gate_desc* g, const void* x, int32_t* idx_out,
             float* logits_out, void* workspace, size_t ws_bytes, void* stream);

/* The same gate for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience).  Typical such callers: a serving loop that must never enter
 * the CUDA allocator once it is running, a plug-in that is handed only its input and output
 * buffers, code running while the process's memory pool is fully handed out.  The pooling scratch
 * lives in a fixed 4 MiB array inside the library image (every GPU that loads the library keeps it
 * until the process exits), so the call takes no workspace and performs no allocation of any kind.
 *   - Limit: B * (splits * c_valid + C_mlp) <= 1,048,576 floats, where splits (1..64) is the
 *     row-band count the gate picks for this GPU; larger problems return DSN_ERR_WORKSPACE and
 *     launch nothing.  The ResNet-50 and ViT workloads fit (128 samples x (4 splits x 1024 + 128) on a
 *     148-SM GPU, 1024 x (1 x 768 + 128)).
 *   - The context's device must be the current device (else DSN_ERR_INVALID_ARG).
 *   - The first call on a device looks up the array's device address (a synchronous runtime
 *     query); make that first call before starting any stream capture.
 *   - All calls on one GPU share the array and it keeps the previous call's contents.  Nothing has
 *     to start at zero (each call overwrites every value it later reads), but two calls that
 *     overlap on the GPU (different streams, or different contexts of one process) race on it:
 *     keep calls to this entry point ordered on one stream per GPU.
 * Arguments and results are those of dsn_gate. */
int dsn_gate_static(dsn_ctx* ctx, const dsn_gate_desc* g, const void* x, int32_t* idx_out,
                    float* logits_out, void* stream);

/* Double-headed gate (Sec. 3.5): the routing head of dsn_gate plus the channel-attention head that
 * shares W1: scale[i][c] = 1 + tanh(b3[c] + sum_j W3[c][j] * ReLU(W1 X_E + b1)[j]), c < c_valid.
 * W3: device [C_full][C_mlp] fp32, b3: device [C_full] or NULL.  scale_out: device [B][c_valid] fp32.
 * idx_out / logits_out as in dsn_gate (both heads always run).  Workspace as for dsn_gate. */
int dsn_gate_attention(dsn_ctx* ctx, const dsn_gate_desc* g, const float* W3, const float* b3, const void* x,
                       int32_t* idx_out, float* logits_out, float* scale_out, void* workspace, size_t ws_bytes,
                       void* stream);

/* Applies the attention head: y[p or i][r][c] = x[i][r][c] * scale[i][c] for c < c_valid (bf16 or fp32
 * activations, fp32 scale).  With r != NULL and to_grouped = 1 the result is written in grouped
 * order (position p holds sample perm[p]), i.e. the scaling is fused with the gather; otherwise y is
 * in input order.  x and y may be the same buffer when the order does not change. */
int dsn_scale_channels(dsn_ctx* ctx, const dsn_routing* r, int32_t to_grouped, int32_t dtype, int32_t B,
                       int32_t R, int32_t c_valid, const void* x, int64_t ldx, const float* scale, void* y,
                       int64_t ldy, void* stream);

/* Split batch norm with re-calibration (Sec. 3.3): gamma[:c] * (X - mu_t) / sigma_t + beta[:c] with
 * per-route statistics.  At inference it is the per-path per-channel affine a_t = gamma / sigma_t,
 * b_t = beta - gamma * mu_t / sigma_t, which the sliced layers apply in their epilogue
 * (bn_scale / bn_shift).  gamma, beta: device [C]; mu, sigma: device [T][C]; outputs device [T][C]. */
int dsn_resbn_fold(dsn_ctx* ctx, int32_t T, int32_t C, const float* gamma, const float* beta, const float* mu,
                   const float* sigma, float* scale_out, float* shift_out, void* stream);

/* ---- routing (stable grouping by path index; one-hot routing of Sec. 3.1) -------------- */
/* idx: device [B], values in [0, T).  Fills out->counts/offsets/perm/inv_perm (device arrays the
 * caller allocated, G = T, B as given); integer-exact and deterministic.  A value outside
 * [0, T) sets DSN_ERR_BAD_INDEX in the status word; that sample joins no group and the unused
 * tail of perm is set to -1. */
int dsn_route(dsn_ctx* ctx, const int32_t* idx, int32_t B, int32_t T, dsn_routing* out, void* stream);

/* ---- gather / scatter between input order and grouped order ---------------------------- */
/* Copies, for every sample, R rows of the leading k[t] columns (t = its path; k host [T]).
 * to_grouped = 1: dst position p <- src sample perm[p]; 0: dst sample perm[p] <- src position p. */
int dsn_permute_rows(dsn_ctx* ctx, const dsn_routing* r, int32_t dtype, int32_t R, int32_t T,
                     const int32_t* k /* host [T] */, const void* src, int64_t ld_src, void* dst,
                     int64_t ld_dst, int32_t to_grouped, void* stream);

/* ---- sliced layers --------------------------------------------------------------------- */
size_t dsn_linear_workspace_bytes(const dsn_linear_desc* d, int32_t B);
size_t dsn_conv_workspace_bytes(const dsn_conv_desc* d, int32_t B);
/* x, y: device, 16-byte aligned, laid out as d->in_order / d->out_order say.  r: routing of the
 * batch (r->B samples).  workspace may be NULL when the size query returns 0. */
int dsn_sliced_linear(dsn_ctx* ctx, const dsn_linear_desc* d, const dsn_routing* r, const void* x,
                      void* y, void* workspace, size_t ws_bytes, void* stream);
int dsn_sliced_conv(dsn_ctx* ctx, const dsn_conv_desc* d, const dsn_routing* r, const void* x,
                    void* y, void* workspace, size_t ws_bytes, void* stream);

int dsn_sliced_depthwise(dsn_ctx* ctx, const dsn_depthwise_desc* d, const dsn_routing* r, const void* x, void* y,
                         void* stream);

/* qkv, out: device bf16, 16-byte aligned.  fp32 scores and softmax, bf16 probabilities for the
 * second contraction, bf16 output. */
int dsn_sliced_attention(dsn_ctx* ctx, const dsn_attention_desc* d, const dsn_routing* r, const void* qkv,
                         void* out, void* stream);

/* ---- whole dynamic block (Eq. (dyn_net)) ------------------------------------------------ */
size_t dsn_layer_workspace_bytes(const dsn_layer_desc* L);
/* Gate (or the given indices) -> routing -> the block's layers, all layers under the one decision
 * (Sec. 5).  Batches of at most two samples per SM pair whose samples have 150..256 rows (14x14
 * images, 197 tokens) run their 2-3 sliced layers as ONE launch in which every SM pair walks whole
 * samples through the layers (skip features included); otherwise (and whenever the block holds the attention core
 * or a depthwise element) one launch per layer.  The two forms agree to within one bfloat16 rounding step of an
 * output on a few percent of the elements (the 3x3 layer sums its taps in a different order), not bit for bit.
 * x, y in input order.  idx_in: device [B], required when L->gate is NULL, ignored otherwise.
 * r_out (optional): receives pointers into the workspace holding the block's routing arrays
 * (valid until the workspace is reused).  idx_out (optional): device [B], the gate's choice. */
int dsn_layer_forward(dsn_ctx* ctx, const dsn_layer_desc* L, const void* x, const int32_t* idx_in,
                      void* y, dsn_routing* r_out, int32_t* idx_out, void* workspace, size_t ws_bytes,
                      void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DSN_H */
