/*
 * twist.h -- C ABI of the B200-native (sm_100a) hot path of one TwIST training round.
 *
 * One round (paper Sec. 3, overview of the system): sample S structured subnet
 * blueprints (Algorithm 1), gather the kept blocks of every partitioned weight
 * matrix into dense slices (dispatcher, Sec. 3.2), run K local forward/backward
 * SGD steps per subnet on the slices, average every parameter over the subnets
 * that hold it (aggregator, Sec. 3.3), resample.
 *
 * General conventions
 *  - Every function returns a status (TWIST_OK == 0, negative on error), never
 *    throws, never exits.  Except where a function says otherwise it allocates
 *    nothing, does not synchronise, and only enqueues work on `stream`
 *    (a cudaStream_t passed as void*; NULL is the default stream).
 *  - "device" pointers are CUDA device memory owned by the caller; they must stay
 *    valid until the stream has run the call.  "host" pointers are read during the
 *    call only.  Base pointers must be 16-byte aligned (byte masks: 8-byte); a misaligned
 *    pointer returns TWIST_ERR_SHAPE, it is never dereferenced.
 *  - Storage layout: every partitioned matrix is row-major with one row per hidden
 *    neuron / head dimension and d_model contiguous, so that a block -- a run of whole rows --
 *    is one contiguous piece of memory (block definition of Sec. 3.1):
 *        W_gate, W_up, W_down : [F, d];  W_qkv : [(H + 2 H_kv) d_head, d];  W_o : [H d_head, d].
 *    up/gate/qkv rows are output features (y = x W^T), down/o rows are input features (y = h W).
 *    Slices and activations of the S subnets are packed [S][rows][cols], dense.
 *  - dtype TWIST_BF16: weights, stored activations and stored activation gradients are
 *    bf16; products accumulate in fp32; each slice has an fp32 master copy that SGD
 *    updates.  dtype TWIST_FP32: everything is fp32 and the slice is its own master.
 *  - Row widths (d_model, f_sub, a_sub, ...) must be multiples of 8 elements in bf16.
 *  - Kernels that wait on hardware barriers bound every wait; on expiry they record
 *    TWIST_ERR_DEVICE_TIMEOUT in a device status word (read it with twist_device_status)
 *    and return instead of hanging.
 */
#ifndef TWIST_H_
#define TWIST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  TWIST_OK = 0,
  TWIST_ERR_NULL = -1,           /* a required pointer is NULL */
  TWIST_ERR_SHAPE = -2,          /* a size is non-positive, misaligned or inconsistent */
  TWIST_ERR_INFEASIBLE = -3,     /* N_sub violates the size bound of Sec. 3.1 */
  TWIST_ERR_BAD_INDEX = -4,      /* an index array entry is out of range / unsorted */
  TWIST_ERR_UNSUPPORTED = -5,    /* valid request outside what the kernels implement */
  TWIST_ERR_WORKSPACE = -6,      /* workspace missing or too small */
  TWIST_ERR_CUDA = -7,           /* a CUDA runtime/driver call failed (see twist_last_cuda_error) */
  TWIST_ERR_DEVICE_TIMEOUT = -8  /* a bounded device-side wait expired */
};

enum { TWIST_FP32 = 0, TWIST_BF16 = 1 };
enum { TWIST_FFN_RELU = 0, TWIST_FFN_GELU = 1, TWIST_FFN_SWIGLU = 2 };
enum { TWIST_MODE_COVER = 0, TWIST_MODE_IID = 1 };
enum { TWIST_KIND_FFN = 0, TWIST_KIND_HEAD = 1 };
enum { TWIST_PROJ_QKV = 0, TWIST_PROJ_O = 1 };

#define TWIST_MAX_SUBNETS 32
#define TWIST_MAX_BLOCKS 16384   /* blocks per layer and kind the sampler kernel handles */
#define TWIST_MAX_COMMON 256     /* common blocks |C| per layer and kind */

/* ---------------------------------------------------------------------------------------------
 * twist_plan -- the shapes of one workload plus a cache of encoded TMA tensor maps (the paper has no counterpart:
 * it is plumbing of this implementation).  The grouped GEMM and attention kernels address their operands through
 * tensor maps that the host encodes from (base address, dimensions, box).  Calls that carry a plan
 * (the `plan` field of their argument struct) look each map up in the plan's cache first, so a training loop that
 * passes the same buffers every step encodes nothing after its first step.  A cached map never goes stale: it
 * is a pure function of its key.  Calls without a plan (plan == NULL) encode their maps every time; both forms
 * compute the same thing.
 *  - twist_plan_create validates the configuration (TWIST_ERR_SHAPE / _INFEASIBLE / _UNSUPPORTED) and allocates
 *    host memory only; the plan is owned by the caller and freed with twist_plan_destroy, after which no call may
 *    carry it.  A plan may be shared by host threads (its cache is locked).
 *  - twist_workspace_bytes: device scratch that covers every scratch argument (loss_ws, the stand-alone loss's
 *    ws, the layer normalisation's ws) of the local-step calls of this workload -- partitioned or shared layers,
 *    gathered or masked workers.
 *  - twist_plan_stats: maps cached, cache hits and misses so far (any pointer may be NULL). */
typedef struct twist_plan twist_plan;
typedef struct {
  uint32_t struct_size;       /* sizeof(twist_config): versions the struct */
  int32_t n_layers, d_model, n_heads /* 0: no attention blocks */, n_kv_heads, d_head, d_ff;
  int32_t ffn_kind;           /* TWIST_FFN_* */
  int32_t n_subnets;          /* S */
  int32_t ffn_block;          /* neurons per FFN block (Sec. 3.1: d_inner / R) */
  int32_t ffn_keep, head_keep;   /* N_sub per kind, in blocks */
  int32_t sample_mode;        /* TWIST_MODE_* */
  int32_t dtype;              /* TWIST_FP32 / TWIST_BF16 */
  int32_t tokens;             /* T: tokens per subnet and local step */
  int32_t reserved;
  uint64_t seed;
} twist_config;
int32_t twist_plan_create(const twist_config* cfg /*host*/, twist_plan** out);
int32_t twist_plan_destroy(twist_plan* plan);
int32_t twist_workspace_bytes(const twist_plan* plan, size_t* bytes);
int32_t twist_plan_stats(twist_plan* plan, uint64_t* cached, uint64_t* hits, uint64_t* misses);

uint32_t twist_abi_version(void);
const char* twist_strerror(int32_t status);
/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char* twist_last_cuda_error(void);
/* Reads (and clears) the device status word.  Synchronises the device.  *code is TWIST_OK,
 * TWIST_ERR_DEVICE_TIMEOUT (a bounded wait of a kernel ran out) or TWIST_ERR_BAD_INDEX (a kernel met an
 * index entry outside its range and skipped it); the time-out wins when both happened. */
int32_t twist_device_status(int32_t* code);
/* Self-test of the give-up path of the kernels' bounded waits (the paper has no counterpart; for tests and
 * bring-up).  Launches one CTA pair with the roles, barriers and exit sequence of the GEMM kernel whose
 * barriers nobody arrives at; every wait gives up after limit_ns (1 .. 100 000 000) of wall time, the pair
 * drains, frees its tensor memory and returns.  Afterwards twist_device_status reports
 * TWIST_ERR_DEVICE_TIMEOUT once, and the device stays usable. */
int32_t twist_selftest_wait(uint64_t limit_ns, void* stream);

/* ---------------------------------------------------------------------------------------------
 * twist_sample_masks -- subnet generator, Algorithm 1 ("Generate Training Subnet Blueprint").
 *
 * For each of n_layers consecutive layers (layer_begin ...) and one block kind, builds the
 * blueprint A [S][n_sub] (rows sorted ascending):  common blocks C, then a seeded random
 * order of the non-common blocks dealt round-robin to the subnets (every block is held at
 * least once), then each subnet fills up to n_sub with distinct random blocks it lacks, then
 * sort.  TWIST_MODE_IID skips the round-robin deal (independent random subnets; used where
 * n_sub is below the bound of Sec. 3.1).  Random draws are a counter-based 64-bit hash of
 * (seed, round, layer, kind, stream, subnet, block); results are a pure function of those.
 * Also writes the index data the aggregator (Sec. 3.3) needs: cover[l][b] = bitmask of the
 * subnets holding block b, pos[l][s][b] = rank of b in A[s] or -1.
 *
 *  common      host, n_common sorted distinct block ids (may be NULL when n_common == 0)
 *  idx         device out, int32 [n_layers][S][n_sub]
 *  cover       device out, uint32 [n_layers][n_full]
 *  pos         device out, int32 [n_layers][S][n_full]
 * Errors: INFEASIBLE when (n_full + (S-1)|C|)/S <= n_sub <= n_full fails in COVER mode (IID
 * needs |C| <= n_sub <= n_full); UNSUPPORTED when n_full > TWIST_MAX_BLOCKS, S > 32 or
 * n_common > TWIST_MAX_COMMON; BAD_INDEX when `common` is unsorted or out of range.
 */
int32_t twist_sample_masks(uint64_t seed, uint64_t round, int32_t layer_begin, int32_t n_layers, int32_t kind,
                           int32_t n_full, int32_t n_subnets, int32_t n_sub,
                           const int32_t* common, int32_t n_common, int32_t sample_mode,
                           int32_t* idx, uint32_t* cover, int32_t* pos, void* stream);

/* Activation masks of Masked / Hybrid TwIST (Sec. 4.1) from the aggregator's cover masks: for the subnets
 * subnet_begin .. subnet_begin + n_subnets - 1,  mask[s][b*block_rows + i] = 1 if subnet s holds block b, else 0.
 *   cover [n_full] device uint32 (one layer);  mask [n_subnets][n_full*block_rows] device uint8: out. */
int32_t twist_hidden_mask(const uint32_t* cover /*device*/, int32_t n_full, int32_t block_rows, int32_t subnet_begin,
                          int32_t n_subnets, uint8_t* mask /*device*/, void* stream);

/* KV groups under grouped-query attention (an extension; the paper's attention is plain
 * multi-head, App. A): group g = h / (n_heads / n_kv_heads) is held by subnet s iff one of its
 * query heads is.  Writes kv_idx [n_layers][S][n_kv_heads] (sorted kept groups, then -1),
 * kv_count [n_layers][S], kv_cols [n_layers][S] = kv_count * d_head (valid K or V columns of the
 * subnet's projection), kv_cover [n_layers][n_kv_heads], kv_pos [n_layers][S][n_kv_heads]; all device. */
/* Column mask of a masked worker's full-width QKV projection (Sec. 4.1) from the aggregator's cover masks:
 * for subnets subnet_begin .. +n_subnets-1, mask[s][c] = 1 iff column c of [Q heads | K groups | V groups] belongs to
 * a head (head_cover, uint32 [n_heads]) or KV group (kv_cover, uint32 [n_kv_heads]) the subnet holds;
 * count[s] = number of marked columns.  mask [n_subnets][(n_heads + 2 n_kv_heads) d_head] uint8, count [n_subnets]
 * int32; all device, one layer. */
int32_t twist_qkv_col_mask(const uint32_t* head_cover, const uint32_t* kv_cover, int32_t n_heads, int32_t n_kv_heads,
                           int32_t d_head, int32_t subnet_begin, int32_t n_subnets, uint8_t* mask, int32_t* count,
                           void* stream);

/* Head mask on the attention core's output (Sec. 4.1: the module output is multiplied element-wise by the mask):
 * out[s][t][c] = mask[s][c] ? in[s][t][c] : 0 for bf16 activations [S][T][width] and a uint8 mask [S][width]
 * (width a multiple of 8; in == out allowed).  All device. */
int32_t twist_apply_col_mask(const void* in, const uint8_t* mask, void* out, int32_t n_subnets, int32_t tokens,
                             int32_t width, void* stream);

int32_t twist_kv_groups(const int32_t* head_idx, int32_t n_layers, int32_t n_subnets, int32_t head_keep,
                        int32_t n_heads, int32_t n_kv_heads, int32_t d_head, int32_t* kv_idx, int32_t* kv_count,
                        int32_t* kv_cols, uint32_t* kv_cover, int32_t* kv_pos, void* stream);

/* ---------------------------------------------------------------------------------------------
 * twist_gather_subnets -- dispatcher, Sec. 3.2: the kept blocks of a matrix are concatenated
 * into one dense sub-matrix per subnet.
 *
 * One call moves up to TWIST_MAX_SEGMENTS row ranges ("segments", e.g. gate, up, down, Q, K, V,
 * O of one layer) in a single launch.  For segment g, subnet s, kept entry j < n_keep and
 * i < block_rows:
 *   dst[s*dst_subnet_stride + (dst_row_offset + j*block_rows + i)*d + :]
 *       = src[(src_row_offset + idx[s*idx_stride + j]*block_rows + i)*d + :]
 * (bit copy); the same values widened to fp32 go to dst_master when it is not NULL.  Entries
 * j >= count[s] (count may be NULL = all valid) are written as zeros (padding of ragged KV rows).
 * Index data is checked on the device: a valid entry idx[..] outside [0, n_blocks) is not followed -- its
 * destination rows are left untouched and TWIST_ERR_BAD_INDEX is recorded in the device status word
 * (twist_device_status); the other rows are gathered as usual.
 */
#define TWIST_MAX_SEGMENTS 8
typedef struct {
  const void* src;            /* device, full matrix [rows_full][d] in `dtype` */
  void* dst;                  /* device, slices in `dtype` */
  float* dst_master;          /* device fp32 copy of dst (same geometry) or NULL */
  const int32_t* idx;         /* device int32 [S][idx_stride], kept block ids */
  const int32_t* count;       /* device int32 [S] valid entries per subnet, or NULL */
  int32_t idx_stride;
  int32_t n_keep;             /* entries written per subnet */
  int32_t block_rows;         /* rows per block */
  int32_t n_blocks;           /* blocks in the partitioned range of src: every idx entry must lie in [0, n_blocks) */
  int64_t src_row_offset;     /* first row of the partitioned range inside src */
  int64_t dst_subnet_stride;  /* elements between consecutive subnets in dst / dst_master */
  int64_t dst_row_offset;     /* first destination row inside a subnet's slice */
} twist_gather_segment;

int32_t twist_gather_subnets(const twist_gather_segment* segs /*host*/, int32_t n_segs, int32_t n_subnets,
                             int32_t d, int32_t dtype, void* stream);

/* ---------------------------------------------------------------------------------------------
 * twist_aggregate -- aggregator, Sec. 3.3:  p <- sum_i p_i 1[p in W_i] / sum_i 1[p in W_i].
 *
 * For every block b of a segment whose cover mask (restricted to live_subnets) is non-zero,
 * each of its rows becomes the fp32 sum, in ascending subnet order, of the subnets' master rows
 * divided (IEEE division) by the number of subnets summed.  The result is written to dst_f32
 * (if not NULL) and, rounded to nearest-even, to dst (bf16 dtype) -- the copy the next gather
 * reads.  Blocks held by no live subnet are neither read nor written.  One writer per row, fixed
 * order, no atomics: results are deterministic.
 *   src (subnet s, block b at rank pos[s][b]) row i:
 *       sub[s*sub_subnet_stride + (sub_row_offset + pos[s*n_full + b]*block_rows + i)*d + :]
 * Index data is checked on the device: when cover says subnet s holds block b but pos[s][b] is outside
 * [0, n_keep), the block's rows are left untouched and TWIST_ERR_BAD_INDEX is recorded in the device
 * status word; the other rows are aggregated as usual.
 */
typedef struct {
  void* dst;                  /* device, full matrix in `dtype` (bf16: rounded shadow; fp32: the result) */
  float* dst_f32;             /* device fp32 full-precision result (bf16 dtype only), may be NULL */
  const float* sub;           /* device fp32 slices (masters in bf16 dtype, the slices in fp32 dtype) */
  const uint32_t* cover;      /* device uint32 [n_full] */
  const int32_t* pos;         /* device int32 [S][n_full] */
  int32_t n_full;             /* blocks in this segment */
  int32_t block_rows;
  int64_t dst_row_offset;     /* first row of the partitioned range inside dst */
  int64_t sub_subnet_stride;  /* elements between subnets in sub */
  int64_t sub_row_offset;     /* first row of this segment inside a subnet's slice */
  /* Hybrid TwIST (Sec. 4.1): the worker `central_subnet` trained its blocks in place on a full-width fp32
   * matrix under an activation mask instead of on a slice; its row for (block b, row i) is
   * central[(dst_row_offset + b*block_rows + i)*d + :].  central may be dst_f32 itself (every element is read
   * before it is written, by the same thread).  NULL: every subnet is read from `sub`. */
  const float* central;
  int32_t central_subnet;
  int32_t n_keep;             /* blocks of this segment in a subnet's slice: pos of a held block must lie in [0, n_keep) */
} twist_aggregate_segment;

int32_t twist_aggregate(const twist_aggregate_segment* segs /*host*/, int32_t n_segs, int32_t n_subnets,
                        int32_t d, int32_t dtype, uint32_t live_subnets, void* stream);

/* The aggregator in two halves, for subnets spread over several GPUs (Sec. 3.3; the server of Sec. 4.1 receives the
 * workers' parameters and averages them).  Every GPU holds the whole model, the blueprints of all S subnets (the
 * sampler is a pure function of the seed) and the slices of its own subnets subnet_begin .. subnet_begin +
 * n_subnets - 1.
 *   twist_aggregate_partial: for every block of a segment, each row of dst_f32 (fp32 dtype: of dst) becomes the fp32
 *     sum, in ascending subnet order, of the rows of this GPU's live holders -- zeros where it has none.  `sub` and
 *     `pos` hold only this GPU's subnets (numbered from 0), `cover` and live_subnets number the subnets globally.
 *     dst_f32 (dst) is the GPU's partial-sum buffer, in the geometry of the full matrix; the bf16 dst is not written.
 *     `central` must be NULL.
 *   (the caller then adds the partial-sum buffers of all GPUs up, e.g. with an NCCL all-reduce)
 *   twist_aggregate_finish: `central` holds the reduced sums (full-matrix geometry, like the Hybrid worker's matrix);
 *     every row of a block held by c > 0 live subnets (of all n_subnets = S) becomes central_row / c (IEEE
 *     division), written to dst_f32 (if not NULL; it may be `central` itself) and, rounded, to dst; blocks held by
 *     none are left untouched.  `sub` and `pos` are not read.
 * The sum over GPUs is associated differently from twist_aggregate's single running sum, so the two agree to fp32
 * rounding of count additions, not bit for bit; with one GPU (subnet_begin 0, all S subnets) they are bit-identical.
 * Status codes and index checks as for twist_aggregate. */
int32_t twist_aggregate_partial(const twist_aggregate_segment* segs /*host*/, int32_t n_segs, int32_t n_subnets,
                                int32_t subnet_begin, int32_t d, int32_t dtype, uint32_t live_subnets, void* stream);
int32_t twist_aggregate_finish(const twist_aggregate_segment* segs /*host*/, int32_t n_segs, int32_t n_subnets,
                               int32_t d, int32_t dtype, uint32_t live_subnets, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Local training on the dense slices (workers of Sec. 4.1 "True TwIST"; FFN of App. A:
 * y = C relu(W x); the GELU and SwiGLU variants are the workloads').  All S subnets run in one
 * grouped launch per contraction.  out_scale is the activation-shift correction sqrt(N_full/N_sub)
 * of Sec. 3.4 (pass 1 to disable it).
 *
 * twist_subnet_ffn_fwd:
 *   MLP:    pre = X W_up^T;                 hh = act(pre);               Y = out_scale * hh W_down
 *   SwiGLU: pre = [X W_gate^T | X W_up^T];  hh = silu(G) * U;            Y = out_scale * hh W_down
 * twist_subnet_ffn_bwd (exact chain rule):
 *   dHh = out_scale * dY W_down^T;  dpre = dHh * act'(pre)  (SwiGLU: dG = dHh U silu'(G), dU = dHh silu(G));
 *   dX = dpre W_gu;  dW_gu = dpre^T X;  dW_down = out_scale * hh^T dY;
 *   if lr != 0:  master -= lr * dW (fp32), compute copy = round(master)   [plain SGD]
 */
/* Optimiser of the fused weight update.  TWIST_OPT_SGD (the zero-initialised default): w <- w - lr dW.
 * TWIST_OPT_ADAM (the optimiser of the paper's experiments, Sec. 5 Setup; bf16 dtype only), in its standard form:
 *   m <- beta1 m + (1 - beta1) g;  v <- beta2 v + (1 - beta2) g^2;
 *   w <- w - lr (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps),   step = 1, 2, ... within a round.
 * The moments are fp32 arrays shaped like the masters, owned by the caller; they belong to the worker's copy of
 * the slice: zero them when the slices are gathered (the paper exchanges parameters only, never optimiser state). */
enum { TWIST_OPT_SGD = 0, TWIST_OPT_ADAM = 1 };
typedef struct {
  int32_t kind, step;
  float beta1, beta2, eps;
} twist_optimizer;

typedef struct {
  int32_t ffn_kind, dtype, n_subnets, tokens, d_model, f_sub;
  float out_scale, lr;
  const void* x;        /* device [S][T][d] */
  void* w_gu;           /* device [S][g*f_sub][d], g = 2 (SwiGLU: gate rows then up rows) or 1 */
  void* w_down;         /* device [S][f_sub][d] */
  float* w_gu_master;   /* device fp32 masters (bf16 dtype, bwd only) */
  float* w_down_master;
  void* pre;            /* device [S][T][g*f_sub]  fwd: out, bwd: in */
  void* hh;             /* device [S][T][f_sub]    fwd: out, bwd: in */
  void* y;              /* device [S][T][d]        fwd: out (may be NULL with fused loss, bf16 dtype) */
  const void* dy;       /* device [S][T][d]        bwd: in (written by a forward call with fused loss) */
  void* dpre;           /* device [S][T][g*f_sub]  bwd: out (gradient w.r.t. pre) */
  void* dx;             /* device [S][T][d]        bwd: out, may be NULL */
  float* dw_gu;         /* device fp32 [S][g*f_sub][d] gradient dump, may be NULL (required in fp32 dtype) */
  float* dw_down;       /* device fp32 [S][f_sub][d]   gradient dump, may be NULL (required in fp32 dtype) */
  /* Optional fused loss of the forward call (see "Fused loss" below); all NULL / 0 to leave it out. */
  const void* tgt;      /* device [S][T][d] regression target */
  float* loss;          /* device fp32 [S]: out */
  void* loss_ws;        /* device scratch, at least twist_fused_loss_workspace_bytes(S, T, d) bytes */
  size_t loss_ws_bytes;
  /* Optional skip connections of the chained transformer layer (App. A, Transformer Layer Architecture:
   * Y = Y_attnlayer + Y_ffn).  fwd: y = y_residual + out_scale * hh W_down;  bwd: dx = dx_residual + dpre W_gu
   * (the gradient arriving over the skip connection).  Each sum is rounded once.  NULL: no addend.
   * Not combinable with the fused loss. */
  const void* y_residual;   /* device [S][T][d] */
  const void* dx_residual;  /* device [S][T][d] */
  twist_optimizer opt;      /* bwd: optimiser of the fused update */
  float *m_gu, *v_gu;       /* device fp32 Adam moments of w_gu   [S][g*f_sub][d] */
  float *m_down, *v_down;   /* device fp32 Adam moments of w_down [S][f_sub][d] */
  /* Optional activation mask (Sec. 4.1, Masked TwIST: y = M * f(x)): device uint8 [S][f_sub], 1 = neuron active,
   * 0 = masked out.  The weights are then the full-width model (f_sub = all neurons) and worker s behaves like
   * the subnet of its active neurons: fwd hh = mask * act(pre) (pre is stored unmasked), bwd dHh = mask * dHh, so
   * the gradients of masked neurons' rows are exactly zero and the fused update leaves them untouched (Hybrid
   * TwIST's central model trains this way on its full copy).  NULL: no mask.  bf16 dtype only. */
  const uint8_t* hidden_mask;
  twist_plan* plan;         /* optional: tensor maps come from this plan's cache (see twist_plan) */
  /* bwd, bf16 dtype: non-zero when the fp32 masters hold nothing yet (the slices were gathered without
   * dst_master).  The update then reads the bf16 weights instead -- a freshly gathered slice's master is exactly
   * its widening -- and writes the masters, also when lr == 0.  Pass it on the first backward call after a gather,
   * 0 afterwards.  It saves the gather 4 of its 8 bytes per kept element. */
  int32_t master_from_slice;
} twist_ffn_args;

/* Fused loss.  When `tgt` is set, twist_subnet_ffn_fwd / twist_subnet_attn_proj_fwd also evaluate the loss
 * of twist_mse_fwd_bwd on their output inside the producing kernel: loss[s] is written, and the
 * gradient of the loss with respect to the output is written where the backward call reads it
 * (twist_ffn_args.dy, twist_proj_args.d_out), exactly as if twist_mse_fwd_bwd had been called on the
 * stored output.  The output itself (y / out) may then be NULL: it is not stored.  Results are
 * deterministic (fixed summation order). */
size_t twist_fused_loss_workspace_bytes(int32_t n_subnets, int32_t tokens, int32_t width);

int32_t twist_subnet_ffn_fwd(const twist_ffn_args* a /*host*/, void* stream);
int32_t twist_subnet_ffn_bwd(const twist_ffn_args* a /*host*/, void* stream);

/* Attention projections on the kept heads (App. A, Multi-Head Attention: Q_h = X W^Q_h ...,
 * Y_attn = Concat(heads) C^attn).
 *   which == TWIST_PROJ_QKV:  out [S][T][n] = out_scale * in [S][T][d] W^T,  W [S][n][d],  n = a_sub + 2 kv_sub
 *                             (the paper scales only the block output: pass out_scale = 1 here)
 *   which == TWIST_PROJ_O:    out [S][T][d] = out_scale * in [S][T][n] W,  W [S][n][d],  n = a_sub
 * bwd: d_in (may be NULL), dW = (QKV) d_out^T in | (O) out_scale * in^T d_out, SGD as above. */
typedef struct {
  int32_t which, dtype, n_subnets, tokens, d_model, n;
  float out_scale, lr;
  const void* in;       /* device */
  void* w;              /* device [S][n][d] */
  float* w_master;      /* device fp32 master (bf16 dtype, bwd only) */
  void* out;            /* fwd: out (may be NULL with fused loss, bf16 dtype) */
  const void* d_out;    /* bwd: in (written by a forward call with fused loss) */
  void* d_in;           /* bwd: out, may be NULL */
  float* dw;            /* device fp32 [S][n][d] gradient dump, may be NULL (required in fp32 dtype) */
  /* Optional fused loss of the forward call (see "Fused loss"); all NULL / 0 to leave it out. */
  const void* tgt;      /* device, same shape as the output */
  float* loss;          /* device fp32 [S]: out */
  void* loss_ws;        /* device scratch, at least twist_fused_loss_workspace_bytes(S, T, output width) bytes */
  size_t loss_ws_bytes;
  const int32_t* valid_cols;   /* column mask of twist_mse_fwd_bwd (device int32 [S]) or NULL */
  int32_t seg_begin, seg_width;
  /* Optional skip connections (App. A: Y_attnlayer = X + Y_attn).  TWIST_PROJ_O fwd: out = out_residual + out_scale * in W;
   * TWIST_PROJ_QKV bwd: d_in = d_in_residual + d_out W.  NULL: no addend.  Not combinable with the fused loss. */
  const void* out_residual;    /* device [S][T][d] */
  const void* d_in_residual;   /* device [S][T][d] */
  twist_optimizer opt;         /* bwd: optimiser of the fused update */
  float *m, *v;                /* device fp32 Adam moments of w [S][n][d] */
  /* Optional head mask of a masked worker (Sec. 4.1, Masked TwIST: the worker holds the full-width projections and
   * behaves like the subnet of the heads it "holds"): device uint8 [S][n], 1 for the rows of W (columns of the QKV
   * output / of the output projection's input) that belong to held heads, constant over aligned groups of 8.
   *   TWIST_PROJ_QKV fwd with fused loss: only marked columns count -- loss = mean over T x valid_cols[s] elements,
   *     zero gradient elsewhere, so the rows of W of the other heads get exactly zero gradient;
   *     valid_cols[s] must then hold the number of marked columns (twist_qkv_col_mask writes both).
   *   TWIST_PROJ_O bwd: d_in is multiplied by the mask.  (The output projection's input `in` is expected to be
   *     masked already, as the attention core's output under a head mask is.)
   * NULL: no mask.  bf16 dtype only. */
  const uint8_t* col_mask;
  twist_plan* plan;            /* optional: tensor maps come from this plan's cache */
  int32_t master_from_slice;   /* bwd: as in twist_ffn_args */
} twist_proj_args;

int32_t twist_subnet_attn_proj_fwd(const twist_proj_args* a /*host*/, void* stream);
int32_t twist_subnet_attn_proj_bwd(const twist_proj_args* a /*host*/, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Attention core of the kept heads (App. A, Multi-Head Attention: head_h = softmax(Q_h K_h^T / sqrt(d_head)) V_h),
 * the step between the QKV projection and the output projection in the chained (STACK) composition of
 * the transformer layer.  Causal within each of the n_seqs sequences of seq_len tokens (T = n_seqs * seq_len).
 *   qkv    [S][T][a' + 2 kv_max d_head]: Q of the kept heads | K of the kept KV positions | V of the same
 *   out    [S][T][a'], a' = head_keep * d_head: the concatenated heads
 *   lse    [S][head_keep][T] fp32: log-sum-exp of each score row (fwd: out; bwd: in)
 * bwd:  d_qkv [S][T][a' + 2 kv_max d_head] from d_out [S][T][a'] (exact chain rule; the probabilities are recomputed
 *       from lse); delta [S][head_keep][T] is fp32 scratch.  K/V positions a subnet does not hold
 *       (kv position >= kv_count[s]) get zero gradient.
 * Grouped-query sharing (an extension, the paper's attention is plain multi-head): when head_idx is set, kept head hq
 * of subnet s reads KV position kv_pos[s][head_idx[s][hq] / (n_heads / n_kv_heads)]; heads that share a position add
 * up in dK and dV.  head_idx == NULL: head hq reads position hq (kv_max must equal head_keep).
 * dtype TWIST_BF16 only; d_head in {8, 16, 32, 64, 128}.  fp32 arithmetic, deterministic (one writer per result). */
typedef struct {
  int32_t dtype, n_subnets, n_seqs, seq_len, head_keep, kv_max, d_head, n_heads, n_kv_heads;
  const void* qkv;           /* device */
  void* out;                 /* device  fwd: out, bwd: in */
  float* lse;                /* device */
  const void* d_out;         /* device  bwd: in */
  void* d_qkv;               /* device  bwd: out */
  float* delta;              /* device  bwd: scratch */
  const int32_t* head_idx;   /* device int32 [S][head_keep] or NULL */
  const int32_t* kv_pos;     /* device int32 [S][n_kv_heads] (required with head_idx) */
  const int32_t* kv_count;   /* device int32 [S] or NULL (every subnet holds kv_max positions) */
  twist_plan* plan;          /* optional: tensor maps come from this plan's cache */
} twist_attn_core_args;

int32_t twist_attn_core_fwd(const twist_attn_core_args* a /*host*/, void* stream);
int32_t twist_attn_core_bwd(const twist_attn_core_args* a /*host*/, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Layer normalisation of the pre-LN transformer layer (App. A, Layer Normalization: z = (x - mu) / sigma with
 * mu, sigma the mean and standard deviation of a token's d_model elements, y = gamma * z + b; Transformer
 * Layer Architecture: one normalisation before the attention block, one before the FFN block, the skip
 * connections around them).  sigma = sqrt(var + eps); eps = 0 is the printed formula.  Used by the chained
 * (STACK) composition.  gamma and b are shared parameters (Sec. 3.1: everything outside the blocks is shared):
 * every worker holds a copy, gamma / beta [S][d_model] fp32, trains it, and the aggregator averages the copies
 * (twist_gather_subnets / twist_aggregate in TWIST_FP32 with one block held by all subnets).
 *   fwd:  y [S][T][d] = gamma[s] * (x - mean) * rstd + beta[s];  mean, rstd [S][T] fp32 are written (bwd reads them)
 *   bwd:  dx = (dz - mean_d(dz) - z mean_d(dz z)) * rstd (+ dx_residual, one rounding for the sum), dz = dy * gamma,
 *         dgamma[s] = sum_t dy z,  dbeta[s] = sum_t dy  (fixed summation order: deterministic), then the optimiser
 *         step on gamma / beta when lr != 0 (twist_optimizer as in the GEMM calls; moments [S][d] fp32).
 *         dx may alias dy or dx_residual.
 * dtype TWIST_BF16 only (bf16 activations, fp32 arithmetic); d_model a multiple of 8, at most 4096.
 * ws: device scratch of at least twist_layernorm_workspace_bytes(S, T, d) bytes (bwd only). */
typedef struct {
  int32_t dtype, n_subnets, tokens, d_model;
  float eps, lr;
  const void* x;            /* device [S][T][d] */
  void* y;                  /* device [S][T][d]   fwd: out */
  float* mean;              /* device [S][T]      fwd: out, bwd: in */
  float* rstd;              /* device [S][T]      fwd: out, bwd: in */
  float* gamma;             /* device [S][d]      bwd: updated when lr != 0 */
  float* beta;              /* device [S][d] */
  const void* dy;           /* device [S][T][d]   bwd: in, gradient w.r.t. y */
  void* dx;                 /* device [S][T][d]   bwd: out */
  const void* dx_residual;  /* device [S][T][d]   bwd: optional addend (gradient over the skip connection) */
  float* dgamma;            /* device [S][d]      bwd: optional gradient dumps */
  float* dbeta;
  void* ws;                 /* device scratch (bwd) */
  size_t ws_bytes;
  twist_optimizer opt;
  float *m_gamma, *v_gamma, *m_beta, *v_beta;   /* device fp32 Adam moments [S][d] */
} twist_layernorm_args;

size_t twist_layernorm_workspace_bytes(int32_t n_subnets, int32_t tokens, int32_t d_model);
int32_t twist_layernorm_fwd(const twist_layernorm_args* a /*host*/, void* stream);
int32_t twist_layernorm_bwd(const twist_layernorm_args* a /*host*/, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Loss of the local steps: mean squared error against a target, per subnet, and its gradient.
 *   loss[s] = mean over the valid elements of (y - t)^2;   dy = 2 (y - t) / n_valid  (zero where invalid)
 * Valid columns: all `width` columns when valid_cols is NULL.  Otherwise columns [0, seg_begin) are
 * valid and the remaining columns form groups of seg_width columns each, of which the first
 * valid_cols[s] (device int32 [S]) are valid -- the zero-padded K and V column groups of a subnet
 * that kept fewer KV groups than the maximum.  (seg_begin = 0, seg_width = width gives a prefix mask.)
 *  ws / ws_bytes: device scratch of at least twist_mse_workspace_bytes(S) bytes (per-block partial
 *  sums; summed in a fixed order, so the loss is deterministic).
 */
size_t twist_mse_workspace_bytes(int32_t n_subnets);
int32_t twist_mse_fwd_bwd(const void* y, const void* tgt, void* dy, float* loss, int32_t n_subnets, int32_t tokens,
                          int32_t width, const int32_t* valid_cols, int32_t seg_begin, int32_t seg_width,
                          int32_t dtype, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * twist_mse_fwd_bwd_noalloc -- the same loss and gradient as twist_mse_fwd_bwd, for callers that
 * cannot provide scratch memory.  (The paper has no counterpart: this entry point exists for the
 * integration, not for the method.)
 *
 * Who needs it: code that runs where device allocation is forbidden or unavailable -- inside a
 * region where cudaMalloc would synchronise or fail (a latency-critical serving loop, a callback, a
 * host that hands this library a fixed set of buffers and nothing else), or a plug-in with no
 * allocator of its own.  twist_mse_fwd_bwd needs a caller-provided workspace for its per-block
 * partial sums; this variant keeps those partial sums in an array that lives inside the library.
 *
 * Limits and behaviour
 *  - The array is fixed-size device memory (TWIST_NOALLOC_MAX_SUBNETS x 1024 floats = 128 KB) that
 *    every GPU which loads the library holds until the process exits.
 *  - n_subnets > TWIST_NOALLOC_MAX_SUBNETS returns TWIST_ERR_UNSUPPORTED; nothing is launched.
 *  - No cudaMalloc, cudaFree or other allocating call is made, here or in a library on its behalf.
 *  - The first call on each device looks up the array's device address (once per device, with that
 *    device current).  Make that first call outside any stream capture.  The address is remembered for
 *    as long as the device's primary context lives; a process that destroys that context
 *    (cudaDeviceReset) must not call this entry point on the device again.
 *  - All calls share the one array, which keeps whatever the previous call left in it.  Nothing in it
 *    has to start at zero: each call overwrites every partial sum it later reads.  Two calls that
 *    overlap on the GPU (different streams, or different host threads without ordering) race on the
 *    array and give wrong losses; order them on one stream or with events.
 *  - Arguments, results and error codes are otherwise those of twist_mse_fwd_bwd.
 */
#define TWIST_NOALLOC_MAX_SUBNETS 32
int32_t twist_mse_fwd_bwd_noalloc(const void* y, const void* tgt, void* dy, float* loss, int32_t n_subnets,
                                  int32_t tokens, int32_t width, const int32_t* valid_cols, int32_t seg_begin,
                                  int32_t seg_width, int32_t dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TWIST_H_ */
