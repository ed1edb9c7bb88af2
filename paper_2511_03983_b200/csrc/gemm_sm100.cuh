// Grouped bf16 GEMM for sm_100a: TMA -> shared-memory ring -> tcgen05.mma (fp32 accumulators in
// tensor memory, double buffered) -> fused epilogues.  Persistent CTA pairs (clusters of two CTAs on
// neighbouring SMs, one pair-wide 256 x 256 tile at a time) walk the tile list of all S subnets
// ("groups"), so the S independent problems of a local-training step are one launch.
//
// A pair shares one tile: CTA r of the pair loads the A rows [128 r, 128 r + 128) and the B columns
// [128 r, 128 r + 128) of the tile into its own shared memory, and the leader (r = 0) issues
// tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and writes each CTA's 128 accumulator
// rows into that CTA's tensor memory.  Per SM and k-block this moves 32 KB from L2 instead of the
// 48 KB a single-CTA 128 x 256 tile needs; no load is multicast.
//
//   D[g] (M x N) = op(A[g]) op(B[g]),  contraction length K, for g < groups.
// Operands are dense row-major [groups][rows][cols] bf16.  "K-major" = the contraction index is the
// contiguous one (A stored [M][K], B stored [N][K]); "MN-major" = the other index is contiguous
// (A stored [K][M], B stored [K][N]).  The three layouts the training step needs:
//   NT (A K-major, B K-major)   x W^T            : up/gate/qkv forward, dHh, dA
//   NN (A K-major, B MN-major)  h W              : down / o forward, dX
//   TN (A MN-major, B MN-major) act^T other      : every weight gradient (contraction over tokens)
//
// Warp roles (320 threads per CTA): warps 0-7 epilogue (warp w owns TMEM lanes 32 (w & 3) .. +31 and half w >> 2 of
// the columns), warp 8 TMA producer (one lane), warp 9 TMEM allocator (both CTAs) + MMA issuer (one lane, leader
// CTA only).  Eight epilogue warps, two per scheduler: a single warp per scheduler cannot hide the latency of its
// own dependent instructions, and short-K tiles were bound by the epilogue's issue rate.
// Barriers: both producers' copies complete on the leader's "full" barrier; the leader's
// tcgen05.commit signals "stage empty" and "accumulator full" in both CTAs; the epilogue warps of both
// CTAs arrive on the leader's "accumulator empty" barrier.
// Every mbarrier wait is bounded in wall time; on expiry the CTA records a timeout and leaves.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace twist {

enum { MAJOR_K = 0, MAJOR_MN = 1 };
enum { EPI_STORE = 0, EPI_SWIGLU_FWD = 1, EPI_ACT_FWD = 2, EPI_DSWIGLU = 3, EPI_DACT = 4, EPI_SGD = 5, EPI_MSE = 6, EPI_RESID = 7,
       EPI_MSE_NOY = 8 /* EPI_MSE without storing D: one box per chunk, so twice as many chunk buffers */,
       EPI_ADAM = 9 /* weight gradient with the Adam update fused, like EPI_SGD */,
       EPI_SGD_LONG = 10 /* EPI_SGD for long contractions: one staged chunk per warp, full operand ring */ };

enum { L2_NORMAL = 0, L2_EVICT_FIRST = 1, L2_EVICT_LAST = 2 };

constexpr int kBM = 256, kBN = 256, kBK = 64, kUmmaK = 16;   // tile of a CTA pair
constexpr int kCtaM = kBM / 2, kCtaN = kBN / 2;   // rows of A / columns of B that one CTA of the pair loads
constexpr int kABytes = kCtaM * kBK * 2;          // 16 KB
constexpr int kBBytes = kCtaN * kBK * 2;          // 16 KB
constexpr int kStageBytes = kABytes + kBBytes;    // 32 KB per CTA and stage
constexpr int kEpiWarps = 8;                      // epilogue warps: two per tensor-memory lane quarter
constexpr int kGemmThreads = (kEpiWarps + 2) * 32;
// Epilogue staging: every epilogue warp owns 8 KB in which 32-row x 32-column bf16 boxes (2 KB, 64-byte rows,
// 64-byte swizzle) travel between global memory and the warp by TMA: operands the epilogue reads arrive as boxes,
// results leave as boxes, so every global access of the epilogue is a full-line bulk transfer.
constexpr int kEpiBoxBytes = 32 * 32 * 2;
constexpr int kCtrlBytes = 512;
// Shared memory per epilogue (EPI_* values are defined above): the staged epilogues own 8 KB per warp; the fused SGD
// update, whose chunk is two fp32 master boxes and one bf16 weight box, 12 KB (two chunks in flight) and pays
// for them with one stage of the operand ring (4 instead of 5: the weight-gradient contraction is the longest of
// all, while at short contractions its time is the masters' read-modify-write, which staging makes asynchronous:
// +19 % on the 1024-token workload).  At long contractions the shorter ring costs more (32768 tokens: 2.5 % of the 7B
// round's weight-gradient time; 8192 tokens at d = 768: 1.5 - 6 % of the backward phases), so those use EPI_SGD_LONG: the same staged update with one chunk
// buffer per warp (6 KB; the epilogue is rare there and need not overlap its own loads) and all five stages.
// The Adam update works from registers and stages nothing.
__host__ __device__ constexpr bool epi_staged(int epi) { return epi != 9 /*EPI_ADAM*/; }
__host__ __device__ constexpr int epi_warp_bytes(int epi) { return epi == 5 /*EPI_SGD*/ ? 12288 : epi == 10 /*EPI_SGD_LONG*/ ? 6144 : 8192; }
__host__ __device__ constexpr int gemm_stages(int epi) { return epi == 5 /*EPI_SGD*/ ? 4 : 5; }
__host__ __device__ constexpr int gemm_epi_region(int epi) { return epi_staged(epi) ? kEpiWarps * epi_warp_bytes(epi) : 0; }
__host__ __device__ constexpr int gemm_smem_bytes(int epi) {
  return gemm_stages(epi) * kStageBytes + gemm_epi_region(epi) + 1024 /*alignment slack*/ + kCtrlBytes;
}
constexpr int kTmemCols = 512;                    // two 128 x 256 fp32 accumulators per CTA

struct GemmParams {
  int M, N, K;          // per group.  EPI_SWIGLU_FWD: N = f_sub (neurons); the tile holds 128 gate + 128 up columns
  int groups;
  int m_tiles, n_tiles;
  int raster_m;         // m-tiles per raster band (set by the launcher from the operand layout)
  int hint_a, hint_b;   // hinted instantiations: L2 eviction priority of the A / B operand loads (L2_* above)
  int hint_epi;         // ... and of the boxes the epilogue reads and writes
  int b_split;          // EPI_SWIGLU_FWD: row of the first "up" weight inside B (= f_sub)
  int act_kind;         // TWIST_FFN_*
  float scale, lr;
  __nv_bfloat16* out0;  // STORE: D [g][M][N].  *_FWD: pre.  D*: dpre.  SGD: bf16 compute copy of the weights.  MSE: D or null
  __nv_bfloat16* out1;  // *_FWD: hh [g][M][f_sub].  MSE: gradient of the loss w.r.t. D, [g][M][N]
  const __nv_bfloat16* in0;   // DSWIGLU / DACT: pre.  MSE: target [g][M][N].  RESID: addend [g][M][N]
  float* master;        // SGD: fp32 master weights [g][M][N] (updated when lr != 0)
  int master_init;      // SGD / ADAM: the masters hold nothing yet - read the bf16 weights (out0) instead, whose exact
                        // widening they are, and write the masters (also when lr == 0)
  float* adam_m;        // ADAM: first / second moment of the group's weights, fp32 [g][M][N]
  float* adam_v;
  float beta1, beta2, adam_eps, bias1, bias2;   // ADAM: decay rates, epsilon, 1 / (1 - beta^t)
  const uint8_t* hmask;  // activation and STORE epilogues: per group N bytes, 1 = column active, 0 = masked out; may be null
  const uint8_t* col_mask;   // MSE: per group N bytes, 1 = column counts in the loss (valid_cols[g] = how many do); may be null
  float* dw;            // SGD: optional fp32 gradient dump [g][M][N].  MSE: partial sums, 16 per tile (2 CTAs x 8 warps)
  const int32_t* valid_cols;   // MSE: valid columns per column group and subnet [groups], or null (all valid)
  int seg_begin, seg_width;    // MSE: columns [0, seg_begin) valid, then groups of seg_width columns (see twist_mse_fwd_bwd)
  int* status;          // device status word
  // MSE: when done_ctr is set, the CTA that finishes last reduces the partial sums into loss_out[groups] itself
  // (same order and arithmetic as finish_fused_loss, which is then not needed).  Every CTA of the grid adds one to
  // *done_ctr, which wraps to zero at the grid size: launches that share a counter must be ordered (one stream).
  float* loss_out;
  unsigned* done_ctr;
  // Wave synchronisation (null: off).  Every CTA of the grid adds one to *wave_ctr per wave (= per tile of its own,
  // plus once for a last wave it has no tile in); wave w may start once the counter has (nearly) reached
  // wave_base + (w + 1) * gridDim.x.  The counter is never reset: the host advances wave_base by n_waves * grid
  // per launch.  Launched cooperatively, so that all CTAs are resident while they wait for one another.
  unsigned* wave_ctr;
  unsigned wave_base;
  int n_waves;
};

// Tensor maps of the epilogue's boxes (box = 32 columns x 32 rows of a dense bf16 [groups][M][cols] tensor):
//   STORE: 0 D.            MSE: 0 target (in), 1 dD (out), 2 D (out, optional).
//   SWIGLU_FWD: 0 G, 1 U (the two halves of pre), 2 hh.        ACT_FWD: 0 pre, 1 hh.
//   DSWIGLU: 0 G, 1 U (in), 2 dG, 3 dU (out).                  DACT: 0 pre (in), 1 dpre (out).
//   RESID: 0 addend (in), 1 D (out).
//   SGD: 0 fp32 masters [groups][M][N] (box = 16 columns x 32 rows, the same 64-byte rows; in and out),
//        2 bf16 weights (out; in instead of the masters when they are created from the weights).
struct EpiMaps { CUtensorMap m[4]; };

// Boxes per chunk buffer, how many of them are read from global memory first, and buffers per warp.
__host__ __device__ constexpr int epi_slots(int epi) {
  return (epi == EPI_SWIGLU_FWD || epi == EPI_SGD || epi == EPI_SGD_LONG) ? 3
         : (epi == EPI_MSE || epi == EPI_ACT_FWD || epi == EPI_DSWIGLU) ? 2 : 1;
}
__host__ __device__ constexpr int epi_in_slots(int epi) {
  return (epi == EPI_DSWIGLU || epi == EPI_SGD || epi == EPI_SGD_LONG) ? 2
         : (epi == EPI_MSE || epi == EPI_MSE_NOY || epi == EPI_DACT || epi == EPI_RESID) ? 1 : 0;
}
// chunk buffers per warp: what fits, rounded down to a power of two (4, 2 or 1)
__host__ __device__ constexpr int epi_bufs(int epi) {
  return epi_warp_bytes(epi) / (epi_slots(epi) * kEpiBoxBytes) >= 4 ? 4 : epi_warp_bytes(epi) / (epi_slots(epi) * kEpiBoxBytes) >= 2 ? 2 : 1;
}

// Registers of one 32-column chunk of accumulator words.
template <int EPI> struct EpiAcc { uint32_t r0[32]; };
// Eight consecutive mask bytes of group g starting at column `col` (a multiple of 8, col + 8 <= N) as factors.
__device__ inline void mask8(const uint8_t* hmask, int g, int N, int col, float (&m)[8]) {
  uint2 w;
  asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(w.x), "=r"(w.y) : "l"(hmask + (long long)g * N + col));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = (float)((w.x >> (8 * i)) & 1u);
    m[4 + i] = (float)((w.y >> (8 * i)) & 1u);
  }
}
template <> struct EpiAcc<EPI_SWIGLU_FWD> { uint32_t r0[32], r1[32]; };

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
// Cluster helpers: rank of this CTA in its pair, address of a shared-memory location of CTA `rank`
// in the cluster-wide shared window, arrival on a barrier given by such an address, cluster barrier.
__device__ inline uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ inline uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
  return r;
}
__device__ inline void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ inline void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tensor memory of a CTA pair: the same warp of both CTAs allocates `cols` columns together and writes the base
// address to `slot` (shared memory); pair_teardown is the common exit of such a pair.
__device__ inline void pair_tmem_alloc(volatile uint32_t* slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
               ::"r"(smem_u32(const_cast<uint32_t*>(slot))), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
// Called by every thread of both CTAs once their roles are done (or gave up).  If a wait ran out, copies that
// may still be in flight get time to land before shared memory is released.  Neither CTA leaves (nor frees
// tensor memory) while the other may still signal its barriers, read its shared memory or write its accumulators.
__device__ inline void pair_teardown(volatile int* abort_flag, bool alloc_warp, uint32_t tmem_base, uint32_t cols) {
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    drain_after_abort(abort_flag);
    __syncthreads();
  }
  cluster_sync_all();
  if (alloc_warp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(cols) : "memory");
  }
}
// All CTAs of the launch start their next tile together.  Why: the CTA pairs of a wave stream the same operand rows
// and columns along the contraction and share them through L2 only while they stay within an L2's worth of one
// another; left alone they drift apart over a long contraction, the same tiles are then fetched from DRAM several
// times, and the extra DRAM traffic costs power - hence clock - under the board's power cap.  Bounded like every wait.
__device__ inline bool wave_barrier(unsigned* ctr, unsigned target, volatile int* abort_flag, int* status) {
  atomicAdd(ctr, 1u);
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if ((int)(v - target) >= 0) return true;
    if ((it & 63u) == 0 && (*abort_flag || global_timer_ns() - t0 > kWaitLimitNs)) {
      *abort_flag = 1;
      note_status(status, (int)TWIST_ERR_DEVICE_TIMEOUT);
      return false;
    }
    __nanosleep(200);
  }
}

// Tiled copy into this CTA's shared memory; completion bytes are counted on `bar`, which may be a
// barrier of the other CTA of the pair (cluster-window address).
__device__ inline void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// The same copy with an L2 eviction policy made by l2_policy().
__device__ inline void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                   uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%3, %4, %5}], [%2], %6;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
// Arrives, once the MMAs issued so far have completed, on the barrier at this shared-memory offset in
// both CTAs of the pair.
__device__ inline void tc_commit_pair(uint32_t bar) {
  const uint16_t both = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(both) : "memory");
}
__device__ inline void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 256 (over the CTA pair), N = 256, operand majors as given.
__host__ __device__ constexpr uint32_t instr_desc(int a_major, int b_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_major << 15) | ((uint32_t)b_major << 16) |
         ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------
// Epilogue helpers
// ---------------------------------------------------------------------------------------------
__device__ inline uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ inline float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ inline float bf_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

// Stores 32 consecutive bf16 (packed in 16 words) of one row; only the first `valid` (multiple of 8) columns.
__device__ inline void store_row32(__nv_bfloat16* dst, const uint32_t (&w)[16], int valid) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if (8 * q < valid) d[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
}
__device__ inline void load_row32(const __nv_bfloat16* src, uint32_t (&w)[16], int valid) {
  const uint4* s = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 v = (8 * q < valid) ? s[q] : make_uint4(0, 0, 0, 0);
    w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
  }
}

// 1 / (1 + e^-x) with the hardware exponential and approximate reciprocal (error ~1e-7 relative, far below
// the bf16 rounding of every value it feeds); the IEEE division costs several times the rest of the epilogue.
__device__ inline float sigmoid_fast(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }

// Exact-erf GELU x Phi(x) and its derivative Phi(x) + x phi(x) for the bf16 epilogues, eight elements at a time.
// erf by the rational approximation 7.1.26 of Abramowitz & Stegun (absolute error <= 1.5e-7, far below the bf16
// rounding of every value it feeds); its exponential exp(-x^2 / 2) is also the Gaussian density the derivative needs,
// so one exponential and one approximate reciprocal serve both.  (The library erff costs several times the rest of
// the epilogue.)  The eight elements advance stage by stage: an epilogue warp has its scheduler to itself, so the
// only latency hiding there is comes from independent instructions of the same warp.
__device__ inline void gelu_parts8(const float (&x)[8], float (&cdf)[8], float (&pdf_x)[8]) {
  // v = |x| sqrt(log2(e) / 2): exp(-x^2 / 2) = 2^(-v^2), and the rational argument p |x| / sqrt(2) = kP v
  constexpr float kV = 0.84932180028801904f;           // sqrt(log2(e) / 2)
  constexpr float kP = 0.3275911f / 1.2011224087864498f;   // p / sqrt(log2(e))
  float v[8], t[8], e[8], poly[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = fabsf(x[i]) * kV;
#pragma unroll
  for (int i = 0; i < 8; ++i) asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t[i]) : "f"(fmaf(kP, v[i], 1.f)));
#pragma unroll
  for (int i = 0; i < 8; ++i) asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e[i]) : "f"(-v[i] * v[i]));   // exp(-x^2 / 2)
#pragma unroll
  for (int i = 0; i < 8; ++i) poly[i] = fmaf(t[i], 1.061405429f, -1.453152027f);
#pragma unroll
  for (int i = 0; i < 8; ++i) poly[i] = fmaf(t[i], poly[i], 1.421413741f);
#pragma unroll
  for (int i = 0; i < 8; ++i) poly[i] = fmaf(t[i], poly[i], -0.284496736f);
#pragma unroll
  for (int i = 0; i < 8; ++i) poly[i] = fmaf(t[i], poly[i], 0.254829592f);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float half_erf = fmaf(-0.5f * poly[i] * t[i], e[i], 0.5f);               // erf(|x| / sqrt(2)) / 2
    cdf[i] = 0.5f + copysignf(half_erf, x[i]);
    pdf_x[i] = x[i] * 0.3989422804014327f * e[i];                                  // x phi(x)
  }
}
// act(x) for eight pre-activations (ReLU or GELU), and act'(x).
__device__ inline void act_fwd8(const float (&x)[8], int kind, float (&y)[8]) {
  if (kind == TWIST_FFN_RELU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = fmaxf(x[i], 0.f);
    return;
  }
  float cdf[8], pdf_x[8];
  gelu_parts8(x, cdf, pdf_x);
#pragma unroll
  for (int i = 0; i < 8; ++i) y[i] = x[i] * cdf[i];
}
__device__ inline void act_grad8(const float (&x)[8], int kind, float (&g)[8]) {
  if (kind == TWIST_FFN_RELU) {
#pragma unroll
    for (int i = 0; i < 8; ++i) g[i] = x[i] > 0.f ? 1.f : 0.f;
    return;
  }
  float cdf[8], pdf_x[8];
  gelu_parts8(x, cdf, pdf_x);
#pragma unroll
  for (int i = 0; i < 8; ++i) g[i] = cdf[i] + pdf_x[i];
}

// Tile index -> (group, m_tile, n_tile): groups outermost; inside a group, bands of raster_m m-tiles, n-tiles
// next, m-tiles innermost.  The 74 tiles in flight stream their operands through L2 together, so what a wave reads
// from DRAM is one copy of the A rows and B columns it spans, plus whatever of them did not stay in L2 since the
// last wave.  Measured on the 7B-shaped launches (DRAM bytes read per layer-step, round time):
//   token-major launches (M = tokens, B = a weight slice): raster_m = 1, i.e. a wave is "a few m-tiles x every
//     n-tile" - A streams through once, B is shared by the whole wave; bands of 8 read 25 % more, panels of 4 - 12
//     n-tiles 10 - 100 % more;
//   weight-gradient launches (both operands activations streamed along a long contraction): the squarest wave,
//     bands of 8 m-tiles (8 x 9 tiles), reads least.
__device__ inline void tile_coords(const GemmParams& p, int tile, int& g, int& mt, int& nt) {
  const int per_group = p.m_tiles * p.n_tiles;
  g = tile / per_group;
  const int r = tile - g * per_group;
  const int band = r / (p.raster_m * p.n_tiles);
  const int m_first = band * p.raster_m;
  const int band_h = min(p.raster_m, p.m_tiles - m_first);
  const int rr = r - band * p.raster_m * p.n_tiles;
  nt = rr / band_h;
  mt = m_first + (rr - nt * band_h);
}

// HINTED: the operand and epilogue copies carry the L2 eviction policies of GemmParams::hint_* (a separate
// instantiation, not a run-time choice: the producer's issue latency is on the critical path of the operand ring, and
// both a branch and a predicated pair of copies per load cost the weight-gradient launches 3 - 10 %).
template <int A_MAJOR, int B_MAJOR, int EPI, bool HINTED = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ EpiMaps tmE, const GemmParams p) {
  constexpr bool kStaged = epi_staged(EPI);
  constexpr int kStages = gemm_stages(EPI);
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t epi_base = smem_base + kStages * kStageBytes;
  const uint32_t bar_base = epi_base + gemm_epi_region(EPI);
  volatile uint32_t* ctrl = reinterpret_cast<volatile uint32_t*>(smem_gen + kStages * kStageBytes + gemm_epi_region(EPI));
  // control block: 8-byte barriers full[kStages], empty[kStages], tmem_full[2], tmem_empty[2]; then the TMEM base
  // address and the abort flag (4 bytes each, within the first 160 bytes for at most 7 stages); at byte 192 the
  // 32 "box arrived" barriers of the epilogue warps (8 per warp).  Same offsets in both CTAs of the pair.
  auto in_bar = [&](int w, uint32_t buf) { return bar_base + 192u + 8u * (4u * w + buf); };
  auto full_bar = [&](int i) { return bar_base + 8u * i; };
  auto empty_bar = [&](int i) { return bar_base + 8u * (kStages + i); };
  auto tfull_bar = [&](int i) { return bar_base + 8u * (2 * kStages + i); };
  auto tempty_bar = [&](int i) { return bar_base + 8u * (2 * kStages + 2 + i); };
  volatile uint32_t* tmem_slot = ctrl + 2 * (2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 2 * (2 * kStages + 4) + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();               // 0: leader of the pair (issues the MMAs)
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int total_tiles = p.groups * p.m_tiles * p.n_tiles;
  const int num_kb = (p.K + kBK - 1) / kBK;

  if (warp == kEpiWarps && lane == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int i = 0; i < kStages; ++i) { mbar_init(full_bar(i), 1); mbar_init(empty_bar(i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), 2 * kEpiWarps); }   // epilogue warps of both CTAs
    if (kStaged)
      for (int w = 0; w < kEpiWarps; ++w)
        for (int b = 0; b < 4; ++b) mbar_init(in_bar(w, b), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kEpiWarps + 1) pair_tmem_alloc(tmem_slot, (uint32_t)kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers exist before anything is signalled across the pair
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The set-up above touches nothing an earlier launch wrote, so it may overlap that launch's tail; from here on
  // this launch reads its operands.  (Its own successor may in turn be placed as soon as these CTAs have gone.)
  griddep_launch_dependents();
  griddep_wait();

  if (warp == kEpiWarps) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      unsigned wave = 0;
      const uint64_t pol_a = HINTED ? l2_policy(p.hint_a) : 0, pol_b = HINTED ? l2_policy(p.hint_b) : 0;
      auto load_a = [&](uint32_t dst, uint32_t bar, int c0, int c1, int c2) {
        if constexpr (HINTED) tma_load_3d(dst, &tmA, bar, c0, c1, c2, pol_a); else tma_load_3d(dst, &tmA, bar, c0, c1, c2);
      };
      auto load_b = [&](uint32_t dst, uint32_t bar, int c0, int c1, int c2) {
        if constexpr (HINTED) tma_load_3d(dst, &tmB, bar, c0, c1, c2, pol_b); else tma_load_3d(dst, &tmB, bar, c0, c1, c2);
      };
      for (int tile = pair; ok && tile < total_tiles; tile += num_pairs, ++wave) {
        int g, mt, nt;
        tile_coords(p, tile, g, mt, nt);
        // (the last eighth of the CTAs is not waited for: rough lockstep is all the L2 needs, and the stragglers'
        // share of a wave would otherwise be idle time for everyone)
        if (p.wave_ctr && !wave_barrier(p.wave_ctr, p.wave_base + (wave + 1u) * gridDim.x - (gridDim.x >> 3), abort_flag,
                                        p.status)) {
          ok = false;
          break;
        }
        const int m0 = mt * kBM + (int)rank * kCtaM;
        // B rows (K-major) / columns (MN-major) of this CTA.  SwiGLU forward: the leader loads 128 gate
        // rows, the peer the matching 128 up rows, so accumulator columns 0..127 are G and 128..255 are U.
        const int n0 = (EPI == EPI_SWIGLU_FWD) ? (rank ? p.b_split : 0) + nt * kCtaN : nt * kBN + (int)rank * kCtaN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int stage = it % kStages;
          const uint32_t phase = (it / kStages) & 1u;
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * kStageBytes);   // both CTAs' bytes
          const uint32_t bar = map_to_cta(full_bar(stage), 0);
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          const uint32_t b_dst = a_dst + kABytes;
          const int k0 = kb * kBK;
          if (A_MAJOR == MAJOR_K) {
            load_a(a_dst, bar, k0, m0, g);                       // box 64 (K) x 128 rows
          } else {
#pragma unroll
            for (int j = 0; j < kCtaM / 64; ++j) load_a(a_dst + j * 8192, bar, m0 + 64 * j, k0, g);   // 64 (M) x 64 (K)
          }
          if (B_MAJOR == MAJOR_K) {
            load_b(b_dst, bar, k0, n0, g);                       // box 64 (K) x 128 rows
          } else {
#pragma unroll
            for (int j = 0; j < kCtaN / 64; ++j) load_b(b_dst + j * 8192, bar, n0 + 64 * j, k0, g);   // 64 (N) x 64 (K)
          }
        }
      }
      // a wave this CTA has no tile in (the last, partial one) still gets its arrival: the count per wave is uniform
      if (p.wave_ctr && ok)
        for (; (int)wave < p.n_waves; ++wave) atomicAdd(p.wave_ctr, 1u);
    }
  } else if (warp == kEpiWarps + 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc(A_MAJOR, B_MAJOR);
      constexpr uint32_t a_lbo = A_MAJOR == MAJOR_K ? 16u : (uint32_t)kBK * 128u;
      constexpr uint32_t b_lbo = B_MAJOR == MAJOR_K ? 16u : (uint32_t)kBK * 128u;
      constexpr uint32_t a_kstep = A_MAJOR == MAJOR_K ? (kUmmaK * 2) : (kUmmaK * 128);   // bytes per 16 of K
      constexpr uint32_t b_kstep = B_MAJOR == MAJOR_K ? (kUmmaK * 2) : (kUmmaK * 128);
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = pair; ok && tile < total_tiles; tile += num_pairs, ++tl) {
        const uint32_t slot = tl & 1u, acc_phase = (tl >> 1) & 1u;
        if (!mbar_wait(tempty_bar(slot), acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + slot * kBN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int stage = it % kStages;
          const uint32_t phase = (it / kStages) & 1u;
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_base + stage * kStageBytes;
          const uint32_t b_addr = a_addr + kABytes;
          const uint64_t a_desc = smem_desc(a_addr, a_lbo, 1024u);
          const uint64_t b_desc = smem_desc(b_addr, b_lbo, 1024u);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            tc_mma_bf16(d_tmem, a_desc + (uint64_t)((k * a_kstep) >> 4), b_desc + (uint64_t)((k * b_kstep) >> 4), idesc,
                        (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit_pair(empty_bar(stage));      // frees the stage in both CTAs when these MMAs have read it
        }
        if (ok) tc_commit_pair(tfull_bar(slot)); // accumulator complete, in both CTAs
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 0..3
    // Thread (warp w, lane l) owns accumulator row 32 w + l of this CTA and walks it in chunks of 32 columns;
    // the tensor-memory load of chunk c + 1 is in flight while chunk c is processed.
    // Warp w reads tensor-memory lanes 32 (w & 3) .. +31 (the rows of that quarter) and the columns of half w >> 2:
    // 128 of the tile's 256 output columns (SwiGLU forward: 64 of its 128 neurons, as 64 G and 64 U columns).
    constexpr int kTileN = (EPI == EPI_SWIGLU_FWD) ? kCtaN : kBN;     // output columns (neurons) per tile
    constexpr int kHalfN = kTileN / 2;                                // ... per warp
    constexpr int kChunks = kHalfN / 32;
    const int quarter = warp & 3, half = warp >> 2;
    const uint32_t tempty_leader[2] = {map_to_cta(tempty_bar(0), 0), map_to_cta(tempty_bar(1), 0)};
    uint32_t tl = 0;
    bool ok = true;

    if constexpr (EPI == EPI_ADAM) {
      // Weight-gradient tiles with the Adam step (three fp32 streams per weight: too many for the staging buffers):
      // plain vector accesses to the fp32 rows; the master values of the next chunk are loaded ahead.
      for (int tile = pair; ok && tile < total_tiles; tile += num_pairs, ++tl) {
        int g, mt, nt;
        tile_coords(p, tile, g, mt, nt);
        const uint32_t slot = tl & 1u, acc_phase = (tl >> 1) & 1u;
        const int row = mt * kBM + (int)rank * kCtaM + quarter * 32 + lane;
        const bool row_ok = row < p.M;
        const uint32_t t_row = tmem_base + slot * kBN + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * kHalfN);
        const long long grow = (long long)g * p.M + row;      // row index over all groups
        const int n_base = nt * kBN + half * kHalfN;
        float4 mv[2][8];
        EpiAcc<EPI> acc[2];
        const bool do_update = p.lr != 0.f || p.master_init != 0;
        auto load_master = [&](int c, float4 (&m)[8]) {
          const int n = n_base + 32 * c;
          const int valid = (row_ok && n < p.N && do_update) ? min(32, p.N - n) : 0;
          if (p.master_init) {      // first update since the slices were gathered: the master is the widened bf16 weight
            const uint4* src = reinterpret_cast<const uint4*>(p.out0 + grow * p.N + n);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 v = (8 * q < valid) ? src[q] : make_uint4(0, 0, 0, 0);
              m[2 * q] = make_float4(bf_lo(v.x), bf_hi(v.x), bf_lo(v.y), bf_hi(v.y));
              m[2 * q + 1] = make_float4(bf_lo(v.z), bf_hi(v.z), bf_lo(v.w), bf_hi(v.w));
            }
          } else {
            const float4* src = reinterpret_cast<const float4*>(p.master + grow * p.N + n);
#pragma unroll
            for (int q = 0; q < 8; ++q) m[q] = (4 * q < valid) ? src[q] : make_float4(0.f, 0.f, 0.f, 0.f);
          }
        };
        load_master(0, mv[0]);
        if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(slot), acc_phase, abort_flag, p.status))) { ok = false; break; }
        tc_fence_after();
        tc_ld32(t_row, acc[0].r0);
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          tc_wait_ld();
          if (c + 1 < kChunks) {
            tc_ld32(t_row + 32 * (c + 1), acc[(c + 1) & 1].r0);
            load_master(c + 1, mv[(c + 1) & 1]);
          }
          const int n = n_base + 32 * c;
          if (row_ok && n < p.N) {
            const int valid = min(32, p.N - n);
            const uint32_t* r = acc[c & 1].r0;
            float* master = p.master + grow * p.N + n;
            float* dw = p.dw ? p.dw + grow * p.N + n : nullptr;
            __nv_bfloat16* w16 = p.out0 + grow * p.N + n;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (4 * q < valid) {
                const float4 gq = make_float4(p.scale * __uint_as_float(r[4 * q]), p.scale * __uint_as_float(r[4 * q + 1]),
                                              p.scale * __uint_as_float(r[4 * q + 2]), p.scale * __uint_as_float(r[4 * q + 3]));
                if (dw) *reinterpret_cast<float4*>(dw + 4 * q) = gq;
                if (do_update) {        // master -= lr * step (fp32); compute copy = bf16(master)
                  float4 m = mv[c & 1][q];
                  if constexpr (EPI == EPI_ADAM) {
                    // m1 <- b1 m1 + (1 - b1) g;  m2 <- b2 m2 + (1 - b2) g^2;  step = (m1 / (1 - b1^t)) / (sqrt(m2 / (1 - b2^t)) + eps)
                    float* pm1 = p.adam_m + grow * p.N + n + 4 * q;
                    float* pm2 = p.adam_v + grow * p.N + n + 4 * q;
                    float4 m1 = *reinterpret_cast<const float4*>(pm1), m2 = *reinterpret_cast<const float4*>(pm2);
                    const float gv[4] = {gq.x, gq.y, gq.z, gq.w};
                    float* a1 = &m1.x; float* a2 = &m2.x; float* wv = &m.x;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                      a1[e] = fmaf(p.beta1, a1[e], (1.f - p.beta1) * gv[e]);
                      a2[e] = fmaf(p.beta2, a2[e], (1.f - p.beta2) * gv[e] * gv[e]);
                      wv[e] -= p.lr * (a1[e] * p.bias1) / (sqrtf(a2[e] * p.bias2) + p.adam_eps);
                    }
                    *reinterpret_cast<float4*>(pm1) = m1;
                    *reinterpret_cast<float4*>(pm2) = m2;
                  } else {
                    m.x -= p.lr * gq.x; m.y -= p.lr * gq.y; m.z -= p.lr * gq.z; m.w -= p.lr * gq.w;
                  }
                  *reinterpret_cast<float4*>(master + 4 * q) = m;
                  *reinterpret_cast<uint2*>(w16 + 4 * q) = make_uint2(pack2(m.x, m.y), pack2(m.z, m.w));
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_leader[slot]);      // accumulator slot free again
      }
    } else {
      // Staged epilogues.  Chunk number gc (counted over all tiles of this CTA) uses buffer gc % kBufs of the
      // warp: kSlots boxes of 2 KB.  Boxes the chunk reads are requested kBufs / 2 chunks ahead, results are
      // written over them in place (each thread touches only its own row) and leave as bulk stores; a buffer
      // is refilled or rewritten only after the bulk store that last read it has finished reading.
      constexpr int kSlots = epi_slots(EPI), kIn = epi_in_slots(EPI), kBufs = epi_bufs(EPI);
      constexpr bool kIsMse = EPI == EPI_MSE || EPI == EPI_MSE_NOY;
      // Inputs are requested kAhead chunks ahead into the buffer that chunk gc + kAhead - kBufs used; only that
      // chunk's store has to be finished, so up to kBufs - kAhead younger stores may still be reading.
      constexpr int kAhead = kBufs > 1 ? kBufs / 2 : 1;
      const uint32_t wbase = epi_base + (uint32_t)warp * epi_warp_bytes(EPI);
      auto box = [&](uint32_t gc, int slot) { return wbase + ((gc & (kBufs - 1)) * kSlots + slot) * kEpiBoxBytes; };
      // 16-byte piece q (0..3) of this thread's row inside a box (64-byte rows, 64-byte swizzle)
      const uint32_t row_off = (uint32_t)lane * 64u;
      const uint32_t sw = ((uint32_t)lane >> 1) & 3u;
      auto piece = [&](uint32_t box_addr, int q) { return box_addr + row_off + ((((uint32_t)q) ^ sw) << 4); };
      // Coordinates (group, first row of this warp, first column) of the tile being processed and of the CTA's next
      // tile, so that requesting a chunk's inputs costs no index arithmetic (kAhead < kChunks: a requested chunk
      // lies in one of the two).
      struct TileAt { int g, row0, n0; bool valid; };
      auto locate = [&](int tile) {
        TileAt t;
        t.valid = tile < total_tiles;
        t.g = 0; t.row0 = 0; t.n0 = 0;
        if (t.valid) {
          int mt, nt;
          tile_coords(p, tile, t.g, mt, nt);
          t.row0 = mt * kBM + (int)rank * kCtaM + quarter * 32;
          t.n0 = nt * kTileN + half * kHalfN;
        }
        return t;
      };
      TileAt cur = locate(pair), nxt = locate(pair + num_pairs);
      // EPI_SGD: whether this launch updates the weights at all (otherwise it only dumps gradients and stages nothing)
      constexpr bool kSgd = EPI == EPI_SGD || EPI == EPI_SGD_LONG;
      const bool sgd_update = kSgd && (p.lr != 0.f || p.master_init != 0);
      const uint64_t pol_epi = HINTED ? l2_policy(p.hint_epi) : 0;
      auto box_load = [&](uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
        if constexpr (HINTED) tma_load_3d_local(dst, map, bar, c0, c1, c2, pol_epi); else tma_load_3d_local(dst, map, bar, c0, c1, c2);
      };
      auto box_store = [&](const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
        if constexpr (HINTED) tma_store_3d(map, src, c0, c1, c2, pol_epi); else tma_store_3d(map, src, c0, c1, c2);
      };
      auto request_inputs = [&](uint32_t gc) {      // lane 0 only; gc / kChunks is tl or tl + 1
        if (kIn == 0) return;
        const TileAt& t = (gc / kChunks == tl) ? cur : nxt;
        if (!t.valid) return;
        const uint32_t bar = in_bar(warp, gc & (kBufs - 1));
        const int n = t.n0 + 32 * (int)(gc % kChunks);
        if constexpr (kSgd) {
          if (!sgd_update) return;
          if (p.master_init) {      // the masters do not exist yet: the bf16 weights, whose widening they are
            mbar_expect_tx(bar, kEpiBoxBytes);
            box_load(box(gc, 2), &tmE.m[2], bar, n, t.row0, t.g);
          } else {                  // two boxes of 16 fp32 columns
            mbar_expect_tx(bar, 2 * kEpiBoxBytes);
            box_load(box(gc, 0), &tmE.m[0], bar, n, t.row0, t.g);
            box_load(box(gc, 1), &tmE.m[0], bar, n + 16, t.row0, t.g);
          }
          return;
        }
        mbar_expect_tx(bar, kIn * kEpiBoxBytes);
#pragma unroll
        for (int i = 0; i < kIn; ++i) box_load(box(gc, i), &tmE.m[i], bar, n, t.row0, t.g);
      };
      if (lane == 0) {
        for (uint32_t gc = 0; gc < (uint32_t)kAhead; ++gc) request_inputs(gc);
      }

      for (int tile = pair; ok && tile < total_tiles; tile += num_pairs, ++tl) {
        if (tl > 0) { cur = nxt; nxt = locate(tile + num_pairs); }
        const int g = cur.g, nt_n0 = cur.n0;
        const uint32_t slot = tl & 1u, acc_phase = (tl >> 1) & 1u;
        const int row0 = cur.row0;
        const bool row_ok = row0 + lane < p.M;
        const uint32_t t_row = tmem_base + slot * kBN + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * kHalfN);
        const int n_base = nt_n0;
        EpiAcc<EPI> acc[2];
        float loss_acc = 0.f, kfac = 0.f;
        int vc = 0;
        if constexpr (kIsMse) {
          vc = p.valid_cols ? min(max(p.valid_cols[g], 0), p.seg_width) : p.seg_width;
          const int n_valid = p.seg_begin + ((p.N - p.seg_begin) / p.seg_width) * vc;
          kfac = n_valid > 0 ? 2.0f / ((float)p.M * (float)n_valid) : 0.f;      // no valid column: zero loss, zero gradient
        }
        auto load_acc = [&](int c, EpiAcc<EPI>& a) {
          tc_ld32(t_row + 32 * c, a.r0);
          if constexpr (EPI == EPI_SWIGLU_FWD) tc_ld32(t_row + kCtaN + 32 * c, a.r1);      // U: 128 columns after G
        };
        if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(slot), acc_phase, abort_flag, p.status))) { ok = false; break; }
        tc_fence_after();
        load_acc(0, acc[0]);
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          const uint32_t gc = tl * kChunks + c;
          const int n = n_base + 32 * c;
          if (kIn > 0 && (!kSgd || sgd_update)) {      // this chunk's boxes have arrived
            if (!__all_sync(0xffffffffu, mbar_wait(in_bar(warp, gc & (kBufs - 1)), (gc / kBufs) & 1u, abort_flag, p.status))) { ok = false; break; }
          } else if (!kSgd) {      // the bulk store that last read this buffer is done with it
            if (lane == 0) bulk_wait_read<kBufs - 1>();
            __syncwarp();
          }
          tc_wait_ld();
          if (c + 1 < kChunks) load_acc(c + 1, acc[(c + 1) & 1]);
          const EpiAcc<EPI>& a = acc[c & 1];
          const uint32_t b0 = box(gc, 0), b1 = box(gc, kSlots > 1 ? 1 : 0), b2 = box(gc, kSlots > 2 ? 2 : 0);

          // ---- compute this thread's 32 columns; results go to the boxes, 8 columns (16 bytes) at a time
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t* r = a.r0 + 8 * q;
            float hm[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
            if constexpr (EPI == EPI_SWIGLU_FWD || EPI == EPI_ACT_FWD || EPI == EPI_DSWIGLU || EPI == EPI_DACT ||
                          EPI == EPI_STORE) {
              if (p.hmask && n + 8 * q < p.N) mask8(p.hmask, g, p.N, n + 8 * q, hm);     // uniform branch
            }
            if constexpr (EPI == EPI_STORE) {
              float sc[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) sc[e] = p.scale * hm[e];
              sts128(piece(b0, q), make_uint4(pack2(sc[0] * __uint_as_float(r[0]), sc[1] * __uint_as_float(r[1])),
                                              pack2(sc[2] * __uint_as_float(r[2]), sc[3] * __uint_as_float(r[3])),
                                              pack2(sc[4] * __uint_as_float(r[4]), sc[5] * __uint_as_float(r[5])),
                                              pack2(sc[6] * __uint_as_float(r[6]), sc[7] * __uint_as_float(r[7]))));
            } else if constexpr (kIsMse) {
              const uint4 tv = lds128(piece(b0, q));
              const uint32_t tw[4] = {tv.x, tv.y, tv.z, tv.w};
              // validity is constant over aligned groups of 8 columns (seg_begin, seg_width, vc are multiples of 8)
              const int col = n + 8 * q;
              bool cv = row_ok && col < p.N;
              if (p.col_mask) {                             // arbitrary column set (constant over aligned groups of 8)
                cv = cv && p.col_mask[(long long)g * p.N + col] != 0;
              } else if (p.valid_cols && col >= p.seg_begin) {     // masked column groups (uniform branch; few groups: no division)
                int rel = col - p.seg_begin;
                while (rel >= p.seg_width) rel -= p.seg_width;
                cv = cv && rel < vc;
              }
              uint32_t wy[4], wd[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                wy[h] = pack2(p.scale * __uint_as_float(r[2 * h]), p.scale * __uint_as_float(r[2 * h + 1]));
                const float d0 = cv ? bf_lo(wy[h]) - bf_lo(tw[h]) : 0.f;
                const float d1 = cv ? bf_hi(wy[h]) - bf_hi(tw[h]) : 0.f;
                loss_acc += d0 * d0 + d1 * d1;
                wd[h] = pack2(kfac * d0, kfac * d1);
              }
              sts128(piece(b0, q), make_uint4(wd[0], wd[1], wd[2], wd[3]));
              if constexpr (EPI == EPI_MSE) sts128(piece(b1, q), make_uint4(wy[0], wy[1], wy[2], wy[3]));
            } else if constexpr (EPI == EPI_SWIGLU_FWD) {
              const uint32_t* ru = a.r1 + 8 * q;
              uint32_t wg[4], wu[4], wh[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                const float g0 = __uint_as_float(r[2 * h]), g1 = __uint_as_float(r[2 * h + 1]);
                const float u0 = __uint_as_float(ru[2 * h]), u1 = __uint_as_float(ru[2 * h + 1]);
                wg[h] = pack2(g0, g1);
                wu[h] = pack2(u0, u1);
                wh[h] = pack2(g0 * sigmoid_fast(g0) * u0 * hm[2 * h], g1 * sigmoid_fast(g1) * u1 * hm[2 * h + 1]);
              }
              sts128(piece(b0, q), make_uint4(wg[0], wg[1], wg[2], wg[3]));
              sts128(piece(b1, q), make_uint4(wu[0], wu[1], wu[2], wu[3]));
              sts128(piece(b2, q), make_uint4(wh[0], wh[1], wh[2], wh[3]));
            } else if constexpr (EPI == EPI_ACT_FWD) {
              uint32_t wp[4], wh[4];
              float xin[8], yv[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) xin[i] = __uint_as_float(r[i]);
              act_fwd8(xin, p.act_kind, yv);
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                wp[h] = pack2(xin[2 * h], xin[2 * h + 1]);
                wh[h] = pack2(yv[2 * h] * hm[2 * h], yv[2 * h + 1] * hm[2 * h + 1]);
              }
              sts128(piece(b0, q), make_uint4(wp[0], wp[1], wp[2], wp[3]));
              sts128(piece(b1, q), make_uint4(wh[0], wh[1], wh[2], wh[3]));
            } else if constexpr (EPI == EPI_DSWIGLU) {
              const uint4 gv = lds128(piece(b0, q)), uv = lds128(piece(b1, q));
              const uint32_t pg[4] = {gv.x, gv.y, gv.z, gv.w}, pu[4] = {uv.x, uv.y, uv.z, uv.w};
              uint32_t wg[4], wu[4];
#pragma unroll
              for (int h = 0; h < 4; ++h) {
                float dg[2], du[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                  const float dh = p.scale * __uint_as_float(r[2 * h + e]) * hm[2 * h + e];
                  const float gt = e ? bf_hi(pg[h]) : bf_lo(pg[h]);
                  const float up = e ? bf_hi(pu[h]) : bf_lo(pu[h]);
                  const float sg = sigmoid_fast(gt);
                  dg[e] = dh * up * (sg * (1.f + gt * (1.f - sg)));
                  du[e] = dh * (gt * sg);
                }
                wg[h] = pack2(dg[0], dg[1]);
                wu[h] = pack2(du[0], du[1]);
              }
              sts128(piece(b0, q), make_uint4(wg[0], wg[1], wg[2], wg[3]));
              sts128(piece(b1, q), make_uint4(wu[0], wu[1], wu[2], wu[3]));
            } else if constexpr (kSgd) {
              // columns 8 q .. 8 q + 7 of the chunk: two 16-byte pieces of a master box, one piece of the weight box
              float gv[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) gv[e] = p.scale * __uint_as_float(r[e]);
              if (p.dw && row_ok && n + 8 * q < p.N) {      // optional gradient dump (tests, the fp32 parity checks)
                float* dwp = p.dw + ((long long)g * p.M + row0 + lane) * p.N + n + 8 * q;
                *reinterpret_cast<float4*>(dwp) = make_float4(gv[0], gv[1], gv[2], gv[3]);
                *reinterpret_cast<float4*>(dwp + 4) = make_float4(gv[4], gv[5], gv[6], gv[7]);
              }
              if (sgd_update) {
                const uint32_t mb = (q < 2) ? b0 : b1;          // master box holding these columns
                const int pq = 2 * (q & 1);                      // its first 16-byte piece
                float m[8];
                if (p.master_init) {
                  const uint4 wv = lds128(piece(b2, q));
                  m[0] = bf_lo(wv.x); m[1] = bf_hi(wv.x); m[2] = bf_lo(wv.y); m[3] = bf_hi(wv.y);
                  m[4] = bf_lo(wv.z); m[5] = bf_hi(wv.z); m[6] = bf_lo(wv.w); m[7] = bf_hi(wv.w);
                } else {
                  const uint4 lo = lds128(piece(mb, pq)), hi = lds128(piece(mb, pq + 1));
                  m[0] = __uint_as_float(lo.x); m[1] = __uint_as_float(lo.y); m[2] = __uint_as_float(lo.z); m[3] = __uint_as_float(lo.w);
                  m[4] = __uint_as_float(hi.x); m[5] = __uint_as_float(hi.y); m[6] = __uint_as_float(hi.z); m[7] = __uint_as_float(hi.w);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) m[e] -= p.lr * gv[e];       // master -= lr * g (fp32)
                sts128(piece(mb, pq), make_uint4(__float_as_uint(m[0]), __float_as_uint(m[1]), __float_as_uint(m[2]), __float_as_uint(m[3])));
                sts128(piece(mb, pq + 1), make_uint4(__float_as_uint(m[4]), __float_as_uint(m[5]), __float_as_uint(m[6]), __float_as_uint(m[7])));
                sts128(piece(b2, q), make_uint4(pack2(m[0], m[1]), pack2(m[2], m[3]), pack2(m[4], m[5]), pack2(m[6], m[7])));   // compute copy
              }
            } else if constexpr (EPI == EPI_RESID) {   // D = addend + scale * acc, rounded once
              const uint4 av = lds128(piece(b0, q));
              const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
              uint32_t w[4];
#pragma unroll
              for (int h = 0; h < 4; ++h)
                w[h] = pack2(fmaf(p.scale, __uint_as_float(r[2 * h]), bf_lo(aw[h])),
                             fmaf(p.scale, __uint_as_float(r[2 * h + 1]), bf_hi(aw[h])));
              sts128(piece(b0, q), make_uint4(w[0], w[1], w[2], w[3]));
            } else {   // EPI_DACT
              const uint4 pv = lds128(piece(b0, q));
              const uint32_t pp[4] = {pv.x, pv.y, pv.z, pv.w};
              uint32_t w[4];
              float xin[8], gv[8];
#pragma unroll
              for (int h = 0; h < 4; ++h) { xin[2 * h] = bf_lo(pp[h]); xin[2 * h + 1] = bf_hi(pp[h]); }
              act_grad8(xin, p.act_kind, gv);
#pragma unroll
              for (int h = 0; h < 4; ++h)
                w[h] = pack2(p.scale * __uint_as_float(r[2 * h]) * gv[2 * h] * hm[2 * h],
                             p.scale * __uint_as_float(r[2 * h + 1]) * gv[2 * h + 1] * hm[2 * h + 1]);
              sts128(piece(b0, q), make_uint4(w[0], w[1], w[2], w[3]));
            }
          }

          // ---- the boxes leave by bulk store (rows / columns outside the tensor are clipped)
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            const int rr = row0, gg = g;
            if constexpr (EPI == EPI_STORE) {
              box_store(&tmE.m[0], b0, n, rr, gg);
            } else if constexpr (kIsMse) {
              box_store(&tmE.m[1], b0, n, rr, gg);
              if constexpr (EPI == EPI_MSE) box_store(&tmE.m[2], b1, n, rr, gg);
            } else if constexpr (EPI == EPI_SWIGLU_FWD) {
              box_store(&tmE.m[0], b0, n, rr, gg);
              box_store(&tmE.m[1], b1, n, rr, gg);
              box_store(&tmE.m[2], b2, n, rr, gg);
            } else if constexpr (EPI == EPI_ACT_FWD) {
              box_store(&tmE.m[0], b0, n, rr, gg);
              box_store(&tmE.m[1], b1, n, rr, gg);
            } else if constexpr (EPI == EPI_DSWIGLU) {
              box_store(&tmE.m[2], b0, n, rr, gg);
              box_store(&tmE.m[3], b1, n, rr, gg);
            } else if constexpr (kSgd) {
              if (sgd_update) {
                box_store(&tmE.m[0], b0, n, rr, gg);
                box_store(&tmE.m[0], b1, n + 16, rr, gg);
                box_store(&tmE.m[2], b2, n, rr, gg);
              }
            } else {   // DACT, RESID
              box_store(&tmE.m[1], b0, n, rr, gg);
            }
            bulk_commit();
            if (kIn > 0) {     // refill the buffer whose store is old enough to have finished reading
              bulk_wait_read<kBufs - kAhead>();
              request_inputs(gc + kAhead);
            }
          }
        }
        if (!ok) break;
        // accumulator slot free again
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_leader[slot]);
        if constexpr (kIsMse) {   // per-warp partial sum of squared errors, fixed order
          for (int o = 16; o > 0; o >>= 1) loss_acc += __shfl_xor_sync(0xffffffffu, loss_acc, o);
          if (lane == 0) p.dw[((long long)tile * 2 + rank) * kEpiWarps + warp] = loss_acc;
        }
      }
      if (lane == 0) bulk_wait_read<0>();      // shared memory stays valid until the last store has read it
      __syncwarp();
    }
  }

  if constexpr (EPI == EPI_MSE || EPI == EPI_MSE_NOY) {
    if (p.done_ctr) {      // the last CTA to get here turns the partial sums into the losses
      __shared__ int last_cta;
      if (warp < kEpiWarps && lane == 0) __threadfence();        // this warp's partial sums are visible device-wide
      __syncthreads();
      if (threadIdx.x == 0) {
        const unsigned before = atomicInc(p.done_ctr, gridDim.x - 1u);
        last_cta = before == gridDim.x - 1u;
      }
      __syncthreads();
      if (last_cta && warp < kEpiWarps) {
        __threadfence();
        const long long per_group = (long long)p.m_tiles * p.n_tiles * 2 * kEpiWarps;
        for (int g = warp; g < p.groups; g += kEpiWarps) {
          const float* src = p.dw + (long long)g * per_group;
          double acc = 0.0;
          for (long long i = lane; i < per_group; i += 32) acc += (double)__ldcg(src + i);
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          if (lane == 0) {
            const int vc = p.valid_cols ? min(max(p.valid_cols[g], 0), p.seg_width) : p.seg_width;
            const long long n_valid = p.seg_begin + (long long)((p.N - p.seg_begin) / p.seg_width) * vc;
            p.loss_out[g] = n_valid > 0 ? (float)(acc / ((double)p.M * (double)n_valid)) : 0.f;
          }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  pair_teardown(abort_flag, warp == kEpiWarps + 1, tmem_base, (uint32_t)kTmemCols);
}

// Host side ------------------------------------------------------------------------------------

struct GemmOperand {
  const void* ptr;     // dense bf16 [groups][rows][cols]
  int rows, cols;
};

// layout: 0 NT, 1 NN, 2 TN.  Returns a TWIST_* status.
int launch_gemm_bf16(int layout, int epi, const GemmOperand& A, const GemmOperand& B, GemmParams p, cudaStream_t st);

// EPI_MSE: number of fp32 partial sums the kernel writes (GemmParams::dw) for `groups` problems of M x N,
// and the fixed-order reduction of those partials into loss[groups].
size_t fused_loss_partials(int groups, int M, int N);
// Counter for GemmParams::done_ctr on stream `st`, or null when the launch has to be followed by finish_fused_loss
// (stream being captured, or more streams in use than there are counters).
unsigned* fused_loss_counter(cudaStream_t st);
int finish_fused_loss(const float* partial, int groups, int M, int N, const int32_t* valid_cols, int seg_begin,
                      int seg_width, float* loss, cudaStream_t st);

}  // namespace twist
