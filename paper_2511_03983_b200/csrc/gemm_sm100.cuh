// Grouped bf16 GEMM for sm_100a: TMA -> shared-memory ring -> tcgen05.mma (fp32 accumulators in
// tensor memory, double buffered) -> fused epilogues.  One persistent CTA per SM walks the tile list
// of all S subnets ("groups"), so the S independent problems of a local-training step are one launch.
//
//   D[g] (M x N) = op(A[g]) op(B[g]),  contraction length K, for g < groups.
// Operands are dense row-major [groups][rows][cols] bf16.  "K-major" = the contraction index is the
// contiguous one (A stored [M][K], B stored [N][K]); "MN-major" = the other index is contiguous
// (A stored [K][M], B stored [K][N]).  The three layouts the training step needs:
//   NT (A K-major, B K-major)   x W^T            : up/gate/qkv forward, dHh, dA
//   NN (A K-major, B MN-major)  h W              : down / o forward, dX
//   TN (A MN-major, B MN-major) act^T other      : every weight gradient (contraction over tokens)
//
// Warp roles (192 threads): warps 0-3 epilogue (warp w owns TMEM lanes 32w..32w+31), warp 4 TMA
// producer (one lane), warp 5 TMEM allocator + MMA issuer (one lane).
// Every mbarrier wait is bounded in wall time; on expiry the CTA records a timeout and leaves.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace twist {

enum { MAJOR_K = 0, MAJOR_MN = 1 };
enum { EPI_STORE = 0, EPI_SWIGLU_FWD = 1, EPI_ACT_FWD = 2, EPI_DSWIGLU = 3, EPI_DACT = 4, EPI_SGD = 5 };

constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4, kUmmaK = 16;
constexpr int kABytes = kBM * kBK * 2;            // 16 KB
constexpr int kBBytes = kBN * kBK * 2;            // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;    // 48 KB
constexpr int kGemmThreads = 192;
constexpr int kGemmSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kTmemCols = 512;                    // two 128 x 256 fp32 accumulators
constexpr int kRasterGroupM = 16;                 // m-tiles per raster group (L2 reuse of A and B tiles)

struct GemmParams {
  int M, N, K;          // per group.  EPI_SWIGLU_FWD: N = f_sub (neurons); the tile holds 128 gate + 128 up columns
  int groups;
  int m_tiles, n_tiles;
  int b_split;          // EPI_SWIGLU_FWD: row of the first "up" weight inside B (= f_sub)
  int act_kind;         // TWIST_FFN_*
  float scale, lr;
  __nv_bfloat16* out0;  // STORE: D [g][M][N].  *_FWD: pre.  D*: dpre.  SGD: bf16 compute copy of the weights
  __nv_bfloat16* out1;  // *_FWD: hh [g][M][f_sub]
  const __nv_bfloat16* in0;   // DSWIGLU / DACT: pre
  float* master;        // SGD: fp32 master weights [g][M][N] (updated when lr != 0)
  float* dw;            // SGD: optional fp32 gradient dump [g][M][N]
  int* status;          // device status word
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ inline void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ inline void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ inline uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done;
}
__device__ inline uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait: gives up after ~2 s of wall time or as soon as another role of the CTA gave up.
__device__ inline bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0) {
      if (*abort_flag || global_timer_ns() - t0 > 2000000000ull) {
        *abort_flag = 1;
        atomicExch(status, (int)TWIST_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ inline void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ inline void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ inline void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ inline void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ inline void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (128-byte swizzle, descriptor version 1 of this architecture).
__device__ inline uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 256, operand majors as given.
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

__device__ inline float act_fwd(float x, int kind) {
  return kind == TWIST_FFN_RELU ? fmaxf(x, 0.f) : 0.5f * x * (1.f + erff(x * 0.70710678118654752f));
}
__device__ inline float act_grad(float x, int kind) {
  if (kind == TWIST_FFN_RELU) return x > 0.f ? 1.f : 0.f;
  return 0.5f * (1.f + erff(x * 0.70710678118654752f)) + x * 0.3989422804014327f * __expf(-0.5f * x * x);
}

// Tile index -> (group, m_tile, n_tile): groups outermost; inside a group, raster groups of
// kRasterGroupM m-tiles, n-tiles next, m-tiles innermost, so that concurrently running CTAs share
// a small set of A and B tiles in L2.
__device__ inline void tile_coords(const GemmParams& p, int tile, int& g, int& mt, int& nt) {
  const int per_group = p.m_tiles * p.n_tiles;
  g = tile / per_group;
  const int r = tile - g * per_group;
  const int band = r / (kRasterGroupM * p.n_tiles);
  const int m_first = band * kRasterGroupM;
  const int band_h = min(kRasterGroupM, p.m_tiles - m_first);
  const int rr = r - band * kRasterGroupM * p.n_tiles;
  nt = rr / band_h;
  mt = m_first + (rr - nt * band_h);
}

template <int A_MAJOR, int B_MAJOR, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  volatile uint32_t* ctrl = reinterpret_cast<volatile uint32_t*>(smem_gen + kStages * kStageBytes);
  // control block (in 4-byte words): full[4] @0, empty[4] @8, tmem_full[2] @16, tmem_empty[2] @20, tmem ptr @24, abort @25
  auto full_bar = [&](int i) { return bar_base + 8u * i; };
  auto empty_bar = [&](int i) { return bar_base + 8u * (kStages + i); };
  auto tfull_bar = [&](int i) { return bar_base + 8u * (2 * kStages + i); };
  auto tempty_bar = [&](int i) { return bar_base + 8u * (2 * kStages + 2 + i); };
  volatile uint32_t* tmem_slot = ctrl + 2 * (2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 2 * (2 * kStages + 4) + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = p.groups * p.m_tiles * p.n_tiles;
  const int num_kb = (p.K + kBK - 1) / kBK;

  if (warp == 4 && lane == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int i = 0; i < kStages; ++i) { mbar_init(full_bar(i), 1); mbar_init(empty_bar(i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        int g, mt, nt;
        tile_coords(p, tile, g, mt, nt);
        const int m0 = mt * kBM;
        const int n0 = nt * (EPI == EPI_SWIGLU_FWD ? kBN / 2 : kBN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int stage = it % kStages;
          const uint32_t phase = (it / kStages) & 1u;
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          const uint32_t bar = full_bar(stage);
          mbar_expect_tx(bar, kStageBytes);
          const uint32_t a_dst = smem_base + stage * kStageBytes;
          const uint32_t b_dst = a_dst + kABytes;
          const int k0 = kb * kBK;
          if (A_MAJOR == MAJOR_K) {
            tma_load_3d(a_dst, &tmA, bar, k0, m0, g);                       // box 64 (K) x 128 rows
          } else {
#pragma unroll
            for (int j = 0; j < kBM / 64; ++j) tma_load_3d(a_dst + j * 8192, &tmA, bar, m0 + 64 * j, k0, g);   // 64 (M) x 64 (K)
          }
          if (B_MAJOR == MAJOR_K) {
            const int r0 = n0;
            const int r1 = (EPI == EPI_SWIGLU_FWD) ? p.b_split + n0 : n0 + 128;
            tma_load_3d(b_dst, &tmB, bar, k0, r0, g);                       // box 64 (K) x 128 rows
            tma_load_3d(b_dst + 16384, &tmB, bar, k0, r1, g);
          } else {
#pragma unroll
            for (int j = 0; j < kBN / 64; ++j) tma_load_3d(b_dst + j * 8192, &tmB, bar, n0 + 64 * j, k0, g);   // 64 (N) x 64 (K)
          }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(A_MAJOR, B_MAJOR);
      constexpr uint32_t a_lbo = A_MAJOR == MAJOR_K ? 16u : (uint32_t)kBK * 128u;
      constexpr uint32_t b_lbo = B_MAJOR == MAJOR_K ? 16u : (uint32_t)kBK * 128u;
      constexpr uint32_t a_kstep = A_MAJOR == MAJOR_K ? (kUmmaK * 2) : (kUmmaK * 128);   // bytes per 16 of K
      constexpr uint32_t b_kstep = B_MAJOR == MAJOR_K ? (kUmmaK * 2) : (kUmmaK * 128);
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tl) {
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
          tc_commit(empty_bar(stage));          // frees the stage when these MMAs have read it
        }
        if (ok) tc_commit(tfull_bar(slot));     // accumulator complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 0..3
    uint32_t tl = 0;
    bool ok = true;
    for (int tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, ++tl) {
      int g, mt, nt;
      tile_coords(p, tile, g, mt, nt);
      const uint32_t slot = tl & 1u, acc_phase = (tl >> 1) & 1u;
      if (!mbar_wait(tfull_bar(slot), acc_phase, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const int row = mt * kBM + warp * 32 + lane;
      const bool row_ok = row < p.M;
      const uint32_t t_row = tmem_base + slot * kBN + ((uint32_t)(warp * 32) << 16);
      const long long grow = (long long)g * p.M + row;      // row index over all groups

      if (EPI == EPI_STORE) {
        const int n0 = nt * kBN;
        __nv_bfloat16* out = p.out0 + grow * p.N;
        for (int c = 0; c < kBN / 32; ++c) {
          const int n = n0 + 32 * c;
          if (n >= p.N) break;
          uint32_t r[32];
          tc_ld32(t_row + 32 * c, r);
          tc_wait_ld();
          if (row_ok) {
            uint32_t w[16];
#pragma unroll
            for (int q = 0; q < 16; ++q)
              w[q] = pack2(p.scale * __uint_as_float(r[2 * q]), p.scale * __uint_as_float(r[2 * q + 1]));
            store_row32(out + n, w, min(32, p.N - n));
          }
        }
      } else if (EPI == EPI_SWIGLU_FWD) {
        const int j0 = nt * (kBN / 2);
        const int f = p.N;
        __nv_bfloat16* pre = p.out0 + grow * (2LL * f);
        __nv_bfloat16* hh = p.out1 + grow * f;
        for (int c = 0; c < kBN / 64; ++c) {
          const int j = j0 + 32 * c;
          if (j >= f) break;
          uint32_t rg[32], ru[32];
          tc_ld32(t_row + 32 * c, rg);
          tc_ld32(t_row + kBN / 2 + 32 * c, ru);
          tc_wait_ld();
          if (row_ok) {
            uint32_t wg[16], wu[16], wh[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              const float g0 = __uint_as_float(rg[2 * q]), g1 = __uint_as_float(rg[2 * q + 1]);
              const float u0 = __uint_as_float(ru[2 * q]), u1 = __uint_as_float(ru[2 * q + 1]);
              wg[q] = pack2(g0, g1);
              wu[q] = pack2(u0, u1);
              wh[q] = pack2(g0 / (1.f + __expf(-g0)) * u0, g1 / (1.f + __expf(-g1)) * u1);
            }
            const int valid = min(32, f - j);
            store_row32(pre + j, wg, valid);
            store_row32(pre + f + j, wu, valid);
            store_row32(hh + j, wh, valid);
          }
        }
      } else if (EPI == EPI_ACT_FWD) {
        const int n0 = nt * kBN;
        __nv_bfloat16* pre = p.out0 + grow * p.N;
        __nv_bfloat16* hh = p.out1 + grow * p.N;
        for (int c = 0; c < kBN / 32; ++c) {
          const int n = n0 + 32 * c;
          if (n >= p.N) break;
          uint32_t r[32];
          tc_ld32(t_row + 32 * c, r);
          tc_wait_ld();
          if (row_ok) {
            uint32_t wp[16], wh[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              const float a0 = __uint_as_float(r[2 * q]), a1 = __uint_as_float(r[2 * q + 1]);
              wp[q] = pack2(a0, a1);
              wh[q] = pack2(act_fwd(a0, p.act_kind), act_fwd(a1, p.act_kind));
            }
            const int valid = min(32, p.N - n);
            store_row32(pre + n, wp, valid);
            store_row32(hh + n, wh, valid);
          }
        }
      } else if (EPI == EPI_DSWIGLU) {
        const int n0 = nt * kBN;
        const int f = p.N;
        const __nv_bfloat16* pre = p.in0 + grow * (2LL * f);
        __nv_bfloat16* dpre = p.out0 + grow * (2LL * f);
        for (int c = 0; c < kBN / 32; ++c) {
          const int j = n0 + 32 * c;
          if (j >= f) break;
          uint32_t r[32];
          tc_ld32(t_row + 32 * c, r);
          tc_wait_ld();
          if (row_ok) {
            const int valid = min(32, f - j);
            uint32_t pg[16], pu[16], wg[16], wu[16];
            load_row32(pre + j, pg, valid);
            load_row32(pre + f + j, pu, valid);
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              float dg[2], du[2];
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const float dh = p.scale * __uint_as_float(r[2 * q + h]);
                const float gt = h ? bf_hi(pg[q]) : bf_lo(pg[q]);
                const float up = h ? bf_hi(pu[q]) : bf_lo(pu[q]);
                const float sg = 1.f / (1.f + __expf(-gt));
                dg[h] = dh * up * (sg * (1.f + gt * (1.f - sg)));
                du[h] = dh * (gt * sg);
              }
              wg[q] = pack2(dg[0], dg[1]);
              wu[q] = pack2(du[0], du[1]);
            }
            store_row32(dpre + j, wg, valid);
            store_row32(dpre + f + j, wu, valid);
          }
        }
      } else if (EPI == EPI_DACT) {
        const int n0 = nt * kBN;
        const __nv_bfloat16* pre = p.in0 + grow * p.N;
        __nv_bfloat16* dpre = p.out0 + grow * p.N;
        for (int c = 0; c < kBN / 32; ++c) {
          const int n = n0 + 32 * c;
          if (n >= p.N) break;
          uint32_t r[32];
          tc_ld32(t_row + 32 * c, r);
          tc_wait_ld();
          if (row_ok) {
            const int valid = min(32, p.N - n);
            uint32_t pp[16], w[16];
            load_row32(pre + n, pp, valid);
#pragma unroll
            for (int q = 0; q < 16; ++q)
              w[q] = pack2(p.scale * __uint_as_float(r[2 * q]) * act_grad(bf_lo(pp[q]), p.act_kind),
                           p.scale * __uint_as_float(r[2 * q + 1]) * act_grad(bf_hi(pp[q]), p.act_kind));
            store_row32(dpre + n, w, valid);
          }
        }
      } else {   // EPI_SGD: acc = dW tile; master -= lr * scale * acc; compute copy = bf16(master)
        const int n0 = nt * kBN;
        float* master = p.master + grow * p.N;
        float* dw = p.dw ? p.dw + grow * p.N : nullptr;
        __nv_bfloat16* w16 = p.out0 + grow * p.N;
        for (int c = 0; c < kBN / 32; ++c) {
          const int n = n0 + 32 * c;
          if (n >= p.N) break;
          uint32_t r[32];
          tc_ld32(t_row + 32 * c, r);
          tc_wait_ld();
          if (row_ok) {
            const int valid = min(32, p.N - n);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              if (4 * q < valid) {
                float4 gq = make_float4(p.scale * __uint_as_float(r[4 * q]), p.scale * __uint_as_float(r[4 * q + 1]),
                                        p.scale * __uint_as_float(r[4 * q + 2]), p.scale * __uint_as_float(r[4 * q + 3]));
                if (dw) *reinterpret_cast<float4*>(dw + n + 4 * q) = gq;
                if (p.lr != 0.f) {
                  float4 m = *reinterpret_cast<const float4*>(master + n + 4 * q);
                  m.x -= p.lr * gq.x; m.y -= p.lr * gq.y; m.z -= p.lr * gq.z; m.w -= p.lr * gq.w;
                  *reinterpret_cast<float4*>(master + n + 4 * q) = m;
                  *reinterpret_cast<uint2*>(w16 + n + 4 * q) = make_uint2(pack2(m.x, m.y), pack2(m.z, m.w));
                }
              }
            }
          }
        }
      }
      // accumulator slot free again
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(slot));
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait expired: give copies that may still be in flight time to land before shared memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
  }
}

// Host side ------------------------------------------------------------------------------------

struct GemmOperand {
  const void* ptr;     // dense bf16 [groups][rows][cols]
  int rows, cols;
};

// layout: 0 NT, 1 NN, 2 TN.  Returns a TWIST_* status.
int launch_gemm_bf16(int layout, int epi, const GemmOperand& A, const GemmOperand& B, GemmParams p, cudaStream_t st);

}  // namespace twist
