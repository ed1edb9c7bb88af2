// Tensor-core forward of the attention core (App. A: head_h = softmax(Q_h K_h^T / sqrt(d_head)) V_h, causal per
// sequence) for d_head = 64, on tcgen05 with accumulators in tensor memory.
//
// One CTA per (block of 128 queries, kept head, sequence).  K and V arrive by TMA in tiles of 128 keys (K-major,
// 128-byte swizzle); the unit of S, P and the softmax is a half block of 64 keys:
//   S = Q K^T        one 128 x 64 x 64 MMA chain per half block into one of two S buffers in tensor memory, issued two
//                    half blocks ahead: the threads do not wait for it
//   softmax          thread = query row: the 64 scores are read from tensor memory once and stay in registers
//                    (maximum, exponentials), running maximum / sum kept in registers, P written to one of two P
//                    buffers in tensor memory (bf16 pairs, lane = query row) as the A operand of the next MMA: it
//                    never passes through shared memory, whose bandwidth the operand reads of the MMAs already load
//   O += P V         128 x 64 x 64 MMA chain accumulating in tensor memory, V as the MN-major B operand (rows =
//                    keys as they lie in memory); runs while the threads are at the next half block
// P and O are expressed relative to a reference maximum that follows the running maximum lazily: only when a
// row's maximum has grown by more than kRescaleLog2 since the reference was set does its warp rescale O in
// tensor memory (and the running sum), after waiting for the O += P V issued so far; otherwise
// P = 2^(s - ref) <= 2^kRescaleLog2 simply accumulates.  O / l is the same quotient for any reference.  The threads
// therefore never read an output block: per half block they read S, write P and go on.
// Warps 0-3: softmax / output; warp 4, one lane: TMA and MMA issue.
// Backward (same tile sizes; probabilities recomputed from the stored log-sum-exp, dS = P (dP - delta)):
//   dQ kernel     one CTA per query block: per key block S = Q K^T and dP = dO V^T into tensor memory, the threads
//                 write dS (bf16 pairs) into tensor memory as the A operand, dQ += dS K accumulates in tensor memory
//                 over the key blocks.
//   dK/dV kernel  one CTA per (key block, KV position): for every kept head that reads the position and every
//                 query block at or after the key block, the transposed tiles S^T = K Q^T and dP^T = V dO^T (rows =
//                 keys), the threads write P^T and dS^T back into tensor memory as A operands, and dV += P^T dO,
//                 dK += dS^T Q accumulate in tensor memory.
// No probability or score gradient ever passes through shared memory: its bandwidth is what the operand reads of
// the MMAs need.
// Every wait is bounded; on expiry the CTA records TWIST_ERR_DEVICE_TIMEOUT and leaves.
#include "attn_core.cuh"
#include "ptx.cuh"

namespace twist {
namespace {

constexpr int kDh = 64;                 // head dimension of this kernel
constexpr int kBq = 128, kBk = 128;     // queries per CTA, keys per block
constexpr int kTileBytes = 128 * kDh * 2;            // a 128-row tile of Q, K or V: 16 KB
constexpr int kFwdThreads = 160;
constexpr int kFwdSmem = kTileBytes * 5 + 1024 + 256;   // Q, K[2], V[2], alignment, barriers: two CTAs per SM
constexpr int kHalf = 64;                // forward: keys per S / P half block
constexpr int kFwdTmemCols = 256;       // S halves: columns 0..63 and 64..127, O: 128..191, P halves (bf16 pairs): 192..223, 224..255
constexpr float kRescaleLog2 = 8.f;     // growth of a row maximum (log2 domain) tolerated before O is rescaled

__device__ inline void mma1(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// A operand in tensor memory (lane = row of A, two 16-bit elements of the contraction per 32-bit column)
__device__ inline void mma1_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ inline void commit1(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// fp32 accumulate, bf16 x bf16, M x N tile, operand majors (0: K-major, 1: MN-major)
__host__ __device__ constexpr uint32_t idesc_bf16(int a_major, int b_major, int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_major << 15) | ((uint32_t)b_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ inline uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
// 2^x by the special-function unit (about 2 ulp, flushes denormals, 2^-inf = 0): exp2f() would wrap the same
// instruction in range fix-ups that cost more issue slots than the rest of the softmax.
__device__ inline float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Softmax of one half block (64 keys) for this thread's query row.  The 64 scores are read from tensor memory once
// and stay in registers through the maximum, the (rare) rescale and the exponentials; m is the reference maximum
// (log2 domain), l the sum relative to it; P = 2^(s * scale - m) goes (bf16 pairs) into the A operand in tensor
// memory.  MASKED: only columns <= k_lim are visible (the diagonal block; k_lim may be negative); the other blocks
// carry no per-element predicate.  `p_free()` is called (by the whole warp) before P is overwritten, `rescale(corr)`
// when some row of the warp moves its reference: it multiplies the row's O by corr.
template <bool MASKED, typename PFree, typename Rescale>
__device__ inline bool softmax_half(uint32_t t_s, uint32_t t_p, int k_lim, float scale_log2, float& m, float& l,
                                    PFree&& p_free, Rescale&& rescale) {
  uint32_t va[32], vb[32];
  tc_ld32(t_s, va);
  tc_ld32(t_s + 32, vb);
  tc_wait_ld();
  float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
#pragma unroll
  for (int i = 0; i < 32; ++i)
    if (!MASKED || i <= k_lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(va[i]));
#pragma unroll
  for (int i = 0; i < 32; ++i)
    if (!MASKED || 32 + i <= k_lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(vb[i]));
  const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
  const float m_blk = mx * scale_log2;                 // scale > 0: the maximum commutes with the scaling
  if (!p_free()) return false;                         // warp-uniform
  if (__any_sync(0xffffffffu, m_blk > m + kRescaleLog2)) {
    const float m_new = fmaxf(m, m_blk);
    const float corr = ex2_fast(m - m_new);            // 0 for a first block (m = -inf), 1 where nothing moved
    l *= corr;
    m = m_new;
    if (!rescale(corr)) return false;
  }
  float sum4[4] = {0.f, 0.f, 0.f, 0.f};
  auto emit = [&](const uint32_t (&v)[32], int c) {
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      float p0 = ex2_fast(fmaf(__uint_as_float(v[2 * i]), scale_log2, -m));
      float p1 = ex2_fast(fmaf(__uint_as_float(v[2 * i + 1]), scale_log2, -m));
      if (MASKED) {
        p0 = (32 * c + 2 * i <= k_lim) ? p0 : 0.f;
        p1 = (32 * c + 2 * i + 1 <= k_lim) ? p1 : 0.f;
      }
      sum4[i & 3] += p0 + p1;
      w[i] = pack2(p0, p1);
    }
    tc_st16(t_p + 16 * c, w);                          // 32 keys = 16 columns of packed bf16 pairs
  };
  emit(va, 0);
  emit(vb, 1);
  tc_wait_st();
  l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
  return true;
}

// Stores 32 accumulator columns (scaled) of this thread's row as bf16.
__device__ inline void store_acc32(__nv_bfloat16* dst, const uint32_t (&v)[32], float sc) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4)
    d[q4] = make_uint4(pack2(sc * __uint_as_float(v[8 * q4]), sc * __uint_as_float(v[8 * q4 + 1])),
                       pack2(sc * __uint_as_float(v[8 * q4 + 2]), sc * __uint_as_float(v[8 * q4 + 3])),
                       pack2(sc * __uint_as_float(v[8 * q4 + 4]), sc * __uint_as_float(v[8 * q4 + 5])),
                       pack2(sc * __uint_as_float(v[8 * q4 + 6]), sc * __uint_as_float(v[8 * q4 + 7])));
}

// qkv viewed as [S * n_seqs][seq_len][nq]: rows past the end of a sequence read as zeros.
__global__ void __maxnreg__(200) attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQKV,
                                                                     const AttnParams p, int* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_s = base, k_s = base + kTileBytes, v_s = base + 3 * kTileBytes;
  const uint32_t bar0 = base + 5 * kTileBytes;
  volatile uint32_t* ctrl = reinterpret_cast<volatile uint32_t*>(gen + 5 * kTileBytes);
  // Two CTAs share an SM (their startup, softmax and MMA phases interleave); K and V are double-buffered.
  // barriers (8 bytes each): 0 q_full, 1-2 k_full, 3-4 v_full, 5-6 v_free, 7-8 s_full, 9-10 p_ready, 11-12 pv_done;
  // then the TMEM base address and the abort flag
  enum { Q_FULL = 0, K_FULL = 1, V_FULL = 3, V_FREE = 5, S_FULL = 7, P_READY = 9, PV_DONE = 11, N_BARS = 13 };
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = ctrl + 32;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 33);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qb = blockIdx.x, hq = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int nblk = qb + 1;                               // causal: key blocks 0 .. qb
  const int n_half = 2 * nblk;                           // half blocks of 64 keys: the unit of S, P and the softmax
  if (threadIdx.x == 128) {
    tma_prefetch_desc(&tmQKV);
    for (int i = 0; i < N_BARS; ++i) mbar_init(bar(i), (i == P_READY || i == P_READY + 1) ? 128 : 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kFwdTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_s = tmem, tm_o = tmem + 128, tm_p = tmem + 192;

  if (warp == 4) {
    if (lane == 0) {
      const int kvp = kv_position(p, s, hq);
      const int z = blockIdx.z;
      const int k_col = p.a_sub + kvp * kDh, v_col = k_col + p.kv_max * kDh;
      auto load_k = [&](int j) {
        const int st = j & 1;
        mbar_expect_tx(bar(K_FULL + st), kTileBytes);
        tma_load_3d_local(k_s + st * kTileBytes, &tmQKV, bar(K_FULL + st), k_col, j * kBk, z);
      };
      auto load_v = [&](int j) {
        const int st = j & 1;
        mbar_expect_tx(bar(V_FULL + st), kTileBytes);
        tma_load_3d_local(v_s + st * kTileBytes, &tmQKV, bar(V_FULL + st), v_col, j * kBk, z);
      };
      mbar_expect_tx(bar(Q_FULL), kTileBytes);
      tma_load_3d_local(q_s, &tmQKV, bar(Q_FULL), hq * kDh, qb * kBq, z);
      load_k(0);
      load_v(0);
      if (nblk > 1) { load_k(1); load_v(1); }
      constexpr uint32_t idesc_s = idesc_bf16(0, 0, kBq, kHalf);     // S = Q K^T : both K-major
      constexpr uint32_t idesc_o = idesc_bf16(0, 1, kBq, kDh);       // O = P V   : V MN-major
      // S of half block hb: Q against key rows 64 (hb & 1) .. of tile hb / 2 (64 rows of 128 bytes = 8 KB further on)
      auto mma_s = [&](int hb) {
        const uint64_t a = smem_desc(q_s, 16u, 1024u);
        const uint64_t bd = smem_desc(k_s + ((hb >> 1) & 1) * kTileBytes + (hb & 1) * (kHalf * 128), 16u, 1024u);
#pragma unroll
        for (int k = 0; k < kDh / 16; ++k) mma1(tm_s + (uint32_t)(hb & 1) * kHalf, a + 2u * k, bd + 2u * k, idesc_s, k != 0);
        commit1(bar(S_FULL + (hb & 1)));
      };
      bool ok = mbar_wait_cta(bar(Q_FULL), 0, abort_flag, status) && mbar_wait_cta(bar(K_FULL), 0, abort_flag, status);
      if (ok) {
        tc_fence_after();
        mma_s(0);
        mma_s(1);
      }
      for (int hb = 0; ok && hb < n_half; ++hb) {
        const int j = hb >> 1, st = j & 1, h = hb & 1;
        // P of half block hb is in tensor memory and S(hb) has been read: its S columns are free, and after the
        // second half so is K(j)'s buffer
        if (!mbar_wait_cta(bar(P_READY + h), (hb >> 1) & 1, abort_flag, status)) break;
        tc_fence_after();
        if (h == 1 && j + 2 < nblk) load_k(j + 2);
        if (h == 0 && !mbar_wait_cta(bar(V_FULL + st), (j >> 1) & 1, abort_flag, status)) break;     // V of block j
        tc_fence_after();
        const uint64_t bd = smem_desc(v_s + st * kTileBytes, (uint32_t)kDh * 128u, 1024u);
#pragma unroll
        for (int k = 0; k < kHalf / 16; ++k)                                      // 16 keys = 8 columns of P
          mma1_ta(tm_o, tm_p + (uint32_t)h * (kHalf / 2) + 8u * k, bd + (uint64_t)(((4 * h + k) * 16 * 128) >> 4), idesc_o,
                  (hb | k) != 0);
        commit1(bar(PV_DONE + h));                                                // P(hb) consumed
        // S two half blocks ahead, into the buffer the threads have just read: they never wait for it.  Issued after
        // O += P V of this half block, so that its completion (S_FULL) also tells the threads that P (hb & 1) has been
        // read and may be overwritten.
        if (hb + 2 < n_half) {
          if (h == 0 && !mbar_wait_cta(bar(K_FULL + ((j + 1) & 1)), ((j + 1) >> 1) & 1, abort_flag, status)) break;
          tc_fence_after();
          mma_s(hb + 2);
        }
        if (h == 1) {
          commit1(bar(V_FREE + st));                                              // V buffer free
          if (j + 2 < nblk) {
            if (!mbar_wait_cta(bar(V_FREE + st), (j >> 1) & 1, abort_flag, status)) break;
            load_v(j + 2);
          }
        }
      }
    }
  } else {
    // ---- softmax warps: thread = query row
    const int r = warp * 32 + lane;
    const int qi = qb * kBq + r;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const uint32_t t_s = tm_s + lane_off, t_o = tm_o + lane_off, t_p = tm_p + lane_off;
    float m = -INFINITY, l = 0.f;
    bool ok = true;
    for (int hb = 0; hb < n_half; ++hb) {
      const int h = hb & 1;
      if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(S_FULL + h), (hb >> 1) & 1, abort_flag, status))) { ok = false; break; }
      tc_fence_after();
      // P (hb & 1) may be overwritten: O += P V of half block hb - 2 was issued before S(hb), whose completion the
      // warp has just seen
      auto p_free = [&]() { return true; };
      // whole warp: O row *= corr in tensor memory, once every O += P V issued so far is complete (the latest is that
      // of half block hb - 1; the next one is not issued before this warp has delivered P(hb))
      auto rescale = [&](float corr) {
        if (hb == 0) return true;                        // nothing accumulated yet
        if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(PV_DONE + ((hb - 1) & 1)), ((hb - 1) >> 1) & 1, abort_flag, status)))
          return false;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < kDh / 32; ++c) {
          uint32_t v[32];
          tc_ld32(t_o + 32 * c, v);
          tc_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * corr);
          tc_st32(t_o + 32 * c, v);
        }
        tc_wait_st();
        return true;
      };
      bool fine;
      const uint32_t ts = t_s + (uint32_t)h * kHalf, tp = t_p + (uint32_t)h * (kHalf / 2);
      if ((hb >> 1) == qb) fine = softmax_half<true>(ts, tp, qi - (hb >> 1) * kBk - h * kHalf, p.scale_log2, m, l, p_free, rescale);
      else fine = softmax_half<false>(ts, tp, kHalf, p.scale_log2, m, l, p_free, rescale);
      if (!fine) { ok = false; break; }
      tc_fence_before();
      mbar_arrive(bar(P_READY + h));
    }
    // the last O += P V (and with it every earlier one) complete
    if (ok && __all_sync(0xffffffffu, mbar_wait_cta(bar(PV_DONE + ((n_half - 1) & 1)), ((n_half - 1) >> 1) & 1, abort_flag, status))) {
      tc_fence_after();
      const float inv = 1.f / l;
      const long long row = (long long)s * p.T + (long long)b * p.seq_len + qi;
#pragma unroll
      for (int c = 0; c < kDh / 32; ++c) {
        uint32_t v[32];
        tc_ld32(t_o + 32 * c, v);
        tc_wait_ld();
        if (qi < p.seq_len) store_acc32(p.out + row * p.a_sub + hq * kDh + 32 * c, v, inv);
      }
      if (qi < p.seq_len)
        p.lse[((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len + qi] = (m + log2f(l)) * 0.6931471805599453f;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {     // a wait expired: let copies that may still be in flight land before shared memory is released
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 4) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kFwdTmemCols) : "memory");
  }
}

constexpr int kBwdTmemCols = 512;
constexpr int kBwdThreads = 288;        // 8 element-wise warps (two per tensor-memory lane quarter) + the control warp

// Element-wise steps of the dQ kernel, for this thread's query row and its 64 key columns (chunks c0 and c0 + 1 of 32
// columns).  They are split so that the tensor pipe can work on dP while the threads are busy with the exponentials:
//   probs_from_s   P = exp2(S * scale - lse2) where visible (column <= k_lim), kept in registers (fp32);
//   ds_from_dp     dS = P * (dP - dl), packed bf16 pairs into tensor memory at column 16 c of `ds` (the A operand of
//                  dQ += dS K).
template <bool MASKED>
__device__ inline void probs_from_s(uint32_t t_s, int c0, int k_lim, float scale_log2, float lse2, float (&pr)[64]) {
  uint32_t va[32], vb[32];
  tc_ld32(t_s + 32 * c0, va);
  tc_wait_ld();
  tc_ld32(t_s + 32 * (c0 + 1), vb);
  auto chunk = [&](const uint32_t (&v)[32], int cc) {
    const int c = c0 + cc;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      float x = ex2_fast(fmaf(__uint_as_float(v[i]), scale_log2, -lse2));
      if (MASKED) x = (32 * c + i <= k_lim) ? x : 0.f;
      pr[32 * cc + i] = x;
    }
  };
  chunk(va, 0);
  tc_wait_ld();
  chunk(vb, 1);
}
__device__ inline void ds_from_dp(uint32_t t_dp, int c0, float dl, uint32_t ds, const float (&pr)[64]) {
  uint32_t va[32], vb[32];
  tc_ld32(t_dp + 32 * c0, va);
  tc_wait_ld();
  tc_ld32(t_dp + 32 * (c0 + 1), vb);
  auto chunk = [&](const uint32_t (&v)[32], int cc) {
    uint32_t w[16];
#pragma unroll
    for (int e = 0; e < 16; ++e)
      w[e] = pack2(pr[32 * cc + 2 * e] * (__uint_as_float(v[2 * e]) - dl),
                   pr[32 * cc + 2 * e + 1] * (__uint_as_float(v[2 * e + 1]) - dl));
    tc_st16(ds + 16 * (c0 + cc), w);
  };
  chunk(va, 0);
  tc_wait_ld();
  chunk(vb, 1);
  tc_wait_st();
}

// ---- dQ: grid (query blocks, kept heads, S * n_seqs).  Per key block j: S = Q K^T and dP = dO V^T (128 x 128)
// into tensor memory, the threads write dS (bf16 pairs) into tensor memory as the A operand, dQ += dS K accumulates
// in tensor memory.
// S is double-buffered in tensor memory and issued two blocks ahead, dP one block ahead right after the threads
// released it, so both are complete before the threads need them: the threads turn S(j) into probabilities (the
// expensive half of their work) while dP(j) is still being computed.  K / V blocks are triple-buffered.
constexpr int kDqStages = 3;
constexpr int kDqSmem = kTileBytes * (2 + 2 * kDqStages) + 1024 + 256;    // Q, dO, K[3], V[3]
__global__ void __launch_bounds__(kBwdThreads) attn_dq_tc_kernel(const __grid_constant__ CUtensorMap tmQKV,
                                                                 const __grid_constant__ CUtensorMap tmDO,
                                                                 const AttnParams p, int* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t q_s = base, do_s = base + kTileBytes, k_s = base + 2 * kTileBytes,
                 v_s = k_s + kDqStages * kTileBytes;
  const uint32_t bar0 = v_s + kDqStages * kTileBytes;
  volatile uint32_t* ctrl = reinterpret_cast<volatile uint32_t*>(gen + (2 + 2 * kDqStages) * kTileBytes);
  // barriers: 0 q_full, 1-3 kv_full, 4-6 kv_free, 7-8 s_full, 9 dp_full, 10 ds_ready, 11 dq_full
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = ctrl + 32;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 33);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qb = blockIdx.x, hq = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int nblk = qb + 1;
  if (threadIdx.x == 256) {
    tma_prefetch_desc(&tmQKV);
    tma_prefetch_desc(&tmDO);
    for (int i = 0; i < 12; ++i) mbar_init(bar(i), i == 10 ? 256 : 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kBwdTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_dp = tmem + 256, tm_dq = tmem + 384, tm_ds = tmem + 448;      // S(j) at columns 128 (j & 1)

  if (warp == 8) {
    if (lane == 0) {
      const int kvp = kv_position(p, s, hq);
      const int z = blockIdx.z;
      const int k_col = p.a_sub + kvp * kDh, v_col = k_col + p.kv_max * kDh;
      auto load_kv = [&](int j) {
        const int st = j % kDqStages;
        mbar_expect_tx(bar(1 + st), 2 * kTileBytes);
        tma_load_3d_local(k_s + st * kTileBytes, &tmQKV, bar(1 + st), k_col, j * kBk, z);
        tma_load_3d_local(v_s + st * kTileBytes, &tmQKV, bar(1 + st), v_col, j * kBk, z);
      };
      mbar_expect_tx(bar(0), 2 * kTileBytes);
      tma_load_3d_local(q_s, &tmQKV, bar(0), hq * kDh, qb * kBq, z);
      tma_load_3d_local(do_s, &tmDO, bar(0), hq * kDh, qb * kBq, z);
      for (int j = 0; j < kDqStages && j < nblk; ++j) load_kv(j);
      constexpr uint32_t idesc_s = idesc_bf16(0, 0, kBq, kBk);       // S = Q K^T, dP = dO V^T : both K-major
      constexpr uint32_t idesc_q = idesc_bf16(0, 1, kBq, kDh);       // dQ = dS K : K as the MN-major B operand
      auto mma_s = [&](int j) {
        const uint64_t aq = smem_desc(q_s, 16u, 1024u), bk = smem_desc(k_s + (j % kDqStages) * kTileBytes, 16u, 1024u);
#pragma unroll
        for (int k = 0; k < kDh / 16; ++k) mma1(tmem + 128u * (j & 1), aq + 2u * k, bk + 2u * k, idesc_s, k != 0);
        commit1(bar(7 + (j & 1)));
      };
      auto mma_dp = [&](int j) {
        const uint64_t ao = smem_desc(do_s, 16u, 1024u), bv = smem_desc(v_s + (j % kDqStages) * kTileBytes, 16u, 1024u);
#pragma unroll
        for (int k = 0; k < kDh / 16; ++k) mma1(tm_dp, ao + 2u * k, bv + 2u * k, idesc_s, k != 0);
        commit1(bar(9));
      };
      bool ok = mbar_wait_cta(bar(0), 0, abort_flag, status) && mbar_wait_cta(bar(1), 0, abort_flag, status);
      if (ok) {
        tc_fence_after();
        mma_s(0);
        mma_dp(0);
        if (nblk > 1) {
          ok = mbar_wait_cta(bar(2), 0, abort_flag, status);
          if (ok) {
            tc_fence_after();
            mma_s(1);
          }
        }
      }
      for (int j = 0; ok && j < nblk; ++j) {
        const int st = j % kDqStages;
        // dS(j) is in tensor memory; S(j) and dP(j) have been read (the threads read S before dP)
        if (!mbar_wait_cta(bar(10), j & 1, abort_flag, status)) break;
        tc_fence_after();
        const uint64_t bd = smem_desc(k_s + st * kTileBytes, (uint32_t)kDh * 128u, 1024u);
#pragma unroll
        for (int k = 0; k < kBk / 16; ++k)               // 16 keys = 8 columns of dS
          mma1_ta(tm_dq, tm_ds + 8u * k, bd + (uint64_t)((k * 16 * 128) >> 4), idesc_q, (j | k) != 0);
        commit1(bar(4 + st));                            // block j's K / V are consumed
        if (j + 1 == nblk) commit1(bar(11));
        // dP of the next block after dQ of this one: its commit then also tells the threads that dS may be rewritten
        // (block j + 1 arrived before S(j + 1) was issued)
        if (j + 1 < nblk) mma_dp(j + 1);
        if (j + 2 < nblk) {
          const int j2 = j + 2;
          if (!mbar_wait_cta(bar(1 + j2 % kDqStages), (j2 / kDqStages) & 1, abort_flag, status)) break;
          tc_fence_after();
          mma_s(j2);                                     // into the buffer S(j) has just left
        }
        if (j + kDqStages < nblk) {
          if (!mbar_wait_cta(bar(4 + st), (j / kDqStages) & 1, abort_flag, status)) break;
          load_kv(j + kDqStages);
        }
      }
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane;
    const int qi = qb * kBq + r;
    const bool row_ok = qi < p.seq_len;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const long long stat = ((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len + qi;
    const float lse2 = row_ok ? p.lse[stat] * 1.4426950408889634f : 0.f;
    const float dl = row_ok ? p.delta[stat] : 0.f;
    bool ok = true;
    for (int j = 0; j < nblk; ++j) {
      float pr[64];
      if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(7 + (j & 1)), (j >> 1) & 1, abort_flag, status))) { ok = false; break; }
      tc_fence_after();
      const int k_lim = !row_ok ? -1 : ((j == qb) ? qi - j * kBk : kBk);
      const uint32_t t_s = tmem + lane_off + 128u * (j & 1);
      if (__any_sync(0xffffffffu, k_lim < kBk))      // warp-uniform: the tensor-memory loads inside are warp-wide
        probs_from_s<true>(t_s, 2 * half, k_lim, p.scale_log2, lse2, pr);
      else
        probs_from_s<false>(t_s, 2 * half, k_lim, p.scale_log2, lse2, pr);
      if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(9), j & 1, abort_flag, status))) { ok = false; break; }
      tc_fence_after();
      ds_from_dp(tm_dp + lane_off, 2 * half, dl, tm_ds + lane_off, pr);
      tc_fence_before();
      mbar_arrive(bar(10));
    }
    if (ok && __all_sync(0xffffffffu, mbar_wait_cta(bar(11), 0, abort_flag, status))) {
      tc_fence_after();
      uint32_t v[32];
      tc_ld32(tm_dq + lane_off + 32 * half, v);
      tc_wait_ld();
      if (row_ok) {
        const long long row = (long long)s * p.T + (long long)b * p.seq_len + qi;
        store_acc32(p.d_qkv + row * p.nq + hq * kDh + 32 * half, v, p.scale_log2 * 0.6931471805599453f);   // / sqrt(d_head)
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kBwdTmemCols) : "memory");
  }
}

// ---- dK, dV: grid (key blocks, KV positions, S * n_seqs).  Units (kept head, query block) stream through with the
// same schedule as the dQ kernel (S two units ahead, dP one).  The score tiles are computed with the keys as rows, S^T = K Q^T and dP^T = V dO^T (128 keys x 128 queries), so that the thread that owns
// tensor-memory lane r owns key r: the probabilities it forms are rows of P^T and dS^T, which is exactly the A operand
// of dV += P^T dO and dK += dS^T Q.  They are written back into tensor memory (packed bf16 pairs, over the first half
// of the thread's own 64 score columns) and never touch shared memory; the softmax statistics, now per column, are
// staged in shared memory once per unit.  Per unit the MMAs read 96 KB of operands from shared memory instead of 160
// KB and the threads write none.
constexpr int kDkvStages = 3;
constexpr int kDkvSmem = kTileBytes * (2 + 2 * kDkvStages) + 1024 + 256;   // K, V, Q[3], dO[3]

// Thread = key row r, 64 query columns starting at col0 (= 64 (warp >> 2)); `stat` = shared-memory address of the 64
// per-query values (log-sum-exp in the log2 domain, +inf for queries past the sequence end).  P^T goes to registers
// and, packed, to columns 0..31 of the thread's own score columns at t_s.
template <bool MASKED>
__device__ inline void probs_from_st(uint32_t t_s, uint32_t stat, int r, int col0, float scale_log2, float (&pr)[64]) {
  uint32_t va[32], vb[32];
  tc_ld32(t_s, va);
  tc_wait_ld();
  tc_ld32(t_s + 32, vb);
  auto chunk = [&](const uint32_t (&v)[32], int cc) {
#pragma unroll
    for (int q4 = 0; q4 < 8; ++q4) {
      const uint4 lv = lds128(stat + 16u * (8 * cc + q4));
      const float l4[4] = {__uint_as_float(lv.x), __uint_as_float(lv.y), __uint_as_float(lv.z), __uint_as_float(lv.w)};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int i = 4 * q4 + e;
        float x = ex2_fast(fmaf(__uint_as_float(v[i]), scale_log2, -l4[e]));
        if (MASKED) x = (col0 + 32 * cc + i >= r) ? x : 0.f;       // causal: key <= query
        pr[32 * cc + i] = x;
      }
    }
    uint32_t w[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) w[e] = pack2(pr[32 * cc + 2 * e], pr[32 * cc + 2 * e + 1]);
    tc_st16(t_s + 16 * cc, w);          // over score columns this thread has already read
  };
  chunk(va, 0);
  tc_wait_ld();
  chunk(vb, 1);
}
// dS^T = P^T * (dP^T - delta[query]), packed over the first half of the thread's own dP^T columns.
__device__ inline void ds_from_dpt(uint32_t t_dp, uint32_t stat, const float (&pr)[64]) {
  uint32_t va[32], vb[32];
  tc_ld32(t_dp, va);
  tc_wait_ld();
  tc_ld32(t_dp + 32, vb);
  auto chunk = [&](const uint32_t (&v)[32], int cc) {
    uint32_t w[16];
#pragma unroll
    for (int q4 = 0; q4 < 8; ++q4) {
      const uint4 dv = lds128(stat + 16u * (8 * cc + q4));
      const int i = 4 * q4;
      w[2 * q4] = pack2(pr[32 * cc + i] * (__uint_as_float(v[i]) - __uint_as_float(dv.x)),
                        pr[32 * cc + i + 1] * (__uint_as_float(v[i + 1]) - __uint_as_float(dv.y)));
      w[2 * q4 + 1] = pack2(pr[32 * cc + i + 2] * (__uint_as_float(v[i + 2]) - __uint_as_float(dv.z)),
                            pr[32 * cc + i + 3] * (__uint_as_float(v[i + 3]) - __uint_as_float(dv.w)));
    }
    tc_st16(t_dp + 16 * cc, w);
  };
  chunk(va, 0);
  tc_wait_ld();
  chunk(vb, 1);
  tc_wait_st();
}

__global__ void __launch_bounds__(kBwdThreads) attn_dkv_tc_kernel(const __grid_constant__ CUtensorMap tmQKV,
                                                                    const __grid_constant__ CUtensorMap tmDO,
                                                                    const AttnParams p, int* status) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ int match[64];
  __shared__ int n_match_s;
  __shared__ __align__(16) float stat_w[8][2][64];       // per element-wise warp: [lse2 | delta][its 64 queries]
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t k_s = base, v_s = base + kTileBytes, q_s = base + 2 * kTileBytes, do_s = q_s + kDkvStages * kTileBytes;
  const uint32_t bar0 = do_s + kDkvStages * kTileBytes;
  volatile uint32_t* ctrl = reinterpret_cast<volatile uint32_t*>(gen + (2 + 2 * kDkvStages) * kTileBytes);
  // barriers: 0 kv_full, 1-3 q_full, 4-6 q_free, 7-8 s_full, 9 dp_full, 10 pds_ready, 11 acc_full
  auto bar = [&](int i) { return bar0 + 8u * i; };
  volatile uint32_t* tmem_slot = ctrl + 32;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 33);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kb = blockIdx.x, kvp = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int nqb = (p.seq_len + kBq - 1) / kBq;
  const int held = p.kv_count ? p.kv_count[s] : p.kv_max;
  if (threadIdx.x == 256) {
    tma_prefetch_desc(&tmQKV);
    tma_prefetch_desc(&tmDO);
    for (int i = 0; i < 12; ++i) mbar_init(bar(i), i == 10 ? 256 : 1);
    *abort_flag = 0;
    int n = 0;
    if (kvp < held)
      for (int hq = 0; hq < p.heads && n < 64; ++hq)
        if (kv_position(p, s, hq) == kvp) match[n++] = hq;
    n_match_s = n;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(const_cast<uint32_t*>(tmem_slot))), "r"((uint32_t)kBwdTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tm_dp = tmem + 256, tm_dv = tmem + 384, tm_dk = tmem + 448;   // S^T(n) at columns 128 (n & 1)
  const int per_head = nqb - kb;                         // query blocks kb .. nqb-1
  const int total = n_match_s * per_head;                // units (head, query block)

  if (warp == 8) {
    if (lane == 0 && total > 0) {
      const int z = blockIdx.z;
      auto load_q = [&](int n) {
        const int st = n % kDkvStages, hq = match[n / per_head], i = kb + n % per_head;
        mbar_expect_tx(bar(1 + st), 2 * kTileBytes);
        tma_load_3d_local(q_s + st * kTileBytes, &tmQKV, bar(1 + st), hq * kDh, i * kBq, z);
        tma_load_3d_local(do_s + st * kTileBytes, &tmDO, bar(1 + st), hq * kDh, i * kBq, z);
      };
      mbar_expect_tx(bar(0), 2 * kTileBytes);
      tma_load_3d_local(k_s, &tmQKV, bar(0), p.a_sub + kvp * kDh, kb * kBk, z);
      tma_load_3d_local(v_s, &tmQKV, bar(0), p.a_sub + (p.kv_max + kvp) * kDh, kb * kBk, z);
      for (int n = 0; n < kDkvStages && n < total; ++n) load_q(n);
      constexpr uint32_t idesc_s = idesc_bf16(0, 0, kBk, kBq);       // S^T = K Q^T, dP^T = V dO^T : both K-major
      constexpr uint32_t idesc_a = idesc_bf16(0, 1, kBk, kDh);       // dV += P^T dO, dK += dS^T Q : B MN-major
      auto mma_s = [&](int n) {
        const uint64_t ak = smem_desc(k_s, 16u, 1024u), bq = smem_desc(q_s + (n % kDkvStages) * kTileBytes, 16u, 1024u);
#pragma unroll
        for (int k = 0; k < kDh / 16; ++k) mma1(tmem + 128u * (n & 1), ak + 2u * k, bq + 2u * k, idesc_s, k != 0);
        commit1(bar(7 + (n & 1)));
      };
      auto mma_dp = [&](int n) {
        const uint64_t av = smem_desc(v_s, 16u, 1024u), bo = smem_desc(do_s + (n % kDkvStages) * kTileBytes, 16u, 1024u);
#pragma unroll
        for (int k = 0; k < kDh / 16; ++k) mma1(tm_dp, av + 2u * k, bo + 2u * k, idesc_s, k != 0);
        commit1(bar(9));
      };
      bool ok = mbar_wait_cta(bar(0), 0, abort_flag, status) && mbar_wait_cta(bar(1), 0, abort_flag, status);
      if (ok) {
        tc_fence_after();
        mma_s(0);
        mma_dp(0);
        if (total > 1) {
          ok = mbar_wait_cta(bar(2), 0, abort_flag, status);
          if (ok) {
            tc_fence_after();
            mma_s(1);
          }
        }
      }
      for (int n = 0; ok && n < total; ++n) {
        const int st = n % kDkvStages;
        // P^T and dS^T of unit n are in tensor memory (inside the S^T(n) and dP^T columns)
        if (!mbar_wait_cta(bar(10), n & 1, abort_flag, status)) break;
        tc_fence_after();
        const uint32_t t_p = tmem + 128u * (n & 1);
        const uint64_t bo = smem_desc(do_s + st * kTileBytes, (uint32_t)kDh * 128u, 1024u);
        const uint64_t bq = smem_desc(q_s + st * kTileBytes, (uint32_t)kDh * 128u, 1024u);
        // contraction over the 128 queries, 16 per step: 8 packed columns, the two 64-query halves 64 columns apart
#pragma unroll
        for (int k = 0; k < kBq / 16; ++k)
          mma1_ta(tm_dv, t_p + 64u * (k >> 2) + 8u * (k & 3), bo + (uint64_t)(k * 128), idesc_a, (n | k) != 0);
#pragma unroll
        for (int k = 0; k < kBq / 16; ++k)
          mma1_ta(tm_dk, tm_dp + 64u * (k >> 2) + 8u * (k & 3), bq + (uint64_t)(k * 128), idesc_a, (n | k) != 0);
        commit1(bar(4 + st));                            // unit n's Q / dO are consumed
        if (n + 1 == total) commit1(bar(11));
        // in issue order behind the MMAs that read dS^T(n) / P^T(n) out of the columns they overwrite
        if (n + 1 < total) mma_dp(n + 1);                // unit n + 1 arrived before S^T(n + 1) was issued
        if (n + 2 < total) {
          const int n2 = n + 2;
          if (!mbar_wait_cta(bar(1 + n2 % kDkvStages), (n2 / kDkvStages) & 1, abort_flag, status)) break;
          tc_fence_after();
          mma_s(n2);
        }
        if (n + kDkvStages < total) {
          if (!mbar_wait_cta(bar(4 + st), (n / kDkvStages) & 1, abort_flag, status)) break;
          load_q(n + kDkvStages);
        }
      }
    }
  } else {
    const int quarter = warp & 3, half = warp >> 2;
    const int r = quarter * 32 + lane;                   // key row of this thread
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    // Each warp stages the statistics of its own 64 queries (lane l: queries l and l + 32 of its half), one unit
    // ahead in registers, so no barrier between warps is needed.
    struct Stat { float l0, l1, d0, d1; };
    auto load_stat = [&](int n) {
      Stat o;
      o.l0 = INFINITY; o.l1 = INFINITY; o.d0 = 0.f; o.d1 = 0.f;      // no probability mass past the sequence end
      if (n >= total) return o;
      const int hq = match[n / per_head], i = kb + n % per_head;
      const int q0 = i * kBq + 64 * half + lane;
      const long long at = ((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len + q0;
      if (q0 < p.seq_len) { o.l0 = p.lse[at] * 1.4426950408889634f; o.d0 = p.delta[at]; }
      if (q0 + 32 < p.seq_len) { o.l1 = p.lse[at + 32] * 1.4426950408889634f; o.d1 = p.delta[at + 32]; }
      return o;
    };
    Stat staged = load_stat(0);
    const uint32_t st_lse = smem_u32(&stat_w[warp][0][0]), st_dl = smem_u32(&stat_w[warp][1][0]);
    bool ok = true;
    for (int n = 0; n < total; ++n) {
      float pr[64];
      __syncwarp();                                      // the previous unit's reads of the staging area are done
      stat_w[warp][0][lane] = staged.l0;
      stat_w[warp][0][lane + 32] = staged.l1;
      stat_w[warp][1][lane] = staged.d0;
      stat_w[warp][1][lane + 32] = staged.d1;
      __syncwarp();
      staged = load_stat(n + 1);                         // in flight during this unit
      const int i = kb + n % per_head;
      if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(7 + (n & 1)), (n >> 1) & 1, abort_flag, status))) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_s = tmem + lane_off + 128u * (n & 1) + 64u * half;
      if (i == kb) probs_from_st<true>(t_s, st_lse, r, 64 * half, p.scale_log2, pr);      // diagonal block
      else probs_from_st<false>(t_s, st_lse, r, 64 * half, p.scale_log2, pr);
      if (!__all_sync(0xffffffffu, mbar_wait_cta(bar(9), n & 1, abort_flag, status))) { ok = false; break; }
      tc_fence_after();
      ds_from_dpt(tm_dp + lane_off + 64u * half, st_dl, pr);
      tc_fence_before();
      mbar_arrive(bar(10));
    }
    // thread r owns key kb * 128 + r; the first four warps store dV, the others dK
    const int kj = kb * kBk + r;
    const long long row = (long long)s * p.T + (long long)b * p.seq_len + kj;
    __nv_bfloat16* dst = p.d_qkv + row * p.nq + p.a_sub + ((half ? 0 : p.kv_max) + kvp) * kDh;
    if (total == 0) {                                    // a KV position this subnet does not hold: zero gradient
      if (kj < p.seq_len)
        for (int c = 0; c < kDh / 8; ++c) reinterpret_cast<uint4*>(dst)[c] = make_uint4(0, 0, 0, 0);
    } else if (ok && __all_sync(0xffffffffu, mbar_wait_cta(bar(11), 0, abort_flag, status))) {
      tc_fence_after();
      const float sc = half ? p.scale_log2 * 0.6931471805599453f : 1.f;          // dK carries 1 / sqrt(d_head)
#pragma unroll
      for (int c = 0; c < kDh / 32; ++c) {
        uint32_t v[32];
        tc_ld32((half ? tm_dk : tm_dv) + lane_off + 32 * c, v);
        tc_wait_ld();
        if (kj < p.seq_len) store_acc32(dst + 32 * c, v, sc);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kBwdTmemCols) : "memory");
  }
}

}  // namespace

// Map over a bf16 activation [S * n_seqs][seq_len][width], box = 64 columns x 128 rows of one sequence.
static int sequence_map(CUtensorMap* tm, const void* ptr, int width, const AttnParams& p, int n_subnets) {
  const unsigned long long dims[3] = {(unsigned long long)width, (unsigned long long)p.seq_len,
                                      (unsigned long long)n_subnets * p.n_seqs};
  const unsigned long long strides[2] = {(unsigned long long)width * 2, (unsigned long long)p.seq_len * width * 2};
  const unsigned box[3] = {64, 128, 1};
  return encode_map_3d_bf16(tm, ptr, dims, strides, box, 128);
}

int attn_bwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st) {
  if (p.d_head != kDh || p.nq % 8 != 0) return TWIST_ERR_UNSUPPORTED;
  CUtensorMap tq, tdo;
  int rc = sequence_map(&tq, p.qkv, p.nq, p, n_subnets);
  if (rc != TWIST_OK) return rc;
  rc = sequence_map(&tdo, p.d_out, p.a_sub, p, n_subnets);
  if (rc != TWIST_OK) return rc;
  static bool configured[64] = {false};
  const int slot = device_slot();
  if (!configured[slot]) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(attn_dq_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDqSmem));
    TWIST_CUDA_TRY(cudaFuncSetAttribute(attn_dkv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDkvSmem));
    configured[slot] = true;
  }
  int* status = device_status_ptr();
  if (!status) return TWIST_ERR_CUDA;
  const int nb = (p.seq_len + kBq - 1) / kBq;
  attn_dq_tc_kernel<<<dim3(nb, p.heads, n_subnets * p.n_seqs), kBwdThreads, kDqSmem, st>>>(tq, tdo, p, status);
  TWIST_LAUNCH_CHECK();
  attn_dkv_tc_kernel<<<dim3(nb, p.kv_max, n_subnets * p.n_seqs), kBwdThreads, kDkvSmem, st>>>(tq, tdo, p, status);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int attn_fwd_tc(const AttnParams& p, int n_subnets, cudaStream_t st) {
  if (p.d_head != kDh || p.nq % 8 != 0) return TWIST_ERR_UNSUPPORTED;
  CUtensorMap tm;
  int rc = sequence_map(&tm, p.qkv, p.nq, p, n_subnets);
  if (rc != TWIST_OK) return rc;
  static bool configured[64] = {false};
  const int slot = device_slot();
  if (!configured[slot]) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFwdSmem));
    configured[slot] = true;
  }
  int* status = device_status_ptr();
  if (!status) return TWIST_ERR_CUDA;
  const dim3 grid((p.seq_len + kBq - 1) / kBq, p.heads, n_subnets * p.n_seqs);
  attn_fwd_tc_kernel<<<grid, kFwdThreads, kFwdSmem, st>>>(tm, p, status);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

}  // namespace twist
