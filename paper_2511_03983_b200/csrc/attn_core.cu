// twist_attn_core_fwd / twist_attn_core_bwd: the softmax core between the QKV projection and the
// output projection of the kept heads (App. A, Multi-Head Attention:
// head_h = softmax(Q_h K_h^T / sqrt(d_head)) V_h), causal within each sequence, with optional
// grouped-query sharing of K/V.  Needed by the chained (STACK) composition only.
//
// d_head = 64 runs on the tensor cores (attn_core_tc.cu); the kernels in this file serve the other head sizes (and
// the delta reduction of every size).
// These are plain fp32 SIMT kernels (bf16 storage, fp32 arithmetic): one group of G threads owns
// one query (forward, dQ) or one key (dK/dV) with DPT = d_head / G of its dimensions in registers;
// the other side streams through shared memory in tiles of 64 rows.  The forward keeps a running
// maximum and sum (one rescale per 8 keys) and stores the log-sum-exp; the backward recomputes
// the probabilities from it.  Every result has one writer: deterministic, no atomics.
#include "attn_core.cuh"
#include "plan.cuh"

namespace twist {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnTile = 64;      // rows of the streamed side per shared-memory tile
constexpr float kLog2e = 1.4426950408889634f;

__device__ inline float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ inline float bf_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
__device__ inline uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Loads DPT bf16 values (a thread's part of a row) from global memory as floats; zeros when !ok.
template <int DPT>
__device__ inline void load_part(const __nv_bfloat16* src, float (&v)[DPT], bool ok) {
#pragma unroll
  for (int c = 0; c < DPT / 8; ++c) {
    const uint4 w = ok ? reinterpret_cast<const uint4*>(src)[c] : make_uint4(0, 0, 0, 0);
    v[8 * c] = bf_lo(w.x); v[8 * c + 1] = bf_hi(w.x); v[8 * c + 2] = bf_lo(w.y); v[8 * c + 3] = bf_hi(w.y);
    v[8 * c + 4] = bf_lo(w.z); v[8 * c + 5] = bf_hi(w.z); v[8 * c + 6] = bf_lo(w.w); v[8 * c + 7] = bf_hi(w.w);
  }
}
template <int DPT>
__device__ inline void store_part(__nv_bfloat16* dst, const float (&v)[DPT]) {
#pragma unroll
  for (int c = 0; c < DPT / 8; ++c)
    reinterpret_cast<uint4*>(dst)[c] = make_uint4(pack2(v[8 * c], v[8 * c + 1]), pack2(v[8 * c + 2], v[8 * c + 3]),
                                                  pack2(v[8 * c + 4], v[8 * c + 5]), pack2(v[8 * c + 6], v[8 * c + 7]));
}
// Part of row `j` of a shared-memory tile [rows][d_head] (bf16) as floats.
template <int DPT>
__device__ inline void tile_part(const __nv_bfloat16* tile, int j, int d_head, int part, float (&v)[DPT]) {
  const uint4* src = reinterpret_cast<const uint4*>(tile + (long long)j * d_head + part * DPT);
#pragma unroll
  for (int c = 0; c < DPT / 8; ++c) {
    const uint4 w = src[c];
    v[8 * c] = bf_lo(w.x); v[8 * c + 1] = bf_hi(w.x); v[8 * c + 2] = bf_lo(w.y); v[8 * c + 3] = bf_hi(w.y);
    v[8 * c + 4] = bf_lo(w.z); v[8 * c + 5] = bf_hi(w.z); v[8 * c + 6] = bf_lo(w.w); v[8 * c + 7] = bf_hi(w.w);
  }
}
// Cooperative copy of `rows` rows of d_head bf16 (row stride ld elements, first row may be short of the sequence
// end: rows beyond n_valid are zero) into a shared tile.
__device__ inline void fill_tile(__nv_bfloat16* tile, const __nv_bfloat16* src, long long ld, int d_head, int n_valid) {
  const int chunks = d_head / 8;
  for (int e = threadIdx.x; e < kAttnTile * chunks; e += kAttnThreads) {
    const int r = e / chunks, c = e - r * chunks;
    const uint4 w = r < n_valid ? reinterpret_cast<const uint4*>(src + r * ld)[c] : make_uint4(0, 0, 0, 0);
    reinterpret_cast<uint4*>(tile + (long long)r * d_head)[c] = w;
  }
}
template <int G>
__device__ inline float group_sum(float v) {
#pragma unroll
  for (int o = G / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int DPT>
__device__ inline float dot(const float (&a)[DPT], const float (&b)[DPT]) {
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < DPT; ++i) s = fmaf(a[i], b[i], s);
  return s;
}

// ---------------------------------------------------------------------------------------------
// Forward: grid (query blocks, kept heads, S * n_seqs); a group of G threads per query.
// ---------------------------------------------------------------------------------------------
template <int DPT, int G>
__global__ void __launch_bounds__(kAttnThreads) attn_fwd_kernel(const AttnParams p) {
  __shared__ __align__(16) __nv_bfloat16 Ks[kAttnTile * DPT * G];
  __shared__ __align__(16) __nv_bfloat16 Vs[kAttnTile * DPT * G];
  constexpr int QB = kAttnThreads / G;
  const int dh = DPT * G;
  const int hq = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int part = threadIdx.x % G, qi = blockIdx.x * QB + threadIdx.x / G;
  const bool q_ok = qi < p.seq_len;
  const int kvp = kv_position(p, s, hq);
  const long long row0 = (long long)s * p.T + (long long)b * p.seq_len;          // first token row of the sequence
  const __nv_bfloat16* base = p.qkv + row0 * p.nq;
  float q[DPT], o[DPT];
  load_part<DPT>(base + (long long)qi * p.nq + hq * dh + part * DPT, q, q_ok);
#pragma unroll
  for (int i = 0; i < DPT; ++i) { q[i] *= p.scale_log2; o[i] = 0.f; }
  float m = -INFINITY, l = 0.f;
  const int q_last = min(p.seq_len, (blockIdx.x + 1) * QB) - 1;                  // last query of the block
  for (int k0 = 0; k0 <= q_last; k0 += kAttnTile) {
    __syncthreads();
    const int n_valid = min(kAttnTile, p.seq_len - k0);
    fill_tile(Ks, base + (long long)k0 * p.nq + p.a_sub + kvp * dh, p.nq, dh, n_valid);
    fill_tile(Vs, base + (long long)k0 * p.nq + p.a_sub + p.kv_max * dh + kvp * dh, p.nq, dh, n_valid);
    __syncthreads();
    const int j_end = min(n_valid, q_last - k0 + 1);                             // block-uniform
    for (int j0 = 0; j0 < j_end; j0 += 8) {
      float sc[8];
      float cm = -INFINITY;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        float kf[DPT];
        tile_part<DPT>(Ks, min(j0 + u, kAttnTile - 1), dh, part, kf);
        const float t = group_sum<G>(dot<DPT>(q, kf));
        const bool live = q_ok && (j0 + u < j_end) && (k0 + j0 + u <= qi);
        sc[u] = live ? t : -INFINITY;
        cm = fmaxf(cm, sc[u]);
      }
      const float m_new = fmaxf(m, cm);
      if (m_new == -INFINITY) continue;                                          // nothing visible yet (group-uniform)
      const float corr = exp2f(m - m_new);
      l *= corr;
#pragma unroll
      for (int i = 0; i < DPT; ++i) o[i] *= corr;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float pu = exp2f(sc[u] - m_new);                                   // 0 for masked keys
        l += pu;
        float vf[DPT];
        tile_part<DPT>(Vs, min(j0 + u, kAttnTile - 1), dh, part, vf);
#pragma unroll
        for (int i = 0; i < DPT; ++i) o[i] = fmaf(pu, vf[i], o[i]);
      }
      m = m_new;
    }
  }
  if (q_ok) {
    const float inv = 1.f / l;
#pragma unroll
    for (int i = 0; i < DPT; ++i) o[i] *= inv;
    store_part<DPT>(p.out + (row0 + qi) * p.a_sub + hq * dh + part * DPT, o);
    if (part == 0)
      p.lse[((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len + qi] = (m + log2f(l)) * 0.6931471805599453f;
  }
}

// delta[s][hq][t] = sum over the head's dimensions of dA * A
__global__ void attn_delta_kernel(const AttnParams p, long long n) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;          // (s, hq, t)
  if (e >= n) return;
  const int t = (int)(e % p.T);
  const int hq = (int)((e / p.T) % p.heads);
  const int s = (int)(e / ((long long)p.T * p.heads));
  const long long off = ((long long)s * p.T + t) * p.a_sub + hq * p.d_head;
  float acc = 0.f;
  for (int c = 0; c < p.d_head / 8; ++c) {
    const uint4 a = reinterpret_cast<const uint4*>(p.out + off)[c];
    const uint4 g = reinterpret_cast<const uint4*>(p.d_out + off)[c];
    acc += bf_lo(a.x) * bf_lo(g.x) + bf_hi(a.x) * bf_hi(g.x) + bf_lo(a.y) * bf_lo(g.y) + bf_hi(a.y) * bf_hi(g.y) +
           bf_lo(a.z) * bf_lo(g.z) + bf_hi(a.z) * bf_hi(g.z) + bf_lo(a.w) * bf_lo(g.w) + bf_hi(a.w) * bf_hi(g.w);
  }
  p.delta[e] = acc;
}

// ---------------------------------------------------------------------------------------------
// dQ: same decomposition as the forward.  P = exp(S - lse), dP = dO V^T, dS = P (dP - delta), dQ = dS K / sqrt(d).
// ---------------------------------------------------------------------------------------------
template <int DPT, int G>
__global__ void __launch_bounds__(kAttnThreads) attn_dq_kernel(const AttnParams p) {
  __shared__ __align__(16) __nv_bfloat16 Ks[kAttnTile * DPT * G];
  __shared__ __align__(16) __nv_bfloat16 Vs[kAttnTile * DPT * G];
  constexpr int QB = kAttnThreads / G;
  const int dh = DPT * G;
  const int hq = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int part = threadIdx.x % G, qi = blockIdx.x * QB + threadIdx.x / G;
  const bool q_ok = qi < p.seq_len;
  const int kvp = kv_position(p, s, hq);
  const long long row0 = (long long)s * p.T + (long long)b * p.seq_len;
  const __nv_bfloat16* base = p.qkv + row0 * p.nq;
  float q[DPT], go[DPT], dq[DPT];
  load_part<DPT>(base + (long long)qi * p.nq + hq * dh + part * DPT, q, q_ok);
  load_part<DPT>(p.d_out + (row0 + qi) * p.a_sub + hq * dh + part * DPT, go, q_ok);
#pragma unroll
  for (int i = 0; i < DPT; ++i) { q[i] *= p.scale_log2; dq[i] = 0.f; }
  const long long stat = ((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len + qi;
  const float lse2 = q_ok ? p.lse[stat] * kLog2e : 0.f;
  const float dl = q_ok ? p.delta[stat] : 0.f;
  const int q_last = min(p.seq_len, (blockIdx.x + 1) * QB) - 1;
  for (int k0 = 0; k0 <= q_last; k0 += kAttnTile) {
    __syncthreads();
    const int n_valid = min(kAttnTile, p.seq_len - k0);
    fill_tile(Ks, base + (long long)k0 * p.nq + p.a_sub + kvp * dh, p.nq, dh, n_valid);
    fill_tile(Vs, base + (long long)k0 * p.nq + p.a_sub + p.kv_max * dh + kvp * dh, p.nq, dh, n_valid);
    __syncthreads();
    const int j_end = min(n_valid, q_last - k0 + 1);
    for (int j = 0; j < j_end; ++j) {
      float kf[DPT], vf[DPT];
      tile_part<DPT>(Ks, j, dh, part, kf);
      tile_part<DPT>(Vs, j, dh, part, vf);
      const float sc = group_sum<G>(dot<DPT>(q, kf));
      const float dp = group_sum<G>(dot<DPT>(go, vf));
      const bool live = q_ok && (k0 + j <= qi);
      const float ds = live ? exp2f(sc - lse2) * (dp - dl) : 0.f;
#pragma unroll
      for (int i = 0; i < DPT; ++i) dq[i] = fmaf(ds, kf[i], dq[i]);
    }
  }
  if (q_ok) {
    const float sc = p.scale_log2 / kLog2e;                                       // 1 / sqrt(d_head)
#pragma unroll
    for (int i = 0; i < DPT; ++i) dq[i] *= sc;
    store_part<DPT>(p.d_qkv + (row0 + qi) * p.nq + hq * dh + part * DPT, dq);
  }
}

// ---------------------------------------------------------------------------------------------
// dK, dV: grid (key blocks, KV positions, S * n_seqs); a group of G threads per key; the queries of every
// kept head that reads this KV position stream through shared memory.  dV = P^T dO, dK = dS^T Q / sqrt(d).
// KV positions the subnet does not hold (padding columns) get zeros.
// ---------------------------------------------------------------------------------------------
template <int DPT, int G>
__global__ void __launch_bounds__(kAttnThreads) attn_dkv_kernel(const AttnParams p) {
  __shared__ __align__(16) __nv_bfloat16 Qs[kAttnTile * DPT * G];
  __shared__ __align__(16) __nv_bfloat16 Gs[kAttnTile * DPT * G];
  __shared__ float Ls[kAttnTile], Ds[kAttnTile];
  constexpr int KB = kAttnThreads / G;
  const int dh = DPT * G;
  const int kvp = blockIdx.y, s = blockIdx.z / p.n_seqs, b = blockIdx.z - s * p.n_seqs;
  const int part = threadIdx.x % G, kj = blockIdx.x * KB + threadIdx.x / G;
  const bool k_ok = kj < p.seq_len;
  const long long row0 = (long long)s * p.T + (long long)b * p.seq_len;
  const __nv_bfloat16* base = p.qkv + row0 * p.nq;
  const int k_col = p.a_sub + kvp * dh + part * DPT, v_col = k_col + p.kv_max * dh;
  float kf[DPT], vf[DPT], dk[DPT], dv[DPT];
#pragma unroll
  for (int i = 0; i < DPT; ++i) { dk[i] = 0.f; dv[i] = 0.f; }
  const int held = p.kv_count ? p.kv_count[s] : p.kv_max;
  if (kvp < held) {                                                               // block-uniform
    load_part<DPT>(base + (long long)kj * p.nq + k_col, kf, k_ok);
    load_part<DPT>(base + (long long)kj * p.nq + v_col, vf, k_ok);
    const int k_first = blockIdx.x * KB;                                          // first key of the block
    for (int hq = 0; hq < p.heads; ++hq) {
      if (kv_position(p, s, hq) != kvp) continue;                                 // block-uniform
      const long long stat0 = ((long long)s * p.heads + hq) * p.T + (long long)b * p.seq_len;
      for (int q0 = (k_first / kAttnTile) * kAttnTile; q0 < p.seq_len; q0 += kAttnTile) {
        __syncthreads();
        const int n_valid = min(kAttnTile, p.seq_len - q0);
        fill_tile(Qs, base + (long long)q0 * p.nq + hq * dh, p.nq, dh, n_valid);
        fill_tile(Gs, p.d_out + (row0 + q0) * p.a_sub + hq * dh, p.a_sub, dh, n_valid);
        if (threadIdx.x < kAttnTile) {
          const bool ok = threadIdx.x < n_valid;
          Ls[threadIdx.x] = ok ? p.lse[stat0 + q0 + threadIdx.x] * kLog2e : 0.f;
          Ds[threadIdx.x] = ok ? p.delta[stat0 + q0 + threadIdx.x] : 0.f;
        }
        __syncthreads();
        for (int i = 0; i < n_valid; ++i) {
          float qf[DPT], gf[DPT];
          tile_part<DPT>(Qs, i, dh, part, qf);
          tile_part<DPT>(Gs, i, dh, part, gf);
          const float sc = group_sum<G>(dot<DPT>(qf, kf)) * p.scale_log2;
          const float dp = group_sum<G>(dot<DPT>(gf, vf));
          const bool live = k_ok && (q0 + i >= kj);
          const float pr = live ? exp2f(sc - Ls[i]) : 0.f;
          const float ds = pr * (dp - Ds[i]);
#pragma unroll
          for (int e = 0; e < DPT; ++e) {
            dv[e] = fmaf(pr, gf[e], dv[e]);
            dk[e] = fmaf(ds, qf[e], dk[e]);
          }
        }
      }
    }
    const float sc = p.scale_log2 / kLog2e;
#pragma unroll
    for (int i = 0; i < DPT; ++i) dk[i] *= sc;
  }
  if (k_ok) {
    store_part<DPT>(p.d_qkv + (row0 + kj) * p.nq + k_col, dk);
    store_part<DPT>(p.d_qkv + (row0 + kj) * p.nq + v_col, dv);
  }
}

int check(const twist_attn_core_args* a) {
  if (!a) return TWIST_ERR_NULL;
  if (a->dtype != TWIST_BF16) return TWIST_ERR_UNSUPPORTED;
  if (a->n_subnets <= 0 || a->n_seqs <= 0 || a->seq_len <= 0 || a->head_keep <= 0 || a->kv_max <= 0 || a->d_head <= 0)
    return TWIST_ERR_SHAPE;
  if (a->d_head != 8 && a->d_head != 16 && a->d_head != 32 && a->d_head != 64 && a->d_head != 128) return TWIST_ERR_UNSUPPORTED;
  if ((long long)a->n_subnets * a->n_seqs > 65535 || a->head_keep > 65535) return TWIST_ERR_UNSUPPORTED;
  if (a->head_idx) {
    if (!a->kv_pos || a->n_heads <= 0 || a->n_kv_heads <= 0 || a->n_heads % a->n_kv_heads != 0) return TWIST_ERR_SHAPE;
  } else if (a->kv_max != a->head_keep) {
    return TWIST_ERR_SHAPE;
  }
  if (!a->qkv || !a->lse) return TWIST_ERR_NULL;
  if (!aligned16(a->qkv)) return TWIST_ERR_SHAPE;
  return TWIST_OK;
}

AttnParams make_params(const twist_attn_core_args* a) {
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.qkv = static_cast<const __nv_bfloat16*>(a->qkv);
  p.out = static_cast<__nv_bfloat16*>(a->out);
  p.lse = a->lse;
  p.d_out = static_cast<const __nv_bfloat16*>(a->d_out);
  p.d_qkv = static_cast<__nv_bfloat16*>(a->d_qkv);
  p.delta = a->delta;
  p.head_idx = a->head_idx; p.kv_pos = a->kv_pos; p.kv_count = a->kv_count;
  p.n_seqs = a->n_seqs; p.seq_len = a->seq_len; p.heads = a->head_keep; p.kv_max = a->kv_max; p.d_head = a->d_head;
  p.per_group = a->head_idx ? a->n_heads / a->n_kv_heads : 1;
  p.n_kv_heads = a->n_kv_heads;
  p.a_sub = a->head_keep * a->d_head;
  p.nq = p.a_sub + 2 * a->kv_max * a->d_head;
  p.T = a->n_seqs * a->seq_len;
  p.scale_log2 = kLog2e / sqrtf((float)a->d_head);
  p.status = device_status_ptr();
  return p;
}

template <int DPT, int G>
int run(const AttnParams& p, int n_subnets, bool backward, cudaStream_t st) {
  const int rows_per_block = kAttnThreads / G;
  const dim3 grid_q((p.seq_len + rows_per_block - 1) / rows_per_block, p.heads, n_subnets * p.n_seqs);
  if (!backward) {
    attn_fwd_kernel<DPT, G><<<grid_q, kAttnThreads, 0, st>>>(p);
    TWIST_LAUNCH_CHECK();
    return TWIST_OK;
  }
  const long long n = (long long)n_subnets * p.heads * p.T;
  attn_delta_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(p, n);
  TWIST_LAUNCH_CHECK();
  if (DPT * G == 64) return attn_bwd_tc(p, n_subnets, st);                         // tensor-core dQ and dK/dV
  attn_dq_kernel<DPT, G><<<grid_q, kAttnThreads, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  const dim3 grid_k(grid_q.x, p.kv_max, grid_q.z);
  attn_dkv_kernel<DPT, G><<<grid_k, kAttnThreads, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int dispatch(const AttnParams& p, int n_subnets, bool backward, cudaStream_t st) {
  if (!p.status) return TWIST_ERR_CUDA;
  switch (p.d_head) {
    case 8: return run<8, 1>(p, n_subnets, backward, st);
    case 16: return run<16, 1>(p, n_subnets, backward, st);
    case 32: return run<32, 1>(p, n_subnets, backward, st);
    case 64:
      if (!backward) return attn_fwd_tc(p, n_subnets, st);                          // tensor-core forward
      return run<32, 2>(p, n_subnets, backward, st);
    case 128: return run<32, 4>(p, n_subnets, backward, st);
    default: return TWIST_ERR_UNSUPPORTED;
  }
}

}  // namespace
}  // namespace twist

extern "C" int32_t twist_attn_core_fwd(const twist_attn_core_args* a, void* stream) {
  using namespace twist;
  int rc = check(a);
  if (rc != TWIST_OK) return rc;
  if (!a->out || !aligned16(a->out)) return a->out ? TWIST_ERR_SHAPE : TWIST_ERR_NULL;
  PlanScope scope(a->plan);
  return dispatch(make_params(a), a->n_subnets, false, static_cast<cudaStream_t>(stream));
}

extern "C" int32_t twist_attn_core_bwd(const twist_attn_core_args* a, void* stream) {
  using namespace twist;
  int rc = check(a);
  if (rc != TWIST_OK) return rc;
  if (!a->out || !a->d_out || !a->d_qkv || !a->delta) return TWIST_ERR_NULL;
  if (!aligned16(a->out) || !aligned16(a->d_out) || !aligned16(a->d_qkv)) return TWIST_ERR_SHAPE;
  PlanScope scope(a->plan);
  return dispatch(make_params(a), a->n_subnets, true, static_cast<cudaStream_t>(stream));
}
