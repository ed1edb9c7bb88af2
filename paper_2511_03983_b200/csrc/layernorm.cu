// twist_layernorm_fwd / twist_layernorm_bwd: the two layer normalisations of the pre-LN transformer layer
// (App. A, Layer Normalization and Transformer Layer Architecture):  z = (x - mu) / sigma per token,
// y = gamma * z + b.  HBM-bound row kernels for the chained (STACK) composition; bf16 activations, fp32
// statistics and parameters.  gamma and b are shared parameters: every worker holds and trains a copy
// ([S][d] here), the aggregator averages the copies.
//
// Forward and input gradient: one warp per token row, the row held in registers (16-byte accesses, at most
// 16 per lane: d_model <= 4096), mean and variance in two register passes.  The parameter gradients
// dgamma = sum_t dy * z, db = sum_t dy are column sums over all tokens: a second kernel forms partial sums
// over chunks of rows (thread = 8 adjacent columns), a finishing kernel adds the chunks in a fixed order and
// applies the optimiser step, so the result is deterministic.
#include <math.h>

#include "common.cuh"

namespace twist {
namespace {

constexpr int kLnMaxVec = 16;          // uint4 (8 bf16) per lane: rows of up to 32 * 16 * 8 = 4096 elements
constexpr int kLnRowsPerChunk = 256;   // rows per partial sum of the parameter gradients

__device__ inline float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ inline float bf_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }
__device__ inline uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ inline void unpack8(const uint4& v, float (&f)[8]) {
  f[0] = bf_lo(v.x); f[1] = bf_hi(v.x); f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
  f[4] = bf_lo(v.z); f[5] = bf_hi(v.z); f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}
__device__ inline float warp_sum(float v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

struct LnArgs {
  const __nv_bfloat16* x;        // [rows][d]
  __nv_bfloat16* y;              // fwd out
  float* mean;                   // [rows]
  float* rstd;                   // [rows]
  const float* gamma;            // [S][d]
  const float* beta;             // [S][d]
  const __nv_bfloat16* dy;       // bwd in
  const __nv_bfloat16* residual; // bwd in, may be null
  __nv_bfloat16* dx;             // bwd out
  long long rows;                // S * T
  int T, d;
  float eps;
};

// Eight consecutive fp32 parameters.
__device__ inline void load8(const float* p, float (&f)[8]) {
  const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

template <int NV>
__global__ void __launch_bounds__(256) ln_fwd_kernel(const LnArgs a) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int nvec = a.d / 8;
  const float inv_d = 1.0f / (float)a.d;
  for (long long r = warp0; r < a.rows; r += nwarps) {
    const uint4* src = reinterpret_cast<const uint4*>(a.x + r * a.d);
    uint4 v[NV];
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = i * 32 + lane;
      v[i] = c < nvec ? src[c] : make_uint4(0, 0, 0, 0);
      float f[8];
      unpack8(v[i], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) sum += f[e];
    }
    const float mu = warp_sum(sum) * inv_d;
    float sq = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      if (i * 32 + lane < nvec) {
        float f[8];
        unpack8(v[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) sq += (f[e] - mu) * (f[e] - mu);
      }
    }
    const float rs = 1.0f / sqrtf(warp_sum(sq) * inv_d + a.eps);
    const int s = (int)(r / a.T);
    const float* g = a.gamma + (long long)s * a.d;
    const float* b = a.beta + (long long)s * a.d;
    uint4* dst = reinterpret_cast<uint4*>(a.y + r * a.d);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = i * 32 + lane;
      if (c < nvec) {
        float f[8], gg[8], bb[8];
        unpack8(v[i], f);
        load8(g + 8 * c, gg);
        load8(b + 8 * c, bb);
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = fmaf(gg[e], (f[e] - mu) * rs, bb[e]);
        dst[c] = make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
      }
    }
    if (lane == 0) { a.mean[r] = mu; a.rstd[r] = rs; }
  }
}

// dx = rstd * (dz - mean(dz) - z * mean(dz * z)) [+ residual],  dz = dy * gamma,  z = (x - mean) * rstd.
template <int NV>
__global__ void __launch_bounds__(256) ln_bwd_dx_kernel(const LnArgs a) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int nvec = a.d / 8;
  const float inv_d = 1.0f / (float)a.d;
  for (long long r = warp0; r < a.rows; r += nwarps) {
    const uint4* xs = reinterpret_cast<const uint4*>(a.x + r * a.d);
    const uint4* ds = reinterpret_cast<const uint4*>(a.dy + r * a.d);
    const float mu = a.mean[r], rs = a.rstd[r];
    const int s = (int)(r / a.T);
    const float* g = a.gamma + (long long)s * a.d;
    uint4 xv[NV], dv[NV];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = i * 32 + lane;
      if (c < nvec) {
        xv[i] = xs[c];
        dv[i] = ds[c];
        float xf[8], df[8], gg[8];
        unpack8(xv[i], xf);
        unpack8(dv[i], df);
        load8(g + 8 * c, gg);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float dz = df[e] * gg[e];
          s1 += dz;
          s2 += dz * ((xf[e] - mu) * rs);
        }
      } else {
        xv[i] = make_uint4(0, 0, 0, 0);
        dv[i] = make_uint4(0, 0, 0, 0);
      }
    }
    const float c1 = warp_sum(s1) * inv_d, c2 = warp_sum(s2) * inv_d;
    uint4* dst = reinterpret_cast<uint4*>(a.dx + r * a.d);
    const uint4* res = a.residual ? reinterpret_cast<const uint4*>(a.residual + r * a.d) : nullptr;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = i * 32 + lane;
      if (c < nvec) {
        float xf[8], df[8], gg[8], rf[8];
        unpack8(xv[i], xf);
        unpack8(dv[i], df);
        load8(g + 8 * c, gg);
        if (res) unpack8(res[c], rf);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float z = (xf[e] - mu) * rs;
          const float v = rs * (df[e] * gg[e] - c1 - z * c2);
          xf[e] = res ? v + rf[e] : v;                       // one rounding for the sum
        }
        dst[c] = make_uint4(pack2(xf[0], xf[1]), pack2(xf[2], xf[3]), pack2(xf[4], xf[5]), pack2(xf[6], xf[7]));
      }
    }
  }
}

// Partial sums of dgamma and db over a chunk of rows: grid (column blocks of 256, row chunks, subnets);
// thread (row group w = threadIdx.x / 32, lane) owns 8 adjacent columns and every 8th row of the chunk; the
// eight row groups are added in shared memory in a fixed order.  partial: [S][chunks][2][d].
__global__ void __launch_bounds__(256) ln_bwd_param_kernel(const LnArgs a, int chunks, float* __restrict__ partial) {
  __shared__ float red[8][32][17];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int col = (blockIdx.x * 32 + lane) * 8;
  const int chunk = blockIdx.y, s = blockIdx.z;
  const int r0 = chunk * kLnRowsPerChunk, r1 = min(a.T, r0 + kLnRowsPerChunk);
  float ag[8], ab[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) { ag[e] = 0.f; ab[e] = 0.f; }
  if (col < a.d) {
    for (int t = r0 + w; t < r1; t += 8) {
      const long long r = (long long)s * a.T + t;
      const float mu = a.mean[r], rs = a.rstd[r];
      float xf[8], df[8];
      unpack8(*reinterpret_cast<const uint4*>(a.x + r * a.d + col), xf);
      unpack8(*reinterpret_cast<const uint4*>(a.dy + r * a.d + col), df);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        ag[e] += df[e] * ((xf[e] - mu) * rs);
        ab[e] += df[e];
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) { red[w][lane][e] = ag[e]; red[w][lane][8 + e] = ab[e]; }
  __syncthreads();
  if (w == 0 && col < a.d) {
    float* out = partial + ((long long)s * chunks + chunk) * 2 * a.d;
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      float t = 0.f;
      for (int k = 0; k < 8; ++k) t += red[k][lane][e];      // fixed order
      out[(e >> 3) * a.d + col + (e & 7)] = t;
    }
  }
}

struct LnUpdate {
  float* gamma; float* beta;             // [S][d], updated when lr != 0
  float* dgamma; float* dbeta;           // optional dumps [S][d]
  float *m_g, *v_g, *m_b, *v_b;          // Adam moments [S][d]
  float lr, beta1, beta2, eps, bias1, bias2;
  int adam;
};

__device__ inline float opt_step(float w, float g, float* m, float* v, long long i, const LnUpdate& u) {
  if (u.lr == 0.f) return w;
  if (!u.adam) return w - u.lr * g;
  const float m1 = fmaf(u.beta1, m[i], (1.f - u.beta1) * g);
  const float m2 = fmaf(u.beta2, v[i], (1.f - u.beta2) * g * g);
  m[i] = m1;
  v[i] = m2;
  return w - u.lr * (m1 * u.bias1) / (sqrtf(m2 * u.bias2) + u.eps);
}

// One thread per (subnet, column): adds the chunks in ascending order, then the optimiser step.
__global__ void ln_finish_kernel(const float* __restrict__ partial, int chunks, int d, long long n, const LnUpdate u) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // s * d + col
  if (i >= n) return;
  const long long s = i / d;
  const int col = (int)(i - s * d);
  float dg = 0.f, db = 0.f;
  for (int c = 0; c < chunks; ++c) {
    const float* p = partial + (s * chunks + c) * 2 * d;
    dg += p[col];
    db += p[d + col];
  }
  if (u.dgamma) u.dgamma[i] = dg;
  if (u.dbeta) u.dbeta[i] = db;
  u.gamma[i] = opt_step(u.gamma[i], dg, u.m_g, u.v_g, i, u);
  u.beta[i] = opt_step(u.beta[i], db, u.m_b, u.v_b, i, u);
}

int row_grid(long long rows) {
  const long long want = (rows + 7) / 8;
  const long long cap = (long long)sm_count() * 8;
  return (int)(want < 1 ? 1 : (want < cap ? want : cap));
}

int check(const twist_layernorm_args* a) {
  if (!a) return TWIST_ERR_NULL;
  if (a->dtype != TWIST_BF16) return TWIST_ERR_UNSUPPORTED;
  if (a->n_subnets <= 0 || a->tokens <= 0 || a->d_model <= 0 || a->d_model % 8 != 0 || !(a->eps >= 0.f)) return TWIST_ERR_SHAPE;
  if (a->d_model > 32 * kLnMaxVec * 8) return TWIST_ERR_UNSUPPORTED;
  if (!a->x || !a->mean || !a->rstd || !a->gamma || !a->beta) return TWIST_ERR_NULL;
  const void* ptrs[] = {a->x, a->y, a->gamma, a->beta, a->dy, a->dx, a->dx_residual, a->dgamma, a->dbeta, a->ws,
                        a->m_gamma, a->v_gamma, a->m_beta, a->v_beta};
  for (const void* p : ptrs)
    if (!aligned16(p)) return TWIST_ERR_SHAPE;
  return TWIST_OK;
}

LnArgs make_args(const twist_layernorm_args* a) {
  LnArgs p;
  memset(&p, 0, sizeof(p));
  p.x = static_cast<const __nv_bfloat16*>(a->x);
  p.y = static_cast<__nv_bfloat16*>(a->y);
  p.mean = a->mean; p.rstd = a->rstd; p.gamma = a->gamma; p.beta = a->beta;
  p.dy = static_cast<const __nv_bfloat16*>(a->dy);
  p.residual = static_cast<const __nv_bfloat16*>(a->dx_residual);
  p.dx = static_cast<__nv_bfloat16*>(a->dx);
  p.rows = (long long)a->n_subnets * a->tokens;
  p.T = a->tokens; p.d = a->d_model; p.eps = a->eps;
  return p;
}

}  // namespace
}  // namespace twist

using namespace twist;

extern "C" size_t twist_layernorm_workspace_bytes(int32_t n_subnets, int32_t tokens, int32_t d_model) {
  if (n_subnets <= 0 || tokens <= 0 || d_model <= 0) return 0;
  const size_t chunks = ((size_t)tokens + kLnRowsPerChunk - 1) / kLnRowsPerChunk;
  return (size_t)n_subnets * chunks * 2 * (size_t)d_model * sizeof(float);
}

extern "C" int32_t twist_layernorm_fwd(const twist_layernorm_args* a, void* stream) {
  int rc = check(a);
  if (rc != TWIST_OK) return rc;
  if (!a->y) return TWIST_ERR_NULL;
  const LnArgs p = make_args(a);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int grid = row_grid(p.rows);
  const int nv = (p.d / 8 + 31) / 32;
  if (nv <= 1) ln_fwd_kernel<1><<<grid, 256, 0, st>>>(p);
  else if (nv <= 2) ln_fwd_kernel<2><<<grid, 256, 0, st>>>(p);
  else if (nv <= 4) ln_fwd_kernel<4><<<grid, 256, 0, st>>>(p);
  else if (nv <= 8) ln_fwd_kernel<8><<<grid, 256, 0, st>>>(p);
  else ln_fwd_kernel<16><<<grid, 256, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

extern "C" int32_t twist_layernorm_bwd(const twist_layernorm_args* a, void* stream) {
  int rc = check(a);
  if (rc != TWIST_OK) return rc;
  if (!a->dy || !a->dx) return TWIST_ERR_NULL;
  if (!a->ws || a->ws_bytes < twist_layernorm_workspace_bytes(a->n_subnets, a->tokens, a->d_model)) return TWIST_ERR_WORKSPACE;
  LnUpdate u;
  memset(&u, 0, sizeof(u));
  u.gamma = a->gamma; u.beta = a->beta; u.dgamma = a->dgamma; u.dbeta = a->dbeta; u.lr = a->lr;
  if (a->opt.kind == TWIST_OPT_ADAM && a->lr != 0.f) {
    if (!a->m_gamma || !a->v_gamma || !a->m_beta || !a->v_beta) return TWIST_ERR_NULL;
    if (a->opt.step < 1 || !(a->opt.beta1 >= 0.f && a->opt.beta1 < 1.f) || !(a->opt.beta2 >= 0.f && a->opt.beta2 < 1.f) ||
        !(a->opt.eps >= 0.f))
      return TWIST_ERR_SHAPE;
    u.adam = 1;
    u.m_g = a->m_gamma; u.v_g = a->v_gamma; u.m_b = a->m_beta; u.v_b = a->v_beta;
    u.beta1 = a->opt.beta1; u.beta2 = a->opt.beta2; u.eps = a->opt.eps;
    u.bias1 = (float)(1.0 / (1.0 - pow((double)a->opt.beta1, (double)a->opt.step)));
    u.bias2 = (float)(1.0 / (1.0 - pow((double)a->opt.beta2, (double)a->opt.step)));
  } else if (a->opt.kind != TWIST_OPT_SGD && a->opt.kind != TWIST_OPT_ADAM) {
    return TWIST_ERR_SHAPE;
  }
  const LnArgs p = make_args(a);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int grid = row_grid(p.rows);
  const int nv = (p.d / 8 + 31) / 32;
  // the parameter gradients read the same dy and x as the input gradient and are formed first, so that dx may
  // overwrite dy or the residual in place (a warp reads its whole row before it writes it)
  const int chunks = (p.T + kLnRowsPerChunk - 1) / kLnRowsPerChunk;
  float* partial = static_cast<float*>(a->ws);
  ln_bwd_param_kernel<<<dim3((p.d / 8 + 31) / 32, chunks, a->n_subnets), 256, 0, st>>>(p, chunks, partial);
  TWIST_LAUNCH_CHECK();
  if (nv <= 1) ln_bwd_dx_kernel<1><<<grid, 256, 0, st>>>(p);
  else if (nv <= 2) ln_bwd_dx_kernel<2><<<grid, 256, 0, st>>>(p);
  else if (nv <= 4) ln_bwd_dx_kernel<4><<<grid, 256, 0, st>>>(p);
  else if (nv <= 8) ln_bwd_dx_kernel<8><<<grid, 256, 0, st>>>(p);
  else ln_bwd_dx_kernel<16><<<grid, 256, 0, st>>>(p);
  TWIST_LAUNCH_CHECK();
  const long long n = (long long)a->n_subnets * p.d;
  ln_finish_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(partial, chunks, p.d, n, u);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}
