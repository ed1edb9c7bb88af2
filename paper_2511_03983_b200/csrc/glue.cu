// Glue of the local training steps: the MSE loss with its gradient (both dtypes), and the small
// fp32 SIMT kernels (grouped GEMM, activations, SGD) behind the TWIST_FP32 path, which exists for
// the tiny fp32 workload only and is not tuned: the tensor-core path is the bf16 one.
#include "glue.cuh"

namespace twist {

namespace {

constexpr int kMseBlocks = 1024;   // partial sums per subnet (upper bound on gridDim.x)

__device__ inline float block_reduce_sum(float v, float* scratch) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float t = 0.f;
  if (warp == 0) {
    t = lane < nw ? scratch[lane] : 0.f;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  }
  return t;   // valid in thread 0
}

// Column validity: [0, seg_begin) valid; then groups of seg_width columns whose first vc are valid.
__device__ inline bool col_valid(int col, int seg_begin, int seg_width, int vc) {
  return col < seg_begin || (col - seg_begin) % seg_width < vc;
}
__device__ inline int valid_count(int width, int seg_begin, int seg_width, int vc) {
  return seg_begin + ((width - seg_begin) / seg_width) * vc;
}

// y, tgt, dy: [S][T][width]; one grid row per subnet; partial[s][blockIdx.x] = sum of squared errors.
template <bool BF16>
__global__ void __launch_bounds__(256) mse_kernel(const void* __restrict__ y_, const void* __restrict__ t_,
                                                  void* __restrict__ dy_, int tokens, int width,
                                                  const int32_t* __restrict__ valid_cols, int seg_begin, int seg_width,
                                                  float* __restrict__ partial) {
  __shared__ float scratch[8];
  const int s = blockIdx.y;
  const int vc = valid_cols ? min(max(valid_cols[s], 0), seg_width) : seg_width;
  const long long n = (long long)tokens * width;
  const int n_valid = valid_count(width, seg_begin, seg_width, vc);
  const float k = n_valid > 0 ? 2.0f / ((float)tokens * (float)n_valid) : 0.f;     // no valid column: zero gradient
  float acc = 0.f;
  if (BF16) {
    const uint4* y = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(y_) + (long long)s * n);
    const uint4* t = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(t_) + (long long)s * n);
    uint4* dy = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dy_) + (long long)s * n);
    const long long chunks = n / 8;
    for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < chunks; c += (long long)gridDim.x * blockDim.x) {
      const int col0 = (int)((c * 8) % width);
      uint4 yv = y[c], tv = t[c], out;
      const uint32_t* yp = &yv.x; const uint32_t* tp = &tv.x; uint32_t* op = &out.x;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float y0 = __uint_as_float(yp[q] << 16), y1 = __uint_as_float(yp[q] & 0xFFFF0000u);
        float t0 = __uint_as_float(tp[q] << 16), t1 = __uint_as_float(tp[q] & 0xFFFF0000u);
        float d0 = col_valid(col0 + 2 * q, seg_begin, seg_width, vc) ? y0 - t0 : 0.f;
        float d1 = col_valid(col0 + 2 * q + 1, seg_begin, seg_width, vc) ? y1 - t1 : 0.f;
        acc += d0 * d0 + d1 * d1;
        __nv_bfloat162 g = __floats2bfloat162_rn(k * d0, k * d1);
        op[q] = *reinterpret_cast<uint32_t*>(&g);
      }
      dy[c] = out;
    }
  } else {
    const float* y = static_cast<const float*>(y_) + (long long)s * n;
    const float* t = static_cast<const float*>(t_) + (long long)s * n;
    float* dy = static_cast<float*>(dy_) + (long long)s * n;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
      const int col = (int)(e % width);
      float d = col_valid(col, seg_begin, seg_width, vc) ? y[e] - t[e] : 0.f;
      acc += d * d;
      dy[e] = k * d;
    }
  }
  float tot = block_reduce_sum(acc, scratch);
  if (threadIdx.x == 0) partial[(long long)s * kMseBlocks + blockIdx.x] = tot;
}

// loss[s] = (sum of the subnet's partials, fixed order) / (T vc)
__global__ void mse_finish_kernel(const float* __restrict__ partial, int nblocks, int tokens, int width,
                                  const int32_t* __restrict__ valid_cols, int seg_begin, int seg_width,
                                  float* __restrict__ loss) {
  const int s = blockIdx.x, lane = threadIdx.x;
  double acc = 0.0;
  for (int i = lane; i < nblocks; i += 32) acc += (double)partial[(long long)s * kMseBlocks + i];
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const int vc = valid_cols ? min(max(valid_cols[s], 0), seg_width) : seg_width;
    const int n_valid = valid_count(width, seg_begin, seg_width, vc);
    loss[s] = n_valid > 0 ? (float)(acc / ((double)tokens * (double)n_valid)) : 0.f;
  }
}

// D[g] (M x N) = scale * op(A[g]) op(B[g]);  TA: A stored [K][M];  BNK: B stored [N][K] (else [K][N]).
template <bool TA, bool BNK>
__global__ void __launch_bounds__(256) sgemm_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                    float* __restrict__ D, int M, int N, int K, int lda, int ldb,
                                                    int ldd, long long sA, long long sB, long long sD, float scale) {
  __shared__ float As[16][17], Bs[16][17];
  const int g = blockIdx.z;
  A += g * sA; B += g * sB; D += g * sD;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m = blockIdx.y * 16 + ty, n = blockIdx.x * 16 + tx;
  float acc = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    {   // As[ty][tx] = A(m0+ty, k0+tx)
      int mm = blockIdx.y * 16 + ty, kk = k0 + tx;
      As[ty][tx] = (mm < M && kk < K) ? (TA ? A[(long long)kk * lda + mm] : A[(long long)mm * lda + kk]) : 0.f;
      int kb = k0 + ty, nn = blockIdx.x * 16 + tx;   // Bs[ty][tx] = B(k0+ty, n0+tx)
      Bs[ty][tx] = (kb < K && nn < N) ? (BNK ? B[(long long)nn * ldb + kb] : B[(long long)kb * ldb + nn]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) acc = fmaf(As[ty][k], Bs[k][tx], acc);
    __syncthreads();
  }
  if (m < M && n < N) D[(long long)m * ldd + n] = scale * acc;
}

__device__ inline float gelu_f(float x) { return 0.5f * x * (1.f + erff(x * 0.70710678118654752f)); }
__device__ inline float gelu_grad_f(float x) {
  return 0.5f * (1.f + erff(x * 0.70710678118654752f)) + x * 0.3989422804014327f * expf(-0.5f * x * x);
}

// pre [rows][g f] -> hh [rows][f]
__global__ void act_fwd_f32_kernel(const float* __restrict__ pre, float* __restrict__ hh, long long rows, int f, int kind) {
  const long long n = rows * f;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / f; const int j = (int)(e - r * f);
    if (kind == TWIST_FFN_SWIGLU) {
      float gte = pre[r * 2 * f + j], up = pre[r * 2 * f + f + j];
      hh[e] = gte / (1.f + expf(-gte)) * up;
    } else {
      float u = pre[e];
      hh[e] = kind == TWIST_FFN_RELU ? fmaxf(u, 0.f) : gelu_f(u);
    }
  }
}

// In place: dpre holds dHh (SwiGLU: in columns f..2f-1 of each row) and becomes the gradient w.r.t. pre.
__global__ void act_bwd_f32_kernel(const float* __restrict__ pre, float* __restrict__ dpre, long long rows, int f, int kind) {
  const long long n = rows * f;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / f; const int j = (int)(e - r * f);
    if (kind == TWIST_FFN_SWIGLU) {
      float gte = pre[r * 2 * f + j], up = pre[r * 2 * f + f + j], dh = dpre[r * 2 * f + f + j];
      float sg = 1.f / (1.f + expf(-gte));
      dpre[r * 2 * f + j] = dh * up * (sg * (1.f + gte * (1.f - sg)));
      dpre[r * 2 * f + f + j] = dh * (gte * sg);
    } else {
      float u = pre[e];
      dpre[e] = dpre[e] * (kind == TWIST_FFN_RELU ? (u > 0.f ? 1.f : 0.f) : gelu_grad_f(u));
    }
  }
}

__global__ void sgd_f32_kernel(float* __restrict__ w, const float* __restrict__ dw, float lr, long long n) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x)
    w[e] = w[e] - lr * dw[e];
}

int ew_grid(long long n) {
  long long b = (n + 255) / 256;
  long long cap = (long long)sm_count() * 8;
  return (int)(b < 1 ? 1 : (b < cap ? b : cap));
}

}  // namespace

int sgemm_f32(bool ta, bool bnk, const float* A, const float* B, float* D, int M, int N, int K, int lda, int ldb,
              int ldd, long long sA, long long sB, long long sD, int groups, float scale, cudaStream_t st) {
  dim3 grid((N + 15) / 16, (M + 15) / 16, groups);
  if (!ta && bnk) sgemm_kernel<false, true><<<grid, 256, 0, st>>>(A, B, D, M, N, K, lda, ldb, ldd, sA, sB, sD, scale);
  else if (!ta && !bnk) sgemm_kernel<false, false><<<grid, 256, 0, st>>>(A, B, D, M, N, K, lda, ldb, ldd, sA, sB, sD, scale);
  else if (ta && !bnk) sgemm_kernel<true, false><<<grid, 256, 0, st>>>(A, B, D, M, N, K, lda, ldb, ldd, sA, sB, sD, scale);
  else return TWIST_ERR_UNSUPPORTED;
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int act_fwd_f32(const float* pre, float* hh, long long rows, int f, int kind, cudaStream_t st) {
  act_fwd_f32_kernel<<<ew_grid(rows * f), 256, 0, st>>>(pre, hh, rows, f, kind);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int act_bwd_f32(const float* pre, float* dpre, long long rows, int f, int kind, cudaStream_t st) {
  act_bwd_f32_kernel<<<ew_grid(rows * f), 256, 0, st>>>(pre, dpre, rows, f, kind);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int sgd_f32(float* w, const float* dw, float lr, long long n, cudaStream_t st) {
  sgd_f32_kernel<<<ew_grid(n), 256, 0, st>>>(w, dw, lr, n);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

}  // namespace twist

extern "C" size_t twist_mse_workspace_bytes(int32_t n_subnets) {
  return n_subnets > 0 ? (size_t)n_subnets * twist::kMseBlocks * sizeof(float) : 0;
}

extern "C" int32_t twist_mse_fwd_bwd(const void* y, const void* tgt, void* dy, float* loss, int32_t n_subnets,
                                     int32_t tokens, int32_t width, const int32_t* valid_cols, int32_t seg_begin,
                                     int32_t seg_width, int32_t dtype, void* ws, size_t ws_bytes, void* stream) {
  using namespace twist;
  if (!y || !tgt || !dy || !loss) return TWIST_ERR_NULL;
  if (n_subnets <= 0 || tokens <= 0 || width <= 0) return TWIST_ERR_SHAPE;
  if (dtype != TWIST_FP32 && dtype != TWIST_BF16) return TWIST_ERR_SHAPE;
  if (dtype == TWIST_BF16 && width % 8 != 0) return TWIST_ERR_SHAPE;
  if (!aligned16(y) || !aligned16(tgt) || !aligned16(dy)) return TWIST_ERR_SHAPE;
  if (!valid_cols) { seg_begin = 0; seg_width = width; }
  if (seg_begin < 0 || seg_begin >= width || seg_width <= 0 || (width - seg_begin) % seg_width != 0) return TWIST_ERR_SHAPE;
  if (!ws || ws_bytes < twist_mse_workspace_bytes(n_subnets)) return TWIST_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long n = (long long)tokens * width;
  const long long work = dtype == TWIST_BF16 ? n / 8 : n;
  long long nb = (work + 256 * 4 - 1) / (256 * 4);
  const long long cap = ((long long)sm_count() * 8 + n_subnets - 1) / n_subnets;
  if (nb > cap) nb = cap;
  if (nb > kMseBlocks) nb = kMseBlocks;
  if (nb < 1) nb = 1;
  float* partial = static_cast<float*>(ws);
  if (dtype == TWIST_BF16)
    mse_kernel<true><<<dim3((unsigned)nb, n_subnets), 256, 0, st>>>(y, tgt, dy, tokens, width, valid_cols, seg_begin,
                                                                    seg_width, partial);
  else
    mse_kernel<false><<<dim3((unsigned)nb, n_subnets), 256, 0, st>>>(y, tgt, dy, tokens, width, valid_cols, seg_begin,
                                                                     seg_width, partial);
  TWIST_LAUNCH_CHECK();
  mse_finish_kernel<<<n_subnets, 32, 0, st>>>(partial, (int)nb, tokens, width, valid_cols, seg_begin, seg_width, loss);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the loss.  Its partial sums live in a file-scope device array, so a
// caller that cannot allocate (or was given no workspace to pass on) can still compute the loss.
// In host code `g_noalloc_partials` is only a handle for the runtime, not a device address: the
// address is looked up once per device and that pointer is what the kernels receive.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) float g_noalloc_partials[TWIST_NOALLOC_MAX_SUBNETS * twist::kMseBlocks];

namespace {
constexpr int kMaxDevices = 64;
float* g_noalloc_addr[kMaxDevices] = {nullptr};   // per device; written once, racing first calls write the same value

// Device address of the scratch array on the current device (first call per device does the lookup).
int noalloc_scratch(float** out) {
  int dev = -1;
  TWIST_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return TWIST_ERR_UNSUPPORTED;
  if (!g_noalloc_addr[dev]) {
    void* p = nullptr;
    TWIST_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_partials));
    if (!p) return TWIST_ERR_CUDA;
    g_noalloc_addr[dev] = static_cast<float*>(p);
  }
  *out = g_noalloc_addr[dev];
  return TWIST_OK;
}
}  // namespace

extern "C" int32_t twist_mse_fwd_bwd_noalloc(const void* y, const void* tgt, void* dy, float* loss, int32_t n_subnets,
                                             int32_t tokens, int32_t width, const int32_t* valid_cols,
                                             int32_t seg_begin, int32_t seg_width, int32_t dtype, void* stream) {
  if (n_subnets > TWIST_NOALLOC_MAX_SUBNETS) return TWIST_ERR_UNSUPPORTED;   // beyond the built-in scratch
  if (n_subnets <= 0) return TWIST_ERR_SHAPE;
  float* scratch = nullptr;
  int rc = noalloc_scratch(&scratch);
  if (rc != TWIST_OK) return rc;
  // Every partial sum that the finishing kernel reads is written by this call's first kernel, so the
  // contents left by an earlier call never need clearing.
  return twist_mse_fwd_bwd(y, tgt, dy, loss, n_subnets, tokens, width, valid_cols, seg_begin, seg_width, dtype, scratch,
                           (size_t)TWIST_NOALLOC_MAX_SUBNETS * twist::kMseBlocks * sizeof(float), stream);
}
