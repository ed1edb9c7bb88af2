// Host-side launchers of the small fp32 SIMT kernels behind the TWIST_FP32 path.
#pragma once
#include "common.cuh"

namespace twist {

// D[g] (M x N, ld ldd) = scale * op(A[g]) op(B[g]).  ta: A stored [K][M]; bnk: B stored [N][K], else [K][N].
int sgemm_f32(bool ta, bool bnk, const float* A, const float* B, float* D, int M, int N, int K, int lda, int ldb,
              int ldd, long long sA, long long sB, long long sD, int groups, float scale, cudaStream_t st);
int act_fwd_f32(const float* pre, float* hh, long long rows, int f, int kind, cudaStream_t st);
int act_bwd_f32(const float* pre, float* dpre, long long rows, int f, int kind, cudaStream_t st);
int sgd_f32(float* w, const float* dw, float lr, long long n, cudaStream_t st);

}  // namespace twist
