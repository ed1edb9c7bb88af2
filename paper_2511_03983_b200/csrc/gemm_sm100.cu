// Host side of the grouped tcgen05 GEMM: tensor-map encoding and kernel dispatch.
#include "gemm_sm100.cuh"

#include <cudaTypedefs.h>

namespace twist {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 3-D map over dense bf16 [groups][rows][cols]; box = 64 contiguous elements x box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero (ragged M / N / K tails need no special code).
int make_map(CUtensorMap* map, const GemmOperand& op, int groups, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) { note_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled entry point"); return TWIST_ERR_CUDA; }
  cuuint64_t dims[3] = {(cuuint64_t)op.cols, (cuuint64_t)op.rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)op.cols * 2, (cuuint64_t)op.rows * (cuuint64_t)op.cols * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(op.ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    note_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return TWIST_ERR_CUDA;
  }
  return TWIST_OK;
}

template <int AM, int BM_, int EPI>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(gemm_kernel<AM, BM_, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kGemmSmemBytes));
    configured = true;
  }
  const int tiles = p.groups * p.m_tiles * p.n_tiles;
  const int grid = tiles < sm_count() ? tiles : sm_count();
  gemm_kernel<AM, BM_, EPI><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(ta, tb, p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

}  // namespace

int launch_gemm_bf16(int layout, int epi, const GemmOperand& A, const GemmOperand& B, GemmParams p, cudaStream_t st) {
  if (!A.ptr || !B.ptr) return TWIST_ERR_NULL;
  if (p.M <= 0 || p.N <= 0 || p.K <= 0 || p.groups <= 0) return TWIST_ERR_SHAPE;
  if (A.cols % 8 || B.cols % 8 || p.N % 8) return TWIST_ERR_SHAPE;            // 16-byte rows for TMA and the epilogue
  if (!aligned16(A.ptr) || !aligned16(B.ptr)) return TWIST_ERR_SHAPE;
  const int a_major = layout == 2 ? MAJOR_MN : MAJOR_K;
  const int b_major = layout == 0 ? MAJOR_K : MAJOR_MN;
  p.m_tiles = (p.M + kBM - 1) / kBM;
  p.n_tiles = epi == EPI_SWIGLU_FWD ? (p.N + kBN / 2 - 1) / (kBN / 2) : (p.N + kBN - 1) / kBN;
  if ((long long)p.groups * p.m_tiles * p.n_tiles > 0x7fffffffLL) return TWIST_ERR_UNSUPPORTED;
  p.status = device_status_ptr();
  if (!p.status) return TWIST_ERR_CUDA;
  CUtensorMap ta, tb;
  int rc = make_map(&ta, A, p.groups, a_major == MAJOR_K ? 128 : 64);
  if (rc != TWIST_OK) return rc;
  rc = make_map(&tb, B, p.groups, b_major == MAJOR_K ? 128 : 64);
  if (rc != TWIST_OK) return rc;
  if (layout == 0) {
    switch (epi) {
      case EPI_STORE: return launch<MAJOR_K, MAJOR_K, EPI_STORE>(ta, tb, p, st);
      case EPI_SWIGLU_FWD: return launch<MAJOR_K, MAJOR_K, EPI_SWIGLU_FWD>(ta, tb, p, st);
      case EPI_ACT_FWD: return launch<MAJOR_K, MAJOR_K, EPI_ACT_FWD>(ta, tb, p, st);
      case EPI_DSWIGLU: return launch<MAJOR_K, MAJOR_K, EPI_DSWIGLU>(ta, tb, p, st);
      case EPI_DACT: return launch<MAJOR_K, MAJOR_K, EPI_DACT>(ta, tb, p, st);
      default: return TWIST_ERR_UNSUPPORTED;
    }
  }
  if (layout == 1 && epi == EPI_STORE) return launch<MAJOR_K, MAJOR_MN, EPI_STORE>(ta, tb, p, st);
  if (layout == 2 && epi == EPI_SGD) return launch<MAJOR_MN, MAJOR_MN, EPI_SGD>(ta, tb, p, st);
  return TWIST_ERR_UNSUPPORTED;
}

}  // namespace twist
