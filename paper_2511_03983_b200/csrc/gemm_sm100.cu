// Host side of the grouped tcgen05 GEMM: tensor-map encoding and kernel dispatch.
#include "gemm_sm100.cuh"

#include <cudaTypedefs.h>

#include <mutex>

#include "plan.cuh"

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

// Encodes a 3-D tiled bf16 tensor map, or takes it from the calling thread's active plan (plan.cuh).
int encode_or_cached(CUtensorMap* map, const void* ptr, const cuuint64_t dims[3], const cuuint64_t strides[2],
                     const cuuint32_t box[3], CUtensorMapSwizzle swizzle, CUtensorMapL2promotion promotion,
                     const char* what, CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16) {
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.ptr = ptr;
  for (int i = 0; i < 3; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  key.strides[0] = strides[0]; key.strides[1] = strides[1];
  key.swizzle = (unsigned)swizzle; key.promotion = (unsigned)promotion | ((unsigned)dtype << 16);
  if (plan_lookup(key, map)) return TWIST_OK;
  EncodeTiledFn fn = encode_fn();
  if (!fn) { note_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled entry point"); return TWIST_ERR_CUDA; }
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, dtype, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, promotion, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    note_cuda_error(cudaErrorInvalidValue, what);
    return TWIST_ERR_CUDA;
  }
  plan_store(key, *map);
  return TWIST_OK;
}

// 3-D map over dense bf16 [groups][rows][cols]; box = 64 contiguous elements x box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero (ragged M / N / K tails need no special code).
int make_map(CUtensorMap* map, const GemmOperand& op, int groups, int box_rows) {
  cuuint64_t dims[3] = {(cuuint64_t)op.cols, (cuuint64_t)op.rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)op.cols * 2, (cuuint64_t)op.rows * (cuuint64_t)op.cols * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  return encode_or_cached(map, op.ptr, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          "cuTensorMapEncodeTiled");
}

// CTA pairs that can be resident at once (one CTA per SM, pairs on neighbouring SMs); queried once per
// kernel instance and device.  More tiles than pairs: the persistent pairs stride over the tile list.
template <int AM, int BM_, int EPI, bool HINTED>
int resident_pairs(int* out) {
  static int cached[64] = {0};
  int dev = 0;
  TWIST_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return TWIST_ERR_UNSUPPORTED;
  if (cached[dev] == 0) {
    TWIST_CUDA_TRY(cudaFuncSetAttribute(gemm_kernel<AM, BM_, EPI, HINTED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        gemm_smem_bytes(EPI)));
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(2 * (sm_count() / 2));
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = gemm_smem_bytes(EPI);
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_kernel<AM, BM_, EPI, HINTED>, &cfg) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = sm_count() / 2;
    }
    cached[dev] = n < sm_count() / 2 ? n : sm_count() / 2;
  }
  *out = cached[dev];
  return TWIST_OK;
}

// 3-D map over a bf16 tensor [groups][rows][cols] whose rows are `row_stride` elements apart, for the
// epilogue's 32 x 32 boxes (64-byte rows in shared memory, 64-byte swizzle).  Loads read zeros outside
// the tensor, stores write nothing there.
int make_box_map(CUtensorMap* map, const void* ptr, int rows, int cols, long long row_stride, int groups) {
  if (!ptr || !aligned16(ptr) || (row_stride * 2) % 16 != 0) return TWIST_ERR_SHAPE;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)row_stride * 2, (cuuint64_t)rows * (cuuint64_t)row_stride * 2};
  cuuint32_t box[3] = {32, 32, 1};
  return encode_or_cached(map, ptr, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          "cuTensorMapEncodeTiled (epilogue box)");
}

// The same box geometry (64-byte rows, 32 rows, 64-byte swizzle) over an fp32 tensor [groups][rows][cols]: 16 columns.
int make_box_map_f32(CUtensorMap* map, const void* ptr, int rows, int cols, int groups) {
  if (!ptr || !aligned16(ptr) || cols % 4 != 0) return TWIST_ERR_SHAPE;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)rows * (cuuint64_t)cols * 4};
  cuuint32_t box[3] = {16, 32, 1};
  return encode_or_cached(map, ptr, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          "cuTensorMapEncodeTiled (fp32 epilogue box)", CU_TENSOR_MAP_DATA_TYPE_FLOAT32);
}

// Tensor maps of the boxes each epilogue reads and writes (layout of EpiMaps in the kernel header).
int make_epilogue_maps(int epi, const GemmParams& p, const CUtensorMap& filler, EpiMaps* e) {
  for (int i = 0; i < 4; ++i) e->m[i] = filler;          // unused entries stay valid descriptors
  const int M = p.M, N = p.N, G = p.groups;
  int rc = TWIST_OK;
  auto mk = [&](int i, const void* ptr, int cols, long long stride) {
    if (rc == TWIST_OK) rc = make_box_map(&e->m[i], ptr, M, cols, stride, G);
  };
  switch (epi) {
    case EPI_STORE: mk(0, p.out0, N, N); break;
    case EPI_MSE: mk(0, p.in0, N, N); mk(1, p.out1, N, N); mk(2, p.out0, N, N); break;
    case EPI_MSE_NOY: mk(0, p.in0, N, N); mk(1, p.out1, N, N); break;
    case EPI_SWIGLU_FWD: mk(0, p.out0, N, 2LL * N); mk(1, p.out0 + N, N, 2LL * N); mk(2, p.out1, N, N); break;
    case EPI_ACT_FWD: mk(0, p.out0, N, N); mk(1, p.out1, N, N); break;
    case EPI_DSWIGLU:
      mk(0, p.in0, N, 2LL * N); mk(1, p.in0 + N, N, 2LL * N);
      mk(2, p.out0, N, 2LL * N); mk(3, p.out0 + N, N, 2LL * N);
      break;
    case EPI_DACT:
    case EPI_RESID: mk(0, p.in0, N, N); mk(1, p.out0, N, N); break;
    case EPI_SGD:
    case EPI_SGD_LONG:                                     // staged only when the launch updates the weights
      if (p.lr != 0.f || p.master_init) {
        if (rc == TWIST_OK) rc = make_box_map_f32(&e->m[0], p.master, M, N, G);
        mk(2, p.out0, N, N);
      }
      break;
    default: break;                                        // EPI_ADAM: plain global accesses
  }
  return rc;
}

// Wave synchronisation, host side.  One never-reset device counter per stream (up to kWaveSlots streams per device;
// further streams run unsynchronised); the host keeps the value each counter will have when the launches issued so
// far on its stream have finished.  Launches on one stream are ordered, so they can share a counter.
constexpr int kSgdLongK = 8192;         // contraction length from which the fused SGD update keeps the full operand ring
constexpr size_t kHintMinABytes = (size_t)32 << 20;   // A rows of one group from which a token-major launch uses L2 hints
constexpr int kPdlMaxWaves = 32;        // launches of at most this many waves of tiles are launched programmatically
constexpr int kWaveSlots = 64;
constexpr int kWaveMinKBlocks = 32;     // contractions shorter than this (K < 2048) lose more to the wait than they save
__device__ unsigned g_wave_ctr[kWaveSlots];
__device__ unsigned g_done_ctr[kWaveSlots];     // GemmParams::done_ctr, one per stream like the wave counters
struct WaveState {
  std::mutex mu;
  unsigned* dev = nullptr;              // device address of g_wave_ctr on this device
  unsigned* done = nullptr;             // ... and of g_done_ctr
  cudaStream_t owner[kWaveSlots];
  unsigned base[kWaveSlots];
  int used = 0;
};
WaveState g_wave[64];

// Picks the counter of stream `st` and reserves n_waves * grid arrivals on it.  Returns false when the launch
// should run without wave synchronisation.
// Slot of stream `st` in the per-stream counter tables (w.mu held); -1: none left, or the stream is being captured
// (the counters' sequence lives partly on the host and a captured launch may be replayed on any stream).
int stream_slot(WaveState& w, cudaStream_t st) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) {
    cudaGetLastError();
    return -1;
  }
  if (!w.dev) {
    void *a = nullptr, *b = nullptr;
    if (cudaGetSymbolAddress(&a, g_wave_ctr) != cudaSuccess || cudaGetSymbolAddress(&b, g_done_ctr) != cudaSuccess || !a || !b) {
      cudaGetLastError();
      return -1;
    }
    w.dev = static_cast<unsigned*>(a);
    w.done = static_cast<unsigned*>(b);
  }
  for (int i = 0; i < w.used; ++i)
    if (w.owner[i] == st) return i;
  if (w.used == kWaveSlots) return -1;
  w.owner[w.used] = st;
  w.base[w.used] = 0;
  return w.used++;
}

// Picks the counter of stream `st` and reserves n_waves * grid arrivals on it.  Returns false when the launch
// should run without wave synchronisation.
bool wave_reserve(cudaStream_t st, int n_waves, int grid, GemmParams* p) {
  WaveState& w = g_wave[device_slot()];
  std::lock_guard<std::mutex> lock(w.mu);
  const int slot = stream_slot(w, st);
  if (slot < 0) return false;
  p->wave_ctr = w.dev + slot;
  p->wave_base = w.base[slot];
  p->n_waves = n_waves;
  w.base[slot] += (unsigned)n_waves * (unsigned)grid;       // wraps like the device counter
  return true;
}
// Takes a reservation back (the launch did not happen).
void wave_unreserve(const GemmParams& p, int grid) {
  WaveState& w = g_wave[device_slot()];
  std::lock_guard<std::mutex> lock(w.mu);
  w.base[p.wave_ctr - w.dev] -= (unsigned)p.n_waves * (unsigned)grid;
}

template <int AM, int BM_, int EPI, bool HINTED>
int launch_as(const CUtensorMap& ta, const CUtensorMap& tb, GemmParams p, cudaStream_t st) {
  int pairs = 0;
  int rc = resident_pairs<AM, BM_, EPI, HINTED>(&pairs);
  if (rc != TWIST_OK) return rc;
  const int tiles = p.groups * p.m_tiles * p.n_tiles;
  const int grid = 2 * (tiles < pairs ? tiles : pairs);
  EpiMaps te;
  rc = make_epilogue_maps(EPI, p, ta, &te);
  if (rc != TWIST_OK) return rc;
  const int smem = gemm_smem_bytes(EPI);
  const int n_waves = (tiles + grid / 2 - 1) / (grid / 2);
  p.wave_ctr = nullptr;
  if (n_waves >= 2 && (p.K + kBK - 1) / kBK >= kWaveMinKBlocks && wave_reserve(st, n_waves, grid, &p)) {
    // cooperative: the grid starts only when all of its CTAs can be resident, so the waits cannot starve
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeCooperative;
    attr.val.cooperative = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, gemm_kernel<AM, BM_, EPI, HINTED>, ta, tb, te, p) == cudaSuccess) return TWIST_OK;
    cudaGetLastError();                 // not launchable that way here: run it unsynchronised
    wave_unreserve(p, grid);
    p.wave_ctr = nullptr;
  }
  // Short launches (a few waves of tiles, where start-up is a visible share: the d = 768 shapes gained 1.1 %):
  // programmatic stream serialisation, so that the CTAs' set-up (barriers, tensor-memory allocation, the pair's
  // rendezvous) overlaps the tail of the previous launch.  The kernel waits for that launch to complete before it
  // reads anything.  Not inside a stream capture.
  if (n_waves <= kPdlMaxWaves) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
      cudaLaunchConfig_t cfg;
      memset(&cfg, 0, sizeof(cfg));
      cfg.gridDim = dim3(grid);
      cfg.blockDim = dim3(kGemmThreads);
      cfg.dynamicSmemBytes = smem;
      cfg.stream = st;
      cudaLaunchAttribute attr;
      attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr.val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = &attr;
      cfg.numAttrs = 1;
      if (cudaLaunchKernelEx(&cfg, gemm_kernel<AM, BM_, EPI, HINTED>, ta, tb, te, p) == cudaSuccess) return TWIST_OK;
    }
    cudaGetLastError();                   // not launchable that way: plain launch
  }
  gemm_kernel<AM, BM_, EPI, HINTED><<<grid, kGemmThreads, smem, st>>>(ta, tb, te, p);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

// L2 eviction priorities, for token-major launches (A = activation rows, B = a weight slice) whose activations do not
// fit in L2 anyway: the weight slice is what every wave of tiles reads again, the activation rows pass through once,
// and so does what the epilogue reads and writes - without the hints the stream of activations and results pushes
// the weights out between waves (7B shapes, 8192 tokens: the up-projection read 2.05 GB from DRAM for 0.9 GB of
// operands, 1.75 GB with them; the dX launch 2.41 -> 1.63 GB; the 32768-token round gained 0.5 - 0.9 % over the
// plain copies).  Smaller launches, whose results the next launch finds in L2, lose 1 - 2 % to any hint;
// weight-gradient launches (both operands stream along the contraction) gain nothing; launches too short for wave
// synchronisation lose 6 % (their tiles drift apart, and an activation row marked evict-first is gone before the
// last tile of the wave asks for it).  All of those keep the plain copies.
template <int AM, int BM_, int EPI>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, GemmParams p, cudaStream_t st) {
  if constexpr (AM == MAJOR_K) {
    if ((size_t)p.M * (size_t)p.K * 2 >= kHintMinABytes && (p.K + kBK - 1) / kBK >= kWaveMinKBlocks) {
      p.hint_a = L2_EVICT_FIRST;
      p.hint_b = L2_EVICT_LAST;
      p.hint_epi = L2_EVICT_FIRST;
      return launch_as<AM, BM_, EPI, true>(ta, tb, p, st);
    }
  }
  return launch_as<AM, BM_, EPI, false>(ta, tb, p, st);
}

// loss[g] = (sum of the group's partial sums, fixed order) / (tokens * valid columns of the group)
__global__ void fused_loss_finish_kernel(const float* __restrict__ partial, long long per_group, int tokens, int width,
                                         const int32_t* __restrict__ valid_cols, int seg_begin, int seg_width,
                                         float* __restrict__ loss) {
  const int g = blockIdx.x, lane = threadIdx.x;
  const float* src = partial + (long long)g * per_group;
  double acc = 0.0;
  for (long long i = lane; i < per_group; i += 32) acc += (double)src[i];
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) {
    const int vc = valid_cols ? min(max(valid_cols[g], 0), seg_width) : seg_width;
    const long long n_valid = seg_begin + (long long)((width - seg_begin) / seg_width) * vc;
    loss[g] = n_valid > 0 ? (float)(acc / ((double)tokens * (double)n_valid)) : 0.f;
  }
}

// Self-test of the give-up path: a CTA pair with the GEMM's roles, barriers nobody ever arrives at, the same bounded
// wait (with a short limit) and the same exit (abort flag, drain, pair barrier, tensor-memory release).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
selftest_wait_kernel(unsigned long long limit_ns, int* status) {
  __shared__ __align__(8) unsigned long long bars[3];
  __shared__ uint32_t tmem_slot_s;
  __shared__ int abort_s;
  volatile uint32_t* tmem_slot = &tmem_slot_s;
  volatile int* abort_flag = &abort_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == kEpiWarps && lane == 0) {
    for (int i = 0; i < 3; ++i) mbar_init(smem_u32(&bars[i]), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kEpiWarps + 1) pair_tmem_alloc(tmem_slot, 32u);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  if (warp == kEpiWarps) {                       // producer role: "stage empty" never comes
    if (lane == 0) mbar_wait_for(smem_u32(&bars[0]), 0, abort_flag, status, limit_ns);
  } else if (warp == kEpiWarps + 1) {            // MMA issuer role (leader only): "stage full" never comes
    if (lane == 0 && cluster_rank() == 0) mbar_wait_for(smem_u32(&bars[1]), 0, abort_flag, status, limit_ns);
  } else {                                       // epilogue role: "accumulator full" never comes; warp-uniform outcome
    (void)__all_sync(0xffffffffu, mbar_wait_for(smem_u32(&bars[2]), 0, abort_flag, status, limit_ns));
  }
  pair_teardown(abort_flag, warp == kEpiWarps + 1, tmem_base, 32u);
}

}  // namespace

// After a kernel gave up (a bounded wait ran out) its wave counter is short of what the host booked: start over.
// Called with the device idle.
void reset_wave_sync() {
  WaveState& w = g_wave[device_slot()];
  std::lock_guard<std::mutex> lock(w.mu);
  static const unsigned zeros[kWaveSlots] = {0};
  if (cudaMemcpyToSymbol(g_wave_ctr, zeros, sizeof(zeros)) != cudaSuccess) cudaGetLastError();
  if (cudaMemcpyToSymbol(g_done_ctr, zeros, sizeof(zeros)) != cudaSuccess) cudaGetLastError();
  for (int i = 0; i < kWaveSlots; ++i) w.base[i] = 0;
}

int encode_map_3d_bf16(CUtensorMap* map, const void* ptr, const unsigned long long dims[3],
                       const unsigned long long strides[2], const unsigned box[3], int swizzle_bytes) {
  if (!ptr || !aligned16(ptr) || strides[0] % 16 || strides[1] % 16) return TWIST_ERR_SHAPE;
  cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
  cuuint64_t st[2] = {strides[0], strides[1]};
  cuuint32_t bx[3] = {box[0], box[1], box[2]};
  return encode_or_cached(map, ptr, d, st, bx, swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, "cuTensorMapEncodeTiled");
}

size_t fused_loss_partials(int groups, int M, int N) {
  const size_t m_tiles = (size_t)(M + kBM - 1) / kBM, n_tiles = (size_t)(N + kBN - 1) / kBN;
  return (size_t)groups * m_tiles * n_tiles * 2 * kEpiWarps;
}

unsigned* fused_loss_counter(cudaStream_t st) {
  WaveState& w = g_wave[device_slot()];
  std::lock_guard<std::mutex> lock(w.mu);
  const int slot = stream_slot(w, st);
  return slot < 0 ? nullptr : w.done + slot;
}

int finish_fused_loss(const float* partial, int groups, int M, int N, const int32_t* valid_cols, int seg_begin,
                      int seg_width, float* loss, cudaStream_t st) {
  const long long per_group = (long long)(fused_loss_partials(groups, M, N) / (size_t)groups);
  fused_loss_finish_kernel<<<groups, 32, 0, st>>>(partial, per_group, M, N, valid_cols, seg_begin, seg_width, loss);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}

int launch_gemm_bf16(int layout, int epi, const GemmOperand& A, const GemmOperand& B, GemmParams p, cudaStream_t st) {
  if (!A.ptr || !B.ptr) return TWIST_ERR_NULL;
  if (p.M <= 0 || p.N <= 0 || p.K <= 0 || p.groups <= 0) return TWIST_ERR_SHAPE;
  if (A.cols % 8 || B.cols % 8 || p.N % 8) return TWIST_ERR_SHAPE;            // 16-byte rows for TMA and the epilogue
  if (!aligned16(A.ptr) || !aligned16(B.ptr)) return TWIST_ERR_SHAPE;
  const int a_major = layout == 2 ? MAJOR_MN : MAJOR_K;
  const int b_major = layout == 0 ? MAJOR_K : MAJOR_MN;
  p.m_tiles = (p.M + kBM - 1) / kBM;
  p.n_tiles = epi == EPI_SWIGLU_FWD ? (p.N + kCtaN - 1) / kCtaN : (p.N + kBN - 1) / kBN;
  if ((long long)p.groups * p.m_tiles * p.n_tiles > 0x7fffffffLL) return TWIST_ERR_UNSUPPORTED;
  p.raster_m = layout == 2 ? 8 : 1;      // see tile_coords
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
      case EPI_MSE: return launch<MAJOR_K, MAJOR_K, EPI_MSE>(ta, tb, p, st);
      case EPI_MSE_NOY: return launch<MAJOR_K, MAJOR_K, EPI_MSE_NOY>(ta, tb, p, st);
      default: return TWIST_ERR_UNSUPPORTED;
    }
  }
  if (layout == 1 && epi == EPI_STORE) return launch<MAJOR_K, MAJOR_MN, EPI_STORE>(ta, tb, p, st);
  if (layout == 1 && epi == EPI_MSE) return launch<MAJOR_K, MAJOR_MN, EPI_MSE>(ta, tb, p, st);
  if (layout == 1 && epi == EPI_MSE_NOY) return launch<MAJOR_K, MAJOR_MN, EPI_MSE_NOY>(ta, tb, p, st);
  if (layout == 1 && epi == EPI_RESID) return launch<MAJOR_K, MAJOR_MN, EPI_RESID>(ta, tb, p, st);
  if (layout == 2 && epi == EPI_SGD) {
    // staged update, except at the longest contractions (see gemm_stages)
    if (p.K >= kSgdLongK) return launch<MAJOR_MN, MAJOR_MN, EPI_SGD_LONG>(ta, tb, p, st);
    return launch<MAJOR_MN, MAJOR_MN, EPI_SGD>(ta, tb, p, st);
  }
  if (layout == 2 && epi == EPI_ADAM) return launch<MAJOR_MN, MAJOR_MN, EPI_ADAM>(ta, tb, p, st);
  return TWIST_ERR_UNSUPPORTED;
}

}  // namespace twist

extern "C" int32_t twist_selftest_wait(uint64_t limit_ns, void* stream) {
  using namespace twist;
  if (limit_ns == 0 || limit_ns > 100000000ull) return TWIST_ERR_SHAPE;       // at most 0.1 s
  int* status = device_status_ptr();
  if (!status) return TWIST_ERR_CUDA;
  selftest_wait_kernel<<<2, kGemmThreads, 0, static_cast<cudaStream_t>(stream)>>>(limit_ns, status);
  TWIST_LAUNCH_CHECK();
  return TWIST_OK;
}
