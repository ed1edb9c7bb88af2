// Status plumbing of the C ABI: error strings, last CUDA error, device status word.
#include "common.cuh"

namespace twist {

static __device__ int g_device_status = 0;

static thread_local char t_cuda_error[256] = "";

void note_cuda_error(cudaError_t e, const char* where) {
  snprintf(t_cuda_error, sizeof(t_cuda_error), "%s: %s (%s)", cudaGetErrorName(e), cudaGetErrorString(e), where);
  cudaGetLastError();  // clear the sticky-less error so later launches are not blamed for it
}

int* device_status_ptr() {
  int* p = nullptr;
  if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_device_status) != cudaSuccess) return nullptr;
  return p;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace twist

extern "C" {

uint32_t twist_abi_version(void) { return 3u; }

const char* twist_strerror(int32_t status) {
  switch (status) {
    case TWIST_OK: return "ok";
    case TWIST_ERR_NULL: return "a required pointer is NULL";
    case TWIST_ERR_SHAPE: return "bad shape, size or alignment";
    case TWIST_ERR_INFEASIBLE: return "subnet size violates (N_full + (S-1)|C|)/S <= N_sub <= N_full";
    case TWIST_ERR_BAD_INDEX: return "index array entry out of range or unsorted";
    case TWIST_ERR_UNSUPPORTED: return "request outside the implemented range";
    case TWIST_ERR_WORKSPACE: return "workspace missing or too small";
    case TWIST_ERR_CUDA: return "CUDA call failed";
    case TWIST_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
  }
}

const char* twist_last_cuda_error(void) { return twist::t_cuda_error; }

int32_t twist_device_status(int32_t* code) {
  if (!code) return TWIST_ERR_NULL;
  int v = 0;
  TWIST_CUDA_TRY(cudaDeviceSynchronize());
  TWIST_CUDA_TRY(cudaMemcpyFromSymbol(&v, twist::g_device_status, sizeof(int)));
  if (v != 0) {
    int zero = 0;
    TWIST_CUDA_TRY(cudaMemcpyToSymbol(twist::g_device_status, &zero, sizeof(int)));
    if (v == TWIST_ERR_DEVICE_TIMEOUT) twist::reset_wave_sync();      // a kernel that gave up left its wave count short
  }
  *code = v;
  return TWIST_OK;
}

}  // extern "C"
