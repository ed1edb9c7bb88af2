// Shared host/device helpers of the TwIST CUDA library (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "../../include/twist.h"

namespace twist {

// Device status word: a kernel whose bounded wait expires stores TWIST_ERR_DEVICE_TIMEOUT there.
// Kernels receive its device address as an argument (one word per device, defined in common.cu).
int* device_status_ptr();

void note_cuda_error(cudaError_t e, const char* where);
// Resets the grouped GEMM's wave-synchronisation counters of the current device (device idle); gemm_sm100.cu.
void reset_wave_sync();
int sm_count();
// Index of the current device for per-device caches (kernel attributes are per device), 0 when it cannot be read
// or exceeds the cache size.
inline int device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  return dev;
}

#define TWIST_CUDA_TRY(expr)                                   \
  do {                                                         \
    cudaError_t e__ = (expr);                                  \
    if (e__ != cudaSuccess) {                                  \
      ::twist::note_cuda_error(e__, #expr);                    \
      return TWIST_ERR_CUDA;                                   \
    }                                                          \
  } while (0)

#define TWIST_LAUNCH_CHECK() TWIST_CUDA_TRY(cudaPeekAtLastError())

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace twist
