// Shared host/device helpers of the CUDA library (never included by the CPU oracle).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "cwl.h"

#define CWL_CUDA_TRY(expr)                        \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) return CWL_ERR_CUDA;   \
  } while (0)

namespace cwl {

constexpr int kQ24 = 1 << 24;

// Records a device-side problem without trapping: bit `code` of the caller's status word.
__device__ __forceinline__ void flag_status(int32_t* status_word, int code) {
  if (status_word != nullptr) atomicOr(status_word, 1 << code);
}

__host__ __device__ __forceinline__ int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
__host__ __device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace cwl
