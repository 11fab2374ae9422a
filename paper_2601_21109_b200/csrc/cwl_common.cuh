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

// Programmatic dependent launch.  A kernel launched with launch_chained() may have its CTAs placed while the kernel
// before it in the stream is still running; it must call pdl_wait() before its first access to global memory, which
// returns once that kernel has completed and its writes are visible.  pdl_launch_dependents() lets the NEXT chained
// launch do the same with respect to this kernel.  Both do nothing in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// true while `stream` records into a CUDA graph (chained launches then keep the plain stream order)
inline bool stream_is_capturing(cudaStream_t stream) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) { cudaGetLastError(); return true; }
  return st != cudaStreamCaptureStatusNone;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(bool chained, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                  cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = chained ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace cwl
