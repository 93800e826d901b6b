// Shared host-side plumbing of the library: status codes, CUDA error capture, argument checks.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "../../include/shadowsync.h"

namespace ss {

extern thread_local int g_last_cuda_error;

inline ss_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return SS_ERR_CUDA;
}

#define SS_CUDA(expr)                                  \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) return ss::cuda_fail(e__); \
  } while (0)

// Launch check: picks up a failed launch without synchronising.
#define SS_LAUNCH_OK()                                  \
  do {                                                  \
    cudaError_t e__ = cudaGetLastError();               \
    if (e__ != cudaSuccess) return ss::cuda_fail(e__);  \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline cudaStream_t as_stream(ss_stream s) { return reinterpret_cast<cudaStream_t>(s); }

// SS_OK when the current device is compute capability 10.x, cached per device.
ss_status check_arch();
int num_sms();

}  // namespace ss
