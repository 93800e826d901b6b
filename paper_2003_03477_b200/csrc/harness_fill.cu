// Device-side fill of synthetic tables with counter-based uniform values (input generation only).
#include "common.cuh"
#include "../../include/shadowsync_harness.h"

namespace ss {
__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

__global__ void __launch_bounds__(256)
fill_uniform_kernel(float* __restrict__ dst, int64_t count, uint64_t key, uint64_t counter0, float scale, float mid) {
  int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  const int64_t stride = (int64_t)gridDim.x * 256;
  for (; i < count; i += stride) {
    const uint64_t h = mix64(key + (counter0 + (uint64_t)i + 1ull) * 0x9E3779B97F4A7C15ull);
    const uint32_t u = (uint32_t)(h >> 32);
    const float x = __fadd_rn(__fmul_rn((float)(u >> 8), 5.9604644775390625e-8f), -0.5f);
    dst[i] = __fadd_rn(__fmul_rn(x, scale), mid);
  }
}
}  // namespace ss

extern "C" ss_status ssh_fill_uniform(float* dst, int64_t count, uint64_t key, uint64_t counter0, float scale,
                                      float mid, ss_stream stream) {
  if (!dst) return SS_ERR_NULL;
  if (count < 0) return SS_ERR_SHAPE;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  if (count == 0) return SS_OK;
  int64_t blocks = (count + 255) / 256;
  const int64_t cap = (int64_t)ss::num_sms() * 32;
  if (blocks > cap) blocks = cap;
  ss::fill_uniform_kernel<<<(unsigned)blocks, 256, 0, ss::as_stream(stream)>>>(dst, count, key, counter0, scale, mid);
  SS_LAUNCH_OK();
  return SS_OK;
}
