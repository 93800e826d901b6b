// Status strings, device checks, float->bf16 conversion.
#include "common.cuh"

namespace ss {
thread_local int g_last_cuda_error = 0;

static int g_arch_ok[64];   // 0 unknown, 1 ok, -1 not sm_100
static int g_sms[64];

ss_status check_arch() {
  int dev = 0;
  SS_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SS_ERR_ARCH;
  if (g_arch_ok[dev] == 0) {
    int major = 0, sms = 0;
    SS_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    SS_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    g_sms[dev] = sms;
    g_arch_ok[dev] = (major == 10) ? 1 : -1;
  }
  return g_arch_ok[dev] == 1 ? SS_OK : SS_ERR_ARCH;
}

int num_sms() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (g_arch_ok[dev] == 0) check_arch();
  return g_sms[dev] > 0 ? g_sms[dev] : 148;
}

__global__ void to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += stride) dst[i] = __float2bfloat16_rn(src[i]);
}
}  // namespace ss

extern "C" {

const char* ss_status_str(ss_status s) {
  switch (s) {
    case SS_OK: return "ok";
    case SS_ERR_NULL: return "a required pointer is NULL";
    case SS_ERR_SHAPE: return "bad shape or size";
    case SS_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
    case SS_ERR_DTYPE: return "unsupported dtype or missing bf16 buffer";
    case SS_ERR_WORKSPACE: return "workspace too small";
    case SS_ERR_ARCH: return "device is not sm_100";
    case SS_ERR_CUDA: return "CUDA call failed (see ss_last_cuda_error)";
    case SS_ERR_RANGE: return "scalar argument out of range";
    default: return "unknown status";
  }
}

int ss_last_cuda_error(void) { return ss::g_last_cuda_error; }

int ss_num_sms(void) {
  if (ss::check_arch() == SS_ERR_CUDA) return -1;
  return ss::num_sms();
}

ss_status ss_to_bf16(const float* src, void* dst, int64_t n, ss_stream stream) {
  if (!src || !dst) return SS_ERR_NULL;
  if (n < 0) return SS_ERR_SHAPE;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  if (n == 0) return SS_OK;
  int64_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  ss::to_bf16_kernel<<<(unsigned)blocks, 256, 0, ss::as_stream(stream)>>>(src, (__nv_bfloat16*)dst, n);
  SS_LAUNCH_OK();
  return SS_OK;
}

}  // extern "C"
