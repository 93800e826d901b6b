// GEMM interface shared by the SIMT and the tensor-core kernels of the MLP.
//
//   C[m, n] = sum_k A(m, k) * B(n, k)        m < M, n < N, k < K
//
// followed by one epilogue: + bias[n], ReLU, multiply by (mask[m, n] > 0) for n < mask_cols, then
// columns [0, lo_cols) go to out_lo (float or bf16, leading dimension ld_lo) and columns
// [lo_cols, N) to the float matrix out_hi at column n - lo_cols.
#pragma once
#include "common.cuh"

namespace ss {

enum OperandKind { OP_F32 = 0, OP_BF16 = 1, OP_F32_ROUND_BF16 = 2 };

struct Epilogue {
  const float* bias = nullptr;
  int relu = 0;
  const void* mask = nullptr;   // activation whose sign gates the gradient
  int mask_bf16 = 0;
  int64_t ld_mask = 0;
  int mask_cols = 0;
  void* out_lo = nullptr;
  int lo_bf16 = 0;
  int64_t ld_lo = 0;
  int lo_cols = 0;
  float* out_hi = nullptr;
  int64_t ld_hi = 0;
};

struct Operand {
  const void* p;
  int kind;            // OperandKind
  int64_t s_row, s_k;  // element strides: A(m,k) = p[m*s_row + k*s_k]
};

// Any shape, any strides; fp32 FMA accumulation in ascending k.
ss_status gemm_simt(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st);
// bf16 operands on the tensor cores (tcgen05); see gemm_tc_eligible for what it accepts.
bool gemm_tc_eligible(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep);
// k_splits > 1 cuts K into slices computed by different CTAs; slice z stores its fp32 partial product at
// out_lo + z * split_stride (plain stores only: no bias, ReLU, mask or bf16 output); the caller adds the slices.
ss_status gemm_tc(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st,
                  int k_splits, int64_t split_stride);
// Several independent products (each eligible for gemm_tc, at most kTcMaxGroup) in ONE launch of 128 x 128 tiles.
constexpr int kTcMaxGroup = 4;
struct TcJob {
  int M, N, K;
  Operand A, B;
  Epilogue ep;
  int k_splits;
  int64_t split_stride;
};
ss_status gemm_tc_group(const TcJob* jobs, int n, cudaStream_t st);
// Tensor cores when eligible, SIMT otherwise.
ss_status gemm(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st);
// The device error flag raised by a bounded wait that ran out (0 = none); synchronises the device.
int read_device_error(bool clear);

__device__ __forceinline__ float epilogue_value(const Epilogue& ep, float v, int64_t m, int n) {
  if (ep.bias) v += ep.bias[n];
  if (ep.relu) v = fmaxf(v, 0.f);
  if (ep.mask && n < ep.mask_cols) {
    const float a = ep.mask_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(ep.mask)[m * ep.ld_mask + n])
                                 : reinterpret_cast<const float*>(ep.mask)[m * ep.ld_mask + n];
    if (!(a > 0.f)) v = 0.f;
  }
  return v;
}

__device__ __forceinline__ void epilogue_store(const Epilogue& ep, float v, int64_t m, int n) {
  if (n < ep.lo_cols) {
    if (ep.lo_bf16) {
      reinterpret_cast<__nv_bfloat16*>(ep.out_lo)[m * ep.ld_lo + n] = __float2bfloat16_rn(v);
    } else {
      reinterpret_cast<float*>(ep.out_lo)[m * ep.ld_lo + n] = v;
    }
  } else if (ep.out_hi) {
    ep.out_hi[m * ep.ld_hi + (n - ep.lo_cols)] = v;
  }
}

}  // namespace ss
