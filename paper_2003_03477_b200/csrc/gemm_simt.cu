// SIMT GEMM with arbitrary operand strides: the float path of the small configuration and the
// layers that are no dense contraction (13 input features, a single output logit).
#include "gemm.cuh"
#include "profile.cuh"

namespace ss {

constexpr int kTM = 64, kTN = 64, kTK = 16;

template <int KIND>
__device__ __forceinline__ float load_op(const void* p, int64_t i) {
  if (KIND == OP_F32) return reinterpret_cast<const float*>(p)[i];
  if (KIND == OP_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
  return __bfloat162float(__float2bfloat16_rn(reinterpret_cast<const float*>(p)[i]));
}

template <int KA, int KB>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int M, int N, int K, const void* __restrict__ A, int64_t sam, int64_t sak,
                 const void* __restrict__ B, int64_t sbn, int64_t sbk, Epilogue ep) {
  __shared__ float As[kTK][kTM + 4];
  __shared__ float Bs[kTK][kTN + 4];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * kTM, n0 = blockIdx.x * kTN;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += kTK) {
    // stage the two operand tiles; the thread->element map follows the contiguous dimension
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int r, k;
      if (sak == 1) { r = (tid >> 4) + 16 * i; k = tid & 15; } else { r = tid & 63; k = (tid >> 6) + 4 * i; }
      const int gm = m0 + r, gk = k0 + k;
      As[k][r] = (gm < M && gk < K) ? load_op<KA>(A, (int64_t)gm * sam + (int64_t)gk * sak) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int r, k;
      if (sbk == 1) { r = (tid >> 4) + 16 * i; k = tid & 15; } else { r = tid & 63; k = (tid >> 6) + 4 * i; }
      const int gn = n0 + r, gk = k0 + k;
      Bs[k][r] = (gn < N && gk < K) ? load_op<KB>(B, (int64_t)gn * sbn + (int64_t)gk * sbk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      epilogue_store(ep, epilogue_value(ep, acc[i][j], m, n), m, n);
    }
  }
}

ss_status gemm_simt(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st) {
  if (M <= 0 || N <= 0) return SS_OK;
  dim3 grid((N + kTN - 1) / kTN, (M + kTM - 1) / kTM);
#define SS_GO(KA, KB)                                                                                         \
  gemm_simt_kernel<KA, KB><<<grid, 256, 0, st>>>(M, N, K, A.p, A.s_row, A.s_k, B.p, B.s_row, B.s_k, ep)
  const int key = A.kind * 3 + B.kind;
  SS_TIMED("gemm_simt_kernel", st);
  switch (key) {
    case OP_F32 * 3 + OP_F32: SS_GO(OP_F32, OP_F32); break;
    case OP_BF16 * 3 + OP_BF16: SS_GO(OP_BF16, OP_BF16); break;
    case OP_F32_ROUND_BF16 * 3 + OP_BF16: SS_GO(OP_F32_ROUND_BF16, OP_BF16); break;
    case OP_BF16 * 3 + OP_F32_ROUND_BF16: SS_GO(OP_BF16, OP_F32_ROUND_BF16); break;
    default: return SS_ERR_DTYPE;
  }
#undef SS_GO
  SS_LAUNCH_OK();
  return SS_OK;
}

}  // namespace ss
