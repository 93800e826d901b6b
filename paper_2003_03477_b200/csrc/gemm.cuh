// GEMM interface shared by the SIMT and the tensor-core kernels of the MLP.
//
//   C[m, n] = sum_k A(m, k) * B(n, k)        m < M, n < N, k < K
//
// followed by one epilogue: + bias[n], ReLU, multiply by (mask[m, n] > 0) for n < mask_cols (mask_cols > 0), then
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
  // Tensor-core kernels only.  bits_out: besides out_lo (bf16), one bit per element "the stored value is positive",
  // bit n % 32 of word [m * ld_bits_out + n / 32]: the ReLU-gradient mask of the backward pass at 1/16 of the bytes.
  // mask_bits: such a word array of the producing layer; when given it is used instead of `mask` (same meaning).
  // Both pitches are multiples of 4 words and the arrays 16-byte aligned.
  uint32_t* bits_out = nullptr;
  int64_t ld_bits_out = 0;
  const uint32_t* mask_bits = nullptr;
  int64_t ld_mask_bits = 0;
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

// A flow: several products (each eligible for gemm_tc, at most kTcMaxFlow) in ONE persistent launch whose CTAs draw
// output tiles from a shared counter, in the order the products are listed.  A product may read, as its A operand,
// what an EARLIER product of the same flow writes (out_lo); its tiles then wait for the row blocks they need:
//   dep_mode 1  A(m, k) rows are the producer's output rows (a layer reading the previous layer's activations, an
//               input gradient reading the gradient above it): tile row block y waits for the producer's row block y.
//               dep_k_blocks > 0: only the first dep_k_blocks 64-wide k blocks of A come from the producer (the
//               concat buffer, whose first columns are the bottom MLP's output): the tile contracts the other
//               k blocks first and waits only then.
//   dep_mode 2  A is the producer's output read transposed (a weight gradient contracting over the batch): k block
//               kb waits for the producer's row block holding batch rows 64 kb .. 64 kb + 63.
// signal_cols: only output tiles that start below this column report completion (0 = all): what later products read.
// Waiting never deadlocks: a tile only waits for tiles that were drawn before it, by CTAs that are running.
constexpr int kTcMaxFlow = 12;
struct TcJob {
  int M, N, K;
  Operand A, B;
  Epilogue ep;
  int k_splits = 1;
  int64_t split_stride = 0;
  int dep = -1;            // index of the producing job in the same flow, -1: A is complete before the launch
  int dep_mode = 0;
  int dep_k_blocks = 0;
  int signal_cols = 0;
};
// Control words of a flow in device memory: the tile counter, the exit ticket and per (job, 128-row block) completion
// counts (plus one total per job).  They must be zero when the launch starts; the kernel leaves them zero when it ends without an error.
inline size_t tc_flow_ctrl_ints(int max_rows) { return 2 + (size_t)kTcMaxFlow * (size_t)((max_rows + 127) / 128 + 1); }
// ctrl == nullptr: tiles are assigned round-robin instead (only for flows without dependencies).
// max_ctas <= 0: one CTA per SM at most.
ss_status gemm_tc_flow(const TcJob* jobs, int n, int* ctrl, int max_rows, int max_ctas, cudaStream_t st);
// CTAs a flow with dependencies takes when the caller gives no number (0: the built-in default, negative: no
// change); returns the number now in effect.
int set_flow_ctas(int ctas);
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
