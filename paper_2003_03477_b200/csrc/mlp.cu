// Bottom MLP -> concat -> top MLP -> sigmoid/BCE, its backward pass and the dense Adagrad update.
#include "gemm.cuh"
#include "profile.cuh"
#include "mlp_plan.cuh"

namespace ss {

// dz[b] = (prob[b] - y[b]) / B, stored as float or bf16 (a [B,1] gradient matrix).
__global__ void dz_kernel(const float* __restrict__ prob, const float* __restrict__ labels, int B, void* __restrict__ dz,
                          int as_bf16) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const float v = (prob[b] - labels[b]) / (float)B;
  if (as_bf16) reinterpret_cast<__nv_bfloat16*>(dz)[b] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(dz)[b] = v;
}

// ---------------------------------------------------------------------------------------------
// Reductions over the batch that are no dense contraction: bias gradients, the gradient of the
// single-logit layer and of the 13-input layer.  All have the form
//     out[c * s_cols + j] = sum_b M[b, c] * S[b, j]          (S absent: s_cols = 1, S = 1)
// One launch takes a list of such jobs.  A block owns 32 columns c and a slice of the batch; its 8
// row groups add their rows in ascending order, the groups are added in order, and a second kernel
// adds the slices in order: every sum has a fixed association.
// ---------------------------------------------------------------------------------------------
constexpr int kMaxJobs = 2 * kMaxLayers + 2;
constexpr int kMaxSCols = 16;

struct RedJob {
  const void* M; const void* S;
  int64_t ldm, lds;
  int m_kind, s_kind;      // OperandKind
  int ncols, s_cols;
  int tile0;               // first column tile of this job in grid.x
  int part_off;            // offset of this job's outputs in a partial row
  int64_t out_off;         // offset into the flat gradient vector
};
struct RedJobs {
  RedJob job[kMaxJobs];
  int njobs, ntiles, total;   // total = outputs over all jobs
};

__device__ __forceinline__ float load_kind(const void* p, int kind, int64_t i) {
  if (kind == OP_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
  const float v = reinterpret_cast<const float*>(p)[i];
  return kind == OP_F32 ? v : __bfloat162float(__float2bfloat16_rn(v));
}

constexpr int kRedRows = 256;     // most rows of the batch a block takes (bounds the staged S tile)
constexpr int kRedWide = 256;     // columns per block of a job without a second factor matrix (s_cols = 1)

// Eight consecutive elements M[row, c .. c+7] as floats; elements at or beyond ncols read as zero.  One
// 128-bit load (bf16) or two (float) when the address allows it, element loads otherwise.
__device__ __forceinline__ void load8_kind(const void* p, int kind, int64_t row, int64_t ld, int c, int ncols, bool vec_ok,
                                           float (&v)[8]) {
  if (vec_ok && c + 8 <= ncols) {
    if (kind == OP_BF16) {
      const uint4 q = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p) + row * ld + c);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[2 * j] = __uint_as_float(w[j] << 16);                // a bf16 is the upper half of a float
        v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    } else {
      const float4* q = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + row * ld + c);
      const float4 a = q[0], b = q[1];
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
      if (kind == OP_F32_ROUND_BF16) {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __bfloat162float(__float2bfloat16_rn(v[j]));
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = (c + j < ncols) ? load_kind(p, kind, row * ld + c + j) : 0.f;
  }
}

__global__ void __launch_bounds__(256)
batch_reduce_partial_kernel(const __grid_constant__ RedJobs jobs, int B, int rows_per_split, float* __restrict__ partial) {
  // S rows of this block's batch slice, as float; then the row groups' sums (8 x 256 or 8 x 32 x 17 floats)
  constexpr int kPartFloats = 8 * 32 * (kMaxSCols + 1);
  static_assert(kPartFloats >= kRedRows * kMaxSCols && kPartFloats >= 8 * kRedWide, "one buffer serves all three uses");
  __shared__ __align__(16) float s_tile[kPartFloats];
  __shared__ RedJob s_job;
  if (threadIdx.x == 0) {
    int j = 0;
    while (j + 1 < jobs.njobs && (int)blockIdx.x >= jobs.job[j + 1].tile0) ++j;
    s_job = jobs.job[j];
  }
  __syncthreads();
  const RedJob J = s_job;                                    // the job's fields in registers
  const int cx = threadIdx.x & 31, ry = threadIdx.x >> 5;
  const int sc = J.s_cols;
  const int r0 = blockIdx.y * rows_per_split;
  const int r1 = min(B, r0 + rows_per_split);
  const int nrows = r1 - r0;

  if (sc == 1) {
    // ---- no second factor, or a single column of one (S[b]): a warp reads 256 consecutive columns of a row,
    // eight per lane; warp ry adds rows ry, ry+8, ... in ascending order, then the eight warps are added in order.
    const int c = ((int)blockIdx.x - J.tile0) * kRedWide + 8 * cx;
    const bool vec_ok = J.m_kind == OP_BF16 ? ((J.ldm & 7) == 0 && (reinterpret_cast<uintptr_t>(J.M) & 15u) == 0)
                                            : ((J.ldm & 3) == 0 && (reinterpret_cast<uintptr_t>(J.M) & 15u) == 0);
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
    if (c < J.ncols) {
      for (int rr = ry; rr < nrows; rr += 32) {
        float m[4][8], sv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {                          // four rows in flight per thread
          const int r = rr + 8 * u;
          if (r < nrows) {
            load8_kind(J.M, J.m_kind, r0 + r, J.ldm, c, J.ncols, vec_ok, m[u]);
            sv[u] = J.S ? load_kind(J.S, J.s_kind, (int64_t)(r0 + r) * J.lds) : 1.f;
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) m[u][j] = 0.f;
            sv[u] = 0.f;
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (J.S) {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] = fmaf(m[u][j], sv[u], acc[j]);
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[j] += m[u][j];
          }
        }
      }
    }
    float* part = s_tile;                                      // [8][256]
    float4* pw = reinterpret_cast<float4*>(part + ry * kRedWide + 8 * cx);
    pw[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    pw[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    __syncthreads();
    const int co = ((int)blockIdx.x - J.tile0) * kRedWide + (int)threadIdx.x;
    if (co < J.ncols) {
      float t = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) t += part[r * kRedWide + threadIdx.x];
      partial[(int64_t)blockIdx.y * jobs.total + J.part_off + co] = t;
    }
    return;
  }

  // ---- a second factor with several columns (the layer with few inputs): 32 columns c per block, each thread
  // keeps one sum per column of S
  const int c = ((int)blockIdx.x - J.tile0) * 32 + cx;
  // S rows as float, padded with zeros to kMaxSCols columns so that the inner product needs no column test
  for (int i = threadIdx.x; i < nrows * kMaxSCols; i += 256) {
    const int rr = i / kMaxSCols, q = i % kMaxSCols;
    s_tile[i] = q < sc ? load_kind(J.S, J.s_kind, (int64_t)(r0 + rr) * J.lds + q) : 0.f;
  }
  __syncthreads();
  float acc[kMaxSCols];
#pragma unroll
  for (int q = 0; q < kMaxSCols; ++q) acc[q] = 0.f;
  if (c < J.ncols) {
    // four rows of M in flight per thread; rows are added in ascending order
    for (int rr = ry; rr < nrows; rr += 32) {
      float m[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        m[u] = (rr + 8 * u < nrows) ? load_kind(J.M, J.m_kind, (int64_t)(r0 + rr + 8 * u) * J.ldm + c) : 0.f;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (rr + 8 * u < nrows) {
          const float4* srow = reinterpret_cast<const float4*>(s_tile + (rr + 8 * u) * kMaxSCols);
#pragma unroll
          for (int q4 = 0; q4 < kMaxSCols / 4; ++q4) {
            const float4 sv = srow[q4];                    // one 128-bit broadcast read for four columns
            acc[4 * q4 + 0] = fmaf(m[u], sv.x, acc[4 * q4 + 0]);
            acc[4 * q4 + 1] = fmaf(m[u], sv.y, acc[4 * q4 + 1]);
            acc[4 * q4 + 2] = fmaf(m[u], sv.z, acc[4 * q4 + 2]);
            acc[4 * q4 + 3] = fmaf(m[u], sv.w, acc[4 * q4 + 3]);
          }
        }
      }
    }
  }
  __syncthreads();                                           // the S tile is no longer read
  float (*part)[32][kMaxSCols + 1] = reinterpret_cast<float (*)[32][kMaxSCols + 1]>(s_tile);   // [8][32][17]
#pragma unroll
  for (int q = 0; q < kMaxSCols; ++q) part[ry][cx][q] = acc[q];
  __syncthreads();
  if (ry == 0 && c < J.ncols) {
    float* dst = partial + (int64_t)blockIdx.y * jobs.total + J.part_off + (int64_t)c * sc;
    for (int q = 0; q < sc; ++q) {
      float t = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) t += part[r][cx][q];
      dst[q] = t;
    }
  }
}

// The single-logit layer, the sigmoid and the loss in one launch:
//   logit[b] = sum_k X[b, k] * w[k] + bias;  prob[b] = sigmoid(logit[b]);
//   loss = mean_b( max(z,0) - z*y + log(1+exp(-|z|)) ).
// One warp per sample (eight consecutive k per lane and round, fixed shuffle tree); a block adds the loss terms of
// its eight samples in order and leaves the sum in part[block]; the block that draws the last ticket adds the
// blocks' sums in a fixed order (which block that is does not matter) and clears the ticket for the next call.
__global__ void __launch_bounds__(256)
logit_loss_kernel(const void* __restrict__ X, int x_kind, int64_t ldx, const void* __restrict__ w, int w_kind, int K,
                  const float* __restrict__ bias, const float* __restrict__ labels, int B, float* __restrict__ logit,
                  float* __restrict__ prob, float* __restrict__ loss, float* part, unsigned int* ticket) {
  __shared__ float s_term[8];
  __shared__ float s_red[256];
  __shared__ int s_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + warp;
  float s = 0.f;
  if (b < B) {
    const bool al_x = (reinterpret_cast<uintptr_t>(X) & 15u) == 0, al_w = (reinterpret_cast<uintptr_t>(w) & 15u) == 0;
    const bool vec_x = al_x && (x_kind == OP_BF16 ? (ldx & 7) == 0 : (ldx & 3) == 0);
    for (int k0 = 8 * lane; k0 < K; k0 += 256) {
      float xv[8], wv[8];
      load8_kind(X, x_kind, b, ldx, k0, K, vec_x, xv);
      load8_kind(w, w_kind, 0, 0, k0, K, al_w, wv);
#pragma unroll
      for (int j = 0; j < 8; ++j) s = fmaf(xv[j], wv[j], s);
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) s += __shfl_down_sync(0xffffffffu, s, off);
  if (lane == 0) {
    float t = 0.f;
    if (b < B) {
      const float z = s + bias[0], y = labels[b];
      const float e = expf(-fabsf(z));
      logit[b] = z;
      prob[b] = (z >= 0.f) ? 1.f / (1.f + e) : e / (1.f + e);
      t = fmaxf(z, 0.f) - z * y + log1pf(e);
    }
    s_term[warp] = t;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
#pragma unroll
    for (int r = 0; r < 8; ++r) t += s_term[r];
    part[blockIdx.x] = t;
    __threadfence();
    s_last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  float a = 0.f;
  for (int i = threadIdx.x; i < (int)gridDim.x; i += 256) a += __ldcg(part + i);
  s_red[threadIdx.x] = a;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if (threadIdx.x < off) s_red[threadIdx.x] += s_red[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    loss[0] = s_red[0] / (float)B;
    *ticket = 0u;
  }
}

// The backward of the single-logit layer with the loss gradient folded in:
//   dz[b] = (prob[b] - y[b]) / B   (rounded to bf16 in bf16 mode, and stored: the reductions read it)
//   dX[b, k] = dz[b] * w[k], gated by X[b, k] > 0.
// One thread per eight consecutive k of a row (K is a multiple of 8: hidden widths are).
template <bool BF16>
__global__ void __launch_bounds__(256)
dz_outer_mask_kernel(const float* __restrict__ prob, const float* __restrict__ labels, const void* __restrict__ w,
                     const void* __restrict__ X, int B, int K, void* __restrict__ dz, void* __restrict__ dX) {
  const int kc = K >> 3;
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= (int64_t)B * kc) return;
  const int b = (int)(i / kc), c = (int)(i - (int64_t)b * kc) * 8;
  float d = (prob[b] - labels[b]) / (float)B;
  if (BF16) {
    const __nv_bfloat16 dh = __float2bfloat16_rn(d);
    d = __bfloat162float(dh);
    if (c == 0) reinterpret_cast<__nv_bfloat16*>(dz)[b] = dh;
    const uint4 xq = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(X) + (int64_t)b * K + c);
    const uint4 wq = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(w) + c);
    const uint32_t xw[4] = {xq.x, xq.y, xq.z, xq.w}, ww[4] = {wq.x, wq.y, wq.z, wq.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float x0 = __uint_as_float(xw[j] << 16), x1 = __uint_as_float(xw[j] & 0xFFFF0000u);
      const float w0 = __uint_as_float(ww[j] << 16), w1 = __uint_as_float(ww[j] & 0xFFFF0000u);
      const float v0 = x0 > 0.f ? d * w0 : 0.f, v1 = x1 > 0.f ? d * w1 : 0.f;
      __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
      o[j] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(dX) + (int64_t)b * K + c) = make_uint4(o[0], o[1], o[2], o[3]);
  } else {
    if (c == 0) reinterpret_cast<float*>(dz)[b] = d;
    const float4* xq = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(X) + (int64_t)b * K + c);
    const float4* wq = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(w) + c);
    float4* oq = reinterpret_cast<float4*>(reinterpret_cast<float*>(dX) + (int64_t)b * K + c);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float4 x = xq[h], ww = wq[h];
      oq[h] = make_float4(x.x > 0.f ? d * ww.x : 0.f, x.y > 0.f ? d * ww.y : 0.f, x.z > 0.f ? d * ww.z : 0.f,
                          x.w > 0.f ? d * ww.w : 0.f);
    }
  }
}

// Where the gradient of each parameter tensor is found when the update kernel runs.
//   GRAD_FLAT    in the flat gradient vector itself (a GEMM wrote it there)
//   GRAD_SLICES  nsplit K slices of a weight-gradient GEMM: src[off + z*stride + i]
//   GRAD_BATCH   nsplit batch slices of the batched reduction (bias, skinny weights): src[off + z*stride + i]
// Elements that belong to no tensor (pads of the layout) have gradient zero.
enum { GRAD_FLAT = 0, GRAD_SLICES = 1, GRAD_BATCH = 2 };
constexpr int kMaxGradRanges = 2 * kMaxLayers;
struct GradTable {
  int n;
  int64_t begin[kMaxGradRanges], end[kMaxGradRanges], off[kMaxGradRanges], stride[kMaxGradRanges];
  int kind[kMaxGradRanges], nsplit[kMaxGradRanges];
};

// Element-wise Adagrad over the flat parameter vector; refreshes the bf16 mirror.  The slices of a
// gradient are added in slice order.  A zero gradient (pads, dead units) leaves the element
// untouched.  g_out (nullable, may alias g) receives the assembled gradient.
// A thread owns two float4 positions, 256 apart; the parameter and accumulator loads of both go out
// before the gradient is looked up, so one round of memory latency covers all of a thread's loads.
constexpr int kAdaPerThread = 2;

__device__ __forceinline__ float4 assemble_grad(const GradTable& tab, int64_t i, const float* g, const float* __restrict__ gpart,
                                                const float* __restrict__ bpart) {
  const int64_t e = i * 4;
  float4 gv = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int t = 0; t < tab.n; ++t) {
    if (e >= tab.begin[t] && e < tab.end[t]) {               // tensors start on multiples of 32: no float4 straddles a start
      const int64_t rel = e - tab.begin[t];
      if (tab.kind[t] == GRAD_FLAT) {
        gv = reinterpret_cast<const float4*>(g)[i];
      } else if (tab.kind[t] == GRAD_SLICES) {               // sizes are multiples of 8: aligned float4 loads
        const float4* p = reinterpret_cast<const float4*>(gpart + tab.off[t] + rel);
        const int ns = tab.nsplit[t];
        const int64_t st4 = tab.stride[t] >> 2;
        gv = p[0];
        if (ns == 2) {
          const float4 q = p[st4];
          gv.x += q.x; gv.y += q.y; gv.z += q.z; gv.w += q.w;
        } else {
          for (int z = 1; z < ns; ++z) {
            const float4 q = p[(int64_t)z * st4];
            gv.x += q.x; gv.y += q.y; gv.z += q.z; gv.w += q.w;
          }
        }
      } else {                                               // any size: scalar loads, elements past the end stay zero
        const int64_t left = tab.end[t] - e;
        const float* p = bpart + tab.off[t] + rel;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        for (int z = 0; z < tab.nsplit[t]; ++z) {
          const float* q = p + (int64_t)z * tab.stride[t];
#pragma unroll
          for (int k = 0; k < 4; ++k) if (k < left) v[k] += q[k];
        }
        gv = make_float4(v[0], v[1], v[2], v[3]);
      }
      break;
    }
  }
  return gv;
}

__global__ void __launch_bounds__(256)
adagrad_kernel(float* __restrict__ w, float* __restrict__ acc, const float* g, const float* __restrict__ gpart,
               const float* __restrict__ bpart, const __grid_constant__ GradTable tab,
               __nv_bfloat16* __restrict__ mirror, int64_t n4, float lr, float eps, float* g_out, int apply) {
  const int64_t i0 = (int64_t)blockIdx.x * (256 * kAdaPerThread) + threadIdx.x;
  float4 wv[kAdaPerThread], av[kAdaPerThread], gv[kAdaPerThread];
#pragma unroll
  for (int u = 0; u < kAdaPerThread; ++u) {
    const int64_t i = i0 + 256 * u;
    if (apply && i < n4) {
      wv[u] = reinterpret_cast<float4*>(w)[i];
      av[u] = reinterpret_cast<float4*>(acc)[i];
    }
  }
#pragma unroll
  for (int u = 0; u < kAdaPerThread; ++u) {
    const int64_t i = i0 + 256 * u;
    if (i < n4) gv[u] = assemble_grad(tab, i, g, gpart, bpart);
  }
#pragma unroll
  for (int u = 0; u < kAdaPerThread; ++u) {
    const int64_t i = i0 + 256 * u;
    if (i >= n4) continue;
    if (g_out) reinterpret_cast<float4*>(g_out)[i] = gv[u];
    if (!apply) continue;
#define SS_UPD(F)                                        \
    if (gv[u].F != 0.f) {                                \
      av[u].F = fmaf(gv[u].F, gv[u].F, av[u].F);         \
      wv[u].F -= lr * gv[u].F / (sqrtf(av[u].F) + eps);  \
    }
    SS_UPD(x) SS_UPD(y) SS_UPD(z) SS_UPD(w)
#undef SS_UPD
    reinterpret_cast<float4*>(w)[i] = wv[u];
    reinterpret_cast<float4*>(acc)[i] = av[u];
    if (mirror) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(wv[u].x, wv[u].y), hi = __floats2bfloat162_rn(wv[u].z, wv[u].w);
      uint2 r;
      r.x = *reinterpret_cast<uint32_t*>(&lo);
      r.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(mirror)[i] = r;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The layer that reads the dense features (at most 16 inputs) is no dense contraction either:
//   Y[b, o] = ReLU( sum_k bf16(x[b, k]) * W[o, k] + bias[o] ),   stored as bf16.
// The weights sit in shared memory as [k][o]; a thread computes eight consecutive outputs of one
// sample with fp32 FMAs in ascending k.
// ---------------------------------------------------------------------------------------------
constexpr int kFewInputs = 16;
constexpr int kFirstRowsMax = 32;   // most samples per block (the launch picks 8, 16 or 32 so that the grid is about two blocks per SM)

__global__ void __launch_bounds__(256)
few_inputs_layer_kernel(const float* __restrict__ x, int K, const __nv_bfloat16* __restrict__ W, const float* __restrict__ bias,
                        int relu, int B, int N, __nv_bfloat16* __restrict__ Y, int64_t ldy, int rows_per_block,
                        uint8_t* __restrict__ bits /*nullable: one bit per output "positive", rows of ld_bits bytes*/,
                        int64_t ld_bits) {
  extern __shared__ __align__(16) __nv_bfloat16 s_w[];       // [K][N]
  __shared__ float s_x[kFirstRowsMax][kFewInputs];           // the block's samples, rounded to bf16, zero beyond K
  const int b0 = blockIdx.x * rows_per_block;
  const int rows = min(rows_per_block, B - b0);
  for (int o = threadIdx.x; o < N; o += 256) {               // W is [o][k]
#pragma unroll 4
    for (int k = 0; k < K; ++k) s_w[k * N + o] = W[(int64_t)o * K + k];
  }
  for (int i = threadIdx.x; i < rows_per_block * kFewInputs; i += 256) {
    const int r = i / kFewInputs, k = i % kFewInputs;
    s_x[r][k] = (r < rows && k < K) ? __bfloat162float(__float2bfloat16_rn(x[(int64_t)(b0 + r) * K + k])) : 0.f;
  }
  __syncthreads();
  const int nchunk = N >> 3;
  for (int item = threadIdx.x; item < rows * nchunk; item += 256) {
    const int r = item / nchunk, o = (item - r * nchunk) * 8;
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
    for (int k = 0; k < kFewInputs; ++k) {
      if (k < K) {
        const float xv = s_x[r][k];
        const uint4 q = *reinterpret_cast<const uint4*>(s_w + k * N + o);
        const uint32_t ww[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] = fmaf(xv, __uint_as_float(ww[j] << 16), acc[2 * j]);
          acc[2 * j + 1] = fmaf(xv, __uint_as_float(ww[j] & 0xFFFF0000u), acc[2 * j + 1]);
        }
      }
    }
    const float4 b0v = reinterpret_cast<const float4*>(bias + o)[0], b1v = reinterpret_cast<const float4*>(bias + o)[1];
    const float bv[8] = {b0v.x, b0v.y, b0v.z, b0v.w, b1v.x, b1v.y, b1v.z, b1v.w};
    uint32_t out[4];
    uint32_t pos = 0;                                          // bit j: output o + j is positive as stored
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v0 = acc[2 * j] + bv[2 * j], v1 = acc[2 * j + 1] + bv[2 * j + 1];
      if (relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
      __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
      out[j] = *reinterpret_cast<uint32_t*>(&h);
      const uint32_t lo = out[j] & 0xFFFFu, hi = out[j] >> 16;
      pos |= (uint32_t)((lo & 0x8000u) == 0 && (lo & 0x7FFFu) != 0) << (2 * j);
      pos |= (uint32_t)((hi & 0x8000u) == 0 && (hi & 0x7FFFu) != 0) << (2 * j + 1);
    }
    *reinterpret_cast<uint4*>(Y + (int64_t)(b0 + r) * ldy + o) = make_uint4(out[0], out[1], out[2], out[3]);
    if (bits) bits[(int64_t)(b0 + r) * ld_bits + (o >> 3)] = (uint8_t)pos;   // byte o / 8 of the row's little-endian words
  }
}

// Collects the tensor-core products of a pass into flows (one persistent launch each, see gemm.cuh) and remembers
// which job of the open flow writes which tensor, so that a later product reading that tensor waits for its row
// blocks inside the launch instead of for a kernel boundary.
static_assert(kTcMaxFlow == 12, "the control-word region of the workspace is sized for 12 products per flow");
struct FlowBuilder {
  TcJob jobs[kTcMaxFlow];
  int n = 0;
  int writer[kMaxLayers];      // writer[l]: job of the open flow whose output is the tensor attached to layer l, or -1
  int* ctrl;
  int max_rows;
  cudaStream_t st;
  FlowBuilder(int* ctrl_, int max_rows_, cudaStream_t st_) : ctrl(ctrl_), max_rows(max_rows_), st(st_) {
    for (int l = 0; l < kMaxLayers; ++l) writer[l] = -1;
  }
  // launches what has been collected; everything it writes is complete for whatever follows on the stream
  ss_status flush() {
    if (n == 0) return SS_OK;
    const ss_status r = gemm_tc_flow(jobs, n, (n == 1 && jobs[0].dep < 0) ? nullptr : ctrl, max_rows, 0, st);
    n = 0;
    for (int l = 0; l < kMaxLayers; ++l) writer[l] = -1;
    return r;
  }
  // adds a job; `reads` is the layer whose tensor is its A operand (or -1); returns the job's index or a negative status
  int add(TcJob j, int reads, int dep_mode, int dep_k_blocks) {
    if (n == kTcMaxFlow) {
      const ss_status r = flush();
      if (r != SS_OK) return r;
    }
    if (reads >= 0 && writer[reads] >= 0) {
      j.dep = writer[reads]; j.dep_mode = dep_mode; j.dep_k_blocks = dep_k_blocks;
    }
    jobs[n] = j;
    return n++;
  }
};

// How layer l (not the last) of the forward pass is computed, and with which operands: the forward pass runs it, the
// backward pass asks the same question to know whether the layer left the sign bits of its output (bits[l]).
enum { FWD_FEW_INPUTS = 0, FWD_TENSOR_CORE = 1, FWD_SIMT = 2 };
struct FwdLayer { Operand A, Bm; Epilogue ep; int how; };
static FwdLayer describe_fwd_layer(const MlpPlan& p, int l, int B, const float* w, const void* w_bf16, const float* dense,
                                   const float* concat_f32, const void* concat_bf16, char* ws) {
  const LayerInfo& L = p.layer[l];
  const int act_kind = p.bf16 ? OP_BF16 : OP_F32;
  FwdLayer f;
  if (l == 0) f.A = Operand{dense, p.bf16 ? OP_F32_ROUND_BF16 : OP_F32, p.n_dense, 1};
  else if (l == p.nb) f.A = Operand{p.bf16 ? (const void*)concat_bf16 : (const void*)concat_f32, act_kind, p.W, 1};
  else f.A = Operand{ws + p.act[l - 1], act_kind, L.in, 1};
  f.Bm = p.bf16 ? Operand{reinterpret_cast<const __nv_bfloat16*>(w_bf16) + L.w_off, OP_BF16, L.in, 1}
                : Operand{w + L.w_off, OP_F32, L.in, 1};
  f.ep.bias = w + L.b_off;
  f.ep.relu = L.relu;
  f.ep.lo_cols = L.out;
  if (l == p.nb - 1) {
    f.ep.out_lo = p.bf16 ? const_cast<void*>(concat_bf16) : (void*)concat_f32; f.ep.lo_bf16 = p.bf16; f.ep.ld_lo = p.W;
  } else {
    f.ep.out_lo = ws + p.act[l]; f.ep.lo_bf16 = p.bf16; f.ep.ld_lo = L.out;
  }
  const size_t few_smem = (size_t)L.in * L.out * 2;
  if (p.bf16 && l == 0 && L.in <= kFewInputs && few_smem <= 48 * 1024 && (f.ep.ld_lo & 7) == 0 && aligned16(f.ep.out_lo))
    f.how = FWD_FEW_INPUTS;
  else if (gemm_tc_eligible(B, L.out, L.in, f.A, f.Bm, f.ep))
    f.how = FWD_TENSOR_CORE;
  else
    f.how = FWD_SIMT;
  return f;
}

static ss_status check_common(const MlpPlan& p, int B, const void* concat_f32, const void* concat_bf16,
                              const void* w_bf16, void* ws, size_t ws_bytes) {
  if (B < 1) return SS_ERR_SHAPE;
  if (!ws) return SS_ERR_NULL;
  if (p.bf16 && (!concat_bf16 || !w_bf16)) return SS_ERR_DTYPE;
  if (!p.bf16 && !concat_f32) return SS_ERR_NULL;
  if (!aligned16(ws) || (concat_f32 && !aligned16(concat_f32)) || (concat_bf16 && !aligned16(concat_bf16)) ||
      (w_bf16 && !aligned16(w_bf16)))
    return SS_ERR_ALIGN;
  if (ws_bytes < p.total) return SS_ERR_WORKSPACE;
  return check_arch();
}

}  // namespace ss

extern "C" {

int64_t ss_mlp_param_count(const ss_mlp_desc* desc) {
  ss::MlpPlan p;
  if (ss::make_mlp_plan(desc, 0, &p) != SS_OK) return -1;
  return p.P;
}

ss_status ss_mlp_param_offsets(const ss_mlp_desc* desc, int64_t* w_off, int64_t* b_off) {
  if (!w_off || !b_off) return SS_ERR_NULL;
  ss::MlpPlan p;
  ss_status st = ss::make_mlp_plan(desc, 0, &p);
  if (st != SS_OK) return st;
  for (int l = 0; l < p.nl; ++l) { w_off[l] = p.layer[l].w_off; b_off[l] = p.layer[l].b_off; }
  return SS_OK;
}

size_t ss_mlp_workspace_bytes(const ss_mlp_desc* desc, int B) {
  ss::MlpPlan p;
  if (ss::make_mlp_plan(desc, B, &p) != SS_OK) return 0;
  return p.total;
}

ss_status ss_mlp_fwd(const ss_mlp_desc* desc, const float* w, const void* w_bf16, const float* dense,
                     float* concat_f32, void* concat_bf16, int B, const float* labels, float* logit, float* prob,
                     float* loss, void* workspace, size_t workspace_bytes, ss_stream stream) {
  using namespace ss;
  if (!w || !dense || !labels || !logit || !prob || !loss) return SS_ERR_NULL;
  MlpPlan p;
  ss_status st = make_mlp_plan(desc, B, &p);
  if (st != SS_OK) return st;
  st = check_common(p, B, concat_f32, concat_bf16, w_bf16, workspace, workspace_bytes);
  if (st != SS_OK) return st;
  if (!aligned16(w)) return SS_ERR_ALIGN;
  cudaStream_t cs = as_stream(stream);
  char* ws = reinterpret_cast<char*>(workspace);
  const int act_kind = p.bf16 ? OP_BF16 : OP_F32;
  // the loss kernel's ticket and the control words of the tensor-core flows start at zero (the workspace arrives
  // uninitialised); both clear themselves after use
  SS_CUDA(cudaMemsetAsync(ws + p.loss_part, 0, p.ctrl + p.ctrl_bytes - p.loss_part, cs));
  FlowBuilder flow(reinterpret_cast<int*>(ws + p.ctrl), p.ctrl_rows, cs);

  for (int l = 0; l < p.nl; ++l) {
    const LayerInfo& L = p.layer[l];
    const FwdLayer f = describe_fwd_layer(p, l, B, w, w_bf16, dense, concat_f32, concat_bf16, ws);
    const Operand& A = f.A;
    const Operand& Bm = f.Bm;
    const Epilogue& ep = f.ep;
    if (l == p.nl - 1) {   // one output unit: a dot product per sample
      st = flow.flush();
      if (st != SS_OK) return st;
      unsigned int* ticket = reinterpret_cast<unsigned int*>(ws + p.loss_part);
      { SS_TIMED("logit_loss_kernel", cs);
      logit_loss_kernel<<<(B + 7) / 8, 256, 0, cs>>>(A.p, A.kind, A.s_row, Bm.p, Bm.kind, L.in, w + L.b_off, labels, B, logit,
                                                     prob, loss, reinterpret_cast<float*>(ticket + 4), ticket);
      }
      SS_LAUNCH_OK();
      break;
    }
    if (f.how == FWD_FEW_INPUTS) {
      int rows = 8;                                            // every block stages the whole weight matrix
      while (rows < kFirstRowsMax && (B + rows - 1) / rows > 2 * num_sms()) rows *= 2;
      SS_TIMED("few_inputs_layer_kernel", cs);
      few_inputs_layer_kernel<<<(B + rows - 1) / rows, 256, (size_t)L.in * L.out * 2, cs>>>(
          dense, L.in, reinterpret_cast<const __nv_bfloat16*>(w_bf16) + L.w_off, ep.bias, ep.relu, B, L.out,
          reinterpret_cast<__nv_bfloat16*>(ep.out_lo), ep.ld_lo, rows, reinterpret_cast<uint8_t*>(ws + p.bits[l]),
          (int64_t)p.ld_bits[l] * 4);
      SS_LAUNCH_OK();
      continue;
    }
    if (f.how == FWD_TENSOR_CORE) {
      // The whole chain of tensor-core layers is ONE launch: layer l's tiles wait for the row blocks of layer l - 1
      // they read.  The first top layer reads the concat buffer, of which only the first D0 columns come from the
      // bottom MLP: it contracts the pooled embeddings first and waits for the bottom output only then.
      TcJob j;
      j.M = B; j.N = L.out; j.K = L.in; j.A = A; j.B = Bm; j.ep = ep;
      j.ep.bits_out = reinterpret_cast<uint32_t*>(ws + p.bits[l]);   // the backward pass masks with these
      j.ep.ld_bits_out = p.ld_bits[l];
      const int idx = flow.add(j, l - 1, 1, l == p.nb ? (p.D0 + 63) / 64 : 0);
      if (idx < 0) return (ss_status)idx;
      flow.writer[l] = idx;
      continue;
    }
    st = flow.flush();
    if (st != SS_OK) return st;
    st = gemm_simt(B, L.out, L.in, A, Bm, ep, cs);
    if (st != SS_OK) return st;
  }
  return SS_OK;
}

ss_status ss_mlp_bwd(const ss_mlp_desc* desc, float* w, void* w_bf16, float* adagrad_acc, float* grads,
                     const float* dense, const float* concat_f32, const void* concat_bf16, const float* labels,
                     const float* prob, int B, float lr, float eps, int apply_update, float* grad_pooled,
                     int64_t ld_grad, void* workspace, size_t workspace_bytes, ss_stream stream) {
  using namespace ss;
  if (!w || !dense || !labels || !prob || !grad_pooled) return SS_ERR_NULL;
  if (apply_update && !adagrad_acc) return SS_ERR_NULL;
  MlpPlan p;
  ss_status st = make_mlp_plan(desc, B, &p);
  if (st != SS_OK) return st;
  st = check_common(p, B, concat_f32, concat_bf16, w_bf16, workspace, workspace_bytes);
  if (st != SS_OK) return st;
  if (!aligned16(w) || (adagrad_acc && !aligned16(adagrad_acc)) || (grads && !aligned16(grads)) ||
      !aligned16(grad_pooled) || (ld_grad & 3))
    return SS_ERR_ALIGN;
  if (ld_grad < p.W - p.D0) return SS_ERR_SHAPE;
  if (!(lr >= 0.f) || !(eps >= 0.f)) return SS_ERR_RANGE;
  cudaStream_t cs = as_stream(stream);
  char* ws = reinterpret_cast<char*>(workspace);
  const int act_kind = p.bf16 ? OP_BF16 : OP_F32;
  float* g = grads ? grads : reinterpret_cast<float*>(ws + p.grads);

  const int last = p.nl - 1;
  const int dz_kind = p.bf16 ? OP_BF16 : OP_F32;
  if (last == p.nb) {   // a single top layer: its input gradient is a GEMM's; otherwise dz comes out of the fused kernel below
    SS_TIMED("dz_kernel", cs);
    dz_kernel<<<(B + 255) / 256, 256, 0, cs>>>(prob, labels, B, ws + p.dact[last], p.bf16);
  }
  SS_LAUNCH_OK();

  float* gpart = reinterpret_cast<float*>(ws + p.gpart);
  GradTable tab;
  tab.n = 0;
  auto add_range = [&](int64_t begin, int64_t count, int kind, int64_t off, int64_t stride, int nsplit) {
    const int t = tab.n++;
    tab.begin[t] = begin; tab.end[t] = begin + count; tab.kind[t] = kind; tab.off[t] = off; tab.stride[t] = stride;
    tab.nsplit[t] = nsplit;
  };
  RedJobs jobs;
  jobs.njobs = 0; jobs.ntiles = 0; jobs.total = 0;
  auto add_job = [&](const void* M, int m_kind, int64_t ldm, int ncols, const void* S, int s_kind, int64_t lds,
                     int s_cols, int64_t out_off) {
    RedJob& J = jobs.job[jobs.njobs++];
    J.M = M; J.m_kind = m_kind; J.ldm = ldm; J.ncols = ncols;
    J.S = S; J.s_kind = s_kind; J.lds = lds; J.s_cols = s_cols;
    J.tile0 = jobs.ntiles; J.part_off = jobs.total; J.out_off = out_off;
    jobs.ntiles += s_cols == 1 ? (ncols + kRedWide - 1) / kRedWide : (ncols + 31) / 32;
    jobs.total += ncols * s_cols;
  };

  // All tensor-core products of the pass -- per layer the input gradient dX = dY W (which produces the next dY) and
  // the weight gradient dW = dY^T X -- form ONE flow, input gradient first: a product that reads a dY written inside
  // the flow waits for the row blocks it needs (dX by tile row, dW by k block, since it contracts over the batch).
  FlowBuilder flow(reinterpret_cast<int*>(ws + p.ctrl), p.ctrl_rows, cs);   // writer[l]: the job that writes dact[l]
  for (int l = last; l >= 0; --l) {
    const LayerInfo& L = p.layer[l];
    const void* G = ws + p.dact[l];
    // input of layer l
    Operand X;
    if (l == 0) X = Operand{dense, p.bf16 ? OP_F32_ROUND_BF16 : OP_F32, 1, p.n_dense};
    else if (l == p.nb) X = Operand{p.bf16 ? concat_bf16 : (const void*)concat_f32, act_kind, 1, p.W};
    else X = Operand{ws + p.act[l - 1], act_kind, 1, L.in};
    // dX[b, i] = sum_o G[b, o] * W[o, i], gated by the ReLU of the producing layer
    if (l == 0) {
    } else if (l == last && l != p.nb) {
      const void* wl = p.bf16 ? (const void*)(reinterpret_cast<const __nv_bfloat16*>(w_bf16) + L.w_off) : (const void*)(w + L.w_off);
      const int64_t cnt = (int64_t)B * (L.in >> 3);            // L.in is a hidden width: a multiple of 8
      { SS_TIMED("dz_outer_mask_kernel", cs);
      if (p.bf16)
        dz_outer_mask_kernel<true><<<(unsigned)((cnt + 255) / 256), 256, 0, cs>>>(prob, labels, wl, ws + p.act[l - 1], B, L.in,
                                                                                  ws + p.dact[last], ws + p.dact[l - 1]);
      else
        dz_outer_mask_kernel<false><<<(unsigned)((cnt + 255) / 256), 256, 0, cs>>>(prob, labels, wl, ws + p.act[l - 1], B, L.in,
                                                                                   ws + p.dact[last], ws + p.dact[l - 1]);
      }
      SS_LAUNCH_OK();
    } else {
      Operand A{G, act_kind, L.out, 1};
      Operand Wt = p.bf16 ? Operand{reinterpret_cast<const __nv_bfloat16*>(w_bf16) + L.w_off, OP_BF16, 1, L.in}
                          : Operand{w + L.w_off, OP_F32, 1, L.in};
      Epilogue ep;
      ep.mask_bf16 = p.bf16;
      ep.out_lo = ws + p.dact[l - 1]; ep.lo_bf16 = p.bf16;
      if (l == p.nb) {
        ep.mask = p.bf16 ? concat_bf16 : (const void*)concat_f32; ep.ld_mask = p.W; ep.mask_cols = p.D0;
        ep.ld_lo = p.D0; ep.lo_cols = p.D0;
        ep.out_hi = grad_pooled; ep.ld_hi = ld_grad;
      } else {
        ep.mask = ws + p.act[l - 1]; ep.ld_mask = L.in; ep.mask_cols = L.in;
        ep.ld_lo = L.in; ep.lo_cols = L.in;
      }
      // the sign bits of the producing layer's output, where its forward kernel left them
      if (p.bf16 && describe_fwd_layer(p, l - 1, B, w, w_bf16, dense, concat_f32, concat_bf16, ws).how != FWD_SIMT) {
        ep.mask_bits = reinterpret_cast<const uint32_t*>(ws + p.bits[l - 1]);
        ep.ld_mask_bits = p.ld_bits[l - 1];
      }
      if (gemm_tc_eligible(B, L.in, L.out, A, Wt, ep)) {
        TcJob j;
        j.M = B; j.N = L.in; j.K = L.out; j.A = A; j.B = Wt; j.ep = ep;
        if (l == p.nb) j.signal_cols = p.D0;                   // later products read the bottom MLP's part only
        const int idx = flow.add(j, l, 1, 0);
        if (idx < 0) return (ss_status)idx;
        // the weight gradient below reads dact[l] as well: the entry of layer l stays as it is
        const int keep = flow.writer[l];
        flow.writer[l - 1] = idx;
        flow.writer[l] = keep;
      } else {
        st = flow.flush();
        if (st != SS_OK) return st;
        st = gemm_simt(B, L.in, L.out, A, Wt, ep, cs);
        if (st != SS_OK) return st;
      }
    }
    // db[o] = sum_b G[b, o]
    add_job(G, act_kind, L.out, L.out, nullptr, 0, 0, 1, L.b_off);
    // dW[o, i] = sum_b G[b, o] * X[b, i]
    if (l == last) {
      add_job(X.p, X.kind, X.s_k, L.in, G, dz_kind, 1, 1, L.w_off);          // out = 1: dW[i] = sum_b X[b,i] dz[b]
    } else if (l == 0 && L.in <= kMaxSCols) {
      add_job(G, act_kind, L.out, L.out, X.p, X.kind, X.s_k, L.in, L.w_off);  // few inputs: dW[o, :] per column o
    } else {
      Operand A{G, act_kind, 1, L.out};
      Epilogue ep;
      ep.out_lo = g + L.w_off; ep.lo_bf16 = 0; ep.ld_lo = L.in; ep.lo_cols = L.in;
      if (gemm_tc_eligible(L.out, L.in, B, A, X, ep)) {
        // K = batch may be cut into slices; the update kernel adds them in slice order.
        const int64_t size = (int64_t)L.in * L.out;
        const int ks = p.k_splits[l];
        if (ks > 1) {
          ep.out_lo = gpart + p.gpart_off[l];
          add_range(L.w_off, size, GRAD_SLICES, p.gpart_off[l], size, ks);
        } else {
          add_range(L.w_off, size, GRAD_FLAT, 0, 0, 1);
        }
        TcJob j;
        j.M = L.out; j.N = L.in; j.K = B; j.A = A; j.B = X; j.ep = ep; j.k_splits = ks; j.split_stride = size;
        const int idx = flow.add(j, l, 2, 0);
        if (idx < 0) return (ss_status)idx;
      } else {
        st = flow.flush();
        if (st != SS_OK) return st;
        st = gemm_simt(L.out, L.in, B, A, X, ep, cs);
        if (st != SS_OK) return st;
        add_range(L.w_off, (int64_t)L.in * L.out, GRAD_FLAT, 0, 0, 1);
      }
    }
  }
  st = flow.flush();
  if (st != SS_OK) return st;
  {
    // all batch reductions of the pass in one launch; the update kernel adds the batch slices
    int rows = ((B + p.red_splits - 1) / p.red_splits + 7) & ~7;   // <= kRedRows by the choice of red_splits
    const int nsplit = (B + rows - 1) / rows;
    float* partial = reinterpret_cast<float*>(ws + p.red_partial);
    { SS_TIMED("batch_reduce_partial_kernel", cs);
    batch_reduce_partial_kernel<<<dim3(jobs.ntiles, nsplit), 256, 0, cs>>>(jobs, B, rows, partial);
    }
    SS_LAUNCH_OK();
    for (int j = 0; j < jobs.njobs; ++j)
      add_range(jobs.job[j].out_off, (int64_t)jobs.job[j].ncols * jobs.job[j].s_cols, GRAD_BATCH, jobs.job[j].part_off,
                jobs.total, nsplit);
    const int64_t n4 = p.P / 4;
    SS_TIMED("adagrad_kernel", cs);
    adagrad_kernel<<<(unsigned)((n4 + 256 * kAdaPerThread - 1) / (256 * kAdaPerThread)), 256, 0, cs>>>(w, adagrad_acc, g, gpart, partial, tab,
                                                                 reinterpret_cast<__nv_bfloat16*>(w_bf16), n4, lr, eps,
                                                                 (grads || !apply_update) ? g : nullptr, apply_update);
    SS_LAUNCH_OK();
  }
  return SS_OK;
}

// ---- normalised entropy (Section 4, "Evaluation Metrics") --------------------------------------
}  // extern "C"

namespace ss {
// acc[0] += sum_b cross-entropy(z_b, y_b), acc[1] += sum_b y_b, acc[2] += B; one block, fixed tree, double.
__global__ void __launch_bounds__(1024)
ne_accumulate_kernel(const float* __restrict__ logit, const float* __restrict__ labels, int B, double* __restrict__ acc) {
  __shared__ double red[2][1024];
  double ce = 0.0, pos = 0.0;
  for (int b = threadIdx.x; b < B; b += 1024) {
    const double z = logit[b], y = labels[b];
    ce += fmax(z, 0.0) - z * y + log1p(exp(-fabs(z)));
    pos += y;
  }
  red[0][threadIdx.x] = ce;
  red[1][threadIdx.x] = pos;
  __syncthreads();
  for (int off = 512; off >= 1; off >>= 1) {
    if (threadIdx.x < off) {
      red[0][threadIdx.x] += red[0][threadIdx.x + off];
      red[1][threadIdx.x] += red[1][threadIdx.x + off];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) { acc[0] += red[0][0]; acc[1] += red[1][0]; acc[2] += (double)B; }
}

// NE = (mean cross-entropy) / (entropy of the empirical click rate p = acc[1]/acc[2])
__global__ void ne_value_kernel(const double* __restrict__ acc, double* __restrict__ out) {
  const double n = acc[2], p = acc[1] / n;
  out[0] = (acc[0] / n) / -(p * log(p) + (1.0 - p) * log(1.0 - p));
}
}  // namespace ss

extern "C" {

ss_status ss_ne_accumulate(const float* logit, const float* labels, int B, double* acc, ss_stream stream) {
  if (!logit || !labels || !acc) return SS_ERR_NULL;
  if (B < 1) return SS_ERR_SHAPE;
  if (reinterpret_cast<uintptr_t>(acc) & 7u) return SS_ERR_ALIGN;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  SS_TIMED("ne_accumulate_kernel", ss::as_stream(stream));
  ss::ne_accumulate_kernel<<<1, 1024, 0, ss::as_stream(stream)>>>(logit, labels, B, acc);
  SS_LAUNCH_OK();
  return SS_OK;
}

ss_status ss_ne_value(const double* acc, double* out, ss_stream stream) {
  if (!acc || !out) return SS_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(acc) | reinterpret_cast<uintptr_t>(out)) & 7u) return SS_ERR_ALIGN;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  ss::ne_value_kernel<<<1, 1, 0, ss::as_stream(stream)>>>(acc, out);
  SS_LAUNCH_OK();
  return SS_OK;
}

}  // extern "C"
