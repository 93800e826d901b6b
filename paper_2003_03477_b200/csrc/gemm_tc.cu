// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   C[m, n] = sum_k A(m, k) * B(n, k)
//
// One CTA computes a 128 x 128 tile (128 x 256 for large products, 128 x 64 for products with too few
// tiles to occupy the SMs).  One launch may hold several independent products (a group): a CTA finds its
// product from its block index.  Warp 0 (one lane) streams 128 x 64 / 64 x 128 operand tiles
// into a ring of shared-memory stages (3, 4 or 6 deep) with TMA (128-byte swizzle), the first round before the
// warps meet; warp 1 (one lane) issues tcgen05.mma (M = 128, N = 64, 128 or 256, K = 16, accumulators in tensor
// memory) and releases stages with tcgen05.commit; warps 2-5 wait for the accumulator, read it with tcgen05.ld
// (one row per thread) and apply the epilogue (bias, ReLU, ReLU-gradient mask, bf16 / fp32 stores), through a
// transposition in shared memory for the short CTAs of a training step.
//
// Either operand may be K-major (k contiguous in memory: the forward pass reads activations [B, in]
// and weights [out, in] this way) or MN-major (m or n contiguous: the backward pass reads the same
// buffers transposed, dW = dY^T X and dX = dY W), so no transposed copy of any matrix is ever made.
// K-major tiles are one TMA box of 128 rows x 64 k; MN-major tiles are two boxes of 64 k x 64 m, the
// canonical 128-byte-swizzle layouts of the shared-memory matrix descriptor in both cases.
//
// Every mbarrier wait is bounded: when it runs out the kernel raises a device error flag, stops
// waiting, drains, frees its tensor memory and returns; the host reads the flag (ss_device_error).
#include <cuda.h>
#include <cudaTypedefs.h>
#include "gemm.cuh"
#include "profile.cuh"

namespace ss {

constexpr int kBM = 128, kBK = 64;   // tile rows and k depth; the tile width kBN (64, 128 or 256) is a template parameter
// Ring depth: 3 stages (97 KiB, two CTAs per SM) for the small GEMMs of a training step, where several
// replicas' kernels share the SMs and a second resident CTA hides more latency than a deeper ring does;
// 6 stages (193 KiB, one CTA per SM) for large products that fill the machine on their own.
constexpr int kStagesSmall = 3, kStagesLarge = 6;
// 128 x 256 tiles (4 stages of 48 KiB) for products large enough to fill the machine with them: a quarter less
// shared-memory traffic per flop than 128 x 128, which is what bounds the 128-wide tile.
constexpr int kStagesWide = 4;
constexpr int kTileBytes = kBM * kBK * 2;                 // 16 KiB: the A tile, and every 128 columns of the B tile
__host__ __device__ constexpr int stage_bytes(int bn) { return kTileBytes + bn * kBK * 2; }
constexpr int kTcThreads = 192;
constexpr int kStgLd = 36;                                // floats per row of an epilogue warp's 32 x 32 staging block
constexpr size_t tc_smem_bytes(int stages, int bn) { return (size_t)stages * stage_bytes(bn) + 1024 /*alignment slack*/ + 256 /*barriers*/; }
constexpr long long kWaitCycles = 400ll * 1000 * 1000;    // ~0.2 s: far beyond any legitimate wait
constexpr long long kWaitCyclesAborted = 2ll * 1000 * 1000;

__device__ int g_device_error = 0;   // 0 ok; otherwise the code of the first wait that ran out

struct TcParams {
  int M, N, K;
  int a_mn, b_mn;          // 1 = MN-major operand
  int k_splits;            // the K range is cut into this many slices; slice z writes out_lo + z*split_stride
  int64_t split_stride;    // in floats
  Epilogue ep;
  int* err;
};

// One product of a launch: its tensor maps, its parameters and its share of the (one-dimensional) grid.
// CTA `cta_begin + (z * grid_y + y) * grid_x + x` computes tile (row block y, column block x) of K slice z.
struct TcProblem {
  CUtensorMap map_a, map_b;
  TcParams p;
  int cta_begin, grid_x, grid_y;
};
template <int NP>
struct TcGroup {
  TcProblem prob[NP];
  int n;
};

// ---------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait.  Returns false (and records `code`) when the limit is reached.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* aborted, int* err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  const long long limit = *aborted ? kWaitCyclesAborted : kWaitCycles;
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) {
      *aborted = 1;
      atomicCAS(err, 0, code);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// ---------------------------------------------------------------------------------------- kernel
template <int kStages, int kBN, int NP, bool kDirect>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const __grid_constant__ TcGroup<NP> grp) {
  extern __shared__ uint8_t smem_raw[];
  int pj = 0;
  if (NP > 1) {
    while (pj + 1 < grp.n && (int)blockIdx.x >= grp.prob[pj + 1].cta_begin) ++pj;
  }
  const TcProblem& prob = grp.prob[pj];
  const TcParams& p = prob.p;
  const CUtensorMap& map_a = prob.map_a;
  const CUtensorMap& map_b = prob.map_b;
  const int cta_local = (int)blockIdx.x - prob.cta_begin;
  const int tile_x = cta_local % prob.grid_x;
  const int tile_y = (cta_local / prob.grid_x) % prob.grid_y;
  const int slice_z = cta_local / (prob.grid_x * prob.grid_y);
  constexpr int kStageBytes = stage_bytes(kBN);
  constexpr int kTmemCols = kBN;                           // one fp32 accumulator column per tile column
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned swizzle atoms
  uint8_t* gen = smem_raw + (tiles - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(gen + (size_t)kStages * kStageBytes);
  const uint32_t bar0 = tiles + kStages * kStageBytes;
  // bars: [0,S) full, [S,2S) empty, [2S] accumulator ready; then tmem base and the abort flag
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 1);
  volatile int* aborted = reinterpret_cast<volatile int*>(tmem_slot + 1);
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  const uint32_t acc_bar = bar0 + 8u * (2 * kStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = tile_y * kBM, n0 = tile_x * kBN;
  const int nk_all = (p.K + kBK - 1) / kBK;
  const int kb_begin = (int)((int64_t)nk_all * slice_z / p.k_splits);
  const int nk = (int)((int64_t)nk_all * (slice_z + 1) / p.k_splits) - kb_begin;   // >= 1: k_splits <= nk_all

  // one stage of operand tiles for k block kb of this CTA's slice
  auto load_stage = [&](int kb) {
    const int s = kb % kStages;
    mbar_expect_tx(full(s), kStageBytes);
    const uint32_t sa = tiles + s * kStageBytes, sb = sa + kTileBytes;
    const int k0 = (kb_begin + kb) * kBK;
    if (p.a_mn) {                       // A stored [K, M]: two boxes of 64 k-rows x 64 m
      tma_load_2d(sa, &map_a, full(s), m0, k0);
      tma_load_2d(sa + kTileBytes / 2, &map_a, full(s), m0 + 64, k0);
    } else {                            // A stored [M, K]: one box of 128 rows x 64 k
      tma_load_2d(sa, &map_a, full(s), k0, m0);
    }
    if (p.b_mn) {
#pragma unroll
      for (int a = 0; a < kBN / 64; ++a) tma_load_2d(sb + a * (kTileBytes / 2), &map_b, full(s), n0 + 64 * a, k0);
    } else {
      tma_load_2d(sb, &map_b, full(s), k0, n0);
    }
  };
  const int n_early = nk < kStages ? nk : kStages;           // the ring starts empty: its first round needs no wait
  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_a)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_b)) : "memory");
    for (int s = 0; s < kStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    mbar_init(acc_bar, 1);
    *aborted = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // the first round of loads goes out before tensor memory is allocated and the warps meet
    for (int kb = 0; kb < n_early; ++kb) load_stage(kb);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int kb = n_early; kb < nk; ++kb) {
        const int s = kb % kStages;
        const uint32_t ph = (kb / kStages) & 1;
        if (!mbar_wait(empty(s), ph ^ 1u, aborted, p.err, 1)) break;
        load_stage(kb);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: D = f32, A = B = bf16, majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
                             ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
      // K-major: 8-row groups 1024 B apart (SBO), K step of 16 elements = 32 B inside the swizzle span.
      // MN-major: 64-wide m atoms 8192 B apart (LBO), 8-k groups 1024 B apart (SBO), K step of 16 = 2048 B.
      const uint32_t a_lbo = p.a_mn ? 8192u : 16u, a_step = p.a_mn ? 2048u : 32u;
      const uint32_t b_lbo = p.b_mn ? 8192u : 16u, b_step = p.b_mn ? 2048u : 32u;
      for (int kb = 0; kb < nk; ++kb) {
        const int s = kb % kStages;
        const uint32_t ph = (kb / kStages) & 1;
        mbar_wait(full(s), ph, aborted, p.err, 2);
        tc_fence_after();
        const uint32_t sa = tiles + s * kStageBytes, sb = sa + kTileBytes;
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
          const uint64_t ad = smem_desc(sa + k * a_step, a_lbo, 1024u);
          const uint64_t bd = smem_desc(sb + k * b_step, b_lbo, 1024u);
          tc_mma(tmem, ad, bd, idesc, (kb > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(empty(s));              // frees the stage when these MMAs have read it
      }
      tc_commit(acc_bar);                 // accumulator complete
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 2..5
    const int q = warp & 3;               // tensor-memory lane quadrant this warp may read
    const Epilogue& ep = p.ep;
    mbar_wait(acc_bar, 0, aborted, p.err, 3);
    tc_fence_after();
    if constexpr (kDirect) {
      // Machine-filling products (their epilogue is a small part of a long CTA): every thread stores the
      // accumulator row it reads, 32 consecutive columns at a time.
      const int64_t m = (int64_t)m0 + 32 * q + lane;
      const bool m_ok = m < p.M;
#pragma unroll 1
      for (int c = 0; c < kBN / 32; ++c) {
        const int nb = n0 + 32 * c;
        if (nb >= p.N) break;
        uint32_t r[32];
        tc_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(32 * c), r);
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if (ep.bias) {
#pragma unroll
          for (int j = 0; j < 32; ++j) if (nb + j < p.N) v[j] += __ldg(ep.bias + nb + j);
        }
        if (ep.relu) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
        }
        if (!m_ok) continue;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const int n = nb + 8 * g;
          if (n >= p.N) break;
          float* x = v + 8 * g;
          if (ep.mask && n < ep.mask_cols) {                       // bf16 activation of the producing layer
            const uint4 mk = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(ep.mask) + m * ep.ld_mask + n);
            const uint32_t w[4] = {mk.x, mk.y, mk.z, mk.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              // a bf16 is positive iff its sign bit is clear and it is not zero
              const uint32_t lo = w[j] & 0xFFFFu, hi = w[j] >> 16;
              if (!((lo & 0x8000u) == 0 && (lo & 0x7FFFu) != 0)) x[2 * j] = 0.f;
              if (!((hi & 0x8000u) == 0 && (hi & 0x7FFFu) != 0)) x[2 * j + 1] = 0.f;
            }
          }
          if (n < ep.lo_cols) {
            if (ep.lo_bf16) {
              uint4 o;
              o.x = pack2(x[0], x[1]); o.y = pack2(x[2], x[3]); o.z = pack2(x[4], x[5]); o.w = pack2(x[6], x[7]);
              *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(ep.out_lo) + m * ep.ld_lo + n) = o;
            } else {
              float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(ep.out_lo) + (int64_t)slice_z * p.split_stride + m * ep.ld_lo + n);
              o[0] = make_float4(x[0], x[1], x[2], x[3]);
              o[1] = make_float4(x[4], x[5], x[6], x[7]);
            }
          } else if (ep.out_hi) {
            float4* o = reinterpret_cast<float4*>(ep.out_hi + m * ep.ld_hi + (n - ep.lo_cols));
            o[0] = make_float4(x[0], x[1], x[2], x[3]);
            o[1] = make_float4(x[4], x[5], x[6], x[7]);
          }
        }
      }
    } else {
      // tcgen05.ld hands a thread one accumulator row; stores of that shape put 32 different rows into one
      // instruction.  For the short CTAs of a training step each warp turns its 32 x 32 block round in shared
      // memory (the operand ring is idle once the accumulator is complete) and continues with four consecutive
      // columns per lane, eight lanes per row: bias, ReLU, mask and stores touch whole 64- or 128-byte row segments.
      float* stg = reinterpret_cast<float*>(gen) + q * (32 * kStgLd);   // rows of 36 floats: 128-bit accesses without bank conflicts
      const int cl = 4 * (lane & 7), rl = lane >> 3;
#pragma unroll 1
      for (int c = 0; c < kBN / 32; ++c) {
        const int nb = n0 + 32 * c;
        if (nb >= p.N) break;
        uint32_t r[32];
        tc_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(32 * c), r);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<uint4*>(stg + lane * kStgLd + 4 * j) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        __syncwarp();
        const int n = nb + cl;
        if (n < p.N) {                       // N is a multiple of 8: four columns are inside together or not at all
          float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
          if (ep.bias) bv = __ldg(reinterpret_cast<const float4*>(ep.bias + n));
          const bool masked = ep.mask && n < ep.mask_cols;
          // the mask words of all eight rows are requested before any is used: one round of load latency, not eight
          uint2 mk[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int64_t m = (int64_t)m0 + 32 * q + rl + 4 * i;
            mk[i] = make_uint2(0x3F803F80u, 0x3F803F80u);   // four positive values: nothing is masked
            if (masked && m < p.M)
              mk[i] = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(ep.mask) + m * ep.ld_mask + n);
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int row = rl + 4 * i;
            const int64_t m = (int64_t)m0 + 32 * q + row;
            if (m >= p.M) continue;
            const float4 sv = *reinterpret_cast<const float4*>(stg + row * kStgLd + cl);
            float x0 = sv.x + bv.x, x1 = sv.y + bv.y, x2 = sv.z + bv.z, x3 = sv.w + bv.w;
            if (ep.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); x2 = fmaxf(x2, 0.f); x3 = fmaxf(x3, 0.f); }
            // bf16 activation of the producing layer: positive iff sign clear and not zero
            if (!((mk[i].x & 0x8000u) == 0 && (mk[i].x & 0x7FFFu) != 0)) x0 = 0.f;
            if (!((mk[i].x & 0x80000000u) == 0 && (mk[i].x & 0x7FFF0000u) != 0)) x1 = 0.f;
            if (!((mk[i].y & 0x8000u) == 0 && (mk[i].y & 0x7FFFu) != 0)) x2 = 0.f;
            if (!((mk[i].y & 0x80000000u) == 0 && (mk[i].y & 0x7FFF0000u) != 0)) x3 = 0.f;
            if (n < ep.lo_cols) {
              if (ep.lo_bf16) {
                uint2 o;
                o.x = pack2(x0, x1); o.y = pack2(x2, x3);
                *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(ep.out_lo) + m * ep.ld_lo + n) = o;
              } else {
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(ep.out_lo) + (int64_t)slice_z * p.split_stride + m * ep.ld_lo + n) =
                    make_float4(x0, x1, x2, x3);
              }
            } else if (ep.out_hi) {
              *reinterpret_cast<float4*>(ep.out_hi + m * ep.ld_hi + (n - ep.lo_cols)) = make_float4(x0, x1, x2, x3);
            }
          }
        }
        __syncwarp();                        // the block is read before the next one overwrites it
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------- host side
static PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

// bf16 matrix with `inner` contiguous elements per row, `outer` rows, row pitch ld elements.
static bool make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld, int box_inner,
                     int box_outer) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

static int* device_error_ptr() {
  static int* ptr[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_device_error) != cudaSuccess) return nullptr;
    ptr[dev] = reinterpret_cast<int*>(p);
  }
  return ptr[dev];
}

bool gemm_tc_eligible(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep) {
  if (A.kind != OP_BF16 || B.kind != OP_BF16) return false;
  if (M < 1 || N < 8 || K < 16 || (N & 7)) return false;
  auto ok = [](const Operand& o) {
    const bool kmaj = o.s_k == 1, mnmaj = o.s_row == 1 && o.s_k != 1;
    if (!kmaj && !mnmaj) return false;
    const int64_t ld = kmaj ? o.s_row : o.s_k;
    return (ld & 7) == 0 && aligned16(o.p);
  };
  if (!ok(A) || !ok(B)) return false;
  if ((ep.lo_cols & 7) || (ep.mask && ((ep.mask_cols & 7) || !ep.mask_bf16 || (ep.ld_mask & 7) || !aligned16(ep.mask))))
    return false;
  if (ep.out_lo && (!aligned16(ep.out_lo) || (ep.ld_lo & (ep.lo_bf16 ? 7 : 3)))) return false;
  if (ep.out_hi && (!aligned16(ep.out_hi) || (ep.ld_hi & 3))) return false;
  if (ep.lo_cols < N && !ep.out_hi) return false;
  return true;
}

// Tile width and ring depth of a launch.
enum TcVariant { TC_SMALL = 0, TC_LARGE = 1, TC_WIDE = 2, TC_NARROW = 3 };
// Products of at least this many flops (4096 x 1024 x 1024) take the 128 x 256 tiles even when they fill the SMs less than
// twice: their CTAs run long enough for the tile's lower shared-memory traffic per flop to outweigh the smaller grid
// (the 3.6 GFLOP products of a 2048-sample step are below it: wide tiles cost that step 3 %).
constexpr double kHeavyFlops = 8589934592.0;
constexpr int kStagesNarrow = 4;   // 128 x 64 tiles: 4 stages of 24 KiB, two CTAs per SM (measured: giving a launch of at most one CTA
                                   // per SM the whole shared memory as a deeper ring lowers whole-step throughput by 3-5 %)

template <int kStages, int kBN, int NP, bool kDirect>
static ss_status launch_group(const TcGroup<NP>& g, int total_ctas, cudaStream_t st) {
  static bool attr_set[64];
  int dev = 0;
  SS_CUDA(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    SS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<kStages, kBN, NP, kDirect>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)tc_smem_bytes(kStages, kBN)));
    attr_set[dev] = true;
  }
  { SS_TIMED("gemm_tc_kernel", st);
  gemm_tc_kernel<kStages, kBN, NP, kDirect><<<total_ctas, kTcThreads, tc_smem_bytes(kStages, kBN), st>>>(g);
  }
  SS_LAUNCH_OK();
  return SS_OK;
}

// Fills one problem of a group for tile width bn; returns its CTA count (0 on failure).
static int fill_problem(TcProblem* pr, const TcJob& j, int bn, int cta_begin, int* err) {
  TcParams& p = pr->p;
  p.M = j.M; p.N = j.N; p.K = j.K;
  p.a_mn = (j.A.s_k != 1);
  p.b_mn = (j.B.s_k != 1);
  const int nk_all = (j.K + kBK - 1) / kBK;
  int ks = j.k_splits < 1 ? 1 : j.k_splits;
  if (ks > nk_all) ks = nk_all;
  p.k_splits = ks;
  p.split_stride = j.split_stride;
  p.ep = j.ep;
  p.err = err;
  const bool oka = p.a_mn ? make_map(&pr->map_a, j.A.p, j.M, j.K, j.A.s_k, 64, 64)
                          : make_map(&pr->map_a, j.A.p, j.K, j.M, j.A.s_row, 64, kBM);
  const bool okb = p.b_mn ? make_map(&pr->map_b, j.B.p, j.N, j.K, j.B.s_k, 64, 64)
                          : make_map(&pr->map_b, j.B.p, j.K, j.N, j.B.s_row, 64, bn);
  if (!oka || !okb) return 0;
  pr->cta_begin = cta_begin;
  pr->grid_x = (j.N + bn - 1) / bn;
  pr->grid_y = (j.M + kBM - 1) / kBM;
  return pr->grid_x * pr->grid_y * ks;
}

static bool splits_ok(const TcJob& j) {
  const Epilogue& ep = j.ep;                 // slices are plain fp32 sums
  return j.k_splits <= 1 || !(ep.lo_bf16 || ep.lo_cols < j.N || ep.bias || ep.relu || ep.mask);
}

ss_status gemm_tc_group(const TcJob* jobs, int n, cudaStream_t st) {
  if (n < 1 || n > kTcMaxGroup) return SS_ERR_SHAPE;
  for (int i = 0; i < n; ++i)
    if (!splits_ok(jobs[i])) return SS_ERR_SHAPE;
  int* err = device_error_ptr();
  if (!err) return SS_ERR_CUDA;
  if (n == 1) {
    const TcJob& j = jobs[0];
    const int nk_all = (j.K + kBK - 1) / kBK;
    int ks = j.k_splits < 1 ? 1 : j.k_splits;
    if (ks > nk_all) ks = nk_all;
    const int nk_slice = (nk_all + ks - 1) / ks;
    const long long mt = (j.M + kBM - 1) / kBM;
    const long long ctas128 = (long long)((j.N + 127) / 128) * mt * ks;
    const long long ctas256 = (long long)((j.N + 255) / 256) * mt * ks;
    int variant = TC_SMALL;
    const bool heavy = 2.0 * j.M * j.N * j.K >= kHeavyFlops;
    if (j.N >= 256 && (ctas256 >= 2ll * num_sms() || heavy) && nk_slice >= 2 * kStagesWide) variant = TC_WIDE;
    else if (ctas128 >= 2ll * num_sms() && nk_slice >= 2 * kStagesLarge) variant = TC_LARGE;
    else if (j.N <= 64 || 2 * ctas128 <= num_sms()) variant = TC_NARROW;    // a narrow product, or too few 128-wide tiles to occupy the SMs
    const int bn = variant == TC_WIDE ? 256 : (variant == TC_NARROW ? 64 : 128);
    alignas(64) TcGroup<1> g;
    g.n = 1;
    const int ctas = fill_problem(&g.prob[0], j, bn, 0, err);
    if (ctas < 1) return SS_ERR_CUDA;
    switch (variant) {
      case TC_WIDE: return launch_group<kStagesWide, 256, 1, true>(g, ctas, st);
      case TC_LARGE: return launch_group<kStagesLarge, 128, 1, true>(g, ctas, st);
      case TC_NARROW: return launch_group<kStagesNarrow, 64, 1, false>(g, ctas, st);
      default: return launch_group<kStagesSmall, 128, 1, false>(g, ctas, st);
    }
  }
  // a group made of wide products that is heavy as a whole takes the 128 x 256 tiles as well
  double flops = 0.0;
  bool wide = true;
  for (int i = 0; i < n; ++i) {
    const TcJob& j = jobs[i];
    flops += 2.0 * j.M * j.N * j.K;
    const int nk_all = (j.K + kBK - 1) / kBK;
    const int ks = j.k_splits < 1 ? 1 : (j.k_splits > nk_all ? nk_all : j.k_splits);
    if (j.N < 256 || (nk_all + ks - 1) / ks < 2 * kStagesWide) wide = false;
  }
  wide = wide && flops >= 2.0 * kHeavyFlops;
  alignas(64) TcGroup<kTcMaxGroup> g;
  g.n = n;
  int total = 0;
  for (int i = 0; i < n; ++i) {
    const int ctas = fill_problem(&g.prob[i], jobs[i], wide ? 256 : 128, total, err);
    if (ctas < 1) return SS_ERR_CUDA;
    total += ctas;
  }
  for (int i = n; i < kTcMaxGroup; ++i) g.prob[i] = g.prob[n - 1];   // never selected; keeps the parameter block defined
  if (wide) return launch_group<kStagesWide, 256, kTcMaxGroup, true>(g, total, st);
  return launch_group<kStagesSmall, 128, kTcMaxGroup, false>(g, total, st);
}

ss_status gemm_tc(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st,
                  int k_splits, int64_t split_stride) {
  TcJob j{M, N, K, A, B, ep, k_splits, split_stride};
  return gemm_tc_group(&j, 1, st);
}

int read_device_error(bool clear) {
  int* d = device_error_ptr();
  if (!d) return -1;
  int v = 0;
  if (cudaMemcpy(&v, d, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
  if (clear && v != 0) {
    int z = 0;
    cudaMemcpy(d, &z, sizeof(int), cudaMemcpyHostToDevice);
  }
  return v;
}

ss_status gemm(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st) {
  if (gemm_tc_eligible(M, N, K, A, B, ep)) return gemm_tc(M, N, K, A, B, ep, st, 1, 0);
  return gemm_simt(M, N, K, A, B, ep, st);
}

}  // namespace ss

extern "C" {

int ss_device_error(int clear) { return ss::read_device_error(clear != 0); }

ss_status ss_gemm_bf16(const void* a, int a_mn_major, int64_t lda, const void* b, int b_mn_major, int64_t ldb,
                       float* c, int64_t ldc, int M, int N, int K, int force_simt, ss_stream stream) {
  using namespace ss;
  if (!a || !b || !c) return SS_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || lda < 1 || ldb < 1 || ldc < N) return SS_ERR_SHAPE;
  ss_status stt = check_arch();
  if (stt != SS_OK) return stt;
  Operand A{a, OP_BF16, a_mn_major ? 1 : lda, a_mn_major ? lda : 1};
  Operand B{b, OP_BF16, b_mn_major ? 1 : ldb, b_mn_major ? ldb : 1};
  Epilogue ep;
  ep.out_lo = c; ep.lo_bf16 = 0; ep.ld_lo = ldc; ep.lo_cols = N;
  if (force_simt) return gemm_simt(M, N, K, A, B, ep, as_stream(stream));
  if (!gemm_tc_eligible(M, N, K, A, B, ep)) return SS_ERR_ALIGN;
  return gemm_tc(M, N, K, A, B, ep, as_stream(stream), 1, 0);
}

}  // extern "C"
