// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores (tcgen05) of sm_100a, as a persistent kernel.
//
//   C[m, n] = sum_k A(m, k) * B(n, k)
//
// One launch (a "flow") holds one or several products.  Its CTAs (at most one per SM) stay resident and draw
// 128 x kBN output tiles from a counter in device memory, in the order the products are listed.  Inside a CTA
// three roles run concurrently on their own warps:
//   warp 0 (one lane)  draws tiles and streams 128 x 64 / 64 x kBN operand tiles into a ring of shared-memory
//                      stages with TMA (128-byte swizzle), running ahead into the next tile;
//   warp 1 (one lane)  issues tcgen05.mma (M = 128, N = 16..kBN, K = 16) into one of TWO accumulators in tensor
//                      memory and releases stages with tcgen05.commit;
//   warps 2-5          read a finished accumulator with tcgen05.ld (one row per thread) and apply the epilogue
//                      (bias, ReLU, ReLU-gradient mask, bf16 / fp32 stores), while the MMA warp already fills the
//                      other accumulator.
// Set-up (barriers, tensor memory, descriptor prefetch) is paid once per CTA, not once per tile.
//
// A product may read what an earlier product of the same flow writes (a layer reading the previous layer's
// activations, a weight gradient reading the gradient tensor an input-gradient product produces).  Finished tiles
// count up a per-(product, row block) word in device memory; the TMA role of a dependent tile waits for the words
// it needs before it loads the operand (release / acquire at device scope, plus a proxy fence because the data is
// written through the generic proxy and read by TMA).  A tile only ever waits for tiles drawn before it, by CTAs
// that are running, so the wait ends whatever else occupies the device.
//
// Either operand may be K-major (k contiguous in memory: the forward pass reads activations [B, in]
// and weights [out, in] this way) or MN-major (m or n contiguous: the backward pass reads the same
// buffers transposed, dW = dY^T X and dX = dY W), so no transposed copy of any matrix is ever made.
// K-major tiles are one TMA box of 128 rows x 64 k; MN-major tiles are boxes of 64 k x 64 m, the
// canonical 128-byte-swizzle layouts of the shared-memory matrix descriptor in both cases.
//
// Every wait (mbarrier or dependency word) is bounded: when it runs out the kernel raises a device error flag,
// every role stops, nothing more is stored, outstanding copies are awaited, tensor memory is freed and the kernel
// returns; the host reads the flag (ss_device_error).
#include <cuda.h>
#include <cudaTypedefs.h>
#include "gemm.cuh"
#include "profile.cuh"

// Hook for a time-stamp trace of the roles (a development harness defines it before including this file); no code here.
#ifndef SS_TC_TRACE
#define SS_TC_TRACE(id, tile)
#endif

namespace ss {

constexpr int kBM = 128, kBK = 64;   // tile rows and k depth; the tile width kBN (128 or 256) is a template parameter
constexpr int kTileBytes = kBM * kBK * 2;                 // 16 KiB: the A tile, and every 128 columns of the B tile
__host__ __device__ constexpr int stage_bytes(int bn) { return kTileBytes + bn * kBK * 2; }
constexpr int kEpiWarps = 4;                              // one per tensor-memory lane quadrant
constexpr int kTcThreads = 64 + 32 * kEpiWarps;
constexpr int kQueue = 4;                                 // tiles a CTA may have drawn and not yet finished
// Ring depth: 5 stages of 32 KiB for 128-wide tiles and for CTA pairs, 3 stages of 48 KiB for 256-wide tiles (a
// quarter less shared-memory traffic per flop than 128-wide ones); one CTA per SM in every case.
constexpr int kStagesNarrow = 5, kStagesWide = 3, kStagesPair = 5;
constexpr int kCtlBytes = 512;                            // barriers, tile queue, tensor-memory address, abort flag
// Per epilogue warp: two 4 KiB slabs (32 rows x 128 bytes, 128-byte swizzle) from which TMA stores pieces of the
// output (one is filled while the other is being read), and the tile's bias values.
constexpr int kSlabBytes = 32 * 128;
constexpr int kBiasBytes = 256 * 4;
constexpr int kEpiWarpBytes = 2 * kSlabBytes + kBiasBytes;
constexpr size_t tc_smem_bytes(int stages, int load_n, size_t meta_bytes) {
  return (size_t)stages * stage_bytes(load_n) + kEpiWarps * kEpiWarpBytes + 1024 /*alignment slack*/ + kCtlBytes + meta_bytes;
}
constexpr long long kWaitCycles = 400ll * 1000 * 1000;    // ~0.2 s: far beyond any legitimate wait

__device__ int g_device_error = 0;   // 0 ok; otherwise the code of the first wait that ran out

struct TcParams {
  int M, N, K;
  int a_mn, b_mn;          // 1 = MN-major operand
  int k_splits;            // the K range is cut into this many slices; slice z writes out_lo + z*split_stride
  int64_t split_stride;    // in floats
  int dep, dep_mode, dep_k_blocks, dep_need;   // see TcJob; dep_need = arrivals that complete a row block of `dep`
  int dep_need_all;        // arrivals that complete all of `dep`
  int signal_x;            // tiles with x < signal_x report completion
  int tma_out;             // 1: outputs leave through shared memory and TMA stores, the mask arrives by TMA
  Epilogue ep;
};

// One product of a flow: its tensor maps, its parameters and its share of the tile sequence.
// Tile `tile_begin + (z * grid_y + y) * grid_x + x` is (row block y, column block x) of K slice z.
// Everything but the tensor maps is copied into shared memory when a CTA starts and from there into registers when a
// role takes up a tile: the parameter block is indexed by a run-time product number, and reading it field by field
// inside the loops would put a constant-bank load in front of every use.
struct TcMeta {
  TcParams p;
  int tile_begin, grid_x, grid_y, pad;
};
struct TcProblem {
  CUtensorMap map_a, map_b;
  CUtensorMap map_lo, map_hi;             // out_lo (3-d for float: column, row, K slice), out_hi; used when tma_out
  TcMeta meta;
};
template <int NP>
struct TcFlow {
  TcProblem prob[NP];
  int n, total_tiles;
  int* ctrl;               // [0] tile counter, [1] exit ticket, [2 + j * rb_stride + rb] completions; nullptr: round-robin
  int rb_stride;
  int* err;
};

// ---------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One try: the hardware may park the thread for up to the given time while the phase is incomplete (it is woken
// when the phase completes), so a waiting role leaves the issue slots to the other warps of the SM.
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
  return ok;
}
// Bounded wait.  Returns false when the limit is reached (records `code`) or another role has given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* aborted, int* err, int code) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*aborted) return false;
    if (clock64() - t0 > kWaitCycles) {
      *aborted = 1;
      atomicCAS(err, 0, code);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Bounded wait for a completion word of the flow to reach `need`.
__device__ __forceinline__ bool wait_count(const int* word, int need, volatile int* aborted, int* err) {
  if (ld_acquire(word) < need) {
    const long long t0 = clock64();
    while (ld_acquire(word) < need) {
      if (*aborted) return false;
      if (clock64() - t0 > kWaitCycles) {
        *aborted = 1;
        atomicCAS(err, 0, 4);
        return false;
      }
      __nanosleep(200);
    }
  }
  // what the other CTAs stored through the generic proxy is read by TMA (async proxy) from here on
  asm volatile("fence.proxy.async;" ::: "memory");
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// ---- CTA pairs (cta_group::2): two CTAs of a cluster share one 256-row MMA
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {   // the same offset in another CTA of the cluster
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load of one CTA of a pair; the bytes are counted on a barrier that may live in the other CTA (no multicast:
// each CTA fetches its own tiles)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {          // arrives on the barrier at this offset in both CTAs
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
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

// Two bits for a packed pair of bf16: each "the value is positive" (sign clear and not zero).
__device__ __forceinline__ uint32_t positive2(uint32_t packed) {
  const uint32_t lo = packed & 0xFFFFu, hi = packed >> 16;
  return (uint32_t)((lo & 0x8000u) == 0 && (lo & 0x7FFFu) != 0) | ((uint32_t)((hi & 0x8000u) == 0 && (hi & 0x7FFFu) != 0) << 1);
}
__device__ __forceinline__ uint32_t pick4(const uint4& v, int i) {
  return (i & 2) ? ((i & 1) ? v.w : v.z) : ((i & 1) ? v.y : v.x);
}
__device__ __forceinline__ void put4(uint4& v, int i, uint32_t w) {
  if (i == 0) v.x = w; else if (i == 1) v.y = w; else if (i == 2) v.z = w; else v.w = w;
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

// A tile of the flow: which product, which block, which K range.
struct TileAt {
  int j, x, y, z, kb_begin, nk;
};
__device__ __forceinline__ TileAt locate_tile(const TcMeta* meta, int n, int t) {
  int j = 0;
  while (j + 1 < n && t >= meta[j + 1].tile_begin) ++j;
  const int gx = meta[j].grid_x, gy = meta[j].grid_y, K = meta[j].p.K, ks = meta[j].p.k_splits;
  const int local = t - meta[j].tile_begin;
  TileAt a;
  a.j = j;
  a.x = local % gx;
  a.y = (local / gx) % gy;
  a.z = local / (gx * gy);
  const int nk_all = (K + kBK - 1) / kBK;
  a.kb_begin = (int)((int64_t)nk_all * a.z / ks);
  a.nk = (int)((int64_t)nk_all * (a.z + 1) / ks) - a.kb_begin;   // >= 1: k_splits <= nk_all
  return a;
}

// ---------------------------------------------------------------------------------------- kernel
// kPair: the CTAs come in pairs (clusters of two).  A pair computes a 256 x kBN tile with one tcgen05.mma.cta_group::2
// per k step, issued by the pair's first CTA: each CTA holds its 128 rows of A, HALF of the B tile (the tensor cores of
// both SMs read both halves) and the accumulator of its own 128 rows.  Per flop a CTA loads and reads a third less
// shared memory than with 128 x 256 tiles of its own, which is what bounds those.  Tiles are assigned round-robin to
// the pairs (no dependencies between products in this mode).
// 112 registers a thread (the epilogue would take 144; capped, it recomputes a few addresses and spills nothing): a
// CTA of this kernel sits beside the blocks of other streams' kernels, which get the registers it leaves.
template <int kStages, int kBN, int NP, bool kPair>
__global__ void __maxnreg__(112)
gemm_tc_kernel(const __grid_constant__ TcFlow<NP> flow) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int kLoadN = kPair ? kBN / 2 : kBN;            // columns of B this CTA loads
  constexpr int kTileM = kPair ? 2 * kBM : kBM;            // rows of a tile
  constexpr int kStageBytes = stage_bytes(kLoadN);
  constexpr int kTmemCols = 2 * kBN;                       // two accumulators of kBN fp32 columns
  const uint32_t rank = kPair ? cluster_rank() : 0u;       // 0: the CTA that issues the pair's MMAs
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned swizzle atoms
  uint8_t* gen = smem_raw + (tiles - raw);
  const uint32_t epi0 = tiles + kStages * kStageBytes;            // 1024-byte aligned: stages are multiples of 1 KiB
  uint8_t* epi_gen = gen + (size_t)kStages * kStageBytes;
  uint8_t* ctl = epi_gen + kEpiWarps * kEpiWarpBytes;
  const uint32_t bar0 = epi0 + kEpiWarps * kEpiWarpBytes;
  // barriers: [0,S) full, [S,2S) empty, then accumulator full[2], empty[2], queue full[kQueue], empty[kQueue]
  constexpr int kNumBars = 2 * kStages + 4 + 2 * kQueue;
  int* tile_q = reinterpret_cast<int*>(ctl + 8 * kNumBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tile_q + kQueue);
  volatile int* aborted = reinterpret_cast<volatile int*>(tmem_slot + 1);
  TcMeta* meta = reinterpret_cast<TcMeta*>(ctl + kCtlBytes);
  static_assert(8 * kNumBars + 4 * kQueue + 8 <= kCtlBytes, "control region");
  static_assert(sizeof(TcMeta) % 4 == 0, "copied word by word");
  const int n_prob = flow.n;
  for (int j = 0; j < n_prob; ++j) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&flow.prob[j].meta);
    uint32_t* dst = reinterpret_cast<uint32_t*>(meta + j);
    for (int i = threadIdx.x; i < (int)(sizeof(TcMeta) / 4); i += kTcThreads) dst[i] = src[i];
  }
  auto full = [&](int s) { return bar0 + 8u * s; };
  auto empty = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto acc_full = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto acc_empty = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  auto q_full = [&](int s) { return bar0 + 8u * (2 * kStages + 4 + s); };
  auto q_empty = [&](int s) { return bar0 + 8u * (2 * kStages + 4 + kQueue + s); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int j = 0; j < flow.n; ++j) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&flow.prob[j].map_a)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&flow.prob[j].map_b)) : "memory");
    }
    for (int s = 0; s < kStages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), kPair ? 2 * kEpiWarps : kEpiWarps); }
    for (int s = 0; s < kQueue; ++s) { mbar_init(q_full(s), 1); mbar_init(q_empty(s), 1 + kEpiWarps); }
    *aborted = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();                           // the other CTA's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  int* const done0 = flow.ctrl ? flow.ctrl + 2 : nullptr;
  if (threadIdx.x == 0) SS_TC_TRACE(1, -1);

  if (warp == 0) {
    // ------------------------------------------------------------------ tile scheduler + TMA producer
    if (lane == 0) {
      uint32_t it = 0;                                     // stages filled so far (over all tiles)
      // the ticket of the next tile is drawn while the current one is loaded (the counter is a round trip to L2 away);
      // tickets are still drawn in order by a running CTA and worked off in order, which is all the waiting needs
      const int unit = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x, n_units = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
      int t_next = flow.ctrl ? atomicAdd(flow.ctrl, 1) : unit;
      for (uint32_t qi = 0;; ++qi) {
        const int qs = qi % kQueue;
        if (!mbar_wait(q_empty(qs), ((qi / kQueue) & 1) ^ 1u, aborted, flow.err, 5)) break;
        int t = t_next;
        if (t >= flow.total_tiles) t = -1;
        if (t >= 0) t_next = flow.ctrl ? atomicAdd(flow.ctrl, 1) : (int)(unit + (qi + 1) * n_units);
        tile_q[qs] = t;
        mbar_arrive(q_full(qs));
        if (t < 0) break;
        SS_TC_TRACE(2, t);
        const TileAt a = locate_tile(meta, n_prob, t);
        const TcProblem& pr = flow.prob[a.j];
        const int m0 = a.y * kTileM + (int)rank * kBM, n0 = a.x * kBN + (int)rank * kLoadN;   // this CTA's rows, its part of B
        int dep_mode = 0, dep_need = 0, dep_kb = 0;
        const int* dep_words = nullptr;
        const int a_mn = meta[a.j].p.a_mn, b_mn = meta[a.j].p.b_mn, K = meta[a.j].p.K;
        if (meta[a.j].p.dep >= 0) {
          dep_mode = meta[a.j].p.dep_mode; dep_need = meta[a.j].p.dep_need;
          dep_kb = meta[a.j].p.k_splits == 1 ? meta[a.j].p.dep_k_blocks : 0;
          dep_words = done0 + meta[a.j].p.dep * flow.rb_stride;
        }
        // k blocks [0, nd) of this tile's range wait for the producing product (taken last); the others do not
        int nd = 0;
        if (dep_mode == 1) nd = (dep_kb > 0 && dep_kb < a.nk) ? dep_kb : a.nk;
        bool dep_ok = (nd == 0);
        int rb_ready = -1;                                 // dep_mode 2: the producer's row blocks up to here are complete
        if (dep_mode == 2 && ld_acquire(dep_words + flow.rb_stride - 1) >= meta[a.j].p.dep_need_all) {
          asm volatile("fence.proxy.async;" ::: "memory");
          rb_ready = 0x7fffffff;                           // the producing product is complete: nothing to wait for
        }
        bool failed = false;
        for (int i = 0; i < a.nk; ++i) {
          int kb = i + nd;
          if (kb >= a.nk) kb -= a.nk;                      // independent k blocks first
          if (!dep_ok && kb < nd) {
            if (!wait_count(dep_words + a.y, dep_need, aborted, flow.err)) { failed = true; break; }
            dep_ok = true;
          }
          const int k0 = (a.kb_begin + kb) * kBK;
          if (dep_mode == 2) {
            int rb = (k0 + kBK - 1) / kBM;                 // a 64-row k block lies inside one 128-row block
            const int rb_last = (K - 1) / kBM;
            if (rb > rb_last) rb = rb_last;
            if (rb > rb_ready) {
              if (!wait_count(dep_words + rb, dep_need, aborted, flow.err)) { failed = true; break; }
              rb_ready = rb;
            }
          }
          const int s = it % kStages;
          if (!mbar_wait(empty(s), ((it / kStages) & 1) ^ 1u, aborted, flow.err, 1)) { failed = true; break; }
          const uint32_t sa = tiles + s * kStageBytes, sb = sa + kTileBytes;
          if (kPair) {
            // both CTAs' tiles are counted on the first CTA's barrier, which its MMA thread waits on
            const uint32_t bar = map_to_cta(full(s), 0);
            if (rank == 0) mbar_expect_tx(full(s), 2 * kStageBytes);
            if (a_mn) {
              tma_load_2d_pair(sa, &pr.map_a, bar, m0, k0);
              tma_load_2d_pair(sa + kTileBytes / 2, &pr.map_a, bar, m0 + 64, k0);
            } else {
              tma_load_2d_pair(sa, &pr.map_a, bar, k0, m0);
            }
            if (b_mn) {
#pragma unroll
              for (int h = 0; h < kLoadN / 64; ++h) tma_load_2d_pair(sb + h * (kTileBytes / 2), &pr.map_b, bar, n0 + 64 * h, k0);
            } else {
#pragma unroll
              for (int h = 0; h < kLoadN / 128; ++h) tma_load_2d_pair(sb + h * kTileBytes, &pr.map_b, bar, k0, n0 + 128 * h);
            }
          } else {
          mbar_expect_tx(full(s), kStageBytes);
          if (a_mn) {                         // A stored [K, M]: two boxes of 64 k-rows x 64 m
            tma_load_2d(sa, &pr.map_a, full(s), m0, k0);
            tma_load_2d(sa + kTileBytes / 2, &pr.map_a, full(s), m0 + 64, k0);
          } else {                            // A stored [M, K]: one box of 128 rows x 64 k
            tma_load_2d(sa, &pr.map_a, full(s), k0, m0);
          }
          if (b_mn) {
#pragma unroll
            for (int h = 0; h < kBN / 64; ++h) tma_load_2d(sb + h * (kTileBytes / 2), &pr.map_b, full(s), n0 + 64 * h, k0);
          } else {
#pragma unroll
            for (int h = 0; h < kBN / 128; ++h) tma_load_2d(sb + h * kTileBytes, &pr.map_b, full(s), k0, n0 + 128 * h);
          }
          }
          ++it;
          if (i == 0) SS_TC_TRACE(3, t);
        }
        if (failed) break;
        SS_TC_TRACE(4, t);
      }
      if (*aborted) {
        // the copies still in flight land in this CTA's shared memory: wait for them (bounded) before leaving
        const uint32_t first = it > (uint32_t)kStages ? it - kStages : 0u;
        for (uint32_t i = first; i < it; ++i) {
          const long long t0 = clock64();
          while (!mbar_try_wait(full(i % kStages), (i / kStages) & 1) && clock64() - t0 < 4000000ll) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      uint32_t it = 0, at = 0;                             // stages consumed, tiles accumulated
      for (uint32_t qi = 0;; ++qi) {
        const int qs = qi % kQueue;
        if (!mbar_wait(q_full(qs), (qi / kQueue) & 1, aborted, flow.err, 6)) break;
        const int t = tile_q[qs];
        mbar_arrive(q_empty(qs));
        if (t < 0) break;
        if (kPair && rank != 0) continue;                  // the pair's MMAs are issued by its first CTA
        const TileAt a = locate_tile(meta, n_prob, t);
        const int a_mn = meta[a.j].p.a_mn, b_mn = meta[a.j].p.b_mn;
        int n_mma = meta[a.j].p.N - a.x * kBN;             // columns of this tile, rounded up to the instruction's granule
        n_mma = n_mma >= kBN ? kBN : ((n_mma + 15) & ~15);
        if (kPair) n_mma = kBN;                            // each CTA holds exactly half of the instruction's columns
        // instruction descriptor: D = f32, A = B = bf16, majors, N >> 3, M >> 4
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
                               ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
        // K-major: 8-row groups 1024 B apart (SBO), K step of 16 elements = 32 B inside the swizzle span.
        // MN-major: 64-wide m atoms 8192 B apart (LBO), 8-k groups 1024 B apart (SBO), K step of 16 = 2048 B.
        const uint32_t a_lbo = a_mn ? 8192u : 16u, a_step = a_mn ? 2048u : 32u;
        const uint32_t b_lbo = b_mn ? 8192u : 16u, b_step = b_mn ? 2048u : 32u;
        const int buf = at & 1;
        if (!mbar_wait(acc_empty(buf), ((at >> 1) & 1) ^ 1u, aborted, flow.err, 7)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + (uint32_t)(buf * kBN);
        bool failed = false;
        for (int i = 0; i < a.nk; ++i) {
          const int s = it % kStages;
          if (!mbar_wait(full(s), (it / kStages) & 1, aborted, flow.err, 2)) { failed = true; break; }
          if (i == 0) SS_TC_TRACE(5, t);
          tc_fence_after();
          const uint32_t sa = tiles + s * kStageBytes, sb = sa + kTileBytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            const uint64_t ad = smem_desc(sa + k * a_step, a_lbo, 1024u);
            const uint64_t bd = smem_desc(sb + k * b_step, b_lbo, 1024u);
            if (kPair) tc_mma_pair(d_tmem, ad, bd, idesc, (i > 0 || k > 0) ? 1u : 0u);
            else tc_mma(d_tmem, ad, bd, idesc, (i > 0 || k > 0) ? 1u : 0u);
          }
          if (kPair) tc_commit_pair(empty(s));   // frees the stage in both CTAs when these MMAs have read it
          else tc_commit(empty(s));
          ++it;
        }
        if (failed) break;
        if (kPair) tc_commit_pair(acc_full(buf));   // accumulator complete, in both CTAs
        else tc_commit(acc_full(buf));
        SS_TC_TRACE(6, t);
        ++at;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps 2..5
    const int q = warp & 3;               // tensor-memory lane quadrant this warp may read
    uint8_t* const slab_gen = epi_gen + q * kEpiWarpBytes;              // [out 0][out 1][bias]
    const uint32_t slab_out = epi0 + q * kEpiWarpBytes;
    float* const s_bias = reinterpret_cast<float*>(slab_gen + 2 * kSlabBytes);
    uint32_t n_stores = 0;                // slabs handed to TMA so far (they alternate)
    uint32_t at = 0;
    for (uint32_t qi = 0;; ++qi) {
      const int qs = qi % kQueue;
      if (!mbar_wait(q_full(qs), (qi / kQueue) & 1, aborted, flow.err, 8)) break;
      const int t = tile_q[qs];
      __syncwarp();
      if (lane == 0) mbar_arrive(q_empty(qs));
      if (t < 0) break;
      const TileAt a = locate_tile(meta, n_prob, t);
      const Epilogue ep = meta[a.j].p.ep;                  // by value: registers
      struct { int M, N, signal_x; int64_t split_stride; } p = {meta[a.j].p.M, meta[a.j].p.N, meta[a.j].p.signal_x,
                                                                 meta[a.j].p.split_stride};
      const int m0 = a.y * kTileM + (int)rank * kBM, n0 = a.x * kBN;
      const int buf = at & 1;
      const bool tma_out = meta[a.j].p.tma_out != 0;
      const TcProblem& pr = flow.prob[a.j];
      // Everything the epilogue needs from memory is requested as soon as the tile is known, so that it arrives while
      // the tensor cores still work on the tile: the tile's bias values (every thread needs all of them: one 16-byte
      // load per lane into the warp's shared memory) and the thread's words of the ReLU-gradient mask.
      if (ep.bias) {
#pragma unroll
        for (int i = 0; i < kBN / 128; ++i) {
          const int n = n0 + 128 * i + 4 * lane;
          float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
          if (n < p.N) bv = __ldg(reinterpret_cast<const float4*>(ep.bias + n));   // N is a multiple of 8
          *reinterpret_cast<float4*>(s_bias + 128 * i + 4 * lane) = bv;
        }
      }
      // the row's mask words (one bit per column), when the producing layer left them: 16 bytes per 128 columns
      const int64_t mrow = (int64_t)m0 + 32 * q + lane;
      const bool use_bits = ep.mask_bits != nullptr;
      uint4 mq0 = make_uint4(~0u, ~0u, ~0u, ~0u), mq1 = mq0;
      if (use_bits && mrow < p.M) {
        if (n0 < ep.mask_cols) mq0 = __ldg(reinterpret_cast<const uint4*>(ep.mask_bits + mrow * ep.ld_mask_bits + (n0 >> 5)));
        if (kBN > 128 && n0 + 128 < ep.mask_cols)
          mq1 = __ldg(reinterpret_cast<const uint4*>(ep.mask_bits + mrow * ep.ld_mask_bits + ((n0 + 128) >> 5)));
      }
      __syncwarp();                                        // the bias values are in shared memory
      if (!mbar_wait(acc_full(buf), (at >> 1) & 1, aborted, flow.err, 3)) break;
      if (threadIdx.x == 64) SS_TC_TRACE(7, t);
      tc_fence_after();
      if (tma_out) {
        // The thread holds 32 consecutive columns of its accumulator row at a time.  It applies bias / ReLU / mask,
        // writes the row piece into the warp's slab in the 128-byte-swizzle layout, and one lane hands the slab to
        // TMA, which stores whole rows of it (and clips what lies beyond the matrix).  A slab is 64 columns of bf16
        // output (two pieces) or 32 columns of float output.
        const int sw = lane & 7;
        const uint32_t row_off = (uint32_t)lane * 128u;
        uint4 bq = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          const int nb = n0 + 32 * c;
          if (nb >= p.N) break;
          const int odd = c & 1;
          uint32_t r[32];
          tc_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kBN + 32 * c), r);
          float v[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
          if (ep.bias) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 bv = *reinterpret_cast<const float4*>(s_bias + 32 * c + j);   // the same address in every lane
              v[j] += bv.x; v[j + 1] += bv.y; v[j + 2] += bv.z; v[j + 3] += bv.w;
            }
          }
          if (ep.relu) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
          }
          if (use_bits && nb < ep.mask_cols) {               // (a tile with a mask takes this path only with mask words)
            uint32_t w = pick4((kBN > 128 && c >= 4) ? mq1 : mq0, c & 3);
            if (nb + 32 > ep.mask_cols) w |= ~0u << (ep.mask_cols - nb);   // columns from mask_cols on are not masked
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (!((w >> j) & 1u)) v[j] = 0.f;
          }
          const bool to_lo = nb < ep.lo_cols;
          if (to_lo && ep.lo_bf16) {
            uint8_t* const slab = slab_gen + (n_stores & 1) * kSlabBytes;
            if (!odd) {
              if (lane == 0) tma_store_wait_read1();       // this slab's previous contents have been read (the other may be in flight)
              __syncwarp();
            }
            uint32_t wbits = 0;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 o;
              o.x = pack2(v[8 * g], v[8 * g + 1]); o.y = pack2(v[8 * g + 2], v[8 * g + 3]);
              o.z = pack2(v[8 * g + 4], v[8 * g + 5]); o.w = pack2(v[8 * g + 6], v[8 * g + 7]);
              *reinterpret_cast<uint4*>(slab + row_off + ((uint32_t)((g + 4 * odd) ^ sw) << 4)) = o;
              wbits |= (positive2(o.x) | (positive2(o.y) << 2) | (positive2(o.z) << 4) | (positive2(o.w) << 6)) << (8 * g);
            }
            if (ep.bits_out) {                             // the words of 128 columns leave together
              put4(bq, c & 3, wbits);
              if ((c & 3) == 3 || nb + 32 >= p.N) {
                if (mrow < p.M && !*aborted)
                  *reinterpret_cast<uint4*>(ep.bits_out + mrow * ep.ld_bits_out + ((n0 + 128 * (c >> 2)) >> 5)) = bq;
                bq = make_uint4(0u, 0u, 0u, 0u);
              }
            }
            if (odd || nb + 32 >= p.N || nb + 32 >= ep.lo_cols) {   // the slab is complete (or the output ends here)
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
              if (lane == 0 && !*aborted) {
                tma_store_2d(&pr.map_lo, slab_out + (n_stores & 1) * kSlabBytes, nb - 32 * odd, m0 + 32 * q);
                tma_store_commit();
              }
              ++n_stores;
            }
          } else {
            uint8_t* const slab = slab_gen + (n_stores & 1) * kSlabBytes;
            if (lane == 0) tma_store_wait_read1();
            __syncwarp();
#pragma unroll
            for (int g = 0; g < 8; ++g)
              *reinterpret_cast<float4*>(slab + row_off + ((uint32_t)(g ^ sw) << 4)) =
                  make_float4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0 && !*aborted) {
              if (to_lo) tma_store_3d(&pr.map_lo, slab_out + (n_stores & 1) * kSlabBytes, nb, m0 + 32 * q, a.z);
              else tma_store_2d(&pr.map_hi, slab_out + (n_stores & 1) * kSlabBytes, nb - ep.lo_cols, m0 + 32 * q);
              tma_store_commit();
            }
            ++n_stores;
          }
        }
      } else {
      // tcgen05.ld hands a thread one accumulator row, 32 consecutive columns at a time: the thread applies the
      // epilogue to its row and stores 16-byte pieces of it (whole 32-byte sectors per pair of stores).
      const int64_t m = (int64_t)m0 + 32 * q + lane;
      const bool m_ok = m < p.M && !*aborted;
#pragma unroll 1
      for (int c = 0; c < kBN / 32; ++c) {
        const int nb = n0 + 32 * c;
        if (nb >= p.N) break;
        uint32_t r[32];
        tc_ld32(tmem + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * kBN + 32 * c), r);
        if (!m_ok) continue;
        float v[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if (ep.bias) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 bv = *reinterpret_cast<const float4*>(s_bias + 32 * c + j);   // the same address in every lane
            v[j] += bv.x; v[j + 1] += bv.y; v[j + 2] += bv.z; v[j + 3] += bv.w;
          }
        }
        if (ep.relu) {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.f);
        }
        uint32_t dbits = 0;
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
              dbits |= (positive2(o.x) | (positive2(o.y) << 2) | (positive2(o.z) << 4) | (positive2(o.w) << 6)) << (8 * g);
            } else {
              float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(ep.out_lo) + (int64_t)a.z * p.split_stride + m * ep.ld_lo + n);
              o[0] = make_float4(x[0], x[1], x[2], x[3]);
              o[1] = make_float4(x[4], x[5], x[6], x[7]);
            }
          } else if (ep.out_hi) {
            float4* o = reinterpret_cast<float4*>(ep.out_hi + m * ep.ld_hi + (n - ep.lo_cols));
            o[0] = make_float4(x[0], x[1], x[2], x[3]);
            o[1] = make_float4(x[4], x[5], x[6], x[7]);
          }
        }
        if (ep.bits_out && ep.lo_bf16 && nb < ep.lo_cols) ep.bits_out[m * ep.ld_bits_out + (nb >> 5)] = dbits;
      }
      }
      // the accumulator may be overwritten: this warp's reads of it are complete
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (kPair) mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));   // the MMA thread of the pair's first CTA waits for both
        else mbar_arrive(acc_empty(buf));
      }
      if (threadIdx.x == 64) SS_TC_TRACE(8, t);
      // completion word of the row block, for the products that read this output
      if (done0 && a.x < p.signal_x) {
        if (tma_out && lane == 0) tma_store_wait_all();    // what this warp's TMA stores wrote is complete in memory
        __threadfence();
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          atomicAdd(done0 + a.j * flow.rb_stride + a.y, 1);
          __threadfence();
          atomicAdd(done0 + a.j * flow.rb_stride + flow.rb_stride - 1, 1);   // after the row block's own word
        }
      }
      ++at;
    }
    if (lane == 0) tma_store_wait_all();                   // the slabs are read before the CTA gives up its shared memory
  }

  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();                           // neither CTA leaves while the other may still signal it
  if (warp == 1) {
    tc_fence_after();
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
  // the last CTA to leave clears the control words for the next launch (every other CTA is past its last access)
  if (flow.ctrl && threadIdx.x == 0 && !*aborted) {
    __threadfence();
    if (atomicAdd(flow.ctrl + 1, 1) == (int)gridDim.x - 1) {
      const int words = 2 + flow.n * flow.rb_stride;
      for (int i = 0; i < words; ++i) flow.ctrl[i] = 0;
      __threadfence();
    }
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

// Matrix with `inner` contiguous elements per row, `outer` rows, row pitch ld elements (and `planes` such matrices
// plane_stride elements apart when rank is 3); 128-byte swizzle, so box_inner * element size is at most 128 bytes.
static bool make_map_any(CUtensorMap* map, CUtensorMapDataType dt, int esize, const void* base, int64_t inner, int64_t outer,
                         int64_t ld, int box_inner, int box_outer, int rank = 2, int64_t planes = 1, int64_t plane_stride = 0) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)ld * esize, (cuuint64_t)plane_stride * esize};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}
static bool make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld, int box_inner,
                     int box_outer) {
  return make_map_any(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, inner, outer, ld, box_inner, box_outer);
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

template <int kStages, int kBN, bool kPair>
static ss_status launch_flow(const TcFlow<kTcMaxFlow>& f, int ctas, cudaStream_t st) {
  static bool attr_set[64];
  int dev = 0;
  SS_CUDA(cudaGetDevice(&dev));
  const size_t smem = tc_smem_bytes(kStages, kPair ? kBN / 2 : kBN, sizeof(TcMeta) * kTcMaxFlow);
  if (dev >= 0 && dev < 64 && !attr_set[dev]) {
    SS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<kStages, kBN, kTcMaxFlow, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem));
    attr_set[dev] = true;
  }
  { SS_TIMED("gemm_tc_kernel", st);
  if (kPair) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctas, 1, 1);
    cfg.blockDim = dim3(kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SS_CUDA(cudaLaunchKernelEx(&cfg, gemm_tc_kernel<kStages, kBN, kTcMaxFlow, kPair>, f));
  } else {
    gemm_tc_kernel<kStages, kBN, kTcMaxFlow, kPair><<<ctas, kTcThreads, smem, st>>>(f);
  }
  }
  SS_LAUNCH_OK();
  return SS_OK;
}

// Fills one problem of a flow for tile width bn; returns its tile count (0 on failure).
static int fill_problem(TcProblem* pr, const TcJob& j, int bn, int tile_begin, int tile_m = kBM) {
  TcParams& p = pr->meta.p;
  p.M = j.M; p.N = j.N; p.K = j.K;
  p.a_mn = (j.A.s_k != 1);
  p.b_mn = (j.B.s_k != 1);
  const int nk_all = (j.K + kBK - 1) / kBK;
  int ks = j.k_splits < 1 ? 1 : j.k_splits;
  if (ks > nk_all) ks = nk_all;
  p.k_splits = ks;
  p.split_stride = j.split_stride;
  p.ep = j.ep;
  p.dep = -1; p.dep_mode = 0; p.dep_k_blocks = 0; p.dep_need = 0; p.dep_need_all = 0;
  const bool oka = p.a_mn ? make_map(&pr->map_a, j.A.p, j.M, j.K, j.A.s_k, 64, 64)
                          : make_map(&pr->map_a, j.A.p, j.K, j.M, j.A.s_row, 64, kBM);
  const bool okb = p.b_mn ? make_map(&pr->map_b, j.B.p, j.N, j.K, j.B.s_k, 64, 64)
                          : make_map(&pr->map_b, j.B.p, j.K, j.N, j.B.s_row, 64, 128);
  if (!oka || !okb) return 0;
  // Outputs through TMA stores: every 64-column piece of a tile lies on one side of the lo / hi boundary.
  const Epilogue& ep = j.ep;
  p.tma_out = 0;
  pr->map_lo = pr->map_a; pr->map_hi = pr->map_a;   // defined, unused unless tma_out
  // (a mask must come as sign bits; a mask given by values only takes the epilogue with plain loads and stores)
  if (ep.out_lo && ep.lo_cols > 0 && ((ep.lo_cols & 63) == 0 || ep.lo_cols >= j.N) && (!ep.mask || ep.mask_bits)) {
    bool ok = true;
    if (ep.lo_bf16) {
      ok = make_map_any(&pr->map_lo, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ep.out_lo, ep.lo_cols < j.N ? ep.lo_cols : j.N, j.M,
                        ep.ld_lo, 64, 32);
    } else {
      const int64_t plane = ks > 1 ? j.split_stride : (int64_t)ep.ld_lo * j.M;
      ok = (plane & 3) == 0 && make_map_any(&pr->map_lo, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ep.out_lo,
                                            ep.lo_cols < j.N ? ep.lo_cols : j.N, j.M, ep.ld_lo, 32, 32, 3, ks, plane);
    }
    if (ok && ep.lo_cols < j.N)
      ok = ep.out_hi && make_map_any(&pr->map_hi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ep.out_hi, j.N - ep.lo_cols, j.M, ep.ld_hi, 32, 32);
    p.tma_out = ok ? 1 : 0;
  }
  pr->meta.tile_begin = tile_begin;
  pr->meta.grid_x = (j.N + bn - 1) / bn;
  pr->meta.grid_y = (j.M + tile_m - 1) / tile_m;
  pr->meta.pad = 0;
  int sx = pr->meta.grid_x;
  if (j.signal_cols > 0 && (j.signal_cols + bn - 1) / bn < sx) sx = (j.signal_cols + bn - 1) / bn;
  p.signal_x = sx;
  return pr->meta.grid_x * pr->meta.grid_y * ks;
}

static bool splits_ok(const TcJob& j) {
  const Epilogue& ep = j.ep;                 // slices are plain fp32 sums
  return j.k_splits <= 1 || !(ep.lo_bf16 || ep.lo_cols < j.N || ep.bias || ep.relu || ep.mask);
}

constexpr int kFlowCtasDefault = 32;
static int g_flow_ctas = 0;     // 0: kFlowCtasDefault
int set_flow_ctas(int ctas) {
  if (ctas >= 0) g_flow_ctas = ctas;
  return g_flow_ctas > 0 ? g_flow_ctas : kFlowCtasDefault;
}

ss_status gemm_tc_flow(const TcJob* jobs, int n, int* ctrl, int max_rows, int max_ctas, cudaStream_t st) {
  if (n < 1 || n > kTcMaxFlow) return SS_ERR_SHAPE;
  double flops = 0.0;
  for (int i = 0; i < n; ++i) {
    const TcJob& j = jobs[i];
    if (!splits_ok(j)) return SS_ERR_SHAPE;
    if (j.dep >= i || (j.dep >= 0 && (!ctrl || j.dep_mode < 1 || j.dep_mode > 2 || jobs[j.dep].k_splits > 1))) return SS_ERR_SHAPE;
    if (j.dep >= 0 && jobs[j.dep].M > max_rows) return SS_ERR_SHAPE;
    flops += 2.0 * j.M * j.N * j.K;
  }
  int* err = device_error_ptr();
  if (!err) return SS_ERR_CUDA;
  // A flow with dependencies keeps CTAs waiting for one another, and a CTA, waiting or not, holds its SM's shared
  // memory and a third of its registers, which the other streams' kernels then lack.  Measured with all replicas of
  // a model training at once (examples/s at 16 / 32 / 64 / 148 CTAs per flow): four replicas, batch 2048: 15.0 /
  // 16.0 / 15.2 / 13.4 M; eight replicas, batch 1024: 13.1 / 13.6 / 12.6 / 11.8 M; sixteen replicas of a model ten
  // times as large, batch 4096: 7.9 / 8.4 / 7.0 / 7.2 M -- while a flow alone on the device is fastest with a CTA on
  // every SM.  So a flow takes 32 CTAs unless the caller says otherwise (set_flow_ctas).
  int ctas = num_sms();
  if (ctrl && max_ctas <= 0) max_ctas = g_flow_ctas > 0 ? g_flow_ctas : kFlowCtasDefault;
  if (max_ctas > 0 && max_ctas < ctas) ctas = max_ctas;
  // 128 x 256 tiles where the flow has at least one of them for each of its CTAs (a third less shared-memory traffic
  // per flop than 128 x 128; a narrower product then has one partly empty tile per row block); 256 x 256 tiles on
  // CTA pairs where, in addition, every product is at least that wide, no product waits for another (tiles then go
  // round-robin) and there is no K slicing
  long long t256 = 0, t_pair = 0;
  bool pair = ctrl == nullptr;
  for (int i = 0; i < n; ++i) {
    const long long ks = jobs[i].k_splits < 1 ? 1 : jobs[i].k_splits;
    t256 += (long long)((jobs[i].N + 255) / 256) * ((jobs[i].M + kBM - 1) / kBM) * ks;
    t_pair += (long long)((jobs[i].N + 255) / 256) * ((jobs[i].M + 2 * kBM - 1) / (2 * kBM));
    if (ks > 1 || jobs[i].dep >= 0 || jobs[i].N < 256) pair = false;
  }
  const bool wide = t256 >= ctas;
  pair = pair && wide && t_pair >= num_sms() / 2;
  const int bn = wide ? 256 : 128;
  alignas(64) TcFlow<kTcMaxFlow> f;
  f.n = n;
  int total = 0;
  for (int i = 0; i < n; ++i) {
    const int tiles = fill_problem(&f.prob[i], jobs[i], bn, total, pair ? 2 * kBM : kBM);
    if (tiles < 1) return SS_ERR_CUDA;
    total += tiles;
  }
  for (int i = 0; i < n; ++i) {
    const TcJob& j = jobs[i];
    if (j.dep < 0) continue;
    TcParams& p = f.prob[i].meta.p;
    p.dep = j.dep; p.dep_mode = j.dep_mode; p.dep_k_blocks = j.dep_k_blocks;
    p.dep_need = kEpiWarps * f.prob[j.dep].meta.p.signal_x;  // every epilogue warp reports per tile
    p.dep_need_all = p.dep_need * f.prob[j.dep].meta.grid_y;
  }
  for (int i = n; i < kTcMaxFlow; ++i) f.prob[i] = f.prob[n - 1];   // never selected; keeps the parameter block defined
  f.total_tiles = total;
  f.ctrl = ctrl;
  f.rb_stride = (max_rows + kBM - 1) / kBM + 1;    // per product: one word per row block, then their total
  f.err = err;
  if (pair) {
    ctas &= ~1;                                            // whole pairs
    if (2 * total < ctas) ctas = 2 * total;
    return launch_flow<kStagesPair, 256, true>(f, ctas, st);
  }
  if (total < ctas) ctas = total;
  if (wide) return launch_flow<kStagesWide, 256, false>(f, ctas, st);
  return launch_flow<kStagesNarrow, 128, false>(f, ctas, st);
}

ss_status gemm_tc(int M, int N, int K, const Operand& A, const Operand& B, const Epilogue& ep, cudaStream_t st,
                  int k_splits, int64_t split_stride) {
  TcJob j;
  j.M = M; j.N = N; j.K = K; j.A = A; j.B = B; j.ep = ep; j.k_splits = k_splits; j.split_stride = split_stride;
  return gemm_tc_flow(&j, 1, nullptr, 0, 0, st);
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

int ss_mlp_set_flow_ctas(int ctas) { return ss::set_flow_ctas(ctas); }

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
