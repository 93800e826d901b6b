// Embedding-bag forward (sum pooling) and the deterministic backward fused with row-wise Adagrad.
//
// Forward: a group of G = D/4 lanes owns one bag; every lane keeps one float4 column slice of the
// pooled vector in registers and walks the bag's rows with 128-bit loads (rows are D*4 contiguous
// bytes, so a group reads whole rows, fully coalesced).  Row loads of four lookups are issued
// together so several gathers are in flight per lane.
//
// Backward: (1) keys t*N+row, (2) stable LSD radix sort of (key, position) with a hand-written
// histogram / scan / ranked-scatter pass per digit, (3) head flags + scan -> unique keys and segment
// offsets, (4) the sorted lookups are cut into windows of 16 consecutive positions; a lane group
// sums the gradients of each run of equal keys inside its window in position order.  A run that
// lies inside one window is final and is updated at once; a run that crosses a window edge leaves a
// partial sum, and a second kernel adds the partials of such a row in window order and updates it.
// Work per group is the same whatever the skew of the row distribution, and every sum has a fixed
// association, so results do not depend on scheduling.
#include "common.cuh"
#include "profile.cuh"

namespace ss {

// ======================================================================================
// forward
// ======================================================================================
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
  return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}

__device__ __forceinline__ uint2 bf16x4(float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  return r;
}

// G lanes per bag (power of two <= 32); NV float4 slices per lane (NV*G*4 >= D).
// Grid: x over the samples of a table (256 / G bags per block), y = table: no division finds (t, b), and all
// addressing inside a table is 32-bit (N * D / 4 < 2^32 is checked by the host).
template <int G, int NV>
__global__ void __launch_bounds__(256)
embbag_fwd_kernel(const float* __restrict__ tables, int T, uint32_t N, int D,
                  const int32_t* __restrict__ indices, const int32_t* __restrict__ offsets, int B,
                  float* __restrict__ out_f32, int64_t ld_f32,
                  __nv_bfloat16* __restrict__ out_bf16, int64_t ld_bf16, int col0,
                  int32_t* __restrict__ d_status) {
  const int b = blockIdx.x * (256 / G) + threadIdx.x / G;
  const int lane = threadIdx.x % G;
  const int t = blockIdx.y;
  if (b >= B) return;
  const int32_t* off = offsets + (int64_t)t * B + b;
  int lo = off[0], hi = off[1];
  // the index list ends where the last bag ends; a bag that is not inside [0, L] in ascending order is treated as empty
  const int L = __ldg(offsets + (int64_t)T * B);
  int bad = 0;
  if (lo < 0 || hi < lo || hi > L) { bad |= SS_DEV_BAD_OFFSET; lo = hi = 0; }
  const uint32_t nvec = (uint32_t)D >> 2;
  const float4* tab = reinterpret_cast<const float4*>(tables + (int64_t)t * N * D);

  float4 acc[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);

  // kRows lookups per round: their indices are loaded first, then their rows; a lookup beyond the bag's end or with
  // an index outside the table reads nothing and adds zeros.  Six rows (one float4 each) or four (two float4 each) in
  // flight per lane still fit 32 registers and were the fastest of 4 / 6 / 8 and 2 / 3 / 4.
  constexpr int kRows = NV >= 2 ? 4 : 6;
  for (int j = lo; j < hi; j += kRows) {
    uint32_t idx[kRows];
#pragma unroll
    for (int u = 0; u < kRows; ++u) idx[u] = (j + u < hi) ? (uint32_t)indices[j + u] : 0xffffffffu;
    float4 rowv[kRows][NV];
#pragma unroll
    for (int u = 0; u < kRows; ++u) {
      const bool ok = idx[u] < N;                            // one unsigned compare: negative indices are huge
      if (!ok && j + u < hi) bad |= SS_DEV_BAD_INDEX;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const uint32_t c = lane + v * G;
        rowv[u][v] = (ok && c < nvec) ? __ldg(tab + (idx[u] * nvec + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < kRows; ++u)      // lookups are added in bag order
#pragma unroll
      for (int v = 0; v < NV; ++v) acc[v] = add4(acc[v], rowv[u][v]);
  }

#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int c = lane + v * G;
    if (c < (int)nvec) {
      const int64_t col = (int64_t)col0 + (int64_t)t * D + 4 * c;
      if (out_f32) *reinterpret_cast<float4*>(out_f32 + (int64_t)b * ld_f32 + col) = acc[v];
      if (out_bf16) *reinterpret_cast<uint2*>(out_bf16 + (int64_t)b * ld_bf16 + col) = bf16x4(acc[v]);
    }
  }
  if (bad && d_status) atomicOr(d_status, bad);
}

template <int G, int NV>
static void launch_fwd(const float* tables, int T, int64_t N, int D, const int32_t* indices,
                       const int32_t* offsets, int B, float* out_f32, int64_t ld_f32, __nv_bfloat16* out_bf16,
                       int64_t ld_bf16, int col0, int32_t* d_status, cudaStream_t st) {
  // rows of 65..128 floats: two float4 per lane and 16 lanes per bag (measured faster than 32 lanes with one each;
  // for narrower rows the single-float4 form is the faster one)
  constexpr int FG = (NV == 1 && G == 32) ? 16 : G, FNV = (NV == 1 && G == 32) ? 2 : NV;
  const int per_block = 256 / FG;
  const dim3 blocks((unsigned)((B + per_block - 1) / per_block), (unsigned)T);
  { SS_TIMED("embbag_fwd_kernel", st);
  embbag_fwd_kernel<FG, FNV><<<blocks, 256, 0, st>>>(tables, T, (uint32_t)N, D, indices, offsets, B, out_f32, ld_f32,
                                                      out_bf16, ld_bf16, col0, d_status);
  }
}

// ======================================================================================
// backward: keys, radix sort, unique, windowed segment reduction, row-wise Adagrad
// ======================================================================================
constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kSortIPT = 16;                              // items per thread
constexpr int kSortTile = kSortThreads * kSortIPT;        // 4096 items per block
constexpr int kMaxBins = 512;
constexpr int kWin = 16;                                  // sorted positions per reduction window
constexpr int kScanThreads = 1024;

struct BwdPlan {
  int64_t L;
  int nblk;          // sort tiles
  int bits, passes, digit_bits, bins;
  int nwin;
  int nblk_u;        // blocks of the unique pass (1024 items each)
  size_t off_keys_a, off_keys_b, off_pos_a, off_pos_b, off_bag, off_hist, off_bintot, off_usum, off_uniq, off_seg,
      off_uidx, off_sbag, off_partial, off_long, off_gsum, off_scalars, total;
};

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static BwdPlan make_plan(int T, int64_t N, int D, int64_t L) {
  BwdPlan p{};
  p.L = L;
  p.nblk = (int)((L + kSortTile - 1) / kSortTile);
  if (p.nblk < 1) p.nblk = 1;
  const uint64_t maxkey = (uint64_t)T * (uint64_t)N;     // sentinel for skipped lookups
  p.bits = 1;
  while ((maxkey >> p.bits) != 0) ++p.bits;
  p.passes = (p.bits + 8) / 9;
  p.digit_bits = (p.bits + p.passes - 1) / p.passes;
  p.bins = 1 << p.digit_bits;
  p.nwin = (int)((L + kWin - 1) / kWin);
  if (p.nwin < 1) p.nwin = 1;
  p.nblk_u = (int)((L + kScanThreads - 1) / kScanThreads);
  if (p.nblk_u < 1) p.nblk_u = 1;
  size_t o = 0;
  const size_t l4 = align256((size_t)(L > 0 ? L : 1) * 4);
  p.off_keys_a = o; o += l4;
  p.off_keys_b = o; o += l4;
  p.off_pos_a = o; o += l4;
  p.off_pos_b = o; o += l4;
  p.off_bag = o; o += l4;
  p.off_hist = o; o += align256((size_t)p.nblk * p.bins * 4);
  p.off_bintot = o; o += align256((size_t)kMaxBins * 4);
  p.off_usum = o; o += align256((size_t)(p.nblk_u + 1) * 4);
  p.off_uniq = o; o += l4;
  p.off_seg = o; o += align256((size_t)(L + 1) * 4);
  p.off_uidx = o; o += l4;
  p.off_sbag = o; o += l4;
  p.off_partial = o; o += align256((size_t)p.nwin * 2 * (size_t)D * 4);
  p.off_long = o; o += align256((size_t)p.nwin * 4);
  const uint64_t umax = (uint64_t)L < maxkey ? (uint64_t)L : maxkey;   // distinct rows cannot exceed either
  p.off_gsum = o; o += align256((size_t)(umax > 0 ? umax : 1) * (size_t)D * 4);
  p.off_scalars = o; o += 256;
  p.total = o;
  return p;
}

// ---- (1) keys ---------------------------------------------------------------------------
// One thread per bag: key = t*N + row for each of its lookups, and the bag id of each position.
// Every position in [0, L) is written by somebody: a bag owns [lo, hi) with both ends clamped to
// [0, L] (consecutive bags share an end, so the clamped ranges tile [clamp(off[0]), clamp(off[T*B])) even
// when the offsets are not monotone), the first and the last bag also take what lies before and after.
// Positions of a malformed bag, and lookups with a row index outside the table, get the sentinel key.
__device__ __forceinline__ void build_keys_block(int blk, const int32_t* __restrict__ indices,
                                                 const int32_t* __restrict__ offsets, int T, int64_t N, int B, int64_t L,
                                                 uint32_t* __restrict__ keys, int32_t* __restrict__ bag_of,
                                                 int32_t* __restrict__ d_status) {
  const int64_t bag = (int64_t)blk * 256 + threadIdx.x;
  const int64_t nbags = (int64_t)T * B;
  if (bag >= nbags) return;
  const uint32_t sentinel = (uint32_t)((uint64_t)T * (uint64_t)N);
  const int t = (int)(bag / B);
  const int lo = offsets[bag], hi = offsets[bag + 1];
  const int64_t clo = lo < 0 ? 0 : (lo > L ? L : lo), chi = hi < 0 ? 0 : (hi > L ? L : hi);
  const bool well_formed = (lo == clo) && (hi == chi) && (lo <= hi);
  int bad = well_formed ? 0 : SS_DEV_BAD_OFFSET;
  for (int64_t j = clo; j < chi; ++j) {
    uint32_t key = sentinel;
    if (well_formed) {
      const int idx = indices[j];
      if (idx >= 0 && idx < N) key = (uint32_t)((uint64_t)t * (uint64_t)N + (uint64_t)idx);
      else bad |= SS_DEV_BAD_INDEX;
    }
    keys[j] = key;
    bag_of[j] = (int32_t)bag;
  }
  if (bag == 0) {
    if (lo != 0) bad |= SS_DEV_BAD_OFFSET;
    for (int64_t j = 0; j < clo; ++j) { keys[j] = sentinel; bag_of[j] = 0; }
  }
  if (bag == nbags - 1) {
    if (hi != L) bad |= SS_DEV_BAD_OFFSET;
    for (int64_t j = chi; j < L; ++j) { keys[j] = sentinel; bag_of[j] = 0; }
  }
  if (bad && d_status) atomicOr(d_status, bad);
}

__global__ void __launch_bounds__(256)
build_keys_kernel(const int32_t* __restrict__ indices, const int32_t* __restrict__ offsets, int T, int64_t N,
                  int B, int64_t L, uint32_t* __restrict__ keys, int32_t* __restrict__ bag_of,
                  int32_t* __restrict__ d_status, const int32_t* __restrict__ run_if) {
  if (run_if && *run_if == 0) return;                     // the per-table sort already produced the result
  build_keys_block(blockIdx.x, indices, offsets, T, N, B, L, keys, bag_of, d_status);
}

// ---- (2) radix sort pass ----------------------------------------------------------------
// Lanes of the warp that hold the same digit, from one ballot per digit bit (cost independent of how many
// distinct digits the warp holds).  `digit` is below 2^nbits, or exactly 2^nbits for a lane past the end.
__device__ __forceinline__ uint32_t same_digit_lanes(uint32_t digit, int nbits) {
  uint32_t peers = 0xffffffffu;
  for (int b = 0; b <= nbits; ++b) {
    const bool bit = (digit >> b) & 1u;
    const uint32_t m = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? m : ~m;
  }
  return peers;
}

// hist[bin * nblk + blk] = number of keys of tile blk whose digit is bin.  Lanes holding the same
// digit are counted together, so a hot row does not serialise on one counter.
// Reads of data that other blocks of the same launch may have written (the single-launch form below) bypass L1.
__device__ __forceinline__ void sort_hist_block(int blk, uint32_t* cnt /*shared, kMaxBins*/, const uint32_t* keys, int64_t L,
                                                int shift, int bins, int nblk, uint32_t* hist) {
  for (int i = threadIdx.x; i < bins; i += kSortThreads) cnt[i] = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const int64_t base = (int64_t)blk * kSortTile;
  const uint32_t mask = (uint32_t)bins - 1u;
  const int nbits = 31 - __clz(bins);
  uint32_t digit[kSortIPT];
#pragma unroll
  for (int k = 0; k < kSortIPT; ++k) {                      // all loads first, then the counting
    const int64_t i = base + (int64_t)k * kSortThreads + threadIdx.x;
    digit[k] = (i < L) ? ((__ldcg(keys + i) >> shift) & mask) : (uint32_t)bins;
  }
#pragma unroll
  for (int k = 0; k < kSortIPT; ++k) {
    const uint32_t peers = same_digit_lanes(digit[k], nbits);
    if (digit[k] < (uint32_t)bins && lane == (__ffs(peers) - 1))
      atomicAdd(&cnt[digit[k]], (uint32_t)__popc(peers));   // integer counts: order-free
  }
  __syncthreads();
  for (int i = threadIdx.x; i < bins; i += kSortThreads) hist[(int64_t)i * nblk + blk] = cnt[i];
}

__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const uint32_t* __restrict__ keys, int64_t L, int shift, int bins, int nblk,
                 uint32_t* __restrict__ hist, const int32_t* __restrict__ run_if) {
  __shared__ uint32_t cnt[kMaxBins];
  if (run_if && *run_if == 0) return;
  sort_hist_block(blockIdx.x, cnt, keys, L, shift, bins, nblk, hist);
}

// One warp per bin: exclusive scan of that bin's per-tile counts in place, bin total to bintot[bin].
__device__ __forceinline__ void bin_scan_block(int blk, uint32_t* hist, int bins, int nblk, uint32_t* bintot) {
  const int bin = blk * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (bin >= bins) return;
  uint32_t* row = hist + (int64_t)bin * nblk;
  uint32_t carry = 0;
  for (int b0 = 0; b0 < nblk; b0 += 32) {
    const int b = b0 + lane;
    const uint32_t v = (b < nblk) ? __ldcg(row + b) : 0u;
    uint32_t inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, inc, off);
      if (lane >= off) inc += n;
    }
    if (b < nblk) row[b] = carry + inc - v;
    carry += __shfl_sync(0xffffffffu, inc, 31);
  }
  if (lane == 0) bintot[bin] = carry;
}

__global__ void __launch_bounds__(256)
bin_scan_kernel(uint32_t* __restrict__ hist, int bins, int nblk, uint32_t* __restrict__ bintot,
                const int32_t* __restrict__ run_if) {
  if (run_if && *run_if == 0) return;
  bin_scan_block(blockIdx.x, hist, bins, nblk, bintot);
}

// Exclusive scan of m values in place by one block (m is a few thousand at most).
// scalars[2..3] stamp the workspace with the problem it holds a finished sort of; the reduction kernels
// refuse a workspace whose stamp does not match their arguments.
__device__ __forceinline__ int32_t ws_stamp(uint32_t sentinel) { return (int32_t)(sentinel ^ 0x53484144u); }

struct UniqueFinish {      // what the scan of the per-block head counts also writes when it closes the unique pass
  int32_t* seg; int32_t* seg_out; int32_t* d_num_unique; int32_t* scalars;
  int64_t L; uint32_t sentinel;
};

// U distinct keys: close the segment list when there is none, publish U, stamp the workspace.
__device__ __forceinline__ void finish_unique(uint32_t U, const UniqueFinish& f) {
  if (U == 0) { f.seg[0] = 0; if (f.seg_out) f.seg_out[0] = 0; }
  if (f.d_num_unique) *f.d_num_unique = (int32_t)U;
  f.scalars[0] = (int32_t)U;
  f.scalars[1] = 0;                                        // rows whose run crosses a window edge (filled by the window kernel)
  f.scalars[2] = (int32_t)f.L;
  f.scalars[3] = ws_stamp(f.sentinel);
}

__global__ void __launch_bounds__(kScanThreads)
scan_exclusive_kernel(uint32_t* __restrict__ data, int64_t m, uint32_t* __restrict__ total_out, UniqueFinish fin) {
  __shared__ uint32_t part[kScanThreads];
  const int64_t chunk = (m + kScanThreads - 1) / kScanThreads;
  const int64_t lo = (int64_t)threadIdx.x * chunk;
  const int64_t hi = (lo + chunk < m) ? lo + chunk : m;
  uint32_t s = 0;
  for (int64_t i = lo; i < hi; ++i) s += data[i];
  part[threadIdx.x] = s;
  __syncthreads();
  for (int off = 1; off < kScanThreads; off <<= 1) {     // Hillis-Steele inclusive scan of the partials
    uint32_t v = (threadIdx.x >= off) ? part[threadIdx.x - off] : 0u;
    __syncthreads();
    part[threadIdx.x] += v;
    __syncthreads();
  }
  uint32_t run = (threadIdx.x == 0) ? 0u : part[threadIdx.x - 1];
  for (int64_t i = lo; i < hi; ++i) {
    const uint32_t v = data[i];
    data[i] = run;
    run += v;
  }
  if (total_out && threadIdx.x == kScanThreads - 1) *total_out = part[kScanThreads - 1];
  if (fin.scalars && threadIdx.x == kScanThreads - 1) finish_unique(part[kScanThreads - 1], fin);
}

// Stable scatter: warp w of the block owns the contiguous items [w*512, (w+1)*512) of the tile and
// walks them 32 at a time; rank inside a round comes from the lanes holding the same digit, across rounds and warps from
// per-warp running counters that start at (bins before this digit) + (this digit in earlier tiles).
__device__ __forceinline__ void sort_scatter_block(int blk, uint32_t* cnt /*shared: [kSortWarps][bins], binbase[bins], wtot[8]*/,
                                                   const uint32_t* keys_in, const int32_t* pos_in, uint32_t* keys_out,
                                                   int32_t* pos_out, int64_t L, int shift, int bins, int nblk,
                                                   const uint32_t* hist_scanned, const uint32_t* bintot) {
  uint32_t* binbase = cnt + kSortWarps * bins;
  uint32_t* wtot = binbase + bins;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < kSortWarps * bins; i += kSortThreads) cnt[i] = 0;
  // exclusive scan of the bin totals (bins <= 512 = 2 per thread)
  {
    const int i0 = 2 * threadIdx.x, i1 = i0 + 1;
    const uint32_t v0 = (i0 < bins) ? __ldcg(bintot + i0) : 0u, v1 = (i1 < bins) ? __ldcg(bintot + i1) : 0u;
    uint32_t inc = v0 + v1;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, inc, off);
      if (lane >= off) inc += n;
    }
    if (lane == 31) wtot[warp] = inc;
    __syncthreads();
    uint32_t wbase = 0;
    for (int w = 0; w < warp; ++w) wbase += wtot[w];
    const uint32_t excl = wbase + inc - (v0 + v1);
    if (i0 < bins) binbase[i0] = excl;
    if (i1 < bins) binbase[i1] = excl + v0;
  }
  __syncthreads();
  const uint32_t mask = (uint32_t)bins - 1u;
  const int nbits = 31 - __clz(bins);
  const int64_t wbase = (int64_t)blk * kSortTile + (int64_t)warp * (32 * kSortIPT);
  uint32_t key[kSortIPT];
  uint32_t* mycnt = cnt + warp * bins;
#pragma unroll
  for (int k = 0; k < kSortIPT; ++k) {
    const int64_t i = wbase + k * 32 + lane;
    const bool valid = i < L;
    key[k] = valid ? __ldcg(keys_in + i) : 0u;
    const uint32_t digit = valid ? ((key[k] >> shift) & mask) : (uint32_t)bins;   // invalid lanes pair up apart
    const uint32_t peers = same_digit_lanes(digit, nbits);
    if (valid && lane == (__ffs(peers) - 1)) mycnt[digit] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  for (int bin = threadIdx.x; bin < bins; bin += kSortThreads) {
    uint32_t run = binbase[bin] + __ldcg(hist_scanned + (int64_t)bin * nblk + blk);
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
      const uint32_t c = cnt[w * bins + bin];
      cnt[w * bins + bin] = run;
      run += c;
    }
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < kSortIPT; ++k) {
    const int64_t i = wbase + k * 32 + lane;
    const bool valid = i < L;
    const uint32_t digit = valid ? ((key[k] >> shift) & mask) : (uint32_t)bins;
    const uint32_t peers = same_digit_lanes(digit, nbits);
    uint32_t dst = 0;
    if (valid) dst = mycnt[digit] + __popc(peers & ((1u << lane) - 1u));
    __syncwarp();
    if (valid && lane == (__ffs(peers) - 1)) mycnt[digit] += __popc(peers);
    __syncwarp();
    if (valid) {
      keys_out[dst] = key[k];
      pos_out[dst] = pos_in ? __ldcg(pos_in + i) : (int32_t)i;
    }
  }
}

__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* __restrict__ keys_in, const int32_t* __restrict__ pos_in,
                    uint32_t* __restrict__ keys_out, int32_t* __restrict__ pos_out, int64_t L, int shift,
                    int bins, int nblk, const uint32_t* __restrict__ hist_scanned, const uint32_t* __restrict__ bintot,
                    const int32_t* __restrict__ run_if) {
  extern __shared__ uint32_t cnt[];                       // [kSortWarps][bins], then binbase[bins], wtot[8]
  if (run_if && *run_if == 0) return;
  sort_scatter_block(blockIdx.x, cnt, keys_in, pos_in, keys_out, pos_out, L, shift, bins, nblk, hist_scanned, bintot);
}

// ---- (2a) the tiled sort as ONE launch -------------------------------------------------------
// Work items -- key building per 256 bags, then per digit pass: a histogram per tile, a scan per 8 bins, a ranked
// scatter per tile -- are numbered in that order and drawn by the blocks from a counter.  An item of one phase needs
// every item of the phases before it; it waits until that many items have been reported complete.  The items it
// waits for have lower numbers, so they were drawn earlier by blocks that are running: the wait ends however few
// blocks the device keeps resident.  run_if (nullable): the launch does nothing when the word it points to is zero
// (the per-table sort has produced the result).  ctl = {next item, items complete, blocks gone}, zero at launch and
// left zero.  The wait is bounded (about a second); when it runs out the block reports SS_DEV_BAD_WORKSPACE and leaves.
struct TiledSort {
  const int32_t* indices; const int32_t* offsets;
  int T, B; int64_t N, L;
  uint32_t *keys_a, *keys_b; int32_t *pos_a, *pos_b, *bag_of;
  uint32_t *hist, *bintot;
  int32_t* d_status; const int32_t* run_if; int* ctl;
  int passes, digit_bits, bins, nblk, n_key_items, n_scan_items;
};

__global__ void __launch_bounds__(kSortThreads)
tiled_sort_kernel(const TiledSort a) {
  __shared__ uint32_t smem[kSortWarps * kMaxBins + kMaxBins + 8];
  __shared__ int s_item;
  if (a.run_if && *a.run_if == 0) return;
  const int per_pass = 2 * a.nblk + a.n_scan_items;
  const int total = a.n_key_items + a.passes * per_pass;
  for (;;) {
    __syncthreads();                                       // the previous item's shared memory is no longer in use
    if (threadIdx.x == 0) s_item = atomicAdd(a.ctl, 1);
    __syncthreads();
    const int item = s_item;
    if (item >= total) break;
    // phase of the item, and how many items precede that phase
    int need = 0, pass = -1, phase = 0, idx = item;
    if (item >= a.n_key_items) {
      const int r = item - a.n_key_items;
      pass = r / per_pass;
      idx = r - pass * per_pass;
      need = a.n_key_items + pass * per_pass;
      if (idx >= a.nblk) { idx -= a.nblk; need += a.nblk; phase = 1; }
      if (phase == 1 && idx >= a.n_scan_items) { idx -= a.n_scan_items; need += a.n_scan_items; phase = 2; }
    }
    if (threadIdx.x == 0 && need > 0) {
      const long long t0 = clock64();
      int seen;
      do {
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(a.ctl + 1) : "memory");
        if (seen < need && clock64() - t0 > 2000000000ll) { s_item = -1; break; }
      } while (seen < need);
    }
    __syncthreads();
    if (s_item < 0) {                                      // gave up: report, and do not touch the item
      if (threadIdx.x == 0 && a.d_status) atomicOr(a.d_status, SS_DEV_BAD_WORKSPACE);
      break;
    }
    // buffers of this pass: pass 0 reads keys_a (positions = indices), every pass swaps
    const uint32_t* kin = (pass & 1) ? a.keys_b : a.keys_a;
    uint32_t* kout = (pass & 1) ? a.keys_a : a.keys_b;
    const int32_t* pin = pass <= 0 ? nullptr : ((pass & 1) ? a.pos_b : a.pos_a);
    int32_t* pout = (pass & 1) ? a.pos_a : a.pos_b;
    const int shift = pass * a.digit_bits;
    if (pass < 0) build_keys_block(idx, a.indices, a.offsets, a.T, a.N, a.B, a.L, a.keys_a, a.bag_of, a.d_status);
    else if (phase == 0) sort_hist_block(idx, smem, kin, a.L, shift, a.bins, a.nblk, a.hist);
    else if (phase == 1) bin_scan_block(idx, a.hist, a.bins, a.nblk, a.bintot);
    else sort_scatter_block(idx, smem, kin, pin, kout, pout, a.L, shift, a.bins, a.nblk, a.hist, a.bintot);
    __threadfence();                                       // this thread's stores, before the item is reported
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(a.ctl + 1, 1);
  }
  // the last block to leave clears the control words for the next launch
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(a.ctl + 2, 1) == (int)gridDim.x - 1) { a.ctl[0] = 0; a.ctl[1] = 0; a.ctl[2] = 0; __threadfence(); }
  }
}

// ---- (2b) per-table sort in shared memory -------------------------------------------------
// The lookups arrive grouped by table (bags are table-major), so the sort by key = t*N + row is T
// independent sorts by row.  One block per table keeps the table's row ids and a 16-bit position payload
// in shared memory and runs the stable LSD passes there: no global histogram, no scan launches, and only
// T of the SMs are busy while the other streams use the rest.  The result is the same unique stable
// order the tiled passes produce.  A block that cannot take this path (more than kTsCap lookups in its
// table, offsets that are not monotone within [0, L], a row index outside the table) raises *fallback
// and the tiled passes, launched after this kernel, run; otherwise they return at once.
constexpr int kTsThreads = 1024;
constexpr int kTsWarps = kTsThreads / 32;
constexpr int kTsCap = SS_TABLE_SORT_CAP;                  // lookups of one table (24576)
constexpr int kTsMaxBins = 256;
constexpr size_t kTsSmem = (size_t)kTsCap * 8 + (size_t)kTsWarps * kTsMaxBins * 4;   // 229,376 bytes

template <int NB>
__device__ __forceinline__ uint32_t same_digit_lanes_n(uint32_t digit) {
  uint32_t peers = 0xffffffffu;
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    const bool bit = (digit >> b) & 1u;
    const uint32_t m = __ballot_sync(0xffffffffu, bit);
    peers &= bit ? m : ~m;
  }
  return peers;
}

template <int NB>                                          // digit bits, 5..8
__global__ void __launch_bounds__(kTsThreads, 1)
table_sort_kernel(const int32_t* __restrict__ indices, const int32_t* __restrict__ offsets, int T, int64_t N, int B,
                  int64_t L, int passes, uint32_t* __restrict__ keys_out, int32_t* __restrict__ perm_out,
                  int32_t* __restrict__ bag_of, int32_t* __restrict__ fallback) {
  extern __shared__ __align__(16) unsigned char ts_smem[];
  uint32_t* okey = reinterpret_cast<uint32_t*>(ts_smem);              // row id of local position i
  uint16_t* pa = reinterpret_cast<uint16_t*>(okey + kTsCap);          // payload ping
  uint16_t* pb = pa + kTsCap;                                         // payload pong
  uint32_t* cnt = reinterpret_cast<uint32_t*>(pb + kTsCap);           // [kTsWarps][bins]
  __shared__ uint32_t wtot[kTsWarps];
  constexpr int bins = 1 << NB;
  constexpr uint32_t mask = (uint32_t)bins - 1u;
  const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t bag0 = (int64_t)t * B;
  const int seg0 = offsets[bag0], seg1 = offsets[bag0 + B];
  // block-uniform checks of the table's segment
  if (seg0 < 0 || seg1 < seg0 || (int64_t)seg1 > L || seg1 - seg0 > kTsCap || (t == 0 && seg0 != 0) ||
      (t == T - 1 && (int64_t)seg1 != L)) {
    if (tid == 0) atomicOr(fallback, 1);
    return;
  }
  const int n = seg1 - seg0;
  const int n32 = (n + 31) & ~31;                          // padded to whole rounds (kTsCap is a multiple of 32)
  // bag of every local position (16 bits: B <= 65536 is checked by the host), parked in the pong array
  int bad = 0;
  for (int b = tid; b < B; b += kTsThreads) {
    const int lo = offsets[bag0 + b], hi = offsets[bag0 + b + 1];
    if (lo < seg0 || hi < lo || hi > seg1) { bad = 1; continue; }
    for (int j = lo; j < hi; ++j) pb[j - seg0] = (uint16_t)b;
  }
  if (__syncthreads_or(bad)) {
    if (tid == 0) atomicOr(fallback, 1);
    return;
  }
  // pad items carry the largest key and the highest positions, so every stable pass leaves them at the end
#pragma unroll 4
  for (int i = tid; i < n32; i += kTsThreads) {
    uint32_t row = 0xffffffffu;
    if (i < n) {
      const int idx = indices[seg0 + i];
      if (idx < 0 || (int64_t)idx >= N) bad = 1;
      row = (uint32_t)idx;
      bag_of[seg0 + i] = (int32_t)(bag0 + pb[i]);
    }
    okey[i] = row;
    pa[i] = (uint16_t)i;
  }
  if (__syncthreads_or(bad)) {
    if (tid == 0) atomicOr(fallback, 1);
    return;
  }
  const int rounds = (n32 + kTsThreads - 1) / kTsThreads;  // rounds of 32 consecutive items per warp
  const int w0 = warp * rounds * 32;                       // warp w owns items [w0, w0 + 32*rounds)
  const int wend = min(w0 + rounds * 32, n32);
  uint32_t* mycnt = cnt + warp * bins;
  uint16_t* src = pa;
  uint16_t* dst = pb;
  for (int pass = 0; pass < passes; ++pass) {
    const int shift = pass * NB;
    for (int i = tid; i < kTsWarps * bins; i += kTsThreads) cnt[i] = 0;
    __syncthreads();
    // counts per (warp, digit): warp-private counters, equal digits inside a round resolved by the atomic unit
    for (int i = w0 + lane; i < wend; i += 32) atomicAdd(&mycnt[(okey[src[i]] >> shift) & mask], 1u);
    __syncthreads();
    // exclusive scan in (digit, warp) order: thread tid owns q = bins/32 consecutive entries of that order
    {
      constexpr int q = bins >> 5;
      uint32_t c[q];
      uint32_t sum = 0;
#pragma unroll
      for (int u = 0; u < q; ++u) {
        const int e = tid * q + u;
        c[u] = cnt[(e & 31) * bins + (e >> 5)];
        sum += c[u];
      }
      uint32_t inc = sum;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += v;
      }
      if (lane == 31) wtot[warp] = inc;
      __syncthreads();
      if (warp == 0) {
        uint32_t v = wtot[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t u = __shfl_up_sync(0xffffffffu, v, off);
          if (lane >= off) v += u;
        }
        wtot[lane] = v;                                    // inclusive over warps
      }
      __syncthreads();
      uint32_t run = (warp ? wtot[warp - 1] : 0u) + inc - sum;
#pragma unroll
      for (int u = 0; u < q; ++u) {
        const int e = tid * q + u;
        cnt[(e & 31) * bins + (e >> 5)] = run;
        run += c[u];
      }
    }
    __syncthreads();
    // stable scatter: rank inside a round from the lanes holding the same digit, across rounds from the counter
    for (int i = w0 + lane; i < wend; i += 32) {           // whole rounds: the bound is the same for all lanes
      const uint32_t pay = src[i];
      const uint32_t digit = (okey[pay] >> shift) & mask;
      const uint32_t peers = same_digit_lanes_n<NB>(digit);
      const uint32_t below = peers & ((1u << lane) - 1u);
      const uint32_t base = mycnt[digit];
      __syncwarp();
      if (below == 0) mycnt[digit] = base + __popc(peers);
      __syncwarp();
      dst[base + __popc(below)] = (uint16_t)pay;
    }
    __syncthreads();
    uint16_t* sw = src; src = dst; dst = sw;
  }
  const uint32_t key0 = (uint32_t)((uint64_t)t * (uint64_t)N);
  for (int j = tid; j < n; j += kTsThreads) {
    const int pay = src[j];
    keys_out[seg0 + j] = key0 + okey[pay];
    perm_out[seg0 + j] = seg0 + pay;
  }
}

// ---- (3) unique -------------------------------------------------------------------------
__device__ __forceinline__ bool is_head(const uint32_t* keys, int64_t i, uint32_t sentinel) {
  const uint32_t k = keys[i];
  return k < sentinel && (i == 0 || keys[i - 1] != k);
}

__global__ void __launch_bounds__(kScanThreads)
unique_count_kernel(const uint32_t* __restrict__ keys, int64_t L, uint32_t sentinel, uint32_t* __restrict__ usum) {
  const int64_t i = (int64_t)blockIdx.x * kScanThreads + threadIdx.x;
  const int h = (i < L) && is_head(keys, i, sentinel);
  const int c = __syncthreads_count(h);
  if (threadIdx.x == 0) usum[blockIdx.x] = (uint32_t)c;
}

// uniq[u], seg[u] at the head of every segment; uidx[i] = segment of sorted position i; sbag[i] = its bag.
__global__ void __launch_bounds__(kScanThreads)
unique_write_kernel(const uint32_t* __restrict__ keys, int64_t L, uint32_t sentinel,
                    const uint32_t* __restrict__ ubase, int32_t* __restrict__ uniq, int32_t* __restrict__ seg,
                    int32_t* __restrict__ uidx, int32_t* __restrict__ uniq_out, int32_t* __restrict__ seg_out,
                    const int32_t* __restrict__ perm, const int32_t* __restrict__ bag_of, int32_t* __restrict__ sbag) {
  __shared__ uint32_t wsum[32];
  const int64_t i = (int64_t)blockIdx.x * kScanThreads + threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool in = i < L;
  const uint32_t k = in ? keys[i] : sentinel;
  const bool h = in && k < sentinel && (i == 0 || keys[i - 1] != k);
  const uint32_t ballot = __ballot_sync(0xffffffffu, h);
  if (lane == 0) wsum[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    uint32_t v = wsum[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const uint32_t n = __shfl_up_sync(0xffffffffu, v, off);
      if (lane >= off) v += n;
    }
    wsum[lane] = v;                                        // inclusive over warps
  }
  __syncthreads();
  const uint32_t before = ubase[blockIdx.x] + (warp ? wsum[warp - 1] : 0u) + __popc(ballot & ((1u << lane) - 1u));
  if (h) {
    uniq[before] = (int32_t)k;
    seg[before] = (int32_t)i;
    if (uniq_out) uniq_out[before] = (int32_t)k;
    if (seg_out) seg_out[before] = (int32_t)i;
  }
  if (in) uidx[i] = (int32_t)(before + (h ? 1u : 0u)) - 1;
  // bag of every sorted position, so that the reduction reads it with one coalesced load
  if (in && sbag) {
    const int pj = perm[i];
    sbag[i] = (pj >= 0 && pj < L) ? bag_of[pj] : -1;
  }
  // the last valid position closes the last segment: seg[U] = number of valid lookups
  if (in && k < sentinel && (i == L - 1 || keys[i + 1] >= sentinel)) {
    const uint32_t u_end = before + (h ? 1u : 0u);
    seg[u_end] = (int32_t)(i + 1);
    if (seg_out) seg_out[u_end] = (int32_t)(i + 1);
  }
}

__global__ void unique_finish_kernel(const uint32_t* __restrict__ total, int32_t* __restrict__ seg,
                                     int32_t* __restrict__ seg_out, int32_t* __restrict__ d_num_unique,
                                     int32_t* __restrict__ scalars, int64_t L, uint32_t sentinel) {
  const uint32_t U = total ? *total : 0u;
  if (U == 0) { seg[0] = 0; if (seg_out) seg_out[0] = 0; }
  if (d_num_unique) *d_num_unique = (int32_t)U;
  scalars[0] = (int32_t)U;
  scalars[1] = 0;                                          // rows whose run crosses a window edge (filled by the window kernel)
  scalars[2] = (int32_t)L;
  scalars[3] = ws_stamp(sentinel);
}

__device__ __forceinline__ bool ws_matches(const int32_t* scalars, int64_t L, uint32_t sentinel, int32_t* d_status) {
  if (scalars[2] == (int32_t)L && scalars[3] == ws_stamp(sentinel)) return true;
  if (d_status && threadIdx.x == 0 && blockIdx.x == 0) atomicOr(d_status, SS_DEV_BAD_WORKSPACE);
  return false;
}

// ---- (4) windowed segment reduction ---------------------------------------------------------
// A lane group owns a window of kWin consecutive sorted positions and adds the gradient rows of each
// run of equal keys in position order.  A run that lies inside the window is complete: its sum goes
// to gsum[u].  A run that crosses a window edge leaves a partial sum in the window's slot 0 (run
// covers the window's first position) or slot 1.  This kernel serves rows wider than 128 floats (several
// float4 per lane); narrower rows take window_apply_kernel, which also updates the rows.
template <int G, int NV>
__global__ void __launch_bounds__(256)
window_reduce_kernel(const uint32_t* __restrict__ keys, const int32_t* __restrict__ sbag,
                     const int32_t* __restrict__ uidx, int64_t L,
                     uint32_t sentinel, int64_t N, int D, int B, const float* __restrict__ grad, int64_t ld_grad,
                     int col0, float* __restrict__ gsum, float* __restrict__ partial, int32_t* __restrict__ long_list,
                     int32_t* __restrict__ scalars, int nwin, int64_t umax, int32_t* __restrict__ d_status) {
  constexpr int kGroups = 256 / G;
  __shared__ uint32_t s_key[kGroups][kWin + 2];            // [0] = key before the window, [kWin+1] = key after
  __shared__ int32_t s_row[kGroups][kWin];                 // float4 index of the lookup's gradient row
  __shared__ int32_t s_u[kGroups][kWin];
  const int grp = threadIdx.x / G, lane = threadIdx.x % G;
  const int64_t win = (int64_t)blockIdx.x * kGroups + grp;
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) / G * G));
  if (!ws_matches(scalars, L, sentinel, d_status)) return;
  if (win >= nwin) return;
  const int64_t w0 = win * kWin;
  const int nvec = D >> 2;
  const int64_t ld4 = ld_grad >> 2;
  // keys (one before and one after the window included), bag and segment of every position: one round of loads
  for (int i = lane; i < kWin + 2; i += G) {
    const int64_t j = w0 - 1 + i;
    const bool in_range = j >= 0 && j < L;
    const bool body = i >= 1 && i <= kWin;
    uint32_t key = in_range ? keys[j] : sentinel;
    const int sb = (body && in_range) ? sbag[j] : 0;
    const int u = (body && in_range) ? uidx[j] : 0;
    int32_t row = -1;
    if (body && key < sentinel) {
      const int t = (int)((uint32_t)sb / (uint32_t)B);     // bags are table-major: bag = t*B + b (32-bit division)
      const int b = sb - t * B;
      // a consistent workspace never fails these; an inconsistent one must not turn into a wild access
      if (sb >= 0 && (int64_t)key >= (int64_t)t * N && (int64_t)key < (int64_t)(t + 1) * N && u >= 0 && u < umax)
        row = (int32_t)((int64_t)b * ld4 + (int64_t)t * nvec);   // B * ld_grad / 4 < 2^31 is checked on the host
      else
        key = sentinel;
    }
    s_key[grp][i] = key;
    if (body) { s_row[grp][i - 1] = row; s_u[grp][i - 1] = u; }
  }
  __syncwarp(gmask);
  const float4* grad4 = reinterpret_cast<const float4*>(grad + col0);  // col0 is a multiple of 4

  float4 acc[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  int run_start = 0;
  constexpr int kBatch = NV >= 8 ? 1 : (NV >= 4 ? 2 : (NV >= 2 ? 4 : 8));   // gradient rows in flight per lane
  for (int i0 = 0; i0 < kWin; i0 += kBatch) {
    float4 gv[kBatch][NV];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int32_t row = s_row[grp][i0 + u];
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int c = lane + v * G;
        gv[u][v] = (row >= 0 && c < nvec) ? __ldg(grad4 + row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int i = i0 + u;
      const uint32_t key = s_key[grp][1 + i];
      if (key >= sentinel) continue;                       // skipped lookups sort last; nothing follows them
#pragma unroll
      for (int v = 0; v < NV; ++v) acc[v] = add4(acc[v], gv[u][v]);
      const uint32_t next = s_key[grp][2 + i];
      if (next != key || i == kWin - 1) {
        const bool head_open = (run_start == 0) && (s_key[grp][0] == key);
        const bool tail_open = (next == key);              // only possible at the window's last position
        const bool complete = !head_open && !tail_open;
        float4* dst = complete ? reinterpret_cast<float4*>(gsum + (int64_t)s_u[grp][i] * D)
                               : reinterpret_cast<float4*>(partial + ((int64_t)win * 2 + (run_start == 0 ? 0 : 1)) * D);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
          const int c = lane + v * G;
          if (c < nvec) dst[c] = acc[v];
          acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        // the window in which a multi-window run starts enters the row in the list of rows to combine
        if (!head_open && tail_open && lane == 0) {
          const int slot = atomicAdd(&scalars[1], 1);
          if (slot < nwin) long_list[slot] = s_u[grp][i];   // at most one such run per window
        }
        run_start = i + 1;
      }
    }
  }
}

template <int G>
__device__ __forceinline__ void adagrad_one_row(float4 g, uint32_t key, int lane, int nvec, int D, unsigned gmask,
                                                float* __restrict__ tables, float* __restrict__ row_state, float lr,
                                                float eps);

__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// ---- (4b) fused window kernel for rows of at most 4G floats ------------------------------------
// Same windows, same order of additions and same outputs as window_reduce_kernel<G, 1, true>.  The run
// structure of the window is three 16-bit masks (valid, head, tail) built once from the keys; while the
// keys are looked at, the table rows of the window's runs are requested into L2, so that when a run ends
// its row is updated on the spot from the sum in the lanes' registers.  No shared-memory stash: the number
// of windows in flight on an SM is bounded by registers only.
constexpr int kWaThreads = 128;

// Row-wise Adagrad on one row whose gradient is in the lanes' registers, NV float4 per lane (column lane + v*G).
template <int G, int NV>
__device__ __forceinline__ void adagrad_row_nv(const float4 (&g)[NV], uint32_t key, int lane, int nvec, int D,
                                               unsigned gmask, float* __restrict__ tables,
                                               float* __restrict__ row_state, float lr, float eps) {
  float4* row = reinterpret_cast<float4*>(tables + (int64_t)key * D);
  float4 r[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) r[v] = (lane + v * G < nvec) ? row[lane + v * G] : make_float4(0.f, 0.f, 0.f, 0.f);
  const float st = row_state[key];
  float ss = 0.f;
#pragma unroll
  for (int v = 0; v < NV; ++v) ss += g[v].x * g[v].x + g[v].y * g[v].y + g[v].z * g[v].z + g[v].w * g[v].w;
#pragma unroll
  for (int off = G / 2; off >= 1; off >>= 1) ss += __shfl_down_sync(gmask, ss, off, G);
  ss = __shfl_sync(gmask, ss, 0, G);                       // every lane uses lane 0's sum
  const float sn = st + ss * (1.0f / (float)D);            // the reciprocal is loop-invariant at the call sites
  const float scale = __fdividef(lr, sqrtf(sn) + eps);     // within 2 ulp of the quotient
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    if (lane + v * G < nvec) {
      float4 o = r[v];
      o.x -= scale * g[v].x; o.y -= scale * g[v].y; o.z -= scale * g[v].z; o.w -= scale * g[v].w;
      row[lane + v * G] = o;
    }
  }
  __syncwarp(gmask);
  if (lane == 0) row_state[key] = sn;
}

template <int G, int NV>
__global__ void __launch_bounds__(kWaThreads, 8)
window_apply_kernel(const uint32_t* __restrict__ keys, const int32_t* __restrict__ sbag,
                    const int32_t* __restrict__ uidx, int64_t L, uint32_t sentinel, int64_t N, int D, int B,
                    const float* __restrict__ grad, int64_t ld_grad, int col0, float* __restrict__ partial,
                    int32_t* __restrict__ long_list, int32_t* __restrict__ scalars, int nwin, int64_t umax,
                    int32_t* __restrict__ d_status, float* __restrict__ tables, float* __restrict__ row_state,
                    float lr, float eps) {
  constexpr int kGroups = kWaThreads / G;
  __shared__ uint32_t s_key[kGroups][kWin + 2];            // [0] = key before the window, [kWin+1] = key after
  __shared__ int32_t s_row[kGroups][kWin];                 // float4 index of the lookup's gradient row
  __shared__ int32_t s_u[kGroups][kWin];
  const int grp = threadIdx.x / G, lane = threadIdx.x % G;
  const int64_t win = (int64_t)blockIdx.x * kGroups + grp;
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) / G * G));
  if (!ws_matches(scalars, L, sentinel, d_status)) return;
  if (win >= nwin) return;
  const int64_t w0 = win * kWin;
  const int nvec = D >> 2;
  const int64_t ld4 = ld_grad >> 2;
  for (int e = lane; e < kWin + 2; e += G) {
    const int64_t j = w0 - 1 + e;
    const bool in_range = j >= 0 && j < L;
    const bool body = e >= 1 && e <= kWin;
    uint32_t key = in_range ? keys[j] : sentinel;
    const int sb = (body && in_range) ? sbag[j] : 0;
    const int u = (body && in_range) ? uidx[j] : 0;
    int32_t row = -1;
    if (body && key < sentinel) {
      const int t = (int)((uint32_t)sb / (uint32_t)B);     // bags are table-major: bag = t*B + b
      const int b = sb - t * B;
      // a consistent workspace never fails these; an inconsistent one must not turn into a wild access
      if (sb >= 0 && (int64_t)key >= (int64_t)t * N && (int64_t)key < (int64_t)(t + 1) * N && u >= 0 && u < umax) {
        row = (int32_t)((int64_t)b * ld4 + (int64_t)t * nvec);   // B * ld_grad / 4 < 2^31 is checked on the host
        const char* trow = reinterpret_cast<const char*>(tables + (int64_t)key * D);
        for (int o = 0; o < D * 4; o += 128) prefetch_l2(trow + o);     // a repeated key asks for a line already on its way
        prefetch_l2(row_state + key);
      } else {
        key = sentinel;
      }
    }
    s_key[grp][e] = key;
    if (body) { s_row[grp][e - 1] = row; s_u[grp][e - 1] = u; }
  }
  __syncwarp(gmask);
  // valid (bits 16..31) and head (bits 0..15) of the positions this lane owns, then OR over the group
  uint32_t bits = 0;
  for (int i = lane; i < kWin; i += G) {
    const uint32_t k = s_key[grp][1 + i];
    if (k < sentinel) {
      bits |= 0x10000u << i;
      if (i == 0 || s_key[grp][i] != k) bits |= 1u << i;
    }
  }
#pragma unroll
  for (int off = G / 2; off >= 1; off >>= 1) bits |= __shfl_xor_sync(gmask, bits, off, G);
  const uint32_t vm = bits >> 16, hm = bits & 0xffffu;
  // a run ends where the next position starts another run, is a skipped lookup, or lies outside the window
  const uint32_t tm = vm & ((hm >> 1) | (~vm >> 1) | 0x8000u);
  const bool first_open = (vm & 1u) && s_key[grp][0] == s_key[grp][1];
  const bool last_open = (vm >> (kWin - 1) & 1u) && s_key[grp][kWin + 1] == s_key[grp][kWin];
  const float4* grad4 = reinterpret_cast<const float4*>(grad + col0);  // col0 is a multiple of 4

  float4 acc[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  constexpr int kBatch = 8 / NV;                           // gradient rows in flight per lane (8 float4)
#pragma unroll
  for (int i0 = 0; i0 < kWin; i0 += kBatch) {
    float4 gv[kBatch][NV];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int32_t row = s_row[grp][i0 + u];
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int c = lane + v * G;
        gv[u][v] = (row >= 0 && c < nvec) ? __ldg(grad4 + row + c) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int i = i0 + u;
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        if ((hm >> i) & 1u) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        acc[v] = add4(acc[v], gv[u][v]);                   // skipped lookups carry zeros and follow every run
      }
      if ((tm >> i) & 1u) {
        const uint32_t key = s_key[grp][1 + i];
        const bool first = (tm & ((1u << i) - 1u)) == 0u;  // the window's first run holds position 0
        const bool head_open = first && first_open;
        const bool tail_open = (i == kWin - 1) && last_open;
        if (!head_open && !tail_open) {
          adagrad_row_nv<G, NV>(acc, key, lane, nvec, D, gmask, tables, row_state, lr, eps);
        } else {
          // the run goes on in a neighbouring window: its part goes to the window's partial slot
          // (slot 0 when the run holds the window's first position), the combine kernel adds the parts
          float4* dst = reinterpret_cast<float4*>(partial + ((int64_t)win * 2 + (first ? 0 : 1)) * D);
#pragma unroll
          for (int v = 0; v < NV; ++v)
            if (lane + v * G < nvec) dst[lane + v * G] = acc[v];
          if (!head_open && lane == 0) {                   // the window in which a multi-window run starts lists the row
            const int slot = atomicAdd(&scalars[1], 1);
            if (slot < nwin) long_list[slot] = s_u[grp][i];   // at most one such run per window
          }
        }
      }
    }
  }
}

// Row-wise Adagrad on one row whose gradient slice is in the lanes' registers (rows of at most 4G floats).
template <int G>
__device__ __forceinline__ void adagrad_one_row(float4 g, uint32_t key, int lane, int nvec, int D, unsigned gmask,
                                                float* __restrict__ tables, float* __restrict__ row_state, float lr,
                                                float eps) {
  float4* row = reinterpret_cast<float4*>(tables + (int64_t)key * D);
  const float4 r = lane < nvec ? row[lane] : make_float4(0.f, 0.f, 0.f, 0.f);
  const float st = row_state[key];
  float ss = g.x * g.x + g.y * g.y + g.z * g.z + g.w * g.w;
#pragma unroll
  for (int off = G / 2; off >= 1; off >>= 1) ss += __shfl_down_sync(gmask, ss, off, G);
  ss = __shfl_sync(gmask, ss, 0, G);                       // every lane uses lane 0's sum
  const float sn = st + ss * (1.0f / (float)D);            // the reciprocal is loop-invariant at the call sites
  const float scale = __fdividef(lr, sqrtf(sn) + eps);     // within 2 ulp of the quotient
  if (lane < nvec) {
    float4 o = r;
    o.x -= scale * g.x; o.y -= scale * g.y; o.z -= scale * g.z; o.w -= scale * g.w;
    row[lane] = o;
  }
  __syncwarp(gmask);
  if (lane == 0) row_state[key] = sn;
}

// ---- (5) rows whose run crosses window edges: add their window partials ---------------------------
// Rows spanning up to 32 windows: one lane group adds the partials in window order.  Longer rows: one
// block per row, lane group j adds the partials of windows k0+j, k0+j+groups, ... in ascending order and
// the group sums are then added in group order.  The association is fixed by the
// segment's position alone (the order of the list does not matter).
// FUSE (rows of at most 128 floats): the combined sum is not stored; the row is updated here.
template <int G, int NV, bool FUSE>
__global__ void __launch_bounds__(256)
combine_rows_kernel(const int32_t* __restrict__ seg, const int32_t* __restrict__ scalars,
                    const int32_t* __restrict__ long_list, int nwin, int D, const float* __restrict__ partial,
                    float* __restrict__ gsum, int64_t L, uint32_t sentinel, int64_t umax,
                    const int32_t* __restrict__ uniq, float* __restrict__ tables, float* __restrict__ row_state,
                    float lr, float eps) {
  constexpr int kGroups = 256 / G;
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) / G * G));
  extern __shared__ float4 s_part[];                       // [kGroups][D/4]
  const int grp = threadIdx.x / G, lane = threadIdx.x % G;
  const int nvec = D >> 2;
  if (!ws_matches(scalars, L, sentinel, nullptr)) return;
  const int n = min(scalars[1], nwin);
  // Spans of up to kShort windows: one lane group per row, which requests kBatch partials at a time and adds them in
  // window order.  Only the rows with longer spans (the hottest of a skewed table) take a whole block each: a
  // block works through its rows one after the other, so that path must stay short -- but a lane group walking a
  // long span is a chain of dependent rounds at the kernel's tail: of 2 / 4 / 8 / 32 / 128 windows, 8 was the
  // fastest (the call 66.7 us against 69.5 with 32 and 89.8 with 128).
  constexpr int kShort = 8;
  constexpr int kBatch = NV <= 1 ? 8 : (NV <= 2 ? 4 : 2);
  // The two phases are two chains of dependent loads; with enough blocks the first half of the grid takes the long
  // spans (phase B) and the second half the short ones (phase A), so that the chains run side by side instead of
  // one after the other.  A small grid does both in every block.
  const int nb_long = gridDim.x >= 4 ? (int)gridDim.x / 2 : 0;
  const bool do_short = nb_long == 0 || (int)blockIdx.x >= nb_long;
  const bool do_long = nb_long == 0 || (int)blockIdx.x < nb_long;
  const int a_blk = nb_long == 0 ? (int)blockIdx.x : (int)blockIdx.x - nb_long;
  const int a_blocks = nb_long == 0 ? (int)gridDim.x : (int)gridDim.x - nb_long;
  const int b_blocks = nb_long == 0 ? (int)gridDim.x : nb_long;
  // phase A
  for (int i = a_blk * kGroups + grp; do_short && i < n; i += a_blocks * kGroups) {
    const int u = long_list[i];
    if (u < 0 || u >= umax) continue;
    const int s0 = seg[u], s1 = seg[u + 1];
    if (s0 < 0 || s1 <= s0 || s1 > L) continue;
    const int k0 = s0 / kWin, k1 = (s1 - 1) / kWin;
    if (k1 - k0 + 1 > kShort) continue;
    float4 t[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) t[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int kb = k0; kb <= k1; kb += kBatch) {
      float4 pv[kBatch][NV];
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        const int k = kb + j;
        const int slot = (s0 <= k * kWin) ? 0 : 1;         // the run covers the window's first position -> slot 0
        const float4* p = reinterpret_cast<const float4*>(partial + ((int64_t)k * 2 + slot) * D);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
          const int c = lane + v * G;
          pv[j][v] = (k <= k1 && c < nvec) ? p[c] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
#pragma unroll
      for (int j = 0; j < kBatch; ++j)
#pragma unroll
        for (int v = 0; v < NV; ++v) t[v] = add4(t[v], pv[j][v]);   // adding zeros for absent windows changes nothing
    }
    if (!FUSE) {
      float4* dst = reinterpret_cast<float4*>(gsum + (int64_t)u * D);
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int c = lane + v * G;
        if (c < nvec) dst[c] = t[v];
      }
    }
    if (FUSE) {
      const uint32_t key = (uint32_t)uniq[u];
      if (key < sentinel) adagrad_row_nv<G, NV>(t, key, lane, nvec, D, gmask, tables, row_state, lr, eps);
    }
  }
  // phase B: long spans, the whole block per row.  The block owns the list entries blockIdx.x + k*gridDim.x;
  // its threads look at 256 of them at a time (one round of loads) and queue the long ones.
  __shared__ int s_long[256];
  __shared__ int s_nlong;
  for (int64_t base = 0; do_long && (int64_t)blockIdx.x + base * b_blocks < n; base += 256) {
    if (threadIdx.x == 0) s_nlong = 0;
    __syncthreads();
    {
      const int64_t i = (int64_t)blockIdx.x + (base + threadIdx.x) * b_blocks;
      if (i < n) {
        const int u = long_list[i];
        if (u >= 0 && u < umax) {
          const int s0 = seg[u], s1 = seg[u + 1];
          if (s0 >= 0 && s1 > s0 && s1 <= L && (s1 - 1) / kWin - s0 / kWin + 1 > kShort) s_long[atomicAdd(&s_nlong, 1)] = u;
        }
      }
    }
    __syncthreads();
    const int nlong = s_nlong;
  for (int q = 0; q < nlong; ++q) {
    const int u = s_long[q];                               // checked above; uniform over the block
    const int s0 = seg[u], s1 = seg[u + 1];
    const int k0 = s0 / kWin, k1 = (s1 - 1) / kWin;
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = k0 + grp; k <= k1; k += kGroups) {
      const int slot = (s0 <= k * kWin) ? 0 : 1;
      const float4* p = reinterpret_cast<const float4*>(partial + ((int64_t)k * 2 + slot) * D);
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int c = lane + v * G;
        if (c < nvec) acc[v] = add4(acc[v], p[c]);
      }
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int c = lane + v * G;
      if (c < nvec) s_part[grp * nvec + c] = acc[v];
    }
    __syncthreads();
    if (grp == 0) {
      const int used = min(kGroups, k1 - k0 + 1);
      float4* dst = reinterpret_cast<float4*>(gsum + (int64_t)u * D);
      float4 tt[NV];
#pragma unroll
      for (int v = 0; v < NV; ++v) {
        const int c = lane + v * G;
        tt[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < nvec) {
          float4 t = s_part[c];
          for (int j = 1; j < used; ++j) t = add4(t, s_part[j * nvec + c]);
          if (!FUSE) dst[c] = t;
          tt[v] = t;
        }
      }
      if (FUSE) {
        const uint32_t key = (uint32_t)uniq[u];
        if (key < sentinel) adagrad_row_nv<G, NV>(tt, key, lane, nvec, D, gmask, tables, row_state, lr, eps);
      }
    }
    __syncthreads();
  }
  }
}

// ---- (6) row-wise Adagrad, one lane group per four distinct rows ----------------------------------
//   g = gsum[u];  s = state + mean_d g^2;  row -= lr * g / (sqrt(s) + eps)
template <int NV> struct RowsPerGroup { static constexpr int value = NV == 1 ? 4 : (NV == 2 ? 2 : 1); };

template <int G, int NV>
__global__ void __launch_bounds__(256)
apply_rows_kernel(const int32_t* __restrict__ uniq, const int32_t* __restrict__ scalars, int D,
                  const float* __restrict__ gsum, float* __restrict__ tables, float* __restrict__ row_state,
                  float lr, float eps, int64_t L, uint32_t sentinel, int64_t umax,
                  const int32_t* __restrict__ list, int list_cap) {
  constexpr int kGroups = 256 / G;
  constexpr int RB = RowsPerGroup<NV>::value;              // rows per group, their loads issued together
  const int grp = threadIdx.x / G, lane = threadIdx.x % G;
  const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << ((threadIdx.x & 31) / G * G));
  if (!ws_matches(scalars, L, sentinel, nullptr)) return;
  // all distinct rows, or (list given) only the listed ones: the rows whose run crossed window edges
  const int U = list ? min(scalars[1], list_cap) : (int)min((int64_t)scalars[0], umax);
  const int nvec = D >> 2;
  const int64_t u0 = ((int64_t)blockIdx.x * kGroups + grp) * RB;
  if (u0 >= U) return;
  uint32_t key[RB];
  int64_t urow[RB];
  bool valid[RB];
#pragma unroll
  for (int r = 0; r < RB; ++r) {
    valid[r] = u0 + r < U;
    urow[r] = valid[r] ? (list ? (int64_t)list[u0 + r] : u0 + r) : 0;
    if (urow[r] < 0 || urow[r] >= umax) { valid[r] = false; urow[r] = 0; }
    key[r] = valid[r] ? (uint32_t)uniq[urow[r]] : 0u;
    if (key[r] >= sentinel) valid[r] = false;              // never true for a consistent workspace
  }
  float4 g[RB][NV], rw[RB][NV];
  float st[RB];
#pragma unroll
  for (int r = 0; r < RB; ++r) {
    const float4* p = reinterpret_cast<const float4*>(gsum + urow[r] * D);
    const float4* row = reinterpret_cast<const float4*>(tables + (int64_t)key[r] * D);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int c = lane + v * G;
      g[r][v] = (valid[r] && c < nvec) ? p[c] : make_float4(0.f, 0.f, 0.f, 0.f);
      rw[r][v] = (valid[r] && c < nvec) ? row[c] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    st[r] = valid[r] ? row_state[key[r]] : 0.f;
  }
#pragma unroll
  for (int r = 0; r < RB; ++r) {
    float ss = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v)
      ss += g[r][v].x * g[r][v].x + g[r][v].y * g[r][v].y + g[r][v].z * g[r][v].z + g[r][v].w * g[r][v].w;
#pragma unroll
    for (int off = G / 2; off >= 1; off >>= 1) ss += __shfl_down_sync(gmask, ss, off, G);
    ss = __shfl_sync(gmask, ss, 0, G);                     // every lane uses lane 0's sum
    if (!valid[r]) continue;
    const float s = st[r] + ss / (float)D;
    const float scale = lr / (sqrtf(s) + eps);
    float4* row = reinterpret_cast<float4*>(tables + (int64_t)key[r] * D);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const int c = lane + v * G;
      if (c < nvec) {
        float4 o = rw[r][v];
        o.x -= scale * g[r][v].x; o.y -= scale * g[r][v].y; o.z -= scale * g[r][v].z; o.w -= scale * g[r][v].w;
        row[c] = o;
      }
    }
    if (lane == 0) row_state[key[r]] = s;
  }
}

template <int G, int NV>
static void launch_reduce(const BwdPlan& p, char* ws, const uint32_t* keys, const int32_t* perm, int T, int64_t N,
                          int D, int B, const float* grad, int64_t ld_grad, int col0, float* tables,
                          float* row_state, float lr, float eps, int32_t* d_status, cudaStream_t st) {
  constexpr int kGroups = 256 / G;
  const uint64_t maxkey = (uint64_t)T * (uint64_t)N;
  const uint64_t umax = (uint64_t)p.L < maxkey ? (uint64_t)p.L : maxkey;
  const uint32_t sentinel = (uint32_t)((uint64_t)T * (uint64_t)N);
  float* partial = reinterpret_cast<float*>(ws + p.off_partial);
  float* gsum = reinterpret_cast<float*>(ws + p.off_gsum);
  const unsigned blocks = (unsigned)((p.nwin + kGroups - 1) / kGroups);
  int32_t* scalars = reinterpret_cast<int32_t*>(ws + p.off_scalars);
  int32_t* long_list = reinterpret_cast<int32_t*>(ws + p.off_long);
  int32_t* seg = reinterpret_cast<int32_t*>(ws + p.off_seg);
  int32_t* uniq = reinterpret_cast<int32_t*>(ws + p.off_uniq);
  constexpr bool kFuse = (NV == 1);
  // the list of rows crossing window edges starts empty (the apply half may be repeated on one sort)
  cudaMemsetAsync(scalars + 1, 0, sizeof(int32_t), st);
  if (kFuse) {
    // two float4 per lane (half as many lanes per window) wherever the row has at least eight
    constexpr int WG = G >= 8 ? G / 2 : G, WNV = G >= 8 ? 2 : 1;
    constexpr int kWaGroups = kWaThreads / WG;
    SS_TIMED("window_apply_kernel", st);
    window_apply_kernel<WG, WNV><<<(unsigned)((p.nwin + kWaGroups - 1) / kWaGroups), kWaThreads, 0, st>>>(
        keys, reinterpret_cast<int32_t*>(ws + p.off_sbag), reinterpret_cast<int32_t*>(ws + p.off_uidx), p.L, sentinel,
        N, D, B, grad, ld_grad, col0, partial, long_list, scalars, p.nwin, (int64_t)umax, d_status, tables, row_state,
        lr, eps);
  } else {
    SS_TIMED("window_reduce_kernel", st);
    window_reduce_kernel<G, NV><<<blocks, 256, 0, st>>>(
        keys, reinterpret_cast<int32_t*>(ws + p.off_sbag), reinterpret_cast<int32_t*>(ws + p.off_uidx), p.L, sentinel, N, D,
        B, grad, ld_grad, col0, gsum, partial, long_list, scalars, p.nwin, (int64_t)umax, d_status);
  }
  {
    SS_TIMED("combine_rows_kernel", st);
    const int cblocks = p.nwin < num_sms() * 8 ? p.nwin : num_sms() * 8;
    // fused rows of at least eight float4: two float4 per lane, half as many lanes per row, twice as many rows in flight
    constexpr int CG = (kFuse && G >= 8) ? G / 2 : G, CNV = (kFuse && G >= 8) ? 2 : NV;
    combine_rows_kernel<CG, CNV, kFuse><<<cblocks, 256, (size_t)(256 / CG) * D * 4, st>>>(
        seg, scalars, long_list, p.nwin, D, partial, gsum, p.L, sentinel, (int64_t)umax, uniq, tables, row_state, lr, eps);
  }
  if (!kFuse) {
    // rows wider than 128 floats: every distinct row is updated from its sum in gsum
    const uint64_t per_block = (uint64_t)kGroups * RowsPerGroup<NV>::value;
    const unsigned ublocks = (unsigned)((umax + per_block - 1) / per_block);
    SS_TIMED("apply_rows_kernel", st);
    apply_rows_kernel<G, NV><<<ublocks, 256, 0, st>>>(uniq, scalars, D, gsum, tables, row_state, lr, eps, p.L, sentinel,
                                                      (int64_t)umax, nullptr, 0);
  }
}

#define SS_DISPATCH_GNV(D_, CALL)                                                 \
  do {                                                                            \
    const int nvec__ = (D_) / 4;                                                  \
    if (nvec__ <= 4) { CALL(4, 1); }                                              \
    else if (nvec__ <= 8) { CALL(8, 1); }                                         \
    else if (nvec__ <= 16) { CALL(16, 1); }                                       \
    else if (nvec__ <= 32) { CALL(32, 1); }                                       \
    else if (nvec__ <= 64) { CALL(32, 2); }                                       \
    else if (nvec__ <= 128) { CALL(32, 4); }                                      \
    else { CALL(32, 8); }                                                         \
  } while (0)

}  // namespace ss

extern "C" {

ss_status ss_embbag_fwd(const float* tables, int T, int64_t N, int D, const int32_t* indices,
                        const int32_t* offsets, int B, float* out_f32, int64_t ld_f32, void* out_bf16,
                        int64_t ld_bf16, int col0, int32_t* d_status, ss_stream stream) {
  if (!tables || !indices || !offsets) return SS_ERR_NULL;
  if (!out_f32 && !out_bf16) return SS_ERR_NULL;
  if (T < 0 || B < 0 || N <= 0 || D <= 0 || D > 1024 || (D & 3) || col0 < 0) return SS_ERR_SHAPE;
  if ((uint64_t)T * (uint64_t)N >= (1ull << 31) || T > 65535 || (uint64_t)N * (uint64_t)(D / 4) >= (1ull << 32)) return SS_ERR_SHAPE;
  if (!ss::aligned16(tables) || (col0 & 3)) return SS_ERR_ALIGN;
  if (out_f32 && (!ss::aligned16(out_f32) || (ld_f32 & 3) || ld_f32 < col0 + (int64_t)T * D)) return SS_ERR_ALIGN;
  if (out_bf16 && ((reinterpret_cast<uintptr_t>(out_bf16) & 7u) || (ld_bf16 & 3) || ld_bf16 < col0 + (int64_t)T * D))
    return SS_ERR_ALIGN;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  if ((int64_t)T * B == 0) return SS_OK;
  cudaStream_t cs = ss::as_stream(stream);
#define SS_FWD(G_, NV_)                                                                                     \
  ss::launch_fwd<G_, NV_>(tables, T, N, D, indices, offsets, B, out_f32, ld_f32, (__nv_bfloat16*)out_bf16, \
                          ld_bf16, col0, d_status, cs)
  SS_DISPATCH_GNV(D, SS_FWD);
#undef SS_FWD
  SS_LAUNCH_OK();
  return SS_OK;
}

size_t ss_embbag_bwd_workspace_bytes(int T, int64_t N, int D, int B, int64_t L) {
  (void)B;
  if (T < 0 || N <= 0 || D <= 0 || L < 0) return 0;
  return ss::make_plan(T, N, D, L).total;
}

static ss_status bwd_impl(bool do_sort, bool do_apply, float* tables, float* row_state, int T, int64_t N, int D,
                          const int32_t* indices, const int32_t* offsets, int B, int64_t L, const float* grad,
                          int64_t ld_grad, int col0, float lr, float eps, void* workspace, size_t workspace_bytes,
                          int32_t* uniq_keys, int32_t* seg_off, int32_t* perm, int32_t* d_num_unique,
                          int32_t* d_status, ss_stream stream) {
  using namespace ss;
  if (!workspace) return SS_ERR_NULL;
  if (do_sort && ((!indices && L > 0) || !offsets)) return SS_ERR_NULL;
  if (do_apply && (!tables || !row_state || !grad)) return SS_ERR_NULL;
  if (T < 0 || B < 0 || N <= 0 || D <= 0 || D > 1024 || (D & 3) || col0 < 0 || L < 0) return SS_ERR_SHAPE;
  if ((uint64_t)T * (uint64_t)N >= (1ull << 31) || L >= (1ll << 31) - kSortTile) return SS_ERR_SHAPE;
  if (!aligned16(workspace)) return SS_ERR_ALIGN;
  if (do_apply) {
    if (!aligned16(tables) || !aligned16(grad) || (ld_grad & 3) || (col0 & 3)) return SS_ERR_ALIGN;
    if (ld_grad < col0 + (int64_t)T * D || (int64_t)B * ld_grad / 4 >= (1ll << 31)) return SS_ERR_SHAPE;
  }
  const BwdPlan p = make_plan(T, N, D, L);
  if (workspace_bytes < p.total) return SS_ERR_WORKSPACE;
  ss_status stt = check_arch();
  if (stt != SS_OK) return stt;
  cudaStream_t cs = as_stream(stream);
  char* ws = reinterpret_cast<char*>(workspace);
  uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + p.off_keys_a);
  uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + p.off_keys_b);
  int32_t* pos_a = reinterpret_cast<int32_t*>(ws + p.off_pos_a);
  int32_t* pos_b = reinterpret_cast<int32_t*>(ws + p.off_pos_b);
  int32_t* bag_of = reinterpret_cast<int32_t*>(ws + p.off_bag);
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + p.off_hist);
  uint32_t* bintot = reinterpret_cast<uint32_t*>(ws + p.off_bintot);
  uint32_t* usum = reinterpret_cast<uint32_t*>(ws + p.off_usum);
  int32_t* uniq = reinterpret_cast<int32_t*>(ws + p.off_uniq);
  int32_t* seg = reinterpret_cast<int32_t*>(ws + p.off_seg);
  int32_t* uidx = reinterpret_cast<int32_t*>(ws + p.off_uidx);
  int32_t* scalars = reinterpret_cast<int32_t*>(ws + p.off_scalars);
  const uint32_t sentinel = (uint32_t)((uint64_t)T * (uint64_t)N);

  if (L == 0 || (int64_t)T * B == 0) {
    if (do_sort) {
      SS_TIMED("unique_finish_kernel", cs);
      unique_finish_kernel<<<1, 1, 0, cs>>>(nullptr, seg, seg_off, d_num_unique, scalars, L, sentinel);
      SS_LAUNCH_OK();
    }
    return SS_OK;
  }
  // the sorted arrays end up in the buffers the last pass wrote
  const uint32_t* keys_sorted = (p.passes & 1) ? keys_b : keys_a;
  const int32_t* perm_sorted = (p.passes & 1) ? pos_b : pos_a;
  if (do_sort) {

  // (0) one block per table sorts that table's lookups in shared memory; scalars[4] stays 0 when every
  // block could, and the tiled sort below then returns at once
  int32_t* fallback = scalars + 4;
  int* sort_ctl = scalars + 8;                             // control words of the tiled sort: zero at launch, left zero
  // more lookups than T tables of kTsCap can hold: some table is too large for its block, the tiled sort is certain
  const bool try_table_sort = B <= 65536 && L <= (int64_t)T * kTsCap;
  SS_CUDA(cudaMemsetAsync(fallback, 0, 8 * sizeof(int32_t), cs));
  if (try_table_sort) {
    int row_bits = 1;
    while (((uint64_t)(N - 1) >> row_bits) != 0) ++row_bits;
    const int t_passes = (row_bits + 7) / 8;
    int t_digit = (row_bits + t_passes - 1) / t_passes;
    if (t_digit < 5) t_digit = 5;                          // the in-block scan wants at least 32 bins
    static bool attr_set[64];
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64 && !attr_set[dev]) {
      cudaFuncSetAttribute(table_sort_kernel<5>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTsSmem);
      cudaFuncSetAttribute(table_sort_kernel<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTsSmem);
      cudaFuncSetAttribute(table_sort_kernel<7>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTsSmem);
      cudaFuncSetAttribute(table_sort_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTsSmem);
      attr_set[dev] = true;
    }
    SS_TIMED("table_sort_kernel", cs);
#define SS_TS(NB_)                                                                                              \
  table_sort_kernel<NB_><<<T, kTsThreads, kTsSmem, cs>>>(indices, offsets, T, N, B, L, t_passes,                \
                                                         const_cast<uint32_t*>(keys_sorted),                    \
                                                         const_cast<int32_t*>(perm_sorted), bag_of, fallback)
    switch (t_digit) {
      case 5: SS_TS(5); break;
      case 6: SS_TS(6); break;
      case 7: SS_TS(7); break;
      default: SS_TS(8); break;
    }
#undef SS_TS
  }
  SS_LAUNCH_OK();

  // (1) keys and (2) LSD radix sort, `passes` digits of `digit_bits` bits, as one launch (see tiled_sort_kernel)
  {
    TiledSort ts;
    ts.indices = indices; ts.offsets = offsets; ts.T = T; ts.B = B; ts.N = N; ts.L = L;
    ts.keys_a = keys_a; ts.keys_b = keys_b; ts.pos_a = pos_a; ts.pos_b = pos_b; ts.bag_of = bag_of;
    ts.hist = hist; ts.bintot = bintot; ts.d_status = d_status;
    ts.run_if = try_table_sort ? fallback : nullptr;
    ts.ctl = sort_ctl;
    ts.passes = p.passes; ts.digit_bits = p.digit_bits; ts.bins = p.bins; ts.nblk = p.nblk;
    ts.n_key_items = (int)(((int64_t)T * B + 255) / 256);
    ts.n_scan_items = (p.bins + 7) / 8;
    int grid = ts.n_key_items > p.nblk ? ts.n_key_items : p.nblk;
    if (grid > 4 * num_sms()) grid = 4 * num_sms();
    SS_TIMED("tiled_sort_kernel", cs);
    tiled_sort_kernel<<<grid, kSortThreads, 0, cs>>>(ts);
  }
  SS_LAUNCH_OK();
  if (perm) SS_CUDA(cudaMemcpyAsync(perm, perm_sorted, (size_t)L * 4, cudaMemcpyDeviceToDevice, cs));

  // (3) unique keys and segment offsets
  { SS_TIMED("unique_count_kernel", cs);
  unique_count_kernel<<<p.nblk_u, kScanThreads, 0, cs>>>(keys_sorted, L, sentinel, usum);
  }
  { SS_TIMED("scan_exclusive_kernel", cs);
  scan_exclusive_kernel<<<1, kScanThreads, 0, cs>>>(usum, p.nblk_u, usum + p.nblk_u,
                                                    UniqueFinish{seg, seg_off, d_num_unique, scalars, L, sentinel});
  }
  { SS_TIMED("unique_write_kernel", cs);
  unique_write_kernel<<<p.nblk_u, kScanThreads, 0, cs>>>(keys_sorted, L, sentinel, usum, uniq, seg, uidx, uniq_keys, seg_off,
                                                         perm_sorted, bag_of, reinterpret_cast<int32_t*>(ws + p.off_sbag));
  }
  SS_LAUNCH_OK();

  }  // do_sort

  // (4) windowed segment reduction, (5) combine, (6) row-wise Adagrad
  if (do_apply) {
#define SS_RED(G_, NV_) \
  launch_reduce<G_, NV_>(p, ws, keys_sorted, perm_sorted, T, N, D, B, grad, ld_grad, col0, tables, row_state, lr, eps, d_status, cs)
    SS_DISPATCH_GNV(D, SS_RED);
#undef SS_RED
    SS_LAUNCH_OK();
  }
  return SS_OK;
}

ss_status ss_embbag_bwd_adagrad(float* tables, float* row_state, int T, int64_t N, int D, const int32_t* indices,
                                const int32_t* offsets, int B, int64_t L, const float* grad, int64_t ld_grad,
                                int col0, float lr, float eps, void* workspace, size_t workspace_bytes,
                                int32_t* uniq_keys, int32_t* seg_off, int32_t* perm, int32_t* d_num_unique,
                                int32_t* d_status, ss_stream stream) {
  return bwd_impl(true, true, tables, row_state, T, N, D, indices, offsets, B, L, grad, ld_grad, col0, lr, eps, workspace,
                  workspace_bytes, uniq_keys, seg_off, perm, d_num_unique, d_status, stream);
}

ss_status ss_embbag_bwd_sort(int T, int64_t N, int D, const int32_t* indices, const int32_t* offsets, int B, int64_t L,
                             void* workspace, size_t workspace_bytes, int32_t* uniq_keys, int32_t* seg_off,
                             int32_t* perm, int32_t* d_num_unique, int32_t* d_status, ss_stream stream) {
  return bwd_impl(true, false, nullptr, nullptr, T, N, D, indices, offsets, B, L, nullptr, 0, 0, 0.f, 0.f, workspace,
                  workspace_bytes, uniq_keys, seg_off, perm, d_num_unique, d_status, stream);
}

ss_status ss_embbag_bwd_apply(float* tables, float* row_state, int T, int64_t N, int D, int B, int64_t L,
                              const float* grad, int64_t ld_grad, int col0, float lr, float eps, void* workspace,
                              size_t workspace_bytes, int32_t* d_status, ss_stream stream) {
  return bwd_impl(false, true, tables, row_state, T, N, D, nullptr, nullptr, B, L, grad, ld_grad, col0, lr, eps, workspace,
                  workspace_bytes, nullptr, nullptr, nullptr, nullptr, d_status, stream);
}

// ------------------------------------------------------------------------------------------------
// Sort / unique without any caller-provided or allocated scratch.
//
// Some callers of this library may not allocate device memory at the moment they need the sort: a
// host process whose memory pool has already handed every byte of the GPU to other owners, a plug-in
// that runs inside somebody else's serving loop where cudaMalloc's implicit device-wide
// synchronisation would stall unrelated streams, or start-up code that runs before the application's
// allocator exists.  For them the scratch of the sort lives in the array below, which is part of the
// library image: every GPU that loads the library holds these bytes until the process exits.
// ------------------------------------------------------------------------------------------------
constexpr int64_t kNoAllocMaxL = 65536;                       // most lookups one call may sort
constexpr size_t kNoAllocScratchBytes = 2162688;              // 2112 KiB, enough for kNoAllocMaxL lookups
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// Device address of the array for the current device.  The array's name is only a handle on the
// host: the address a kernel can use comes from cudaGetSymbolAddress, asked once per device.
static ss_status noalloc_scratch_ptr(unsigned char** out) {
  static unsigned char* ptr[64];
  int dev = 0;
  SS_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SS_ERR_SHAPE;
  if (!ptr[dev]) {
    void* p = nullptr;
    SS_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    ptr[dev] = reinterpret_cast<unsigned char*>(p);
  }
  *out = ptr[dev];
  return SS_OK;
}

ss_status ss_embbag_bwd_sort_noalloc(int T, int64_t N, const int32_t* indices, const int32_t* offsets, int B,
                                     int64_t L, int32_t* uniq_keys, int32_t* seg_off, int32_t* perm,
                                     int32_t* d_num_unique, int32_t* d_status, ss_stream stream) {
  using namespace ss;
  if (!offsets || (!indices && L > 0) || !uniq_keys || !seg_off || !perm || !d_num_unique) return SS_ERR_NULL;
  if (T < 0 || B < 0 || N <= 0 || L < 0) return SS_ERR_SHAPE;
  if (L > kNoAllocMaxL) return SS_ERR_SHAPE;                   // beyond the built-in scratch: use ss_embbag_bwd_sort
  if ((uint64_t)T * (uint64_t)N >= (1ull << 31)) return SS_ERR_SHAPE;
  ss_status stt = check_arch();
  if (stt != SS_OK) return stt;
  unsigned char* ws = nullptr;
  stt = noalloc_scratch_ptr(&ws);
  if (stt != SS_OK) return stt;
  cudaStream_t cs = as_stream(stream);

  // digit plan of the radix sort (same rule as the workspace variant)
  const uint64_t maxkey = (uint64_t)T * (uint64_t)N;
  int bits = 1;
  while ((maxkey >> bits) != 0) ++bits;
  const int passes = (bits + 8) / 9;
  const int digit_bits = (bits + passes - 1) / passes;
  const int bins = 1 << digit_bits;
  const int nblk = L > 0 ? (int)((L + kSortTile - 1) / kSortTile) : 1;
  const int nblk_u = L > 0 ? (int)((L + kScanThreads - 1) / kScanThreads) : 1;

  // carve the array; every piece is rewritten in full by each call before it is read, so nothing
  // depends on what an earlier call left behind
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += align256(bytes); return r; };
  const size_t l4 = (size_t)kNoAllocMaxL * 4;
  uint32_t* keys_a = reinterpret_cast<uint32_t*>(ws + take(l4));
  uint32_t* keys_b = reinterpret_cast<uint32_t*>(ws + take(l4));
  int32_t* pos_a = reinterpret_cast<int32_t*>(ws + take(l4));
  int32_t* pos_b = reinterpret_cast<int32_t*>(ws + take(l4));
  int32_t* bag_of = reinterpret_cast<int32_t*>(ws + take(l4));
  int32_t* uniq = reinterpret_cast<int32_t*>(ws + take(l4));
  int32_t* uidx = reinterpret_cast<int32_t*>(ws + take(l4));
  int32_t* seg = reinterpret_cast<int32_t*>(ws + take(l4 + 4));
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + take((size_t)(kNoAllocMaxL / kSortTile) * kMaxBins * 4));
  uint32_t* bintot = reinterpret_cast<uint32_t*>(ws + take((size_t)kMaxBins * 4));
  uint32_t* usum = reinterpret_cast<uint32_t*>(ws + take((size_t)(kNoAllocMaxL / kScanThreads + 1) * 4));
  int32_t* scalars = reinterpret_cast<int32_t*>(ws + take(256));
  if (o > kNoAllocScratchBytes) return SS_ERR_WORKSPACE;
  const uint32_t sentinel = (uint32_t)maxkey;

  if (L == 0 || (int64_t)T * B == 0) {
    unique_finish_kernel<<<1, 1, 0, cs>>>(nullptr, seg, seg_off, d_num_unique, scalars, L, sentinel);
    SS_LAUNCH_OK();
    return SS_OK;
  }
  build_keys_kernel<<<(unsigned)(((int64_t)T * B + 255) / 256), 256, 0, cs>>>(indices, offsets, T, N, B, L, keys_a,
                                                                                bag_of, d_status, nullptr);
  SS_LAUNCH_OK();
  uint32_t* kin = keys_a; uint32_t* kout = keys_b;
  int32_t* pin = nullptr;
  int32_t* pout = pos_b;
  int32_t* pnext = pos_a;
  const size_t smem = ((size_t)kSortWarps * bins + bins + 8) * 4;
  for (int pass = 0; pass < passes; ++pass) {
    const int shift = pass * digit_bits;
    sort_hist_kernel<<<nblk, kSortThreads, 0, cs>>>(kin, L, shift, bins, nblk, hist, nullptr);
    bin_scan_kernel<<<(bins + 7) / 8, 256, 0, cs>>>(hist, bins, nblk, bintot, nullptr);
    sort_scatter_kernel<<<nblk, kSortThreads, smem, cs>>>(kin, pin, kout, pout, L, shift, bins, nblk, hist, bintot,
                                                          nullptr);
    SS_LAUNCH_OK();
    uint32_t* tk = kin; kin = kout; kout = tk;
    pin = pout; pout = pnext; pnext = pin;
  }
  SS_CUDA(cudaMemcpyAsync(perm, pin, (size_t)L * 4, cudaMemcpyDeviceToDevice, cs));
  unique_count_kernel<<<nblk_u, kScanThreads, 0, cs>>>(kin, L, sentinel, usum);
  scan_exclusive_kernel<<<1, kScanThreads, 0, cs>>>(usum, nblk_u, usum + nblk_u,
                                                    UniqueFinish{seg, seg_off, d_num_unique, scalars, L, sentinel});
  unique_write_kernel<<<nblk_u, kScanThreads, 0, cs>>>(kin, L, sentinel, usum, uniq, seg, uidx, uniq_keys, seg_off,
                                                       nullptr, nullptr, nullptr);
  SS_LAUNCH_OK();
  return SS_OK;
}

}  // extern "C"
