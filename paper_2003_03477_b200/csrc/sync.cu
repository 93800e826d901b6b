// Background synchronisation kernels: Shadow EASGD, Shadow MA, Shadow BMUF (Algorithms 2, 3, 4).
//
// Each rule is one element-wise pass: a thread owns one float4 position, loads that position from
// all R replicas and from the centre/global copy (R+1 independent 128-bit loads in flight), applies
// the rule in registers and stores everything back.  Traffic is exactly one read and one write of
// every vector, which is what bounds the kernel (HBM for vectors beyond L2).  The replica pointers
// travel in the kernel parameter block, so there is no pointer table in device memory.
#include "common.cuh"
#include "profile.cuh"

namespace ss {

constexpr int kMaxR = 16;

struct SyncPtrs {
  float* w[kMaxR];
  __nv_bfloat16* m[kMaxR];   // bf16 mirrors, only read when MIRROR
};

__device__ __forceinline__ uint2 pack_bf16x4(float4 v) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  return r;
}

enum { RULE_EASGD = 0, RULE_EASGD_LITERAL = 1, RULE_MA = 2, RULE_BMUF = 3, RULE_BMUF_NESTEROV = 4 };

template <int RULE> struct IsBmuf { static constexpr bool value = (RULE == 3 || RULE == 4); };

struct SyncScalars {
  float alpha, eta, mu, inv_r;
};

// One scalar position of a rule.  w[0..R) in/out; c = centre (EASGD) or global (BMUF/MA out); dl = BMUF delta.
template <int RULE, int R>
__device__ __forceinline__ void apply_rule(float (&w)[R], float& c, float& dl, const SyncScalars& s) {
  if (RULE == RULE_EASGD) {
#pragma unroll
    for (int r = 0; r < R; ++r) {          // trainers visit the centre in turn
      float d = s.alpha * (w[r] - c);
      w[r] -= d;
      c += d;
    }
  } else if (RULE == RULE_EASGD_LITERAL) {
#pragma unroll
    for (int r = 0; r < R; ++r) {          // Algorithm 2 line by line: centre first, replica toward the new centre
      c = c + s.alpha * (w[r] - c);
      w[r] = w[r] + s.alpha * (c - w[r]);
    }
  } else {
    float sum = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) sum += w[r];
    float m = sum * s.inv_r;
    if (RULE == RULE_MA) {
      c = m;
    } else {
      dl = s.mu * dl + s.eta * (m - c);
      c = c + dl;
    }
    // Nesterov look-ahead: the replicas are pulled toward where the global model is heading
    const float target = (RULE == RULE_BMUF_NESTEROV) ? c + s.mu * dl : c;
#pragma unroll
    for (int r = 0; r < R; ++r) w[r] = w[r] + s.alpha * (target - w[r]);
  }
}

template <int RULE, int R, bool MIRROR>
__global__ void __launch_bounds__(256)
sync_kernel(SyncPtrs p, float* __restrict__ c, float* __restrict__ delta, int64_t n4, int64_t n, SyncScalars s) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  constexpr bool kReadC = (RULE != RULE_MA);
  if (i < n4) {
    float4 wv[R];
#pragma unroll
    for (int r = 0; r < R; ++r) wv[r] = reinterpret_cast<const float4*>(p.w[r])[i];
    float4 cv = make_float4(0.f, 0.f, 0.f, 0.f), dv = cv;
    if (kReadC) cv = reinterpret_cast<const float4*>(c)[i];
    if (IsBmuf<RULE>::value) dv = reinterpret_cast<const float4*>(delta)[i];

    float a[R];
#define SS_LANE(F)                                         \
    {                                                      \
      _Pragma("unroll") for (int r = 0; r < R; ++r) a[r] = wv[r].F; \
      apply_rule<RULE, R>(a, cv.F, dv.F, s);               \
      _Pragma("unroll") for (int r = 0; r < R; ++r) wv[r].F = a[r]; \
    }
    SS_LANE(x) SS_LANE(y) SS_LANE(z) SS_LANE(w)
#undef SS_LANE

#pragma unroll
    for (int r = 0; r < R; ++r) {
      reinterpret_cast<float4*>(p.w[r])[i] = wv[r];
      if (MIRROR) reinterpret_cast<uint2*>(p.m[r])[i] = pack_bf16x4(wv[r]);
    }
    if (c != nullptr) reinterpret_cast<float4*>(c)[i] = cv;
    if (IsBmuf<RULE>::value) reinterpret_cast<float4*>(delta)[i] = dv;
  }
  // ragged tail (n not a multiple of 4): the first threads of block 0 take one scalar each
  if (blockIdx.x == 0 && threadIdx.x < (int)(n - n4 * 4)) {
    const int64_t k = n4 * 4 + threadIdx.x;
    float a[R];
#pragma unroll
    for (int r = 0; r < R; ++r) a[r] = p.w[r][k];
    float cs = (kReadC ? c[k] : 0.f), ds = (IsBmuf<RULE>::value ? delta[k] : 0.f);
    apply_rule<RULE, R>(a, cs, ds, s);
#pragma unroll
    for (int r = 0; r < R; ++r) {
      p.w[r][k] = a[r];
      if (MIRROR) p.m[r][k] = __float2bfloat16_rn(a[r]);
    }
    if (c != nullptr) c[k] = cs;
    if (IsBmuf<RULE>::value) delta[k] = ds;
  }
}

template <int RULE, int R>
static ss_status launch_r(const SyncPtrs& p, bool mirror, float* c, float* delta, int64_t n,
                          const SyncScalars& s, cudaStream_t st) {
  const int64_t n4 = n / 4;
  int64_t blocks = (n4 + 255) / 256;
  if (blocks == 0) blocks = 1;
  if (blocks > 0x7fffffffLL) return SS_ERR_SHAPE;
  if (mirror)
    { SS_TIMED("sync_kernel", st);
    sync_kernel<RULE, R, true><<<(unsigned)blocks, 256, 0, st>>>(p, c, delta, n4, n, s);
    }
  else
    { SS_TIMED("sync_kernel", st);
    sync_kernel<RULE, R, false><<<(unsigned)blocks, 256, 0, st>>>(p, c, delta, n4, n, s);
    }
  SS_LAUNCH_OK();
  return SS_OK;
}

template <int RULE>
static ss_status launch(int R, const SyncPtrs& p, bool mirror, float* c, float* delta, int64_t n,
                        const SyncScalars& s, cudaStream_t st) {
  switch (R) {
#define SS_CASE(K) case K: return launch_r<RULE, K>(p, mirror, c, delta, n, s, st);
    SS_CASE(1) SS_CASE(2) SS_CASE(3) SS_CASE(4) SS_CASE(5) SS_CASE(6) SS_CASE(7) SS_CASE(8)
    SS_CASE(9) SS_CASE(10) SS_CASE(11) SS_CASE(12) SS_CASE(13) SS_CASE(14) SS_CASE(15) SS_CASE(16)
#undef SS_CASE
  }
  return SS_ERR_SHAPE;
}

static ss_status collect(float* const* w, int R, int64_t n, void* const* w_bf16, float alpha, SyncPtrs* p) {
  if (!w) return SS_ERR_NULL;
  if (R < 1 || R > kMaxR || n < 0) return SS_ERR_SHAPE;
  if (!(alpha >= 0.f && alpha <= 1.f)) return SS_ERR_RANGE;
  for (int r = 0; r < kMaxR; ++r) { p->w[r] = nullptr; p->m[r] = nullptr; }
  for (int r = 0; r < R; ++r) {
    if (!w[r]) return SS_ERR_NULL;
    if (!aligned16(w[r])) return SS_ERR_ALIGN;
    p->w[r] = w[r];
    if (w_bf16) {
      if (!w_bf16[r]) return SS_ERR_NULL;
      if ((reinterpret_cast<uintptr_t>(w_bf16[r]) & 7u) != 0) return SS_ERR_ALIGN;
      p->m[r] = reinterpret_cast<__nv_bfloat16*>(w_bf16[r]);
    }
  }
  return check_arch();
}

}  // namespace ss

extern "C" {

ss_status ss_sync_easgd(float* const* w, int R, float* center, int64_t n, float alpha, int flags,
                        void* const* w_bf16, ss_stream stream) {
  ss::SyncPtrs p;
  if (!center) return SS_ERR_NULL;
  ss_status st = ss::collect(w, R, n, w_bf16, alpha, &p);
  if (st != SS_OK) return st;
  if (!ss::aligned16(center)) return SS_ERR_ALIGN;
  if (n == 0) return SS_OK;
  ss::SyncScalars s{alpha, 0.f, 0.f, 1.f / (float)R};
  if (flags & SS_SYNC_EASGD_LITERAL)
    return ss::launch<ss::RULE_EASGD_LITERAL>(R, p, w_bf16 != nullptr, center, nullptr, n, s, ss::as_stream(stream));
  return ss::launch<ss::RULE_EASGD>(R, p, w_bf16 != nullptr, center, nullptr, n, s, ss::as_stream(stream));
}

ss_status ss_sync_ma(float* const* w, int R, float* global_out, int64_t n, float alpha, int flags,
                     void* const* w_bf16, ss_stream stream) {
  (void)flags;
  ss::SyncPtrs p;
  ss_status st = ss::collect(w, R, n, w_bf16, alpha, &p);
  if (st != SS_OK) return st;
  if (global_out && !ss::aligned16(global_out)) return SS_ERR_ALIGN;
  if (n == 0) return SS_OK;
  ss::SyncScalars s{alpha, 0.f, 0.f, 1.f / (float)R};
  return ss::launch<ss::RULE_MA>(R, p, w_bf16 != nullptr, global_out, nullptr, n, s, ss::as_stream(stream));
}

ss_status ss_sync_bmuf(float* const* w, int R, float* global, float* delta, int64_t n,
                       float alpha, float eta, float mu, int flags, void* const* w_bf16, ss_stream stream) {
  ss::SyncPtrs p;
  if (!global || !delta) return SS_ERR_NULL;
  ss_status st = ss::collect(w, R, n, w_bf16, alpha, &p);
  if (st != SS_OK) return st;
  if (!ss::aligned16(global) || !ss::aligned16(delta)) return SS_ERR_ALIGN;
  if (!(mu >= 0.f && mu < 1.f) || !(eta >= 0.f)) return SS_ERR_RANGE;
  if (n == 0) return SS_OK;
  ss::SyncScalars s{alpha, eta, mu, 1.f / (float)R};
  if (flags & SS_SYNC_BMUF_NESTEROV)
    return ss::launch<ss::RULE_BMUF_NESTEROV>(R, p, w_bf16 != nullptr, global, delta, n, s, ss::as_stream(stream));
  return ss::launch<ss::RULE_BMUF>(R, p, w_bf16 != nullptr, global, delta, n, s, ss::as_stream(stream));
}

// ------------------------------------------------------------------------------------------------
// The shadow thread (Section 3.2, Algorithm 1): a host thread that does nothing but enqueue one
// synchronisation pass after another on the stream it was given, with a bounded number of passes in
// flight.  It shares no event with any training stream and knows nothing about training.
// ------------------------------------------------------------------------------------------------
}  // extern "C"

#include <atomic>
#include <chrono>
#include <thread>

struct ss_shadow {
  int rule, R, flags, device, max_in_flight, pause_us;
  float* w[ss::kMaxR];
  void* m[ss::kMaxR];
  bool mirror;
  float *center, *delta;
  int64_t n, max_rounds;
  float alpha, eta, mu;
  cudaStream_t stream;
  std::atomic<int64_t> rounds{0};
  std::atomic<int> stop{0};
  std::atomic<int> paused{0};      // set by ss_shadow_pause; the thread drains its passes and idles while it is set
  std::atomic<int> idle{0};        // the thread's answer: 1 while it idles with nothing queued
  std::atomic<int> status{SS_OK};
  std::thread thread;
};

static void shadow_main(ss_shadow* h) {
  if (cudaSetDevice(h->device) != cudaSuccess) { h->status = SS_ERR_CUDA; return; }
  const int depth = h->max_in_flight < 1 ? 1 : (h->max_in_flight > 8 ? 8 : h->max_in_flight);
  cudaEvent_t ev[8];
  for (int i = 0; i < depth; ++i)
    if (cudaEventCreateWithFlags(&ev[i], cudaEventDisableTiming) != cudaSuccess) { h->status = SS_ERR_CUDA; return; }
  int64_t k = 0;
  while (!h->stop.load(std::memory_order_relaxed) && k < h->max_rounds) {
    if (h->paused.load(std::memory_order_acquire)) {
      // every pass enqueued so far has completed before the pause is acknowledged
      for (int i = 0; i < depth && i < k; ++i) cudaEventSynchronize(ev[i]);
      h->idle.store(1, std::memory_order_release);
      while (h->paused.load(std::memory_order_acquire) && !h->stop.load(std::memory_order_relaxed))
        std::this_thread::sleep_for(std::chrono::microseconds(20));
      h->idle.store(0, std::memory_order_release);
      continue;
    }
    const int slot = (int)(k % depth);
    if (k >= depth && cudaEventSynchronize(ev[slot]) != cudaSuccess) { h->status = SS_ERR_CUDA; break; }
    ss_status st;
    void* const* mir = h->mirror ? h->m : nullptr;
    if (h->rule == 0) st = ss_sync_easgd(h->w, h->R, h->center, h->n, h->alpha, h->flags, mir, h->stream);
    else if (h->rule == 1) st = ss_sync_ma(h->w, h->R, h->center, h->n, h->alpha, h->flags, mir, h->stream);
    else st = ss_sync_bmuf(h->w, h->R, h->center, h->delta, h->n, h->alpha, h->eta, h->mu, h->flags, mir, h->stream);
    if (st != SS_OK) { h->status = st; break; }
    cudaEventRecord(ev[slot], h->stream);
    h->rounds.store(++k, std::memory_order_relaxed);
    if (h->pause_us > 0) std::this_thread::sleep_for(std::chrono::microseconds(h->pause_us));
  }
  for (int i = 0; i < depth; ++i) {
    cudaEventSynchronize(ev[i]);
    cudaEventDestroy(ev[i]);
  }
  h->idle.store(1, std::memory_order_release);             // ended: nothing in flight
}

extern "C" {

ss_status ss_shadow_start(ss_shadow** out, int rule, float* const* w, int R, float* center, float* delta, int64_t n,
                          float alpha, float eta, float mu, int flags, void* const* w_bf16, ss_stream stream,
                          int max_in_flight, int pause_us, int64_t max_rounds) {
  if (!out || !w || !center) return SS_ERR_NULL;
  if (rule < 0 || rule > 2 || R < 1 || R > ss::kMaxR || n < 0 || max_rounds < 0) return SS_ERR_SHAPE;
  if (rule == 2 && !delta) return SS_ERR_NULL;
  if (!(alpha >= 0.f && alpha <= 1.f)) return SS_ERR_RANGE;
  ss_status st = ss::check_arch();
  if (st != SS_OK) return st;
  ss_shadow* h = new ss_shadow();
  h->rule = rule; h->R = R; h->flags = flags; h->max_in_flight = max_in_flight; h->pause_us = pause_us;
  h->mirror = w_bf16 != nullptr;
  for (int r = 0; r < ss::kMaxR; ++r) { h->w[r] = r < R ? w[r] : nullptr; h->m[r] = (w_bf16 && r < R) ? w_bf16[r] : nullptr; }
  h->center = center; h->delta = delta; h->n = n; h->max_rounds = max_rounds;
  h->alpha = alpha; h->eta = eta; h->mu = mu;
  h->stream = ss::as_stream(stream);
  if (cudaGetDevice(&h->device) != cudaSuccess) { delete h; return SS_ERR_CUDA; }
  h->thread = std::thread(shadow_main, h);
  *out = h;
  return SS_OK;
}

int64_t ss_shadow_rounds(const ss_shadow* h) { return h ? h->rounds.load(std::memory_order_relaxed) : -1; }

ss_status ss_shadow_pause(ss_shadow* h, int paused) {
  if (!h) return SS_ERR_NULL;
  h->paused.store(paused ? 1 : 0, std::memory_order_release);
  if (!paused) return SS_OK;
  // wait (at most ~30 s) until the thread has drained its queued passes and idles, or has ended by itself
  for (int i = 0; i < 1500000; ++i) {
    if (h->idle.load(std::memory_order_acquire) || h->status.load() != SS_OK)
      return (ss_status)h->status.load();
    std::this_thread::sleep_for(std::chrono::microseconds(20));
  }
  return SS_ERR_CUDA;
}

ss_status ss_shadow_stop(ss_shadow* h, int64_t* rounds_out) {
  if (!h) return SS_ERR_NULL;
  h->stop.store(1);
  if (h->thread.joinable()) h->thread.join();
  if (rounds_out) *rounds_out = h->rounds.load();
  const ss_status st = (ss_status)h->status.load();
  delete h;
  return st;
}

}  // extern "C"
