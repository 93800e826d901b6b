// Per-kernel timers (see profile.cuh).
#include <mutex>
#include <string.h>
#include <vector>
#include "common.cuh"
#include "profile.cuh"

namespace ss {

int g_profile_on = 0;

namespace {
struct Rec { const char* name; cudaEvent_t a, b; bool closed; };
std::mutex g_mu;
std::vector<Rec> g_recs;
std::vector<std::pair<cudaEvent_t, cudaEvent_t>> g_pool;
constexpr size_t kMaxRecs = 1 << 16;
}  // namespace

ProfScope::ProfScope(const char* name, cudaStream_t stream) : slot(-1), st(stream) {
  if (!g_profile_on) return;
  std::lock_guard<std::mutex> lk(g_mu);
  if (g_recs.size() >= kMaxRecs) return;
  Rec r{name, nullptr, nullptr, false};
  if (!g_pool.empty()) {
    r.a = g_pool.back().first; r.b = g_pool.back().second;
    g_pool.pop_back();
  } else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) {
    return;
  }
  cudaEventRecord(r.a, st);
  slot = (int)g_recs.size();
  g_recs.push_back(r);
}

ProfScope::~ProfScope() {
  if (slot < 0) return;
  std::lock_guard<std::mutex> lk(g_mu);
  if ((size_t)slot < g_recs.size()) {
    cudaEventRecord(g_recs[slot].b, st);
    g_recs[slot].closed = true;
  }
}

}  // namespace ss

extern "C" {

int ss_profile(int on) {
  const int prev = ss::g_profile_on;
  ss::g_profile_on = on ? 1 : 0;
  return prev;
}

int ss_profile_collect(char* names, size_t names_len, float* ms, int max_records) {
  using namespace ss;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  std::lock_guard<std::mutex> lk(g_mu);
  int n = 0;
  size_t off = 0;
  for (const Rec& r : g_recs) {
    float t = 0.f;
    if (r.closed && cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess && n < max_records && names && ms) {
      const size_t len = strlen(r.name);
      if (off + len + 1 < names_len) {
        memcpy(names + off, r.name, len);
        names[off + len] = '\n';
        off += len + 1;
        ms[n++] = t;
      }
    }
    g_pool.emplace_back(r.a, r.b);
  }
  if (names && names_len) names[off < names_len ? off : names_len - 1] = 0;
  g_recs.clear();
  return n;
}

}  // extern "C"
