// Optional per-kernel timers: when switched on, every kernel launch of the library is bracketed by a pair
// of CUDA events recorded on the launching stream; ss_profile_collect() reads the elapsed times.
// Off by default; must stay off while a stream is being captured into a CUDA graph.
#pragma once
#include <cuda_runtime.h>

namespace ss {

extern int g_profile_on;

struct ProfScope {
  int slot;
  cudaStream_t st;
  ProfScope(const char* name, cudaStream_t stream);
  ~ProfScope();
};

}  // namespace ss

#define SS_PROF_CAT2(a, b) a##b
#define SS_PROF_CAT(a, b) SS_PROF_CAT2(a, b)
// SS_TIMED("name", stream); kernel<<<...>>>(...);   -- times everything up to the end of the enclosing block
#define SS_TIMED(name, stream) ss::ProfScope SS_PROF_CAT(prof_scope_, __LINE__)(name, stream)
