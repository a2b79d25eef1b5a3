// Per-kernel-class timing with CUDA events recorded on the stream each kernel is launched on
// (the main stream, or the side stream of the reductions and column sums; the side stream is
// joined into the main one before collect() waits).
#include <stdio.h>
#include <stdlib.h>

#include "kernels.h"

namespace mbd {

bool pdl_enabled() {
  static const bool on = getenv("MBD_NO_PDL") == nullptr;
  return on;
}

cudaEvent_t Profiler::get_event() {
  if (n_pool > 0) return pool[--n_pool];
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

void Profiler::begin(int cls, double w, cudaStream_t launch_stream) {
  total_launches++;
  if (!on) return;
  cur = launch_stream ? launch_stream : stream;
  if (n_pending == cap) {
    cap = cap ? cap * 2 : 256;
    pending = static_cast<Pending*>(realloc(pending, cap * sizeof(Pending)));
  }
  Pending& p = pending[n_pending];
  p.a = get_event();
  p.b = get_event();
  p.cls = cls;
  work[cls] += w;
  launches[cls]++;
  cudaEventRecord(p.a, cur);
}

void Profiler::end() {
  if (!on) return;
  cudaEventRecord(pending[n_pending].b, cur);
  n_pending++;
}

void Profiler::collect() {
  cudaStreamSynchronize(stream);
  // MBD_PROF_TIMELINE=1: start (since the first bracketed launch) and duration of every launch, both streams
  const bool timeline = n_pending > 0 && getenv("MBD_PROF_TIMELINE") != nullptr;
  for (int i = 0; i < n_pending; ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, pending[i].a, pending[i].b) == cudaSuccess) ms[pending[i].cls] += t;
    if (timeline) {
      float t0 = 0.f;
      cudaEventElapsedTime(&t0, pending[0].a, pending[i].a);
      fprintf(stderr, "timeline %4d  class %2d  start %10.3f ms  duration %8.3f ms\n", i, pending[i].cls, t0, t);
    }
    if (n_pool + 2 > pool_cap) {
      pool_cap = pool_cap ? pool_cap * 2 : 512;
      pool = static_cast<cudaEvent_t*>(realloc(pool, pool_cap * sizeof(cudaEvent_t)));
    }
    pool[n_pool++] = pending[i].a;
    pool[n_pool++] = pending[i].b;
  }
  n_pending = 0;
  (void)cudaGetLastError();
}

void Profiler::reset() {
  collect();
  for (int i = 0; i < NCLS; ++i) { ms[i] = 0; work[i] = 0; launches[i] = 0; }
}

void Profiler::destroy() {
  collect();
  for (int i = 0; i < n_pool; ++i) cudaEventDestroy(pool[i]);
  free(pool);
  free(pending);
  pool = nullptr; pending = nullptr; n_pool = pool_cap = cap = 0;
}

}  // namespace mbd
