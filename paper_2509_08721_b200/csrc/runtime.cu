// Host-side runtime helpers of the library: status text, launch counting and the optional
// per-kernel timing used by benchmarks.
#include "common.cuh"

namespace sapo {
KernelTimer& kernel_timer() {
  static KernelTimer t;
  return t;
}
}  // namespace sapo

extern "C" int sapo_timing_enable(int32_t on) {
  sapo::KernelTimer& t = sapo::kernel_timer();
  if (on && !t.created) {
    for (int i = 0; i < sapo::KernelTimer::MAX_PAIRS; ++i) {
      if (cudaEventCreate(&t.start[i]) != cudaSuccess || cudaEventCreate(&t.stop[i]) != cudaSuccess)
        return SAPO_ERR_CUDA;
    }
    t.created = true;
  }
  t.enabled = on != 0;
  t.n = 0;
  return SAPO_OK;
}

extern "C" int sapo_timing_read(float* h_ms, int32_t* h_launches) {
  sapo::KernelTimer& t = sapo::kernel_timer();
  if (!h_ms || !h_launches) return SAPO_ERR_INVALID_ARG;
  for (int k = 0; k < SAPO_K_COUNT; ++k) { h_ms[k] = 0.f; h_launches[k] = 0; }
  for (int i = 0; i < t.n; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(t.stop[i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, t.start[i], t.stop[i]) != cudaSuccess)
      return SAPO_ERR_CUDA;
    h_ms[t.id[i]] += ms;
    h_launches[t.id[i]] += 1;
  }
  t.n = 0;
  return SAPO_OK;
}

extern "C" int64_t sapo_debug_bounds_violations(void) {
#ifdef SAPO_BOUNDS_CHECK
  const long long a = sapo::bounds_violations_pack(), b = sapo::bounds_violations_lmhead();
  return (a < 0 || b < 0) ? -2 : a + b;
#else
  return -1;      // not a checked build
#endif
}

extern "C" int64_t sapo_launch_count(void) { return sapo::kernel_timer().launches; }

extern "C" const char* sapo_status_string(int32_t code) {
  switch (code) {
    case SAPO_OK: return "ok";
    case SAPO_ERR_INVALID_ARG: return "invalid argument";
    case SAPO_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case SAPO_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SAPO_ERR_CUDA: return "CUDA error";
    case SAPO_ERR_STATIC_SCRATCH_EXCEEDED: return "sizes exceed the built-in static scratch";
    default: return "unknown code";
  }
}
