// Shared host/device helpers of the SAPO B200 library (no method arithmetic here).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sapo.h"

namespace sapo {

// OR a device-detected condition into the caller's status word.
__device__ __forceinline__ void raise_status(int32_t* status, int32_t bit) {
  if (status != nullptr) atomicOr(status, bit);
}

// Checked builds (-DSAPO_BOUNDS_CHECK; the stand-in for a memory checker): every index a kernel
// computes from its arguments or its data before a global-memory access is compared with the
// extent of the array; a violation is counted and the access left out.  Each translation unit
// counts for itself (sapo_debug_bounds_violations adds the counters up).  In regular builds the
// macro is constant true and costs nothing.
#ifdef SAPO_BOUNDS_CHECK
static __device__ unsigned long long g_bounds_violations = 0;
#define SAPO_IN_BOUNDS(cond) ((cond) ? true : (atomicAdd(&g_bounds_violations, 1ull), false))
static inline long long read_bounds_violations() {
  unsigned long long v = 0;
  return cudaMemcpyFromSymbol(&v, g_bounds_violations, sizeof(v)) == cudaSuccess ? (long long)v : -1;
}
#else
#define SAPO_IN_BOUNDS(cond) (true)
static inline long long read_bounds_violations() { return 0; }
#endif
long long bounds_violations_pack();
long long bounds_violations_lmhead();

inline int check_launch() {
  return cudaGetLastError() == cudaSuccess ? SAPO_OK : SAPO_ERR_CUDA;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int MAX_DEVICES = 64;   // devices of one process the per-device caches below cover

// index of the current device, or -1 (no device, or more devices than the caches cover)
inline int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -1;
  return dev;
}

// SM count of the current device (looked up once per device)
inline int sm_count() {
  static int n[MAX_DEVICES] = {0};
  const int dev = current_device();
  if (dev < 0) return 0;
  if (n[dev] == 0 && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 0;
  return n[dev];
}

// Blocks of `threads` threads of `kernel` an SM holds at once.  The grid-stride kernels that stream
// through device memory are launched with at most that many blocks per SM: a larger grid runs in
// waves, and a last wave that is not full leaves bandwidth unused.
template <class Kernel>
inline int resident_blocks_per_sm(Kernel kernel, int threads) {
  int n = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, 0) != cudaSuccess || n < 1) n = 1;
  return n;
}

// Optional per-kernel timing and launch counting (see sapo_timing_* in sapo.h).
// A KernelScope brackets one kernel launch with two CUDA events when timing is on.
struct KernelTimer {
  static constexpr int MAX_PAIRS = 16384;
  bool enabled = false;
  bool created = false;
  int n = 0;
  int id[MAX_PAIRS];
  cudaEvent_t start[MAX_PAIRS], stop[MAX_PAIRS];
  long long launches = 0;
};
KernelTimer& kernel_timer();

struct KernelScope {
  cudaStream_t st; int slot;
  KernelScope(int kernel_id, cudaStream_t s) : st(s), slot(-1) {
    KernelTimer& t = kernel_timer();
    ++t.launches;
    if (t.enabled && t.created && t.n < KernelTimer::MAX_PAIRS) {
      slot = t.n++;
      t.id[slot] = kernel_id;
      cudaEventRecord(t.start[slot], st);
    }
  }
  ~KernelScope() { if (slot >= 0) cudaEventRecord(kernel_timer().stop[slot], st); }
};

template <typename T>
__host__ __device__ constexpr T ceil_div(T a, T b) { return (a + b - 1) / b; }
template <typename T>
__host__ __device__ constexpr T round_up(T a, T b) { return ceil_div(a, b) * b; }

}  // namespace sapo
