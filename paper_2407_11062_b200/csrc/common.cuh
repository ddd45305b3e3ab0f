// Shared device/host helpers of the sm_100a kernels (not part of the C ABI).
#pragma once

#include <atomic>

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "eqat.h"

namespace eqat {

// Codes written to the device status word by a kernel that abandons a wait.
enum WaitSite : int {
  WAIT_NONE = 0,
  WAIT_PRODUCER_EMPTY = 1,    // TMA producer waiting for a free pipeline stage
  WAIT_MMA_FULL = 2,          // MMA issuer waiting for a filled stage
  WAIT_MMA_ACC_EMPTY = 3,     // MMA issuer waiting for the epilogue to drain TMEM
  WAIT_EPI_ACC_FULL = 4,      // epilogue waiting for the accumulator
  WAIT_DEQ_OPERAND_EMPTY = 5, // dequantiser waiting for a free operand stage
  WAIT_TEARDOWN = 6,          // producer draining its copies in flight
  WAIT_STREAM_EMPTY = 7,      // streaming kernels: producer waiting for a free ring stage
  WAIT_STREAM_FULL = 8,       // streaming kernels: consumers waiting for a filled ring stage
  WAIT_SELFTEST = 9           // eqat_selftest_wait_expiry: a wait that nothing ever satisfies
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? EQAT_OK : EQAT_ERR_CUDA; }

// Host-side state that belongs to a device rather than to the process (a kernel attribute lives in the
// device's context, the SM count is a property of the device).  Devices beyond the table are served
// uncached.
constexpr int kMaxCachedDevices = 64;

inline int current_device() {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

// Number of SMs of the current device (0 on error).
inline int sm_count() {
  static std::atomic<int> cache[kMaxCachedDevices];
  const int dev = current_device();
  if (dev < 0) return 0;
  if (dev < kMaxCachedDevices) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int v = 0;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (dev < kMaxCachedDevices) cache[dev].store(v, std::memory_order_relaxed);
  return v;
}

// Raises a kernel's dynamic shared-memory limit once per device (one flag set per kernel: declare a
// function-local static SmemOptIn next to the launch).
struct SmemOptIn {
  std::atomic<uint64_t> done{0};
  template <typename K>
  bool ensure(K kernel, int bytes) {
    const int dev = current_device();
    if (dev < 0) return false;
    const uint64_t bit = 1ull << (dev & 63);
    if (dev < kMaxCachedDevices && (done.load(std::memory_order_acquire) & bit)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (dev < kMaxCachedDevices) done.fetch_or(bit, std::memory_order_release);
    return true;
  }
};

}  // namespace eqat
