// Shared device/host helpers of the sm_100a kernels (not part of the C ABI).
#pragma once

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
  WAIT_TEARDOWN = 6           // producer draining its copies in flight
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? EQAT_OK : EQAT_ERR_CUDA; }

}  // namespace eqat
