// Host launcher of the packed-weight matrix-vector forward (arguments already validated).
#pragma once
#include <cuda_runtime.h>
#include "eqat.h"

namespace eqat {

// True when the few-token kernel handles this problem: groups of at least 64 elements, at most 64 tokens, staged
// activations of at least one token that fit in the shared memory of a CTA, and, where the tokens need several
// launches, a cost estimate below the tiled kernel's.
bool packed_gemv_applies(const eqat_desc& d);
// Y[T,out] = X[T,in] * dequant(Wq)^T for a problem packed_gemv_applies() accepted
int launch_packed_gemv(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                       const void* zq, eqat_bf16* Y, cudaStream_t st);

// Self-test of the matrix-vector kernel's bounded wait (one warp, 1 ms, a barrier nothing signals).
int launch_wait_expiry_gemv(cudaStream_t st);
// Reads and clears the status word of the matrix-vector kernels ({status, wait site}); synchronises.
int read_gemv_status(int* status, int* detail);

}  // namespace eqat
