// Host launcher of the packed-weight matrix-vector forward (arguments already validated).
#pragma once
#include <cuda_runtime.h>
#include "eqat.h"

namespace eqat {

constexpr int kGemvMaxTokens = 4;

// True when a small-batch kernel handles this problem: groups of at least 64 elements and either byte zero points
// (with packed rows that are multiples of 16 bytes) and at most 64 tokens (tensor-core kernel, at most eight tokens per launch; several launches only
// while they are cheaper than the tiled kernel), or at most kGemvMaxTokens tokens and activations (as fp32) that fit
// in the shared memory of one CTA.
bool packed_gemv_applies(const eqat_desc& d);
// Y[T,out] = X[T,in] * dequant(Wq)^T for a problem packed_gemv_applies() accepted
int launch_packed_gemv(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                       const void* zq, eqat_bf16* Y, cudaStream_t st);

// Self-test of the matrix-vector kernel's bounded wait (one warp, 1 ms, a barrier nothing signals).
int launch_wait_expiry_gemv(cudaStream_t st);
// Reads and clears the status word of the matrix-vector kernels ({status, wait site}); synchronises.
int read_gemv_status(int* status, int* detail);

}  // namespace eqat
