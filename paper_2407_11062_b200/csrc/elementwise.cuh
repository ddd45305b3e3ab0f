// Host launchers of the streaming kernels (arguments already validated).
#pragma once
#include <cuda_runtime.h>
#include "eqat.h"

namespace eqat {
int launch_fakequant(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* What, cudaStream_t st);
int launch_ste_bwd(const eqat_desc& d, const eqat_bf16* dWhat, const eqat_bf16* W, const float* s, const float* z,
                   eqat_bf16* dW, float* ds, float* dz, cudaStream_t st);
int launch_minmax(const eqat_desc& d, const eqat_bf16* W, float* s, float* z, cudaStream_t st);
int launch_quantize_pack(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, uint8_t* packed,
                         uint8_t* z8, eqat_fp16* s16, cudaStream_t st);
int launch_pack(const eqat_desc& d, const uint8_t* codes, uint8_t* packed, cudaStream_t st);
int launch_unpack(const eqat_desc& d, const uint8_t* packed, uint8_t* codes, cudaStream_t st);
int launch_pack_zeros(const eqat_desc& d, const uint8_t* z8, uint8_t* packed, cudaStream_t st);
int launch_unpack_zeros(const eqat_desc& d, const uint8_t* packed, uint8_t* z8, cudaStream_t st);
// TMA-staged variants for groups of at most 256 elements (stream.cu).
int launch_fakequant_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* What,
                            cudaStream_t st);
int launch_ste_bwd_stream(const eqat_desc& d, const eqat_bf16* dWhat, const eqat_bf16* W, const float* s,
                          const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st);
int launch_minmax_stream(const eqat_desc& d, const eqat_bf16* W, float* s, float* z, cudaStream_t st);
int launch_quantize_pack_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z,
                                uint8_t* packed, uint8_t* z8, eqat_fp16* s16, cudaStream_t st);
// Self-test of the streaming kernels' bounded wait (one warp, 1 ms, a barrier nothing signals).
int launch_wait_expiry_stream(cudaStream_t st);
// Reads and clears the streaming kernels' status word ({status, wait site}); synchronises.
int read_stream_status(int* status, int* detail);
}  // namespace eqat
