// Host launchers of the tcgen05 GEMM kernels (arguments already validated).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include "eqat.h"

namespace eqat {

// Tensor map of a bf16 matrix [outer, inner] row-major for copies of 64 elements (128 bytes) x box_outer rows
// with the 128-byte swizzle (the driver's encoder is looked up once; false if it is missing or refuses).
bool make_tmap_bf16(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer);
// Tensor map of a byte matrix [outer, inner_bytes] row-major for copies of box_bytes (at most 128) x box_outer
// rows with the 128-byte swizzle; bytes outside the matrix are delivered as zeros.
bool make_tmap_u8(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t outer, uint32_t box_bytes,
                  uint32_t box_outer);

// Y[T,out] = X[T,in] * What[out,in]^T
int launch_dense_fwd(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* What, eqat_bf16* Y, cudaStream_t st);
// dX[T,in] = dY[T,out] * What[out,in]
int launch_dense_dx(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* What, eqat_bf16* dX, cudaStream_t st);
// dWhat[out,in] = dY[T,out]^T * X[T,in]
int launch_dense_dw(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, eqat_bf16* dWhat, cudaStream_t st);
// The same contraction with Eqs. 3-5 applied in its epilogue (group <= 256): writes dW, ds and optionally dz;
// the gradient of W_hat is never stored.
int launch_dense_dw_ste(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, const eqat_bf16* W, const float* s,
                        const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st);
// Y = X * W_hat^T and dX = dY * W_hat with W_hat = Eq. 2 of Eq. 1 of the latent weight, computed inside the
// kernel on each tile of W after it has been copied to shared memory; W_hat is not stored.  The group must be a
// power of two up to 256 or the whole row.
int launch_latent_fwd(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* W, const float* s, const float* z,
                      eqat_bf16* Y, cudaStream_t st);
int launch_latent_dx(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* W, const float* s, const float* z,
                     eqat_bf16* dX, cudaStream_t st);
// Y = X * dequant(Wq)^T and dX = dY * dequant(Wq), codes expanded in shared memory.  zq: zero points as uint8 or,
// with desc.zero_point_format == EQAT_ZP_FP16, as fp16 values.
int launch_packed_fwd(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                      const void* zq, eqat_bf16* Y, cudaStream_t st);
int launch_packed_dx(const eqat_desc& d, const eqat_bf16* dY, const uint8_t* Wq, const eqat_fp16* s16,
                     const void* zq, eqat_bf16* dX, cudaStream_t st);
// ds (and optionally dz) reduced in the epilogue of dY^T * X.  One group per row needs
// packed_ds_workspace_bytes(d) bytes of scratch for the per-tile partial sums (0 otherwise).
size_t packed_ds_workspace_bytes(const eqat_desc& d);
int launch_packed_ds(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* dY, const uint8_t* Wq,
                     const void* zq, const eqat_fp16* s16, float* ds, float* dz, void* workspace, cudaStream_t st);

// Self-test of the bounded wait: one warp waits 1 ms for a barrier that is never signalled, records
// EQAT_ERR_TIMEOUT / WAIT_SELFTEST in the status word and returns.
int launch_wait_expiry_gemm(cudaStream_t st);

// Reads and clears the device status word ({status, wait site}); synchronises.
int read_device_status(int* status, int* detail);

}  // namespace eqat
