// C ABI (include/eqat.h): argument validation on the host, then launches.
#include <stdint.h>

#include "common.cuh"
#include "elementwise.cuh"
#include "gemm.cuh"
#include "gemv.cuh"

namespace {

using namespace eqat;

constexpr int kMaxFusedSteGroup = 256;   // longest group the weight-gradient epilogue reduces by itself

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }

// Geometry every entry point shares.
int check_weight_desc(const eqat_desc* d) {
  if (d == nullptr) return EQAT_ERR_NULL;
  if (d->zero_point_format != EQAT_ZP_U8 && d->zero_point_format != EQAT_ZP_FP16) return EQAT_ERR_UNSUPPORTED;
  if (d->bits < 2 || d->bits > 4) return EQAT_ERR_UNSUPPORTED;
  if (d->dz_mode != 0 && d->dz_mode != 1) return EQAT_ERR_UNSUPPORTED;
  if (d->out_features <= 0 || d->in_features <= 0 || d->group <= 0) return EQAT_ERR_SHAPE;
  if (d->in_features % 128 != 0) return EQAT_ERR_SHAPE;
  if (d->group % 32 != 0 || d->in_features % d->group != 0) return EQAT_ERR_SHAPE;
  if (d->group <= 256 && !is_pow2(d->group)) return EQAT_ERR_UNSUPPORTED;
  if (d->group > 32768) return EQAT_ERR_UNSUPPORTED;
  if ((int64_t)d->out_features * d->in_features > ((int64_t)1 << 34)) return EQAT_ERR_SHAPE;
  return EQAT_OK;
}

// Entry points that read no packed zero points take the default format only.
int check_plain_desc(const eqat_desc* d) {
  const int rc = check_weight_desc(d);
  if (rc != EQAT_OK) return rc;
  return d->zero_point_format == EQAT_ZP_U8 ? EQAT_OK : EQAT_ERR_UNSUPPORTED;
}

int check_gemm_desc(const eqat_desc* d, bool packed) {
  const int rc = packed ? check_weight_desc(d) : check_plain_desc(d);
  if (rc != EQAT_OK) return rc;
  if (d->tokens <= 0 || d->tokens > (int64_t)1 << 30) return EQAT_ERR_SHAPE;
  if (d->out_features % 64 != 0) return EQAT_ERR_SHAPE;
  // packed kernels: a group is a power of two up to 256, or the whole row
  if (packed && d->group > 256 && d->group != d->in_features) return EQAT_ERR_UNSUPPORTED;
  return EQAT_OK;
}

// The kernels that fake-quantise the latent weight tile by tile index groups with a shift, or not at all.
inline bool latent_group_ok(const eqat_desc* d) { return d->group <= 256 || d->group == d->in_features; }

template <typename... P>
int check_ptrs(P... ptrs) {
  const void* v[] = {static_cast<const void*>(ptrs)...};
  for (const void* p : v)
    if (p == nullptr) return EQAT_ERR_NULL;
  for (const void* p : v)
    if (!aligned16(p)) return EQAT_ERR_ALIGN;
  return EQAT_OK;
}

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

// Host-side validation of the layer entry points, one function each, so that the block-level calls can check
// every linear before the first launch.
int v_fakequant_fwd(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* W, const float* s, const float* z,
                    const eqat_bf16* Y, const eqat_bf16* W_hat) {
  int rc = check_gemm_desc(d, false);
  if (rc != EQAT_OK) return rc;
  if ((rc = check_ptrs(X, W, s, z, Y)) != EQAT_OK) return rc;
  if (W_hat == nullptr) return latent_group_ok(d) ? EQAT_OK : EQAT_ERR_UNSUPPORTED;
  return aligned16(W_hat) ? EQAT_OK : EQAT_ERR_ALIGN;
}

int v_fakequant_bwd(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* dY, const eqat_bf16* W, const float* s,
                    const float* z, const eqat_bf16* W_hat, const eqat_bf16* dX, const eqat_bf16* dW, const float* ds,
                    const float* dz, const void* workspace, size_t workspace_bytes) {
  int rc = check_gemm_desc(d, false);
  if (rc != EQAT_OK) return rc;
  if ((rc = check_ptrs(X, dY, W, s, z, dX, dW, ds)) != EQAT_OK) return rc;
  if (dz != nullptr && !aligned16(dz)) return EQAT_ERR_ALIGN;
  if (W_hat != nullptr && !aligned16(W_hat)) return EQAT_ERR_ALIGN;
  if (W_hat == nullptr && !latent_group_ok(d)) return EQAT_ERR_UNSUPPORTED;
  if (d->group > kMaxFusedSteGroup) {
    const size_t need = (size_t)d->out_features * d->in_features * sizeof(eqat_bf16);
    if (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
      return EQAT_ERR_WORKSPACE;
  }
  return EQAT_OK;
}

int v_packed_fwd(const eqat_desc* d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* z,
                 const eqat_bf16* Y) {
  const int rc = check_gemm_desc(d, true);
  return rc != EQAT_OK ? rc : check_ptrs(X, Wq, s16, z, Y);
}

int v_packed_bwd_ds(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* dY, const uint8_t* Wq, const void* z,
                    const eqat_fp16* s16, const float* ds, const float* dz, const void* workspace,
                    size_t workspace_bytes) {
  int rc = check_gemm_desc(d, true);
  if (rc != EQAT_OK) return rc;
  if ((rc = check_ptrs(X, dY, Wq, z, ds)) != EQAT_OK) return rc;
  if (dz != nullptr && (rc = check_ptrs(dz, s16)) != EQAT_OK) return rc;
  const size_t need = packed_ds_workspace_bytes(*d);
  if (need != 0 && (workspace == nullptr || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0))
    return EQAT_ERR_WORKSPACE;
  return EQAT_OK;
}

#define EQAT_TRY(expr)            \
  do {                            \
    const int rc__ = (expr);      \
    if (rc__ != EQAT_OK) return rc__; \
  } while (0)

}  // namespace

extern "C" {

const char* eqat_status_string(int status) {
  switch (status) {
    case EQAT_OK: return "ok";
    case EQAT_ERR_NULL: return "null pointer";
    case EQAT_ERR_SHAPE: return "invalid shape";
    case EQAT_ERR_ALIGN: return "pointer not 16-byte aligned";
    case EQAT_ERR_UNSUPPORTED: return "unsupported bits/group/mode";
    case EQAT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case EQAT_ERR_CUDA: return "CUDA error";
    case EQAT_ERR_TIMEOUT: return "a kernel abandoned a bounded wait";
    default: return "unknown status";
  }
}

int eqat_version(void) { return 100; }

size_t eqat_workspace_bytes(const eqat_desc* d, int op) {
  if (op == EQAT_OP_FAKEQUANT_BWD) {
    if (check_gemm_desc(d, false) != EQAT_OK) return (size_t)-1;
    // groups that fit an output tile are reduced inside the weight-gradient GEMM: nothing to store
    if (d->group <= kMaxFusedSteGroup) return 0;
    return (size_t)d->out_features * d->in_features * sizeof(eqat_bf16);   // dW_hat in bf16
  }
  if (op == EQAT_OP_PACKED_BWD_DS) {
    if (check_gemm_desc(d, true) != EQAT_OK) return (size_t)-1;
    return packed_ds_workspace_bytes(*d);
  }
  return (size_t)-1;
}

int eqat_device_status(int* h_status, int* h_detail) {
  if (h_status == nullptr) return EQAT_ERR_NULL;
  int st[3] = {0, 0, 0}, det[3] = {0, 0, 0};
  EQAT_TRY(read_device_status(&st[0], &det[0]));      // GEMM kernels
  EQAT_TRY(read_stream_status(&st[1], &det[1]));      // staged streaming kernels
  EQAT_TRY(read_gemv_status(&st[2], &det[2]));        // matrix-vector kernels
  const int k = st[0] != EQAT_OK ? 0 : (st[1] != EQAT_OK ? 1 : 2);
  *h_status = st[k];
  if (h_detail != nullptr) *h_detail = det[k];
  return EQAT_OK;
}

int eqat_selftest_wait_expiry(int which, void* stream) {
  if (which == 0) return launch_wait_expiry_gemm(as_stream(stream));
  if (which == 1) return launch_wait_expiry_stream(as_stream(stream));
  if (which == 2) return launch_wait_expiry_gemv(as_stream(stream));
  return EQAT_ERR_UNSUPPORTED;
}

int eqat_minmax_init(const eqat_desc* d, const eqat_bf16* W, float* s, float* z, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(W, s, z));
  return launch_minmax(*d, W, s, z, as_stream(stream));
}

int eqat_fakequant_weight(const eqat_desc* d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* W_hat,
                          void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(W, s, z, W_hat));
  return launch_fakequant(*d, W, s, z, W_hat, as_stream(stream));
}

int qlinear_fakequant_fwd(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* W, const float* s, const float* z,
                          eqat_bf16* Y, eqat_bf16* W_hat, void* stream) {
  EQAT_TRY(v_fakequant_fwd(d, X, W, s, z, Y, W_hat));
  // W_hat not wanted: fake-quantise each tile of W inside the GEMM, after it has reached shared memory
  if (W_hat == nullptr) return launch_latent_fwd(*d, X, W, s, z, Y, as_stream(stream));
  EQAT_TRY(launch_fakequant(*d, W, s, z, W_hat, as_stream(stream)));
  return launch_dense_fwd(*d, X, W_hat, Y, as_stream(stream));
}

int eqat_ste_bwd(const eqat_desc* d, const eqat_bf16* dW_hat, const eqat_bf16* W, const float* s, const float* z,
                 eqat_bf16* dW, float* ds, float* dz, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(dW_hat, W, s, z, dW, ds));
  if (dz != nullptr && !aligned16(dz)) return EQAT_ERR_ALIGN;
  return launch_ste_bwd(*d, dW_hat, W, s, z, dW, ds, dz, as_stream(stream));
}

int qlinear_fakequant_bwd(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* dY, const eqat_bf16* W,
                          const float* s, const float* z, const eqat_bf16* W_hat, eqat_bf16* dX, eqat_bf16* dW,
                          float* ds, float* dz, void* workspace, size_t workspace_bytes, void* stream) {
  EQAT_TRY(v_fakequant_bwd(d, X, dY, W, s, z, W_hat, dX, dW, ds, dz, workspace, workspace_bytes));
  // A group that fits inside one output tile is reduced in the weight-gradient GEMM's epilogue and needs no
  // scratch; a longer one (channel-wise quantisation) spans tiles, so its gradient goes through the workspace
  // and a second kernel.
  const bool fused = d->group <= kMaxFusedSteGroup;
  eqat_bf16* dW_hat = static_cast<eqat_bf16*>(workspace);
  cudaStream_t st = as_stream(stream);
  if (W_hat != nullptr) EQAT_TRY(launch_dense_dx(*d, dY, W_hat, dX, st));
  else EQAT_TRY(launch_latent_dx(*d, dY, W, s, z, dX, st));      // no stored W_hat: Eq. 1-2 inside the dX GEMM
  if (fused) return launch_dense_dw_ste(*d, dY, X, W, s, z, dW, ds, dz, st);
  EQAT_TRY(launch_dense_dw(*d, dY, X, dW_hat, st));
  return launch_ste_bwd(*d, dW_hat, W, s, z, dW, ds, dz, st);
}

int eqat_quantize_pack(const eqat_desc* d, const eqat_bf16* W, const float* s, const float* z, uint8_t* Wq_packed,
                       uint8_t* z8, eqat_fp16* s16, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(W, s, z, Wq_packed, z8, s16));
  return launch_quantize_pack(*d, W, s, z, Wq_packed, z8, s16, as_stream(stream));
}

int eqat_pack(const eqat_desc* d, const uint8_t* codes, uint8_t* Wq_packed, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(codes, Wq_packed));
  return launch_pack(*d, codes, Wq_packed, as_stream(stream));
}

int eqat_unpack(const eqat_desc* d, const uint8_t* Wq_packed, uint8_t* codes, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(Wq_packed, codes));
  return launch_unpack(*d, Wq_packed, codes, as_stream(stream));
}

int eqat_pack_zeros(const eqat_desc* d, const uint8_t* z8, uint8_t* z_packed, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(z8, z_packed));
  if (((int64_t)d->out_features * d->in_features / d->group) % 8 != 0) return EQAT_ERR_SHAPE;
  return launch_pack_zeros(*d, z8, z_packed, as_stream(stream));
}

int eqat_unpack_zeros(const eqat_desc* d, const uint8_t* z_packed, uint8_t* z8, void* stream) {
  EQAT_TRY(check_plain_desc(d));
  EQAT_TRY(check_ptrs(z_packed, z8));
  if (((int64_t)d->out_features * d->in_features / d->group) % 8 != 0) return EQAT_ERR_SHAPE;
  return launch_unpack_zeros(*d, z_packed, z8, as_stream(stream));
}

int qlinear_packed_fwd(const eqat_desc* d, const eqat_bf16* X, const uint8_t* Wq_packed, const eqat_fp16* s16,
                       const void* z, eqat_bf16* Y, void* stream) {
  EQAT_TRY(v_packed_fwd(d, X, Wq_packed, s16, z, Y));
  // a handful of tokens (decoding): one pass over the packed weight instead of near-empty tensor-core tiles
  if (packed_gemv_applies(*d)) return launch_packed_gemv(*d, X, Wq_packed, s16, z, Y, as_stream(stream));
  return launch_packed_fwd(*d, X, Wq_packed, s16, z, Y, as_stream(stream));
}

int qlinear_packed_bwd_dx(const eqat_desc* d, const eqat_bf16* dY, const uint8_t* Wq_packed, const eqat_fp16* s16,
                          const void* z, eqat_bf16* dX, void* stream) {
  EQAT_TRY(v_packed_fwd(d, dY, Wq_packed, s16, z, dX));          // same shape of check: one activation in, one out
  return launch_packed_dx(*d, dY, Wq_packed, s16, z, dX, as_stream(stream));
}

int qlinear_packed_bwd_ds(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* dY, const uint8_t* Wq_packed,
                          const void* z, const eqat_fp16* s16, float* ds, float* dz, void* workspace,
                          size_t workspace_bytes, void* stream) {
  EQAT_TRY(v_packed_bwd_ds(d, X, dY, Wq_packed, z, s16, ds, dz, workspace, workspace_bytes));
  return launch_packed_ds(*d, X, dY, Wq_packed, z, s16, ds, dz, workspace, as_stream(stream));
}

int eqat_block_ap_step(const eqat_block_ap_linear* L, int count, int* h_failed, void* stream) {
  if (h_failed != nullptr) *h_failed = -1;
  if (L == nullptr) return EQAT_ERR_NULL;
  if (count <= 0) return EQAT_ERR_SHAPE;
  for (int i = 0; i < count; ++i) {                         // everything is checked before anything is launched
    int rc = v_fakequant_fwd(&L[i].desc, L[i].X, L[i].W, L[i].s, L[i].z, L[i].Y, L[i].W_hat);
    if (rc == EQAT_OK)
      rc = v_fakequant_bwd(&L[i].desc, L[i].X, L[i].dY, L[i].W, L[i].s, L[i].z, L[i].W_hat, L[i].dX, L[i].dW, L[i].ds,
                           L[i].dz, L[i].workspace, L[i].workspace_bytes);
    if (rc != EQAT_OK) {
      if (h_failed != nullptr) *h_failed = i;
      return rc;
    }
  }
  for (int i = 0; i < count; ++i) {
    int rc = qlinear_fakequant_fwd(&L[i].desc, L[i].X, L[i].W, L[i].s, L[i].z, L[i].Y, L[i].W_hat, stream);
    if (rc == EQAT_OK)
      rc = qlinear_fakequant_bwd(&L[i].desc, L[i].X, L[i].dY, L[i].W, L[i].s, L[i].z, L[i].W_hat, L[i].dX, L[i].dW,
                                 L[i].ds, L[i].dz, L[i].workspace, L[i].workspace_bytes, stream);
    if (rc != EQAT_OK) {                                    // only the runtime can still refuse (EQAT_ERR_CUDA)
      if (h_failed != nullptr) *h_failed = i;
      return rc;
    }
  }
  return EQAT_OK;
}

int eqat_e2e_qp_step(const eqat_e2e_qp_linear* L, int count, int* h_failed, void* stream) {
  if (h_failed != nullptr) *h_failed = -1;
  if (L == nullptr) return EQAT_ERR_NULL;
  if (count <= 0) return EQAT_ERR_SHAPE;
  for (int i = 0; i < count; ++i) {
    int rc = v_packed_fwd(&L[i].desc, L[i].X, L[i].Wq_packed, L[i].s16, L[i].z, L[i].Y);
    if (rc == EQAT_OK) rc = v_packed_fwd(&L[i].desc, L[i].dY, L[i].Wq_packed, L[i].s16, L[i].z, L[i].dX);
    if (rc == EQAT_OK)
      rc = v_packed_bwd_ds(&L[i].desc, L[i].X, L[i].dY, L[i].Wq_packed, L[i].z, L[i].s16, L[i].ds, L[i].dz,
                           L[i].workspace, L[i].workspace_bytes);
    if (rc != EQAT_OK) {
      if (h_failed != nullptr) *h_failed = i;
      return rc;
    }
  }
  for (int i = 0; i < count; ++i) {
    int rc = qlinear_packed_fwd(&L[i].desc, L[i].X, L[i].Wq_packed, L[i].s16, L[i].z, L[i].Y, stream);
    if (rc == EQAT_OK) rc = qlinear_packed_bwd_dx(&L[i].desc, L[i].dY, L[i].Wq_packed, L[i].s16, L[i].z, L[i].dX, stream);
    if (rc == EQAT_OK)
      rc = qlinear_packed_bwd_ds(&L[i].desc, L[i].X, L[i].dY, L[i].Wq_packed, L[i].z, L[i].s16, L[i].ds, L[i].dz,
                                 L[i].workspace, L[i].workspace_bytes, stream);
    if (rc != EQAT_OK) {
      if (h_failed != nullptr) *h_failed = i;
      return rc;
    }
  }
  return EQAT_OK;
}

}  // extern "C"
