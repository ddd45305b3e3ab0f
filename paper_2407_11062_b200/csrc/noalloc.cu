// Block-AP backward for callers that must not allocate device memory.
//
// qlinear_fakequant_bwd needs out*in bf16 values of scratch for the weight
// gradient between its GEMM and its STE kernel when a quantisation group is
// longer than 256 elements (channel-wise quantisation; shorter groups are
// reduced inside the GEMM and leave the scratch untouched), and normally the
// caller allocates that.  Some callers cannot: code that runs after another framework
// has claimed the whole device for its own pool, or inside a section where the
// implicit device-wide synchronisation that cudaMalloc / cudaFree may perform is
// not acceptable.  For them this file keeps the scratch in a fixed array that is
// part of the library image: every GPU that loads the library holds these bytes
// until the process exits, which is why the array is modest and the entry point
// refuses larger problems.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kMaxElems = EQAT_NOALLOC_MAX_WEIGHT_ELEMS;
constexpr int kMaxDevices = 64;

// Device-resident scratch.  In host code this name is only a handle for the
// runtime's symbol table, not a device address: it must go through
// cudaGetSymbolAddress before a kernel can be given it.
static __device__ __align__(256) eqat_bf16 g_noalloc_scratch[kMaxElems];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];      // resolved address per device ordinal, null until set up

// Resolves the array's address on the current device, once per device.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EQAT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return EQAT_ERR_CUDA;
    }
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return EQAT_OK;
}

}  // namespace

extern "C" int qlinear_fakequant_bwd_noalloc(const eqat_desc* d, const eqat_bf16* X, const eqat_bf16* dY,
                                             const eqat_bf16* W, const float* s, const float* z,
                                             const eqat_bf16* W_hat, eqat_bf16* dX, eqat_bf16* dW, float* ds,
                                             float* dz, void* stream) {
  if (d == nullptr) return EQAT_ERR_NULL;
  if (d->out_features <= 0 || d->in_features <= 0) return EQAT_ERR_SHAPE;
  if ((uint64_t)d->out_features * (uint64_t)d->in_features > (uint64_t)kMaxElems) return EQAT_ERR_WORKSPACE;
  void* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != EQAT_OK) return rc;
  // Same kernels, same validation, same results as the caller-allocated variant.
  return qlinear_fakequant_bwd(d, X, dY, W, s, z, W_hat, dX, dW, ds, dz, scratch, kMaxElems * sizeof(eqat_bf16),
                               stream);
}
