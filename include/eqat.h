/*
 * eqat.h - C ABI of the B200 (sm_100a) library for the group-wise low-bit
 * quantised linear layer of EfficientQAT (arXiv 2407.11062).
 *
 * The layer is the one both training phases of the paper run through:
 *   Block-AP (Sec. 3.2): the weight is fake-quantised in the graph,
 *       W_int = clamp(round(W / s) + z, 0, 2^N - 1)          (Eq. 1)
 *       W_hat = (W_int - z) * s                              (Eq. 2)
 *     and W, s, z receive straight-through gradients (appendix "Gradient of
 *     Trainable Parameters in Block-AP", Eqs. 3-5).
 *   E2E-QP (Sec. 3.3): W_int is frozen and stored in N bits, only Eq. 2 runs,
 *     and the step size s is trained with d w_hat / d s = w_q - z.
 *
 * Conventions shared by every entry point
 *   - W is [out_features, in_features] row-major, as in Y = X * W^T.  A
 *     quantisation group is `group` consecutive elements along in_features
 *     inside one row; s and z are [out_features, in_features / group]
 *     row-major.  X is [tokens, in_features], Y and dY are [tokens,
 *     out_features], all row-major and dense (no padding, no strides).
 *   - bf16 / fp16 values are passed as their 16-bit patterns.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless its
 *     name starts with `h_` (host).  The library allocates no memory and keeps
 *     no pointer after a call returns.  Device base pointers must be 16-byte
 *     aligned; nothing more is required (where a kernel has a faster path for
 *     32-byte aligned data it picks it from the pointer).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work on `stream` and return without waiting for it.
 *   - Return value: EQAT_OK, or a negative eqat_status decided on the host
 *     BEFORE anything is launched (outputs untouched), or EQAT_ERR_CUDA if the
 *     runtime rejected a launch.  A kernel that gives up a bounded wait records
 *     it in a device status word read by eqat_device_status().
 *   - Gradients are overwritten, never accumulated.  No bias term (the
 *     quantised layers of the paper have none).
 *   - Tensor contents are not inspected: s <= 0, NaN or Inf give undefined
 *     values (never out-of-bounds accesses).
 *
 * Supported geometry: bits in {2,3,4}; group in {32,64,128,256} or a larger
 * multiple of 32 dividing in_features (e.g. group == in_features, one group
 * per row) for the element-wise and codec entry points; in_features a
 * multiple of 128.  The GEMM entry points also need out_features a multiple
 * of 64; tokens may be any positive number.  The packed-weight GEMMs take
 * group in {32,64,128,256} or group == in_features (channel-wise).
 */
#ifndef EQAT_H_
#define EQAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t eqat_bf16;   /* bfloat16 bit pattern */
typedef uint16_t eqat_fp16;   /* IEEE binary16 bit pattern */

typedef enum {
  EQAT_OK = 0,
  EQAT_ERR_NULL = -1,         /* a required pointer is NULL                          */
  EQAT_ERR_SHAPE = -2,        /* a size is non-positive or violates a divisibility   */
  EQAT_ERR_ALIGN = -3,        /* a device pointer is not 16-byte aligned             */
  EQAT_ERR_UNSUPPORTED = -4,  /* bits / group / mode outside the supported set       */
  EQAT_ERR_WORKSPACE = -5,    /* workspace missing, misaligned or too small          */
  EQAT_ERR_CUDA = -6,         /* the CUDA runtime or driver reported an error        */
  EQAT_ERR_TIMEOUT = -7       /* a kernel gave up a bounded wait (device status)     */
} eqat_status;

/* Problem descriptor: plain data, read during the call, never retained. */
typedef struct {
  int32_t bits;               /* N: 2, 3 or 4                                         */
  int32_t group;              /* g: elements per quantisation group along in_features */
  int32_t out_features;
  int32_t in_features;
  int64_t tokens;             /* rows of X / dY (ignored by weight-only entry points) */
  int32_t dz_mode;            /* clamped-branch value of d w_hat / d z:
                                 0 = -s (derivative of Eq. 2 at a saturated code),
                                 1 = -1 (Eq. 4 as printed)                            */
  int32_t zero_point_format;  /* how the packed-weight (E2E-QP) entry points read their
                                 zero points: EQAT_ZP_U8 or EQAT_ZP_FP16; must be
                                 EQAT_ZP_U8 (0) for every other entry point           */
} eqat_desc;

/* Zero points of the packed-weight entry points.  EQAT_ZP_U8: one byte per group,
 * the frozen N-bit integers of the hand-off.  EQAT_ZP_FP16: one fp16 value per
 * group, used as it is (not rounded): the variant of Sec. 3.3 that also trains z
 * and therefore keeps it in FP16 (2 + 32/64 = 2.50 bits per weight at w2g64 in
 * the paper's table of E2E-QP variants). */
enum { EQAT_ZP_U8 = 0, EQAT_ZP_FP16 = 1 };

/* Operations that need caller-provided scratch memory (eqat_workspace_bytes). */
enum { EQAT_OP_FAKEQUANT_BWD = 1, EQAT_OP_PACKED_BWD_DS = 2 };

const char* eqat_status_string(int status);
int eqat_version(void);

/* Bytes of device scratch the given operation needs for this problem (0 if none,
 * (size_t)-1 if desc/op is invalid).  The workspace must be 256-byte aligned. */
size_t eqat_workspace_bytes(const eqat_desc* desc, int op);

/* Reads and clears the device status word of the current device (synchronises
 * the device).  *h_status receives EQAT_OK or EQAT_ERR_TIMEOUT; *h_detail (may be
 * NULL) a code naming the wait that was abandoned. */
int eqat_device_status(int* h_status, int* h_detail);

/* Diagnostic of the bounded waits (no counterpart in the paper).  Every wait of
 * a kernel on a barrier has a time limit, after which the kernel records
 * EQAT_ERR_TIMEOUT in the device status word, abandons its work and returns
 * normally.  This call enqueues one warp that waits, with a limit of 1 ms, on a
 * barrier that nothing ever signals, through the very wait routine of the GEMM
 * kernels (which = 0), of the streaming kernels (which = 1) or of the
 * few-token forward kernel (which = 2); afterwards
 * eqat_device_status() must report EQAT_ERR_TIMEOUT once and EQAT_OK from then
 * on.  It touches no tensor. */
int eqat_selftest_wait_expiry(int which, void* stream);

/* ------------------------------------------------------------------ helpers */

/* Round-to-nearest initialisation of the quantisation parameters from each
 * group's range (the paper does not describe its initialisation; this is the
 * min/max rule):  s = max((max - min) / (2^N - 1), 2^-14),
 * z = clamp(-round(min / s), 0, 2^N - 1), evaluated in binary32.
 *   W [out,in] bf16 (in)   s, z [out,in/g] fp32 (out; z is integer valued) */
int eqat_minmax_init(const eqat_desc* desc, const eqat_bf16* W, float* s, float* z, void* stream);

/* ------------------------------------------------------------------ Block-AP */

/* Eq. 1 followed by Eq. 2: W_hat = (clamp(round(W/s) + round(z), 0, 2^N-1) - round(z)) * s.
 * The quotient W/s is an IEEE binary32 division, rounded half-to-even.
 *   W [out,in] bf16, s, z [out,in/g] fp32 (in)   W_hat [out,in] bf16 (out) */
int eqat_fakequant_weight(const eqat_desc* desc, const eqat_bf16* W, const float* s, const float* z,
                          eqat_bf16* W_hat, void* stream);

/* Block-AP forward (Sec. 3.2): W_hat as above, then Y = X * W_hat^T with fp32
 * accumulation.  Two forms, same Y bit for bit:
 *   - W_hat != NULL: W_hat is computed once by a streaming kernel and written out
 *     (the backward pass can then read it); the faster form.
 *   - W_hat == NULL: nothing is stored; every tile of W is fake-quantised inside
 *     the GEMM after it has been copied to shared memory (Eq. 1-2 "integrated
 *     within the computation graph" taken literally).  It saves out*in*2 bytes of
 *     memory and costs more time, because each tile of W is quantised once per
 *     512 tokens instead of once.  Needs group <= 256 or group == in_features.
 *   X [T,in] bf16, W, s, z (in)   Y [T,out] bf16, W_hat [out,in] bf16 (out, optional) */
int qlinear_fakequant_fwd(const eqat_desc* desc, const eqat_bf16* X, const eqat_bf16* W, const float* s,
                          const float* z, eqat_bf16* Y, eqat_bf16* W_hat, void* stream);

/* Straight-through backward of the fake quantiser (Eqs. 3-5, upper bound read
 * as 2^N - 1 as in Eq. 1, bounds inclusive).  With p = round(w/s) + round(z):
 *   dW      = dW_hat            if 0 <= p <= 2^N-1, else 0
 *   ds[o,g] = sum over the group of dW_hat * (round(w/s) - w/s | -z | 2^N-1-z)
 *   dz[o,g] = sum over the group of dW_hat * (0 | -s | -s)      (dz_mode 1: -1)
 *   dW_hat, W [out,in] bf16, s, z fp32 (in)   dW bf16, ds, dz fp32 (out)
 * dz may be NULL (not computed). */
int eqat_ste_bwd(const eqat_desc* desc, const eqat_bf16* dW_hat, const eqat_bf16* W, const float* s,
                 const float* z, eqat_bf16* dW, float* ds, float* dz, void* stream);

/* Block-AP backward: dX = dY * W_hat, dW_hat = dY^T * X, then Eqs. 3-5 as in
 * eqat_ste_bwd.  W_hat is the array qlinear_fakequant_fwd stored, or NULL, in
 * which case the dX GEMM fake-quantises W tile by tile itself (same dX; same
 * restriction on the group as in the forward).  With groups of up to 256 elements Eqs. 3-5 are applied to the
 * fp32 accumulators of dW_hat inside the same kernel and dW_hat is never
 * stored; longer groups (channel-wise) keep dW_hat in bf16 in the workspace and
 * run eqat_ste_bwd on it.  Needs eqat_workspace_bytes(desc,
 * EQAT_OP_FAKEQUANT_BWD) bytes of scratch: 0 for groups of up to 256 elements
 * (workspace may then be NULL), out*in*2 bytes for longer ones.
 *   X [T,in], dY [T,out], W, W_hat [out,in] bf16, s, z (in)
 *   dX [T,in] bf16, dW [out,in] bf16, ds, dz [out,in/g] fp32 (out) */
int qlinear_fakequant_bwd(const eqat_desc* desc, const eqat_bf16* X, const eqat_bf16* dY, const eqat_bf16* W,
                          const float* s, const float* z, const eqat_bf16* W_hat,
                          eqat_bf16* dX, eqat_bf16* dW, float* ds, float* dz,
                          void* workspace, size_t workspace_bytes, void* stream);

/* The same computation as qlinear_fakequant_bwd, for callers that cannot
 * allocate device memory (no counterpart in the paper: it is a deployment
 * convenience of this library).  Typical cases: the process's device memory is
 * already owned by another framework's pool, or the caller sits in a section
 * where the device-wide synchronisation that cudaMalloc / cudaFree may imply is
 * not acceptable.  The out*in bf16 values of scratch live in a fixed array
 * inside the library, so
 *   - out_features * in_features must not exceed EQAT_NOALLOC_MAX_WEIGHT_ELEMS
 *     (8 MiB of bf16); larger problems return EQAT_ERR_WORKSPACE and launch
 *     nothing.  Every GPU that loads the library holds those 8 MiB until exit;
 *   - the first call on each device looks the array's address up (a runtime
 *     call that is not stream work).  With CUDA's lazy module loading that
 *     look-up is also the moment the device actually sets the 8 MiB aside, so
 *     make that first call (any small valid problem will do) early: before
 *     another framework claims the rest of the device's memory, and before any
 *     stream capture begins on that device.  EQAT_ERR_CUDA from a first call
 *     means the array could not be reserved;
 *   - all calls on a device share the one array.  Its previous contents do not
 *     matter (every value read is written earlier in the same call), but two
 *     calls whose kernels overlap on the GPU (different streams) race on it:
 *     serialise them;
 *   - it calls no cudaMalloc, cudaFree or other allocating routine.
 * Arguments, outputs and status codes are otherwise those of
 * qlinear_fakequant_bwd. */
#define EQAT_NOALLOC_MAX_WEIGHT_ELEMS (4u << 20)
int qlinear_fakequant_bwd_noalloc(const eqat_desc* desc, const eqat_bf16* X, const eqat_bf16* dY,
                                  const eqat_bf16* W, const float* s, const float* z, const eqat_bf16* W_hat,
                                  eqat_bf16* dX, eqat_bf16* dW, float* ds, float* dz, void* stream);

/* ------------------------------------------------------------------ storage format */
/* The paper stores W_int and z in N bits and s in fp16 (Sec. 3.2, last
 * paragraph; N + (N+16)/g bits per parameter, appendix "Size of Quantized
 * Models") but gives no bit order.  This library's: each row of W_int is a
 * dense little-endian bit stream, code j in stream bits [N*j, N*j+N), stream
 * bit b = bit (b % 8) of byte (b / 8); row pitch in*N/8 bytes. */

/* Hand-off from Block-AP to E2E-QP: codes of Eq. 1 packed, zero points as
 * bytes, step sizes rounded to fp16.
 *   W, s, z (in)   Wq_packed [out, in*N/8] u8, z8 [out,in/g] u8, s16 [out,in/g] fp16 (out) */
int eqat_quantize_pack(const eqat_desc* desc, const eqat_bf16* W, const float* s, const float* z,
                       uint8_t* Wq_packed, uint8_t* z8, eqat_fp16* s16, void* stream);

/* codes [out,in] u8 (each < 2^N) <-> Wq_packed [out, in*N/8]. */
int eqat_pack(const eqat_desc* desc, const uint8_t* codes, uint8_t* Wq_packed, void* stream);
int eqat_unpack(const eqat_desc* desc, const uint8_t* Wq_packed, uint8_t* codes, void* stream);

/* Zero points for storage: z8 [out*in/g] u8 <-> one flat N-bit stream of
 * out*in/g*N/8 bytes with the same bit rule (the count must be a multiple of 8). */
int eqat_pack_zeros(const eqat_desc* desc, const uint8_t* z8, uint8_t* z_packed, void* stream);
int eqat_unpack_zeros(const eqat_desc* desc, const uint8_t* z_packed, uint8_t* z8, void* stream);

/* ------------------------------------------------------------------ E2E-QP */

/* In the three calls below `z` is [out,in/g] uint8, or [out,in/g] fp16 when
 * desc->zero_point_format is EQAT_ZP_FP16. */

/* Y = X * ((W_int - z) * s)^T, the packed codes expanded tile by tile in
 * shared memory inside the GEMM (Eq. 2; Sec. 3.3).  With few tokens (decoding)
 * and groups of at least 64 a matrix-vector kernel streams the packed weight
 * instead and does not round (W_int - z) * s to bf16.  It takes up to eight
 * tokens per launch, and up to 64 tokens go through it in slices (one pass over
 * the packed weight per slice) while that is cheaper than the tiled kernel; a
 * token's result does not depend on how the tokens were sliced.
 *   X [T,in] bf16, Wq_packed, s16, z (in)   Y [T,out] bf16 (out) */
int qlinear_packed_fwd(const eqat_desc* desc, const eqat_bf16* X, const uint8_t* Wq_packed,
                       const eqat_fp16* s16, const void* z, eqat_bf16* Y, void* stream);

/* dX = dY * ((W_int - z) * s).
 *   dY [T,out] bf16, Wq_packed, s16, z (in)   dX [T,in] bf16 (out) */
int qlinear_packed_bwd_dx(const eqat_desc* desc, const eqat_bf16* dY, const uint8_t* Wq_packed,
                          const eqat_fp16* s16, const void* z, eqat_bf16* dX, void* stream);

/* Step-size gradient (Sec. 3.3, d w_hat/d s = w_q - z):
 *   ds[o,g] = sum_{j in g} (sum_t dY[t,o] X[t,j]) * (W_int[o,j] - z[o,g]),
 * reduced in the epilogue of the weight-gradient GEMM; the [out,in] weight
 * gradient is never written to memory.  If dz is not NULL it also receives the
 * zero-point gradient of the same layer (the Sec. 3.3 variant that trains z),
 * dz[o,g] = -s[o,g] * sum_{j in g} G[o,j]; s16 is then required, else it may be
 * NULL.  Needs eqat_workspace_bytes(desc, EQAT_OP_PACKED_BWD_DS) bytes of
 * scratch: 0 for groups of up to 256 elements (workspace may then be NULL);
 * with one group per row the sums of the 256-column tiles of a row pass through
 * it and are added up in a fixed order.
 *   X [T,in], dY [T,out] bf16, Wq_packed, z (in)   ds [out,in/g] fp32 (out) */
int qlinear_packed_bwd_ds(const eqat_desc* desc, const eqat_bf16* X, const eqat_bf16* dY,
                          const uint8_t* Wq_packed, const void* z, const eqat_fp16* s16,
                          float* ds, float* dz, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------ whole blocks */

/* Both phases of the paper work on one transformer block at a time (Block-AP,
 * Sec. 3.2: "training of all parameters" of a block; E2E-QP, Sec. 3.3: every
 * quantised linear of the network with frozen codes), so a training step calls
 * the layer entry points above once per linear of the block (seven in a Llama
 * decoder block).  The two calls below take the block's linears as a HOST array
 * and do exactly that, in array order, on one stream:
 *   eqat_block_ap_step : qlinear_fakequant_fwd, then qlinear_fakequant_bwd
 *   eqat_e2e_qp_step   : qlinear_packed_fwd, qlinear_packed_bwd_dx,
 *                        qlinear_packed_bwd_ds
 * Every linear is validated on the host before the first launch: on an error
 * nothing has been enqueued, the status is that of the first offending linear
 * and *h_failed (may be NULL) receives its index.  The fields have the meaning
 * of the same-named arguments of the layer entry points (W_hat, dz, workspace
 * optional as there).  The arrays are read during the call and not retained. */
typedef struct {
  eqat_desc desc;
  const eqat_bf16* X;         /* [T,in]                          */
  const eqat_bf16* dY;        /* [T,out]                         */
  const eqat_bf16* W;         /* [out,in] latent weight          */
  const float* s;             /* [out,in/g]                      */
  const float* z;             /* [out,in/g]                      */
  eqat_bf16* Y;               /* [T,out]   (out)                 */
  eqat_bf16* W_hat;           /* [out,in]  (out, may be NULL)    */
  eqat_bf16* dX;              /* [T,in]    (out)                 */
  eqat_bf16* dW;              /* [out,in]  (out)                 */
  float* ds;                  /* [out,in/g] (out)                */
  float* dz;                  /* [out,in/g] (out, may be NULL)   */
  void* workspace;            /* eqat_workspace_bytes(EQAT_OP_FAKEQUANT_BWD), may be NULL if 0 */
  size_t workspace_bytes;
} eqat_block_ap_linear;

typedef struct {
  eqat_desc desc;
  const eqat_bf16* X;         /* [T,in]                          */
  const eqat_bf16* dY;        /* [T,out]                         */
  const uint8_t* Wq_packed;   /* [out, in*N/8]                   */
  const eqat_fp16* s16;       /* [out,in/g]                      */
  const void* z;              /* [out,in/g] uint8 or fp16 (desc.zero_point_format) */
  eqat_bf16* Y;               /* [T,out]   (out)                 */
  eqat_bf16* dX;              /* [T,in]    (out)                 */
  float* ds;                  /* [out,in/g] (out)                */
  float* dz;                  /* [out,in/g] (out, may be NULL)   */
  void* workspace;            /* eqat_workspace_bytes(EQAT_OP_PACKED_BWD_DS), may be NULL if 0 */
  size_t workspace_bytes;
} eqat_e2e_qp_linear;

int eqat_block_ap_step(const eqat_block_ap_linear* h_linears, int count, int* h_failed, void* stream);
int eqat_e2e_qp_step(const eqat_e2e_qp_linear* h_linears, int count, int* h_failed, void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* EQAT_H_ */
