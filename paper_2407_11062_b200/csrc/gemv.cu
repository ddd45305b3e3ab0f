// Packed-weight forward for a handful of tokens (decode-time inference):
//     Y[T,out] = X[T,in] * dequant(Wq)^T,   T <= 4,
// the matrix-vector case of the E2E-QP forward (Eq. 2 on frozen codes).  The
// 256-row tensor-core tiles of gemm.cu would be almost empty here; the work is
// one pass over the packed weight, so the kernel is a stream over its bytes.
//
// Mapping: a CTA owns 32 consecutive weight rows, lane = row, and its 16 warps
// split the row into contiguous runs of 64-code units.  All lanes of a warp are
// on the same columns, so the activations are read from shared memory as
// broadcasts (one wavefront per 16-byte load); each warp stages the columns of
// its own units there as fp32, together with their sum over every 64-column unit.
//
// Arithmetic: a code q is dropped into the top mantissa bits of the float 1.0,
// giving 1 + q/2^N with two logic operations and no int-to-float conversion.
// For a unit with step size s and zero point z
//     sum_j (q_j - z) s x_j = s (2^N * sum_j (1 + q_j/2^N) x_j - (2^N + z) * sum_j x_j),
// all in fp32, so the dequantised weight is never rounded to bf16 here.
#include "common.cuh"
#include "gemv.cuh"
#include "ptx.cuh"

namespace eqat {
namespace {

constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kRows = 32;                   // weight rows per CTA = lanes
constexpr size_t kMaxSmem = 200 * 1024;

__host__ __device__ inline size_t smem_floats(int T, int in_features) {
  return (size_t)T * in_features + (size_t)T * (in_features >> 6) + (size_t)kWarps * T * 32;
}

// Code c (0..63) of a 64-code unit held in 2*BITS words, as the float 1 + q/2^BITS.
template <int BITS>
__device__ __forceinline__ float code_as_float(const uint32_t (&w)[2 * BITS], int c) {
  const int bit = BITS * c, word = bit >> 5, off = bit & 31;
  constexpr int pos = 23 - BITS;            // lowest mantissa bit the code occupies
  uint32_t t;
  if (off + BITS <= 32) {
    t = off <= pos ? w[word] << (pos - off) : w[word] >> (off - pos);
  } else {
    t = __funnelshift_r(w[word], w[word + 1], off - pos);      // 3-bit codes that straddle two words
  }
  // (t & mask) | 1.0f as one three-input logic operation: both constants are passed in registers, which the
  // compiler otherwise folds into two instructions with one immediate each.
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(t), "r"(((1u << BITS) - 1u) << pos), "r"(0x3F800000u));
  return __uint_as_float(r);
}

template <int BITS>
__device__ __forceinline__ void load_unit(const uint8_t* p, uint32_t (&w)[2 * BITS]) {
  if constexpr (BITS == 3) {
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      const uint2 t = __ldg(reinterpret_cast<const uint2*>(p) + i);
      w[2 * i] = t.x; w[2 * i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < BITS / 2; ++i) {
      const uint4 t = __ldg(reinterpret_cast<const uint4*>(p) + i);
      w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
    }
  }
}

template <int BITS, int T>
__global__ void __launch_bounds__(kThreads)
packed_gemv_kernel(const eqat_bf16* __restrict__ X, const uint8_t* __restrict__ Wq, const eqat_fp16* __restrict__ s16,
                   const void* __restrict__ zq, eqat_bf16* __restrict__ Y, int out_features, int in_features,
                   int group_shift, int groups_per_row, int sectors, int z_fp16) {
  extern __shared__ __align__(16) float smem_f[];
  const int units = in_features >> 6;
  float* xs = smem_f;                                   // [T][in]
  float* xsum = xs + (size_t)T * in_features;           // [T][units]
  float* part = xsum + (size_t)T * units;               // [warps][T][32]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const int row = blockIdx.x * kRows + lane;
  const bool live = row < out_features;
  const uint8_t* wrow = Wq + (size_t)(live ? row : 0) * ((size_t)in_features * BITS / 8);
  const eqat_fp16* srow = s16 + (size_t)(live ? row : 0) * groups_per_row;
  // zero points: one byte each, or (z_fp16) one fp16 value each; kept as 16 raw bits next to the step size
  const size_t zrow = (size_t)(live ? row : 0) * groups_per_row;
  const uint8_t* z8 = static_cast<const uint8_t*>(zq);
  const eqat_fp16* z16 = static_cast<const eqat_fp16*>(zq);
  // whole pairs of units per warp (in_features is a multiple of 128): a pair is 32-byte aligned for 2- and
  // 4-bit codes, and lies in one group or in two consecutive ones
  const int pairs = units >> 1;
  const int u_begin = 2 * (int)((long)pairs * warp / kWarps), u_end = 2 * (int)((long)pairs * (warp + 1) / kWarps);
  constexpr float kScale = (float)(1 << BITS);

  float acc[T];
#pragma unroll
  for (int t = 0; t < T; ++t) acc[t] = 0.0f;
  // Units are taken kBatch at a time and the next batch is requested before the current one is used, so every
  // lane keeps 128 bytes of its row in flight: the rows of a warp are kilobytes apart, and with one unit per
  // request the kernel waited on DRAM latency instead of streaming.
  constexpr int kBatch = BITS == 2 ? 4 : 2;
  uint32_t w_nxt[kBatch][2 * BITS];
  uint32_t sz_nxt[kBatch];                              // fp16 step size | zero point << 16, fetched with the codes
  auto fetch = [&](int u0) {
#pragma unroll
    for (int k = 0; k < kBatch; k += 2)
      if (u0 + k < u_end) {
        const uint8_t* src = wrow + (size_t)(u0 + k) * (8 * BITS);
        // `sectors`: the packed matrix starts on a 32-byte boundary, so every pair of units does too and is
        // fetched as whole 32-byte sectors; otherwise with 16-byte (3-bit: 8-byte) loads
        bool fetched = false;
        if constexpr (BITS == 2) {
          if (sectors) {                                // both units: one 32-byte sector
            ptx::ldg_256(src, reinterpret_cast<uint32_t(&)[8]>(w_nxt[k][0]));
            fetched = true;
          }
        } else if constexpr (BITS == 4) {
          if (sectors) {
            ptx::ldg_256(src, w_nxt[k]);
            ptx::ldg_256(src + 32, w_nxt[k + 1]);
            fetched = true;
          }
        }
        if (!fetched) {
          load_unit<BITS>(src, w_nxt[k]);
          load_unit<BITS>(src + 8 * BITS, w_nxt[k + 1]);
        }
        const int g = ((u0 + k) << 6) >> group_shift;
        if (group_shift == 6) {
          const uint32_t s2 = __ldg(reinterpret_cast<const uint32_t*>(srow + g));
          if (z_fp16) {
            const uint32_t z2 = __ldg(reinterpret_cast<const uint32_t*>(z16 + zrow + g));
            sz_nxt[k] = (s2 & 0xFFFFu) | (z2 << 16);
            sz_nxt[k + 1] = (s2 >> 16) | (z2 & 0xFFFF0000u);
          } else {
            const uint32_t z2 = __ldg(reinterpret_cast<const unsigned short*>(z8 + zrow + g));
            sz_nxt[k] = (s2 & 0xFFFFu) | ((z2 & 0xFFu) << 16);
            sz_nxt[k + 1] = (s2 >> 16) | ((z2 >> 8) << 16);
          }
        } else {
          const uint32_t zraw = z_fp16 ? (uint32_t)__ldg(z16 + zrow + g) : (uint32_t)__ldg(z8 + zrow + g);
          sz_nxt[k] = sz_nxt[k + 1] = (uint32_t)__ldg(srow + g) | (zraw << 16);
        }
      }
  };
  fetch(u_begin);                                       // in flight while this warp stages its activations

  // A warp reads only the columns of its own units, so it stages just those (bf16 -> fp32) and their per-unit
  // sums itself: no CTA-wide barrier before the main loop.
  {
    const int nu = u_end - u_begin;
    for (int i = lane; i < T * nu * 8; i += 32) {       // one 16-byte piece (8 bf16) per iteration
      const int t = i / (nu * 8), r8 = i - t * (nu * 8);
      const size_t e0 = (size_t)t * in_features + (size_t)u_begin * 64 + (size_t)r8 * 8;
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(X + e0));
      const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
      float4 lo, hi;
      lo.x = __uint_as_float(r[0] << 16); lo.y = __uint_as_float(r[0] & 0xFFFF0000u);
      lo.z = __uint_as_float(r[1] << 16); lo.w = __uint_as_float(r[1] & 0xFFFF0000u);
      hi.x = __uint_as_float(r[2] << 16); hi.y = __uint_as_float(r[2] & 0xFFFF0000u);
      hi.z = __uint_as_float(r[3] << 16); hi.w = __uint_as_float(r[3] & 0xFFFF0000u);
      reinterpret_cast<float4*>(xs + e0)[0] = lo;
      reinterpret_cast<float4*>(xs + e0)[1] = hi;
    }
    __syncwarp();
    for (int i = 0; i < T * nu; ++i) {                  // two elements per lane, fixed-order tree
      const int t = i / nu, u = u_begin + (i - t * nu);
      const float* xu = xs + (size_t)t * in_features + (size_t)u * 64;
      float v = xu[lane] + xu[32 + lane];
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
      if (lane == 0) xsum[t * units + u] = v;
    }
    __syncwarp();
  }
#pragma unroll 1
  for (int u0 = u_begin; u0 < u_end; u0 += kBatch) {
    uint32_t w[kBatch][2 * BITS], sz[kBatch];
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      sz[k] = sz_nxt[k];
#pragma unroll
      for (int i = 0; i < 2 * BITS; ++i) w[k][i] = w_nxt[k][i];
    }
    fetch(u0 + kBatch);
#pragma unroll
    for (int k = 0; k < kBatch; ++k) {
      const int u = u0 + k;
      if (u < u_end) {
        const float s = __half2float(__ushort_as_half((unsigned short)(sz[k] & 0xFFFFu)));
        const float z = z_fp16 ? __half2float(__ushort_as_half((unsigned short)(sz[k] >> 16))) : (float)(sz[k] >> 16);
        // four independent partial sums per token and kAhead activation loads in flight: the loop is otherwise a
        // single chain of dependent multiply-adds behind one shared-memory load
        constexpr int kAhead = T == 1 ? 4 : (T == 2 ? 2 : 1);
        float d4[T][4];
#pragma unroll
        for (int t = 0; t < T; ++t)
#pragma unroll
          for (int e = 0; e < 4; ++e) d4[t][e] = 0.0f;
#pragma unroll
        for (int j = 0; j < 64; j += 4 * kAhead) {
          float4 xv[kAhead][T];
#pragma unroll
          for (int a = 0; a < kAhead; ++a)
#pragma unroll
            for (int t = 0; t < T; ++t)
              xv[a][t] = *reinterpret_cast<const float4*>(xs + (size_t)t * in_features + (size_t)u * 64 + j + 4 * a);
#pragma unroll
          for (int a = 0; a < kAhead; ++a) {
            const int c = j + 4 * a;
            const float q0 = code_as_float<BITS>(w[k], c), q1 = code_as_float<BITS>(w[k], c + 1),
                        q2 = code_as_float<BITS>(w[k], c + 2), q3 = code_as_float<BITS>(w[k], c + 3);
#pragma unroll
            for (int t = 0; t < T; ++t) {
              d4[t][0] = fmaf(q0, xv[a][t].x, d4[t][0]);
              d4[t][1] = fmaf(q1, xv[a][t].y, d4[t][1]);
              d4[t][2] = fmaf(q2, xv[a][t].z, d4[t][2]);
              d4[t][3] = fmaf(q3, xv[a][t].w, d4[t][3]);
            }
          }
        }
        float dot[T];
#pragma unroll
        for (int t = 0; t < T; ++t) dot[t] = (d4[t][0] + d4[t][1]) + (d4[t][2] + d4[t][3]);
#pragma unroll
        for (int t = 0; t < T; ++t)
          acc[t] = fmaf(s, fmaf(kScale, dot[t], -(kScale + z) * xsum[t * units + u]), acc[t]);
      }
    }
  }
#pragma unroll
  for (int t = 0; t < T; ++t) part[(warp * T + t) * 32 + lane] = acc[t];
  __syncthreads();
  if (warp < T && live) {
    float v = 0.0f;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) v += part[(wv * T + warp) * 32 + lane];      // fixed order: deterministic
    Y[(size_t)warp * out_features + row] = (eqat_bf16)(pack_bf16x2(v, 0.0f) & 0xFFFFu);
  }
}

template <int BITS, int T>
int launch_one(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* zq,
               eqat_bf16* Y, int group_shift, cudaStream_t st) {
  auto kern = packed_gemv_kernel<BITS, T>;
  const size_t smem = smem_floats(T, d.in_features) * sizeof(float);
  if (smem > 48 * 1024) {
    static SmemOptIn opt_in;        // raise the kernel's shared-memory limit once per device
    if (!opt_in.ensure(kern, (int)kMaxSmem)) return EQAT_ERR_CUDA;
  }
  const int grid = (d.out_features + kRows - 1) / kRows;
  const int sectors = (reinterpret_cast<uintptr_t>(Wq) & 31u) == 0 ? 1 : 0;
  kern<<<grid, kThreads, smem, st>>>(X, Wq, s16, zq, Y, d.out_features, d.in_features, group_shift,
                                     d.in_features / d.group, sectors, d.zero_point_format == EQAT_ZP_FP16 ? 1 : 0);
  return launch_status();
}

template <int BITS>
int launch_bits(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* zq,
                eqat_bf16* Y, int group_shift, cudaStream_t st) {
  switch ((int)d.tokens) {
    case 1: return launch_one<BITS, 1>(d, X, Wq, s16, zq, Y, group_shift, st);
    case 2: return launch_one<BITS, 2>(d, X, Wq, s16, zq, Y, group_shift, st);
    case 3: return launch_one<BITS, 3>(d, X, Wq, s16, zq, Y, group_shift, st);
    default: return launch_one<BITS, 4>(d, X, Wq, s16, zq, Y, group_shift, st);
  }
}

}  // namespace

bool packed_gemv_applies(const eqat_desc& d) {
  // a 64-code unit must lie inside one group: groups of 32 go through the tiled kernel
  return d.tokens >= 1 && d.tokens <= kGemvMaxTokens && d.group >= 64 &&
         smem_floats((int)d.tokens, d.in_features) * sizeof(float) <= kMaxSmem;
}

int launch_packed_gemv(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                       const void* zq, eqat_bf16* Y, cudaStream_t st) {
  int group_shift = 31;                                  // one group per row: every group index shifts to 0
  if (d.group <= 256) {
    group_shift = 0;
    while ((1 << group_shift) < d.group) ++group_shift;
  }
  switch (d.bits) {
    case 2: return launch_bits<2>(d, X, Wq, s16, zq, Y, group_shift, st);
    case 3: return launch_bits<3>(d, X, Wq, s16, zq, Y, group_shift, st);
    default: return launch_bits<4>(d, X, Wq, s16, zq, Y, group_shift, st);
  }
}

}  // namespace eqat
