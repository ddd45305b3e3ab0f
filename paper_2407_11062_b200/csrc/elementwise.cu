// Streaming (HBM-bound) kernels: fake quantiser, its straight-through
// backward with per-group reductions, min/max initialisation and the N-bit
// codec.  Every kernel moves 16-byte vectors with fully coalesced accesses; a
// quantisation group (contiguous along in_features, hence contiguous in the
// flattened weight) is owned by group/8 adjacent lanes of one warp, so group
// sums are fixed-order warp shuffles and the results are run-to-run identical.
#include "common.cuh"
#include "codec.cuh"
#include "elementwise.cuh"

namespace eqat {

namespace {

constexpr int kThreads = 256;

struct Vec8 { float v[8]; };

__device__ __forceinline__ Vec8 load_bf16x8(const eqat_bf16* p, size_t vec) {
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p) + vec);
  Vec8 o;
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o.v[2 * i] = __uint_as_float(w[i] << 16);
    o.v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
  return o;
}

__device__ __forceinline__ void store_bf16x8(eqat_bf16* p, size_t vec, const Vec8& x) {
  uint4 raw;
  raw.x = pack_bf16x2(x.v[0], x.v[1]);
  raw.y = pack_bf16x2(x.v[2], x.v[3]);
  raw.z = pack_bf16x2(x.v[4], x.v[5]);
  raw.w = pack_bf16x2(x.v[6], x.v[7]);
  reinterpret_cast<uint4*>(p)[vec] = raw;
}

// Eq. 1 for one element: the quotient t, its rounding r and the pre-clamp value
// p.  The quotient is a correctly rounded binary32 division and the rounding is
// half-to-even: this pair of choices defines the integer code.
__device__ __forceinline__ void quant_terms(float w, float s, float zr, float& t, float& r, float& p) {
  t = __fdiv_rn(w, s);
  r = rintf(t);
  p = r + zr;
}

__device__ __forceinline__ float clamp_code(float p, float Q) { return fminf(fmaxf(p, 0.0f), Q); }

// ------------------------------------------------------------------ Eq. 1 + Eq. 2
// (used for groups longer than 256 elements; shorter groups take the staged kernel in stream.cu)
__global__ void __launch_bounds__(kThreads)
fakequant_kernel(const eqat_bf16* __restrict__ W, const float* __restrict__ s, const float* __restrict__ z,
                 eqat_bf16* __restrict__ What, size_t n_vec, uint32_t vec_per_group, float Q) {
  const size_t base = (size_t)blockIdx.x * (kThreads * 2) + threadIdx.x;
  const size_t vi[2] = {base, base + kThreads};
  Vec8 w[2];
  float sv[2], zv[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    if (vi[u] < n_vec) {
      w[u] = load_bf16x8(W, vi[u]);
      const uint32_t g = (uint32_t)vi[u] / vec_per_group;
      sv[u] = __ldg(s + g);
      zv[u] = rintf(__ldg(z + g));
    }
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    if (vi[u] < n_vec) {
      Vec8 o;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        float t, r, p;
        quant_terms(w[u].v[i], sv[u], zv[u], t, r, p);
        o.v[i] = (clamp_code(p, Q) - zv[u]) * sv[u];
      }
      store_bf16x8(What, vi[u], o);
    }
  }
}

// ------------------------------------------------------------------ Eqs. 3-5 + group sums
// (groups of at most 256 elements are handled by the staged kernel in stream.cu)
// One block per group, for groups longer than 256 elements (e.g. channel-wise).
__global__ void __launch_bounds__(kThreads)
ste_bwd_long_group_kernel(const eqat_bf16* __restrict__ dWhat, const eqat_bf16* __restrict__ W,
                          const float* __restrict__ s, const float* __restrict__ z,
                          eqat_bf16* __restrict__ dW, float* __restrict__ ds, float* __restrict__ dz,
                          int vec_per_group, float Q, int dz_literal) {
  __shared__ float red_s[kThreads / 32], red_z[kThreads / 32];
  const size_t g = blockIdx.x;
  const float sv = __ldg(s + g);
  const float zr = rintf(__ldg(z + g));
  const float dz_clamped = dz_literal ? -1.0f : -sv;
  float acc_s = 0.0f, acc_z = 0.0f;
  for (int k = threadIdx.x; k < vec_per_group; k += kThreads) {
    const size_t v = g * (size_t)vec_per_group + k;
    const Vec8 gr = load_bf16x8(dWhat, v);
    const Vec8 w = load_bf16x8(W, v);
    Vec8 o;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float t, r, p;
      quant_terms(w.v[i], sv, zr, t, r, p);
      const bool below = p < 0.0f;
      const bool above = p > Q;
      const bool inside = !(below || above);
      o.v[i] = inside ? gr.v[i] : 0.0f;
      acc_s = fmaf(gr.v[i], inside ? (r - t) : (below ? -zr : Q - zr), acc_s);
      acc_z = fmaf(gr.v[i], inside ? 0.0f : dz_clamped, acc_z);
    }
    store_bf16x8(dW, v, o);
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    acc_s += __shfl_xor_sync(0xFFFFFFFFu, acc_s, d);
    acc_z += __shfl_xor_sync(0xFFFFFFFFu, acc_z, d);
  }
  if ((threadIdx.x & 31) == 0) { red_s[threadIdx.x >> 5] = acc_s; red_z[threadIdx.x >> 5] = acc_z; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.0f, b = 0.0f;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) { a += red_s[i]; b += red_z[i]; }
    ds[g] = a;
    if (dz != nullptr) dz[g] = b;
  }
}

// ------------------------------------------------------------------ min/max initialisation
__device__ __forceinline__ void minmax_finish(float mx, float mn, float Q, float* s, float* z, size_t g) {
  float sv = __fdiv_rn(mx - mn, Q);
  sv = fmaxf(sv, 6.103515625e-05f);                 // 2^-14, smallest normal fp16
  float zv = -rintf(__fdiv_rn(mn, sv));
  zv = fminf(fmaxf(zv, 0.0f), Q) + 0.0f;
  s[g] = sv;
  z[g] = zv;
}

// (groups of at most 256 elements are handled by the staged kernel in stream.cu)
__global__ void __launch_bounds__(kThreads)
minmax_long_group_kernel(const eqat_bf16* __restrict__ W, float* __restrict__ s, float* __restrict__ z,
                         int vec_per_group, float Q) {
  __shared__ float red_mx[kThreads / 32], red_mn[kThreads / 32];
  const size_t g = blockIdx.x;
  float mx = -INFINITY, mn = INFINITY;
  for (int k = threadIdx.x; k < vec_per_group; k += kThreads) {
    const Vec8 w = load_bf16x8(W, g * (size_t)vec_per_group + k);
#pragma unroll
    for (int i = 0; i < 8; ++i) { mx = fmaxf(mx, w.v[i]); mn = fminf(mn, w.v[i]); }
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, d));
    mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, d));
  }
  if ((threadIdx.x & 31) == 0) { red_mx[threadIdx.x >> 5] = mx; red_mn[threadIdx.x >> 5] = mn; }
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) { mx = fmaxf(mx, red_mx[i]); mn = fminf(mn, red_mn[i]); }
    minmax_finish(mx, mn, Q, s, z, g);
  }
}

// ------------------------------------------------------------------ codec
template <int BITS>
__device__ __forceinline__ void store_words(uint8_t* packed, size_t chunk, const uint32_t (&w)[BITS]) {
  uint32_t* dst = reinterpret_cast<uint32_t*>(packed) + chunk * BITS;   // chunk*BITS*4 bytes: 4-byte aligned
  if constexpr (BITS == 2) {
    *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
  } else if constexpr (BITS == 4) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  } else {
#pragma unroll
    for (int i = 0; i < BITS; ++i) dst[i] = w[i];
  }
}

template <int BITS>
__device__ __forceinline__ void load_words(const uint8_t* packed, size_t chunk, uint32_t (&w)[BITS]) {
  const uint32_t* src = reinterpret_cast<const uint32_t*>(packed) + chunk * BITS;
  if constexpr (BITS == 2) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(src)); w[0] = t.x; w[1] = t.y;
  } else if constexpr (BITS == 4) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(src)); w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
  } else {
#pragma unroll
    for (int i = 0; i < BITS; ++i) w[i] = __ldg(src + i);
  }
}

// One thread quantises 32 consecutive weights (one 64-byte run) and emits their packed words.
template <int BITS>
__global__ void __launch_bounds__(kThreads)
quantize_pack_kernel(const eqat_bf16* __restrict__ W, const float* __restrict__ s, const float* __restrict__ z,
                     uint8_t* __restrict__ packed, uint8_t* __restrict__ z8, eqat_fp16* __restrict__ s16,
                     size_t n_chunk, uint32_t chunk_per_group) {
  const size_t c = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (c >= n_chunk) return;
  constexpr float Q = (float)((1 << BITS) - 1);
  const uint32_t g = (uint32_t)c / chunk_per_group;
  const float sv = __ldg(s + g);
  const float zr = rintf(__ldg(z + g));
  uint32_t codes[32];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const Vec8 w = load_bf16x8(W, c * 4 + k);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float t, r, p;
      quant_terms(w.v[i], sv, zr, t, r, p);
      codes[8 * k + i] = (uint32_t)clamp_code(p, Q);
    }
  }
  uint32_t words[BITS];
  pack32<BITS>(codes, words);
  store_words<BITS>(packed, c, words);
  if ((uint32_t)c % chunk_per_group == 0) {
    z8[g] = (uint8_t)clamp_code(zr, Q);
    s16[g] = __half_as_ushort(__float2half_rn(sv));
  }
}

template <int BITS>
__global__ void __launch_bounds__(kThreads)
pack_kernel(const uint8_t* __restrict__ codes8, uint8_t* __restrict__ packed, size_t n_chunk) {
  const size_t c = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (c >= n_chunk) return;
  constexpr uint32_t mask = (1u << BITS) - 1u;
  uint32_t codes[32];
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(codes8) + c * 2 + k);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 16; ++i) codes[16 * k + i] = (w[i >> 2] >> (8 * (i & 3))) & mask;
  }
  uint32_t words[BITS];
  pack32<BITS>(codes, words);
  store_words<BITS>(packed, c, words);
}

// WIDE: the output is 32-byte aligned, so a thread's 32 codes go out as one store (a whole sector per lane,
// 1 KB contiguous per warp); otherwise as two 16-byte stores.
template <int BITS, bool WIDE>
__global__ void __launch_bounds__(kThreads)
unpack_kernel(const uint8_t* __restrict__ packed, uint8_t* __restrict__ codes8, size_t n_chunk) {
  const size_t c = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (c >= n_chunk) return;
  uint32_t words[BITS];
  load_words<BITS>(packed, c, words);
  uint32_t codes[32];
  unpack32<BITS>(words, codes);
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int j = 4 * i;
    w[i] = codes[j] | (codes[j + 1] << 8) | (codes[j + 2] << 16) | (codes[j + 3] << 24);
  }
  if constexpr (WIDE) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(codes8 + c * 32), "r"(w[0]), "r"(w[1]),
                 "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
  } else {
    reinterpret_cast<uint4*>(codes8)[c * 2] = make_uint4(w[0], w[1], w[2], w[3]);
    reinterpret_cast<uint4*>(codes8)[c * 2 + 1] = make_uint4(w[4], w[5], w[6], w[7]);
  }
}

// Flat stream of small arrays (zero points): one thread per 8 codes <-> `bits` bytes.
__global__ void pack8_kernel(const uint8_t* __restrict__ codes8, uint8_t* __restrict__ packed, size_t n8, int bits) {
  const size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= n8) return;
  const uint32_t mask = (1u << bits) - 1u;
  uint32_t acc = 0u;
  for (int j = 0; j < 8; ++j) acc |= ((uint32_t)codes8[i * 8 + j] & mask) << (bits * j);
  for (int b = 0; b < bits; ++b) packed[i * bits + b] = (uint8_t)(acc >> (8 * b));
}

__global__ void unpack8_kernel(const uint8_t* __restrict__ packed, uint8_t* __restrict__ codes8, size_t n8, int bits) {
  const size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= n8) return;
  const uint32_t mask = (1u << bits) - 1u;
  uint32_t acc = 0u;
  for (int b = 0; b < bits; ++b) acc |= (uint32_t)packed[i * bits + b] << (8 * b);
  for (int j = 0; j < 8; ++j) codes8[i * 8 + j] = (uint8_t)((acc >> (bits * j)) & mask);
}

inline unsigned blocks_for(size_t items, size_t per_block) { return (unsigned)((items + per_block - 1) / per_block); }

}  // namespace

// ------------------------------------------------------------------ host launchers
int launch_fakequant(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* What,
                     cudaStream_t st) {
  if (d.group <= 256) return launch_fakequant_stream(d, W, s, z, What, st);
  const size_t n_vec = (size_t)d.out_features * d.in_features / 8;
  const float Q = (float)((1 << d.bits) - 1);
  fakequant_kernel<<<blocks_for(n_vec, kThreads * 2), kThreads, 0, st>>>(W, s, z, What, n_vec,
                                                                         (uint32_t)d.group / 8, Q);
  return launch_status();
}

int launch_ste_bwd(const eqat_desc& d, const eqat_bf16* dWhat, const eqat_bf16* W, const float* s, const float* z,
                   eqat_bf16* dW, float* ds, float* dz, cudaStream_t st) {
  if (d.group <= 256) return launch_ste_bwd_stream(d, dWhat, W, s, z, dW, ds, dz, st);
  const float Q = (float)((1 << d.bits) - 1);
  const size_t n_groups = (size_t)d.out_features * d.in_features / d.group;
  ste_bwd_long_group_kernel<<<(unsigned)n_groups, kThreads, 0, st>>>(dWhat, W, s, z, dW, ds, dz, d.group / 8, Q,
                                                                     d.dz_mode == 1);
  return launch_status();
}

int launch_minmax(const eqat_desc& d, const eqat_bf16* W, float* s, float* z, cudaStream_t st) {
  if (d.group <= 256) return launch_minmax_stream(d, W, s, z, st);
  const float Q = (float)((1 << d.bits) - 1);
  const size_t n_groups = (size_t)d.out_features * d.in_features / d.group;
  minmax_long_group_kernel<<<(unsigned)n_groups, kThreads, 0, st>>>(W, s, z, d.group / 8, Q);
  return launch_status();
}

int launch_quantize_pack(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, uint8_t* packed,
                         uint8_t* z8, eqat_fp16* s16, cudaStream_t st) {
  if (d.group <= 256) return launch_quantize_pack_stream(d, W, s, z, packed, z8, s16, st);
  const size_t n_chunk = (size_t)d.out_features * d.in_features / 32;
  const unsigned nb = blocks_for(n_chunk, kThreads);
  const uint32_t cpg = (uint32_t)d.group / 32;
  switch (d.bits) {
    case 2: quantize_pack_kernel<2><<<nb, kThreads, 0, st>>>(W, s, z, packed, z8, s16, n_chunk, cpg); break;
    case 3: quantize_pack_kernel<3><<<nb, kThreads, 0, st>>>(W, s, z, packed, z8, s16, n_chunk, cpg); break;
    default: quantize_pack_kernel<4><<<nb, kThreads, 0, st>>>(W, s, z, packed, z8, s16, n_chunk, cpg); break;
  }
  return launch_status();
}

int launch_pack(const eqat_desc& d, const uint8_t* codes, uint8_t* packed, cudaStream_t st) {
  const size_t n_chunk = (size_t)d.out_features * d.in_features / 32;
  const unsigned nb = blocks_for(n_chunk, kThreads);
  switch (d.bits) {
    case 2: pack_kernel<2><<<nb, kThreads, 0, st>>>(codes, packed, n_chunk); break;
    case 3: pack_kernel<3><<<nb, kThreads, 0, st>>>(codes, packed, n_chunk); break;
    default: pack_kernel<4><<<nb, kThreads, 0, st>>>(codes, packed, n_chunk); break;
  }
  return launch_status();
}

int launch_unpack(const eqat_desc& d, const uint8_t* packed, uint8_t* codes, cudaStream_t st) {
  const size_t n_chunk = (size_t)d.out_features * d.in_features / 32;
  const unsigned nb = blocks_for(n_chunk, kThreads);
  const bool wide = (reinterpret_cast<uintptr_t>(codes) & 31u) == 0;
  switch (d.bits * 2 + (wide ? 1 : 0)) {
    case 4: unpack_kernel<2, false><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
    case 5: unpack_kernel<2, true><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
    case 6: unpack_kernel<3, false><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
    case 7: unpack_kernel<3, true><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
    case 8: unpack_kernel<4, false><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
    default: unpack_kernel<4, true><<<nb, kThreads, 0, st>>>(packed, codes, n_chunk); break;
  }
  return launch_status();
}

int launch_pack_zeros(const eqat_desc& d, const uint8_t* z8, uint8_t* packed, cudaStream_t st) {
  const size_t n8 = (size_t)d.out_features * d.in_features / d.group / 8;
  pack8_kernel<<<blocks_for(n8, kThreads), kThreads, 0, st>>>(z8, packed, n8, d.bits);
  return launch_status();
}

int launch_unpack_zeros(const eqat_desc& d, const uint8_t* packed, uint8_t* z8, cudaStream_t st) {
  const size_t n8 = (size_t)d.out_features * d.in_features / d.group / 8;
  unpack8_kernel<<<blocks_for(n8, kThreads), kThreads, 0, st>>>(packed, z8, n8, d.bits);
  return launch_status();
}

}  // namespace eqat
