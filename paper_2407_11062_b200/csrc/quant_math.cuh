// Element arithmetic of Eq. 1 shared by the streaming kernels and by the GEMM
// epilogue that applies Eqs. 3-5 to the weight gradient while it is still in
// tensor memory.
#pragma once
#include <stdint.h>

#include "common.cuh"

namespace eqat {

__device__ __forceinline__ void unpack8(const uint4& raw, float (&v)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

__device__ __forceinline__ uint4 pack8(const float (&v)[8]) {
  return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
                    pack_bf16x2(v[6], v[7]));
}

// 1/s to within 1 ulp (rcp.approx.f32); NaN, which forces the exact path below for the whole group, when the
// reciprocal is subnormal or not finite and the error bound would not hold, or when the rounded zero point zr lies
// outside [-16, 16] (the shortcut relies on the clamp range [-zr, Q - zr] lying within [-16, 31], see below).
__device__ __forceinline__ float group_rcp(float s, float zr) {
  float rs;
  asm("rcp.approx.f32 %0, %1;" : "=f"(rs) : "f"(s));
  const bool ok = fabsf(rs) >= 1.17549435e-38f && fabsf(rs) <= 3.402823466e+38f && fabsf(zr) <= 16.0f;
  return ok ? rs : __int_as_float(0x7FC00000);
}

// Eq. 1 for the eight elements of a vector: r = round(w/s) and the STE term
// r - w/s.  The code is DEFINED by a correctly rounded binary32 division
// followed by round-half-to-even, r = rintf(__fdiv_rn(w, s)).  Division and
// rintf run on the quarter-rate special-function pipe, which would cap these
// kernels below the memory roofline, so the common case takes a shortcut that
// provably gives the same r:
//   with rs a reciprocal of s good to 1 ulp, the exact product w*rs differs from
//   the exact quotient by at most 2^-23 |q| and from rn(w/s) by at most
//   1.5 * 2^-23 |q|.  r0 = rint(w*rs) (one fused multiply-add with 1.5 * 2^23,
//   which rounds the exact product half-to-even, then a subtraction) can differ
//   from rint(rn(w/s)) only if a half-integer lies between the two values; for
//   |q| <= 32.5 that needs w*rs within 1.5 * 2^-23 * 32.5 < 2^-17 of a half-integer.
//   d = w*rs - r0 (one more fused multiply-add) is the distance to the integer.
//   An element with |d| >= 0.5 - 2^-17 (or NaN) is redone with the exact
//   sequence: a few elements per thousand on min/max-initialised bf16 weights,
//   whose quotients are ratios of small integers and hit exact half-integers.
//   Quotients beyond 32.5 in magnitude need no care: every caller clamps r to
//   [-zr, Q - zr], which group_rcp keeps inside [-16, 31]; there r >= 33 or
//   r <= -33, r0 is within 1 of r (or as huge, or as infinite), and both clamp to
//   the same end.  (r itself is then not the defined value; only its clamp is.)
// The STE term r - w/s is returned as -d in the common case (2^-23 relative away
// from the exact one, immaterial for a gradient).
__device__ __forceinline__ void quotient_round8(const float (&w)[8], float s, float rs, float (&r)[8],
                                                float (&r_minus_t)[8]) {
  float dq[2] = {0.0f, 0.0f};                       // largest |d| of elements 0..3 and 4..7
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float r0 = fmaf(w[i], rs, 12582912.0f) - 12582912.0f;
    const float d = fmaf(w[i], rs, -r0);
    r[i] = r0;
    r_minus_t[i] = -d;
    dq[i >> 2] = fmaxf(dq[i >> 2], fabsf(d));
  }
  // fmaxf drops NaNs, so a NaN reciprocal (group_rcp's way of asking for the exact path) is tested by itself; a NaN
  // weight makes r NaN on either path
  const bool all_exact = rs != rs;
  if (!(fmaxf(dq[0], dq[1]) < 0.49999237060546875f) || all_exact) {
    // Some lane of every second warp lands here (bf16 weights over a min/max grid hit exact half-integer quotients
    // in a few elements per thousand), and the whole warp walks what that lane walks.  So the walk goes by halves
    // of the vector: a half with an element to redo is three times rarer than a vector with one.
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (!(dq[h] < 0.49999237060546875f) || all_exact) {
#pragma unroll
        for (int i = 4 * h; i < 4 * h + 4; ++i) {
          if (!(fabsf(r_minus_t[i]) < 0.49999237060546875f)) {
            const float q = __fdiv_rn(w[i], s);
            r[i] = rintf(q);
            r_minus_t[i] = r[i] - q;
          }
        }
      }
    }
  }
}

}  // namespace eqat
