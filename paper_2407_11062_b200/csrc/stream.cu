// Streaming kernels with TMA-staged inputs: fake quantiser (Eq. 1 + Eq. 2), its
// straight-through backward (Eqs. 3-5), min/max initialisation and quantise +
// pack, for groups of at most 256 elements.
//
// These kernels move 2-6 bytes per element and would be bound by HBM bandwidth
// if the instruction stream per element were short enough; at 10-25 executed
// instructions per element it is the issue rate of the SM that decides, so the
// layout is chosen to keep everything that is per group or per access out of
// the per-element count:
//   * the loads are taken out of the compute threads altogether.  Each
//     persistent CTA has one producer thread that streams 16 KB tiles of the
//     input(s) into a shared-memory ring with tensor copies
//     (cp.async.bulk.tensor, completion on an mbarrier) while 8 consumer warps
//     compute; the flattened weight is described to the copy engine as a matrix
//     of 128-byte rows with the 128-byte swizzle;
//   * a consumer lane owns 32 CONSECUTIVE elements (half a row of the tile, four
//     16-byte vectors, always inside one quantisation group), so the group's
//     step size, zero point, reciprocal and clamp bounds are set up once per 32
//     elements, the group sums need one shuffle per doubling of the group
//     beyond 32, and the lane writes 64 contiguous bytes.  The swizzle makes
//     the lanes' 16-byte shared-memory reads conflict-free although they are 64
//     bytes apart.
// Three CTAs fit on an SM (24 consumer warps, up to 190 KB of reads in flight).
//
// Group sums are fixed-order (serial inside a lane, then a shuffle tree), so
// results are run-to-run identical.
#include <cuda.h>

#include "common.cuh"
#include "elementwise.cuh"
#include "gemm.cuh"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace eqat {

__device__ int g_stream_status[2];   // [0] = eqat_status, [1] = WaitSite

namespace {

constexpr int kConsumers = 256;
constexpr int kThreadsS = kConsumers + 32;           // + one producer warp
constexpr int kLaneElems = 32;                       // consecutive elements per consumer lane and tile
constexpr int kTileRows = kConsumers / 2;            // 128-byte rows per tile (two lanes per row)
constexpr int kTileElems = kConsumers * kLaneElems;  // 8192
constexpr int kTileBytes = kTileElems * 2;           // 16 KB per input stream
constexpr uint64_t kStreamWaitLimitNs = 2000000000ull;
// Ring depth and CTAs per SM.  The stage a consumer works on is released as soon as its vectors are in
// registers, so a few stages are enough to keep the copy engine busy.
#ifndef EQAT_STREAM_CTAS1
#define EQAT_STREAM_CTAS1 3
#define EQAT_STREAM_STAGES1 4
#endif
constexpr int kStages1 = EQAT_STREAM_STAGES1, kCtas1 = EQAT_STREAM_CTAS1;   // kernels with one input stream
constexpr int kStages2 = 2, kCtas2 = 3;                                    // two input streams (32 KB per stage)

template <int NIN, int STAGES>
struct Ring {
  static constexpr int kStages = STAGES;
  static constexpr int kStageBytes = NIN * kTileBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*control block*/;
};

struct RingCtl {
  uint64_t full[8];
  uint64_t empty[8];
  int abort;
};
static_assert(sizeof(RingCtl) <= 256, "ring control block must fit its reservation");

__device__ __forceinline__ bool ring_wait(uint32_t bar, uint32_t parity, volatile int* abort, int site,
                                          uint32_t sleep_ns, uint64_t limit_ns = kStreamWaitLimitNs) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t n = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if (sleep_ns != 0) __nanosleep(sleep_ns);
    if ((++n & 31u) == 0u) {
      if (*abort) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) {
        *abort = 1;
        atomicExch(&g_stream_status[1], site);
        atomicExch(&g_stream_status[0], (int)EQAT_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Runs `body(e0, raw, params)` on every consumer lane for every tile this CTA
// owns: e0 is the index of the lane's first element, raw[i][u] the lane's
// vector u (elements e0 + 8u .. e0 + 8u + 7) of input stream i, and params what
// `fetch(e0)` returned for this tile.  fetch is called one tile ahead, so the
// small per-group loads it makes (step size, zero point) are in flight while
// the previous tile is being computed.  The maps describe each input as
// [n_elem / 64, 64] bf16; rows beyond the end read as zeros, and a lane whose
// e0 is at or beyond n_elem must ignore its vectors.
template <int NIN, int STAGES, typename Params, typename Fetch, typename Body>
__device__ __forceinline__ void stream_tiles(const CUtensorMap* const (&maps)[NIN], size_t n_elem, Fetch&& fetch,
                                             Body&& body) {
  using R = Ring<NIN, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_addr(smem_raw);
  const uint32_t smem_base = (raw_addr + 1023u) & ~1023u;            // stages are 1024-byte aligned (swizzle period)
  RingCtl* ctl = reinterpret_cast<RingCtl*>(smem_raw + (smem_base - raw_addr) + R::kStages * R::kStageBytes);
  volatile int* abort_flag = &ctl->abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t n_tiles = (n_elem + kTileElems - 1) / kTileElems;

  if (threadIdx.x == 0) {
    for (int s = 0; s < R::kStages; ++s) {
      ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), kConsumers / 32);
    }
    ctl->abort = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();

  if (warp == kConsumers / 32) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < NIN; ++i) ptx::tma_prefetch_desc(maps[i]);
      int stage = 0;
      uint32_t phase = 0;
      size_t issued = 0;
      bool ok = true;
      for (size_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        if (!ring_wait(ptx::smem_addr(&ctl->empty[stage]), phase ^ 1u, abort_flag, WAIT_STREAM_EMPTY, 32)) {
          ok = false;
          break;
        }
        ptx::fence_proxy_async_smem();                             // consumers' reads of this stage before the copy's writes
        const uint32_t full = ptx::smem_addr(&ctl->full[stage]);
        ptx::mbar_expect_tx(full, NIN * kTileBytes);               // rows past the end are zero-filled and counted
#pragma unroll
        for (int i = 0; i < NIN; ++i)
          ptx::tma_load_2d(smem_base + stage * R::kStageBytes + i * kTileBytes, maps[i], 0, (int)(tile * kTileRows), full);
        ++issued;
        if (++stage == R::kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok || *abort_flag) {
        // every copy this thread started must land before the CTA exits
        const size_t first = issued > (size_t)R::kStages ? issued - R::kStages : 0;
        for (size_t i = first; i < issued; ++i) {
          const uint32_t bar = ptx::smem_addr(&ctl->full[i % R::kStages]);
          const uint32_t par = (uint32_t)((i / R::kStages) & 1);
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(bar, par)) {
            if (ptx::globaltimer_ns() - t0 > 50000000ull) {
              atomicExch(&g_stream_status[1], (int)WAIT_TEARDOWN);
              break;
            }
          }
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- consumers
    // lane t owns half (t & 1) of row (t >> 1): 16-byte chunk c of a row sits at chunk (c ^ (row & 7))
    const uint32_t row = threadIdx.x >> 1;
    const uint32_t row_off = row * 128u, sx = row & 7u, c0 = (threadIdx.x & 1u) * 4u;
    int stage = 0;
    uint32_t phase = 0;
    Params next = fetch((size_t)blockIdx.x * kTileElems + (size_t)threadIdx.x * kLaneElems);
    for (size_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
      const Params cur = next;
      if (tile + gridDim.x < n_tiles) next = fetch((tile + gridDim.x) * kTileElems + (size_t)threadIdx.x * kLaneElems);
      // the lanes of a warp leave together: the bodies shuffle across the whole warp
      const bool got = ring_wait(ptx::smem_addr(&ctl->full[stage]), phase, abort_flag, WAIT_STREAM_FULL, 0);
      if (!__all_sync(0xFFFFFFFFu, got)) break;
      uint4 raw[NIN][4];
      const uint32_t st = smem_base + stage * R::kStageBytes + row_off;
#pragma unroll
      for (int i = 0; i < NIN; ++i)
#pragma unroll
        for (int u = 0; u < 4; ++u) raw[i][u] = ptx::lds_128(st + i * kTileBytes + (((c0 + u) ^ sx) << 4));
      // The stage is handed back before the compute.  Its next user is a copy of the asynchronous proxy, which
      // is not ordered after these generic-proxy reads by the barrier alone: without a proxy fence on the way
      // a few lanes read rows of the tile four steps ahead (seen on 8192 x 8192 weights with three CTAs per SM).
      // The readers fence here, and the producer fences again between its wait and the copy.
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->empty[stage]));   // the stage can be refilled now
      if (++stage == R::kStages) { stage = 0; phase ^= 1u; }
      body(tile * kTileElems + (size_t)threadIdx.x * kLaneElems, raw, cur);
    }
  }
}

// Step size and (already rounded) zero point of the group a lane's elements belong to.
struct GroupParams {
  float s, z;
};

__device__ __forceinline__ GroupParams fetch_group(const float* __restrict__ s, const float* __restrict__ z, size_t e0,
                                                   size_t n_elem, int group_shift) {
  GroupParams p{1.0f, 0.0f};
  if (e0 < n_elem) {
    p.s = __ldg(s + (e0 >> group_shift));
    p.z = __ldg(z + (e0 >> group_shift));
  }
  return p;
}

// A lane's 64 output bytes: two 32-byte stores where the tensor allows it, four 16-byte stores otherwise.
__device__ __forceinline__ void store_lane(eqat_bf16* dst, const uint4 (&o)[4], bool wide) {
  if (wide) {
#pragma unroll
    for (int h = 0; h < 2; ++h)
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 16 * h), "r"(o[2 * h].x),
                   "r"(o[2 * h].y), "r"(o[2 * h].z), "r"(o[2 * h].w), "r"(o[2 * h + 1].x), "r"(o[2 * h + 1].y),
                   "r"(o[2 * h + 1].z), "r"(o[2 * h + 1].w) : "memory");
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u) reinterpret_cast<uint4*>(dst)[u] = o[u];
  }
}

// ------------------------------------------------------------------ Eq. 1 + Eq. 2
// (clamp(r + z, 0, Q) - z) * s == clamp(r, -z, Q - z) * s for integer r and z.
__global__ void __launch_bounds__(kThreadsS, kCtas1)
fakequant_stream_kernel(const __grid_constant__ CUtensorMap map_w, const float* __restrict__ s,
                        const float* __restrict__ z, eqat_bf16* __restrict__ What, size_t n_elem, int group_shift,
                        float Q, int wide) {
  const CUtensorMap* const maps[1] = {&map_w};
  stream_tiles<1, kStages1, GroupParams>(maps, n_elem,
      [&](size_t e0) { return fetch_group(s, z, e0, n_elem, group_shift); },
      [&](size_t e0, const uint4 (&raw)[1][4], const GroupParams& gp) {
    if (e0 >= n_elem) return;
    const float sv = gp.s;
    const float zr = rintf(gp.z);
    const float rs = group_rcp(sv, zr);
    const float lo = -zr, hi = Q - zr;
    uint4 o[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float w[8], r[8], rt[8];
      unpack8(raw[0][u], w);
      quotient_round8(w, sv, rs, r, rt);
#pragma unroll
      for (int i = 0; i < 8; ++i) w[i] = fminf(fmaxf(r[i], lo), hi) * sv;
      o[u] = pack8(w);
    }
    store_lane(What + e0, o, wide != 0);
  });
}

// ------------------------------------------------------------------ Eqs. 3-5 + group sums
// With lo = -z, hi = Q - z and c = clamp(r, lo, hi): the element is in range iff
// c == r, and on the clamped branches Eq. 3's value (-z or Q - z) is c itself.
// Eq. 4 is a constant per group times the sum of the gradient over the clamped
// elements.  LPG = lanes per group (group / 32).
template <int LPG>
__global__ void __launch_bounds__(kThreadsS, kCtas2)
ste_bwd_stream_kernel(const __grid_constant__ CUtensorMap map_g, const __grid_constant__ CUtensorMap map_w,
                      const float* __restrict__ s, const float* __restrict__ z, eqat_bf16* __restrict__ dW,
                      float* __restrict__ ds, float* __restrict__ dz, size_t n_elem, float Q, int dz_literal, int wide) {
  const CUtensorMap* const maps[2] = {&map_g, &map_w};
  constexpr int group_shift = LPG == 1 ? 5 : LPG == 2 ? 6 : LPG == 4 ? 7 : 8;
  stream_tiles<2, kStages2, GroupParams>(maps, n_elem,
      [&](size_t e0) { return fetch_group(s, z, e0, n_elem, group_shift); },
      [&](size_t e0, const uint4 (&raw)[2][4], const GroupParams& gp) {
    const bool live = e0 < n_elem;                      // uniform over the lanes of a group
    float acc_s = 0.0f, acc_g = 0.0f;
    const float sv = gp.s;
    if (live) {
      const float zr = rintf(gp.z);
      const float rs = group_rcp(sv, zr);
      const float lo = -zr, hi = Q - zr;
      uint4 o[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float gr[8], w[8], r[8], rt[8];
        unpack8(raw[0][u], gr);
        unpack8(raw[1][u], w);
        quotient_round8(w, sv, rs, r, rt);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float c = fminf(fmaxf(r[i], lo), hi);
          const bool inside = (c == r[i]);
          acc_s = fmaf(gr[i], inside ? rt[i] : c, acc_s);     // Eq. 3
          acc_g += inside ? 0.0f : gr[i];                      // Eq. 4
          w[i] = inside ? gr[i] : 0.0f;                        // Eq. 5
        }
        o[u] = pack8(w);
      }
      store_lane(dW + e0, o, wide != 0);
    }
#pragma unroll
    for (int d = LPG / 2; d >= 1; d >>= 1) {
      acc_s += __shfl_xor_sync(0xFFFFFFFFu, acc_s, d);
      acc_g += __shfl_xor_sync(0xFFFFFFFFu, acc_g, d);
    }
    if (live && (threadIdx.x % LPG) == 0) {
      const size_t g = e0 >> group_shift;
      ds[g] = acc_s;
      if (dz != nullptr) dz[g] = (dz_literal ? -1.0f : -sv) * acc_g;
    }
  });
}

// ------------------------------------------------------------------ min/max initialisation
struct NoParams {};

__device__ __forceinline__ uint32_t bf162_max(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t bf162_min(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmin2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}

template <int LPG>
__global__ void __launch_bounds__(kThreadsS, kCtas1)
minmax_stream_kernel(const __grid_constant__ CUtensorMap map_w, float* __restrict__ s, float* __restrict__ z,
                     size_t n_elem, float Q) {
  const CUtensorMap* const maps[1] = {&map_w};
  constexpr int group_shift = LPG == 1 ? 5 : LPG == 2 ? 6 : LPG == 4 ? 7 : 8;
  stream_tiles<1, kStages1, NoParams>(maps, n_elem, [](size_t) { return NoParams{}; },
      [&](size_t e0, const uint4 (&raw)[1][4], const NoParams&) {
    // extrema on packed bf16 pairs (exact: comparisons only), widened to fp32 at the end
    uint32_t mx2 = 0xFF80FF80u, mn2 = 0x7F807F80u;      // (-inf, -inf) and (+inf, +inf) as bf16 pairs
    const bool live = e0 < n_elem;                      // uniform over the lanes of a group
    if (live) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint4 r4 = raw[0][u];
        mx2 = bf162_max(mx2, bf162_max(bf162_max(r4.x, r4.y), bf162_max(r4.z, r4.w)));
        mn2 = bf162_min(mn2, bf162_min(bf162_min(r4.x, r4.y), bf162_min(r4.z, r4.w)));
      }
    }
#pragma unroll
    for (int d = LPG / 2; d >= 1; d >>= 1) {
      mx2 = bf162_max(mx2, __shfl_xor_sync(0xFFFFFFFFu, mx2, d));
      mn2 = bf162_min(mn2, __shfl_xor_sync(0xFFFFFFFFu, mn2, d));
    }
    if (live && (threadIdx.x % LPG) == 0) {
      const float mx = fmaxf(__uint_as_float(mx2 << 16), __uint_as_float(mx2 & 0xFFFF0000u));
      const float mn = fminf(__uint_as_float(mn2 << 16), __uint_as_float(mn2 & 0xFFFF0000u));
      // s = max((max - min) / Q, 2^-14), z = clamp(-round(min / s), 0, Q), all in binary32
      float sv = __fdiv_rn(mx - mn, Q);
      sv = fmaxf(sv, 6.103515625e-05f);
      float zv = -rintf(__fdiv_rn(mn, sv));
      zv = fminf(fmaxf(zv, 0.0f), Q) + 0.0f;
      s[e0 >> group_shift] = sv;
      z[e0 >> group_shift] = zv;
    }
  });
}

// ------------------------------------------------------------------ quantise + pack (hand-off)
// A lane turns its 32 weights into 32 codes = BITS consecutive 32-bit words of the
// little-endian stream (code j of the lane at bits [BITS*j, BITS*j + BITS)).
//
// Only the clamped code is wanted here, not r or r - w/s, which allows a shorter
// exact evaluation of Eq. 1 than quotient_round8.  With cz = 2^23 + zr (an
// integer) t = fma(w, rs, cz) rounds w*rs + zr to an integer held in the low
// mantissa bits of t whenever the sum is in [0, 2^23), and lands below 2^23
// (code 0 after the clamp) when it is negative.  The code is DEFINED through
// y0 = rn(w / s).  Take the two reciprocals rs_lo = rs (1 - 2^-16) and
// rs_hi = rs (1 + 2^-16), rs good to 1 ulp: the exact products w*rs_lo and
// w*rs_hi enclose y0 with a margin of 2^-17 |y0| on either side, and rounding is
// monotone, so when t_lo == t_hi every value between the products, y0 among
// them, rounds to the same integer; y0 itself cannot be an exact tie then, since
// a tie strictly inside the interval would separate t_lo from t_hi.  (The
// integer added before rounding changes which neighbour a tie goes to, but a tie
// never reaches this branch.)  When they differ (the quotient is within about
// 2^-16 |y0| of a rounding boundary: a few elements per thousand) the element
// is redone with the defining sequence.  Two multiply-adds and one logic
// operation per element, and the clamped t feeds the bit packing directly: its
// low bits ARE the code.
template <int BITS>
__global__ void __launch_bounds__(kThreadsS, kCtas1)
quantize_pack_stream_kernel(const __grid_constant__ CUtensorMap map_w, const float* __restrict__ s,
                            const float* __restrict__ z, uint8_t* __restrict__ packed, uint8_t* __restrict__ z8,
                            eqat_fp16* __restrict__ s16, size_t n_elem, int group_shift) {
  const CUtensorMap* const maps[1] = {&map_w};
  constexpr float Q = (float)((1 << BITS) - 1);
  constexpr float kTwo23 = 8388608.0f;
  // sum over the 8 codes of a vector of the bit pattern of 2^23 shifted to the code's place (mod 2^32)
  constexpr uint32_t kBias = (uint32_t)(0x4B000000ull * (((1ull << (8 * BITS)) - 1ull) / ((1ull << BITS) - 1ull)));
  stream_tiles<1, kStages1, GroupParams>(maps, n_elem,
      [&](size_t e0) { return fetch_group(s, z, e0, n_elem, group_shift); },
      [&](size_t e0, const uint4 (&raw)[1][4], const GroupParams& gp) {
    if (e0 >= n_elem) return;
    const float sv = gp.s;
    const float zr = rintf(gp.z);
    const float rs = group_rcp(sv, zr);                 // NaN: the whole group takes the defining sequence
    const bool exact_only = !(fabsf(rs) >= 2.5e-38f);   // (also when rs_lo would lose bits to underflow)
    const float rs_lo = rs * 0.9999847412109375f, rs_hi = rs * 1.0000152587890625f;
    const float cz = kTwo23 + zr;
    uint32_t piece[4];                                  // vector u's 8 codes, code i at bits [BITS*i, BITS*i + BITS)
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float w[8], t[8];
      unpack8(raw[0][u], w);
      uint32_t differ[2] = {exact_only ? 1u : 0u, exact_only ? 1u : 0u};   // elements 0..3 and 4..7
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        t[i] = fmaf(w[i], rs_lo, cz);
        differ[i >> 2] |= __float_as_uint(t[i]) ^ __float_as_uint(fmaf(w[i], rs_hi, cz));
      }
      if ((differ[0] | differ[1]) != 0u) {
        // the whole warp walks what one lane walks, so the walk goes by halves of the vector (see quotient_round8)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (differ[h] != 0u) {
#pragma unroll
            for (int i = 4 * h; i < 4 * h + 4; ++i) {
              if (exact_only || !(t[i] == fmaf(w[i], rs_hi, cz))) {
                const float r = rintf(__fdiv_rn(w[i], sv));
                t[i] = (r + zr) + kTwo23;
              }
            }
          }
        }
      }
      uint32_t acc = 0u;
#pragma unroll
      for (int i = 7; i >= 0; --i)
        acc = (acc << BITS) + __float_as_uint(fminf(fmaxf(t[i], kTwo23), kTwo23 + Q));
      piece[u] = acc - kBias;
    }
    if ((e0 & (((size_t)1 << group_shift) - 1)) == 0) {
      const size_t g = e0 >> group_shift;
      z8[g] = (uint8_t)(__float_as_uint(fminf(fmaxf(zr, 0.0f), Q) + 8388608.0f) & 0xFFu);
      s16[g] = __half_as_ushort(__float2half_rn(sv));
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(packed) + (e0 >> 5) * BITS;
    if constexpr (BITS == 2) {
      *reinterpret_cast<uint2*>(dst) = make_uint2(piece[0] | (piece[1] << 16), piece[2] | (piece[3] << 16));
    } else if constexpr (BITS == 3) {
      dst[0] = piece[0] | (piece[1] << 24);
      dst[1] = (piece[1] >> 8) | (piece[2] << 16);
      dst[2] = (piece[2] >> 16) | (piece[3] << 8);
    } else {
      *reinterpret_cast<uint4*>(dst) = make_uint4(piece[0], piece[1], piece[2], piece[3]);
    }
  });
}

// The give-up path of ring_wait alone: one warp, a barrier nothing signals, a short limit.
__global__ void ring_wait_expiry_kernel(uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_addr(&bar), 1);
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  (void)ring_wait(ptx::smem_addr(&bar), 0u, &abort_word, WAIT_SELFTEST, 0, limit_ns);
}

// The flattened [out, in] weight as rows of 64 elements, one tile of kTileRows rows per copy.
inline bool weight_map(CUtensorMap* tm, const eqat_bf16* p, size_t n_elem) {
  return make_tmap_bf16(tm, p, 64, n_elem / 64, kTileRows);
}

inline bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// Persistent grid: every CTA resident at once, never more CTAs than tiles.  The kernel is a template
// argument so that each kernel has its own per-device state: the shared-memory opt-in and the number of
// CTAs that fit on an SM (both asked of the runtime once per device).
template <auto kernel, typename... Args>
int launch_stream(int smem_bytes, size_t n_elem, cudaStream_t st, Args... args) {
  static SmemOptIn opt_in;
  static std::atomic<int> ctas_per_sm[kMaxCachedDevices];
  if (!opt_in.ensure(kernel, smem_bytes)) return EQAT_ERR_CUDA;
  const int dev = current_device(), sms = sm_count();
  if (dev < 0 || sms <= 0) return EQAT_ERR_CUDA;
  int per_sm = dev < kMaxCachedDevices ? ctas_per_sm[dev].load(std::memory_order_relaxed) : 0;
  if (per_sm <= 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreadsS, smem_bytes) != cudaSuccess ||
        per_sm <= 0) {
      (void)cudaGetLastError();
      return EQAT_ERR_CUDA;
    }
    if (dev < kMaxCachedDevices) ctas_per_sm[dev].store(per_sm, std::memory_order_relaxed);
  }
  const size_t tiles = (n_elem + kTileElems - 1) / kTileElems;
  const size_t resident = (size_t)sms * per_sm;
  const unsigned grid = (unsigned)(tiles < resident ? tiles : resident);
  kernel<<<grid, kThreadsS, smem_bytes, st>>>(args...);
  return launch_status();
}

inline int group_shift_of(int group) {
  int sh = 5;
  while ((1 << sh) < group) ++sh;
  return sh;
}

}  // namespace

int launch_fakequant_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* What,
                            cudaStream_t st) {
  const size_t n_elem = (size_t)d.out_features * d.in_features;
  const float Q = (float)((1 << d.bits) - 1);
  CUtensorMap mw;
  if (!weight_map(&mw, W, n_elem)) return EQAT_ERR_CUDA;
  return launch_stream<fakequant_stream_kernel>(Ring<1, kStages1>::kSmemBytes, n_elem, st, mw, s, z, What, n_elem,
                                                group_shift_of(d.group), Q, (int)aligned32(What));
}

int launch_ste_bwd_stream(const eqat_desc& d, const eqat_bf16* dWhat, const eqat_bf16* W, const float* s,
                          const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st) {
  const size_t n_elem = (size_t)d.out_features * d.in_features;
  const float Q = (float)((1 << d.bits) - 1);
  const int lit = d.dz_mode == 1, wide = (int)aligned32(dW);
  CUtensorMap mg, mw;
  if (!weight_map(&mg, dWhat, n_elem) || !weight_map(&mw, W, n_elem)) return EQAT_ERR_CUDA;
  constexpr int smem = Ring<2, kStages2>::kSmemBytes;
  switch (d.group) {
    case 32:  return launch_stream<ste_bwd_stream_kernel<1>>(smem, n_elem, st, mg, mw, s, z, dW, ds, dz, n_elem, Q, lit, wide);
    case 64:  return launch_stream<ste_bwd_stream_kernel<2>>(smem, n_elem, st, mg, mw, s, z, dW, ds, dz, n_elem, Q, lit, wide);
    case 128: return launch_stream<ste_bwd_stream_kernel<4>>(smem, n_elem, st, mg, mw, s, z, dW, ds, dz, n_elem, Q, lit, wide);
    default:  return launch_stream<ste_bwd_stream_kernel<8>>(smem, n_elem, st, mg, mw, s, z, dW, ds, dz, n_elem, Q, lit, wide);
  }
}

int launch_minmax_stream(const eqat_desc& d, const eqat_bf16* W, float* s, float* z, cudaStream_t st) {
  const size_t n_elem = (size_t)d.out_features * d.in_features;
  const float Q = (float)((1 << d.bits) - 1);
  CUtensorMap mw;
  if (!weight_map(&mw, W, n_elem)) return EQAT_ERR_CUDA;
  constexpr int smem = Ring<1, kStages1>::kSmemBytes;
  switch (d.group) {
    case 32:  return launch_stream<minmax_stream_kernel<1>>(smem, n_elem, st, mw, s, z, n_elem, Q);
    case 64:  return launch_stream<minmax_stream_kernel<2>>(smem, n_elem, st, mw, s, z, n_elem, Q);
    case 128: return launch_stream<minmax_stream_kernel<4>>(smem, n_elem, st, mw, s, z, n_elem, Q);
    default:  return launch_stream<minmax_stream_kernel<8>>(smem, n_elem, st, mw, s, z, n_elem, Q);
  }
}

int launch_quantize_pack_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z,
                                uint8_t* packed, uint8_t* z8, eqat_fp16* s16, cudaStream_t st) {
  const size_t n_elem = (size_t)d.out_features * d.in_features;
  const int gs = group_shift_of(d.group);
  CUtensorMap mw;
  if (!weight_map(&mw, W, n_elem)) return EQAT_ERR_CUDA;
  constexpr int smem = Ring<1, kStages1>::kSmemBytes;
  switch (d.bits) {
    case 2:  return launch_stream<quantize_pack_stream_kernel<2>>(smem, n_elem, st, mw, s, z, packed, z8, s16, n_elem, gs);
    case 3:  return launch_stream<quantize_pack_stream_kernel<3>>(smem, n_elem, st, mw, s, z, packed, z8, s16, n_elem, gs);
    default: return launch_stream<quantize_pack_stream_kernel<4>>(smem, n_elem, st, mw, s, z, packed, z8, s16, n_elem, gs);
  }
}

int launch_wait_expiry_stream(cudaStream_t st) {
  ring_wait_expiry_kernel<<<1, 32, 0, st>>>(1000000ull);   // 1 ms
  return launch_status();
}

int read_stream_status(int* status, int* detail) {
  int h[2] = {0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess) return EQAT_ERR_CUDA;
  if (cudaMemcpyFromSymbol(h, g_stream_status, sizeof(h)) != cudaSuccess) return EQAT_ERR_CUDA;
  const int zero[2] = {0, 0};
  if (cudaMemcpyToSymbol(g_stream_status, zero, sizeof(zero)) != cudaSuccess) return EQAT_ERR_CUDA;
  *status = h[0];
  *detail = h[1];
  return EQAT_OK;
}

}  // namespace eqat
