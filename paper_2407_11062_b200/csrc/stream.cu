// Streaming kernels with TMA-staged inputs: fake quantiser (Eq. 1 + Eq. 2), its
// straight-through backward (Eqs. 3-5), min/max initialisation and quantise +
// pack, for groups of at most 256 elements.
//
// These kernels are bound by HBM bandwidth, and what decides how close they
// get to it is the number of bytes in flight per SM.  A plain "load, compute,
// store" thread keeps its loads in flight only until its arithmetic starts,
// and the arithmetic here is long (a division-free but exact quantiser per
// element).  So the loads are taken out of the compute threads: each persistent
// CTA has one producer thread that streams 8-16 KB chunks of the input(s) into
// a four-stage shared-memory ring with bulk asynchronous copies (cp.async.bulk,
// completion on an mbarrier), several chunks ahead, while 8 consumer warps pull
// 16-byte vectors from the ring, compute, and write results to global memory
// with coalesced 16-byte stores.  Three CTAs fit on an SM, so 150-190 KB of
// reads are in flight per SM whatever the consumers are doing.
//
// A quantisation group is contiguous in the flattened weight and owned by
// group/8 adjacent lanes of one warp; group sums are fixed-order shuffles, so
// results are run-to-run identical.
#include "common.cuh"
#include "elementwise.cuh"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace eqat {

__device__ int g_stream_status[2];   // [0] = eqat_status, [1] = WaitSite

namespace {

constexpr int kConsumers = 256;
constexpr int kThreadsS = kConsumers + 32;           // + one producer warp
// VPT = 16-byte vectors per consumer thread and chunk (a chunk is VPT * 4 KB per
// input stream): 4 for the one-input fake quantiser, 2 for the two-input STE
// backward, whose consumers need twice the registers per vector.
constexpr uint64_t kStreamWaitLimitNs = 2000000000ull;

template <int NIN, int VPT>
struct Ring {
  static constexpr int kChunkVec = VPT * kConsumers;          // vectors per chunk and stream
  static constexpr int kChunkBytes = kChunkVec * 16;
  static constexpr int kStages = 4;
  static constexpr int kStageBytes = NIN * kChunkBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 256;
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

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Runs `body(v, raw, params)` on every consumer thread for every chunk this CTA
// owns: v is the index of the thread's first vector, raw[i][u] the thread's
// vector u (v + u * 256) of input stream i, and params what `fetch(v)` returned
// for this chunk.  fetch is called one chunk ahead, so the small per-group loads
// it makes (step size, zero point) are in flight while the previous chunk is
// being computed instead of stalling this one.  Vectors at or beyond n_vec hold
// stale shared memory and must be ignored by the body.
template <int NIN, int VPT, typename Params, typename Fetch, typename Body>
__device__ __forceinline__ void stream_chunks(const uint8_t* const (&src)[NIN], size_t n_vec, Fetch&& fetch,
                                              Body&& body) {
  using R = Ring<NIN, VPT>;
  constexpr int kChunkVec = R::kChunkVec, kChunkBytes = R::kChunkBytes;
  extern __shared__ __align__(128) uint8_t smem[];
  RingCtl* ctl = reinterpret_cast<RingCtl*>(smem + R::kStages * R::kStageBytes);
  volatile int* abort_flag = &ctl->abort;
  const uint32_t smem_base = ptx::smem_addr(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t n_chunks = (n_vec + kChunkVec - 1) / kChunkVec;

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
      int stage = 0;
      uint32_t phase = 0;
      size_t issued = 0;
      bool ok = true;
      for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        if (!ring_wait(ptx::smem_addr(&ctl->empty[stage]), phase ^ 1u, abort_flag, WAIT_STREAM_EMPTY, 32)) {
          ok = false;
          break;
        }
        const size_t v0 = chunk * kChunkVec;
        const uint32_t bytes = (uint32_t)((n_vec - v0 < (size_t)kChunkVec ? n_vec - v0 : (size_t)kChunkVec) * 16);
        const uint32_t full = ptx::smem_addr(&ctl->full[stage]);
        ptx::mbar_expect_tx(full, NIN * bytes);
#pragma unroll
        for (int i = 0; i < NIN; ++i)
          bulk_load(smem_base + stage * R::kStageBytes + i * kChunkBytes, src[i] + v0 * 16, bytes, full);
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
    int stage = 0;
    uint32_t phase = 0;
    Params next = fetch((size_t)blockIdx.x * kChunkVec + threadIdx.x);
    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
      const Params cur = next;
      if (chunk + gridDim.x < n_chunks) next = fetch((chunk + gridDim.x) * kChunkVec + threadIdx.x);
      // the lanes of a warp leave together: the bodies shuffle across the whole warp
      const bool got = ring_wait(ptx::smem_addr(&ctl->full[stage]), phase, abort_flag, WAIT_STREAM_FULL, 0);
      if (!__all_sync(0xFFFFFFFFu, got)) break;
      uint4 raw[NIN][VPT];
      const uint8_t* st = smem + stage * R::kStageBytes;
#pragma unroll
      for (int i = 0; i < NIN; ++i)
#pragma unroll
        for (int u = 0; u < VPT; ++u)
          raw[i][u] = *reinterpret_cast<const uint4*>(st + i * kChunkBytes + (u * kConsumers + threadIdx.x) * 16);
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->empty[stage]));   // the stage can be refilled now
      if (++stage == R::kStages) { stage = 0; phase ^= 1u; }
      body(chunk * kChunkVec + threadIdx.x, raw, cur);
    }
  }
}

constexpr int kFakequantVpt = 4, kSteVpt = 2, kMinmaxVpt = 4, kPackVpt = 4;

// Step size and zero point of the groups of a thread's vectors.
template <int VPT>
struct GroupParams {
  float s[VPT], z[VPT];
};

template <int VPT>
__device__ __forceinline__ GroupParams<VPT> fetch_groups(const float* __restrict__ s, const float* __restrict__ z,
                                                    size_t v0, size_t n_vec, int vec_shift) {
  GroupParams<VPT> p;
#pragma unroll
  for (int u = 0; u < VPT; ++u) {
    const size_t v = v0 + (size_t)u * kConsumers;
    p.s[u] = 1.0f;
    p.z[u] = 0.0f;
    if (v < n_vec) {
      p.s[u] = __ldg(s + (v >> vec_shift));
      p.z[u] = __ldg(z + (v >> vec_shift));
    }
  }
  return p;
}

// ------------------------------------------------------------------ Eq. 1 + Eq. 2
// (clamp(r + z, 0, Q) - z) * s == clamp(r, -z, Q - z) * s for integer r and z.
__global__ void __launch_bounds__(kThreadsS)
fakequant_stream_kernel(const eqat_bf16* __restrict__ W, const float* __restrict__ s, const float* __restrict__ z,
                        eqat_bf16* __restrict__ What, size_t n_vec, int vec_shift, float Q) {
  const uint8_t* const src[1] = {reinterpret_cast<const uint8_t*>(W)};
  constexpr int VPT = kFakequantVpt;
  stream_chunks<1, VPT, GroupParams<VPT>>(src, n_vec,
      [&](size_t v0) { return fetch_groups<VPT>(s, z, v0, n_vec, vec_shift); },
      [&](size_t v0, const uint4 (&raw)[1][VPT], const GroupParams<VPT>& gp) {
#pragma unroll
    for (int u = 0; u < VPT; ++u) {
      const size_t v = v0 + (size_t)u * kConsumers;
      if (v < n_vec) {
        const float sv = gp.s[u];
        const float zr = rintf(gp.z[u]);
        const float rs = group_rcp(sv, zr);
        const float lo = -zr, hi = Q - zr;
        float w[8], r[8], rt[8];
        unpack8(raw[0][u], w);
        quotient_round8(w, sv, rs, r, rt);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = fminf(fmaxf(r[i], lo), hi) * sv;
        reinterpret_cast<uint4*>(What)[v] = pack8(w);
      }
    }
  });
}

// ------------------------------------------------------------------ Eqs. 3-5 + group sums
// With lo = -z, hi = Q - z and c = clamp(r, lo, hi): the element is in range iff
// c == r, and on the clamped branches Eq. 3's value (-z or Q - z) is c itself.
// Eq. 4 is a constant per group times the sum of the gradient over the clamped
// elements.  LPG = lanes per group (group / 8).
template <int LPG>
__global__ void __launch_bounds__(kThreadsS)
ste_bwd_stream_kernel(const eqat_bf16* __restrict__ dWhat, const eqat_bf16* __restrict__ W,
                      const float* __restrict__ s, const float* __restrict__ z, eqat_bf16* __restrict__ dW,
                      float* __restrict__ ds, float* __restrict__ dz, size_t n_vec, float Q, int dz_literal) {
  const uint8_t* const src[2] = {reinterpret_cast<const uint8_t*>(dWhat), reinterpret_cast<const uint8_t*>(W)};
  constexpr int vec_shift = LPG == 4 ? 2 : LPG == 8 ? 3 : LPG == 16 ? 4 : 5;
  constexpr int VPT = kSteVpt;
  stream_chunks<2, VPT, GroupParams<VPT>>(src, n_vec,
      [&](size_t v0) { return fetch_groups<VPT>(s, z, v0, n_vec, vec_shift); },
      [&](size_t v0, const uint4 (&raw)[2][VPT], const GroupParams<VPT>& gp) {
#pragma unroll
    for (int u = 0; u < VPT; ++u) {
      const size_t v = v0 + (size_t)u * kConsumers;
      const bool live = v < n_vec;                      // uniform over the lanes of a group
      const size_t g = v / LPG;
      float acc_s = 0.0f, acc_g = 0.0f;
      const float sv = gp.s[u];
      if (live) {
        const float zr = rintf(gp.z[u]);
        const float rs = group_rcp(sv, zr);
        const float lo = -zr, hi = Q - zr;
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
        reinterpret_cast<uint4*>(dW)[v] = pack8(w);
      }
#pragma unroll
      for (int d = LPG / 2; d >= 1; d >>= 1) {
        acc_s += __shfl_xor_sync(0xFFFFFFFFu, acc_s, d);
        acc_g += __shfl_xor_sync(0xFFFFFFFFu, acc_g, d);
      }
      if (live && (v % LPG) == 0) {
        ds[g] = acc_s;
        if (dz != nullptr) dz[g] = (dz_literal ? -1.0f : -sv) * acc_g;
      }
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
__global__ void __launch_bounds__(kThreadsS)
minmax_stream_kernel(const eqat_bf16* __restrict__ W, float* __restrict__ s, float* __restrict__ z, size_t n_vec,
                     float Q) {
  const uint8_t* const src[1] = {reinterpret_cast<const uint8_t*>(W)};
  constexpr int VPT = kMinmaxVpt;
  static_assert(kMinmaxVpt <= 4 && LPG >= 4, "one lane of a group finishes one of the thread's vectors");
  stream_chunks<1, VPT, NoParams>(src, n_vec, [](size_t) { return NoParams{}; },
      [&](size_t v0, const uint4 (&raw)[1][VPT], const NoParams&) {
    // Reduce each of the thread's VPT vectors over the lanes of its group (every lane ends up with the
    // group's extrema), then let lane u of the group finish vector u: one pass of the division code for
    // all VPT groups instead of VPT passes with one active lane per group.
    float mx_sel = 0.0f, mn_sel = 0.0f;
    const int sub = threadIdx.x % LPG;
#pragma unroll
    for (int u = 0; u < VPT; ++u) {
      const size_t v = v0 + (size_t)u * kConsumers;
      // extrema on packed bf16 pairs (exact: comparisons only), widened to fp32 at the end
      uint32_t mx2 = 0xFF80FF80u, mn2 = 0x7F807F80u;    // (-inf, -inf) and (+inf, +inf) as bf16 pairs
      if (v < n_vec) {                                  // uniform over the lanes of a group
        const uint4 r4 = raw[0][u];
        mx2 = bf162_max(bf162_max(r4.x, r4.y), bf162_max(r4.z, r4.w));
        mn2 = bf162_min(bf162_min(r4.x, r4.y), bf162_min(r4.z, r4.w));
      }
#pragma unroll
      for (int d = LPG / 2; d >= 1; d >>= 1) {
        mx2 = bf162_max(mx2, __shfl_xor_sync(0xFFFFFFFFu, mx2, d));
        mn2 = bf162_min(mn2, __shfl_xor_sync(0xFFFFFFFFu, mn2, d));
      }
      if (sub == u) {
        mx_sel = fmaxf(__uint_as_float(mx2 << 16), __uint_as_float(mx2 & 0xFFFF0000u));
        mn_sel = fminf(__uint_as_float(mn2 << 16), __uint_as_float(mn2 & 0xFFFF0000u));
      }
    }
    const size_t v = v0 - sub + (size_t)sub * kConsumers;          // first vector of the group this lane finishes
    if (sub < VPT && v < n_vec) {
      // s = max((max - min) / Q, 2^-14), z = clamp(-round(min / s), 0, Q), all in binary32
      float sv = __fdiv_rn(mx_sel - mn_sel, Q);
      sv = fmaxf(sv, 6.103515625e-05f);
      float zv = -rintf(__fdiv_rn(mn_sel, sv));
      zv = fminf(fmaxf(zv, 0.0f), Q) + 0.0f;
      s[v / LPG] = sv;
      z[v / LPG] = zv;
    }
  });
}

// ------------------------------------------------------------------ quantise + pack (hand-off)
// A thread turns one vector (8 weights) into 8*BITS bits; four adjacent lanes
// hold 32 consecutive codes, which lane 0 of the four assembles into BITS
// 32-bit words of the little-endian stream and stores.
template <int BITS>
__global__ void __launch_bounds__(kThreadsS)
quantize_pack_stream_kernel(const eqat_bf16* __restrict__ W, const float* __restrict__ s, const float* __restrict__ z,
                            uint8_t* __restrict__ packed, uint8_t* __restrict__ z8, eqat_fp16* __restrict__ s16,
                            size_t n_vec, int vec_shift) {
  const uint8_t* const src[1] = {reinterpret_cast<const uint8_t*>(W)};
  constexpr int VPT = kPackVpt;
  constexpr float Q = (float)((1 << BITS) - 1);
  stream_chunks<1, VPT, GroupParams<VPT>>(src, n_vec,
      [&](size_t v0) { return fetch_groups<VPT>(s, z, v0, n_vec, vec_shift); },
      [&](size_t v0, const uint4 (&raw)[1][VPT], const GroupParams<VPT>& gp) {
#pragma unroll
    for (int u = 0; u < VPT; ++u) {
      const size_t v = v0 + (size_t)u * kConsumers;
      const bool live = v < n_vec;                      // uniform over each 4 adjacent lanes (n_vec % 4 == 0)
      uint32_t piece = 0u;                              // this vector's 8 codes, code i at bits [BITS*i, BITS*i+BITS)
      if (live) {
        const float sv = gp.s[u];
        const float zr = rintf(gp.z[u]);
        const float rs = group_rcp(sv, zr);
        float w[8], r[8], rt[8];
        unpack8(raw[0][u], w);
        quotient_round8(w, sv, rs, r, rt);
        // The piece is sum_i code_i * 2^(BITS*i) with code_i = clamp(r_i + zr, 0, Q): evaluated by Horner's rule on the
        // integer-valued floats (exact: below 2^24), with one conversion per 16 or 24 bits instead of an add, a mask,
        // a shift and an or per code.
        constexpr float kRadix = (float)(1 << BITS);
        constexpr int kHalf = BITS == 4 ? 4 : 8;                                 // codes per conversion
#pragma unroll
        for (int h = 0; h < 8 / kHalf; ++h) {
          float acc = fminf(fmaxf(r[h * kHalf + kHalf - 1] + zr, 0.0f), Q);
#pragma unroll
          for (int i = kHalf - 2; i >= 0; --i) acc = fmaf(acc, kRadix, fminf(fmaxf(r[h * kHalf + i] + zr, 0.0f), Q));
          piece |= __float2uint_rn(acc) << (h * BITS * kHalf);
        }
        if ((v & (((size_t)1 << vec_shift) - 1)) == 0) {
          const size_t g = v >> vec_shift;
          z8[g] = (uint8_t)(__float_as_uint(fminf(fmaxf(zr, 0.0f), Q) + 8388608.0f) & 0xFFu);
          s16[g] = __half_as_ushort(__float2half_rn(sv));
        }
      }
      if constexpr (BITS == 4) {
        if (live) reinterpret_cast<uint32_t*>(packed)[v] = piece;                // 32 bits per vector: store directly
      } else {
        const uint32_t p1 = __shfl_down_sync(0xFFFFFFFFu, piece, 1);
        const uint32_t p2 = __shfl_down_sync(0xFFFFFFFFu, piece, 2);
        const uint32_t p3 = __shfl_down_sync(0xFFFFFFFFu, piece, 3);
        if (live && (threadIdx.x & 3) == 0) {
          if constexpr (BITS == 2) {
            reinterpret_cast<uint2*>(packed)[v >> 2] = make_uint2(piece | (p1 << 16), p2 | (p3 << 16));
          } else {
            uint32_t* dst = reinterpret_cast<uint32_t*>(packed) + (v >> 2) * 3;
            dst[0] = piece | (p1 << 24);
            dst[1] = (p1 >> 8) | (p2 << 16);
            dst[2] = (p2 >> 16) | (p3 << 8);
          }
        }
      }
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

// Persistent grid: every CTA resident at once, never more CTAs than chunks.  The kernel is a template
// argument so that each kernel has its own per-device state: the shared-memory opt-in and the number of
// CTAs that fit on an SM (both asked of the runtime once per device).
template <auto kernel, typename... Args>
int launch_stream(int smem_bytes, int chunk_vec, size_t n_vec, cudaStream_t st, Args... args) {
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
  const size_t chunks = (n_vec + chunk_vec - 1) / chunk_vec;
  const size_t resident = (size_t)sms * per_sm;
  const unsigned grid = (unsigned)(chunks < resident ? chunks : resident);
  kernel<<<grid, kThreadsS, smem_bytes, st>>>(args...);
  return launch_status();
}

}  // namespace

int launch_fakequant_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z, eqat_bf16* What,
                            cudaStream_t st) {
  const size_t n_vec = (size_t)d.out_features * d.in_features / 8;
  const float Q = (float)((1 << d.bits) - 1);
  int vec_shift = 0;
  while ((8 << vec_shift) < d.group) ++vec_shift;
  using R = Ring<1, kFakequantVpt>;
  return launch_stream<fakequant_stream_kernel>(R::kSmemBytes, R::kChunkVec, n_vec, st, W, s, z, What, n_vec, vec_shift, Q);
}

int launch_ste_bwd_stream(const eqat_desc& d, const eqat_bf16* dWhat, const eqat_bf16* W, const float* s,
                          const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st) {
  const size_t n_vec = (size_t)d.out_features * d.in_features / 8;
  const float Q = (float)((1 << d.bits) - 1);
  const int lit = d.dz_mode == 1;
  using R = Ring<2, kSteVpt>;
  constexpr int smem = R::kSmemBytes, cv = R::kChunkVec;
  switch (d.group) {
    case 32:  return launch_stream<ste_bwd_stream_kernel<4>>(smem, cv, n_vec, st, dWhat, W, s, z, dW, ds, dz, n_vec, Q, lit);
    case 64:  return launch_stream<ste_bwd_stream_kernel<8>>(smem, cv, n_vec, st, dWhat, W, s, z, dW, ds, dz, n_vec, Q, lit);
    case 128: return launch_stream<ste_bwd_stream_kernel<16>>(smem, cv, n_vec, st, dWhat, W, s, z, dW, ds, dz, n_vec, Q, lit);
    default:  return launch_stream<ste_bwd_stream_kernel<32>>(smem, cv, n_vec, st, dWhat, W, s, z, dW, ds, dz, n_vec, Q, lit);
  }
}

int launch_minmax_stream(const eqat_desc& d, const eqat_bf16* W, float* s, float* z, cudaStream_t st) {
  const size_t n_vec = (size_t)d.out_features * d.in_features / 8;
  const float Q = (float)((1 << d.bits) - 1);
  using R = Ring<1, kMinmaxVpt>;
  constexpr int smem = R::kSmemBytes, cv = R::kChunkVec;
  switch (d.group) {
    case 32:  return launch_stream<minmax_stream_kernel<4>>(smem, cv, n_vec, st, W, s, z, n_vec, Q);
    case 64:  return launch_stream<minmax_stream_kernel<8>>(smem, cv, n_vec, st, W, s, z, n_vec, Q);
    case 128: return launch_stream<minmax_stream_kernel<16>>(smem, cv, n_vec, st, W, s, z, n_vec, Q);
    default:  return launch_stream<minmax_stream_kernel<32>>(smem, cv, n_vec, st, W, s, z, n_vec, Q);
  }
}

int launch_quantize_pack_stream(const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z,
                                uint8_t* packed, uint8_t* z8, eqat_fp16* s16, cudaStream_t st) {
  const size_t n_vec = (size_t)d.out_features * d.in_features / 8;
  int vec_shift = 0;
  while ((8 << vec_shift) < d.group) ++vec_shift;
  using R = Ring<1, kPackVpt>;
  constexpr int smem = R::kSmemBytes, cv = R::kChunkVec;
  switch (d.bits) {
    case 2:  return launch_stream<quantize_pack_stream_kernel<2>>(smem, cv, n_vec, st, W, s, z, packed, z8, s16, n_vec, vec_shift);
    case 3:  return launch_stream<quantize_pack_stream_kernel<3>>(smem, cv, n_vec, st, W, s, z, packed, z8, s16, n_vec, vec_shift);
    default: return launch_stream<quantize_pack_stream_kernel<4>>(smem, cv, n_vec, st, W, s, z, packed, z8, s16, n_vec, vec_shift);
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
