// tcgen05 GEMM kernels for the quantised linear layer.
//
// One persistent, warp-specialised kernel template computes
//     D[M,N] = sum_k A[m,k] * B[n,k]          (bf16 x bf16 -> fp32 in TMEM)
// for the three contractions of the layer.  Each operand is either K-major
// (rows of K contiguous elements) or MN-major (the row-major transpose), so no
// transposed copy of X, dY or W_hat is ever materialised:
//     Y    = X  * W_hat^T : A = X  [T,in]  K-major,  B = W_hat [out,in] K-major
//     dX   = dY * W_hat   : A = dY [T,out] K-major,  B = W_hat [out,in] MN-major
//     dW^  = dY^T * X     : A = dY [T,out] MN-major, B = X     [T,in]  MN-major
//
// Roles inside a CTA (one CTA per SM, (MT*128) x BN output tile, 64-deep K blocks;
// MT = 1 with two TMEM accumulator sets so the epilogue overlaps the next tile,
// MT = 2 for the packed-weight kernels so each expanded B stage feeds two MMAs):
//   warp 0      TMA producer: fills a ring of 128B-swizzled shared-memory stages
//   warp 1      MMA issuer: one thread issues tcgen05.mma into one of two TMEM
//               accumulators, frees stages with tcgen05.commit
//   warps 2-5   epilogue: tcgen05.ld the finished accumulator (one TMEM lane
//               quadrant each); with MT = 1 the next tile is already being
//               multiplied meanwhile
//   warps 2-17  (packed-weight kernels only) expand N-bit codes into the bf16 B
//               operand, (q - z) * s exactly, rounded once to bf16.  That operand
//               has a ring of four stages of its own (the TMA-fed A ring has
//               three), and two groups of eight warps take alternate runs of one
//               or two K blocks, one 64-code row per thread and K block, so two
//               stages are being expanded at any time and each group owns two of
//               the four.  Warps 2-5
//               then run the epilogue of the tile (MT = 2: nothing overlaps it
//               anyway, and the other warps meanwhile pre-expand the next tile's
//               first stages up to the point where they need these four)
// The epilogue either stores the tile as bf16; or, for the E2E-QP step-size
// gradient, multiplies each accumulator row by (q - z) of the matching packed
// codes and reduces runs of `group` columns, so the [out,in] weight gradient
// never leaves the chip; or, for the Block-AP weight gradient, applies Eqs. 3-5
// to the accumulators next to the latent weights and writes dW, ds and dz.
// Packed kernels walk their tiles row by row (the few MB of codes stay in L2,
// each activation panel is fetched once); dense kernels in bands of 16 row-tiles.
//
// Every wait on an mbarrier is bounded in time; a role that gives up raises a
// CTA-wide abort flag, records the site in a device status word and all roles
// fall through to a teardown that drains copies in flight and frees TMEM.
#include <cuda.h>

#include "common.cuh"
#include "codec.cuh"
#include "gemm.cuh"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace eqat {

__device__ int g_device_status[2];   // [0] = eqat_status, [1] = WaitSite

namespace {

constexpr int BM = 128;          // rows per MMA = TMEM lanes
constexpr int BK = 64;           // K per stage: one 128-byte swizzle span of bf16
constexpr int UMMA_K = 16;       // K per tcgen05.mma for 16-bit inputs
constexpr int kEpiWarps = 4;       // dense kernels: warps 2-5 are the epilogue
constexpr int kDeqWarps = 16;      // packed kernels: warps 2-17 expand codes; warps 2-5 also run the epilogue
constexpr uint64_t kWaitLimitNs = 2000000000ull;   // 2 s per wait
constexpr uint64_t kDrainLimitNs = 50000000ull;    // 50 ms per stage at teardown

enum Epilogue : int { EPI_STORE = 0, EPI_DS = 1, EPI_STE = 2 };

struct GemmParams {
  int M, N, K;
  eqat_bf16* D;              // EPI_STORE: [M,N] row-major
  // packed weight (B operand of the packed kernels, epilogue operand of EPI_DS)
  const uint8_t* Wq;         // [out, in*bits/8]
  const eqat_fp16* s16;      // [out, in/group]
  const uint8_t* z8;         // [out, in/group]
  int out_features, in_features;
  int group_shift;           // log2(group)
  int wq_sectors;            // Wq is 32-byte aligned: a thread may fetch a whole 32-byte sector with one load
  float* ds;                 // EPI_DS / EPI_STE outputs [out, in/group]
  float* dz;                 // may be null
  // EPI_STE: latent weight and Block-AP quantiser parameters of the [out,in] tile rows
  const eqat_bf16* W;        // [out, in]
  const float* s32;          // [out, in/group]
  const float* z32;          // [out, in/group]
  float Q;                   // 2^N - 1
  int dz_literal;            // Eq. 4 clamped branch: -1 instead of -s
};

template <int BN, int MT, bool PACKED>
struct Cfg {
  static constexpr int kTileM = MT * BM;                 // output rows per CTA tile
  static constexpr int kAccSets = MT == 1 ? 2 : 1;       // TMEM holds kAccSets * MT accumulators of BN columns
  static constexpr int kStages = MT == 2 ? 3 : (BN == 256 ? 4 : 6);
  // Packed kernels keep the expanded B operand in a ring of its own, one stage deeper than the TMA-fed A
  // ring: an expansion takes longer than a copy, and the extra B stage is what lets it run a K block further
  // ahead of the tensor core.  Dense kernels keep A and B of a stage side by side.
  static constexpr int kStagesB = PACKED ? kStages + 1 : kStages;
  static constexpr int kABytes = kTileM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kRingBytes = kStages * kABytes + kStagesB * kBBytes;
  __host__ __device__ static constexpr int a_offset(int stage) { return PACKED ? stage * kABytes : stage * kStageBytes; }
  __host__ __device__ static constexpr int b_offset(int stage_b) {
    return PACKED ? kStages * kABytes + stage_b * kBBytes : stage_b * kStageBytes + kABytes;
  }
  static constexpr int kThreads = (2 + (PACKED ? kDeqWarps : kEpiWarps)) * 32;
  static constexpr int kTmemCols = kAccSets * MT * BN;
  static constexpr int kSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
  static_assert(kSmemBytes <= 232448, "stage rings exceed the shared memory of one CTA");
};

struct Control {
  uint64_t full[8];          // A (and, dense kernels, B) stage filled by TMA
  uint64_t empty[8];
  uint64_t full_b[4];        // packed kernels: B stage expanded
  uint64_t empty_b[4];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort;
};
static_assert(sizeof(Control) <= 256, "control block must fit its reservation");

// Bounded wait on an mbarrier phase.  `sleep_ns` > 0 backs off between polls so
// that a role with nothing to do for a long time (the epilogue during a main
// loop, the producer on a full ring) leaves the issue slots to the warps that
// are working; latency-critical waits pass 0.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort, int site,
                                             uint32_t sleep_ns = 0, uint64_t limit_ns = kWaitLimitNs) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t n = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if (sleep_ns != 0) __nanosleep(sleep_ns);
    if ((++n & 31u) == 0u) {
      if (*abort) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) {
        *abort = 1;
        atomicExch(&g_device_status[1], site);
        atomicExch(&g_device_status[0], (int)EQAT_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Shared-memory matrix descriptor, 128-byte swizzle, 8-row atoms 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(1024u >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}

template <bool ROW_ORDER>
__device__ __forceinline__ void tile_coords(int tile, int num_m, int num_n, int& m_blk, int& n_blk) {
  if (ROW_ORDER) {
    // Packed kernels: the B operand (N-bit codes, a few MB) lives in L2 whatever the order, so tiles run along
    // a row of tiles first and each A panel is fetched by one wave of CTAs only.
    m_blk = tile / num_n;
    n_blk = tile - m_blk * num_n;
    return;
  }
  // Bands of 16 row-tiles, row-tile fastest inside a band: the ~148 tiles in
  // flight share 16 A panels and ~9 B panels in L2.
  const int band_tiles = 16 * num_n;
  const int band = tile / band_tiles;
  const int r = tile - band * band_tiles;
  const int m0 = band * 16;
  const int h = min(16, num_m - m0);
  m_blk = m0 + r % h;
  n_blk = r / h;
}

// Expand 64 consecutive codes of one weight row into one 128-byte swizzled
// shared-memory row: element e of the row goes to 16-byte chunk (e/8) ^ rx.
//
// A code q is dropped into bits 16..23 of the float 0x4B000000 (= 2^23), giving
// x = 2^23 + 65536*q exactly.  Then fma(x, s/65536, -(128 + z)*s) = (q - z)*s:
// s is an fp16 value (11 significant bits), so s/65536 and (128 + z)*s are
// exact in fp32 and so is the result; the only rounding is the final one to
// bf16.  4-bit codes reach byte positions with one shift+mask per 4 codes and
// one byte permute each; 3-bit codes are shifted individually; 2-bit codes use
// a 4-entry table per group instead (see below).
struct DequantScale {
  float sp, cz;
  __device__ __forceinline__ DequantScale(float s, float z) : sp(s * (1.0f / 65536.0f)), cz(-(128.0f + z) * s) {}
  __device__ __forceinline__ float operator()(uint32_t xbits) const { return fmaf(__uint_as_float(xbits), sp, cz); }
};

//
// `row_sx` is the shared-memory address of the row XOR (rx << 4): the row is 128-byte aligned, so chunk c
// lies at row_sx ^ (c << 4), one logic operation per store.
__device__ __forceinline__ void store_chunk(uint32_t row_sx, int chunk, const float (&v)[8]) {
  ptx::sts_128(row_sx ^ ((uint32_t)chunk << 4), pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
               pack_bf16x2(v[6], v[7]));
}

// Expands 32 consecutive codes (half h of a 64-code row) into chunks 4h .. 4h+3.
template <int BITS>
__device__ __forceinline__ void dequant_half32(const uint32_t (&w)[BITS], float s, float z, uint32_t row_sx, int h) {
  constexpr uint32_t kMagic = 0x4B000000u;
  if constexpr (BITS == 2) {
    // Four possible values per group: build them once, exactly, as bf16
    // ((q - z)*s has at most 13 significant bits, so the fp32 value is exact and
    // the conversion is the only rounding), then look each code up with a byte
    // permute.  lut01 = (v0, v1), lut23 = (v2, v3); value q occupies bytes 2q, 2q+1
    // of the 8-byte pair, so the selector byte of a code is 0x10 + 0x22*q.
    const float zs = z * s;
    const uint32_t lut01 = pack_bf16x2(-zs, s - zs);
    const uint32_t lut23 = pack_bf16x2(fmaf(2.0f, s, -zs), fmaf(3.0f, s, -zs));
#pragma unroll
    for (int i = 0; i < 2; ++i) {                       // word i: codes 16i .. 16i+15 of the half
      uint32_t sel[4];                                  // byte b of sel[r] = selector byte of code 4b + r
#pragma unroll
      for (int r = 0; r < 4; ++r) sel[r] = ((w[i] >> (2 * r)) & 0x03030303u) * 0x22u + 0x10101010u;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t o[4];
#pragma unroll
        for (int pr = 0; pr < 4; ++pr) {
          const int k = 8 * c + 2 * pr;                 // even code of the pair; k = 4b + r with r in {0, 2}
          const uint32_t b = (uint32_t)(k >> 2), r = (uint32_t)(k & 3);
          const uint32_t pair_sel = __byte_perm(sel[r], sel[r + 1], b | ((4u + b) << 4));
          o[pr] = __byte_perm(lut01, lut23, pair_sel);
        }
        ptx::sts_128(row_sx ^ ((uint32_t)(4 * h + 2 * i + c) << 4), o[0], o[1], o[2], o[3]);
      }
    }
  } else if constexpr (BITS == 4) {
    const DequantScale f(s, z);
#pragma unroll
    for (int i = 0; i < 4; ++i) {                       // word i: codes 8i .. 8i+7 of the half
      const uint32_t m0 = w[i] & 0x0F0F0F0Fu, m1 = (w[i] >> 4) & 0x0F0F0F0Fu;   // byte b = code 2b (+1)
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e)
        v[e] = f(__byte_perm((e & 1) ? m1 : m0, kMagic, 0x7044u | ((uint32_t)(e >> 1) << 8)));
      store_chunk(row_sx, 4 * h + i, v);
    }
  } else {
    const DequantScale f(s, z);
#pragma unroll
    for (int c = 0; c < 4; ++c) {                       // 32 codes = 3 words
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int bit = 3 * (8 * c + e), word = bit >> 5, off = bit & 31;
        uint32_t t;
        if (off <= 16) {
          t = w[word] << (16 - off);
        } else {
          const uint32_t hi = (off + 3 > 32) ? w[word + 1] : 0u;
          t = __funnelshift_r(w[word], hi, off - 16);
        }
        v[e] = f((t & 0x00070000u) | kMagic);
      }
      store_chunk(row_sx, 4 * h + c, v);
    }
  }
}

// 64 codes = 2*BITS consecutive 32-bit words, at a multiple of 8*BITS bytes.
template <int BITS>
__device__ __forceinline__ void load_codes64(const uint8_t* p, uint32_t (&w)[2 * BITS]) {
  if constexpr (BITS == 2) {
    const uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
    w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
  } else if constexpr (BITS == 3) {
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      const uint2 t = __ldg(reinterpret_cast<const uint2*>(p) + i);
      w[2 * i] = t.x; w[2 * i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint4 t = __ldg(reinterpret_cast<const uint4*>(p) + i);
      w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
    }
  }
}

// 4 x 4 transpose of 16-byte pieces inside each quad of lanes.  In: o[4p .. 4p+3] = piece p (8 bf16 columns) of the
// lane's own row.  Out: o[4k .. 4k+3] = piece (lane & 3) of the row owned by lane k of the quad.  Two butterfly
// rounds; in round b the pieces whose index differs from the lane's in bit b change lane and slot.
__device__ __forceinline__ void quad_transpose(uint32_t (&o)[16], int lane) {
#pragma unroll
  for (int b = 1; b >= 0; --b) {
    const bool up = (lane >> b) & 1;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int s0 = b == 1 ? j : 2 * j, s1 = s0 + (1 << b);        // slots that differ in bit b only
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const uint32_t send = up ? o[4 * s0 + w] : o[4 * s1 + w];
        const uint32_t recv = __shfl_xor_sync(0xFFFFFFFFu, send, 1 << b);
        if (up) o[4 * s0 + w] = recv; else o[4 * s1 + w] = recv;
      }
    }
  }
}

// A_MN / B_MN: operand is MN-major.  PACKED: B is expanded from N-bit codes.
// BITS is used by PACKED and by EPI_DS.
template <int BN, int MT, bool A_MN, bool B_MN, bool PACKED, int EPI, int BITS>
__global__ void __launch_bounds__(Cfg<BN, MT, PACKED>::kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const GemmParams p) {
  using C = Cfg<BN, MT, PACKED>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_addr(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;                                  // 1024-byte aligned stages
  const uint32_t smem_base = raw_addr + pad;
  Control* ctl = reinterpret_cast<Control*>(smem + C::kRingBytes);
  volatile int* abort_flag = &ctl->abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int num_m = (p.M + C::kTileM - 1) / C::kTileM;
  const int num_n = (p.N + BN - 1) / BN;
  const int num_tiles = num_m * num_n;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), 1);
    }
    if (PACKED) {
      for (int s = 0; s < C::kStagesB; ++s) {
        ptx::mbar_init(ptx::smem_addr(&ctl->full_b[s]), kDeqWarps / 2);
        ptx::mbar_init(ptx::smem_addr(&ctl->empty_b[s]), 1);
      }
    }
    for (int a = 0; a < C::kAccSets; ++a) {
      ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[a]), 1);
      ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[a]), 4);
    }
    ptx::mbar_init(ptx::smem_addr(&ctl->drain), 1);
    ctl->abort = 0;
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&tmap_a);
    if (!PACKED) ptx::tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_base), C::kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  // ---------------------------------------------------------------- epilogue of one tile
  // Run by four warps, one per TMEM lane quadrant (warp index mod 4).
  const int quad = warp & 3;
  const int row_in_tile = quad * 32 + lane;
  auto epilogue_tile = [&](int m_blk, int n_blk, int acc, uint32_t acc_phase) -> bool {
    // The lanes of a warp must leave together: the store epilogue below shuffles across the whole warp.
    const bool got = wait_bounded(ptx::smem_addr(&ctl->acc_full[acc]), acc_phase, abort_flag, WAIT_EPI_ACC_FULL,
                                  PACKED ? 0 : (MT == 2 ? 512 : 128));
    if (!__all_sync(0xFFFFFFFFu, got)) return false;
    ptx::tc_fence_after();
#pragma unroll 1
    for (int h = 0; h < MT; ++h) {
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((acc * MT + h) * BN);
      const int m = m_blk * C::kTileM + h * BM + row_in_tile;
      if constexpr (EPI == EPI_STORE) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          ptx::tmem_ld_32x32(t_row + c * 32, r);
          ptx::tmem_ld_wait();
          const int col0 = n_blk * BN + c * 32;
          // A lane owns a row, so a plain store instruction would hit 32 different lines, and it is the stores, not
          // the TMEM loads, that set the pace of this epilogue.  The four lanes of a quad therefore trade 16-byte
          // pieces so that each store instruction writes 64 contiguous bytes of one row per quad: 8 lines instead
          // of 32.  (N is a multiple of 16 for every shape the library accepts, so a piece is never ragged.)
          uint32_t o[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) o[i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
          quad_transpose(o, lane);
          const int q = lane & 3;
          if (col0 + q * 8 < p.N) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int mk = m - q + k;
              if (mk < p.M)
                *reinterpret_cast<uint4*>(p.D + (size_t)mk * p.N + col0 + q * 8) =
                    make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            }
          }
        }
      } else if constexpr (EPI == EPI_STE) {
        // Block-AP: the accumulator row is the gradient of row m of W_hat.  Eqs. 3-5 are applied to it here,
        // in fp32, next to the matching latent weights: dW = G where the code is in range, ds and dz are the
        // group sums of G times the partials.  G itself is never written.
        const int groups_per_row = p.N >> p.group_shift;
        const int chunks_per_group = 1 << (p.group_shift - 5);
        const eqat_bf16* wrow = p.W + (size_t)m * p.N;
        eqat_bf16* drow = p.D + (size_t)m * p.N;
        float acc_s = 0.0f, acc_g = 0.0f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          const int col0 = n_blk * BN + c * 32;
          const bool live = m < p.M && col0 < p.N;
          uint4 wraw[4];
          float sv = 1.0f, zr = 0.0f;
          if (live) {
#pragma unroll
            for (int v = 0; v < 4; ++v) wraw[v] = __ldg(reinterpret_cast<const uint4*>(wrow + col0) + v);
            const size_t gi = (size_t)m * groups_per_row + (col0 >> p.group_shift);
            sv = __ldg(p.s32 + gi);
            zr = rintf(__ldg(p.z32 + gi));
          }
          uint32_t r32[32];
          ptx::tmem_ld_32x32(t_row + c * 32, r32);
          ptx::tmem_ld_wait();
          if (live) {
            const float rs = group_rcp(sv, zr);
            const float lo = -zr, hi = p.Q - zr;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              float w[8], r[8], rt[8];
              unpack8(wraw[v], w);
              quotient_round8(w, sv, rs, r, rt);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float gr = __uint_as_float(r32[8 * v + i]);
                const float cl = fminf(fmaxf(r[i], lo), hi);
                const bool inside = (cl == r[i]);
                acc_s = fmaf(gr, inside ? rt[i] : cl, acc_s);     // Eq. 3
                acc_g += inside ? 0.0f : gr;                      // Eq. 4
                w[i] = inside ? gr : 0.0f;                        // Eq. 5
              }
              reinterpret_cast<uint4*>(drow + col0)[v] = pack8(w);
            }
            if (((c + 1) & (chunks_per_group - 1)) == 0) {
              const size_t gi = (size_t)m * groups_per_row + (col0 >> p.group_shift);
              p.ds[gi] = acc_s;
              if (p.dz != nullptr) p.dz[gi] = (p.dz_literal ? -1.0f : -sv) * acc_g;
              acc_s = 0.0f;
              acc_g = 0.0f;
            }
          }
        }
      } else {
        // Row m of the tile is output row o = m of the weight; columns are input
        // features.  ds[o,g] = sum_{j in g} G[o,j] * (q[o,j] - z[o,g]).
        const int groups_per_row = p.in_features >> p.group_shift;
        const int chunks_per_group = 1 << (p.group_shift - 5);
        const uint8_t* qrow = p.Wq + (size_t)m * ((size_t)p.in_features * BITS / 8);
        float acc_s = 0.0f, acc_g = 0.0f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          ptx::tmem_ld_32x32(t_row + c * 32, r);
          ptx::tmem_ld_wait();
          const int col0 = n_blk * BN + c * 32;
          if (m < p.M && col0 < p.N) {
            uint32_t words[BITS];
            const uint32_t* src = reinterpret_cast<const uint32_t*>(qrow) + (size_t)(col0 >> 5) * BITS;
#pragma unroll
            for (int i = 0; i < BITS; ++i) words[i] = __ldg(src + i);
            uint32_t codes[32];
            unpack32<BITS>(words, codes);
            const int g = col0 >> p.group_shift;
            const float zf = (float)__ldg(p.z8 + (size_t)m * groups_per_row + g);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float gv = __uint_as_float(r[i]);
              acc_s = fmaf(gv, (float)codes[i] - zf, acc_s);
              acc_g += gv;
            }
            if (((c + 1) & (chunks_per_group - 1)) == 0) {
              const size_t idx = (size_t)m * groups_per_row + g;
              p.ds[idx] = acc_s;
              if (p.dz != nullptr) p.dz[idx] = -__half2float(__ushort_as_half(__ldg(p.s16 + idx))) * acc_g;
              acc_s = 0.0f;
              acc_g = 0.0f;
            }
          }
        }
      }
    }
    ptx::tc_fence_before();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->acc_empty[acc]));
    return true;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int m_blk, n_blk;
        tile_coords<PACKED>(tile, num_m, num_n, m_blk, n_blk);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bounded(ptx::smem_addr(&ctl->empty[stage]), phase ^ 1u, abort_flag, WAIT_PRODUCER_EMPTY, 64)) {
            ok = false;
            break;
          }
          const uint32_t full = ptx::smem_addr(&ctl->full[stage]);
          const uint32_t a_dst = smem_base + C::a_offset(stage);
          const uint32_t b_dst = smem_base + C::b_offset(stage);
          ptx::mbar_expect_tx(full, PACKED ? C::kABytes : C::kStageBytes);
          if (A_MN) {
#pragma unroll
            for (int b = 0; b < C::kTileM / 64; ++b)
              ptx::tma_load_2d(a_dst + b * (BK * 128), &tmap_a, m_blk * C::kTileM + b * 64, kb * BK, full);
          } else {
            ptx::tma_load_2d(a_dst, &tmap_a, kb * BK, m_blk * C::kTileM, full);
          }
          if (!PACKED) {
            if (B_MN) {
#pragma unroll
              for (int b = 0; b < BN / 64; ++b)
                ptx::tma_load_2d(b_dst + b * (BK * 128), &tmap_b, n_blk * BN + b * 64, kb * BK, full);
            } else {
              ptx::tma_load_2d(b_dst, &tmap_b, kb * BK, n_blk * BN, full);
            }
          }
          ++issued;
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        // Drain: every copy this thread started must land before the CTA exits.
        const long first = issued > C::kStages ? issued - C::kStages : 0;
        for (long i = first; i < issued; ++i) {
          const uint32_t bar = ptx::smem_addr(&ctl->full[i % C::kStages]);
          const uint32_t par = (uint32_t)((i / C::kStages) & 1);
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(bar, par)) {
            if (ptx::globaltimer_ns() - t0 > kDrainLimitNs) {
              atomicExch(&g_device_status[1], (int)WAIT_TEARDOWN);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
      constexpr uint32_t a_lbo = A_MN ? BK * 128 : 16, b_lbo = B_MN ? BK * 128 : 16;
      constexpr uint32_t a_step = A_MN ? UMMA_K * 128 : UMMA_K * 2, b_step = B_MN ? UMMA_K * 128 : UMMA_K * 2;
      constexpr uint32_t a_half = BM * BK * 2;        // second 128-row half of the A stage (either major)
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!wait_bounded(ptx::smem_addr(&ctl->acc_empty[acc]), acc_phase ^ 1u, abort_flag, WAIT_MMA_ACC_EMPTY, 64)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * MT * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bounded(ptx::smem_addr(&ctl->full[stage]), phase, abort_flag, WAIT_MMA_FULL, PACKED ? 32 : 0) ||
              (PACKED &&
               !wait_bounded(ptx::smem_addr(&ctl->full_b[stage_b]), phase_b, abort_flag, WAIT_MMA_FULL, 32))) {
            ok = false;
            break;
          }
          ptx::tc_fence_after();
          const uint32_t a_addr = smem_base + C::a_offset(stage);
          const uint32_t b_addr = smem_base + C::b_offset(PACKED ? stage_b : stage);
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            const uint64_t b_desc = smem_desc(b_addr + kk * b_step, b_lbo);
#pragma unroll
            for (int h = 0; h < MT; ++h)
              ptx::mma_bf16_ss(d_tmem + h * BN, smem_desc(a_addr + h * a_half + kk * a_step, a_lbo), b_desc, idesc,
                               (kb | kk) != 0 ? 1u : 0u);
          }
          ptx::mma_commit(ptx::smem_addr(&ctl->empty[stage]));
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
          if (PACKED) {
            ptx::mma_commit(ptx::smem_addr(&ctl->empty_b[stage_b]));
            if (++stage_b == C::kStagesB) { stage_b = 0; phase_b ^= 1u; }
          }
        }
        if (!ok) break;
        ptx::mma_commit(ptx::smem_addr(&ctl->acc_full[acc]));
        if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
      }
      // All MMAs of this thread must have retired before TMEM is freed.
      ptx::mma_commit(ptx::smem_addr(&ctl->drain));
      wait_bounded(ptx::smem_addr(&ctl->drain), 0u, abort_flag, WAIT_TEARDOWN, 64, kDrainLimitNs * 4);
    }
  } else if (!PACKED) {
    // ------------------------------------------------------------ epilogue warps (dense kernels)
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      int m_blk, n_blk;
      tile_coords<PACKED>(tile, num_m, num_n, m_blk, n_blk);
      if (!epilogue_tile(m_blk, n_blk, acc, acc_phase)) break;
      if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------ dequantisers (+ epilogue on warps 2-5)
    if constexpr (PACKED) {
      // Sixteen warps in two groups of eight: group 0 expands the even K blocks (counted over all tiles of
      // this CTA), group 1 the odd ones, each thread one whole 64-code unit (one 128-byte operand row) of
      // its K blocks.  Two stages are thus being expanded at any time, and the per-K-block bookkeeping
      // (wait, fence, arrive, addresses, step size) is paid once per 64 codes.
      const int t = (threadIdx.x - 64) & 255;                     // unit within the stage
      const int grp = (threadIdx.x - 64) >> 8;                    // 0 or 1
      const size_t pitch = (size_t)p.in_features * BITS / 8;      // bytes per packed row
      const int groups_per_row = p.in_features >> p.group_shift;
      const int chunks_in = p.in_features >> 6;                   // 64-code units per row
      bool ok = true;
      //   B K-major  (Y):  tile row t is weight row n0 + t, unit = kb
      //   B MN-major (dX): k-row kr is weight row kb*64 + kr, unit = n0/64 + box (64-column box)
      // The 8 lanes of a quarter-warp (one 16-byte store wavefront) own 8 consecutive
      // rows, whose swizzled chunks fall in 8 different bank groups.
      const int kr = (t & 7) | ((t >> 5) << 3);                   // MN-major: k-row 0..63
      const int box = (t >> 3) & 3;                               // MN-major: 64-column box 0..3
      const int smem_row_off = B_MN ? (box * (BK * 128) + kr * 128) : t * 128;
      const int rx = B_MN ? (kr & 7) : (t & 7);
      const uint32_t smem_row_sx = (uint32_t)smem_row_off ^ ((uint32_t)rx << 4);   // stage bases are 1024-byte aligned
      // Step sizes and zero points.  With a K-major B operand a thread stays on one
      // weight row for a whole tile and walks its groups in order, so it reads
      // them four groups at a time (one 8-byte and one 4-byte load per four
      // groups, a block ahead of use) instead of one 2-byte and one 1-byte load
      // per K block: 32 lanes on 32 different rows make every such load 32
      // separate L1 transactions, and those were what bounded the kernel.
      const bool sz_blocks = !B_MN && (groups_per_row & 3) == 0;
      struct SzBlock {
        uint2 s4;
        uint32_t z4;
      };
      SzBlock sz_cur = {make_uint2(0u, 0u), 0u}, sz_nxt = {make_uint2(0u, 0u), 0u};
      int sz_blk = -1;
      // Each group takes alternate runs of R consecutive K blocks (counted over all tiles of this CTA).  R = 2
      // for 2-bit codes with a K-major operand: the 2 x 16 bytes of a run are one 32-byte sector of the packed
      // row, fetched by one thread with one load, instead of by two warps at unrelated times.
      // Register ring of two runs: the loads for the thread's next-but-one run (4R K blocks ahead) are issued
      // as soon as the current run has been expanded.
      constexpr int R = (!B_MN && BITS == 2) ? 2 : 1;
      static_assert(C::kStagesB == 4, "stage and phase of a K block are taken from its index mod 4");
      uint32_t ring_w[2][R][2 * BITS];
      float ring_s[2][R], ring_z[2][R];
      const size_t code_step = 2 * R * (B_MN ? (size_t)BK * pitch : (size_t)(8 * BITS));   // bytes per two runs
      const size_t sz_step = B_MN ? (size_t)2 * BK * groups_per_row : 0;                   // groups per two runs
      long gk = 0;                                                // global index of the tile's K block 0
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int m_blk, n_blk;
        tile_coords<PACKED>(tile, num_m, num_n, m_blk, n_blk);
        // this group's first K block of the tile (R = 2: K is a multiple of 128, so gk is even)
        const int kb_first = R * (int)((grp - gk / R) & 1);
        const int wrow0 = B_MN ? kb_first * BK + kr : n_blk * BN + t;
        const int unit0 = B_MN ? n_blk * (BN / 64) + box : kb_first;
        const bool valid = B_MN ? (unit0 < chunks_in) : (wrow0 < p.out_features);
        const uint8_t* code_ptr = p.Wq + (valid ? (size_t)wrow0 * pitch + (size_t)unit0 * (8 * BITS) : 0);
        const size_t g0 = valid ? (size_t)wrow0 * groups_per_row + (B_MN ? ((unit0 << 6) >> p.group_shift) : 0) : 0;
        const eqat_fp16* s_ptr = p.s16 + g0;                      // K-major: group 0 of the row
        const uint8_t* z_ptr = p.z8 + g0;
        auto fetch = [&](int j, int kb) {                         // kb: first K block of the run being fetched
          if (valid) {
            if constexpr (R == 2) {
              // the run's 32 bytes are one sector of the packed row when the matrix itself starts on a 32-byte
              // boundary (row pitch and unit offsets are multiples of 32); otherwise two 16-byte loads
              if (p.wq_sectors) {
                ptx::ldg_256(code_ptr, reinterpret_cast<uint32_t(&)[8]>(ring_w[j][0][0]));
              } else {
                load_codes64<BITS>(code_ptr, ring_w[j][0]);
                load_codes64<BITS>(code_ptr + 8 * BITS, ring_w[j][1]);
              }
            } else {
              load_codes64<BITS>(code_ptr, ring_w[j][0]);
            }
            code_ptr += code_step;
            if (!sz_blocks) {
#pragma unroll
              for (int u = 0; u < R; ++u) {
                const size_t gi = B_MN ? 0 : (size_t)(((kb + u) << 6) >> p.group_shift);
                ring_s[j][u] = __half2float(__ushort_as_half(__ldg(s_ptr + gi)));
                ring_z[j][u] = (float)__ldg(z_ptr + gi);
              }
              if (B_MN) { s_ptr += sz_step; z_ptr += sz_step; }
            }
          }
        };
        auto fetch_sz = [&](SzBlock& b, int blk) {
          if (valid && blk * 4 < groups_per_row) {
            b.s4 = __ldg(reinterpret_cast<const uint2*>(s_ptr + blk * 4));
            b.z4 = __ldg(reinterpret_cast<const uint32_t*>(z_ptr + blk * 4));
          }
        };
#pragma unroll
        for (int j = 0; j < 2; ++j)
          if (kb_first + 2 * R * j < num_kb) fetch(j, kb_first + 2 * R * j);
        if (sz_blocks) {
          const int blk0 = ((kb_first << 6) >> p.group_shift) >> 2;
          fetch_sz(sz_cur, blk0);
          fetch_sz(sz_nxt, blk0 + 1);
          sz_blk = blk0;
        }
        for (int kb0 = kb_first; kb0 < num_kb && ok; kb0 += 4 * R) {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            if constexpr (R == 2) {
              // Both K blocks of a run as one straight-line piece of code (their two stages belong to this group and
              // share a phase): twice the independent work for the scheduler to interleave, one fence and one warp
              // synchronisation for the two stages.
              const int kb = kb0 + 4 * j;                           // even; kb + 1 < num_kb since num_kb is even
              if (ok && kb < num_kb) {
                if (sz_blocks) {
                  const int blk = ((kb << 6) >> p.group_shift) >> 2;
                  if (blk != sz_blk) {
                    sz_cur = sz_nxt;
                    sz_blk = blk;
                    fetch_sz(sz_nxt, blk + 1);
                  }
                }
                const int stage = (int)((gk + kb) & 3);             // 0 or 2; the run's second block is stage + 1
                const uint32_t phase = (uint32_t)(((gk + kb) >> 2) & 1);
                if (!wait_bounded(ptx::smem_addr(&ctl->empty_b[stage]), phase ^ 1u, abort_flag,
                                  WAIT_DEQ_OPERAND_EMPTY) ||
                    !wait_bounded(ptx::smem_addr(&ctl->empty_b[stage + 1]), phase ^ 1u, abort_flag,
                                  WAIT_DEQ_OPERAND_EMPTY)) {
                  ok = false;
                } else {
                  const uint32_t row_sx = smem_base + C::b_offset(stage) + smem_row_sx;
                  if (valid) {
                    float sv[2], zv[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                      sv[u] = ring_s[j][u];
                      zv[u] = ring_z[j][u];
                      if (sz_blocks) {
                        const int sub = (((kb + u) << 6) >> p.group_shift) & 3;
                        const uint32_t sw = (sub & 2) ? sz_cur.s4.y : sz_cur.s4.x;
                        sv[u] = __half2float(__ushort_as_half((unsigned short)((sub & 1) ? (sw >> 16) : (sw & 0xFFFFu))));
                        zv[u] = (float)((sz_cur.z4 >> (8 * sub)) & 0xFFu);
                      }
                    }
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                      const uint32_t rs = row_sx + (uint32_t)u * C::kBBytes;
                      dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][0]), sv[u], zv[u], rs, 0);
                      dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][BITS]), sv[u], zv[u], rs, 1);
                    }
                  } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                      ptx::sts_128(row_sx ^ ((uint32_t)c << 4), 0u, 0u, 0u, 0u);
                      ptx::sts_128((row_sx + C::kBBytes) ^ ((uint32_t)c << 4), 0u, 0u, 0u, 0u);
                    }
                  }
                  if (kb + 8 < num_kb) fetch(j, kb + 8);
                  ptx::fence_proxy_async_smem();
                  __syncwarp();
                  if (lane == 0) {
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->full_b[stage]));
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->full_b[stage + 1]));
                  }
                }
              }
            } else {
#pragma unroll
            for (int u = 0; u < R; ++u) {
              const int kb = kb0 + 2 * R * j + u;
              if (ok && kb < num_kb) {
                if (sz_blocks) {
                  const int blk = ((kb << 6) >> p.group_shift) >> 2;
                  if (blk != sz_blk) {
                    sz_cur = sz_nxt;
                    sz_blk = blk;
                    fetch_sz(sz_nxt, blk + 1);
                  }
                }
                const int stage = (int)((gk + kb) & 3);
                const uint32_t phase = (uint32_t)(((gk + kb) >> 2) & 1);
                if (!wait_bounded(ptx::smem_addr(&ctl->empty_b[stage]), phase ^ 1u, abort_flag,
                                  WAIT_DEQ_OPERAND_EMPTY)) {
                  ok = false;
                } else {
                  const uint32_t row_sx = smem_base + C::b_offset(stage) + smem_row_sx;
                  if (valid) {
                    float sv = ring_s[j][u], zv = ring_z[j][u];
                    if (sz_blocks) {
                      const int sub = ((kb << 6) >> p.group_shift) & 3;
                      const uint32_t sw = (sub & 2) ? sz_cur.s4.y : sz_cur.s4.x;
                      sv = __half2float(__ushort_as_half((unsigned short)((sub & 1) ? (sw >> 16) : (sw & 0xFFFFu))));
                      zv = (float)((sz_cur.z4 >> (8 * sub)) & 0xFFu);
                    }
                    dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][0]), sv, zv, row_sx, 0);
                    dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][BITS]), sv, zv, row_sx, 1);
                  } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c) ptx::sts_128(row_sx ^ ((uint32_t)c << 4), 0u, 0u, 0u, 0u);
                  }
                  if (u == R - 1 && kb - (R - 1) + 4 * R < num_kb) fetch(j, kb - (R - 1) + 4 * R);
                  ptx::fence_proxy_async_smem();
                  __syncwarp();
                  if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->full_b[stage]));
                }
              }
            }
            }
          }
        }
        gk += num_kb;
        ok = __all_sync(0xFFFFFFFFu, ok);                          // a warp gives up as a whole
        if (warp < 2 + kEpiWarps && ok) {
          ok = epilogue_tile(m_blk, n_blk, acc, acc_phase);
          if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  }

  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::kTmemCols);
  }
}

// One warp waits, with a short limit, on an mbarrier that nothing ever arrives at: the give-up path of
// wait_bounded (abort flag, status word, normal return) without any copy or tensor-memory state around it.
__global__ void wait_expiry_kernel(uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_addr(&bar), 1);
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  (void)wait_bounded(ptx::smem_addr(&bar), 0u, &abort_word, WAIT_SELFTEST, 0, limit_ns);
}

// ------------------------------------------------------------------ host side
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

// bf16 matrix [outer, inner] row-major; box = 64 elements (128 bytes) x box_outer rows, 128-byte swizzle.
bool make_tmap(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer) {
  EncodeFn enc = encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {64, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN, int MT, bool A_MN, bool B_MN, bool PACKED, int EPI, int BITS>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const GemmParams& p, cudaStream_t st) {
  using C = Cfg<BN, MT, PACKED>;
  auto kern = gemm_kernel<BN, MT, A_MN, B_MN, PACKED, EPI, BITS>;
  static SmemOptIn opt_in;
  if (!opt_in.ensure(kern, C::kSmemBytes)) return EQAT_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return EQAT_ERR_CUDA;
  const int tiles = ((p.M + C::kTileM - 1) / C::kTileM) * ((p.N + BN - 1) / BN);
  const int grid = tiles < sms ? tiles : sms;
  kern<<<grid, C::kThreads, C::kSmemBytes, st>>>(ta, tb, p);
  return launch_status();
}

// Rows per CTA tile for the dense kernels: 256 (two MMAs per stage, one
// accumulator set, epilogue not overlapped) runs about 6 % faster per flop than
// 128 (measured on 4096^2 x 16384), but its tiles are twice as coarse, so it is
// taken only when the last wave of tiles is still well filled.
int dense_row_tiles(int M, int N) {
  const int sms = sm_count();
  if (sms <= 0) return 1;
  auto fill = [&](int tile_m) {
    const long tiles = (long)((M + tile_m - 1) / tile_m) * ((N + 255) / 256);
    const long waves = (tiles + sms - 1) / sms;
    return (double)tiles / (double)(waves * sms);
  };
  return fill(256) * 1.06 > fill(128) ? 2 : 1;
}

int log2_exact(int v) {
  int s = 0;
  while ((1 << s) < v) ++s;
  return s;
}

GemmParams base_params(int M, int N, int K) {
  GemmParams p{};
  p.M = M; p.N = N; p.K = K;
  return p;
}

void set_output(GemmParams& p, eqat_bf16* D) { p.D = D; }

void set_weight(GemmParams& p, const eqat_desc& d, const uint8_t* Wq, const eqat_fp16* s16, const uint8_t* z8) {
  p.Wq = Wq; p.s16 = s16; p.z8 = z8;
  p.out_features = d.out_features;
  p.in_features = d.in_features;
  p.group_shift = log2_exact(d.group);
  p.wq_sectors = (reinterpret_cast<uintptr_t>(Wq) & 31u) == 0 ? 1 : 0;
}

}  // namespace

int launch_dense_fwd(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* What, eqat_bf16* Y, cudaStream_t st) {
  CUtensorMap ta, tb;
  GemmParams p = base_params((int)d.tokens, d.out_features, d.in_features);
  set_output(p, Y);
  const int mt = dense_row_tiles(p.M, p.N);
  if (!make_tmap(&ta, X, d.in_features, d.tokens, mt * BM) || !make_tmap(&tb, What, d.in_features, d.out_features, 256))
    return EQAT_ERR_CUDA;
  return mt == 2 ? launch<256, 2, false, false, false, EPI_STORE, 2>(ta, tb, p, st)
                 : launch<256, 1, false, false, false, EPI_STORE, 2>(ta, tb, p, st);
}

int launch_dense_dx(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* What, eqat_bf16* dX, cudaStream_t st) {
  CUtensorMap ta, tb;
  GemmParams p = base_params((int)d.tokens, d.in_features, d.out_features);
  set_output(p, dX);
  const int mt = dense_row_tiles(p.M, p.N);
  if (!make_tmap(&ta, dY, d.out_features, d.tokens, mt * BM) || !make_tmap(&tb, What, d.in_features, d.out_features, BK))
    return EQAT_ERR_CUDA;
  return mt == 2 ? launch<256, 2, false, true, false, EPI_STORE, 2>(ta, tb, p, st)
                 : launch<256, 1, false, true, false, EPI_STORE, 2>(ta, tb, p, st);
}

int launch_dense_dw(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, eqat_bf16* dWhat, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap(&ta, dY, d.out_features, d.tokens, BK) || !make_tmap(&tb, X, d.in_features, d.tokens, BK))
    return EQAT_ERR_CUDA;
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  set_output(p, dWhat);
  return dense_row_tiles(p.M, p.N) == 2 ? launch<256, 2, true, true, false, EPI_STORE, 2>(ta, tb, p, st)
                                        : launch<256, 1, true, true, false, EPI_STORE, 2>(ta, tb, p, st);
}

int launch_dense_dw_ste(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, const eqat_bf16* W, const float* s,
                        const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap(&ta, dY, d.out_features, d.tokens, BK) || !make_tmap(&tb, X, d.in_features, d.tokens, BK))
    return EQAT_ERR_CUDA;
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  set_output(p, dW);
  p.W = W; p.s32 = s; p.z32 = z;
  p.ds = ds; p.dz = dz;
  p.group_shift = log2_exact(d.group);
  p.Q = (float)((1 << d.bits) - 1);
  p.dz_literal = d.dz_mode;
  // 128-row tiles: with two accumulator sets this epilogue, the longest of the three, runs under the next tile
  return launch<256, 1, true, true, false, EPI_STE, 2>(ta, tb, p, st);
}

int launch_packed_fwd(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                      const uint8_t* z8, eqat_bf16* Y, cudaStream_t st) {
  CUtensorMap ta;
  if (!make_tmap(&ta, X, d.in_features, d.tokens, 2 * BM)) return EQAT_ERR_CUDA;
  GemmParams p = base_params((int)d.tokens, d.out_features, d.in_features);
  set_output(p, Y);
  set_weight(p, d, Wq, s16, z8);
  switch (d.bits) {
    case 2: return launch<256, 2, false, false, true, EPI_STORE, 2>(ta, ta, p, st);
    case 3: return launch<256, 2, false, false, true, EPI_STORE, 3>(ta, ta, p, st);
    default: return launch<256, 2, false, false, true, EPI_STORE, 4>(ta, ta, p, st);
  }
}

int launch_packed_dx(const eqat_desc& d, const eqat_bf16* dY, const uint8_t* Wq, const eqat_fp16* s16,
                     const uint8_t* z8, eqat_bf16* dX, cudaStream_t st) {
  CUtensorMap ta;
  if (!make_tmap(&ta, dY, d.out_features, d.tokens, 2 * BM)) return EQAT_ERR_CUDA;
  GemmParams p = base_params((int)d.tokens, d.in_features, d.out_features);
  set_output(p, dX);
  set_weight(p, d, Wq, s16, z8);
  switch (d.bits) {
    case 2: return launch<256, 2, false, true, true, EPI_STORE, 2>(ta, ta, p, st);
    case 3: return launch<256, 2, false, true, true, EPI_STORE, 3>(ta, ta, p, st);
    default: return launch<256, 2, false, true, true, EPI_STORE, 4>(ta, ta, p, st);
  }
}

int launch_packed_ds(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* dY, const uint8_t* Wq,
                     const uint8_t* z8, const eqat_fp16* s16, float* ds, float* dz, cudaStream_t st) {
  CUtensorMap ta, tb;
  if (!make_tmap(&ta, dY, d.out_features, d.tokens, BK) || !make_tmap(&tb, X, d.in_features, d.tokens, BK))
    return EQAT_ERR_CUDA;
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  set_weight(p, d, Wq, s16, z8);
  p.ds = ds;
  p.dz = dz;
  const int mt = dense_row_tiles(p.M, p.N);
  switch (d.bits) {
    case 2: return mt == 2 ? launch<256, 2, true, true, false, EPI_DS, 2>(ta, tb, p, st)
                             : launch<256, 1, true, true, false, EPI_DS, 2>(ta, tb, p, st);
    case 3: return mt == 2 ? launch<256, 2, true, true, false, EPI_DS, 3>(ta, tb, p, st)
                             : launch<256, 1, true, true, false, EPI_DS, 3>(ta, tb, p, st);
    default: return mt == 2 ? launch<256, 2, true, true, false, EPI_DS, 4>(ta, tb, p, st)
                            : launch<256, 1, true, true, false, EPI_DS, 4>(ta, tb, p, st);
  }
}

int launch_wait_expiry_gemm(cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(1000000ull);   // 1 ms
  return launch_status();
}

int read_device_status(int* status, int* detail) {
  int h[2] = {0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess) return EQAT_ERR_CUDA;
  if (cudaMemcpyFromSymbol(h, g_device_status, sizeof(h)) != cudaSuccess) return EQAT_ERR_CUDA;
  const int zero[2] = {0, 0};
  if (cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero)) != cudaSuccess) return EQAT_ERR_CUDA;
  *status = h[0];
  if (detail != nullptr) *detail = h[1];
  return EQAT_OK;
}

}  // namespace eqat
