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
// A tile of the output is 256 columns wide and is computed either by one CTA or
// by a PAIR of CTAs (a cluster of two on neighbouring SMs) that share one MMA
// (tcgen05 cta_group::2): each CTA of a pair holds its own rows of A and of the
// accumulator, and only HALF of the B operand; the tensor cores of the two SMs
// exchange the halves.  Per flop a paired CTA therefore stages (loads, or expands
// from packed codes) half the B bytes and reads half the B bytes from shared
// memory, which is what bounds the one-CTA form.  Every CTA fetches its own
// operands with its own loads.
//
// Roles inside a CTA (one CTA per SM; MT*128 output rows per CTA, 64-deep K blocks;
// MT = 1 keeps two TMEM accumulator sets so the epilogue overlaps the next tile,
// MT = 2 feeds two MMAs from each B stage):
//   warp 0      TMA producer: fills a ring of 128B-swizzled shared-memory stages;
//               in a pair the bytes are counted on the first CTA's barrier
//   warp 1      MMA issuer (first CTA of a pair only): one thread issues tcgen05.mma,
//               frees stages in both CTAs with tcgen05.commit; owns the TMEM allocation
//   warps 2-5   epilogue: tcgen05.ld the finished accumulator (one TMEM lane
//               quadrant each)
//   warps 2-17  (packed-weight kernels only) expand N-bit codes into the bf16 B
//               operand, (q - z) * s, rounded once to bf16.  That operand has a
//               ring of its own; the sixteen warps form groups of as many threads
//               as the CTA's B stage has rows (one 64-code row per thread and K
//               block) and the groups take alternate runs of one or two K blocks,
//               two ring stages per group.  Warps 2-5 then run the tile's epilogue.
// The epilogue either stores the tile as bf16; or, for the E2E-QP step-size
// gradient, multiplies each accumulator row by (q - z) of the matching packed
// codes and reduces runs of `group` columns, so the [out,in] weight gradient
// never leaves the chip; or, for the Block-AP weight gradient, applies Eqs. 3-5
// to the accumulators next to the latent weights and writes dW, ds and dz.
// Packed kernels walk their tiles row by row (the few MB of codes stay in L2,
// each activation panel is fetched once); dense kernels in bands of row-tiles.
//
// Every wait on an mbarrier is bounded in time; a role that gives up raises a
// CTA-wide abort flag, records the site in a device status word and all roles
// fall through to a teardown that drains copies in flight and frees TMEM.  The
// CTAs of a pair leave together (cluster barrier), so neither signals a barrier
// of a CTA that is gone.
#include <cuda.h>

#include "common.cuh"
#include "codec.cuh"
#include "gemm.cuh"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace eqat {

__device__ int g_device_status[2];   // [0] = eqat_status, [1] = WaitSite

namespace {

constexpr int BM = 128;          // rows per CTA and MMA = TMEM lanes
constexpr int BN = 256;          // columns per tile
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
  const void* zq;            // [out, in/group]: uint8, or fp16 when z_fp16
  int z_fp16;
  int out_features, in_features;
  int group_shift;           // log2(group) for groups of 32..256 (31 for one group per row: every index shifts to 0)
  int groups_per_row;
  int wq_sectors;            // Wq is 32-byte aligned: a thread may fetch a whole 32-byte sector with one load
  float* ds;                 // EPI_DS / EPI_STE outputs [out, in/group]
  float* dz;                 // may be null
  float* partial;            // EPI_DS, one group per row: per-tile partial sums [2][column tiles][out]
  // EPI_STE: latent weight and Block-AP quantiser parameters of the [out,in] tile rows
  const eqat_bf16* W;        // [out, in]
  const float* s32;          // [out, in/group]
  const float* z32;          // [out, in/group]
  float Q;                   // 2^N - 1
  int dz_literal;            // Eq. 4 clamped branch: -1 instead of -s
};

template <int MT, bool PACKED, bool PAIR>
struct Cfg {
  static constexpr int kCtas = PAIR ? 2 : 1;
  static constexpr int kTileM = MT * BM;                 // output rows per CTA
  static constexpr int kClusterM = kCtas * kTileM;       // output rows per tile
  static constexpr int kBRows = BN / kCtas;              // rows of the B operand staged by one CTA
  static constexpr int kAccSets = MT == 1 ? 2 : 1;       // TMEM holds kAccSets * MT accumulators of BN columns
  static constexpr int kABytes = kTileM * BK * 2;
  static constexpr int kBBytes = kBRows * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  // Dense kernels keep A and B of a stage side by side, as many stages as fit in 192 KB.  Packed kernels keep
  // the expanded B operand in a ring of its own, two stages per group of expansion warps: an expansion takes
  // longer than a copy, and the deeper B ring is what lets it run ahead of the tensor core.
  static constexpr int kStages = PACKED ? 3 : (196608 / kStageBytes);
  static constexpr int kDeqGroups = kDeqWarps * 32 / kBRows;          // 2 (one CTA) or 4 (pair)
  static constexpr int kStagesB = PACKED ? 2 * kDeqGroups : kStages;
  static constexpr int kRingBytes = PACKED ? kStages * kABytes + kStagesB * kBBytes : kStages * kStageBytes;
  __host__ __device__ static constexpr int a_offset(int stage) { return PACKED ? stage * kABytes : stage * kStageBytes; }
  __host__ __device__ static constexpr int b_offset(int stage_b) {
    return PACKED ? kStages * kABytes + stage_b * kBBytes : stage_b * kStageBytes + kABytes;
  }
  static constexpr int kThreads = (2 + (PACKED ? kDeqWarps : kEpiWarps)) * 32;
  static constexpr int kTmemCols = kAccSets * MT * BN;
  static constexpr int kSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 512 /*barriers*/;
  static_assert(!PACKED || MT == 2, "packed kernels use 256 rows per CTA");
  static_assert(kStages <= 8 && kStagesB <= 8, "barrier arrays hold eight stages");
  static_assert(kSmemBytes <= 232448, "stage rings exceed the shared memory of one CTA");
};

struct Control {
  uint64_t full[8];          // A (and, dense kernels, B) stage filled by TMA          (pair: first CTA's is used)
  uint64_t empty[8];         //                                                         (each CTA its own)
  uint64_t full_b[8];        // packed kernels: B stage expanded                        (pair: first CTA's)
  uint64_t empty_b[8];
  uint64_t raw_b[8];         // latent-weight kernels: B stage filled by TMA, not yet fake-quantised (each CTA its own)
  uint64_t acc_full[2];      //                                                         (each CTA its own)
  uint64_t acc_empty[2];     //                                                         (pair: first CTA's)
  uint64_t drain;
  uint32_t tmem_base;
  int abort;
};
static_assert(sizeof(Control) <= 512, "control block must fit its reservation");

// Bounded wait on an mbarrier phase.  `sleep_ns` > 0 backs off between polls so
// that a role with nothing to do for a long time (the epilogue during a main
// loop, the producer on a full ring) leaves the issue slots to the warps that
// are working; latency-critical waits pass 0.  CLUSTER: the barrier is also
// signalled from the other CTA of a pair.
template <bool CLUSTER = false>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort, int site,
                                             uint32_t sleep_ns = 0, uint64_t limit_ns = kWaitLimitNs) {
  auto ready = [&] { return CLUSTER ? ptx::mbar_try_wait_cluster(bar, parity) : ptx::mbar_try_wait(bar, parity); };
  if (ready()) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t n = 0;
  while (!ready()) {
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

template <bool ROW_ORDER, int BAND>
__device__ __forceinline__ void tile_coords(int tile, int num_m, int num_n, int& m_blk, int& n_blk) {
  if (ROW_ORDER) {
    // Packed kernels: the B operand (N-bit codes, a few MB) lives in L2 whatever the order, so tiles run along
    // a row of tiles first and each A panel is fetched by one wave of CTAs only.
    m_blk = tile / num_n;
    n_blk = tile - m_blk * num_n;
    return;
  }
  // Bands of BAND row-tiles (4096 rows), row-tile fastest inside a band: the tiles in flight share the band's A
  // panels and a few B panels in L2.
  const int band_tiles = BAND * num_n;
  const int band = tile / band_tiles;
  const int r = tile - band * band_tiles;
  const int m0 = band * BAND;
  const int h = min(BAND, num_m - m0);
  m_blk = m0 + r % h;
  n_blk = r / h;
}

// ------------------------------------------------------------------ expansion of packed codes
// 64 consecutive codes of one weight row become one 128-byte swizzled shared-memory row: element e of the row
// goes to 16-byte chunk (e/8) ^ rx.  `row_sx` is the shared-memory address of the row XOR (rx << 4): the row is
// 128-byte aligned, so chunk c lies at row_sx ^ (c << 4), one logic operation per store.
//
// 3- and 4-bit codes: a code q is dropped into bits 16..23 of the float 0x4B000000 (= 2^23), giving
// x = 2^23 + 65536*q exactly, and fma(x, s/65536, -(128 + z)*s) = (q - z)*s.  With an integer zero point both
// constants are exact in fp32 (s is an fp16 value, 11 significant bits) and so is the result: the only rounding
// is the final one to bf16.  With a real-valued (fp16) zero point the constant (128 + z)*s is rounded to fp32
// first, an error of at most 2^-17 s.  4-bit codes reach byte positions with one shift+mask per 4 codes and one
// byte permute each; 3-bit codes are shifted individually.
// 2-bit codes: the four possible values of a group are built once as bf16 ((q - z)*s in fp32, rounded once) and
// each code is looked up with a byte permute: lut01 = (v0, v1), lut23 = (v2, v3); value q occupies bytes 2q, 2q+1
// of the 8-byte pair, so the selector byte of a code is 0x10 + 0x22*q.
template <int BITS>
struct GroupValues {
  float sp, cz;
  __device__ __forceinline__ GroupValues() : sp(0.0f), cz(0.0f) {}
  __device__ __forceinline__ GroupValues(float s, float z) : sp(s * (1.0f / 65536.0f)), cz(-(128.0f + z) * s) {}
  __device__ __forceinline__ float operator()(uint32_t xbits) const { return fmaf(__uint_as_float(xbits), sp, cz); }
};
// 3-bit codes are not byte-aligned, and a shift per code costs as much as the multiply-add that follows it.  A
// code may instead sit at any mantissa position p as long as the constants follow it: with x = 2^23 + 2^p * q,
// fma(x, s / 2^p, -(2^(23-p) + z) * s) = (q - z) * s, exact while (2^(23-p) + z) * s is (p >= 11 for 11-bit s and
// z < 8).  Three consecutive codes of the stream land on p = 12, 15, 18 with ONE shift of the word (or of two
// words, for a code that straddles them), so a triple costs one shift instead of three.
template <>
struct GroupValues<3> {
  float sp[3], cz[3];
  __device__ __forceinline__ GroupValues() : sp{0.0f, 0.0f, 0.0f}, cz{0.0f, 0.0f, 0.0f} {}
  __device__ __forceinline__ GroupValues(float s, float z) {
    sp[0] = s * (1.0f / 4096.0f);   cz[0] = -(2048.0f + z) * s;
    sp[1] = s * (1.0f / 32768.0f);  cz[1] = -(256.0f + z) * s;
    sp[2] = s * (1.0f / 262144.0f); cz[2] = -(32.0f + z) * s;
  }
  // code of slot k (0..2) of a triple, still at bits [12 + 3k, 15 + 3k) of `win`
  __device__ __forceinline__ float at(int k, uint32_t win) const {
    return fmaf(__uint_as_float((win & (7u << (12 + 3 * k))) | 0x4B000000u), sp[k], cz[k]);
  }
};

template <>
struct GroupValues<2> {
  uint32_t lut01, lut23;
  __device__ __forceinline__ GroupValues() : lut01(0u), lut23(0u) {}
  __device__ __forceinline__ GroupValues(float s, float z) {
    const float zs = z * s;                              // exact: 11 x 11 significant bits
    lut01 = pack_bf16x2(-zs, s - zs);
    lut23 = pack_bf16x2(fmaf(2.0f, s, -zs), fmaf(3.0f, s, -zs));
  }
};

__device__ __forceinline__ void store_chunk(uint32_t row_sx, int chunk, const float (&v)[8]) {
  ptx::sts_128(row_sx ^ ((uint32_t)chunk << 4), pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]),
               pack_bf16x2(v[6], v[7]));
}

// Expands 32 consecutive codes (half h of a 64-code row) into chunks 4h .. 4h+3.
template <int BITS>
__device__ __forceinline__ void dequant_half32(const uint32_t (&w)[BITS], const GroupValues<BITS>& f, uint32_t row_sx, int h) {
  constexpr uint32_t kMagic = 0x4B000000u;
  if constexpr (BITS == 2) {
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
          o[pr] = __byte_perm(f.lut01, f.lut23, pair_sel);
        }
        ptx::sts_128(row_sx ^ ((uint32_t)(4 * h + 2 * i + c) << 4), o[0], o[1], o[2], o[3]);
      }
    }
  } else if constexpr (BITS == 4) {
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
    // 32 codes = 3 words = 96 bits, code j at bit 3j.  Triple m (codes 3m .. 3m+2) is brought to bits 12..20 of a
    // register by one shift of the stream: the 32-bit window that starts at bit 9m - 12.
    float v[32];
#pragma unroll
    for (int m = 0; m < 11; ++m) {
      const int start = 9 * m - 12;
      uint32_t win;
      if (start < 0) {
        win = w[0] << (-start);
      } else {
        const int word = start >> 5, sh = start & 31;
        const uint32_t hi = word + 1 < 3 ? w[word + 1 < 3 ? word + 1 : 2] : 0u;
        win = sh == 0 ? w[word] : __funnelshift_r(w[word], hi, sh);
      }
#pragma unroll
      for (int k = 0; k < 3; ++k)
        if (3 * m + k < 32) v[3 * m + k] = f.at(k, win);
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) store_chunk(row_sx, 4 * h + c, *reinterpret_cast<const float(*)[8]>(v + 8 * c));
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

// Step sizes and zero points of up to four consecutive groups of one weight row, as fetched: fp16 step sizes in
// s, zero points in z either as bytes (z.x) or as fp16 values.  `count` (1, 2 or 4) consecutive groups starting
// at group index gi, which is a multiple of count; in_features is a multiple of 128, so the vector loads below
// are aligned.
struct GroupParamsRaw {
  uint2 s, z;
};
__device__ __forceinline__ void load_group_params(const GemmParams& p, size_t gi, int count, GroupParamsRaw& r) {
  const eqat_fp16* sp = p.s16 + gi;
  if (count == 1) {
    r.s.x = __ldg(sp);
  } else if (count == 2) {
    r.s.x = __ldg(reinterpret_cast<const uint32_t*>(sp));
  } else {
    r.s = __ldg(reinterpret_cast<const uint2*>(sp));
  }
  if (p.z_fp16) {
    const eqat_fp16* zp = static_cast<const eqat_fp16*>(p.zq) + gi;
    if (count == 1) {
      r.z.x = __ldg(zp);
    } else if (count == 2) {
      r.z.x = __ldg(reinterpret_cast<const uint32_t*>(zp));
    } else {
      r.z = __ldg(reinterpret_cast<const uint2*>(zp));
    }
  } else {
    const uint8_t* zp = static_cast<const uint8_t*>(p.zq) + gi;
    if (count == 1) {
      r.z.x = __ldg(zp);
    } else if (count == 2) {
      r.z.x = __ldg(reinterpret_cast<const unsigned short*>(zp));
    } else {
      r.z.x = __ldg(reinterpret_cast<const uint32_t*>(zp));
    }
  }
}
__device__ __forceinline__ float half_at(const uint2& v, int i) {
  const uint32_t w = (i & 2) ? v.y : v.x;
  return __half2float(__ushort_as_half((unsigned short)((i & 1) ? (w >> 16) : (w & 0xFFFFu))));
}
__device__ __forceinline__ float step_size_at(const GroupParamsRaw& r, int i) { return half_at(r.s, i); }
__device__ __forceinline__ float zero_point_at(const GroupParamsRaw& r, int i, int z_fp16) {
  return z_fp16 ? half_at(r.z, i) : (float)((r.z.x >> (8 * i)) & 0xFFu);
}
// Zero point of one group, whichever way it is stored.
__device__ __forceinline__ float load_zero_point(const GemmParams& p, size_t gi) {
  return p.z_fp16 ? __half2float(__ushort_as_half(__ldg(static_cast<const eqat_fp16*>(p.zq) + gi)))
                  : (float)__ldg(static_cast<const uint8_t*>(p.zq) + gi);
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

// A_MN / B_MN: operand is MN-major.  PACKED: the B operand is produced by the CTA's warps: expanded from N-bit
// codes (BITS = 2, 3, 4), or (BITS = 16, Block-AP) fetched by TMA as the latent bf16 weight and fake-quantised in
// place, Eq. 1 then Eq. 2, before the tensor core reads it.  PAIR: the tile is computed by two CTAs sharing one
// MMA.  BITS is used by PACKED and by EPI_DS.
template <int MT, bool A_MN, bool B_MN, bool PACKED, int EPI, int BITS, bool PAIR>
__global__ void __launch_bounds__(Cfg<MT, PACKED, PAIR>::kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const GemmParams p) {
  using C = Cfg<MT, PACKED, PAIR>;
  constexpr bool LATENT = PACKED && BITS == 16;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_addr(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;                                  // 1024-byte aligned stages
  const uint32_t smem_base = raw_addr + pad;
  Control* ctl = reinterpret_cast<Control*>(smem + C::kRingBytes);
  volatile int* abort_flag = &ctl->abort;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = PAIR ? (int)ptx::cluster_ctarank() : 0;          // this CTA's place in its pair
  const int cluster_id = (int)blockIdx.x / C::kCtas;
  const int num_clusters = (int)gridDim.x / C::kCtas;
  const int num_m = (p.M + C::kClusterM - 1) / C::kClusterM;
  const int num_n = (p.N + BN - 1) / BN;
  const int num_tiles = num_m * num_n;
  const int num_kb = (p.K + BK - 1) / BK;
  constexpr int kBand = 4096 / C::kClusterM;

  // A barrier that both CTAs of a pair signal lives in the first CTA: `lead(bar)` is its address there.
  auto lead = [&](uint32_t bar) -> uint32_t { return PAIR ? ptx::map_to_cta(bar, 0) : bar; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), C::kCtas);
      ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), 1);
    }
    if (PACKED) {
      for (int s = 0; s < C::kStagesB; ++s) {
        ptx::mbar_init(ptx::smem_addr(&ctl->full_b[s]), C::kCtas * (C::kBRows / 32));
        ptx::mbar_init(ptx::smem_addr(&ctl->empty_b[s]), 1);
        ptx::mbar_init(ptx::smem_addr(&ctl->raw_b[s]), 1);
      }
    }
    for (int a = 0; a < C::kAccSets; ++a) {
      ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[a]), 1);
      ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[a]), C::kCtas * kEpiWarps);
    }
    ptx::mbar_init(ptx::smem_addr(&ctl->drain), 1);
    ctl->abort = 0;
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&tmap_a);
    if (!PACKED || LATENT) ptx::tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(ptx::smem_addr(&ctl->tmem_base), C::kTmemCols);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_base), C::kTmemCols);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) {                                                      // the other CTA's barriers exist from here on
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  ptx::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;

  // ---------------------------------------------------------------- epilogue of one tile
  // Run by four warps, one per TMEM lane quadrant (warp index mod 4).  `m0` is the first output row of this CTA's
  // part of the tile.
  const int quad = warp & 3;
  const int row_in_tile = quad * 32 + lane;
  auto epilogue_tile = [&](int m0, int n_blk, int acc, uint32_t acc_phase) -> bool {
    // The lanes of a warp must leave together: the store epilogue below shuffles across the whole warp.
    const bool got = wait_bounded<PAIR>(ptx::smem_addr(&ctl->acc_full[acc]), acc_phase, abort_flag, WAIT_EPI_ACC_FULL,
                                        PACKED ? 0 : (MT == 2 ? 512 : 128));
    if (!__all_sync(0xFFFFFFFFu, got)) return false;
    ptx::tc_fence_after();
#pragma unroll 1
    for (int h = 0; h < MT; ++h) {
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((acc * MT + h) * BN);
      const int m = m0 + h * BM + row_in_tile;
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
        // features.  ds[o,g] = sum_{j in g} G[o,j] * (q[o,j] - z[o,g]).  With one group per row the tile
        // holds 256 of the row's columns: its sums go to the partial arrays and a second kernel adds the
        // column tiles up in a fixed order.
        const bool whole_row = p.partial != nullptr;
        const int chunks_per_group = whole_row ? BN / 32 : 1 << (p.group_shift - 5);
        const uint8_t* qrow = p.Wq + (size_t)m * ((size_t)p.in_features * BITS / 8);
        float acc_s = 0.0f, acc_g = 0.0f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          ptx::tmem_ld_32x32(t_row + c * 32, r);
          ptx::tmem_ld_wait();
          const int col0 = n_blk * BN + c * 32;
          if (m < p.M) {
            if (col0 < p.N) {
              uint32_t words[BITS];
              const uint32_t* src = reinterpret_cast<const uint32_t*>(qrow) + (size_t)(col0 >> 5) * BITS;
#pragma unroll
              for (int i = 0; i < BITS; ++i) words[i] = __ldg(src + i);
              uint32_t codes[32];
              unpack32<BITS>(words, codes);
              const size_t gi = (size_t)m * p.groups_per_row + (col0 >> p.group_shift);
              const float zf = load_zero_point(p, gi);
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float gv = __uint_as_float(r[i]);
                acc_s = fmaf(gv, (float)codes[i] - zf, acc_s);
                acc_g += gv;
              }
            }
            if (((c + 1) & (chunks_per_group - 1)) == 0) {
              if (whole_row) {
                p.partial[(size_t)n_blk * p.M + m] = acc_s;
                p.partial[(size_t)(num_n + n_blk) * p.M + m] = acc_g;
              } else if (col0 < p.N) {
                const size_t gi = (size_t)m * p.groups_per_row + (col0 >> p.group_shift);
                p.ds[gi] = acc_s;
                if (p.dz != nullptr) p.dz[gi] = -__half2float(__ushort_as_half(__ldg(p.s16 + gi))) * acc_g;
              }
              acc_s = 0.0f;
              acc_g = 0.0f;
            }
          }
        }
      }
    }
    ptx::tc_fence_before();
    __syncwarp();
    if (lane == 0) {
      if (PAIR) ptx::mbar_arrive_cluster(lead(ptx::smem_addr(&ctl->acc_empty[acc])));
      else ptx::mbar_arrive(ptx::smem_addr(&ctl->acc_empty[acc]));
    }
    return true;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && LATENT) {
      // Two rings, one thread: the A operand goes to the first CTA's tensor core as it lands, the latent weight
      // goes to this CTA's own warps first (raw_b), which fake-quantise it in place.  The rings have different
      // depths and drain at different times, so the thread polls both and serves whichever has a free stage.
      struct Cursor {
        int tile, kb, m_blk, n_blk;
        long n;
      };
      auto start = [&](Cursor& c) {
        c.tile = cluster_id; c.kb = 0; c.n = 0;
        if (c.tile < num_tiles) tile_coords<PACKED, kBand>(c.tile, num_m, num_n, c.m_blk, c.n_blk);
      };
      auto advance = [&](Cursor& c) {
        ++c.n;
        if (++c.kb == num_kb) {
          c.kb = 0;
          c.tile += num_clusters;
          if (c.tile < num_tiles) tile_coords<PACKED, kBand>(c.tile, num_m, num_n, c.m_blk, c.n_blk);
        }
      };
      Cursor ca, cb;
      start(ca); start(cb);
      uint64_t t_last = ptx::globaltimer_ns();
      uint32_t idle = 0;
      while (ca.tile < num_tiles || cb.tile < num_tiles) {
        bool progress = false;
        if (ca.tile < num_tiles) {
          const int st_a = (int)(ca.n % C::kStages);
          const uint32_t par = (uint32_t)((ca.n / C::kStages) & 1) ^ 1u;
          const uint32_t bar = ptx::smem_addr(&ctl->empty[st_a]);
          if (PAIR ? ptx::mbar_try_wait_cluster(bar, par) : ptx::mbar_try_wait(bar, par)) {
            const uint32_t full = lead(ptx::smem_addr(&ctl->full[st_a]));
            const uint32_t a_dst = smem_base + C::a_offset(st_a);
            const int m0 = ca.m_blk * C::kClusterM + rank * C::kTileM;
            if (PAIR) {
              ptx::mbar_expect_tx_cluster(full, C::kABytes);
              ptx::tma_load_2d_pair(a_dst, &tmap_a, ca.kb * BK, m0, full);
            } else {
              ptx::mbar_expect_tx(full, C::kABytes);
              ptx::tma_load_2d(a_dst, &tmap_a, ca.kb * BK, m0, full);
            }
            advance(ca);
            progress = true;
          }
        }
        if (cb.tile < num_tiles) {
          const int st_b = (int)(cb.n % C::kStagesB);
          const uint32_t par = (uint32_t)((cb.n / C::kStagesB) & 1) ^ 1u;
          const uint32_t bar = ptx::smem_addr(&ctl->empty_b[st_b]);
          if (PAIR ? ptx::mbar_try_wait_cluster(bar, par) : ptx::mbar_try_wait(bar, par)) {
            const uint32_t raw = ptx::smem_addr(&ctl->raw_b[st_b]);
            const uint32_t b_dst = smem_base + C::b_offset(st_b);
            const int n0 = cb.n_blk * BN + rank * C::kBRows;
            ptx::mbar_expect_tx(raw, C::kBBytes);
            if (B_MN) {
#pragma unroll
              for (int b = 0; b < C::kBRows / 64; ++b)
                ptx::tma_load_2d(b_dst + b * (BK * 128), &tmap_b, n0 + b * 64, cb.kb * BK, raw);
            } else {
              ptx::tma_load_2d(b_dst, &tmap_b, cb.kb * BK, n0, raw);
            }
            advance(cb);
            progress = true;
          }
        }
        if (progress) {
          idle = 0;
          t_last = ptx::globaltimer_ns();
        } else {
          __nanosleep(64);
          if ((++idle & 31u) == 0u) {
            if (*abort_flag) break;
            if (ptx::globaltimer_ns() - t_last > kWaitLimitNs) {
              *abort_flag = 1;
              atomicExch(&g_device_status[1], (int)WAIT_PRODUCER_EMPTY);
              atomicExch(&g_device_status[0], (int)EQAT_ERR_TIMEOUT);
              break;
            }
          }
        }
      }
      if (*abort_flag) {                                           // outwait the copies in flight (microseconds)
        const uint64_t t0 = ptx::globaltimer_ns();
        while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
      }
    } else if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      long issued = 0;
      bool ok = true;
      constexpr uint32_t kBytes = PACKED ? C::kABytes : C::kStageBytes;   // this CTA's bytes per stage
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int m_blk, n_blk;
        tile_coords<PACKED, kBand>(tile, num_m, num_n, m_blk, n_blk);
        const int m0 = m_blk * C::kClusterM + rank * C::kTileM;    // this CTA's rows of A
        const int n0 = n_blk * BN + rank * C::kBRows;              // this CTA's rows of B
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bounded<PAIR>(ptx::smem_addr(&ctl->empty[stage]), phase ^ 1u, abort_flag, WAIT_PRODUCER_EMPTY, 64)) {
            ok = false;
            break;
          }
          const uint32_t full = lead(ptx::smem_addr(&ctl->full[stage]));
          const uint32_t a_dst = smem_base + C::a_offset(stage);
          const uint32_t b_dst = smem_base + C::b_offset(stage);
          auto load = [&](uint32_t dst, const CUtensorMap* tm, int c0, int c1) {
            if (PAIR) ptx::tma_load_2d_pair(dst, tm, c0, c1, full);
            else ptx::tma_load_2d(dst, tm, c0, c1, full);
          };
          if (PAIR) ptx::mbar_expect_tx_cluster(full, kBytes);
          else ptx::mbar_expect_tx(full, kBytes);
          if (A_MN) {
#pragma unroll
            for (int b = 0; b < C::kTileM / 64; ++b) load(a_dst + b * (BK * 128), &tmap_a, m0 + b * 64, kb * BK);
          } else {
            load(a_dst, &tmap_a, kb * BK, m0);
          }
          if (!PACKED) {
            if (B_MN) {
#pragma unroll
              for (int b = 0; b < C::kBRows / 64; ++b) load(b_dst + b * (BK * 128), &tmap_b, n0 + b * 64, kb * BK);
            } else {
              load(b_dst, &tmap_b, kb * BK, n0);
            }
          }
          ++issued;
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        // Drain: every copy this thread started must land before the CTA exits.  One CTA alone polls its own
        // barriers; in a pair the byte counts sit on the first CTA's barriers and mix both CTAs' copies, so the
        // thread simply outwaits its copies (they take microseconds).
        if (PAIR) {
          const uint64_t t0 = ptx::globaltimer_ns();
          while (ptx::globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
        } else {
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
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (first CTA of a pair)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                                 ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) |
                                 ((uint32_t)((C::kCtas * BM) >> 4) << 24);
      constexpr uint32_t a_lbo = A_MN ? BK * 128 : 16, b_lbo = B_MN ? BK * 128 : 16;
      constexpr uint32_t a_step = A_MN ? UMMA_K * 128 : UMMA_K * 2, b_step = B_MN ? UMMA_K * 128 : UMMA_K * 2;
      constexpr uint32_t a_half = BM * BK * 2;        // second 128-row half of the CTA's A stage (either major)
      auto commit_both = [&](uint32_t bar) {           // arrives in every CTA of the tile
        if (PAIR) ptx::mma_commit_pair_both(bar);
        else ptx::mma_commit(bar);
      };
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        if (!wait_bounded<PAIR>(ptx::smem_addr(&ctl->acc_empty[acc]), acc_phase ^ 1u, abort_flag, WAIT_MMA_ACC_EMPTY, 64)) break;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * MT * BN);
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bounded<PAIR>(ptx::smem_addr(&ctl->full[stage]), phase, abort_flag, WAIT_MMA_FULL, PACKED ? 32 : 0) ||
              (PACKED &&
               !wait_bounded<PAIR>(ptx::smem_addr(&ctl->full_b[stage_b]), phase_b, abort_flag, WAIT_MMA_FULL, 32))) {
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
            for (int h = 0; h < MT; ++h) {
              const uint64_t a_desc = smem_desc(a_addr + h * a_half + kk * a_step, a_lbo);
              if (PAIR) ptx::mma_bf16_ss_pair(d_tmem + h * BN, a_desc, b_desc, idesc, (kb | kk) != 0 ? 1u : 0u);
              else ptx::mma_bf16_ss(d_tmem + h * BN, a_desc, b_desc, idesc, (kb | kk) != 0 ? 1u : 0u);
            }
          }
          commit_both(ptx::smem_addr(&ctl->empty[stage]));
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
          if (PACKED) {
            commit_both(ptx::smem_addr(&ctl->empty_b[stage_b]));
            if (++stage_b == C::kStagesB) { stage_b = 0; phase_b ^= 1u; }
          }
        }
        if (!ok) break;
        commit_both(ptx::smem_addr(&ctl->acc_full[acc]));
        if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
      }
      // All MMAs of this thread must have retired before TMEM is freed (and, in a pair, before either CTA leaves:
      // the commits above signal barriers in both).
      if (PAIR) ptx::mma_commit_pair(ptx::smem_addr(&ctl->drain));
      else ptx::mma_commit(ptx::smem_addr(&ctl->drain));
      wait_bounded(ptx::smem_addr(&ctl->drain), 0u, abort_flag, WAIT_TEARDOWN, 64, kDrainLimitNs * 4);
    }
  } else if (!PACKED) {
    // ------------------------------------------------------------ epilogue warps (dense kernels)
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = cluster_id; tile < num_tiles; tile += num_clusters) {
      int m_blk, n_blk;
      tile_coords<PACKED, kBand>(tile, num_m, num_n, m_blk, n_blk);
      if (!epilogue_tile(m_blk * C::kClusterM + rank * C::kTileM, n_blk, acc, acc_phase)) break;
      if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
    }
  } else {
    // ------------------------------------------------------------ dequantisers (+ epilogue on warps 2-5)
    if constexpr (PACKED) {
      // The sixteen warps form NG groups of U threads, U = rows of this CTA's B stage: a thread owns one whole
      // 64-code unit (one 128-byte operand row) of each K block its group expands, so the per-K-block
      // bookkeeping (wait, fence, arrive, addresses, step size) is paid once per 64 codes.  The groups take
      // alternate RUNS of R consecutive K blocks, counted over all tiles of this CTA; NG stages are being
      // expanded at any time and each group owns 2R of the 2*NG*... ring stages.
      //   B K-major  (Y):  stage row t is weight row n0 + t, unit = kb
      //   B MN-major (dX): k-row kr is weight row kb*64 + kr, unit = n0/64 + box (64-column box)
      // The 8 lanes of a quarter-warp (one 16-byte store wavefront) own 8 consecutive
      // rows, whose swizzled chunks fall in 8 different bank groups.
      constexpr int U = C::kBRows, NG = C::kDeqGroups;
      constexpr int kBoxes = U / 64;                               // MN-major: 64-column boxes per CTA
      const int tid = (int)threadIdx.x - 64;
      const int t = tid & (U - 1);                                 // unit within the stage
      const int grp = tid / U;
      const size_t pitch = LATENT ? 0 : (size_t)p.in_features * BITS / 8;      // bytes per packed row
      const int chunks_in = p.in_features >> 6;                   // 64-code units per row
      bool ok = true;
      const int kr = (t & 7) | ((t / (8 * kBoxes)) << 3);         // MN-major: k-row 0..63
      const int box = (t >> 3) & (kBoxes - 1);                    // MN-major: 64-column box
      const int smem_row_off = B_MN ? (box * (BK * 128) + kr * 128) : t * 128;
      const int rx = B_MN ? (kr & 7) : (t & 7);
      const uint32_t smem_row_sx = (uint32_t)smem_row_off ^ ((uint32_t)rx << 4);   // stage bases are 1024-byte aligned
      // R = 2 for 2-bit codes with a K-major operand: the 2 x 16 bytes of a run are one 32-byte sector of the
      // packed row, fetched by one thread with one load, instead of by two warps at unrelated times.
      // Register ring of two runs: the loads for the thread's next-but-one run (2*NG*R K blocks ahead) are
      // issued as soon as the current run has been expanded.  A run's step sizes and zero points (one to four
      // consecutive groups of the row) travel with its codes.
      // Latent weights (BITS = 16): the unit's 128 bytes are already in the stage (TMA); only the group's
      // fp32 step size and zero point travel through the ring.
      constexpr int R = (!B_MN && BITS == 2) ? 2 : 1;
      constexpr int kStep = NG * R;                                // K blocks between a group's runs
      static_assert(C::kStagesB == 2 * NG && (C::kStagesB & (C::kStagesB - 1)) == 0, "stage = K block index mod 2*NG");
      constexpr int kCodeWords = LATENT ? 1 : 2 * BITS;
      uint32_t ring_w[2][R][kCodeWords];
      GroupParamsRaw ring_g[2];
      float ring_ls[2][2], ring_lz[2][2];                          // latent weights: s, z of the unit's one or two groups
      // groups per run / per unit, and where a 32-code half finds its group among those fetched
      const int span = B_MN ? 64 : 64 * R;                        // codes of one row a fetch covers
      const int g_count = max(1, span >> p.group_shift);          // 1, 2 or 4
      const bool split_units = p.group_shift == 5;                // groups of 32: the halves of a unit differ
      const size_t code_step = (size_t)kStep * (B_MN ? (size_t)BK * pitch : (size_t)(8 * BITS));   // bytes between runs
      const uint32_t full_b_lead = lead(ptx::smem_addr(&ctl->full_b[0]));
      long gk = 0;                                                // global index of the tile's K block 0
      int acc = 0;
      uint32_t acc_phase = 0;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int m_blk, n_blk;
        tile_coords<PACKED, kBand>(tile, num_m, num_n, m_blk, n_blk);
        // this group's first K block of the tile (R = 2: K is a multiple of 128, so gk is even)
        const int kb_first = R * (int)(((long)grp - gk / R) & (NG - 1));
        const int wrow0 = B_MN ? kb_first * BK + kr : n_blk * BN + rank * U + t;
        const int unit0 = B_MN ? n_blk * (BN / 64) + rank * kBoxes + box : kb_first;
        const bool valid = B_MN ? (unit0 < chunks_in) : (wrow0 < p.out_features);
        const uint8_t* code_ptr = LATENT ? nullptr : p.Wq + (valid ? (size_t)wrow0 * pitch + (size_t)unit0 * (8 * BITS) : 0);
        // first group of the row that a run starting at K block kb needs
        const size_t g_row0 = B_MN ? (size_t)kr * p.groups_per_row + (size_t)((unit0 << 6) >> p.group_shift)
                                   : (size_t)(valid ? wrow0 : 0) * p.groups_per_row;
        auto fetch = [&](int j, int kb) {                         // the run starting at K block kb, into ring slot j
          if constexpr (LATENT) {
            if (valid) {
              const size_t gi = B_MN ? g_row0 + (size_t)kb * BK * p.groups_per_row : g_row0 + (size_t)((kb << 6) >> p.group_shift);
              ring_ls[j][0] = __ldg(p.s32 + gi);
              ring_lz[j][0] = __ldg(p.z32 + gi);
              if (split_units) {
                ring_ls[j][1] = __ldg(p.s32 + gi + 1);
                ring_lz[j][1] = __ldg(p.z32 + gi + 1);
              }
            }
          } else if (valid) {
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
            const size_t gi = B_MN ? g_row0 + (size_t)kb * BK * p.groups_per_row : g_row0 + (size_t)((kb << 6) >> p.group_shift);
            load_group_params(p, gi, g_count, ring_g[j]);
          }
        };
#pragma unroll
        for (int j = 0; j < 2; ++j)
          if (kb_first + kStep * j < num_kb) fetch(j, kb_first + kStep * j);
        for (int kb0 = kb_first; kb0 < num_kb && ok; kb0 += 2 * kStep) {
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int kb = kb0 + kStep * j;                         // first K block of the run (R = 2: kb + 1 < num_kb too)
            if (ok && kb < num_kb) {
              const int stage = (int)((gk + kb) & (C::kStagesB - 1));   // R = 2: even; the run's second block is stage + 1
              const uint32_t phase = (uint32_t)(((gk + kb) / C::kStagesB) & 1);
              // packed codes: the stage must have been released by the tensor core; latent weights: the raw tile
              // must have landed in it
              bool free_stage = LATENT ? wait_bounded(ptx::smem_addr(&ctl->raw_b[stage]), phase, abort_flag, WAIT_DEQ_OPERAND_EMPTY)
                                       : wait_bounded<PAIR>(ptx::smem_addr(&ctl->empty_b[stage]), phase ^ 1u, abort_flag,
                                                            WAIT_DEQ_OPERAND_EMPTY);
              if (R == 2 && free_stage)
                free_stage = wait_bounded<PAIR>(ptx::smem_addr(&ctl->empty_b[stage + 1]), phase ^ 1u, abort_flag,
                                                WAIT_DEQ_OPERAND_EMPTY);
              if (!free_stage) {
                ok = false;
              } else {
                // Both K blocks of a run are one straight-line piece of code (their two stages belong to this group
                // and share a phase): twice the independent work for the scheduler to interleave, one fence and one
                // warp synchronisation for the two stages.
                const uint32_t row_sx = smem_base + C::b_offset(stage) + smem_row_sx;
                if constexpr (LATENT) {
                  // Eq. 1 then Eq. 2 on the unit's 64 latent weights, in place: the same arithmetic, shortcut and
                  // fallback as the stand-alone fake quantiser, so the operand is bit for bit the W_hat it would store.
                  // (Rows or columns past the matrix were zero-filled by the copy and stay zero.)
                  if (valid) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                      const int gsel = split_units ? h : 0;
                      const float sv = ring_ls[j][gsel];
                      const float zr = rintf(ring_lz[j][gsel]);
                      const float rs = group_rcp(sv, zr);
                      const float lo = -zr, hi = p.Q - zr;
#pragma unroll
                      for (int c = 4 * h; c < 4 * h + 4; ++c) {
                        const uint32_t addr = row_sx ^ ((uint32_t)c << 4);
                        float w[8], r[8], rt[8];
                        unpack8(ptx::lds_128(addr), w);
                        quotient_round8(w, sv, rs, r, rt);
#pragma unroll
                        for (int i = 0; i < 8; ++i) w[i] = fminf(fmaxf(r[i], lo), hi) * sv;
                        const uint4 o = pack8(w);
                        ptx::sts_128(addr, o.x, o.y, o.z, o.w);
                      }
                    }
                  }
                } else if (valid) {
                  GroupValues<BITS> gv[R][2];
#pragma unroll
                  for (int u = 0; u < R; ++u) {
                    const int i0 = (u * 64) >> p.group_shift;       // which of the fetched groups (0 for one group per row)
                    gv[u][0] = GroupValues<BITS>(step_size_at(ring_g[j], i0), zero_point_at(ring_g[j], i0, p.z_fp16));
                    gv[u][1] = gv[u][0];
                    if (split_units)
                      gv[u][1] = GroupValues<BITS>(step_size_at(ring_g[j], i0 + 1), zero_point_at(ring_g[j], i0 + 1, p.z_fp16));
                  }
#pragma unroll
                  for (int u = 0; u < R; ++u) {
                    const uint32_t rs = row_sx + (uint32_t)u * C::kBBytes;
                    dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][0]), gv[u][0], rs, 0);
                    dequant_half32<BITS>(reinterpret_cast<const uint32_t(&)[BITS]>(ring_w[j][u][BITS]), gv[u][1], rs, 1);
                  }
                } else {
#pragma unroll
                  for (int u = 0; u < R; ++u)
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                      ptx::sts_128((row_sx + (uint32_t)u * C::kBBytes) ^ ((uint32_t)c << 4), 0u, 0u, 0u, 0u);
                }
                if (kb + 2 * kStep < num_kb) fetch(j, kb + 2 * kStep);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
#pragma unroll
                  for (int u = 0; u < R; ++u) {
                    if (PAIR) ptx::mbar_arrive_cluster(full_b_lead + (uint32_t)(stage + u) * 8u);
                    else ptx::mbar_arrive(ptx::smem_addr(&ctl->full_b[stage + u]));
                  }
                }
              }
            }
          }
        }
        gk += num_kb;
        ok = __all_sync(0xFFFFFFFFu, ok);                          // a warp gives up as a whole
        if (warp < 2 + kEpiWarps && ok) {
          ok = epilogue_tile(m_blk * C::kClusterM + rank * C::kTileM, n_blk, acc, acc_phase);
          if (++acc == C::kAccSets) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  }

  __syncwarp();
  ptx::tc_fence_before();
  __syncthreads();
  if (PAIR) {                                                      // neither CTA leaves while the other may still signal it
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, C::kTmemCols);
    else ptx::tmem_dealloc(tmem_base, C::kTmemCols);
  }
}

// E2E-QP with one group per row: adds up the column tiles' partial sums in a fixed order.
//   ds[o] = sum_n part[0][n][o],   dz[o] = -s[o] * sum_n part[1][n][o]
__global__ void finish_row_sums_kernel(const float* __restrict__ partial, int num_n, int out_features,
                                       const eqat_fp16* __restrict__ s16, float* __restrict__ ds, float* __restrict__ dz) {
  const int o = (int)(blockIdx.x * blockDim.x + threadIdx.x);
  if (o >= out_features) return;
  float a = 0.0f, b = 0.0f;
  for (int n = 0; n < num_n; ++n) {
    a += partial[(size_t)n * out_features + o];
    b += partial[(size_t)(num_n + n) * out_features + o];
  }
  ds[o] = a;
  if (dz != nullptr) dz[o] = -__half2float(__ushort_as_half(__ldg(s16 + o))) * b;
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

}  // namespace

// bf16 matrix [outer, inner] row-major; box = 64 elements (128 bytes) x box_outer rows, 128-byte swizzle.
bool make_tmap_bf16(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer) {
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

bool make_tmap_u8(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t outer, uint32_t box_bytes,
                  uint32_t box_outer) {
  EncodeFn enc = encode_fn();
  if (enc == nullptr) return false;
  const cuuint64_t dims[2] = {inner_bytes, outer};
  const cuuint64_t strides[1] = {inner_bytes};
  const cuuint32_t box[2] = {box_bytes, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

bool make_tmap(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer) {
  return make_tmap_bf16(tm, base, inner, outer, box_outer);
}

// How a contraction's tiles are shaped: rows per CTA (128 * mt) and whether pairs of CTAs share a tile.
struct TileShape {
  int mt;
  bool pair;
  int rows() const { return 128 * mt * (pair ? 2 : 1); }
};

// One operand of a contraction: a bf16 matrix and which way it is walked.
//   K-major : [rows, K] row-major, tiled in boxes of 64 K x `rows per CTA`
//   MN-major: [K, rows] row-major, tiled in boxes of 64 rows x 64 K
struct Operand {
  const void* base;
  uint64_t rows, k;
  bool mn_major;
};

bool operand_tmap(CUtensorMap* tm, const Operand& op, int rows_per_cta) {
  return op.mn_major ? make_tmap(tm, op.base, op.rows, op.k, BK) : make_tmap(tm, op.base, op.k, op.rows, rows_per_cta);
}

template <int MT, bool A_MN, bool B_MN, bool PACKED, int EPI, int BITS, bool PAIR>
int launch(const Operand& a, const Operand& b, const GemmParams& p, cudaStream_t st) {
  using C = Cfg<MT, PACKED, PAIR>;
  auto kern = gemm_kernel<MT, A_MN, B_MN, PACKED, EPI, BITS, PAIR>;
  static SmemOptIn opt_in;
  if (!opt_in.ensure(kern, C::kSmemBytes)) return EQAT_ERR_CUDA;
  CUtensorMap ta, tb;
  if (!operand_tmap(&ta, a, C::kTileM)) return EQAT_ERR_CUDA;
  if (PACKED && BITS != 16) tb = ta;                            // packed codes are fetched with ordinary loads
  else if (!operand_tmap(&tb, b, C::kBRows)) return EQAT_ERR_CUDA;
  const int sms = sm_count();
  if (sms < C::kCtas) return EQAT_ERR_CUDA;
  const int tiles = ((p.M + C::kClusterM - 1) / C::kClusterM) * ((p.N + BN - 1) / BN);
  const int clusters = tiles < sms / C::kCtas ? tiles : sms / C::kCtas;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(clusters * C::kCtas), 1, 1);
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C::kCtas;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = PAIR ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, kern, ta, tb, p) != cudaSuccess) {
    (void)cudaGetLastError();
    return EQAT_ERR_CUDA;
  }
  return launch_status();
}

// Tile shape for a contraction with M output rows.  Pairs of CTAs are what keeps the tensor cores fed (half the
// B traffic per flop), 256 rows per CTA run a few percent faster per flop than 128 but make tiles twice as
// coarse; so the largest shape is taken whose last wave of tiles is still about as full as a finer shape's.
// A problem of at most 128 rows gets single CTAs (a pair's second CTA would have nothing to do).
TileShape choose_shape(int M, int N, bool allow_mt2) {
  const int sms = sm_count();
  if (M <= 128 || sms < 2) return {1, false};
  auto fill = [&](const TileShape& s) {
    const long units = sms / (s.pair ? 2 : 1);
    const long tiles = (long)((M + s.rows() - 1) / s.rows()) * ((N + BN - 1) / BN);
    const long waves = (tiles + units - 1) / units;
    // useful rows / rows computed, times the fill of the last wave
    return ((double)M / ((double)((M + s.rows() - 1) / s.rows()) * s.rows())) * ((double)tiles / (double)(waves * units));
  };
  const TileShape small{1, true}, large{2, true};
  if (allow_mt2 && fill(large) * 1.04 > fill(small)) return large;
  return small;
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

void set_weight(GemmParams& p, const eqat_desc& d, const uint8_t* Wq, const eqat_fp16* s16, const void* zq) {
  p.Wq = Wq; p.s16 = s16; p.zq = zq;
  p.z_fp16 = d.zero_point_format == EQAT_ZP_FP16 ? 1 : 0;
  p.out_features = d.out_features;
  p.in_features = d.in_features;
  const bool whole_row = d.group == d.in_features && d.group > 256;
  p.group_shift = whole_row ? 31 : log2_exact(d.group);
  p.groups_per_row = d.in_features / d.group;
  p.wq_sectors = (reinterpret_cast<uintptr_t>(Wq) & 31u) == 0 ? 1 : 0;
}

// Block-AP quantiser parameters for the kernels that fake-quantise the latent weight themselves.
void set_latent(GemmParams& p, const eqat_desc& d, const eqat_bf16* W, const float* s, const float* z) {
  p.W = W; p.s32 = s; p.z32 = z;
  p.Q = (float)((1 << d.bits) - 1);
  p.out_features = d.out_features;
  p.in_features = d.in_features;
  const bool whole_row = d.group == d.in_features && d.group > 256;
  p.group_shift = whole_row ? 31 : log2_exact(d.group);
  p.groups_per_row = d.in_features / d.group;
}

// Dense contraction with the plain store epilogue, over the three operand layouts.
template <bool A_MN, bool B_MN>
int launch_dense(const Operand& a, const Operand& b, GemmParams& p, cudaStream_t st) {
  const TileShape s = choose_shape(p.M, p.N, true);
  if (!s.pair) return launch<1, A_MN, B_MN, false, EPI_STORE, 2, false>(a, b, p, st);
  return s.mt == 2 ? launch<2, A_MN, B_MN, false, EPI_STORE, 2, true>(a, b, p, st)
                   : launch<1, A_MN, B_MN, false, EPI_STORE, 2, true>(a, b, p, st);
}

template <bool B_MN, int BITS>
int launch_packed(const Operand& a, GemmParams& p, cudaStream_t st) {
  // 256 rows per CTA; pairs as soon as there are more rows than one CTA takes
  return p.M > 256 ? launch<2, false, B_MN, true, EPI_STORE, BITS, true>(a, a, p, st)
                   : launch<2, false, B_MN, true, EPI_STORE, BITS, false>(a, a, p, st);
}

template <int BITS>
int launch_ds(const Operand& a, const Operand& b, GemmParams& p, cudaStream_t st) {
  const TileShape s = choose_shape(p.M, p.N, true);
  if (!s.pair) return launch<1, true, true, false, EPI_DS, BITS, false>(a, b, p, st);
  return s.mt == 2 ? launch<2, true, true, false, EPI_DS, BITS, true>(a, b, p, st)
                   : launch<1, true, true, false, EPI_DS, BITS, true>(a, b, p, st);
}

}  // namespace

int launch_dense_fwd(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* What, eqat_bf16* Y, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.out_features, d.in_features);
  p.D = Y;
  return launch_dense<false, false>({X, (uint64_t)d.tokens, (uint64_t)d.in_features, false},
                                    {What, (uint64_t)d.out_features, (uint64_t)d.in_features, false}, p, st);
}

int launch_dense_dx(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* What, eqat_bf16* dX, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.in_features, d.out_features);
  p.D = dX;
  return launch_dense<false, true>({dY, (uint64_t)d.tokens, (uint64_t)d.out_features, false},
                                   {What, (uint64_t)d.in_features, (uint64_t)d.out_features, true}, p, st);
}

int launch_dense_dw(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, eqat_bf16* dWhat, cudaStream_t st) {
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  p.D = dWhat;
  return launch_dense<true, true>({dY, (uint64_t)d.out_features, (uint64_t)d.tokens, true},
                                  {X, (uint64_t)d.in_features, (uint64_t)d.tokens, true}, p, st);
}

int launch_dense_dw_ste(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* X, const eqat_bf16* W, const float* s,
                        const float* z, eqat_bf16* dW, float* ds, float* dz, cudaStream_t st) {
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  p.D = dW;
  p.W = W; p.s32 = s; p.z32 = z;
  p.ds = ds; p.dz = dz;
  p.group_shift = log2_exact(d.group);
  p.Q = (float)((1 << d.bits) - 1);
  p.dz_literal = d.dz_mode;
  const Operand a{dY, (uint64_t)d.out_features, (uint64_t)d.tokens, true}, b{X, (uint64_t)d.in_features, (uint64_t)d.tokens, true};
  // 128 rows per CTA: with two accumulator sets this epilogue, the longest of the three, runs under the next tile
  return p.M > 128 ? launch<1, true, true, false, EPI_STE, 2, true>(a, b, p, st)
                   : launch<1, true, true, false, EPI_STE, 2, false>(a, b, p, st);
}

int launch_latent_fwd(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* W, const float* s, const float* z,
                      eqat_bf16* Y, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.out_features, d.in_features);
  p.D = Y;
  set_latent(p, d, W, s, z);
  const Operand a{X, (uint64_t)d.tokens, (uint64_t)d.in_features, false}, b{W, (uint64_t)d.out_features, (uint64_t)d.in_features, false};
  return p.M > 256 ? launch<2, false, false, true, EPI_STORE, 16, true>(a, b, p, st)
                   : launch<2, false, false, true, EPI_STORE, 16, false>(a, b, p, st);
}

int launch_latent_dx(const eqat_desc& d, const eqat_bf16* dY, const eqat_bf16* W, const float* s, const float* z,
                     eqat_bf16* dX, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.in_features, d.out_features);
  p.D = dX;
  set_latent(p, d, W, s, z);
  const Operand a{dY, (uint64_t)d.tokens, (uint64_t)d.out_features, false}, b{W, (uint64_t)d.in_features, (uint64_t)d.out_features, true};
  return p.M > 256 ? launch<2, false, true, true, EPI_STORE, 16, true>(a, b, p, st)
                   : launch<2, false, true, true, EPI_STORE, 16, false>(a, b, p, st);
}

int launch_packed_fwd(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                      const void* zq, eqat_bf16* Y, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.out_features, d.in_features);
  p.D = Y;
  set_weight(p, d, Wq, s16, zq);
  const Operand a{X, (uint64_t)d.tokens, (uint64_t)d.in_features, false};
  switch (d.bits) {
    case 2: return launch_packed<false, 2>(a, p, st);
    case 3: return launch_packed<false, 3>(a, p, st);
    default: return launch_packed<false, 4>(a, p, st);
  }
}

int launch_packed_dx(const eqat_desc& d, const eqat_bf16* dY, const uint8_t* Wq, const eqat_fp16* s16,
                     const void* zq, eqat_bf16* dX, cudaStream_t st) {
  GemmParams p = base_params((int)d.tokens, d.in_features, d.out_features);
  p.D = dX;
  set_weight(p, d, Wq, s16, zq);
  const Operand a{dY, (uint64_t)d.tokens, (uint64_t)d.out_features, false};
  switch (d.bits) {
    case 2: return launch_packed<true, 2>(a, p, st);
    case 3: return launch_packed<true, 3>(a, p, st);
    default: return launch_packed<true, 4>(a, p, st);
  }
}

size_t packed_ds_workspace_bytes(const eqat_desc& d) {
  if (!(d.group == d.in_features && d.group > 256)) return 0;
  const size_t num_n = (size_t)(d.in_features + BN - 1) / BN;
  return 2 * num_n * (size_t)d.out_features * sizeof(float);
}

int launch_packed_ds(const eqat_desc& d, const eqat_bf16* X, const eqat_bf16* dY, const uint8_t* Wq,
                     const void* zq, const eqat_fp16* s16, float* ds, float* dz, void* workspace, cudaStream_t st) {
  GemmParams p = base_params(d.out_features, d.in_features, (int)d.tokens);
  set_weight(p, d, Wq, s16, zq);
  p.ds = ds;
  p.dz = dz;
  const bool whole_row = packed_ds_workspace_bytes(d) != 0;
  p.partial = whole_row ? static_cast<float*>(workspace) : nullptr;
  const Operand a{dY, (uint64_t)d.out_features, (uint64_t)d.tokens, true}, b{X, (uint64_t)d.in_features, (uint64_t)d.tokens, true};
  int rc;
  switch (d.bits) {
    case 2: rc = launch_ds<2>(a, b, p, st); break;
    case 3: rc = launch_ds<3>(a, b, p, st); break;
    default: rc = launch_ds<4>(a, b, p, st); break;
  }
  if (rc != EQAT_OK || !whole_row) return rc;
  const int num_n = (d.in_features + BN - 1) / BN;
  finish_row_sums_kernel<<<(d.out_features + 255) / 256, 256, 0, st>>>(p.partial, num_n, d.out_features, s16, ds, dz);
  return launch_status();
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
