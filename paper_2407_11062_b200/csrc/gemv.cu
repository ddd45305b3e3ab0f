// Packed-weight forward for a handful of tokens (decode-time inference):
//     Y[T,out] = X[T,in] * dequant(Wq)^T,
// the matrix-vector case of the E2E-QP forward (Eq. 2 on frozen codes).  The
// 512-row tensor-memory tiles of gemm.cu would be almost empty here; the work is
// one pass over the packed weight, so the kernel is a stream over its bytes that
// builds weight fragments for warp-level matrix instructions in registers.  It
// takes up to eight tokens per launch (more tokens, or rows too long for the
// staged activations, go out as several launches).  The dequantised weight is
// never rounded to bf16 here: the codes enter the matrix instructions as exact
// small numbers and the step size scales fp32 accumulators.
#include <cuda.h>

#include "common.cuh"
#include "gemm.cuh"
#include "gemv.cuh"
#include "ptx.cuh"

namespace eqat {
namespace {

// ====================================================================== codes on tensor-core tiles
// A loop on the ordinary cores spends three instructions per code and token.
// That is several times what the bytes allow, so the codes go through
// warp-level matrix instructions instead (mma.sync m16n8k16, bf16 in, fp32
// out): 16 weight rows by 16 columns against up to 8 tokens per instruction,
// with the weight fragment built in registers, one logic operation per PAIR of
// codes.  (The paired-CTA tensor-memory path of gemm.cu
// wants its operands expanded into shared memory, which is exactly the cost to
// avoid here; and with at most a few tokens there is nothing for a 128-row
// accumulator to amortise.)
//
// Fragment construction, 2-bit codes (3-bit and 4-bit codes: see expand_reg).
// A 32-bit word of the stream holds 16 consecutive codes of one row, code j at
// bits [2j, 2j + 2).  (w >> 2p) & 0x00030003 isolates codes p and p + 8 in the
// two halves of a register; OR-ing 0x4300 into each half makes them the bf16
// numbers 128 + q.  For p = 1, 2 (mod 3) the shift is skipped: a code left at
// bits 2-3 (4-5) of a half with 0x4200 (0x4100) above it is the bf16 number
// 32 + q (8 + q).  Eight registers from ten operations.  The added constants
// and the zero point are taken out again by a fifth instruction per chunk: with
// xb = sum of bias * x and xs = sum of x over the chunk's 64 columns,
//     sum (q - z) x = sum (bias + q) x - (xb - 128 xs) - (128 + z) xs,
// and the fifth instruction multiplies weights -1 and -(128 + z) (the bf16
// pattern 0xC300 | z) with xb - 128 xs and xs, each given as the sum of three
// bf16 numbers (24 significant bits: an fp32 value split without loss), so the
// correction is as exact as if it were done in fp32 and the accumulator of a
// chunk only remains to be scaled by the row's step size.
//
// Mapping.  A task is 16 consecutive weight rows over the whole of K; persistent
// CTAs take tasks round-robin.  The producer thread copies the task's codes into
// a shared-memory ring as [16 rows x 128 bytes] boxes (cp.async.bulk.tensor,
// 128-byte swizzle, bytes past the end of a row arrive as zeros), eight boxes
// per stage.  Consumer warp w owns half of box w/2 of every stage: four chunks
// of 16 bytes = 64 columns = the four words of the four lanes of a quad.  (4-bit
// codes: sixteen boxes per stage, a warp owns a box = four chunks of 32 bytes,
// two words per lane.  3-bit codes: sixteen unswizzled boxes of 96 bytes, a
// warp owns a box = four chunks of 24 bytes, six bytes per lane.)  A chunk lies
// in one quantisation group and its accumulator is scaled by one step size per
// row.  Lane (g, q) of the warp holds rows g and g + 8 and, in instruction m of
// a chunk, supplies four of its 16 codes (2m, 2m+8, 2m+1, 2m+9 for 2-bit codes;
// tc_column gives the order for every width); the activations are staged once
// per CTA in exactly that order, so a lane fetches its fragment of X for an
// instruction with one 8-byte load.  Zero points are one byte each, or fp16
// values (ZF16): then 128 + z is split into three bf16 numbers like the sums
// and the fifth instruction holds all nine products.  The 16 warps' partial sums of a
// task go through a double-buffered shared array to a reducer warp, which adds
// them in a fixed order and stores Y while the consumers are on the next task.
constexpr int kTcMaxTokens = 8;                         // the instruction has eight token columns
constexpr int kTcMaxTotalTokens = 64;                   // up to here, as several launches over slices of the tokens
constexpr int kTcWarps = 16;
constexpr int kTcThreads = (kTcWarps + 2) * 32;        // + producer warp + reducer warp
constexpr int kTcRows = 16;                            // weight rows per task
// Bytes of a row per box of the copy engine: 128 (512 columns of 2-bit codes, 256 of 4-bit codes) or, for 3-bit
// codes, whose 64-column chunks are 24 bytes, 96 (256 columns).
__host__ __device__ constexpr int tc_box_bytes(int bits) { return bits == 3 ? 96 : 128; }
__host__ __device__ constexpr int tc_words_per_lane(int bits) { return bits == 2 ? 1 : 2; }   // per row and chunk
// Boxes per stage: every consumer warp has four chunks of a stage, i.e. half a box of 2-bit codes (8 boxes,
// 16 KB per stage) or a whole box of 3-bit or 4-bit codes (16 boxes, 24 KB or 32 KB per stage).
__host__ __device__ constexpr int tc_boxes_per_stage(int bits) { return bits == 2 ? 8 : 16; }
__host__ __device__ constexpr int tc_box_smem(int bits) { return kTcRows * tc_box_bytes(bits); }   // 2 KB or 1.5 KB
__host__ __device__ constexpr int tc_stage_bytes(int bits) { return tc_boxes_per_stage(bits) * tc_box_smem(bits); }
constexpr int kTcAhead = 3;                            // stages of lead of the parameter loads
constexpr int kTcItems = 5;                            // instructions per chunk: four on codes, one correction
constexpr int kTcMaxStages = 8;
__host__ __device__ constexpr int tc_min_stages(int bits) { return bits == 2 ? 3 : 2; }   // at least 48 KB in flight
constexpr uint64_t kTcWaitLimitNs = 2000000000ull;
constexpr size_t kTcSmemBudget = 227 * 1024;             // the most a CTA can be given (eight tokens of 8192 columns need 225.2 KB)

struct TcCtl {
  uint64_t full[kTcMaxStages];
  uint64_t empty[kTcMaxStages];
  uint64_t part_ready[2];
  uint64_t part_free[2];
  int abort;
};

struct TcLayout {
  size_t xb_off, part_off, ctl_off, total;             // byte offsets from the 1024-byte aligned ring base
  int stages;
};

// Shared-memory plan for T tokens and in_features columns of `bits`-bit codes.
__host__ __device__ inline TcLayout tc_layout(int T, int in_features, int stages, int bits) {
  TcLayout L;
  // chunks of 64 columns, counted up to the end of the last (possibly partial) 128-byte box (512 columns of 2-bit
  // codes, 256 of 4-bit codes): the entries past in_features are zeros, so the compute loop needs no end-of-row case
  const int box_cols = tc_box_bytes(bits) * 8 / bits;
  const size_t chunks = (size_t)((in_features + box_cols - 1) / box_cols) * (box_cols / 64);
  L.stages = stages;
  L.xb_off = (size_t)stages * tc_stage_bytes(bits);
  L.part_off = L.xb_off + chunks * kTcItems * 4 * T * 8;             // permuted bf16 activations + correction terms
  L.ctl_off = L.part_off + (size_t)2 * kTcWarps * kTcRows * kTcMaxTokens * 4;
  L.total = L.ctl_off + sizeof(TcCtl) + 1024 /*alignment slack*/;
  return L;
}

inline int tc_stages_that_fit(int T, int in_features, int bits) {
  for (int st = kTcMaxStages; st >= tc_min_stages(bits); --st)
    if (tc_layout(T, in_features, st, bits).total <= kTcSmemBudget) return st;
  return 0;
}

__device__ int g_gemv_status[2];   // [0] = eqat_status, [1] = WaitSite

__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int* abort, int site, uint32_t sleep_ns,
                                        uint64_t limit_ns = kTcWaitLimitNs) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = ptx::globaltimer_ns();
  uint32_t n = 0;
  while (!ptx::mbar_try_wait(bar, parity)) {
    if (sleep_ns != 0) __nanosleep(sleep_ns);
    if ((++n & 31u) == 0u) {
      if (*abort) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) {
        *abort = 1;
        atomicExch(&g_gemv_status[1], site);
        atomicExch(&g_gemv_status[0], (int)EQAT_ERR_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

// Programmatic dependent launch: let the next launch of the stream start / wait until the launches before this one
// have completed and their writes are visible (both do nothing in a launch without the attribute).
__device__ __forceinline__ void grid_dependents_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// (t & mask) | magic on both halves of a register.
__device__ __forceinline__ uint32_t and_or(uint32_t t, uint32_t mask, uint32_t magic) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(t), "r"(mask), "r"(magic));
  return r;
}

// D += A * B, A 16x16 (row), B 16x8 (col), bf16 inputs, fp32 accumulators.
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The first instruction of a chain: D = A * B (the accumulator input is the constant zero, no register is cleared).
__device__ __forceinline__ void mma_16816_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%10, %10, %10, %10};"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}

// (t & MASK) | magic with the mask as an immediate of the instruction and the magic in a register.  The logic
// instruction takes one immediate; given two compile-time constants the compiler re-creates one of them with a
// move in front of every use, which doubled the instruction count of the expansion.  The callers therefore pass
// magics whose value the compiler cannot see (TcMagics).
template <uint32_t MASK>
__device__ __forceinline__ uint32_t and_imm_or(uint32_t t, uint32_t magic) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(t), "n"(MASK), "r"(magic));
  return r;
}
// The bf16 pairs (128, 128), (32, 32), (8, 8), built from a value that is zero at run time only.
struct TcMagics {
  uint32_t m128, m32, m8, m32_128;                      // the last: 32 in the high half, 128 in the low half
  __device__ __forceinline__ explicit TcMagics(uint32_t zero)
      : m128(0x43004300u | zero), m32(0x42004200u | zero), m8(0x41004100u | zero), m32_128(0x42004300u | zero) {}
};

// Register r (0..7) of the expansion of a lane's 16 codes of one row.
// 2-bit codes: one word, register r holds codes r and r + 8 as a bf16 pair.  Registers 0..2 come from the word
// itself, 3..5 from the word shifted by 6, 6..7 from the word shifted by 12 (the compiler shares the shifts), each
// with the mask and the constant of the position the code is left at (128, 32 or 8).
// 4-bit codes: two words of eight codes, code j at bits [4j, 4j + 4); registers 0..3 hold codes (p, p + 4) of the
// first word, 4..7 of the second, all with the constant 128 (the codes fill the low four mantissa bits, so there
// is no room to skip a shift).
// 3-bit codes: w[0] and w[1] hold the lane's 48 bits (code j at bits [3j, 3j + 3); bits 48 and up of w[1] belong to
// the next lane).  Register r < 6 comes from the 32 bits starting at bit 3r: code r at the bottom of the low half
// (constant 128) and code r + 6 at bits 2-4 of the high half (constant 32, whose last place is a quarter).
// Registers 6 and 7 hold codes (12, 14) and (13, 15), moved to the bottom of their halves one at a time.
template <int BITS>
__device__ __forceinline__ uint32_t expand_reg(const uint32_t (&w)[tc_words_per_lane(BITS)], int r, const TcMagics& k) {
  if constexpr (BITS == 3) {
    if (r < 6) return and_imm_or<0x001C0007u>(r == 0 ? w[0] : __funnelshift_r(w[0], w[1], 3 * r), k.m32_128);
    const uint32_t low = and_imm_or<0x00000007u>(w[1] >> (r == 6 ? 4 : 7), k.m128);
    return and_imm_or<0x00070000u>(w[1] << (r == 6 ? 6 : 3), low);
  } else if constexpr (BITS == 2) {
    const uint32_t t = r < 3 ? w[0] : (r < 6 ? w[0] >> 6 : w[0] >> 12);
    const int pos = r % 3;
    return pos == 0 ? and_imm_or<0x00030003u>(t, k.m128)
                    : (pos == 1 ? and_imm_or<0x000C000Cu>(t, k.m32) : and_imm_or<0x00300030u>(t, k.m8));
  } else {
    return and_imm_or<0x000F000Fu>(w[BITS == 4 ? (r >> 2) : 0] >> (4 * (r & 3)), k.m128);
  }
}
// Which of a lane's 16 columns sits in half `half` (0 = low) of register r (0..7) of the expansion.
template <int BITS>
__host__ __device__ constexpr int tc_column(int r, int half) {
  if (BITS == 3) return r < 6 ? r + 6 * half : r + 6 + 2 * half;
  return BITS == 2 ? r + 8 * half : (r < 4 ? r + 4 * half : r + 4 + 4 * half);
}
// Constant that the expansion adds to column j (0..15) of a lane.
template <int BITS>
__host__ __device__ constexpr float tc_bias(int j) {
  if (BITS == 3) return (j >= 6 && j < 12) ? 32.0f : 128.0f;
  return BITS == 4 ? 128.0f : ((j & 7) % 3 == 0 ? 128.0f : ((j & 7) % 3 == 1 ? 32.0f : 8.0f));
}

template <int BITS, int PARAM_MODE, bool ZF16>
__global__ void __launch_bounds__(kTcThreads, 1)
packed_gemv_tc_kernel(const __grid_constant__ CUtensorMap map_w, const eqat_bf16* __restrict__ X,
                      const eqat_fp16* __restrict__ s16, const void* __restrict__ zq, eqat_bf16* __restrict__ Y,
                      int out_features, int in_features, int group_shift, int groups_per_row, int T, int stages) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_addr(smem_raw);
  const uint32_t ring_addr = (raw_addr + 1023u) & ~1023u;          // boxes are 1024-byte aligned (swizzle period)
  uint8_t* ring = smem_raw + (ring_addr - raw_addr);
  constexpr int kTcBoxBytes = tc_box_bytes(BITS), kTcBoxSmem = tc_box_smem(BITS);
  constexpr int kChunksPerBox = kTcBoxBytes * 8 / BITS / 64;        // 64-column chunks of a row per box: 8 or 4
  constexpr int kChunksPerWarp = 4;                                 // half a box (2-bit codes) or a box (4-bit codes)
  constexpr int kBoxesPerStage = tc_boxes_per_stage(BITS);
  constexpr int kStageBytes = tc_stage_bytes(BITS);
  const TcLayout L = tc_layout(T, in_features, stages, BITS);
  uint2* xb = reinterpret_cast<uint2*>(ring + L.xb_off);           // [chunk][quad lane][token][item] -> 4 bf16
  float* part = reinterpret_cast<float*>(ring + L.part_off);       // [2][warp][row][kTcMaxTokens]
  TcCtl* ctl = reinterpret_cast<TcCtl*>(ring + L.ctl_off);
  volatile int* abort_flag = &ctl->abort;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tasks = out_features / kTcRows;
  const int chunks = in_features >> 6;
  const int row_bytes = in_features * BITS / 8;
  const int n_boxes = (row_bytes + kTcBoxBytes - 1) / kTcBoxBytes;
  const int task_stages = (n_boxes + kBoxesPerStage - 1) / kBoxesPerStage;
  const int chunks_pad = n_boxes * kChunksPerBox;

  // Launched with programmatic stream serialisation: the next launch of the stream may start as soon as every
  // CTA of this grid has got here, and a CTA of this grid may be running while the launch before it still is.
  // Nothing before the wait below touches global memory (the barriers live in this CTA's shared memory); the
  // wait returns once the earlier grids have completed and their writes are visible.
  grid_dependents_launch();
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), 1);
      ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), kTcWarps);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(ptx::smem_addr(&ctl->part_ready[b]), kTcWarps);
      ptx::mbar_init(ptx::smem_addr(&ctl->part_free[b]), 1);
    }
    ctl->abort = 0;
    ptx::fence_mbar_init();
  }
  grid_dependency_wait();

  // Consumers request their first loads before the rest of the set-up: the first unit of the activations and the step
  // sizes / zero points of the first stages.  They are first touches of their pages in this launch, and once the
  // weight stream is running a small load waits behind megabytes of bulk copies.
  const int units = T * chunks_pad * 4;                                // (token, chunk, quad lane): 16 columns each
  auto unit_src = [&](int u) -> const uint4* {
    const int uq = u & 3, cg = (u >> 2) % chunks_pad, t = (u >> 2) / chunks_pad;
    return cg < chunks ? reinterpret_cast<const uint4*>(X + (size_t)t * in_features + (size_t)cg * 64 + uq * 16) : nullptr;
  };
  uint4 x_first[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
  if (warp < kTcWarps && (int)threadIdx.x < units) {
    const uint4* src = unit_src(threadIdx.x);
    if (src != nullptr) { x_first[0] = __ldg(src); x_first[1] = __ldg(src + 1); }
  }

  const int g = lane >> 2, q = lane & 3;
  const int box = BITS == 2 ? warp >> 1 : warp, chunk0 = BITS == 2 ? (warp & 1) * kChunksPerWarp : 0;
  // Step sizes (fp16) and zero points (bytes) of this lane's four chunks of stage k of a task, rows g and g + 8,
  // in up to four slots.  The four chunks are 256 consecutive columns starting at a multiple of 256: four groups
  // of 64 (mode 1), two groups of 128 (mode 2) or part of one larger group (mode 3), fetched with one load per row
  // and kind where the rows of parameters keep the alignment for it; mode 0 fetches chunk by chunk.  Chunk c uses
  // slot c >> kSlotShift.  The loaded registers are not touched before the stage is computed (three stages later):
  // an instruction on them here would wait for the load.
  // Zero points: one byte per slot in z_lo.x / z_hi.x, or (ZF16) one fp16 value per slot like the step sizes.
  struct StageParams { uint2 s_lo, s_hi, z_lo, z_hi; };
  constexpr int kSlotShift = PARAM_MODE == 2 ? 1 : (PARAM_MODE == 3 ? 2 : 0);
  const uint8_t* const z8 = static_cast<const uint8_t*>(zq);
  const eqat_fp16* const z16 = static_cast<const eqat_fp16*>(zq);
  auto fetch = [&](int task, int k) {
    StageParams sp;
    sp.s_lo = sp.s_hi = sp.z_lo = sp.z_hi = make_uint2(0u, 0u);
    const int cg0 = (k * kBoxesPerStage + box) * kChunksPerBox + chunk0;
    if (task < n_tasks && cg0 < chunks) {
      const size_t p_lo = (size_t)(task * kTcRows + g) * groups_per_row, p_hi = p_lo + (size_t)8 * groups_per_row;
      if constexpr (PARAM_MODE == 1) {                    // the row has a multiple of four groups: all four exist
        sp.s_lo = __ldg(reinterpret_cast<const uint2*>(s16 + p_lo + cg0));
        sp.s_hi = __ldg(reinterpret_cast<const uint2*>(s16 + p_hi + cg0));
        if constexpr (ZF16) {
          sp.z_lo = __ldg(reinterpret_cast<const uint2*>(z16 + p_lo + cg0));
          sp.z_hi = __ldg(reinterpret_cast<const uint2*>(z16 + p_hi + cg0));
        } else {
          sp.z_lo.x = __ldg(reinterpret_cast<const uint32_t*>(z8 + p_lo + cg0));
          sp.z_hi.x = __ldg(reinterpret_cast<const uint32_t*>(z8 + p_hi + cg0));
        }
      } else if constexpr (PARAM_MODE == 2) {             // an even number of groups per row: both exist
        const int g0 = cg0 >> 1;
        sp.s_lo.x = __ldg(reinterpret_cast<const uint32_t*>(s16 + p_lo + g0));
        sp.s_hi.x = __ldg(reinterpret_cast<const uint32_t*>(s16 + p_hi + g0));
        if constexpr (ZF16) {
          sp.z_lo.x = __ldg(reinterpret_cast<const uint32_t*>(z16 + p_lo + g0));
          sp.z_hi.x = __ldg(reinterpret_cast<const uint32_t*>(z16 + p_hi + g0));
        } else {
          sp.z_lo.x = __ldg(reinterpret_cast<const uint16_t*>(z8 + p_lo + g0));
          sp.z_hi.x = __ldg(reinterpret_cast<const uint16_t*>(z8 + p_hi + g0));
        }
      } else if constexpr (PARAM_MODE == 3) {
        const int grp = (cg0 << 6) >> group_shift;
        sp.s_lo.x = __ldg(s16 + p_lo + grp);
        sp.s_hi.x = __ldg(s16 + p_hi + grp);
        sp.z_lo.x = ZF16 ? (uint32_t)__ldg(z16 + p_lo + grp) : (uint32_t)__ldg(z8 + p_lo + grp);
        sp.z_hi.x = ZF16 ? (uint32_t)__ldg(z16 + p_hi + grp) : (uint32_t)__ldg(z8 + p_hi + grp);
      } else {
        uint32_t sl[4] = {0u, 0u, 0u, 0u}, sh[4] = {0u, 0u, 0u, 0u}, zl[4] = {0u, 0u, 0u, 0u}, zh[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int c = 0; c < kChunksPerWarp; ++c) {
          if (cg0 + c < chunks) {
            const int grp = ((cg0 + c) << 6) >> group_shift;
            sl[c] = __ldg(s16 + p_lo + grp);
            sh[c] = __ldg(s16 + p_hi + grp);
            zl[c] = ZF16 ? (uint32_t)__ldg(z16 + p_lo + grp) : (uint32_t)__ldg(z8 + p_lo + grp);
            zh[c] = ZF16 ? (uint32_t)__ldg(z16 + p_hi + grp) : (uint32_t)__ldg(z8 + p_hi + grp);
          }
        }
        sp.s_lo = make_uint2(sl[0] | (sl[1] << 16), sl[2] | (sl[3] << 16));
        sp.s_hi = make_uint2(sh[0] | (sh[1] << 16), sh[2] | (sh[3] << 16));
        if constexpr (ZF16) {
          sp.z_lo = make_uint2(zl[0] | (zl[1] << 16), zl[2] | (zl[3] << 16));
          sp.z_hi = make_uint2(zh[0] | (zh[1] << 16), zh[2] | (zh[3] << 16));
        } else {
          sp.z_lo.x = zl[0] | (zl[1] << 8) | (zl[2] << 16) | (zl[3] << 24);
          sp.z_hi.x = zh[0] | (zh[1] << 8) | (zh[2] << 16) | (zh[3] << 24);
        }
      }
    }
    return sp;
  };
  // kTcAhead stages of lead (the ring alone keeps 128 KB per SM in flight, so one stage is not enough)
  StageParams nx[kTcAhead];
  int pf_task = blockIdx.x, pf_k = 0;                     // next (task, stage) to request
  auto advance = [&]() {
    if (++pf_k == task_stages) { pf_k = 0; pf_task += gridDim.x; }
  };
#pragma unroll
  for (int i = 0; i < kTcAhead; ++i) {
    nx[i] = StageParams{make_uint2(0u, 0u), make_uint2(0u, 0u), make_uint2(0u, 0u), make_uint2(0u, 0u)};
    if (warp < kTcWarps) { nx[i] = fetch(pf_task, pf_k); advance(); }
  }

  __syncthreads();

  if (warp == kTcWarps) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      ptx::tma_prefetch_desc(&map_w);
      int slot = 0;
      uint32_t phase = 0;
      size_t issued = 0;
      bool ok = true;
      for (int task = blockIdx.x; task < n_tasks && ok; task += gridDim.x) {
        for (int k = 0; k < task_stages; ++k) {
          if (!tc_wait(ptx::smem_addr(&ctl->empty[slot]), phase ^ 1u, abort_flag, WAIT_STREAM_EMPTY, 32)) {
            ok = false;
            break;
          }
          ptx::fence_proxy_async_smem();                            // consumers' reads of this stage before the copies' writes
          const int nb = min(kBoxesPerStage, n_boxes - k * kBoxesPerStage);
          const uint32_t full = ptx::smem_addr(&ctl->full[slot]);
          ptx::mbar_expect_tx(full, (uint32_t)nb * kTcBoxSmem);     // bytes past the end of a row are zero-filled and counted
          for (int b = 0; b < nb; ++b)
            ptx::tma_load_2d(ring_addr + slot * kStageBytes + b * kTcBoxSmem, &map_w,
                             (k * kBoxesPerStage + b) * kTcBoxBytes, task * kTcRows, full);
          ++issued;
          if (++slot == stages) { slot = 0; phase ^= 1u; }
        }
      }
      if (!ok || *abort_flag) {
        // every copy this thread started must land before the CTA exits
        const size_t first = issued > (size_t)stages ? issued - stages : 0;
        for (size_t i = first; i < issued; ++i) {
          const uint32_t bar = ptx::smem_addr(&ctl->full[i % stages]);
          const uint32_t par = (uint32_t)((i / stages) & 1);
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(bar, par)) {
            if (ptx::globaltimer_ns() - t0 > 50000000ull) {
              atomicExch(&g_gemv_status[1], (int)WAIT_TEARDOWN);
              break;
            }
          }
        }
      }
    }
  } else if (warp == kTcWarps + 1) {
    // ---------------------------------------------------------------- reducer
    int buf = 0;
    uint32_t ready_phase[2] = {0u, 0u};
    for (int task = blockIdx.x; task < n_tasks; task += gridDim.x) {
      const bool got = tc_wait(ptx::smem_addr(&ctl->part_ready[buf]), ready_phase[buf], abort_flag, WAIT_EPI_ACC_FULL, 0);
      if (!__all_sync(0xFFFFFFFFu, got)) break;
      for (int idx = lane; idx < kTcRows * T; idx += 32) {
        const int r = idx & (kTcRows - 1), n = idx >> 4;
        float v = 0.0f;
#pragma unroll
        for (int wv = 0; wv < kTcWarps; ++wv)              // fixed order: deterministic
          v += part[((buf * kTcWarps + wv) * kTcRows + r) * kTcMaxTokens + n];
        Y[(size_t)n * out_features + (size_t)task * kTcRows + r] = (eqat_bf16)(pack_bf16x2(v, 0.0f) & 0xFFFFu);
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->part_free[buf]));
      ready_phase[buf] ^= 1u;
      buf ^= 1;
    }
  } else {
    // ---------------------------------------------------------------- consumers
    // Activations, in fragment order (zeros past in_features): unit (t, chunk, quad lane) = the 16 columns of that
    // lane's word.
    {
      const int tid = threadIdx.x;                                     // 0 .. 511
      for (int u0 = tid - lane; u0 < units; u0 += kTcWarps * 32) {     // warp-uniform bounds: the sums shuffle
        const int u = u0 + lane;
        const bool valid = u < units;
        float sb = 0.0f, sx = 0.0f;
        if (valid) {
          const int uq = u & 3, cg = (u >> 2) % chunks_pad, t = (u >> 2) / chunks_pad;
          uint4 v0 = x_first[0], v1 = x_first[1];
          if (u0 >= kTcWarps * 32) {                                   // later rounds load here
            const uint4* src = unit_src(u);
            v0 = v1 = make_uint4(0u, 0u, 0u, 0u);
            if (src != nullptr) { v0 = __ldg(src); v1 = __ldg(src + 1); }
          }
          const uint32_t r[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          uint32_t h[16];                                              // column j of the word as 16 bits
#pragma unroll
          for (int i = 0; i < 8; ++i) { h[2 * i] = r[i] & 0xFFFFu; h[2 * i + 1] = r[i] >> 16; }
          float sb4[4] = {0.0f, 0.0f, 0.0f, 0.0f}, sx4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
          for (int j = 0; j < 16; ++j) {                               // fixed order, four short chains
            const float xv = __uint_as_float(h[j] << 16);
            sb4[j & 3] = fmaf(tc_bias<BITS>(j), xv, sb4[j & 3]);
            sx4[j & 3] += xv;
          }
          sb = (sb4[0] + sb4[1]) + (sb4[2] + sb4[3]);
          sx = (sx4[0] + sx4[1]) + (sx4[2] + sx4[3]);
#pragma unroll
          for (int m = 0; m < 4; ++m)
            xb[(((size_t)cg * 4 + uq) * T + t) * kTcItems + m] =
                make_uint2(h[tc_column<BITS>(2 * m, 0)] | (h[tc_column<BITS>(2 * m, 1)] << 16),
                           h[tc_column<BITS>(2 * m + 1, 0)] | (h[tc_column<BITS>(2 * m + 1, 1)] << 16));
        }
        sb += __shfl_xor_sync(0xFFFFFFFFu, sb, 1); sx += __shfl_xor_sync(0xFFFFFFFFu, sx, 1);
        sb += __shfl_xor_sync(0xFFFFFFFFu, sb, 2); sx += __shfl_xor_sync(0xFFFFFFFFu, sx, 2);
        if (valid && (u & 3) == 0) {
          // correction item of the chunk: xb - 128 xs and xs, each as three bf16 numbers (round to nearest, the
          // remainders are exact in fp32), in the slots of quad lanes 0 and 1; lanes 2 and 3 supply zeros
          const int cg = (u >> 2) % chunks_pad, t = (u >> 2) / chunks_pad;
          float v[2] = {fmaf(-128.0f, sx, sb), sx};
          uint32_t parts[2][3];
#pragma unroll
          for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int pce = 0; pce < 3; ++pce) {
              const uint32_t hb = pack_bf16x2(v[i], 0.0f) & 0xFFFFu;
              parts[i][pce] = hb;
              v[i] -= __uint_as_float(hb << 16);
            }
          uint2* item = xb + ((size_t)cg * 4 * T + t) * kTcItems + 4;    // + quad lane * T * kTcItems
          item[0 * T * kTcItems] = make_uint2(parts[0][0] | (parts[0][1] << 16), parts[0][2] | (parts[1][0] << 16));
          // the three parts of xs once more per part of a three-part zero point (fp16 zero points; with byte zero
          // points their weights are zero)
          item[1 * T * kTcItems] = make_uint2(parts[1][1] | (parts[1][2] << 16), parts[1][0] | (parts[1][1] << 16));
          item[2 * T * kTcItems] = make_uint2(parts[1][2] | (parts[1][0] << 16), parts[1][1] | (parts[1][2] << 16));
          item[3 * T * kTcItems] = make_uint2(0u, 0u);
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kTcWarps * 32) : "memory");
    }

    // Correction weights by quad lane: lane 0 holds slots 0, 1 (-1, -1) and 8, 9 (-1, -(128 + z)), lane 1 slots
    // 2, 3 (-(128 + z) twice), lanes 2 and 3 zeros.  0xBF80 = -1, 0xC300 | z = -(128 + z) for z < 128.
    const uint32_t mask_a = q == 1 ? 0x007F007Fu : 0u, const_a = q == 0 ? 0xBF80BF80u : (q == 1 ? 0xC300C300u : 0u);
    const uint32_t mask_b = q == 0 ? 0x007F0000u : 0u, const_b = q == 0 ? 0xC300BF80u : 0u;
    // + chunk and item offsets.  Lanes whose token column does not exist read the last token's entry instead of
    // a zero: their accumulator columns are never stored.
    const uint2* xb_lane = xb + ((size_t)q * T + (g < T ? g : T - 1)) * kTcItems;
    const TcMagics magics((uint32_t)stages >> 30);                     // stages is at most kTcMaxStages
    int slot = 0, buf = 0;
    uint32_t phase = 0, free_phase[2] = {0u, 0u};
    bool alive = true;
    for (int task = blockIdx.x; task < n_tasks && alive; task += gridDim.x) {
      float tot[4] = {0.0f, 0.0f, 0.0f, 0.0f};                         // rows g, g + 8 x tokens 2q, 2q + 1
      for (int k = 0; k < task_stages; ++k) {
        const int gbox = k * kBoxesPerStage + box;
        const bool have = gbox < n_boxes;
        const StageParams sp = nx[0];
#pragma unroll
        for (int i = 0; i + 1 < kTcAhead; ++i) nx[i] = nx[i + 1];
        nx[kTcAhead - 1] = fetch(pf_task, pf_k);
        advance();
        const bool got = tc_wait(ptx::smem_addr(&ctl->full[slot]), phase, abort_flag, WAIT_STREAM_FULL, 0);
        if (!__all_sync(0xFFFFFFFFu, got)) { alive = false; break; }
        // a lane's 16 codes per row and chunk
        uint32_t w_lo[kChunksPerWarp][tc_words_per_lane(BITS)], w_hi[kChunksPerWarp][tc_words_per_lane(BITS)];
        if (have) {
          // 16-byte piece c of row r sits at piece (c ^ (r & 7)); rows g and g + 8 share the pattern
          const uint32_t row = ring_addr + slot * kStageBytes + box * kTcBoxSmem + g * kTcBoxBytes;
#pragma unroll
          for (int c = 0; c < kChunksPerWarp; ++c) {
            if constexpr (BITS == 3) {
              // no swizzle; the lane's 6 bytes start at byte 6q of the chunk's 24: the two words around them,
              // shifted down by 0 or 16 bits
              const uint32_t a = row + (uint32_t)(chunk0 + c) * 24u + (uint32_t)((6 * q) >> 2) * 4u;
              uint32_t lo0, lo1, hi0, hi1;
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(lo0) : "r"(a) : "memory");
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(lo1) : "r"(a + 4) : "memory");
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(hi0) : "r"(a + 8 * kTcBoxBytes) : "memory");
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(hi1) : "r"(a + 8 * kTcBoxBytes + 4) : "memory");
              const uint32_t sh = (q & 1) * 16u;
              w_lo[c][0] = __funnelshift_r(lo0, lo1, sh); w_lo[c][1] = lo1 >> sh;
              w_hi[c][0] = __funnelshift_r(hi0, hi1, sh); w_hi[c][1] = hi1 >> sh;
            } else if constexpr (BITS == 2) {                          // word q of the chunk's one piece
              const uint32_t a = row + ((uint32_t)((chunk0 + c) ^ g) << 4) + q * 4;
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w_lo[c][0]) : "r"(a) : "memory");
              asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w_hi[c][0]) : "r"(a + 8 * kTcBoxBytes) : "memory");
            } else {                                                   // words 2q, 2q + 1 of the chunk's two pieces
              const uint32_t a = row + ((uint32_t)(((chunk0 + c) * 2 + (q >> 1)) ^ g) << 4) + (q & 1) * 8;
              asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w_lo[c][0]), "=r"(w_lo[c][1]) : "r"(a) : "memory");
              asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(w_hi[c][0]), "=r"(w_hi[c][1])
                           : "r"(a + 8 * kTcBoxBytes) : "memory");
            }
          }
        }
        // The stage's next user is a copy of the asynchronous proxy, which the barrier alone does not order after
        // these generic-proxy reads: the readers fence here, the producer again between its wait and the copy.
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->empty[slot]));   // the stage can be refilled now
        if (++slot == stages) { slot = 0; phase ^= 1u; }
        if (have) {
#pragma unroll
          for (int c = 0; c < kChunksPerWarp; ++c) {                   // independent chains, no branches
            const int cg = gbox * kChunksPerBox + chunk0 + c;
            const uint2* item = xb_lane + (size_t)cg * (kTcItems * 4) * T;   // the lane's five entries of the chunk
            float D[4];
#pragma unroll
            for (int m = 0; m < 4; ++m) {                              // the four registers of A right before their use
              const uint2 b = item[m];
              const uint32_t a0 = expand_reg<BITS>(w_lo[c], 2 * m, magics), a1 = expand_reg<BITS>(w_hi[c], 2 * m, magics);
              const uint32_t a2 = expand_reg<BITS>(w_lo[c], 2 * m + 1, magics);
              const uint32_t a3 = expand_reg<BITS>(w_hi[c], 2 * m + 1, magics);
              if (m == 0) mma_16816_first(D, a0, a1, a2, a3, b.x, b.y);
              else mma_16816(D, a0, a1, a2, a3, b.x, b.y);
            }
            const int slot = c >> kSlotShift;                          // a constant once the loop is unrolled
            if constexpr (ZF16) {
              // correction with a real zero point: 128 + z as three bf16 numbers (an fp32 value split without
              // loss), each against the three parts of xs
              const uint32_t z2_lo = slot < 2 ? sp.z_lo.x : sp.z_lo.y, z2_hi = slot < 2 ? sp.z_hi.x : sp.z_hi.y;
              uint32_t a[2][2];
#pragma unroll
              for (int hrow = 0; hrow < 2; ++hrow) {
                const uint32_t z2 = hrow == 0 ? z2_lo : z2_hi;
                float t = 128.0f + __half2float(__ushort_as_half((unsigned short)((slot & 1) ? (z2 >> 16) : (z2 & 0xFFFFu))));
                uint32_t n[3];                                         // the negated parts
#pragma unroll
                for (int pce = 0; pce < 3; ++pce) {
                  const uint32_t hb = pack_bf16x2(t, 0.0f) & 0xFFFFu;
                  t -= __uint_as_float(hb << 16);
                  n[pce] = hb ^ 0x8000u;
                }
                a[hrow][0] = q == 0 ? 0xBF80BF80u : (q == 1 ? n[0] * 0x10001u : (q == 2 ? (n[1] | (n[2] << 16)) : 0u));
                a[hrow][1] = q == 0 ? (0xBF80u | (n[0] << 16)) : (q == 1 ? n[1] * 0x10001u : (q == 2 ? n[2] * 0x10001u : 0u));
              }
              const uint2 b = item[4];
              mma_16816(D, a[0][0], a[1][0], a[0][1], a[1][1], b.x, b.y);
            } else {
              // correction: weights -1 and -(128 + z) against the split sums (see the header)
              const uint32_t zz_lo = ((sp.z_lo.x >> (8 * slot)) & 0xFFu) * 0x10001u;
              const uint32_t zz_hi = ((sp.z_hi.x >> (8 * slot)) & 0xFFu) * 0x10001u;
              const uint2 b = item[4];
              mma_16816(D, and_or(zz_lo, mask_a, const_a), and_or(zz_hi, mask_a, const_a), and_or(zz_lo, mask_b, const_b),
                        and_or(zz_hi, mask_b, const_b), b.x, b.y);
            }
            const uint32_t s2_lo = slot < 2 ? sp.s_lo.x : sp.s_lo.y, s2_hi = slot < 2 ? sp.s_hi.x : sp.s_hi.y;
            const float s_lo = __half2float(__ushort_as_half((unsigned short)((slot & 1) ? (s2_lo >> 16) : (s2_lo & 0xFFFFu))));
            const float s_hi = __half2float(__ushort_as_half((unsigned short)((slot & 1) ? (s2_hi >> 16) : (s2_hi & 0xFFFFu))));
            tot[0] = fmaf(s_lo, D[0], tot[0]);
            tot[1] = fmaf(s_lo, D[1], tot[1]);
            tot[2] = fmaf(s_hi, D[2], tot[2]);
            tot[3] = fmaf(s_hi, D[3], tot[3]);
          }
        }
      }
      if (!alive) break;
      const bool free_ok = tc_wait(ptx::smem_addr(&ctl->part_free[buf]), free_phase[buf] ^ 1u, abort_flag,
                                   WAIT_MMA_ACC_EMPTY, 0);
      if (!__all_sync(0xFFFFFFFFu, free_ok)) break;
      float* pw = part + (size_t)((buf * kTcWarps + warp) * kTcRows) * kTcMaxTokens;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int n = 2 * q + e;
        if (n < T) {
          pw[g * kTcMaxTokens + n] = tot[e];
          pw[(g + 8) * kTcMaxTokens + n] = tot[2 + e];
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->part_ready[buf]));
      free_phase[buf] ^= 1u;
      buf ^= 1;
    }
  }
}

// The give-up path of tc_wait alone: one warp, a barrier nothing signals, a short limit.
__global__ void tc_wait_expiry_kernel(uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_addr(&bar), 1);
    abort_word = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  (void)tc_wait(ptx::smem_addr(&bar), 0u, &abort_word, WAIT_SELFTEST, 0, limit_ns);
}

// Tensor map of a byte matrix [outer, inner_bytes] row-major for copies of box_bytes x box_outer rows laid out in
// shared memory as they are (no swizzle): the 96-byte boxes of 3-bit codes.
bool make_tmap_u8_plain(CUtensorMap* tm, const void* base, uint64_t inner_bytes, uint64_t outer, uint32_t box_bytes,
                        uint32_t box_outer) {
  using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static const EncodeFn enc = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  if (enc == nullptr) return false;
  const cuuint64_t dims[2] = {inner_bytes, outer};
  const cuuint64_t strides[1] = {inner_bytes};
  const cuuint32_t box[2] = {box_bytes, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BITS, int PARAM_MODE, bool ZF16>
int launch_tc_mode(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* zq,
                   eqat_bf16* Y, int group_shift, int stages, cudaStream_t st) {
  static SmemOptIn opt_in;
  if (!opt_in.ensure(packed_gemv_tc_kernel<BITS, PARAM_MODE, ZF16>, (int)kTcSmemBudget)) return EQAT_ERR_CUDA;
  CUtensorMap mw;
  const uint64_t row_bytes = (uint64_t)d.in_features * BITS / 8;
  if (!(BITS == 3 ? make_tmap_u8_plain(&mw, Wq, row_bytes, (uint64_t)d.out_features, tc_box_bytes(BITS), kTcRows)
                  : make_tmap_u8(&mw, Wq, row_bytes, (uint64_t)d.out_features, tc_box_bytes(BITS), kTcRows)))
    return EQAT_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return EQAT_ERR_CUDA;
  const int T = (int)d.tokens, n_tasks = d.out_features / kTcRows, ng = d.in_features / d.group;
  const TcLayout L = tc_layout(T, d.in_features, stages, BITS);
  // Programmatic stream serialisation: back-to-back launches of this kernel overlap the tail of one grid with the
  // CTA start-up of the next (the kernel waits for its predecessors before its first global access).  After a
  // kernel that never signals its dependents the launch behaves like an ordinary one.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_tasks < sms ? n_tasks : sms));
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = L.total;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, packed_gemv_tc_kernel<BITS, PARAM_MODE, ZF16>, mw, X, s16, zq, Y,
                         d.out_features, d.in_features, group_shift, ng, T, stages) != cudaSuccess) {
    (void)cudaGetLastError();
    return EQAT_ERR_CUDA;
  }
  return launch_status();
}

template <int BITS, bool ZF16>
int launch_tc_format(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* zq,
                     eqat_bf16* Y, int group_shift, int stages, cudaStream_t st) {
  // how a lane fetches the parameters of its 256 columns of a stage (see the kernel): one load per row and kind
  // where the rows of step sizes and zero points keep the alignment those loads need, chunk by chunk otherwise
  const uintptr_t s_addr = reinterpret_cast<uintptr_t>(s16), z_addr = reinterpret_cast<uintptr_t>(zq);
  const uintptr_t z_unit = ZF16 ? 2 : 1;                 // bytes per zero point
  const int ng = d.in_features / d.group;
  if (d.group == 64 && ng % 4 == 0 && (s_addr & 7u) == 0 && (z_addr & (4 * z_unit - 1)) == 0)
    return launch_tc_mode<BITS, 1, ZF16>(d, X, Wq, s16, zq, Y, group_shift, stages, st);
  if (d.group == 128 && ng % 2 == 0 && (s_addr & 3u) == 0 && (z_addr & (2 * z_unit - 1)) == 0)
    return launch_tc_mode<BITS, 2, ZF16>(d, X, Wq, s16, zq, Y, group_shift, stages, st);
  if (d.group >= 256) return launch_tc_mode<BITS, 3, ZF16>(d, X, Wq, s16, zq, Y, group_shift, stages, st);
  return launch_tc_mode<BITS, 0, ZF16>(d, X, Wq, s16, zq, Y, group_shift, stages, st);
}

template <int BITS>
int launch_tc(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16, const void* zq,
              eqat_bf16* Y, int group_shift, int stages, cudaStream_t st) {
  return d.zero_point_format == EQAT_ZP_FP16 ? launch_tc_format<BITS, true>(d, X, Wq, s16, zq, Y, group_shift, stages, st)
                                             : launch_tc_format<BITS, false>(d, X, Wq, s16, zq, Y, group_shift, stages, st);
}

}  // namespace

// How the tokens go through the kernel: in one launch when the shared-memory plan fits all
// tokens, otherwise (long rows, or more than eight tokens) as several launches over slices of the tokens, each of
// which streams the packed weight once more.  That is taken only while it is clearly cheaper than the tiled kernel
// of gemm.cu.  Cost model (from timings on the Llama-2 7B, 13B and 70B shapes): a launch of this kernel takes about
// 4 us + 0.5 us per token + the packed weight at 2.25 / 2.6 / 3.5 TB/s (2 / 3 / 4-bit codes; 4 % more per further
// token); the tiled kernel takes about 1 / 1.45 / 1.2 us per 64 input columns for any token count below a full
// row-tile, because the K loop of a tile is serial.
struct TcPlan {
  int launches, slice;                                   // slice = tokens per launch (the last one may have fewer)
};

static TcPlan tc_plan(const eqat_desc& d) {
  const TcPlan none{0, 0};
  if (d.bits < 2 || d.bits > 4 || d.group < 64 || d.tokens < 1 || d.tokens > kTcMaxTotalTokens) return none;
  if (((int64_t)d.in_features * d.bits / 8) % 16 != 0) return none;    // the copy engine wants rows of 16-byte multiples
  const int T = (int)d.tokens;
  int fit = T < kTcMaxTokens ? T : kTcMaxTokens;
  while (fit >= 1 && tc_stages_that_fit(fit, d.in_features, d.bits) == 0) --fit;
  if (fit < 1) return none;
  const int launches = (T + fit - 1) / fit, slice = (T + launches - 1) / launches;
  if (launches > 1) {
    const double weight_mb = (double)d.out_features * d.in_features * d.bits / 8.0 / 1.0e6;
    const double stream_tbs = d.bits == 2 ? 2.25 : (d.bits == 3 ? 2.6 : 3.5);
    const double tiled_us = d.in_features / 64.0 * (d.bits == 2 ? 1.0 : (d.bits == 3 ? 1.45 : 1.2));
    const double few_us = launches * (4.0 + 0.5 * slice + weight_mb / stream_tbs * (1.0 + 0.04 * (slice - 1)));
    if (few_us >= 0.8 * tiled_us) return none;
  }
  return TcPlan{launches, slice};
}

bool packed_gemv_applies(const eqat_desc& d) {
  // a 64-column chunk must lie inside one group: groups of 32 go through the tiled kernel
  return d.tokens >= 1 && d.group >= 64 && tc_plan(d).launches > 0;
}

int launch_packed_gemv(const eqat_desc& d, const eqat_bf16* X, const uint8_t* Wq, const eqat_fp16* s16,
                       const void* zq, eqat_bf16* Y, cudaStream_t st) {
  int group_shift = 31;                                  // one group per row: every group index shifts to 0
  if (d.group <= 256) {
    group_shift = 0;
    while ((1 << group_shift) < d.group) ++group_shift;
  }
  const TcPlan plan = tc_plan(d);
  if (plan.launches > 0) {
    for (int t0 = 0; t0 < (int)d.tokens; t0 += plan.slice) {
      eqat_desc part = d;
      part.tokens = (int)d.tokens - t0 < plan.slice ? (int)d.tokens - t0 : plan.slice;
      const int stages = tc_stages_that_fit((int)part.tokens, d.in_features, d.bits);
      const eqat_bf16* Xs = X + (size_t)t0 * d.in_features;
      eqat_bf16* Ys = Y + (size_t)t0 * d.out_features;
      const int rc = d.bits == 2   ? launch_tc<2>(part, Xs, Wq, s16, zq, Ys, group_shift, stages, st)
                     : d.bits == 3 ? launch_tc<3>(part, Xs, Wq, s16, zq, Ys, group_shift, stages, st)
                                   : launch_tc<4>(part, Xs, Wq, s16, zq, Ys, group_shift, stages, st);
      if (rc != EQAT_OK) return rc;
    }
    return EQAT_OK;
  }
  return EQAT_ERR_UNSUPPORTED;                           // not reached for a problem packed_gemv_applies() accepted
}

int launch_wait_expiry_gemv(cudaStream_t st) {
  tc_wait_expiry_kernel<<<1, 32, 0, st>>>(1000000ull);   // 1 ms
  return launch_status();
}

int read_gemv_status(int* status, int* detail) {
  int h[2] = {0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess) return EQAT_ERR_CUDA;
  if (cudaMemcpyFromSymbol(h, g_gemv_status, sizeof(h)) != cudaSuccess) return EQAT_ERR_CUDA;
  const int zero[2] = {0, 0};
  if (cudaMemcpyToSymbol(g_gemv_status, zero, sizeof(zero)) != cudaSuccess) return EQAT_ERR_CUDA;
  *status = h[0];
  *detail = h[1];
  return EQAT_OK;
}

}  // namespace eqat
