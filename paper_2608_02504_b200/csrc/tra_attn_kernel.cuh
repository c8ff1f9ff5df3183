// Dense attention with fused entropy (Eq. 1, Eq. 2, Algorithm 2) and block-sparse attention
// (Eq. 16 as executed over retained blocks) for sm_100a: the kernel template and its launcher.
// Included by one translation unit per (head_dim, block) shape.
//
// One CTA owns two 128-row query tiles of one (batch, head).  Both S = Q K^T and O += P V run on
// the 5th-generation tensor cores (tcgen05.mma, kind::f16, bf16 operands, fp32 accumulators in
// tensor memory).  K/V tiles of the retained key blocks are fetched by TMA into a shared-memory
// ring.  Warp roles:
//   warps 0-3  softmax of query tile 0 (one thread per query row, tcgen05.ld of its S row)
//   warps 4-7  softmax of query tile 1
//   warp  8    TMA producer (Q once, then K_v, V_v for every key block v of the CTA's list)
//   warp  9    tensor-memory allocation and the single MMA-issuing thread
//   warps 10-11 idle: they complete the third warpgroup, whose registers are handed to the softmax
//              warps with setmaxnreg so that a softmax thread can keep its whole S row in registers
// Tensor-memory columns: score buffers SB0 [0,128) and SB1 [128,256), accumulators O0 [256,384) and
// O1 [384,512); the bf16 P of a job overwrites the first half of its score buffer and feeds the PV
// MMA straight from tensor memory.
//
// Jobs.  The key-block list of the CTA is the union of the lists of the query blocks it holds.  A
// job is one (key block of the list, tile that retains it) pair; jobs are numbered in list order,
// tile 0 before tile 1.  Job n computes its scores into buffer n & 1 and accumulates into the O of
// its tile, and the tensor pipe sees  S_0, S_1, [PV_0, S_2], [PV_1, S_3], ...  : the scores of job
// n + 2 are issued right behind the PV of job n, whose P they overwrite.  When both tiles retain a
// key block its two jobs use the two buffers and each tile's softmax runs while the other tile's
// MMAs execute.  When only one tile retains a run of key blocks, that tile's consecutive jobs
// alternate between the two buffers, so the scores of its next block are computed while its
// softmax still works on the current one (a lone tile is not serialised on its own
// S -> softmax -> PV chain).  Dense launches (kDense) have no list and count key blocks instead.
// With kTokenMask the softmax threads also remove, inside every retained block, the keys outside
// their query's disk (Eq. 15).
//
// Online softmax state per row, in the base-2 domain (t = s * sm_scale * log2 e):
//   m  running reference maximum (raised only when the new maximum exceeds it by more than 8,
//      so the O accumulator is rescaled rarely; exact because every term uses the same m),
//   l  = sum 2^(t - m),   a = sum 2^(t - m) (t - m)   (the entropy accumulator of Algorithm 2,
//      centred on m, which keeps its magnitude small).
// At the end  O = o / l,  lse = (m + log2 l) ln 2,  H = ln l - ln 2 * a / l
// (= m + log l - (sum e^(s-m) s) / l of Algorithm 2 with s measured from m).
//
// Every wait on an mbarrier is bounded: after about two seconds the waiting thread records
// TRA_ERR_TIMEOUT in the plan's status word, raises a CTA-wide abort flag and every role leaves
// its loop; tensor memory is released on every path.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "tra_attn_shapes.h"
#include "tra_common.cuh"

namespace {

constexpr int kThreads = 384;         // 12 warps: three per SM sub-partition
constexpr int kRegsSoftmax = 216;     // per-thread registers after setmaxnreg: 2 * 216 + 72 = 3 * 168
constexpr int kRegsControl = 72;
constexpr int kTileM = 128;           // query rows per tile (UMMA M)
constexpr int kMaxBitmapWords = 64;   // key blocks per row <= 2048
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// ------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false = gave up (abort flag raised by this or another thread).
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            int* status, unsigned long long limit_ns = kWaitLimitNs) {
  // The global timer is slow to read, so it is consulted only after many failed polls (each
  // try_wait already suspends the thread for a while): ordinary waits never touch it.
#pragma unroll 1
  for (uint32_t it = 0; it < 4096u; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        tra_set_status(status, TRA_ERR_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}

// A whole warp waits.  Every lane polls: one polling lane followed by a warp vote wakes the warp later,
// and the wake-up latency of the softmax and MMA warps is on the critical path of every key block.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int* status) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, "
      "%4}], [%5];" ::"r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// The MMA warp runs its loop with all 32 lanes (warp-uniform control flow and descriptor
// arithmetic); the tcgen05.mma / tcgen05.commit instructions themselves are issued by one elected lane.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred pe;\n\t"
      "elect.sync _|pe, 0xffffffff;\n\t"
      "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar)
      : "memory");
}
// D[tmem] (+)= A[smem] * B[smem].  Descriptors arrive as (lo, hi) words so that stepping along K
// is one 32-bit add on the issuing thread.
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                          uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, pe;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "elect.sync _|pe, 0xffffffff;\n\t"
      "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, pe;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "elect.sync _|pe, 0xffffffff;\n\t"
      "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
      "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
      "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
      "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// Waits for this thread's tcgen05.ld; the 32 destination registers are named as read-write
// operands so that the compiler cannot move a use of them above the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t* r) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]),
                 "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]),
                 "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                 "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
// Compiler-only fence on 32 registers filled by an earlier tcgen05.ld: keeps their uses below
// the tcgen05.wait::ld that precedes this statement.
__device__ __forceinline__ void reg_fence32(uint32_t* r) {
  asm volatile(""
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]),
                 "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]),
                 "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]),
                 "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]),
                 "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}
__device__ __forceinline__ void tmem_wait_st() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// ---- packed fp32 pairs (sm_100 f32x2 arithmetic: one instruction for two lanes of a row) ----
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// floor(sqrt(n)) for 0 <= n < 2^22 with no conversion instruction (conversions share the
// special-function unit with ex2): n + 0.5 is formed from the 2^23 bit pattern, sqrt.approx of it
// stays at least 0.25 / sqrt(n) away from every integer, and adding 2^23 - 0.5 rounds it down into
// the low mantissa bits.
__device__ __forceinline__ int tra_isqrt_small_nocvt(int n) {
  const float f = __uint_as_float(0x4B000000u | (uint32_t)n) - 8388607.5f;      // n + 0.5, exact
  float r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(f));
  return (int)(__float_as_uint(r + 8388607.5f) & 0x7FFFFFu);
}
// acc_lo += (float)low bf16 of `packed`, acc_hi += (float)high bf16: the mixed-precision add of
// sm_100 widens the bf16 operand itself (no shift / mask to unpack the pair first)
__device__ __forceinline__ void add_bf16_pair(float& acc_lo, float& acc_hi, uint32_t packed) {
  asm("{\n\t.reg .b16 lo, hi;\n\t"
      "mov.b32 {lo, hi}, %2;\n\t"
      "add.rn.f32.bf16 %0, lo, %0;\n\t"
      "add.rn.f32.bf16 %1, hi, %1;\n\t}"
      : "+f"(acc_lo), "+f"(acc_hi)
      : "r"(packed));
}
// bf16x2 with `lo` in the low half
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 format (version 1), as two words:
//   lo = start address >> 4 (14 bits) | leading byte offset >> 4 at bit 16
//   hi = stride byte offset >> 4 | version 1 at bit 14 | SWIZZLE_128B (2) at bits 29..31
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__host__ __device__ constexpr uint32_t desc_hi(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 x bf16, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

template <int D, int BN>
struct Cfg {
  static constexpr int kGroups = kTileM / BN;                 // query blocks per tile
  static constexpr int kBlocksPerCta = 2 * kGroups;
  static constexpr int kQTileBytes = kTileM * D * 2;
  static constexpr int kSlotBytes = BN * D * 2;
  static constexpr int kSlots = (D == 128 && BN > 96) ? 5 : 6;
  static constexpr int kChunks = (BN + 31) / 32;               // 32-key chunks of a score row
  static constexpr int kCols = kChunks * 32;
  static constexpr int kKSlots = 3;                            // block-sparse launches: K ring / V ring
  static constexpr int kVSlots = kSlots - kKSlots;
  static constexpr int kAtoms = D / 64;                        // 64-column swizzle atoms per row
  static constexpr int kQAtomBytes = kTileM * 128;
  static constexpr int kKVAtomBytes = BN * 128;
  static constexpr int kSmemData = 2 * kQTileBytes + kSlots * kSlotBytes;
  // at least 120 KB so that one CTA owns an SM and its whole tensor memory
  static constexpr int kSmemNeeded = kSmemData + 1024 /*alignment slack*/ + 2048 /*barriers, bitmaps*/;
  static constexpr int kSmemBytes = kSmemNeeded > 120 * 1024 ? kSmemNeeded : 120 * 1024;
};

struct SharedCtl {
  uint64_t q_full;
  uint64_t kv_full[6];
  uint64_t kv_release[16];   // ring slots are handed back in release events (see the TMA producer)
  uint64_t s_full[2][2];    // [tile][score buffer]: the scores of a job of that tile in that buffer are complete
  uint64_t p_ready[2][2];   // [score buffer][64-key half of the block]
  uint64_t o_done[2];       // [tile]: a PV whose tile also owns the next job has retired
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
  int dbg_jobs[4];          // bounds-checking build: jobs walked by softmax tile 0 / tile 1 / the MMA warp, entries loaded
  int rmax[4];              // largest candidate index among the video queries of each query block
  uint32_t bitmap[4][kMaxBitmapWords];
};
static_assert(sizeof(SharedCtl) <= 2048, "control block");

// Arguments of the optional token mask inside retained blocks (Eq. 15 applied on top of the block
// list): packed coordinates of the video tokens (padded by one block), thresholds, candidate indices.
struct TokenMaskArgs {
  const tra_block_boxes_t* boxes; // per-block boxes (plan table), for launches without a block list
  const uint32_t* slice;          // one word per 16 positions (plan table): run of one frame row or 0
  const uint32_t* coord_packed;
  const int32_t* theta;
  const uint16_t* ridx;
  int n_video;
  int T;
  int n_radii;                    // candidate indices are clamped to n_radii - 1
};

// ------------------------------------------------------------------------------------ kernel
// kDense: every query block attends to every key block (no block list; row_ptr is not read).
// kLse: the caller wants lse from a launch without entropy; the row sum of the unrounded
// probabilities is then accumulated next to the bf16-rounded one (kEntropy always does).
template <int D, int BN, bool kEntropy, bool kTokenMask, bool kDense, bool kLse, bool kAny>
__global__ void __launch_bounds__(kThreads, 1)
tra_attn_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, __nv_bfloat16* __restrict__ O,
                float* __restrict__ entropy, float* __restrict__ lse,
                const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                const int32_t* __restrict__ tile_pairs, int N, int NB, float scale_log2,
                int* __restrict__ status, TokenMaskArgs tm, int blk_arg,
                const int32_t* __restrict__ slice_raster, int raster_kv) {
  using C = Cfg<D, BN>;
  static_assert(!(kAny && kTokenMask), "the token mask needs blocks of whole 16-key slices");
  // kAny: blocks of blk <= BN tokens (BN = blk rounded up to a multiple of 16).  A key tile is still BN rows,
  // loaded from row v * blk: its last BN - blk rows belong to the next block and are masked as columns; a query
  // tile holds kGroups blocks in its first tile_rows rows and the rest of its 128 rows are computed and dropped.
  const int blk = kAny ? blk_arg : BN;
  const int tile_rows = C::kGroups * blk;
  constexpr bool kExact = kEntropy || kLse;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;                                   // [2 tiles][atoms][128 rows][64] bf16, swizzled
  uint8_t* sKV = smem + 2 * C::kQTileBytes;             // ring of K / V tiles
  SharedCtl* ctl = (SharedCtl*)(smem + C::kSmemData);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  // The two 128-row query tiles of this CTA: consecutive ones, or the pair the block-mask call chose
  // (tiles with similar block lists share a CTA, so that few key blocks serve one tile only).
  // A missing tile (index -1) has no rows and no list.
  const int NT = (N + tile_rows - 1) / tile_rows;
  int tile0 = 2 * (int)blockIdx.x, tile1 = 2 * (int)blockIdx.x + 1;
  if (!kDense && tile_pairs != nullptr) {
    const int32_t* pr = tile_pairs + ((size_t)bh * gridDim.x + blockIdx.x) * 2;
    tile0 = pr[0];
    tile1 = pr[1];
  }
  if (tile0 < 0 || tile0 >= NT) tile0 = -1;
  if (tile1 < 0 || tile1 >= NT) tile1 = -1;
  auto tile_index = [&](int k) { return k ? tile1 : tile0; };
  const int n_words = (NB + 31) >> 5;
  volatile int* abort_flag = &ctl->abort_flag;

  // ---- set-up --------------------------------------------------------------------------
  if (tid == 0) {
    mbar_init(smem_u32(&ctl->q_full), 1);
    for (int i = 0; i < C::kSlots; ++i) {
      mbar_init(smem_u32(&ctl->kv_full[i]), 1);
    }
    for (int i = 0; i < 16; ++i) mbar_init(smem_u32(&ctl->kv_release[i]), 1);
    for (int k = 0; k < 2; ++k) {
      mbar_init(smem_u32(&ctl->s_full[k][0]), 1);
      mbar_init(smem_u32(&ctl->s_full[k][1]), 1);
      mbar_init(smem_u32(&ctl->p_ready[k][0]), 4);     // one lane of each of the four warps of a tile
      mbar_init(smem_u32(&ctl->p_ready[k][1]), 4);
      mbar_init(smem_u32(&ctl->o_done[k]), 1);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(
                     smem_u32(&ctl->tmem_base))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < 4 * kMaxBitmapWords; i += kThreads) (&ctl->bitmap[0][0])[i] = 0u;
  if (tid < 4) {
    ctl->rmax[tid] = -1;
    ctl->dbg_jobs[tid] = 0;
  }
  __syncthreads();
  // Token-mask launch without a block list (Eq. 16 itself): the key blocks a query block can reach
  // at all, from the block boxes and the largest candidate index among its queries — a superset
  // of the blocks that hold a visible key; the token mask inside the kernel does the rest.
  const bool geometric_list = kTokenMask && row_ptr == nullptr;
  if (geometric_list) {
    for (int i = tid; i < 2 * kTileM; i += kThreads) {
      const int t = tile_index(i / kTileM);
      const int row = t * kTileM + i % kTileM;
      if (t >= 0 && row < tm.n_video)
        atomicMax(&ctl->rmax[i / BN], min((int)tm.ridx[(size_t)bh * N + row], tm.n_radii - 1));
    }
    __syncthreads();
    for (int g = 0; g < C::kBlocksPerCta; ++g) {
      const int t = tile_index(g / C::kGroups);
      const int ub = t * C::kGroups + g % C::kGroups;
      if (t < 0 || ub >= NB) continue;
      const bool q_text = (ub + 1) * BN > tm.n_video;        // holds a text query: sees every key
      const int rmax = ctl->rmax[g];
      const tra_block_boxes_t* ubx = tm.boxes + ub;      // read in place: a local copy indexed by a loop
      const int n_ubox = ubx->n_box;                    // variable would live in local memory
      for (int v = tid; v < NB; v += kThreads) {
        bool on = q_text || (v + 1) * BN > tm.n_video;         // text keys are always visible
        if (!on && rmax >= 0) {
          const tra_block_boxes_t* vb = tm.boxes + v;
          const int n_vbox = vb->n_box;
          for (int iu = 0; iu < n_ubox && !on; ++iu) {
            const uint4 au = __ldg(reinterpret_cast<const uint4*>(&ubx->box[iu]));
            const int a_t0 = (int16_t)(au.x & 0xffffu), a_t1 = (int16_t)(au.x >> 16), a_y0 = (int16_t)(au.y & 0xffffu),
                      a_y1 = (int16_t)(au.y >> 16), a_x0 = (int16_t)(au.z & 0xffffu), a_x1 = (int16_t)(au.z >> 16);
            for (int iv = 0; iv < n_vbox && !on; ++iv) {
              const uint4 cu = __ldg(reinterpret_cast<const uint4*>(&vb->box[iv]));
              const int c_t0 = (int16_t)(cu.x & 0xffffu), c_t1 = (int16_t)(cu.x >> 16), c_y0 = (int16_t)(cu.y & 0xffffu),
                        c_y1 = (int16_t)(cu.y >> 16), c_x0 = (int16_t)(cu.z & 0xffffu), c_x1 = (int16_t)(cu.z >> 16);
              const int dt_min = max(0, max(a_t0 - c_t1, c_t0 - a_t1));
              const int gy = max(0, max(a_y0 - c_y1, c_y0 - a_y1));
              const int gx = max(0, max(a_x0 - c_x1, c_x0 - a_x1));
              on = tm.theta[rmax * tm.T + dt_min] >= gy * gy + gx * gx;
            }
          }
        }
        if (on) atomicOr(&ctl->bitmap[g][v >> 5], 1u << (v & 31));
      }
    }
  }
  // key-block bitmaps of the query blocks this CTA holds (block-sparse launches only)
  for (int g = 0; g < C::kBlocksPerCta && !kDense && !geometric_list; ++g) {
    const int t = tile_index(g / C::kGroups);
    const int ub = t * C::kGroups + g % C::kGroups;
    if (t < 0 || ub >= NB) continue;
    {
      const long long r = (long long)bh * NB + ub;
      const int lo = row_ptr[r], hi = row_ptr[r + 1];
#ifdef TRA_DEBUG      // the list of a row lies inside the lists of the launch
      if (tid == 0 && (lo < 0 || hi < lo || hi > row_ptr[(long long)gridDim.y * NB]))
        tra_set_status(status, TRA_ERR_BOUNDS);
#endif
      for (int e = lo + tid; e < hi; e += kThreads) {
        const int v = col_idx[e];
        if (v >= 0 && v < NB) atomicOr(&ctl->bitmap[g][v >> 5], 1u << (v & 31));
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;

  // dense launches: a tile takes part when its first query block exists
  const bool tile1_on = tile1 >= 0;
  const int n_outer = kDense ? 1 : n_words;   // dense launches walk 0 .. NB-1 in one inner loop
  // bitmap of a tile = union over its query blocks
  auto tile_word = [&](int k, int w) -> uint32_t {
    uint32_t x = ctl->bitmap[k * C::kGroups][w];
    if (C::kGroups == 2) x |= ctl->bitmap[k * C::kGroups + 1][w];
    return x;
  };

  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsControl));
  if (warp == 8) {
    // ================================================================== TMA producer
    // One lane runs the producer; with the tensors in raster order the whole warp runs it in step (same state in
    // every lane), so that the sixteen small boxes of a tile are issued by sixteen lanes at once.
    // (slice_raster is set when Q and O are in raster order; raster_kv tells whether K and V are as well)
    const bool wide = slice_raster != nullptr && raster_kv;
    if (lane == 0 || wide) {
      const uint32_t qbar = smem_u32(&ctl->q_full);
      if (lane == 0) mbar_expect_tx(qbar, 2 * C::kQTileBytes);
      if (wide) __syncwarp();
      // Rows [row0, row0 + rows) of the tile-major order into a tile at `dst` (atoms `atom_bytes` apart).  With the
      // tensors in tile-major order that is one box per 64-column atom.  With the tensors in RASTER order
      // (slice_raster != NULL) every 16 consecutive tile-major positions are 16 consecutive raster rows, which
      // start at slice_raster[position / 16]: one box of 16 rows per slice, 2 KB apart in the tile (the swizzle
      // pattern repeats every 8 rows, so the tile in shared memory is the same either way).
      auto load_rows = [&](const CUtensorMap* map, uint32_t dst, uint32_t bar, int row0, int rows, int atom_bytes,
                           bool by_runs) {
        if (!by_runs) {
          if (lane == 0)
            for (int a = 0; a < C::kAtoms; ++a) tma_load_3d(dst + a * atom_bytes, map, bar, a * 64, row0, bh);
        } else if (wide) {
          const int j = lane & 7, a = lane >> 3;           // lane -> (slice, atom)
          if (a < C::kAtoms && j * 16 < rows)
            tma_load_3d(dst + a * atom_bytes + j * 2048, map, bar, a * 64, __ldg(slice_raster + (row0 >> 4) + j), bh);
        } else {                                           // the one producer lane issues every box (Q only)
          for (int j = 0; j * 16 < rows; ++j)
            for (int a = 0; a < C::kAtoms; ++a)
              tma_load_3d(dst + a * atom_bytes + j * 2048, map, bar, a * 64, __ldg(slice_raster + (row0 >> 4) + j), bh);
        }
      };
      for (int k = 0; k < 2; ++k)      // a missing tile loads rows nobody uses
        load_rows(&map_q, smem_u32(sQ + k * C::kQTileBytes), qbar, max(tile_index(k), 0) * tile_rows, kTileM,
                  C::kQAtomBytes, slice_raster != nullptr);
      bool alive = true;
      auto load_tile = [&](const CUtensorMap* map, int slot, int v) {
        const uint32_t fbar = smem_u32(&ctl->kv_full[slot]);
        if (lane == 0) mbar_expect_tx(fbar, C::kSlotBytes);
        if (wide) __syncwarp();
        load_rows(map, smem_u32(sKV + slot * C::kSlotBytes), fbar, v * blk, BN, C::kKVAtomBytes, wide);
      };
      if constexpr (kDense) {
        // Loads go K0, V0, K1, V1, ... into consecutive slots.  The MMA warp hands slots back in
        // release events: event 0 frees K0, event e + 1 frees V_e and K_(e+1) with one commit, so load
        // j is freed by event (j + 1) / 2.  Event r arrives on kv_release[r % 8] as its (r / 8)-th
        // completion; the producer has always passed event r before event r + 8 can be committed.
        int slot = 0, n_load = 0;
        for (int v = 0; v < NB && alive; ++v) {
          for (int kv = 0; kv < 2; ++kv) {
            if (n_load >= C::kSlots) {          // the slot's previous load must have been released
              const int r = (n_load - C::kSlots + 1) >> 1;
              if (!mbar_wait(smem_u32(&ctl->kv_release[r & 7]), (uint32_t)(r >> 3) & 1u, abort_flag, status)) {
                alive = false;
                break;
              }
            }
            ++n_load;
            load_tile(kv == 0 ? &map_k : &map_v, slot, v);
            if (++slot == C::kSlots) slot = 0;
          }
        }
      } else {
        // Block-sparse launches keep K tiles and V tiles in rings of their own (kKSlots + kVSlots
        // slots): the scores of a job are issued two jobs ahead of its PV, so K tiles turn over early
        // and V tiles late, and a lone tile consumes a tile of each per job.  The MMA warp commits
        // once per group of its job stream: commit 0 after the first two S, commit n + 1 after group n
        // (PV of job n, S of job n + 2), on kv_release[c % 16].  With n_last(e) the last job of list
        // entry e, K_e is free after commit max(0, n_last(e) - 1) and V_e after commit n_last(e) + 1.
        // Commits are waited for one by one, in order; the MMA warp cannot get 8 commits ahead.
        // The K loads and the V loads are two streams over the same list, each issued as soon as its
        // own slot is free, so that a V tile waiting for its slot does not hold back the K tiles the
        // next scores need.  Commits are observed one by one, in order (with three K slots the MMA
        // warp cannot get more than six commits ahead of the one the producer looks at).
        struct Stream {
          int w;                       // next bitmap word
          uint32_t bits, word0, word1; // entries of the current word still to load
          uint32_t jobs;               // jobs of the entries already walked
          int e, slot;                 // entries loaded, next slot
          uint32_t f1, f2, f3;         // freeing commits of the tiles of the last three entries
          bool more;                   // an entry is waiting in `bits`
        };
        auto advance = [&](Stream& st) {   // moves to the next entry of the list, if any
          while (st.bits == 0u && st.w < n_words) {
            st.word0 = tile_word(0, st.w);
            st.word1 = tile_word(1, st.w);
            st.bits = st.word0 | st.word1;
            ++st.w;
          }
          st.more = st.bits != 0u;
        };
        auto load_next = [&](Stream& st, bool is_k) {
          const uint32_t low = st.bits & (0u - st.bits);
          st.bits &= ~low;
          const int v = 32 * (st.w - 1) + __ffs(low) - 1;
          const uint32_t n_last = st.jobs + (((st.word0 & low) && (st.word1 & low)) ? 1u : 0u);
          st.jobs = n_last + 1u;
          st.f3 = st.f2, st.f2 = st.f1;
          if (is_k) {
            st.f1 = n_last >= 1u ? n_last - 1u : 0u;
            load_tile(&map_k, st.slot, v);
            if (++st.slot == C::kKSlots) st.slot = 0;
          } else {
            st.f1 = n_last + 1u;
            load_tile(&map_v, C::kKSlots + st.slot, v);
            if (++st.slot == C::kVSlots) st.slot = 0;
          }
          ++st.e;
          advance(st);
        };
        Stream ks = {0, 0u, 0u, 0u, 0u, 0, 0, 0u, 0u, 0u, false}, vs = ks;
        advance(ks);
        advance(vs);
        uint32_t seen = 0;                 // commits 0 .. seen - 1 have completed
        while (alive && (ks.more || vs.more)) {
          bool progress = false;
          if (ks.more && (ks.e < C::kKSlots || ks.f3 < seen)) {
            load_next(ks, true);
            progress = true;
          }
          if (vs.more && (vs.e < C::kVSlots || (C::kVSlots == 2 ? vs.f2 : vs.f3) < seen)) {
            load_next(vs, false);
            progress = true;
          }
          if (!progress) {
            alive = mbar_wait(smem_u32(&ctl->kv_release[seen & 15u]), (seen >> 4) & 1u, abort_flag, status);
            ++seen;
          }
        }
#ifdef TRA_DEBUG
        if (lane == 0) ctl->dbg_jobs[3] = (int)ks.jobs - (ks.e == vs.e ? 0 : 1 << 20);     // both streams walked every entry
#endif
      }
    }
  } else if (warp == 9) {
    // ================================================================== MMA issuer
    {
      constexpr uint32_t kIdescQK = make_idesc(BN, false);
      constexpr uint32_t kIdescPV = make_idesc(D, true);
      bool alive = mbar_wait(smem_u32(&ctl->q_full), 0u, abort_flag, status);
      tc_fence_after();
      uint32_t pv_started = 0;            // bit k: tile k's accumulator holds at least one PV

      // descriptor words: K-major operands (Q, K) step 32 B per k-step inside a 64-column atom and
      // one atom (rows * 128 B) every four k-steps; the MN-major V operand steps 16 rows (2048 B)
      constexpr uint32_t kHi = desc_hi(1024);
      const uint32_t q_lo0 = desc_lo(smem_u32(sQ), 16), q_lo1 = desc_lo(smem_u32(sQ + C::kQTileBytes), 16);
      const uint32_t k_lo0 = desc_lo(smem_u32(sKV), 16);
      const uint32_t v_lo0 = desc_lo(smem_u32(sKV), C::kKVAtomBytes);
      const uint32_t s_full_bar = smem_u32(&ctl->s_full[0][0]);       // [tile][buffer], 8 bytes apart

      auto issue_s = [&](int k, int kslot, int buf) {
        const uint32_t qa = k ? q_lo1 : q_lo0;
        const uint32_t ka = k_lo0 + (uint32_t)kslot * (C::kSlotBytes >> 4);
        const uint32_t d = tmem + buf * 128;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off_q = ((kk >> 2) * C::kQAtomBytes + (kk & 3) * 32) >> 4;
          const uint32_t off_k = ((kk >> 2) * C::kKVAtomBytes + (kk & 3) * 32) >> 4;
          tc_mma_ss(d, qa + off_q, kHi, ka + off_k, kHi, kIdescQK, kk > 0 ? 1u : 0u);
        }
      };
      // PV in 64-key halves: the first half starts as soon as the softmax has stored the first 32
      // packed columns of P
      const uint32_t p_ready_bar = smem_u32(&ctl->p_ready[0][0]);     // [buffer][half], 8 bytes apart
      auto issue_pv = [&](int k, int vslot, int buf, uint32_t parity) -> bool {
        const uint32_t va = v_lo0 + (uint32_t)vslot * (C::kSlotBytes >> 4);
        const uint32_t d = tmem + 256 + k * 128;
        const uint32_t pa = tmem + buf * 128;
        const uint32_t started = (pv_started >> k) & 1u;
#pragma unroll
        for (int half = 0; half < (BN + 63) / 64; ++half) {
          if (!mbar_wait(p_ready_bar + (buf * 2 + half) * 8, parity, abort_flag, status)) return false;
          tc_fence_after();
#pragma unroll
          for (int kk = half * 4; kk < half * 4 + 4 && kk < BN / 16; ++kk)
            tc_mma_ts(d, pa + kk * 8, va + kk * (2048 >> 4), kHi, kIdescPV, kk > 0 ? 1u : started);
        }
        pv_started |= 1u << k;
        return true;
      };

      if constexpr (kDense) {
        // ---- dense launches: every key block, for both tiles (tile 1 when it exists).  A tile keeps
        // its own score buffer; per key block the pipe sees PV_0(e), S_0(e+1), PV_1(e), S_1(e+1).
        int slot = 0;
        uint32_t phase = 0;
        auto advance = [&]() {
          if (++slot == C::kSlots) {
            slot = 0;
            phase ^= 1u;
          }
        };
        uint32_t parity[2] = {0u, 0u};
        bool have = alive && NB > 0;
        if (have) {
          alive = mbar_wait(smem_u32(&ctl->kv_full[slot]), phase, abort_flag, status);   // first K tile
          if (alive) {
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < 2; ++k)
              if (k == 0 || tile1_on) {
                issue_s(k, slot, k);
                tc_commit(s_full_bar + (k * 2 + k) * 8);
              }
            tc_commit(smem_u32(&ctl->kv_release[0]));        // release event 0: K0
            advance();
          }
        }
        uint32_t n_release = 1;
        for (int e = 0; have && alive; ++e) {
          const int vslot = slot;
          const uint32_t vphase = phase;
          advance();
          const int kslot = slot;
          const uint32_t kphase = phase;
          const bool have_next = e + 1 < NB;
          bool v_ready = false, k_ready = false;
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            if (!alive || (k == 1 && !tile1_on)) continue;
            if (!v_ready) {
              alive = mbar_wait(smem_u32(&ctl->kv_full[vslot]), vphase, abort_flag, status);
              v_ready = true;
            }
            if (alive) alive = issue_pv(k, vslot, k, parity[k]);
            if (!alive) break;
            parity[k] ^= 1u;
            if (have_next) {
              if (!k_ready) {
                alive = mbar_wait(smem_u32(&ctl->kv_full[kslot]), kphase, abort_flag, status);
                k_ready = true;
                if (!alive) break;
                tc_fence_after();
              }
              issue_s(k, kslot, k);
              tc_commit(s_full_bar + (k * 2 + k) * 8);
            }
          }
          if (!alive) break;
          tc_commit(smem_u32(&ctl->kv_release[n_release & 7u]));   // V of this block and K of the next
          ++n_release;
          if (have_next) advance();
          have = have_next;
        }
      } else {
        // ---- the job stream: (list entry, tile) pairs in list order, tile 0 before tile 1 -----------
        int w = 0;
        uint32_t bits0 = 0, bits1 = 0;      // remaining bits of the current word, per tile
        auto next_entry = [&](bool& h0, bool& h1) -> bool {
          while (true) {
            const uint32_t u = bits0 | bits1;
            if (u) {
              const uint32_t low = u & (0u - u);
              h0 = (bits0 & low) != 0;
              h1 = (bits1 & low) != 0;
              bits0 &= ~low;
              bits1 &= ~low;
              return true;
            }
            if (w >= n_words) return false;
            bits0 = tile_word(0, w);
            bits1 = tile_word(1, w);
            ++w;
          }
        };
        // a job as flag bits
        constexpr uint32_t kJobValid = 1u, kJobTile1 = 2u, kJobFirst = 4u;    // kJobFirst: the first job of its entry
        bool pending1 = false;              // tile 1's job of the current entry is still to come
        auto next_job = [&]() -> uint32_t {
          if (pending1) {
            pending1 = false;
            return kJobValid | kJobTile1;
          }
          bool h0 = false, h1 = false;
          if (!next_entry(h0, h1)) return 0u;
          pending1 = h0 && h1;
          return kJobValid | kJobFirst | (h0 ? 0u : kJobTile1);
        };
        // Ring positions: K tiles cycle through slots 0 .. kKSlots - 1, V tiles through the slots behind
        // them, one step per list entry (see the TMA producer).
        struct Cursor {
          int slot;
          uint32_t phase;
        };
        Cursor kc = {C::kKSlots - 1, 1u};   // K tile of the entry whose scores were issued last (none yet)
        Cursor vc = {C::kVSlots - 1, 1u};   // V tile of the entry whose PV is being issued (none yet)
        auto wait_k = [&](uint32_t job) -> bool {     // scores of `job` come next: its K tile must have landed
          if (!(job & kJobFirst)) return true;        // the entry's first job already waited
          if (++kc.slot == C::kKSlots) {
            kc.slot = 0;
            kc.phase ^= 1u;
          }
          if (!mbar_wait(smem_u32(&ctl->kv_full[kc.slot]), kc.phase, abort_flag, status)) return false;
          tc_fence_after();
          return true;
        };

        // prologue: the scores of jobs 0 and 1, then commit 0 of the release sequence
        uint32_t cur = next_job();
        uint32_t nxt = cur ? next_job() : 0u;
        if (alive && cur) {
          alive = wait_k(cur);
          if (alive) {
            issue_s((cur & kJobTile1) ? 1 : 0, kc.slot, 0);
            tc_commit(s_full_bar + (((cur & kJobTile1) ? 2 : 0) + 0) * 8);
          }
          if (alive && nxt) {
            alive = wait_k(nxt);
            if (alive) {
              issue_s((nxt & kJobTile1) ? 1 : 0, kc.slot, 1);
              tc_commit(s_full_bar + (((nxt & kJobTile1) ? 2 : 0) + 1) * 8);
            }
          }
          if (alive) tc_commit(smem_u32(&ctl->kv_release[0]));
        }
        // group n: PV of job n, then the scores of job n + 2 into the buffer that PV just read.  What
        // the group needs from the ring is waited for first, so that nothing but the MMAs sits between
        // "P is announced" and "the next scores are issued".
        for (uint32_t n = 0; alive && cur; ++n) {
          const uint32_t ahead = nxt ? next_job() : 0u;
          const int buf = (int)(n & 1u);
          const int tile = (cur & kJobTile1) ? 1 : 0;
          if (cur & kJobFirst) {
            if (++vc.slot == C::kVSlots) {
              vc.slot = 0;
              vc.phase ^= 1u;
            }
            alive = mbar_wait(smem_u32(&ctl->kv_full[C::kKSlots + vc.slot]), vc.phase, abort_flag, status);
          }
          if (alive && ahead) alive = wait_k(ahead);
          if (alive) alive = issue_pv(tile, C::kKSlots + vc.slot, buf, (n >> 1) & 1u);
          if (!alive) break;
          // the next job belongs to the same tile: its softmax already holds scores issued ahead of
          // this PV, so it learns from this commit that the accumulator may be rescaled
          if (nxt && ((nxt ^ cur) & kJobTile1) == 0u) tc_commit(smem_u32(&ctl->o_done[tile]));
          if (ahead) {
            const int atile = (ahead & kJobTile1) ? 1 : 0;
            issue_s(atile, kc.slot, buf);
            tc_commit(s_full_bar + (atile * 2 + buf) * 8);
          }
          tc_commit(smem_u32(&ctl->kv_release[(n + 1u) & 15u]));   // commit n + 1 of the release sequence
          cur = nxt;
          nxt = ahead;
#ifdef TRA_DEBUG
          if (lane == 0) ctl->dbg_jobs[2] = (int)n + 1;
#endif
        }
      }
      // make sure every MMA has retired before tensor memory is released
      tc_commit(smem_u32(&ctl->drain));
      mbar_wait(smem_u32(&ctl->drain), 0u, abort_flag, status);
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    // ================================================================== softmax + epilogue
    const int k = warp >> 2;                         // query tile
    const int r = tid & (kTileM - 1);                // row inside the tile
    const int row = tile_index(k) * tile_rows + r;               // meaningless for a missing tile (index -1)
    const bool row_valid = tile_index(k) >= 0 && r < tile_rows && row < N;
    const int g_own = k * C::kGroups + min(r / blk, C::kGroups - 1);
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t t_o = tmem + lane_base + 256 + k * 128;

    float m = -INFINITY, l = 0.f, a = 0.f;
    float l_exact = 0.f;          // unrounded row sum (kExact: entropy, or lse requested)
    // token mask: this query's coordinate and its row of the threshold table (video queries only)
    bool tm_row = false;
    int qx = 0, qy = 0, qt = 0;
    const int32_t* th_row = nullptr;
    if (kTokenMask && row_valid && row < tm.n_video) {
      const uint32_t c = tm.coord_packed[row];
      qx = tra_coord_x(c);
      qy = tra_coord_y(c);
      qt = tra_coord_t(c);
      th_row = tm.theta + min((int)tm.ridx[(size_t)bh * N + row], tm.n_radii - 1) * tm.T;
      tm_row = true;
    }
    uint32_t n = 0;               // key blocks this tile has processed
    uint32_t job_prev = 0;        // job number of this tile's previous key block
    uint32_t jobs_before = 0;     // jobs of both tiles in the words already walked
    uint32_t s_seen = 0;            // bit b: parity of the completions of s_full[k][b] this thread has waited for
    uint32_t o_seen = 0;            // completions of o_done[k] this thread has waited for
    bool alive = true;

    const int n_dense = (k == 0 || tile1_on) ? NB : 0;
    for (int w = 0; w < n_outer && alive; ++w) {
      uint32_t bits = kDense ? 0u : tile_word(k, w);
      const uint32_t word0 = kDense ? 0u : tile_word(0, w);
      const uint32_t word1 = kDense ? 0u : tile_word(1, w);
      const uint32_t own_bits = kDense ? 0u : ctl->bitmap[g_own][w];
      int v_dense = 0;
      while (kDense ? v_dense < n_dense : bits != 0u) {
        int v;
        uint32_t buf;            // score buffer: a dense tile keeps its own, a sparse job takes job & 1
        bool chained = false;    // sparse: this tile also owned the previous job of the stream
        bool active = true;      // a tile that is one query block retains every block of its list
        if (kDense) {
          v = v_dense++;
          buf = (uint32_t)k;
        } else {
          const uint32_t low = bits & (0u - bits);
          bits &= ~low;
          v = 32 * w + __ffs(low) - 1;
          const uint32_t job = jobs_before + __popc(word0 & (low - 1u)) + __popc(word1 & (low - 1u)) +
                               ((k == 1 && (word0 & low)) ? 1u : 0u);
          buf = job & 1u;
          chained = n > 0 && job_prev + 1u == job;
          job_prev = job;
          if (C::kGroups > 1) active = (own_bits & low) != 0;
        }
        // rows of the tile past its query blocks (kAny) hold no query: no exponentials for them (a warp made of such
        // rows only keeps up with the barriers and writes zeros)
        if (kAny && r >= tile_rows) active = false;
        const int col_limit = min(blk, N - v * blk);
        const uint32_t t_s = tmem + lane_base + buf * 128;

        if (!mbar_wait_warp(smem_u32(&ctl->s_full[k][buf]), (s_seen >> buf) & 1u, abort_flag, status)) {
          alive = false;
          break;
        }
        s_seen ^= 1u << buf;
        tc_fence_after();

        // the whole S row of this thread, straight into registers (one load latency)
        uint32_t sb[C::kCols];
#pragma unroll
        for (int c = 0; c < C::kChunks; ++c) tmem_ld32(t_s + c * 32, &sb[c * 32]);
        tmem_wait_ld(&sb[0]);
#pragma unroll
        for (int c = 1; c < C::kChunks; ++c) reg_fence32(&sb[c * 32]);

        // Columns >= col_limit do not exist: the ragged last key block, and with kAny the tail of every key tile
        // (rows of the next block, and tensor-memory columns past BN that no MMA wrote).  Only the last 16
        // columns of the tile, and those past BN, can be concerned unless the block is the ragged last one.
        if (col_limit < C::kCols) {
          if (col_limit > BN - 16) {        // the usual case with kAny: the block ends in the last 16 rows of the tile
#pragma unroll
            for (int j = BN - 16; j < BN; ++j)
              if (j >= col_limit) sb[j] = __float_as_uint(-1e30f);
#pragma unroll
            for (int j = BN; j < C::kCols; ++j) sb[j] = __float_as_uint(-1e30f);
          } else {
#pragma unroll
            for (int j = 0; j < C::kCols; ++j)
              if (j >= col_limit) sb[j] = __float_as_uint(-1e30f);
          }
        }
        if (kTokenMask && tm_row && active && v * BN < tm.n_video) {
          // keys outside this query's disk at their frame distance do not exist for it (Eq. 15);
          // text keys (index >= n_video) stay visible
          const int k0 = v * BN;
          const int kt0 = tra_coord_t(tm.coord_packed[k0]);
          const int th0 = __ldg(th_row + abs(qt - kt0));
          const int th1 = kt0 + 1 < tm.T ? __ldg(th_row + abs(qt - kt0 - 1)) : th0;
          const uint4* kc4 = reinterpret_cast<const uint4*>(tm.coord_packed + k0);
          const bool one_frame = k0 + BN <= tm.n_video && tra_coord_t(tm.coord_packed[k0 + BN - 1]) == kt0;
          // 16-key slices of the block; the usual case: each is 16 consecutive x of one frame row
          const uint4 sa = __ldg(reinterpret_cast<const uint4*>(tm.slice + (k0 >> 4)));
          const uint4 sb4 = BN > 64 ? __ldg(reinterpret_cast<const uint4*>(tm.slice + (k0 >> 4)) + 1) : sa;
          auto slice_word = [&](int q) -> uint32_t {     // q is a compile-time constant at every use
            const uint4& w4 = q < 4 ? sa : sb4;
            return (q & 3) == 0 ? w4.x : ((q & 3) == 1 ? w4.y : ((q & 3) == 2 ? w4.z : w4.w));
          };
          const uint32_t all_runs = sa.x & sa.y & sa.z & sa.w & sb4.x & sb4.y & sb4.z & sb4.w;
          if (all_runs & (1u << 30)) {
            // A key (x0 + j, ys) is inside the disk iff |x0 + j - qx| <= w with
            // w = floor(sqrt(theta - (ys - qy)^2)): one square root per slice gives the interval of
            // inside keys, 0 <= j + (x0 - qx + w) <= 2 w, as a word of flags; one test per key.
#pragma unroll
            for (int q = 0; q < BN / 16; ++q) {
              const uint32_t sw = slice_word(q);
              const int ts = (int)((sw >> 20) & 1023u), dts = ts - kt0;
              const int th = dts == 0 ? th0
                             : (dts == 1 ? th1 : (TRA_IDX(abs(qt - ts), tm.T, status) ? __ldg(th_row + abs(qt - ts)) : 0));
              const int dy = tra_coord_y(sw) - qy;
              const int rem = th - dy * dy;
              const int w = tra_isqrt_small_nocvt(max(rem, 0));
              // keys j with 0 <= j + bs <= 2 w are inside: one 16-bit word of "inside" flags per slice
              const int bs = w + tra_coord_x(sw) - qx;
              const int lo = max(-bs, 0), hi = min(2 * w - bs, 15);
              const uint32_t inside = (rem >= 0 && hi >= lo) ? ((0xFFFFu >> (15 - hi)) & (0xFFFFu << lo)) : 0u;
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (((inside >> j) & 1u) == 0u) sb[q * 16 + j] = __float_as_uint(-1e30f);
            }
          } else if (one_frame) {       // every key of the block in one frame, some slice not a row run
#pragma unroll
            for (int j4 = 0; j4 < BN / 4; ++j4) {
              const uint4 c4 = __ldg(kc4 + j4);
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                const uint32_t kc = q4 == 0 ? c4.x : (q4 == 1 ? c4.y : (q4 == 2 ? c4.z : c4.w));
                const int dx = qx - tra_coord_x(kc), dy = qy - tra_coord_y(kc);
                if (dx * dx + dy * dy > th0) sb[j4 * 4 + q4] = __float_as_uint(-1e30f);
              }
            }
          } else {
#pragma unroll
            for (int j4 = 0; j4 < BN / 4; ++j4) {
              const uint4 c4 = __ldg(kc4 + j4);
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                const int j = j4 * 4 + q4;
                const uint32_t kc = q4 == 0 ? c4.x : (q4 == 1 ? c4.y : (q4 == 2 ? c4.z : c4.w));
                const int dt = tra_coord_t(kc) - kt0;
                const int th = dt == 0 ? th0
                               : (dt == 1 ? th1
                                          : (TRA_IDX(abs(qt - kt0 - dt), tm.T, status) ? __ldg(th_row + abs(qt - kt0 - dt)) : 0));
                const int dx = qx - tra_coord_x(kc), dy = qy - tra_coord_y(kc);
                if (k0 + j < tm.n_video && dx * dx + dy * dy > th) sb[j] = __float_as_uint(-1e30f);
              }
            }
          }
        }
        float alpha = 1.f;
        bool row_on = active;         // false also when the token mask leaves this row nothing here
        if (active) {
          float mx0 = __uint_as_float(sb[0]), mx1 = __uint_as_float(sb[1]);
#pragma unroll
          for (int j = 2; j + 3 < C::kCols; j += 4) {
            mx0 = fmax3(mx0, __uint_as_float(sb[j]), __uint_as_float(sb[j + 1]));
            mx1 = fmax3(mx1, __uint_as_float(sb[j + 2]), __uint_as_float(sb[j + 3]));
          }
          mx0 = fmax3(mx0, __uint_as_float(sb[C::kCols - 2]), __uint_as_float(sb[C::kCols - 1]));
          const float mx = fmaxf(mx0, mx1);
          if (kTokenMask) row_on = mx > -1e29f;
          const float m_blk = mx * scale_log2;
          if (row_on && m_blk > m + kRescaleThreshold) {   // also the first block (m = -inf)
            alpha = ex2(m - m_blk);                   // 0 when m = -inf
            a = l_exact > 0.f ? alpha * (a + (m - m_blk) * l_exact) : 0.f;
            l *= alpha;
            l_exact *= alpha;
            m = m_blk;
          }
        }
        // A chained job's scores were issued ahead of the previous PV of this tile (job - 1); the MMA
        // warp commits o_done when that PV retires.  Every such commit is waited for exactly once,
        // here: the row maximum above has hidden most of its latency, and the accumulator may be
        // rescaled below.  (A PV of a job <= job - 2 was issued ahead of the S just read, on the same
        // in-order pipe, and the commit that announced S covers every earlier MMA.)
        if (!kDense && chained) {
          if (!mbar_wait_warp(smem_u32(&ctl->o_done[k]), o_seen & 1u, abort_flag, status)) {
            alive = false;
            break;
          }
          ++o_seen;
          tc_fence_after();
        }
        // rescale the O accumulator when some row of this warp raised its reference maximum
        const bool warp_rescale = __any_sync(0xffffffffu, alpha != 1.f) && n > 0;
        if (warp_rescale) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(t_o + c * 32, o);
            tmem_wait_ld(o);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
            tmem_st32(t_o + c * 32, o);
          }
        }
        // probabilities (relative to m), row sum and entropy accumulator; P goes back to tensor
        // memory 32 keys at a time, and each 64-key half is announced to the MMA issuer on its own
        {
          const float neg_m = row_on ? -m : 0.f;
          const uint64_t scale2 = pack2(scale_log2, scale_log2), neg_m2 = pack2(neg_m, neg_m);
          // Row sum of the rounded probabilities, even and odd keys apart.  Launches without entropy add
          // the bf16 halves of a packed pair with the mixed-precision add (two instructions per pair);
          // the fused-entropy launch, whose FMA pipe is busier, unpacks with a shift and a mask and adds
          // the pair at once (measured: -4 % time for the former, +1 % for the latter if swapped).
          uint64_t l2 = 0ull;
          float l_lo = 0.f, l_hi = 0.f;
          uint64_t a2 = 0ull, e2 = 0ull;                 // pairs of partial sums
#pragma unroll
          for (int c = 0; c < C::kChunks; ++c) {
            uint32_t pk[16];
            if (active) {
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const uint64_t t2 = ffma2(pack2(__uint_as_float(sb[c * 32 + j]), __uint_as_float(sb[c * 32 + j + 1])),
                                          scale2, neg_m2);
                float t0, t1, x0, x1;
                unpack2(t2, t0, t1);
                x0 = ex2(t0);
                x1 = ex2(t1);
                // the row sum that normalises O uses the bf16-rounded probabilities the PV MMA
                // consumes, so numerator and denominator of O = (sum p v) / (sum p) agree
                const uint32_t packed = pack_bf16(x0, x1);
                if (kEntropy)
                  l2 = fadd2(l2, pack2(__uint_as_float(packed << 16), __uint_as_float(packed & 0xffff0000u)));
                else
                  add_bf16_pair(l_lo, l_hi, packed);
                if (kExact) {                 // entropy and lse from the unrounded terms
                  const uint64_t x2 = pack2(x0, x1);
                  e2 = fadd2(e2, x2);
                  if (kEntropy) a2 = ffma2(x2, t2, a2);
                }
                pk[j >> 1] = packed;
              }
            } else {                          // this row's query block does not retain the key block
#pragma unroll
              for (int j = 0; j < 16; ++j) pk[j] = 0u;
            }
            tmem_st16(t_s + c * 16, pk);
            if ((c & 1) || c == C::kChunks - 1) {   // a 64-key half of P (the last may be shorter) is complete
              tmem_wait_st();
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&ctl->p_ready[buf][c >> 1]));
            }
          }
          float lo, hi;
          if (kEntropy) unpack2(l2, l_lo, l_hi);
          l += l_lo + l_hi;
          if (kEntropy) {
            unpack2(a2, lo, hi);
            a += lo + hi;
          }
          if (kExact) {
            unpack2(e2, lo, hi);
            l_exact += lo + hi;
          }
        }
        ++n;
      }
      jobs_before += __popc(word0) + __popc(word1);
    }

#ifdef TRA_DEBUG
    if (r == 0) ctl->dbg_jobs[k] = (int)n;
#endif
    // ---- epilogue: O = o / l, entropy, lse ------------------------------------------------
    // the MMA warp commits `drain` behind its last MMA: every PV of both tiles has retired then
    if (alive && n > 0)
      alive = mbar_wait_warp(smem_u32(&ctl->drain), 0u, abort_flag, status);
    if (alive) {
      tc_fence_after();
      const float inv_l = l > 0.f ? 1.f / l : 0.f;
      // the output row: the query's own position, or its raster row when the tensors are in raster order
      const int out_row = !row_valid ? 0 : (slice_raster ? __ldg(slice_raster + (row >> 4)) + (row & 15) : row);
      __nv_bfloat16* orow = O + ((size_t)bh * N + out_row) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o_bits[32];
        float o[32];
        if (n > 0) {
          tmem_ld32(t_o + c * 32, o_bits);
          tmem_wait_ld(o_bits);
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(o_bits[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) o[j] = 0.f;
        }
        if (row_valid) {
          uint4* dst = (uint4*)(orow + c * 32);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 val;
            val.x = pack_bf16(o[q4 * 8 + 0] * inv_l, o[q4 * 8 + 1] * inv_l);
            val.y = pack_bf16(o[q4 * 8 + 2] * inv_l, o[q4 * 8 + 3] * inv_l);
            val.z = pack_bf16(o[q4 * 8 + 4] * inv_l, o[q4 * 8 + 5] * inv_l);
            val.w = pack_bf16(o[q4 * 8 + 6] * inv_l, o[q4 * 8 + 7] * inv_l);
            dst[q4] = val;
          }
        }
      }
      if (row_valid) {
        const size_t idx = (size_t)bh * N + row;
        const float l_out = kExact ? l_exact : l;
        if (kEntropy && entropy) entropy[idx] = l_out > 0.f ? logf(l_out) - kLn2 * a / l_out : 0.f;
        if (lse) lse[idx] = l_out > 0.f ? (m + log2f(l_out)) * kLn2 : -INFINITY;
      }
    }
  }

  // ---- teardown ------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
#ifdef TRA_DEBUG      // every role walked the same job stream (block-sparse launches)
  if (!kDense && tid == 0 && !ctl->abort_flag &&
      (ctl->dbg_jobs[0] + ctl->dbg_jobs[1] != ctl->dbg_jobs[2] || ctl->dbg_jobs[3] != ctl->dbg_jobs[2]))
    tra_set_status(status, TRA_ERR_BOUNDS);
#endif
  if (warp == 9) {
    if (ctl->abort_flag) {
      // let copies and MMAs that were in flight when the CTA gave up land before releasing
      const unsigned long long t0 = globaltimer_ns();
      while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ------------------------------------------------------------------------------------ host
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                    const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                    const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_tiled() {
  static encode_tiled_fn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (encode_tiled_fn)p;
  }
  return fn;
}

// [B*heads, N, d] bf16 viewed as a 3-D tensor (d innermost); box = 64 columns x `rows` tokens.
int make_map(CUtensorMap* map, const void* base, int d, int N, long long BH, int rows) {
  encode_tiled_fn enc = get_encode_tiled();
  if (!enc) return TRA_ERR_CUDA;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * (cuuint64_t)N};
  cuuint32_t box[3] = {64u, (cuuint32_t)rows, 1u};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? TRA_OK : TRA_ERR_CUDA;
}

template <int D, int BN, bool kEntropy, bool kTokenMask, bool kDense, bool kLse, bool kAny = false>
int launch(const tra_attn_args& a) {
  using C = Cfg<D, BN>;
  const tra_plan_t* plan = a.plan;
  CUtensorMap mq, mk, mv;
  int rc;
  const bool raster_kv = (plan->cfg.flags & TRA_ORDER_RASTER) != 0;
  const int32_t* slice_raster = (plan->cfg.flags & (TRA_ORDER_RASTER | TRA_ORDER_RASTER_QO)) ? plan->d_slice_raster
                                                                                              : nullptr;
  // boxes: a whole tile per 64-column atom, or (raster order) one 16-token run
  if ((rc = make_map(&mq, a.Q, D, plan->S, a.BH, slice_raster ? 16 : kTileM)) != TRA_OK) return rc;
  if ((rc = make_map(&mk, a.K, D, plan->S, a.BH, raster_kv ? 16 : BN)) != TRA_OK) return rc;
  if ((rc = make_map(&mv, a.V, D, plan->S, a.BH, raster_kv ? 16 : BN)) != TRA_OK) return rc;
  auto kern = tra_attn_kernel<D, BN, kEntropy, kTokenMask, kDense, kLse, kAny>;
  TokenMaskArgs tm = {plan->d_boxes, plan->d_slice, plan->d_coord_packed, plan->d_theta, a.ridx,
                      plan->N,       plan->cfg.T,   plan->n_radii};
  TRA_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
  const int tile_rows = C::kGroups * (kAny ? plan->cfg.block : BN);      // query rows a tile really holds
  const int n_pairs = ((plan->S + tile_rows - 1) / tile_rows + 1) / 2;
  dim3 grid((unsigned)n_pairs, (unsigned)a.BH);
  kern<<<grid, kThreads, C::kSmemBytes, a.stream>>>(mq, mk, mv, (__nv_bfloat16*)a.O, a.entropy, a.lse, a.row_ptr,
                                                    a.col_idx, a.tile_pairs, plan->S, plan->NB,
                                                    a.sm_scale * kLog2e, plan->d_status, tm, plan->cfg.block,
                                                    slice_raster, raster_kv ? 1 : 0);
  TRA_CUDA_CHECK(cudaGetLastError());
  return TRA_OK;
}

// The launch variants of one (head_dim, block) shape: entropy launches are dense, token-mask
// launches block-sparse (or list-free), a plain launch is either; lse without entropy selects the
// instantiation that also accumulates the unrounded row sum.
template <int D, int BN>
int launch_shape(const tra_attn_args& a) {
  const bool want_lse = a.lse != nullptr;
  if (a.entropy != nullptr) return launch<D, BN, true, false, true, false>(a);
  if (a.ridx != nullptr)
    return want_lse ? launch<D, BN, false, true, false, true>(a) : launch<D, BN, false, true, false, false>(a);
  if (a.row_ptr == nullptr)
    return want_lse ? launch<D, BN, false, false, true, true>(a) : launch<D, BN, false, false, true, false>(a);
  return want_lse ? launch<D, BN, false, false, false, true>(a) : launch<D, BN, false, false, false, false>(a);
}

// Blocks of any size in (BN - 16, BN] (the paper's 40 .. 120-token blocks): dense and block-sparse launches; the
// token mask inside blocks needs whole 16-key slices and is refused.
template <int D, int BN>
int launch_shape_any(const tra_attn_args& a) {
  const bool want_lse = a.lse != nullptr;
  if (a.ridx != nullptr) return TRA_ERR_UNSUPPORTED;
  if (a.entropy != nullptr) return launch<D, BN, true, false, true, false, true>(a);
  if (a.row_ptr == nullptr)
    return want_lse ? launch<D, BN, false, false, true, true, true>(a) : launch<D, BN, false, false, true, false, true>(a);
  return want_lse ? launch<D, BN, false, false, false, true, true>(a) : launch<D, BN, false, false, false, false, true>(a);
}

}  // namespace
