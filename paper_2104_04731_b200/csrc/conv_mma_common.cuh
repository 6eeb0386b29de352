// Device-side building blocks shared by the convolution kernels: bounded mbarrier waits, TMA
// loads, shared-memory and instruction descriptors of tcgen05.mma.kind::i8, tensor-memory loads and
// the fused epilogue (activation step, shift / clip, NKPQ / NPQK stores; Section 5.1's vector unit).
// Included by each kernel translation unit; everything lives in an unnamed namespace.
#pragma once

#include "b2c_internal.h"

namespace b2c {

namespace {

constexpr int kGatherWarps = 8;                    // warps 2..9: operand-A gather, then epilogue
constexpr int kThreads = 64 + 32 * kGatherWarps;  // + warp 0 (TMA producer) and warp 1 (MMA issuer)
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait

struct __align__(8) SharedCtl {
  unsigned long long full[8];
  unsigned long long empty[8];
  unsigned long long tmem_full[4];   // accumulator buffer b complete (MMA warp -> epilogue warps)
  unsigned long long tmem_empty[4];  // accumulator buffer b drained (epilogue warps -> MMA warp)
  uint32_t tmem_base;
  volatile int abort_flag;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// The issue helpers below take `on`: the instruction is predicated on it instead of sitting in a
// divergent branch, so the surrounding loop stays straight-line, warp-uniform code.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %2, 0;\n"
      "@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n}" ::"r"(bar),
      "r"(bytes), "r"(on)
      : "memory");
}
// Non-blocking phase test (never suspends the thread).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// One lane of a converged warp.  Loops of the single-thread roles (TMA issue, MMA issue) are run
// by the whole warp with only the issuing instructions predicated on this lane, so that loop
// counters, barrier addresses and descriptors stay warp-uniform.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n.reg .pred p;\n"
      "elect.sync _|p, 0xffffffff;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait.  Returns false when the block is aborting (this wait or another one expired).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status) {
  const unsigned long long t0 = global_ns();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (ctl->abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      ctl->abort_flag = 1;
      atomicCAS(status, 0, B2C_E_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status) {
#pragma unroll 1
  for (int i = 0; i < 32; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, ctl, status);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                            uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %5, 0;\n"
      "@q cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n}" ::
          "r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(bar), "r"(on)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                   uint32_t bar, uint16_t off_w, uint16_t off_h, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %9, 0;\n"
      "@q cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, "
      "%5}], [%6], {%7, %8};\n}" ::"r"(dst),
      "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(off_w), "h"(off_h), "r"(on)
      : "memory");
}

__device__ __forceinline__ void tma_load_tiled_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                  uint32_t bar, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %7, 0;\n"
      "@q cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], "
      "[%6];\n}" ::"r"(dst),
      "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "r"(on)
      : "memory");
}

// Shared-memory operand descriptor for a K-major tile whose rows are `bk` bytes long and stored
// with the matching 32/64/128-byte swizzle: start address (16-byte units), leading-dimension
// offset unused for swizzled K-major layouts (set to 1), stride between 8-row groups = 8 * bk
// bytes, descriptor version 1, swizzle code in the top three bits.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, int bk) {
  const uint64_t swz = bk == 128 ? 2ull : (bk == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)((8 * bk) >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= swz << 61;
  return d;
}

// A tile may also start at any row of a buffer that TMA filled with the pattern anchored at its
// natural boundary (1024 / 512 / 256 bytes for the 128 / 64 / 32-byte swizzle): the swizzle is a
// function of the shared-memory address bits, applied after the row and chunk offsets have been
// added to the start address, so the same descriptor (base offset 0) with a start address moved by
// whole rows reads the rows further on.  The shift execution relies on this; its parity tests
// cover all three swizzle widths.

// Instruction descriptor for kind::i8: D = s32 (code 2 at bit 4), A = B = signed 8-bit (code 1
// at bits 7 and 10), both operands K-major (no transpose bits), N/8 at bit 17, M/16 at bit 24.
__device__ __forceinline__ uint32_t make_idesc_i8(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

// One reduction block: `ksteps` (1..4) MMAs over consecutive 32-byte slices of the stage (each
// step advances both descriptors by 2 units of 16 bytes).  Issued from one asm block so that the
// predicates and descriptors are formed once and the instructions go out back to back; the first
// step overwrites the accumulator when `accumulate` is 0, the others always add.
__device__ __forceinline__ void mma_i8_block(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t on, int ksteps) {
  asm volatile(
      "{\n"
      ".reg .pred pacc, ptrue, q0, q1, q2, q3;\n"
      ".reg .b64 a1, a2, a3, b1, b2, b3;\n"
      "setp.ne.b32 pacc, %4, 0;\n"
      "setp.eq.b32 ptrue, 0, 0;\n"
      "setp.ne.b32 q0, %5, 0;\n"
      "setp.gt.and.s32 q1, %6, 1, q0;\n"
      "setp.gt.and.s32 q2, %6, 2, q0;\n"
      "setp.gt.and.s32 q3, %6, 3, q0;\n"
      "add.u64 a1, %1, 2;\n"
      "add.u64 b1, %2, 2;\n"
      "add.u64 a2, %1, 4;\n"
      "add.u64 b2, %2, 4;\n"
      "add.u64 a3, %1, 6;\n"
      "add.u64 b3, %2, 6;\n"
      "@q0 tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, pacc;\n"
      "@q1 tcgen05.mma.cta_group::1.kind::i8 [%0], a1, b1, %3, ptrue;\n"
      "@q2 tcgen05.mma.cta_group::1.kind::i8 [%0], a2, b2, %3, ptrue;\n"
      "@q3 tcgen05.mma.cta_group::1.kind::i8 [%0], a3, b3, %3, ptrue;\n"
      "}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(on), "r"(ksteps)
      : "memory");
}
// Up to four MMAs whose descriptors advance by constant steps (one 32-byte slice per tap: the A
// descriptor moves by the tap's pixel shift, the B descriptor to the next resident weight tile).
// One asm block, so that predicates and descriptors are formed once and the instructions go out
// back to back.
__device__ __forceinline__ void mma_i8_run4(uint32_t d_tmem, uint64_t adesc, uint64_t a_step, uint64_t bdesc,
                                            uint64_t b_step, uint32_t idesc, uint32_t accumulate, uint32_t on,
                                            int count) {
  asm volatile(
      "{\n"
      ".reg .pred pacc, ptrue, q0, q1, q2, q3;\n"
      ".reg .b64 a1, a2, a3, b1, b2, b3;\n"
      "setp.ne.b32 pacc, %6, 0;\n"
      "setp.eq.b32 ptrue, 0, 0;\n"
      "setp.ne.b32 q0, %7, 0;\n"
      "setp.gt.and.s32 q1, %8, 1, q0;\n"
      "setp.gt.and.s32 q2, %8, 2, q0;\n"
      "setp.gt.and.s32 q3, %8, 3, q0;\n"
      "add.u64 a1, %1, %2;\n"
      "add.u64 b1, %3, %4;\n"
      "add.u64 a2, a1, %2;\n"
      "add.u64 b2, b1, %4;\n"
      "add.u64 a3, a2, %2;\n"
      "add.u64 b3, b2, %4;\n"
      "@q0 tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %3, %5, pacc;\n"
      "@q1 tcgen05.mma.cta_group::1.kind::i8 [%0], a1, b1, %5, ptrue;\n"
      "@q2 tcgen05.mma.cta_group::1.kind::i8 [%0], a2, b2, %5, ptrue;\n"
      "@q3 tcgen05.mma.cta_group::1.kind::i8 [%0], a3, b3, %5, ptrue;\n"
      "}" ::"r"(d_tmem),
      "l"(adesc), "l"(a_step), "l"(bdesc), "l"(b_step), "r"(idesc), "r"(accumulate), "r"(on), "r"(count)
      : "memory");
}
// Two taps of a filter row with two 32-byte slices each (64-byte channel blocks): four MMAs in one
// asm block.  The second tap's descriptors lie a_step / b_step further on; `taps` is 1 or 2.
__device__ __forceinline__ void mma_i8_pair2(uint32_t d_tmem, uint64_t adesc, uint64_t a_step, uint64_t bdesc,
                                             uint64_t b_step, uint32_t idesc, uint32_t accumulate, uint32_t on,
                                             int taps) {
  asm volatile(
      "{\n"
      ".reg .pred pacc, ptrue, q0, q1;\n"
      ".reg .b64 a1, a2, a3, b1, b2, b3;\n"
      "setp.ne.b32 pacc, %6, 0;\n"
      "setp.eq.b32 ptrue, 0, 0;\n"
      "setp.ne.b32 q0, %7, 0;\n"
      "setp.gt.and.s32 q1, %8, 1, q0;\n"
      "add.u64 a1, %1, 2;\n"
      "add.u64 b1, %3, 2;\n"
      "add.u64 a2, %1, %2;\n"
      "add.u64 b2, %3, %4;\n"
      "add.u64 a3, a2, 2;\n"
      "add.u64 b3, b2, 2;\n"
      "@q0 tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %3, %5, pacc;\n"
      "@q0 tcgen05.mma.cta_group::1.kind::i8 [%0], a1, b1, %5, ptrue;\n"
      "@q1 tcgen05.mma.cta_group::1.kind::i8 [%0], a2, b2, %5, ptrue;\n"
      "@q1 tcgen05.mma.cta_group::1.kind::i8 [%0], a3, b3, %5, ptrue;\n"
      "}" ::"r"(d_tmem),
      "l"(adesc), "l"(a_step), "l"(bdesc), "l"(b_step), "r"(idesc), "r"(accumulate), "r"(on), "r"(taps)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %1, 0;\n"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}" ::"r"(bar),
      "r"(on)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ int8_t requant(int v, int shift) { return (int8_t)max(-128, min(127, v >> shift)); }

// Activation step of Section 5.1's vector unit on a complete sum of output channel k: optional
// per-channel bias, optional ReLU.  (Partial sums of a split reduction are never passed here.)
__device__ __forceinline__ int activate(const ConvArgs& args, int v, int k) {
  if (args.bias != nullptr) v += __ldg(args.bias + k);
  if (args.relu) v = max(v, 0);
  return v;
}

// Loads NC consecutive accumulator columns of this thread's TMEM lane.
template <int NC>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, int32_t* v);
template <>
__device__ __forceinline__ void tmem_ld<16>(uint32_t taddr, int32_t* v) {
  tmem_ld16(taddr, v);
}
template <>
__device__ __forceinline__ void tmem_ld<32>(uint32_t taddr, int32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Epilogue for NC accumulator columns starting at output channel `kbase` of one output pixel
// (one thread = one accumulator row).  Section 5.1's quantisation step (shift, clip) is applied
// here, and the values go to the NKPQ or NPQK tensor; with a split reduction the partial sums
// are added into a zeroed int32 buffer instead.
template <int NC>
__device__ __forceinline__ void store_columns(const ConvArgs& args, int32_t* v, int kbase, bool row_valid,
                                              long long base_nkpq, long long base_npqk, int bias_off = 0) {
  const int K = args.K;
  if (!row_valid || kbase >= K) return;
  const bool nhwc = args.out_layout == B2C_LAYOUT_NHWC;
#ifdef B2C_DEBUG_BOUNDS
  {
    // first and last element this call can touch, in each tensor it writes
    const int cnt = min(NC, K - kbase);
    const long long first = nhwc ? base_npqk + kbase : base_nkpq + (long long)kbase * args.out_PQ;
    const long long last = nhwc ? first + cnt - 1 : first + (long long)(cnt - 1) * args.out_PQ;
    bool ok = true;
    if (args.split_k > 1 && !args.cluster_split) {
      ok = (args.acc == args.y32 ? B2C_O32_OK(args.dbg, 20, args.acc + first, 4) && B2C_O32_OK(args.dbg, 20, args.acc + last, 4)
                                 : B2C_WS_OK(args.dbg, 20, args.acc + first, 4) && B2C_WS_OK(args.dbg, 20, args.acc + last, 4));
    } else {
      if (args.out_mode & B2C_OUT_I32) ok = B2C_O32_OK(args.dbg, 21, args.y32 + first, 4) && B2C_O32_OK(args.dbg, 21, args.y32 + last, 4);
      if (ok && (args.out_mode & B2C_OUT_I8)) ok = B2C_O8_OK(args.dbg, 22, args.y8 + first, 1) && B2C_O8_OK(args.dbg, 22, args.y8 + last, 1);
    }
    if (!ok) return;
  }
#endif
  if (args.split_k > 1 && !args.cluster_split) {
    // Partial sums of the reduction slices meet in global memory; integer addition is
    // associative, so the order of arrival does not change the result.
    int32_t* dst = args.acc + (nhwc ? base_npqk + kbase : base_nkpq + (long long)kbase * args.out_PQ);
    const long long step = nhwc ? 1 : args.out_PQ;
#pragma unroll
    for (int j = 0; j < NC; ++j) {
      if (kbase + j < K) atomicAdd(dst, v[j]);
      dst += step;
    }
    return;
  }
  if (args.bias != nullptr || args.relu) {
#pragma unroll
    for (int j = 0; j < NC; ++j)
      if (kbase + j < K) v[j] = activate(args, v[j], bias_off + kbase + j);
  }
  if (!nhwc) {
    // NKPQ: for a fixed column the 32 lanes of a warp hold 32 consecutive pixels, so every
    // store instruction writes one contiguous run.
    const long long o = base_nkpq + (long long)kbase * args.out_PQ;
    if (kbase + NC <= K && (long long)NC * args.out_PQ < 0x7FFFFFFFLL) {
      // all NC channels exist: no per-column test, and every address is the base plus a 32-bit
      // offset, so the columns are independent instructions
      const int pq = args.out_PQ, shift = args.shift;
      if (args.out_mode & B2C_OUT_I32) {
        int32_t* dst = args.y32 + o;
#pragma unroll
        for (int j = 0; j < NC; ++j) dst[j * pq] = v[j];
      }
      if (args.out_mode & B2C_OUT_I8) {
        int8_t* dst = args.y8 + o;
#pragma unroll
        for (int j = 0; j < NC; ++j) {
          dst[j * pq] = requant(v[j], shift);
        }
      }
      return;
    }
    if (args.out_mode & B2C_OUT_I32) {
      int32_t* dst = args.y32 + o;
#pragma unroll
      for (int j = 0; j < NC; ++j) {
        if (kbase + j < K) *dst = v[j];
        dst += args.out_PQ;
      }
    }
    if (args.out_mode & B2C_OUT_I8) {
      int8_t* dst = args.y8 + o;
#pragma unroll
      for (int j = 0; j < NC; ++j) {
        if (kbase + j < K) *dst = requant(v[j], args.shift);
        dst += args.out_PQ;
      }
    }
  } else {
    // NPQK: a thread owns NC consecutive channels of one pixel: 16-byte vector stores.
    const bool full = kbase + NC <= K;
    if (args.out_mode & B2C_OUT_I32) {
      int32_t* dst = args.y32 + base_npqk + kbase;
      if (full && (K & 3) == 0) {
#pragma unroll
        for (int j = 0; j < NC; j += 4) *reinterpret_cast<int4*>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < NC; ++j)
          if (kbase + j < K) dst[j] = v[j];
      }
    }
    if (args.out_mode & B2C_OUT_I8) {
      int8_t* dst = args.y8 + base_npqk + kbase;
      if (full && (K & 15) == 0) {
#pragma unroll
        for (int g = 0; g < NC; g += 16) {
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            w[j] = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) w[j] |= (uint32_t)(uint8_t)requant(v[g + j * 4 + i], args.shift) << (8 * i);
          }
          *reinterpret_cast<uint4*>(dst + g) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < NC; ++j)
          if (kbase + j < K) dst[j] = requant(v[j], args.shift);
      }
    }
  }
}

// Swapped axis map: this thread's accumulator row is output channel k, and v holds 16 consecutive
// fused pixels m_first .. m_first + 15.  NPQK: for a fixed pixel the 32 lanes of a warp hold 32
// consecutive channels, so every store instruction writes one contiguous run.  NKPQ: the 16 pixels
// of a thread are contiguous while they stay inside one image, and go out as 16-byte vectors when
// the run is complete and aligned.
__device__ __forceinline__ void store_columns_swapped(const ConvArgs& args, int32_t* v, int k, bool row_valid,
                                                      int m_first) {
  if (!row_valid || m_first >= args.Mg) return;
  const int count = min(16, args.Mg - m_first);
#ifdef B2C_DEBUG_BOUNDS
  {
    // output elements of pixels m_first .. m_first + count - 1 in channel k, first and last
    const bool nh = args.out_layout == B2C_LAYOUT_NHWC;
    const int m_last = m_first + count - 1;
    const int n0_ = (int)args.div_pq.div((uint32_t)m_first), n1_ = (int)args.div_pq.div((uint32_t)m_last);
    const long long first = nh ? (long long)m_first * args.K + k : ((long long)n0_ * args.K + k) * args.PQ + (m_first - n0_ * args.PQ);
    const long long last = nh ? (long long)m_last * args.K + k : ((long long)n1_ * args.K + k) * args.PQ + (m_last - n1_ * args.PQ);
    bool ok = true;
    if (args.split_k > 1) {
      ok = (args.acc == args.y32 ? B2C_O32_OK(args.dbg, 23, args.acc + first, 4) && B2C_O32_OK(args.dbg, 23, args.acc + last, 4)
                                 : B2C_WS_OK(args.dbg, 23, args.acc + first, 4) && B2C_WS_OK(args.dbg, 23, args.acc + last, 4));
    } else {
      if (args.out_mode & B2C_OUT_I32) ok = B2C_O32_OK(args.dbg, 24, args.y32 + first, 4) && B2C_O32_OK(args.dbg, 24, args.y32 + last, 4);
      if (ok && (args.out_mode & B2C_OUT_I8)) ok = B2C_O8_OK(args.dbg, 25, args.y8 + first, 1) && B2C_O8_OK(args.dbg, 25, args.y8 + last, 1);
    }
    if (!ok) return;
  }
#endif
  const int n_img = (int)args.div_pq.div((uint32_t)m_first);
  int pq = m_first - n_img * args.PQ;
  const bool nhwc = args.out_layout == B2C_LAYOUT_NHWC;
  const bool split = args.split_k > 1;
  if (!split && (args.bias != nullptr || args.relu)) {
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = activate(args, v[j], k);
  }
  if (nhwc) {
    long long o = (long long)m_first * args.K + k;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (j < count) {
        if (split) {
          atomicAdd(args.acc + o, v[j]);
        } else {
          if (args.out_mode & B2C_OUT_I32) args.y32[o] = v[j];
          if (args.out_mode & B2C_OUT_I8) args.y8[o] = requant(v[j], args.shift);
        }
      }
      o += args.K;
    }
    return;
  }
  long long o = ((long long)n_img * args.K + k) * args.PQ + pq;
  if (!split && count == 16 && pq + 16 <= args.PQ) {
    if (args.out_mode & B2C_OUT_I32) {
      int32_t* dst = args.y32 + o;
      if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
#pragma unroll
        for (int j = 0; j < 16; j += 4) *reinterpret_cast<int4*>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = v[j];
      }
    }
    if (args.out_mode & B2C_OUT_I8) {
      int8_t* dst = args.y8 + o;
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        w[j] = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) w[j] |= (uint32_t)(uint8_t)requant(v[j * 4 + i], args.shift) << (8 * i);
      }
      if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
      } else if ((reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) reinterpret_cast<uint32_t*>(dst)[j] = w[j];
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[j] = (int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xff);
      }
    }
    return;
  }
  // general case: the run crosses an image boundary, is a tail, or adds into the split buffer
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    if (j < count) {
      if (split) {
        atomicAdd(args.acc + o, v[j]);
      } else {
        if (args.out_mode & B2C_OUT_I32) args.y32[o] = v[j];
        if (args.out_mode & B2C_OUT_I8) args.y8[o] = requant(v[j], args.shift);
      }
      ++o;
      if (++pq == args.PQ) {
        pq = 0;
        o += (long long)(args.K - 1) * args.PQ;  // same channel of the next image
      }
    }
  }
}

template <int NC>
__device__ __forceinline__ void epilogue_columns(const ConvArgs& args, uint32_t taddr, int kbase, bool row_valid,
                                                 long long base_nkpq, long long base_npqk, uint32_t exchange_addr,
                                                 int bias_off = 0) {
  int32_t v[NC];
  __syncwarp();
  tmem_ld<NC>(taddr, v);  // warp-collective: executed by all lanes
  if (exchange_addr != 0) {
    // cluster reduction: the partial sums go to this block's exchange tile [column][row]
#pragma unroll
    for (int j = 0; j < NC; ++j)
      asm volatile("st.shared.b32 [%0], %1;" ::"r"(exchange_addr + (uint32_t)j * (kTileM * 4)), "r"(v[j]) : "memory");
    return;
  }
  store_columns<NC>(args, v, kbase, row_valid, base_nkpq, base_npqk, bias_off);
}

}  // namespace
}  // namespace b2c
