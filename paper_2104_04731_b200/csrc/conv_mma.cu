// The convolution kernel: the GEMM intrinsic of the paper's Section 5.1 (8-bit operands, 32-bit
// accumulation, C_xy += A_xz * B_zy^T with B held transposed) realised as tcgen05.mma.kind::i8
// with the accumulator tile in tensor memory, and the vector unit's quantisation step fused
// into the epilogue.
//
// One thread block owns one 128 x tile_n accumulator tile (rows = fused (n, p, q), the Fuse
// rule of Table 2; columns = output channels) and a slice of the reduction.  Warp roles:
//   warp 0      TMA producer (operand B always; operand A for the tiled and im2col-mode maps)
//   warp 1      tensor-memory allocation, MMA issue (one elected lane)
//   warps 2-5   operand-A gather into swizzled shared memory (stencil unroll inside the
//               kernel), then the epilogue: tcgen05.ld, shift / clip, global stores
// Shared-memory stages form a ring guarded by full/empty mbarriers.  Every wait is bounded:
// on expiry the block raises an abort flag, records B2C_E_TIMEOUT in the status word, lets
// copies in flight drain, frees its tensor memory and returns.
#include "b2c_internal.h"

namespace b2c {

namespace {

constexpr int kThreads = 192;
constexpr unsigned long long kWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s per wait

struct __align__(8) SharedCtl {
  unsigned long long full[8];
  unsigned long long empty[8];
  unsigned long long tmem_full;
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
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
      atomicExch(status, B2C_E_TIMEOUT);
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

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          dst),
      "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                   uint32_t bar, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, "
      "%5}], [%6], {%7, %8};" ::"r"(dst),
      "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(off_w), "h"(off_h)
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

// Instruction descriptor for kind::i8: D = s32 (code 2 at bit 4), A = B = signed 8-bit (code 1
// at bits 7 and 10), both operands K-major (no transpose bits), N/8 at bit 17, M/16 at bit 24.
__device__ __forceinline__ uint32_t make_idesc_i8(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
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

template <int AMODE>
__global__ void __launch_bounds__(kThreads) conv_mma_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                                             const __grid_constant__ CUtensorMap tmap_b,
                                                             const ConvArgs args) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * kTileM;
  const int n0 = blockIdx.y * args.tile_n;
  const int kb_begin = (int)((long long)blockIdx.z * args.num_kb / args.split_k);
  const int kb_end = (int)((long long)(blockIdx.z + 1) * args.num_kb / args.split_k);
  const int stages = args.stages;
  const int bk = args.bk;
  const uint32_t a_stage_bytes = kTileM * bk;
  const uint32_t b_stage_bytes = args.tile_n * bk;

  // Stage buffers start on a 1024-byte boundary (the 128-byte swizzle repeats every 1024 bytes).
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base;
  const uint32_t b_base = smem_base + stages * a_stage_bytes;
  uint8_t* smem_aligned = smem_raw + (smem_base - smem_u32(smem_raw));
  GatherEntry* s_table = reinterpret_cast<GatherEntry*>(smem_aligned + stages * (a_stage_bytes + b_stage_bytes));

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&ctl.full[s]), AMODE == A_GATHER ? 1 + 128 : 1);
      mbar_init(smem_u32(&ctl.empty[s]), 1);
    }
    mbar_init(smem_u32(&ctl.tmem_full), 1);
    ctl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(args.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (AMODE == A_GATHER) {
    for (int i = threadIdx.x; i < args.table_len; i += kThreads) s_table[i] = args.table[i];
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = ctl.tmem_base;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int n_img = 0, h_org = 0, w_org = 0;
      if (AMODE == A_IM2COL_TMA) {
        n_img = m0 / args.PQ;
        const int rem = m0 - n_img * args.PQ;
        const int p = rem / args.Q, q = rem - p * args.Q;
        h_org = p * args.stride_h - args.pad_h;
        w_org = q * args.stride_w - args.pad_w;
      }
      int it = 0;
      for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status)) break;
        const uint32_t full = smem_u32(&ctl.full[s]);
        if (AMODE == A_GATHER) {
          mbar_arrive_expect_tx(full, b_stage_bytes);
          tma_load_2d(b_base + s * b_stage_bytes, &tmap_b, kb * bk, n0, full);
        } else if (AMODE == A_TILED) {
          mbar_arrive_expect_tx(full, a_stage_bytes + b_stage_bytes);
          tma_load_2d(a_base + s * a_stage_bytes, &tmap_a, kb * bk, m0, full);
          tma_load_2d(b_base + s * b_stage_bytes, &tmap_b, kb * bk, n0, full);
        } else {
          const int tap = kb / args.kb_per_tap;
          const int cb = kb - tap * args.kb_per_tap;
          const int r = tap / args.S, sx = tap - r * args.S;
          mbar_arrive_expect_tx(full, a_stage_bytes + b_stage_bytes);
          tma_load_im2col_4d(a_base + s * a_stage_bytes, &tmap_a, cb * bk, w_org, h_org, n_img, full,
                             (uint16_t)(sx * args.dil_w), (uint16_t)(r * args.dil_h));
          tma_load_2d(b_base + s * b_stage_bytes, &tmap_b, tap * args.tap_cols + cb * bk, n0, full);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = make_idesc_i8(args.tile_n);
      int it = 0;
      bool ok = true;
      for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, args.status)) {
          ok = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t adesc = make_smem_desc(a_base + s * a_stage_bytes, bk);
        const uint64_t bdesc = make_smem_desc(b_base + s * b_stage_bytes, bk);
        const int ksteps = (kb == args.num_kb - 1) ? args.ksteps_last : args.ksteps_full;
        for (int k = 0; k < ksteps; ++k) {
          // Advancing 32 bytes along the row = 2 units of 16 bytes in the descriptor address.
          mma_i8(tmem_acc, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        mma_commit(smem_u32(&ctl.empty[s]));
      }
      if (ok) mma_commit(smem_u32(&ctl.tmem_full));
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- gather + epilogue warps
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    const int row = quad * 32 + lane;        // accumulator row = A-tile row
    const long long m = (long long)m0 + row;
    const bool row_valid = m < args.Mg;
    int n_img = 0, pq = 0;
    if (row_valid) {
      n_img = (int)(m / args.PQ);
      pq = (int)(m - (long long)n_img * args.PQ);
    }
    bool ok = true;

    if (AMODE == A_GATHER) {
      // Stencil unroll formed in place: this thread writes row `row` of the A tile, 128 bytes
      // per stage, in the 128-byte swizzled order the MMA descriptor expects (16-byte chunk j
      // of row r lives at chunk position j ^ (r & 7)).
      const int p = pq / args.Q, q = pq - p * args.Q;
      const int h0 = row_valid ? p * args.stride_h - args.pad_h : -(1 << 29);
      const int w0 = q * args.stride_w - args.pad_w;
      const int8_t* base =
          args.x + n_img * args.x_stride_n + (long long)(row_valid ? h0 : 0) * args.x_stride_h + (long long)w0 * args.x_stride_w;
      const uint32_t row_off = (uint32_t)row * 128u;
      const uint32_t xr = (uint32_t)(row & 7);
      int it = 0;
      for (int kb = kb_begin; kb < kb_end; ++kb, ++it) {
        const int s = it % stages;
        const uint32_t ph = (uint32_t)(it / stages) & 1u;
        if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status)) {
          ok = false;
          break;
        }
        const uint32_t a_row = a_base + s * a_stage_bytes + row_off;
        const int chunks = (kb == args.num_kb - 1) ? args.ksteps_last * 2 : 8;
        for (int j = 0; j < chunks; ++j) {
          uint32_t wv[4] = {0, 0, 0, 0};
          const GatherEntry* te = s_table + kb * 128 + j * 16;
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const GatherEntry g = te[e];
            const int h = h0 + g.dh, ww = w0 + g.dw;
            uint32_t v = 0;
            if (g.off >= 0 && (unsigned)h < (unsigned)args.H && (unsigned)ww < (unsigned)args.W)
              v = (uint8_t)__ldg(base + g.off);
            wv[e >> 2] |= v << (8 * (e & 3));
          }
          const uint32_t dst = a_row + ((((uint32_t)j) ^ xr) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]),
                       "r"(wv[3])
                       : "memory");
        }
        // Make the generic-proxy writes visible to the tensor core's async proxy, then signal.
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(smem_u32(&ctl.full[s]));
      }
    }

    // ---- epilogue ----
    if (ok) ok = mbar_wait(smem_u32(&ctl.tmem_full), 0u, &ctl, args.status);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
      const uint32_t taddr_row = tmem_acc + ((uint32_t)(quad * 32) << 16);
      const bool split = args.split_k > 1;
      const bool nhwc = args.out_layout == B2C_LAYOUT_NHWC;
      const int K = args.K;
      // Output index of (m, k): NKPQ -> (n*K + k)*PQ + pq ; NPQK -> m*K + k.
      const long long base_nkpq = (long long)n_img * K * args.PQ + pq;
      const long long base_npqk = m * K;
      for (int c0 = 0; c0 < args.tile_n; c0 += 16) {
        int32_t v[16];
        __syncwarp();
        tmem_ld16(taddr_row + (uint32_t)c0, v);  // warp-collective: executed by all lanes
        if (!row_valid) continue;
        const int kbase = n0 + c0;
        if (kbase >= K) continue;
        if (split) {
          // Partial sums of the reduction slices meet in global memory; integer addition is
          // associative, so the order of arrival does not change the result.
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int k = kbase + j;
            if (k < K) {
              const long long o = nhwc ? base_npqk + k : base_nkpq + (long long)k * args.PQ;
              atomicAdd(args.acc + o, v[j]);
            }
          }
        } else if (!nhwc) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int k = kbase + j;
            if (k < K) {
              const long long o = base_nkpq + (long long)k * args.PQ;
              if (args.out_mode & B2C_OUT_I32) args.y32[o] = v[j];
              if (args.out_mode & B2C_OUT_I8) args.y8[o] = requant(v[j], args.shift);
            }
          }
        } else {
          const bool full16 = kbase + 16 <= K;
          if (args.out_mode & B2C_OUT_I32) {
            int32_t* dst = args.y32 + base_npqk + kbase;
            if (full16 && (K & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<int4*>(dst + j) = make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (kbase + j < K) dst[j] = v[j];
            }
          }
          if (args.out_mode & B2C_OUT_I8) {
            int8_t* dst = args.y8 + base_npqk + kbase;
            if (full16 && (K & 15) == 0) {
              uint32_t w[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                w[j] = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) w[j] |= (uint32_t)(uint8_t)requant(v[j * 4 + i], args.shift) << (8 * i);
              }
              *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (kbase + j < K) dst[j] = requant(v[j], args.shift);
            }
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (ctl.abort_flag && threadIdx.x == 0) {
    // Give copies that were already issued time to land before the shared memory is released.
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 50000ull) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(args.tmem_cols)
                 : "memory");
  }
}

}  // namespace

size_t conv_mma_smem_bytes(int amode, const ConvArgs& a) {
  size_t b = 1024 + (size_t)a.stages * (kTileM + a.tile_n) * a.bk;
  if (amode == A_GATHER) b += (size_t)a.table_len * sizeof(GatherEntry);
  return b;
}

cudaError_t launch_conv_mma(int amode, const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const ConvArgs& args,
                            cudaStream_t st) {
  const size_t smem = conv_mma_smem_bytes(amode, args);
  dim3 grid((unsigned)((args.Mg + kTileM - 1) / kTileM), (unsigned)((args.K + args.tile_n - 1) / args.tile_n),
            (unsigned)args.split_k);
  cudaError_t e;
#define B2C_LAUNCH(MODE)                                                                                  \
  {                                                                                                       \
    static size_t configured = 0;                                                                         \
    if (smem > configured) {                                                                              \
      e = cudaFuncSetAttribute(conv_mma_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024); \
      if (e != cudaSuccess) return e;                                                                     \
      configured = 200 * 1024;                                                                            \
    }                                                                                                     \
    conv_mma_kernel<MODE><<<grid, kThreads, smem, st>>>(*tmap_a, *tmap_b, args);                          \
  }
  if (amode == A_TILED) B2C_LAUNCH(A_TILED)
  else if (amode == A_IM2COL_TMA) B2C_LAUNCH(A_IM2COL_TMA)
  else B2C_LAUNCH(A_GATHER)
#undef B2C_LAUNCH
  return cudaGetLastError();
}

}  // namespace b2c
