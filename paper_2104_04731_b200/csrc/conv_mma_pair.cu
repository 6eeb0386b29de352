// Two-SM form of the convolution kernel: a pair of thread blocks on neighbouring SMs (a cluster
// of two) owns one 256 x tile_n accumulator tile and issues tcgen05.mma.cta_group::2.kind::i8.
// The GEMM intrinsic is still that of Section 5.1 (8-bit operands, 32-bit accumulation,
// C_xy += A_xz * B_zy^T, B held transposed); what changes is how the operands are shared: each
// block of the pair loads its own 128 rows of A (fused (n, p, q) pixels) and only HALF of the B
// rows (tile_n / 2 output channels), and the tensor cores of both SMs read the two B halves from
// both shared memories.  Per MMA cycle a block therefore takes a third fewer operand bytes from
// L2 than the one-SM kernel with the same tile_n, which is what bounds the compute-bound shapes.
//
// Roles in each block: warp 0 TMA producer (own A rows, own B half, into the block's own shared
// memory; no cluster multicast), warp 1 MMA issue in the leader block (cluster rank 0; idle in the
// other block after the tensor-memory allocation), warps 2-9 epilogue of the block's own 128
// accumulator rows (tcgen05.ld from the block's own tensor memory, activation step, shift / clip,
// stores).  Barriers: the copies of BOTH blocks complete on the leader's full[s] (the loads carry
// .cta_group::2, which lets a copy signal a barrier in the peer block; the leader's producer
// announces the bytes of both), so the MMA thread waits on one barrier with no hand-over in
// between (a hand-over by a thread of the peer, mbarrier.arrive.release.cluster on the leader's
// barrier, measured about 0.8 us per stage and paced the whole kernel); the leader's commits
// arrive on empty[s] and tmem_full[b] of BOTH blocks (tcgen05.commit with a block mask); the
// epilogue warps of both blocks arrive on the leader's tmem_empty[b].  Every wait is bounded as
// in the one-SM kernel.
#include <algorithm>

#include "conv_mma_common.cuh"

namespace b2c {

namespace {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
  return remote;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Waits that pair with arrivals from the other block of the cluster.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
__device__ __noinline__ bool mbar_wait_cluster_slow(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status) {
  const unsigned long long t0 = global_ns();
  while (true) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (ctl->abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      ctl->abort_flag = 1;
      atomicCAS(status, 0, B2C_E_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status) {
#pragma unroll 1
  for (int i = 0; i < 32; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  return mbar_wait_cluster_slow(bar, parity, ctl, status);
}

// TMA loads of a block of the pair: destination in the executing block's shared memory, completion
// on `bar`, a shared::cluster address that may lie in either block of the pair (.cta_group::2).
__device__ __forceinline__ void tma_pair_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                                 uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %5, 0;\n"
      "@q cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, %3}], "
      "[%4];\n}" ::"r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(bar), "r"(on)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_im2col_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                        uint32_t bar, uint16_t off_w, uint16_t off_h, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\nsetp.ne.b32 q, %9, 0;\n"
      "@q cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, "
      "%3, %4, %5}], [%6], {%7, %8};\n}" ::"r"(dst),
      "l"(map), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(off_w), "h"(off_h), "r"(on)
      : "memory");
}

// Instruction descriptor of the two-SM MMA: as make_idesc_i8, with M = 256 (128 rows per block).
__device__ __forceinline__ uint32_t make_idesc_i8_pair(int n) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// One reduction block of the pair: `ksteps` (1..4) two-SM MMAs over consecutive 32-byte slices.
__device__ __forceinline__ void mma_i8_pair_block(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
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
      "@q0 tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, pacc;\n"
      "@q1 tcgen05.mma.cta_group::2.kind::i8 [%0], a1, b1, %3, ptrue;\n"
      "@q2 tcgen05.mma.cta_group::2.kind::i8 [%0], a2, b2, %3, ptrue;\n"
      "@q3 tcgen05.mma.cta_group::2.kind::i8 [%0], a3, b3, %3, ptrue;\n"
      "}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(on), "r"(ksteps)
      : "memory");
}
// Arrives on the barrier at this shared-memory offset in both blocks of the pair once every MMA
// issued so far has completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar, uint32_t on) {
  asm volatile(
      "{\n.reg .pred q;\n.reg .b16 m;\nsetp.ne.b32 q, %1, 0;\nmov.b16 m, 3;\n"
      "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n}" ::"r"(bar),
      "r"(on)
      : "memory");
}

constexpr int kPackWarps = 4;  // warps 10..13 of the fused form: activation pack
constexpr int kPackGroup = 32 * kPackWarps;

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Pack role (Table 2: Pad, Split, Reorder of the activations, here inside the convolution kernel so
// that the memory-bound rewrite runs beside the tensor-bound main loop).  Each of the four warps is
// a pipeline of its own with one shared-memory buffer.  A warp takes a batch from the global
// counter (one atomic per batch, issued one batch ahead): pk_ct channels x pk_pt pixels of one
// image, i.e. up to four units of 16 channels.  The batch's channel rows arrive by bulk async copies
// (one copy when the batch is contiguous in NCHW); every lane transposes 16 channels x 4 pixels in
// registers and stores 16-byte pieces of the NHWC tensor.  When all lanes have read the buffer the
// next batch's copies are started, and only then does the warp fence its stores and bump the
// image's counter by the number of units: fence and copy latency overlap, and the other three
// warps hide what is left.
__device__ __forceinline__ void fused_pack_role(const ConvArgs& args, uint8_t* buf0, unsigned long long* bars,
                                                SharedCtl* ctl, int pw, int lane) {
  const int C = args.pk_C, HW = args.pk_HW, C_pad = args.pk_Cpad, PT = args.pk_pt, CT = args.pk_ct;
  const int hw_tiles = args.pk_hw_tiles;
  const int cgroups = args.pk_ctiles;                       // batches along the channel axis
  const int bpi = hw_tiles * cgroups;                       // batches per image
  const int total = args.pk_N * bpi;
  const bool row_mode = hw_tiles > 1;
  const int rp = row_mode ? PT : HW;                        // row pitch in shared memory
  uint8_t* my_buf = buf0 + pw * (args.pk_smem / kPackWarps);
  const uint32_t my_buf_a = smem_u32(my_buf);
  const uint32_t bar = smem_u32(&bars[pw]);
  uint32_t parity = 0u;

  // starts the copies of a batch: channels [c0, min(c0 + CT, C)) x pixels [hw0, hw0 + npx) of image n
  auto start_batch = [&](int n, int c0, int hw0, int npx) {
    const int rows = max(0, min(CT, C - c0));
    if (rows == 0) return;
#ifdef B2C_DEBUG_BOUNDS
    // the whole source block of the batch (first byte of the first row .. last byte of the last row);
    // a refused batch completes its barrier phase without copying, so that its consumer's wait ends
    if (!B2C_X_OK(args.dbg, 40, args.pk_src + ((size_t)n * C + c0) * HW + hw0, (long long)(rows - 1) * HW + npx)) {
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
      __syncwarp();
      return;
    }
#endif
    if (lane == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(rows * npx)) : "memory");
    __syncwarp();
    const int8_t* xin = args.pk_src + ((size_t)n * C + c0) * HW + hw0;
    if (row_mode) {
      for (int r = lane; r < rows; r += 32)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         my_buf_a + (uint32_t)(r * rp)),
                     "l"(xin + (size_t)r * HW), "r"((uint32_t)npx), "r"(bar)
                     : "memory");
    } else if (lane == 0) {
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(my_buf_a),
                   "l"(xin), "r"((uint32_t)(rows * HW)), "r"(bar)
                   : "memory");
    }
  };
  auto decode = [&](int batch, int* n, int* c0, int* hw0, int* npx) {
    *n = batch / bpi;
    const int rem = batch - *n * bpi;
    const int hwt = rem / cgroups;
    *c0 = (rem - hwt * cgroups) * CT;
    *hw0 = hwt * PT;
    *npx = min(PT, HW - *hw0);
  };

  int batch = 0, batch_next = 0;
  if (lane == 0) batch = atomicAdd(args.pk_ctl, 1);
  batch = __shfl_sync(0xffffffffu, batch, 0);
  if (batch < total) {
    int n, c0, hw0, npx;
    decode(batch, &n, &c0, &hw0, &npx);
    start_batch(n, c0, hw0, npx);
  }
  while (batch < total) {
    if (lane == 0) batch_next = atomicAdd(args.pk_ctl, 1);  // used after this batch: its latency is hidden
    int n, cg0, hw0, npx;
    decode(batch, &n, &cg0, &hw0, &npx);
    const int units = min(CT, C_pad - cg0) >> 4;
    if (cg0 < C) {
      if (!__all_sync(0xffffffffu, mbar_wait(bar, parity, ctl, args.status))) break;
      parity ^= 1u;
    }
    // item = (group of 4 pixels, unit): the lanes of consecutive units of one pixel write consecutive
    // 16-byte pieces, so a pixel's 64 bytes of this batch leave the SM as whole sectors
    const int items = ((npx + 3) >> 2) * units;
    for (int it = lane; it < items; it += 32) {
      const int pg = it / units, k = it - pg * units;
      const int c0 = cg0 + 16 * k;
      uint32_t w[16];
      if (c0 < C) {
        const uint8_t* tile = my_buf + (16 * k) * rp + pg * 4;
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = *reinterpret_cast<const uint32_t*>(tile + i * rp);
      } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) w[i] = 0;  // channels past C: the zero padding of the channel axis
      }
      int8_t* dst = args.pk_dst + ((size_t)n * HW + hw0 + pg * 4) * C_pad + c0;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (pg * 4 + j < npx) {
          uint32_t o[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t lo = __byte_perm(w[4 * q], w[4 * q + 1], j | ((4 + j) << 4));
            const uint32_t hi = __byte_perm(w[4 * q + 2], w[4 * q + 3], j | ((4 + j) << 4));
            o[q] = __byte_perm(lo, hi, 0x5410);
          }
          if (B2C_WS_OK(args.dbg, 41, dst + (size_t)j * C_pad, 16))
            *reinterpret_cast<uint4*>(dst + (size_t)j * C_pad) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
    }
    __syncwarp();  // every lane has read the buffer: the next batch's copies may land in it
    batch_next = __shfl_sync(0xffffffffu, batch_next, 0);
    if (batch_next < total) {
      int n2, c2, h2, p2;
      decode(batch_next, &n2, &c2, &h2, &p2);
      start_batch(n2, c2, h2, p2);
    }
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(args.pk_ctl + 1 + n, units);
    batch = batch_next;
  }
}

// Producer side of the fused pack: the images a tile reads (rows m_first .. m_first + 127 of the fused
// pixel axis) must be complete before its loads are issued.  Lanes poll different images; the
// generic-proxy writes of the pack warps (any SM) are then ordered before this thread's TMA loads.
__device__ __forceinline__ bool wait_images_packed(const ConvArgs& args, int m_first, int lane, SharedCtl* ctl) {
  bool ok = true;
  if (m_first < args.Mg) {
    const int upi = args.pk_hw_tiles * (args.pk_Cpad >> 4);  // units of one image
    const int n_a = (int)args.div_pq.div((uint32_t)m_first);
    const int n_b = (int)args.div_pq.div((uint32_t)min(m_first + kTileM - 1, args.Mg - 1));
    for (int n = n_a + lane; n <= n_b && ok; n += 32) {
      const int* cnt = args.pk_ctl + 1 + n;
      if (ld_acquire_gpu(cnt) >= upi) continue;
      const unsigned long long t0 = global_ns();
      while (ld_acquire_gpu(cnt) < upi) {
        if (ctl->abort_flag) {
          ok = false;
          break;
        }
        if (global_ns() - t0 > kWaitLimitNs) {
          ctl->abort_flag = 1;
          atomicCAS(args.status, 0, B2C_E_TIMEOUT);
          ok = false;
          break;
        }
        __nanosleep(200);
      }
    }
  }
  ok = __all_sync(0xffffffffu, ok);
  asm volatile("fence.proxy.async.global;" ::: "memory");
  return ok;
}

// PERSIST: 0 = one pair tile per cluster, two blocks resident per SM (one 256-column accumulator each,
// stage ring within half of the shared memory); 1 = 74 clusters walk the tile list, one block per SM,
// two accumulator buffers, the deepest stage ring that fits.
// PACK: the block has four more warps that run the activation pack (persistent channel-pack map only).
template <int AMODE, int PERSIST, bool PACK>
__global__ void __launch_bounds__(PACK ? kThreads + kPackGroup : kThreads, PERSIST == 1 ? 1 : 2)
    conv_mma_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                         const ConvArgs args) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;
  __shared__ __align__(8) unsigned long long pack_bars[kPackWarps];

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0: leader (issues the MMAs), 1: peer
  const int pair_id = (int)(blockIdx.x >> 1);
  const int num_pairs = (int)(gridDim.x >> 1);
  constexpr bool persistent = PERSIST != 0;
  const int tile_first = pair_id;
  const int tile_step = num_pairs;
  const int tile_end = args.num_tiles;
  const int nbuf = persistent ? args.tmem_bufs : 1;  // 1 or 2
  const int stages = args.stages;
  const int bk = args.bk;
  const int half_n = args.tile_n >> 1;  // B rows (output channels) this block loads
  const uint32_t a_stage_bytes = (uint32_t)(kTileM * bk);
  const uint32_t b_stage_bytes = (uint32_t)(half_n * bk);

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base;
  const uint32_t b_base = smem_base + stages * a_stage_bytes;

  if (warp == 0) {
    if (lane < stages) {
      // full[] is used in the leader only: one arrival (its producer) plus the bytes of both blocks
      mbar_init(smem_u32(&ctl.full[lane]), 1);
      mbar_init(smem_u32(&ctl.empty[lane]), 1);
    }
    if (lane == 8) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
        mbar_init(smem_u32(&ctl.tmem_empty[b]), 2 * kGatherWarps);  // the epilogue warps of both blocks
      }
      ctl.abort_flag = 0;
    }
    if (lane == 9) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
    if (lane == 10) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    if (PACK && lane >= 16 && lane < 16 + kPackWarps) mbar_init(smem_u32(&pack_bars[lane - 16]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // both blocks of the pair allocate the same columns together
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(args.tmem_cols * nbuf)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  // the other block's barriers must be initialised before anything arrives on them
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = __shfl_sync(0xffffffffu, ctl.tmem_base, 0);
  pdl_wait();
  // The next kernel of the stream may start its set-up once the leader has issued its last MMA (its
  // blocks then wait in griddepcontrol.wait while this grid's epilogue runs).  An earlier start would
  // park waiting blocks on SMs that blocks of other streams could be using.
  if (rank != 0) pdl_launch_dependents();

#define B2C_PAIR_TILE_ORIGIN(t)                                     \
  const int mt_ = (int)args.div_tiles_n.div((uint32_t)(t));        \
  const int m0 = mt_ * (2 * kTileM) + (int)rank * kTileM;          \
  const int n0 = ((t) - mt_ * args.tiles_n) * args.tile_n;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both blocks)
    int s = 0;
    uint32_t ph = 0;
    uint32_t a_dst = a_base, b_dst = b_base;
    const uint32_t leader_lane = elect_one() ? 1u : 0u;
    bool alive = true;
    for (int t = tile_first; t < tile_end && alive; t += tile_step) {
      B2C_PAIR_TILE_ORIGIN(t)
      int n_img = 0, h_org = 0, w_org = 0, cb = 0, sx = 0, r = 0;
      if (AMODE == A_IM2COL_TMA) {
        n_img = (int)args.div_pq.div((uint32_t)m0);
        const int rem = m0 - n_img * args.PQ;
        const int p = (int)args.div_q.div((uint32_t)rem), q = rem - p * args.Q;
        h_org = p * args.stride_h - args.pad_h;
        w_org = q * args.stride_w - args.pad_w;
      }
      if (PACK && !wait_images_packed(args, m0, lane, &ctl)) break;
      int kcol = 0;
      const int wrow0 = n0 + (int)rank * half_n;  // first output channel of this block's B half
      for (int kb = 0; kb < args.num_kb; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status))) {
          alive = false;
          break;
        }
        // both blocks' copies complete on the leader's barrier; the leader announces the bytes of both
        const uint32_t full = map_to_rank(smem_u32(&ctl.full[s]), 0u);
        if (rank == 0) mbar_arrive_expect_tx(smem_u32(&ctl.full[s]), 2u * (a_stage_bytes + b_stage_bytes), leader_lane);
        if (AMODE == A_TILED) {
          tma_pair_load_2d(a_dst, &tmap_a, kcol, m0, full, leader_lane);
        } else {
          tma_pair_load_im2col_4d(a_dst, &tmap_a, cb * bk, w_org, h_org, n_img, full, (uint16_t)(sx * args.dil_w),
                                  (uint16_t)(r * args.dil_h), leader_lane);
          if (++cb == args.kb_per_tap) {
            cb = 0;
            if (++sx == args.S) {
              sx = 0;
              ++r;
            }
          }
        }
        tma_pair_load_2d(b_dst, &tmap_b, kcol, wrow0, full, leader_lane);
        kcol += bk;
        a_dst += a_stage_bytes;
        b_dst += b_stage_bytes;
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
          a_dst = a_base;
          b_dst = b_base;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 && rank != 0) {
    // (the peer's warp 1 only allocates and frees tensor memory)
  } else if (warp == 1) {
    // ---------------------------------------------------------------- leader: MMA issue for the pair
    const uint32_t idesc = make_idesc_i8_pair(args.tile_n);
    const uint64_t adesc0 = make_smem_desc(a_base, bk);
    const uint64_t bdesc0 = make_smem_desc(b_base, bk);
    const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;
    uint64_t adesc = adesc0, bdesc = bdesc0;
    int s = 0;
    uint32_t ph = 0;
    const uint32_t leader_lane = elect_one() ? 1u : 0u;
    bool alive = true;
    int ti = 0;
    for (int t = tile_first; t < tile_end && alive; t += tile_step, ++ti) {
      const int buf = persistent ? (ti & (nbuf - 1)) : 0;
      const uint32_t use = persistent ? (uint32_t)(ti / nbuf) : 0u;
      if (persistent) {
        // the epilogue warps of both blocks must have drained this accumulator buffer
        if (!__all_sync(0xffffffffu, mbar_wait_cluster(smem_u32(&ctl.tmem_empty[buf]), (use & 1u) ^ 1u, &ctl, args.status))) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
      const uint32_t d_tmem = tmem_acc + (uint32_t)(buf * args.tmem_cols);
      uint32_t accumulate = 0;
      for (int kb = 0; kb < args.num_kb; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, args.status))) {
          alive = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int ksteps = (kb == args.num_kb - 1) ? args.ksteps_last : args.ksteps_full;
        mma_i8_pair_block(d_tmem, adesc, bdesc, idesc, accumulate, leader_lane, ksteps);
        mma_commit_pair(smem_u32(&ctl.empty[s]), leader_lane);
        if (kb == args.num_kb - 1) mma_commit_pair(smem_u32(&ctl.tmem_full[buf]), leader_lane);
        accumulate = 1;
        adesc += a_step;
        bdesc += b_step;
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
          adesc = adesc0;
          bdesc = bdesc0;
        }
      }
    }
    pdl_launch_dependents();
    __syncwarp();
  } else if (PACK && warp >= 2 + kGatherWarps) {
    // ---------------------------------------------------------------- activation pack (both blocks)
    uint8_t* pack_buf = smem_raw + (smem_base - smem_u32(smem_raw)) + args.stage_region;
    fused_pack_role(args, pack_buf, pack_bars, &ctl, warp - (2 + kGatherWarps), lane);
  } else {
    // ---------------------------------------------------------------- epilogue warps (both blocks)
    const int quad = warp & 3;         // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;  // the two warps of a quadrant split the columns
    const int row = quad * 32 + lane;
    const uint32_t leader_empty0 = map_to_rank(smem_u32(&ctl.tmem_empty[0]), 0u);
    const uint32_t leader_empty1 = map_to_rank(smem_u32(&ctl.tmem_empty[1]), 0u);
    bool ok = true;
    int ti = 0;
    for (int t = tile_first; t < tile_end && ok; t += tile_step, ++ti) {
      B2C_PAIR_TILE_ORIGIN(t)
      const unsigned m = (unsigned)m0 + (unsigned)row;
      bool row_valid = m < (unsigned)args.Mg;
      int n_img = 0, pq = 0;
      if (row_valid) {
        n_img = (int)args.div_pq.div(m);
        pq = (int)(m - (unsigned)n_img * (unsigned)args.PQ);
      }
      int out_img = n_img, out_pq = pq;
      if (args.remap == 1 && row_valid) {
        // dilation phase pack: interleave the sub-image results back, drop rows outside the output
        const int ps = (int)args.div_q.div((uint32_t)pq), qs = pq - ps * args.Q;
        const int phases = args.ph_dh * args.ph_dw;
        out_img = n_img / phases;
        const int phs = n_img - out_img * phases;
        const int a = phs / args.ph_dw, b = phs - a * args.ph_dw;
        const int po = (ps - args.ph_pad_h) * args.ph_dh + a + args.out_pad_h;
        const int qo = (qs - args.ph_pad_w) * args.ph_dw + b + args.out_pad_w;
        row_valid = (unsigned)po < (unsigned)args.out_P && (unsigned)qo < (unsigned)args.out_Q;
        out_pq = po * args.out_Q + qo;
      }
      const int buf = persistent ? (ti & (nbuf - 1)) : 0;
      const uint32_t use = persistent ? (uint32_t)(ti / nbuf) : 0u;
      ok = mbar_wait(smem_u32(&ctl.tmem_full[buf]), use & 1u, &ctl, args.status);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (ok) {
        const long long base_nkpq = (long long)out_img * args.y_stride_n + out_pq;
        const long long base_npqk = args.remap ? ((long long)out_img * args.out_PQ + out_pq) * args.K : (long long)m * args.K;
        const int cols = args.tile_n >> 1;  // tile_n >= 32
        const int c_begin = half * cols;
        const uint32_t taddr = tmem_acc + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * args.tmem_cols) + (uint32_t)c_begin;
        if ((cols & 31) == 0) {
          for (int c = 0; c < cols; c += 32)
            epilogue_columns<32>(args, taddr + (uint32_t)c, n0 + c_begin + c, row_valid, base_nkpq, base_npqk, 0u);
        } else {
          for (int c = 0; c < cols; c += 16)
            epilogue_columns<16>(args, taddr + (uint32_t)c, n0 + c_begin + c, row_valid, base_nkpq, base_npqk, 0u);
        }
        if (persistent) {
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(buf ? leader_empty1 : leader_empty0);
        }
      }
    }
  }
#undef B2C_PAIR_TILE_ORIGIN

  // ---------------------------------------------------------------- teardown
  // No block of the pair leaves, or frees tensor memory, while the other may still read its shared
  // memory, arrive on its barriers or write its accumulator.
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (ctl.abort_flag) {
    if (threadIdx.x == 0) {
      const unsigned long long t0 = global_ns();
      while (global_ns() - t0 < 50000ull) __nanosleep(1000);
    }
    __syncthreads();
  }
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(args.tmem_cols * nbuf)
                 : "memory");
  }
}

// Issue rate of the two-SM intrinsic itself: tcgen05.mma.cta_group::2.kind::i8 (M = 256, N = tile_n,
// K = 32) issued back to back by the leader of every pair on operands that already sit in the two
// blocks' shared memory (A: 128 rows per block, B: tile_n / 2 rows per block, each block's tensor core
// reading the other half of B from its peer).  No loads, no epilogue: the denominator for what the
// two-SM schedule can reach at most.
__global__ void __launch_bounds__(64, 1) mma_rate_pair_kernel(int tile_n, int tmem_cols, int blocks_of_four,
                                                              unsigned long long* cycles, int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base, b_base = smem_base + kTileM * 128;
  uint8_t* p = smem_raw + (smem_base - smem_u32(smem_raw));
  for (int i = threadIdx.x * 16; i < (kTileM + tile_n / 2) * 128; i += 64 * 16)
    *reinterpret_cast<uint4*>(p + i) = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl.full[0]), 1);  // (both blocks: the commit arrives on the pair's two barriers)
    ctl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = __shfl_sync(0xffffffffu, ctl.tmem_base, 0);
  if (warp == 0 && rank == 0) {
    const uint32_t idesc = make_idesc_i8_pair(tile_n);
    const uint64_t adesc = make_smem_desc(a_base, 128), bdesc = make_smem_desc(b_base, 128);
    const uint32_t leader = elect_one() ? 1u : 0u;
    const long long t0 = clock64();
    for (int i = 0; i < blocks_of_four; ++i) mma_i8_pair_block(tmem_acc, adesc, bdesc, idesc, i ? 1u : 0u, leader, 4);
    mma_commit_pair(smem_u32(&ctl.full[0]), leader);
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[0]), 0u, &ctl, status));
    const long long t1 = clock64();
    if (lane == 0) cycles[blockIdx.x >> 1] = ok ? (unsigned long long)(t1 - t0) : 0ull;
  }
  // neither block leaves, or frees tensor memory, while the leader's MMAs may still read its shared memory
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

size_t conv_mma_pair_smem_bytes(const ConvArgs& a) { return 1024 + (size_t)a.stage_region + (a.pk_on ? (size_t)a.pk_smem : 0); }

bool fused_pack_geometry(int C, int H, int W, int C_pad, int* ct, int* pt, int* hw_tiles, int* ctiles, int* smem) {
  const int HW = H * W;
  // channels in whole groups of 16 and either the whole image per unit (a multiple of 4 pixels, at most
  // 256) or pixel rows that are multiples of 16 bytes (units of 256 pixels)
  if ((C % 16) != 0 || (HW % 4) != 0 || !(HW <= 256 || (HW % 16) == 0)) return false;
  *pt = HW <= 256 ? HW : 128;
  *hw_tiles = (HW + *pt - 1) / *pt;
  *ct = 64;  // channels per batch (four units of 16)
  *ctiles = (C_pad + *ct - 1) / *ct;
  // one batch buffer per pack warp
  *smem = 4 * ((*ct * *pt + 127) / 128 * 128);
  return true;
}

cudaError_t launch_conv_mma_pair(int amode, const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const ConvArgs& args,
                                 cudaStream_t st) {
  const size_t smem = conv_mma_pair_smem_bytes(args);
  int pairs = args.persistent ? std::min(args.num_tiles, kNumSMs / 2) : args.num_tiles;
  dim3 grid((unsigned)(2 * pairs), 1, 1);
  cudaError_t e;
#define B2C_LAUNCH_PAIR(MODE, PERS, PACK)                                                                      \
  {                                                                                                           \
    static std::atomic<unsigned long long> configured{0};                                                     \
    e = set_max_dynamic_smem_once(configured, (const void*)conv_mma_pair_kernel<MODE, PERS, PACK>, 226 * 1024); \
    if (e != cudaSuccess) return e;                                                                           \
    cudaLaunchConfig_t cfg = {};                                                                              \
    cfg.gridDim = grid;                                                                                       \
    cfg.blockDim = dim3(PACK ? kThreads + kPackGroup : kThreads);                                             \
    cfg.dynamicSmemBytes = smem;                                                                              \
    cfg.stream = st;                                                                                          \
    cudaLaunchAttribute attr[2];                                                                              \
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                          \
    attr[0].val.programmaticStreamSerializationAllowed = 1;                                                   \
    attr[1].id = cudaLaunchAttributeClusterDimension;                                                         \
    attr[1].val.clusterDim.x = 2;                                                                             \
    attr[1].val.clusterDim.y = 1;                                                                             \
    attr[1].val.clusterDim.z = 1;                                                                             \
    cfg.attrs = attr;                                                                                         \
    cfg.numAttrs = 2;                                                                                         \
    if (PERS) {                                                                                               \
      /* a persistent grid is one wave: as many pairs as the device keeps resident at once */                 \
      int resident = 0;                                                                                       \
      if (cudaOccupancyMaxActiveClusters(&resident, conv_mma_pair_kernel<MODE, PERS, PACK>, &cfg) == cudaSuccess && \
          resident > 0 && resident < pairs) {                                                                 \
        pairs = resident;                                                                                     \
        cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);                                                      \
      }                                                                                                       \
      (void)cudaGetLastError();                                                                               \
    }                                                                                                         \
    e = cudaLaunchKernelEx(&cfg, conv_mma_pair_kernel<MODE, PERS, PACK>, *tmap_a, *tmap_b, args);                    \
    if (e != cudaSuccess) return e;                                                                           \
  }
  if (amode == A_TILED && args.persistent) B2C_LAUNCH_PAIR(A_TILED, 1, false)
  else if (amode == A_TILED) B2C_LAUNCH_PAIR(A_TILED, 0, false)
  else if (amode == A_IM2COL_TMA && args.persistent && args.pk_on) B2C_LAUNCH_PAIR(A_IM2COL_TMA, 1, true)
  else if (amode == A_IM2COL_TMA && args.persistent) B2C_LAUNCH_PAIR(A_IM2COL_TMA, 1, false)
  else if (amode == A_IM2COL_TMA) B2C_LAUNCH_PAIR(A_IM2COL_TMA, 0, false)
  else return cudaErrorInvalidValue;
#undef B2C_LAUNCH_PAIR
  return cudaGetLastError();
}

}  // namespace b2c

extern "C" int b2c_measure_mma_rate_pair(int tile_n, int mmas_per_pair, float* device_us, float* cycles_per_mma, void* cuda_stream) {
  using namespace b2c;
  if (!device_us || !cycles_per_mma || mmas_per_pair < 4 || mmas_per_pair > (1 << 22)) return B2C_E_INVALID_ARG;
  if (tile_n != 64 && tile_n != 128 && tile_n != 256) return B2C_E_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const int tmem_cols = tile_n;
  const int pairs = kNumSMs / 2;
  unsigned long long* cyc = nullptr;
  int* status = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  auto fail = [&](cudaError_t e) {
    set_last_cuda_error((int)e);
    cudaFree(cyc);
    cudaFree(status);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    return B2C_E_CUDA;
  };
  cudaError_t e = cudaMalloc(&cyc, pairs * sizeof(unsigned long long));
  if (e == cudaSuccess) e = cudaMemsetAsync(cyc, 0, pairs * sizeof(unsigned long long), st);
  if (e == cudaSuccess) e = cudaMalloc(&status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e != cudaSuccess) return fail(e);
  static std::atomic<unsigned long long> configured{0};
  e = set_max_dynamic_smem_once(configured, (const void*)mma_rate_pair_kernel, 200 * 1024);
  if (e != cudaSuccess) return fail(e);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(2 * pairs));
  cfg.blockDim = dim3(64);
  cfg.dynamicSmemBytes = 120 * 1024;  // more than half of the shared memory: one block per SM
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int fours = mmas_per_pair / 4;
  for (int rep = 0; rep < 2 && e == cudaSuccess; ++rep) {  // the first launch warms up
    e = cudaEventRecord(e0, st);
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, mma_rate_pair_kernel, tile_n, tmem_cols, fours, cyc, status);
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  }
  if (e != cudaSuccess) return fail(e);
  float ms = 0;
  std::vector<unsigned long long> h(pairs);
  int hs = 0;
  e = cudaEventElapsedTime(&ms, e0, e1);
  if (e == cudaSuccess) e = cudaMemcpy(h.data(), cyc, pairs * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(&hs, status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail(e);
  cudaFree(cyc);
  cudaFree(status);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (hs != 0) return hs;
  std::sort(h.begin(), h.end());
  if (h[0] == 0) return B2C_E_TIMEOUT;
  *device_us = ms * 1000.0f;
  *cycles_per_mma = (float)((double)h[pairs / 2] / (double)(fours * 4));  // median over the pairs
  return B2C_OK;
}
