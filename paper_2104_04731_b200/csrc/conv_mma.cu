// The convolution kernel: the GEMM intrinsic of the paper's Section 5.1 (8-bit operands, 32-bit
// accumulation, C_xy += A_xz * B_zy^T with B held transposed) realised as tcgen05.mma.kind::i8
// with the accumulator tile in tensor memory, and the vector unit's quantisation step fused
// into the epilogue.
//
// One thread block owns one 128 x tile_n accumulator tile (rows = fused (n, p, q), the Fuse
// rule of Table 2; columns = output channels) and a slice of the reduction.  Warp roles:
//   warp 0      TMA producer (operand B always; operand A for the tiled and im2col-mode maps)
//   warp 1      tensor-memory allocation, MMA issue (one elected lane)
//   warps 2-9   operand-A gather into swizzled shared memory (stencil unroll inside the
//               kernel), then the epilogue: tcgen05.ld, shift / clip, global stores
// Shared-memory stages form a ring guarded by full/empty mbarriers.  Every wait is bounded:
// on expiry the block raises an abort flag, records B2C_E_TIMEOUT in the status word, lets
// copies in flight drain, frees its tensor memory and returns.
#include <algorithm>

#include "conv_mma_common.cuh"

namespace b2c {

namespace {

// PERSIST: 0 = one tile per block; 1 = persistent, one block per SM (wide tiles, deep stage ring);
// 2 = persistent, three blocks per SM (narrow tiles: short main loops, several epilogues in flight).
template <int AMODE, int PERSIST>
__global__ void __launch_bounds__(kThreads, PERSIST == 1 ? 1 : 3) conv_mma_kernel(const __grid_constant__ CUtensorMap tmap_a,
                                                             const __grid_constant__ CUtensorMap tmap_b,
                                                             const ConvArgs args) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;

  // The warp index is broadcast from lane 0 so that the compiler can prove the role branches below
  // warp-uniform: inside them, loop counters, barrier addresses and above all the MMA descriptors
  // can then live in the uniform datapath that the MMA instruction takes its operands from.
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  // Tile schedule.  Small grids: one tile per block, (blockIdx.x, blockIdx.y) = (row tile, column
  // tile).  Persistent mode (large TMA-fed problems): gridDim.x blocks walk the tile list
  // t = blockIdx.x, blockIdx.x + gridDim.x, ... with the column tile fastest (blocks running at the
  // same time share the A operand in L2), and the accumulator alternates between two tensor-memory
  // buffers so that the epilogue of one tile overlaps the main loop of the next.
  // (PERSIST is a template parameter so that the one-tile-per-block instantiation carries none of
  // the loop, buffer-index and hand-back overhead.)
  constexpr bool persistent = PERSIST != 0;
  const int tile_first = persistent ? (int)blockIdx.x : 0;
  const int tile_step = persistent ? (int)gridDim.x : 1;
  const int tile_end = persistent ? args.num_tiles : 1;
  const int nbuf = persistent ? args.tmem_bufs : 1;  // a power of two, at most 4
  const int nbuf_log2 = nbuf == 4 ? 2 : (nbuf == 2 ? 1 : 0);
#define B2C_TILE_ORIGIN(t)                                                          \
  int m0, n0;                                                                       \
  if (persistent) {                                                                 \
    const int mt_ = (int)args.div_tiles_n.div((uint32_t)(t));                       \
    m0 = mt_ * kTileM;                                                              \
    n0 = ((t) - mt_ * args.tiles_n) * args.tile_n;                                  \
  } else if (args.swap) {                                                           \
    m0 = (int)blockIdx.y * kTileM;     /* accumulator rows: output channels */      \
    n0 = (int)blockIdx.x * args.tile_n; /* accumulator columns: fused pixels */     \
  } else {                                                                          \
    m0 = (int)blockIdx.x * kTileM;                                                  \
    n0 = (int)blockIdx.y * args.tile_n;                                             \
  }
  // blockIdx.z: reduction slice of a split reduction, or the group of a grouped convolution (never both)
  const int grp = args.groups > 1 ? (int)blockIdx.z : 0;
  const unsigned zslice = args.groups > 1 ? 0u : blockIdx.z;
  const int kb_begin = (int)(zslice * (unsigned)args.num_kb / (unsigned)args.split_k);
  const int kb_end = (int)((zslice + 1u) * (unsigned)args.num_kb / (unsigned)args.split_k);
  const int stages = args.stages;
  const int bk = args.bk;
  const uint32_t a_stage_bytes = AMODE == A_SHIFT ? (uint32_t)args.sh_win_bytes : (uint32_t)(kTileM * bk);
  const uint32_t b_stage_bytes = args.tile_n * bk;

  // Stage buffers start on a 1024-byte boundary (the 128-byte swizzle repeats every 1024 bytes).
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base;
  const uint32_t b_base = smem_base + stages * a_stage_bytes;
  uint8_t* smem_aligned = smem_raw + (smem_base - smem_u32(smem_raw));
  uint8_t* smem_extra = smem_aligned + args.stage_region;
  GatherEntry* s_table = reinterpret_cast<GatherEntry*>(smem_extra);              // A_GATHER
  int32_t* s_table32 = reinterpret_cast<int32_t*>(smem_extra);                    // A_STAGED
  uint8_t* s_window = smem_extra + ((args.table_len * 4 + 15) & ~15);             // A_STAGED
  constexpr bool kThreadsFormA = (AMODE == A_GATHER || AMODE == A_STAGED);
  // A 16-column tile is drained by one warp per lane quadrant; the four warps of the second column
  // half then have nothing to do (unless the threads also form the A operand) and stay out of the
  // tile loop, so that they neither poll the barriers nor count in the accumulator hand-back.
  const bool second_half_idle = !kThreadsFormA && args.tile_n < 32;
  // Shift execution with two accumulator buffers: the two warps of a lane quadrant take turns, one
  // draining the even tiles of the block's walk (buffer 0), the other the odd ones (buffer 1), each
  // all columns of its tile.  The work per warp is the same as with split columns, but the per-tile
  // fixed cost (barrier wait, tile coordinates, hand-back) is paid for every second tile only.
  const bool alternate = persistent && AMODE == A_SHIFT && args.tmem_bufs >= 2;
  const int epilogue_warps = (second_half_idle || alternate) ? kGatherWarps / 2 : kGatherWarps;

  if (warp == 0) {
    if (lane < stages) {
      mbar_init(smem_u32(&ctl.full[lane]), kThreadsFormA ? 1 + kGatherWarps : 1);
      mbar_init(smem_u32(&ctl.empty[lane]), 1);
    }
    if (lane == 8) {
      mbar_init(smem_u32(&ctl.tmem_full[0]), 1);
      if (persistent) {
        for (int b = 1; b < 4; ++b) mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
        for (int b = 0; b < 4; ++b) mbar_init(smem_u32(&ctl.tmem_empty[b]), epilogue_warps);
      }
      ctl.abort_flag = 0;
    }
    if (lane == 11 && AMODE == A_SHIFT) mbar_init(smem_u32(&ctl.full[7]), 1);  // resident weights have landed
    if (lane == 9 && !kThreadsFormA) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_a) : "memory");
    if (lane == 10) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                 "r"(args.tmem_cols * nbuf)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (AMODE == A_GATHER) {
    for (int i = threadIdx.x; i < args.table_len; i += kThreads) s_table[i] = args.table[i];
  }
  if (AMODE == A_STAGED) {
    for (int i = threadIdx.x; i < args.table_len; i += kThreads) s_table32[i] = args.table32[i];
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = __shfl_sync(0xffffffffu, ctl.tmem_base, 0);  // same value in every lane, provably
  // Everything above touched only kernel parameters, shared memory and the plan's constant lookup
  // table.  From here on the block reads tensors earlier kernels of the stream produce and writes
  // tensors they may still read.
  pdl_wait();
  pdl_launch_dependents();

  // The loops below keep stage index, phase bit, tap position and addresses as running
  // counters: each role is a single thread, so every integer division in a loop body would
  // cost hundreds of cycles of dependent issue.
  // Which of the two single-thread roles sits in warp 0 and which in warp 1.  The warp that issues
  // the MMAs holds up the other warps of its scheduler while it issues (a per-role clock timeline
  // shows the epilogue warp with the same warp index modulo 4 finishing about one MMA-issue time
  // after its siblings), so blocks that walk tiles side by side on one SM put it on different
  // schedulers: persistent grids are sized in multiples of the SM count, and blocks b, b + 148, ..
  // are taken to share an SM.
  const int mma_warp = persistent ? 1 - (int)((blockIdx.x / kNumSMs) & 1u) : 1;
  const int producer_warp = 1 - mma_warp;
  if (warp == producer_warp) {
    // ---------------------------------------------------------------- TMA producer
    int s = 0;
    uint32_t ph = 0;
    uint32_t a_dst = a_base, b_dst = b_base;
    const uint32_t leader = elect_one() ? 1u : 0u;
    bool alive = true;
    if (AMODE == A_SHIFT) {
      // Resident weights: one box [bk bytes x tile_n channels] per (tap, channel block), once.
      const uint32_t wfull = smem_u32(&ctl.full[7]);
      const int taps = args.sh_R * args.S;
      mbar_arrive_expect_tx(wfull, (uint32_t)args.sh_w_bytes, leader);
      uint32_t w_dst = b_base;
      for (int tap = 0; tap < taps; ++tap)
        for (int cblk = 0; cblk < args.sh_ncb; ++cblk) {
          tma_load_2d(w_dst, &tmap_b, tap * args.tap_cols + cblk * bk, 0, wfull, leader);
          w_dst += b_stage_bytes;
        }
      // One window per tile: the sh_rows padded image rows from the row that holds the tile's first
      // position on, each row by one copy per channel block (zeros outside the image).
      const uint32_t win_tx = (uint32_t)(args.sh_ncb * args.sh_rows * args.sh_row_bytes);
      for (int t = tile_first; t < tile_end; t += tile_step) {
        const uint32_t pos0 = (uint32_t)t * kTileM;
        const uint32_t row0 = args.div_wps.div(pos0);
        int n = (int)args.div_hp.div(row0);
        int hp = (int)row0 - n * args.sh_hp;
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status))) break;
        const uint32_t full = smem_u32(&ctl.full[s]);
        mbar_arrive_expect_tx(full, win_tx, leader);
        uint32_t dst = a_base + s * a_stage_bytes;
        if (args.remap == 3) {
          // two-dimensional tile (image, tile row, tile column): the window is one box of sh_rows rows
          // of sh_wps pixels per channel block, from the tile's first window origin on
          const int img = (int)args.div_tiles_hw.div((uint32_t)t);
          const int rem = t - img * (args.sh_tiles_h * args.sh_tiles_w);
          const int th = (int)args.div_tiles_w.div((uint32_t)rem), tw = rem - th * args.sh_tiles_w;
          for (int cblk = 0; cblk < args.sh_ncb; ++cblk)
            tma_load_tiled_4d(dst + cblk * args.sh_cblk_bytes, &tmap_a, cblk * bk, tw * args.sh_valid_w - args.pad_w,
                              th * (kTileM / args.sh_wps) - args.pad_h, img,
                              full, leader);
        } else
        for (int j = 0; j < args.sh_rows; ++j) {
          for (int cblk = 0; cblk < args.sh_ncb; ++cblk)
            tma_load_tiled_4d(dst + cblk * args.sh_cblk_bytes, &tmap_a, cblk * bk, -args.pad_w, hp - args.pad_h, n, full,
                              leader);
          dst += args.sh_row_bytes;
          if (++hp == args.sh_hp) {
            hp = 0;
            ++n;
          }
        }
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
        }
      }
      alive = false;  // the generic stage loop below is not used
    }
    for (int t = tile_first; t < tile_end && alive; t += tile_step) {
      B2C_TILE_ORIGIN(t)
      int n_img = 0, h_org = 0, w_org = 0, cb = 0, sx = 0, r = 0;
      // Swapped axis map: the activations are the N operand (tile_n pixels from n0 on, into the B
      // region) and the packed weights the 128-row operand (rows m0 .., into the A region).
      const bool swap = args.swap != 0;
      const int pix0 = swap ? n0 : m0;
      const int wrow0 = swap ? m0 : n0;
      if (AMODE == A_IM2COL_TMA) {
        n_img = (int)args.div_pq.div((uint32_t)pix0);
        const int rem = pix0 - n_img * args.PQ;
        const int p = (int)args.div_q.div((uint32_t)rem), q = rem - p * args.Q;
        h_org = p * args.stride_h - args.pad_h;
        w_org = q * args.stride_w - args.pad_w;
        const int tap = kb_begin / args.kb_per_tap;
        cb = kb_begin - tap * args.kb_per_tap;
        r = tap / args.S;
        sx = tap - r * args.S;
      }
      int kcol = kb_begin * bk;  // column of the packed weight matrix = reduction offset in bytes
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status))) {
          alive = false;
          break;
        }
        const uint32_t full = smem_u32(&ctl.full[s]);
        if (kThreadsFormA) {
          mbar_arrive_expect_tx(full, b_stage_bytes, leader);
          tma_load_2d(b_dst, &tmap_b, kcol, n0 + grp * args.K, full, leader);
        } else if (AMODE == A_TILED) {
          mbar_arrive_expect_tx(full, a_stage_bytes + b_stage_bytes, leader);
          tma_load_2d(swap ? b_dst : a_dst, &tmap_a, kcol, pix0, full, leader);
          tma_load_2d(swap ? a_dst : b_dst, &tmap_b, kcol, wrow0, full, leader);
        } else {
          mbar_arrive_expect_tx(full, a_stage_bytes + b_stage_bytes, leader);
          tma_load_im2col_4d(swap ? b_dst : a_dst, &tmap_a, cb * bk, w_org, h_org, n_img, full,
                             (uint16_t)(sx * args.dil_w), (uint16_t)(r * args.dil_h), leader);
          tma_load_2d(swap ? a_dst : b_dst, &tmap_b, kcol, wrow0, full, leader);
          if (++cb == args.kb_per_tap) {
            cb = 0;
            if (++sx == args.S) {
              sx = 0;
              ++r;
            }
          }
        }
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
  } else if (warp == mma_warp) {
    // ---------------------------------------------------------------- MMA issuer
    {
      const uint32_t idesc = make_idesc_i8(args.tile_n);
      const uint64_t adesc0 = make_smem_desc(a_base, bk);
      const uint64_t bdesc0 = make_smem_desc(b_base, bk);
      const uint64_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;
      uint64_t adesc = adesc0, bdesc = bdesc0;
      int s = 0;
      uint32_t ph = 0;
      // The same lane issues every MMA and the commits that track them.
      const uint32_t leader = elect_one() ? 1u : 0u;
      bool alive = true;
      int ti = 0;
      if (AMODE == A_SHIFT) {
        // Stencil as operand shift: all taps of a tile are issued from one staged window, the A
        // descriptor moving (r*dil_h*sh_wps + s*dil_w) pixels per tap, the B descriptor walking the
        // resident weight tiles.
        alive = __all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[7]), 0u, &ctl, args.status));
        const uint32_t cblk_steps = (uint32_t)(bk / kMmaK);
        const uint64_t a_r_step = (uint64_t)((uint32_t)(args.dil_h * args.sh_wps * bk) >> 4);
        const uint64_t a_s_step = args.S == 1 ? a_r_step : (uint64_t)((uint32_t)(args.dil_w * bk) >> 4);
        const uint64_t a_c_step = (uint64_t)((uint32_t)args.sh_cblk_bytes >> 4);
        // (in registers: the loops below are one thread's dependent chain.  A view with one tap per
        // filter row walks its rows as the taps of a single run, so that they share asm blocks.)
        const bool rows_as_taps = args.S == 1;
        const int sh_R = rows_as_taps ? 1 : args.sh_R, sh_S = rows_as_taps ? args.sh_R : args.S, sh_ncb = args.sh_ncb;
        for (int t = tile_first; t < tile_end && alive; t += tile_step, ++ti) {
          const int buf = ti & (nbuf - 1);
          const uint32_t use = (uint32_t)(ti >> nbuf_log2);
          // (votes: the outcome of a wait is the same for all lanes, and saying so keeps the loop's
          // control flow, and with it the descriptor arithmetic, warp-uniform for the compiler)
          if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.tmem_empty[buf]), (use & 1u) ^ 1u, &ctl, args.status))) break;
          if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, args.status))) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t d_tmem = tmem_acc + (uint32_t)(buf * args.tmem_cols);
          const uint32_t pos0 = (uint32_t)t * kTileM;
          const uint32_t rel = pos0 - args.div_wps.div(pos0) * (uint32_t)args.sh_wps;
          // descriptors advance by address deltas in 16-byte units: per filter row, per tap, per
          // channel block, per 32-byte slice
          uint64_t a_row = make_smem_desc(a_base + s * a_stage_bytes + rel * (uint32_t)bk, bk);
          uint64_t bdesc = bdesc0;
          uint32_t accumulate = 0;
          if (sh_ncb == 1 && cblk_steps == 1) {
            // one MMA per tap: runs of up to four taps of a filter row per asm block
            for (int r = 0; r < sh_R; ++r) {
              uint64_t a_tap = a_row;
              for (int sx = 0; sx < sh_S; sx += 4) {
                mma_i8_run4(d_tmem, a_tap, a_s_step, bdesc, b_step, idesc, accumulate, leader, sh_S - sx);
                accumulate = 1;
                a_tap += 4 * a_s_step;
                bdesc += 4 * b_step;
              }
              bdesc -= (uint64_t)((4 - (sh_S & 3)) & 3) * b_step;  // the last run of a row may be short
              a_row += a_r_step;
            }
          } else if (sh_ncb == 1 && cblk_steps == 2) {
            // two MMAs per tap: two taps of a filter row per asm block
            for (int r = 0; r < sh_R; ++r) {
              uint64_t a_tap = a_row;
              for (int sx = 0; sx < sh_S; sx += 2) {
                mma_i8_pair2(d_tmem, a_tap, a_s_step, bdesc, b_step, idesc, accumulate, leader, sh_S - sx);
                accumulate = 1;
                a_tap += 2 * a_s_step;
                bdesc += 2 * b_step;
              }
              bdesc -= (uint64_t)(sh_S & 1) * b_step;  // the last pair of a row may be a single tap
              a_row += a_r_step;
            }
          } else {
            // per tap and channel block: the 32-byte slices of one swizzle row as one asm block
            for (int r = 0; r < sh_R; ++r) {
              uint64_t a_tap = a_row;
              for (int sx = 0; sx < sh_S; ++sx) {
                uint64_t a_c = a_tap;
                for (int cblk = 0; cblk < sh_ncb; ++cblk) {
                  mma_i8_block(d_tmem, a_c, bdesc, idesc, accumulate, leader, (int)cblk_steps);
                  accumulate = 1;
                  a_c += a_c_step;
                  bdesc += b_step;
                }
                a_tap += a_s_step;
              }
              a_row += a_r_step;
            }
          }
          mma_commit(smem_u32(&ctl.empty[s]), leader);
          mma_commit(smem_u32(&ctl.tmem_full[buf]), leader);
          if (++s == stages) {
            s = 0;
            ph ^= 1u;
          }
        }
        alive = false;  // the generic stage loop below is not used
      }
      for (int t = tile_first; t < tile_end && alive; t += tile_step, ++ti) {
      const int buf = persistent ? (ti & (nbuf - 1)) : 0;
      const uint32_t use = persistent ? (uint32_t)(ti >> nbuf_log2) : 0u;
      if (persistent) {
        // the epilogue must have drained this accumulator buffer (first use passes at once)
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.tmem_empty[buf]), (use & 1u) ^ 1u, &ctl, args.status))) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      }
      const uint32_t d_tmem = tmem_acc + (uint32_t)(buf * args.tmem_cols);
      uint32_t accumulate = 0;
      bool ready = false;  // result of the look-ahead test of this stage's full barrier
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!ready && !__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[s]), ph, &ctl, args.status))) {
          alive = false;
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int ksteps = (kb == args.num_kb - 1) ? args.ksteps_last : args.ksteps_full;
        const int s_cur = s;
        const uint64_t a_cur = adesc, b_cur = bdesc;
        adesc += a_step;
        bdesc += b_step;
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
          adesc = adesc0;
          bdesc = bdesc0;
        }
        // Look ahead: test the next stage's barrier now so that its latency overlaps the MMA issue.
        ready = (kb + 1 < kb_end) && __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl.full[s]), ph));
        mma_i8_block(d_tmem, a_cur, b_cur, idesc, accumulate, leader, ksteps);
        mma_commit(smem_u32(&ctl.empty[s_cur]), leader);
        if (kb == kb_end - 1) mma_commit(smem_u32(&ctl.tmem_full[buf]), leader);
        accumulate = 1;
      }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- gather + epilogue warps
    const int quad = warp & 3;          // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;   // two warps share a quadrant and split the columns / chunks
    const int row = quad * 32 + lane;   // accumulator row = A-tile row
    bool ok = alternate || !(second_half_idle && half == 1);
    int ti = 0;
    int s = 0;         // stage ring position of the A-forming threads (runs on across tiles)
    uint32_t ph = 0;
    // two-dimensional tiles: the pixel of this row inside a tile does not change from tile to tile
    // (the tile width is a power of two)
    const int tile_w_log2 = args.remap == 3 ? 31 - __clz(args.sh_wps) : 0;
    const int tile_h3 = kTileM >> tile_w_log2;
    const int row_in_tile = row >> tile_w_log2, col_in_tile = row & ((1 << tile_w_log2) - 1);
    for (int t = tile_first; t < tile_end && ok; t += tile_step, ++ti) {
    if (alternate && (ti & 1) != half) continue;
    B2C_TILE_ORIGIN(t)
    const unsigned m = (unsigned)m0 + (unsigned)row;
    bool row_valid = m < (unsigned)(args.swap ? args.K : args.Mg);
    int n_img = 0, pq = 0;
    if (row_valid && !args.swap && args.remap < 2) {
      n_img = (int)args.div_pq.div(m);
      pq = (int)(m - (unsigned)n_img * (unsigned)args.PQ);
    }
    // Where this row's results go: (out_img, out_pq) in the convolution's own output.  The phase
    // pack interleaves the sub-image results back and drops rows that fall outside the output.
    int out_img = n_img, out_pq = pq;
    if (args.remap == 3 && row_valid) {
      // two-dimensional tiles: tile (image, tile row, tile column), row = pixel (row / 16, row % 16) of it
      const uint32_t tile = (uint32_t)m0 / kTileM;
      out_img = (int)args.div_tiles_hw.div(tile);
      const int rem = (int)tile - out_img * (args.sh_tiles_h * args.sh_tiles_w);
      const int th = (int)args.div_tiles_w.div((uint32_t)rem), tw = rem - th * args.sh_tiles_w;
      const int po = th * tile_h3 + row_in_tile, qo = tw * args.sh_valid_w + col_in_tile;
      row_valid = col_in_tile < args.sh_valid_w && po < args.out_P && qo < args.out_Q;
      out_pq = po * args.out_Q + qo;
    } else if (args.remap == 2 && row_valid) {
      // shift execution: row m is window origin (n, hp, wp) on the padded grid of sh_hp x sh_wps positions
      const uint32_t rowi = args.div_wps.div(m);
      const int wp = (int)(m - rowi * (uint32_t)args.sh_wps);
      out_img = (int)args.div_hp.div(rowi);
      const int hp = (int)rowi - out_img * args.sh_hp;
      row_valid = hp < args.out_P && wp < args.out_Q;
      out_pq = hp * args.out_Q + wp;
    } else if (args.remap && row_valid) {
      const int ps = (int)args.div_q.div((uint32_t)pq), qs = pq - ps * args.Q;
      const int phases = args.ph_dh * args.ph_dw;
      out_img = n_img / phases;
      const int ph = n_img - out_img * phases;
      const int a = ph / args.ph_dw, b = ph - a * args.ph_dw;
      const int po = (ps - args.ph_pad_h) * args.ph_dh + a + args.out_pad_h;
      const int qo = (qs - args.ph_pad_w) * args.ph_dw + b + args.out_pad_w;
      row_valid = (unsigned)po < (unsigned)args.out_P && (unsigned)qo < (unsigned)args.out_Q;
      out_pq = po * args.out_Q + qo;
    }

    if (AMODE == A_GATHER) {
      // Stencil unroll formed in place: this thread writes half of row `row` of the A tile (four
      // 16-byte chunks per stage) in the 128-byte swizzled order the MMA descriptor expects
      // (chunk j of row r lives at chunk position j ^ (r & 7)).
      const int p = (int)args.div_q.div((uint32_t)pq), q = pq - p * args.Q;
      const int h0 = row_valid ? p * args.stride_h - args.pad_h : -(1 << 29);
      const int w0 = q * args.stride_w - args.pad_w;
      const int8_t* base = args.x + grp * args.group_x_stride + n_img * args.x_stride_n + (long long)(row_valid ? h0 : 0) * args.x_stride_h +
                           (long long)w0 * args.x_stride_w;
      const uint32_t row_off = (uint32_t)row * 128u;
      const uint32_t xr = (uint32_t)(row & 7);
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status)) {
          ok = false;
          break;
        }
        const uint32_t a_row = a_base + s * a_stage_bytes + row_off;
        const int chunks = (kb == args.num_kb - 1) ? args.ksteps_last * 2 : 8;
        const GatherEntry* te = s_table + kb * 128 + half * 64;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
          const int j = half * 4 + jj;
          if (j < chunks) {
            uint32_t wv[4] = {0, 0, 0, 0};
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const GatherEntry g = te[jj * 16 + e];
              const int h = h0 + g.dh, ww = w0 + g.dw;
              uint32_t v = 0;
              if (g.off >= 0 && (unsigned)h < (unsigned)args.H && (unsigned)ww < (unsigned)args.W &&
                  B2C_X_OK(args.dbg, 30, base + g.off, 1))
                v = (uint8_t)__ldg(base + g.off);
              wv[e >> 2] |= v << (8 * (e & 3));
            }
            const uint32_t dst = a_row + ((((uint32_t)j) ^ xr) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]),
                         "r"(wv[3]));
          }
        }
        // Make the generic-proxy writes visible to the tensor core's async proxy, then one lane
        // signals for the whole warp.
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl.full[s]));
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
        }
      }
    }

    if (AMODE == A_STAGED) {
      // Stencil unroll from a staged window.  First the 256 threads copy, for every image the tile
      // touches, the input rows its output pixels need into shared memory as a zero-padded window
      // (rows outside the image and the left/right margins are zeros, so the gather below needs no
      // bounds tests); then each thread forms half a row of the A tile per stage from that window.
      const int tg = (int)threadIdx.x - 64;
      // (persistent blocks: every thread must be done reading the previous tile's window)
      if (ti > 0) asm volatile("bar.sync 1, %0;" ::"n"(kGatherWarps * 32) : "memory");
      const unsigned m_last = min((unsigned)m0 + (unsigned)kTileM - 1u, (unsigned)args.Mg - 1u);
      const int img0 = (int)args.div_pq.div((uint32_t)m0);
      const int p_first = (int)args.div_q.div((uint32_t)(m0 - img0 * args.PQ));
      const int img1 = (int)args.div_pq.div(m_last);
      const int p_last = (int)args.div_q.div(m_last - (unsigned)img1 * (unsigned)args.PQ);
      const int parts = img1 - img0 + 1;
      const int wp = args.win_pitch, wr = args.win_rows, C = args.C;
      const int vec_per_row = wp >> 4;
      const int slots = parts * C * wr;
      const bool vec_ok = (args.W & 15) == 0 && (reinterpret_cast<uintptr_t>(args.x) & 15) == 0;
      for (int idx = tg; idx < slots * vec_per_row; idx += kGatherWarps * 32) {
        const int slot = (int)args.div_vec_per_row.div((uint32_t)idx);
        const int v16 = idx - slot * vec_per_row;
        const int part = (int)args.div_c_rows.div((uint32_t)slot);
        const int cj = slot - part * (C * wr);
        const int c = (int)args.div_rows.div((uint32_t)cj);
        const int j = cj - c * wr;
        const int pl = part == 0 ? p_first : 0;
        const int ph_ = part == parts - 1 ? p_last : args.P - 1;
        const int h = pl * args.stride_h - args.pad_h + j;
        const bool row_live = j <= (ph_ - pl) * args.stride_h + args.win_tap_span && (unsigned)h < (unsigned)args.H;
        const int col0 = v16 * 16 - args.win_left;  // image column of the first byte of this vector
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row_live && col0 < args.W && col0 + 16 > 0) {
          const int8_t* src = args.x + grp * args.group_x_stride + (size_t)(img0 + part) * args.x_stride_n + ((size_t)c * args.H + h) * args.W + col0;
          if (vec_ok && col0 >= 0 && col0 + 16 <= args.W) {
            if (B2C_X_OK(args.dbg, 31, src, 16)) val = __ldg(reinterpret_cast<const uint4*>(src));
          } else {
            uint32_t wv[4] = {0, 0, 0, 0};
            for (int b = 0; b < 16; ++b)
              if ((unsigned)(col0 + b) < (unsigned)args.W && B2C_X_OK(args.dbg, 31, src + b, 1))
                wv[b >> 2] |= (uint32_t)(uint8_t)__ldg(src + b) << (8 * (b & 3));
            val = make_uint4(wv[0], wv[1], wv[2], wv[3]);
          }
        }
        *reinterpret_cast<uint4*>(s_window + (size_t)slot * wp + v16 * 16) = val;
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kGatherWarps * 32) : "memory");

      // window position of this pixel's first tap (r = s = 0, c = 0)
      int wbase = -1;
      if (row_valid) {
        const int p = (int)args.div_q.div((uint32_t)pq), q = pq - p * args.Q;
        const int part = n_img - img0;
        const int pl = part == 0 ? p_first : 0;
        wbase = (part * C * wr + (p - pl) * args.stride_h) * wp + args.win_left + q * args.stride_w - args.pad_w;
      }
      const uint32_t row_off = (uint32_t)row * 128u;
      const uint32_t xr = (uint32_t)(row & 7);
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!mbar_wait(smem_u32(&ctl.empty[s]), ph ^ 1u, &ctl, args.status)) {
          ok = false;
          break;
        }
        const uint32_t a_row = a_base + s * a_stage_bytes + row_off;
        const int chunks = (kb == args.num_kb - 1) ? args.ksteps_last * 2 : 8;
        if (args.win_word_mode) {
          // Unit horizontal dilation: the S taps of a (c, r) run are consecutive window bytes.  Runs
          // are padded to a multiple of 4 (the packed weights hold zeros there), so every 32-bit
          // word of the A row is one unaligned word of the window: two aligned loads and a byte
          // permute whose selector depends only on this pixel's window alignment.
          const int32_t* te = s_table32 + kb * 32 + half * 16;
          const uint32_t sel = 0x3210u + 0x1111u * ((uint32_t)wbase & 3u);
          const uint8_t* wrow = s_window + (wbase & ~3);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = half * 4 + jj;
            if (j < chunks) {
              uint32_t wv[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int off = te[jj * 4 + e];
                uint32_t v = 0;
                if (off >= 0 && wbase >= 0) {
                  const uint32_t lo = *reinterpret_cast<const uint32_t*>(wrow + off);
                  const uint32_t hi = *reinterpret_cast<const uint32_t*>(wrow + off + 4);
                  v = __byte_perm(lo, hi, sel);
                }
                wv[e] = v;
              }
              const uint32_t dst = a_row + ((((uint32_t)j) ^ xr) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]),
                           "r"(wv[3]));
            }
          }
        } else {
          const int32_t* te = s_table32 + kb * 128 + half * 64;
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = half * 4 + jj;
            if (j < chunks) {
              uint32_t wv[4] = {0, 0, 0, 0};
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                const int off = te[jj * 16 + e];
                uint32_t v = 0;
                if (off >= 0 && wbase >= 0) v = s_window[wbase + off];
                wv[e >> 2] |= v << (8 * (e & 3));
              }
              const uint32_t dst = a_row + ((((uint32_t)j) ^ xr) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]),
                           "r"(wv[3]));
            }
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl.full[s]));
        if (++s == stages) {
          s = 0;
          ph ^= 1u;
        }
      }
    }

    // ---- epilogue ----
    const int buf = persistent ? (ti & (nbuf - 1)) : 0;
    const uint32_t use = persistent ? (uint32_t)(ti >> nbuf_log2) : 0u;
    if (ok) ok = mbar_wait(smem_u32(&ctl.tmem_full[buf]), use & 1u, &ctl, args.status);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
      // Output index of (m, k): NKPQ -> (n*K + k)*PQ + pq ; NPQK -> m*K + k.
      const long long base_nkpq = (long long)out_img * args.y_stride_n + out_pq + (long long)grp * args.K * args.out_PQ;
      const long long base_npqk = args.remap ? ((long long)out_img * args.out_PQ + out_pq) * args.K : (long long)m * args.K;
      const int cols = alternate ? args.tile_n : (args.tile_n >= 32 ? (args.tile_n >> 1) : 16);  // columns handled by this warp
      const int c_begin = alternate ? 0 : half * cols;
      if (c_begin < args.tile_n) {
        const uint32_t taddr =
            tmem_acc + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * args.tmem_cols) + (uint32_t)c_begin;
        // cluster reduction: the stage buffers are free once the accumulator is complete
        const uint32_t xch = args.cluster_split ? a_base + (uint32_t)row * 4u + (uint32_t)c_begin * (kTileM * 4) : 0u;
        if (args.swap) {
          // accumulator row = output channel m, columns = pixels n0 + c_begin ..
          for (int c = 0; c < cols; c += 16) {
            int32_t v[16];
            __syncwarp();
            tmem_ld<16>(taddr + (uint32_t)c, v);
            store_columns_swapped(args, v, (int)m, row_valid, n0 + c_begin + c);
          }
        } else if ((cols & 31) == 0) {
          for (int c = 0; c < cols; c += 32)
            epilogue_columns<32>(args, taddr + (uint32_t)c, n0 + c_begin + c, row_valid, base_nkpq, base_npqk,
                                 xch ? xch + (uint32_t)c * (kTileM * 4) : 0u, grp * args.K);
        } else {
          for (int c = 0; c < cols; c += 16)
            epilogue_columns<16>(args, taddr + (uint32_t)c, n0 + c_begin + c, row_valid, base_nkpq, base_npqk,
                                 xch ? xch + (uint32_t)c * (kTileM * 4) : 0u, grp * args.K);
        }
      }
      if (persistent) {
        // this warp has read its part of the accumulator buffer: hand it back to the MMA warp
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
      }
    }
    }  // tile loop
  }

  if (args.cluster_split) {
    B2C_TILE_ORIGIN(0)
    // ---------------------------------------------------------------- cluster reduction
    // Barrier 1: every slice's partial tile is in its block's shared memory.  Then block `rank`
    // sums columns [rank * tile_n / split, (rank + 1) * tile_n / split) over all slices, applies the
    // epilogue and stores.  Barrier 2: no block leaves while its tile may still be read.
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
    if (warp >= 2 && !ctl.abort_flag) {
      // Lane g owns accumulator rows 4g .. 4g+3 (one 16-byte vector of the [column][row] tile);
      // warp w takes columns w, w + 8, ... of this block's slice.  All vector loads of a batch of
      // columns (from every slice, starting with the own one) are issued before the first add.
      const int cols_slice = args.tile_n / args.split_k;
      const int col_base = (int)blockIdx.z * cols_slice;
      const uint32_t rank = blockIdx.z;
      const unsigned mrow = (unsigned)m0 + 4u * (unsigned)lane;
      // rows of this lane: valid count, image and pixel of the first row, same-image flag
      int n_img = 0, pq = 0;
      if (mrow < (unsigned)args.Mg) {
        n_img = (int)args.div_pq.div(mrow);
        pq = (int)(mrow - (unsigned)n_img * (unsigned)args.PQ);
      }
      const int rows_valid = (int)min(4u, (unsigned)args.Mg > mrow ? (unsigned)args.Mg - mrow : 0u);
      const bool one_image = rows_valid == 4 && pq + 3 < args.PQ;
      const bool nhwc = args.out_layout == B2C_LAYOUT_NHWC;
      constexpr int kBatch = 4;  // columns in flight per thread: kBatch * split vector loads
      for (int cb = warp - 2; cb < cols_slice; cb += kGatherWarps * kBatch) {
        int32_t acc[kBatch][4];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0;
        for (int rr = 0; rr < args.split_k; ++rr) {
          uint32_t r = rank + (uint32_t)rr;
          if (r >= (uint32_t)args.split_k) r -= (uint32_t)args.split_k;
          int32_t t[kBatch][4];
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            const int c = cb + b * kGatherWarps;
            if (c < cols_slice) {
              const uint32_t local = a_base + (uint32_t)(col_base + c) * (kTileM * 4) + (uint32_t)lane * 16u;
              uint32_t remote;
              asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(r));
              asm volatile("ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [%4];"
                           : "=r"(t[b][0]), "=r"(t[b][1]), "=r"(t[b][2]), "=r"(t[b][3])
                           : "r"(remote)
                           : "memory");
            } else {
              t[b][0] = t[b][1] = t[b][2] = t[b][3] = 0;
            }
          }
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            acc[b][0] += t[b][0];
            acc[b][1] += t[b][1];
            acc[b][2] += t[b][2];
            acc[b][3] += t[b][3];
          }
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int c = cb + b * kGatherWarps;
          const int k = n0 + col_base + c;
          if (c >= cols_slice || k >= args.K || rows_valid == 0) continue;
#ifdef B2C_DEBUG_BOUNDS
          {
            // the rows_valid output elements of channel k this lane writes, first and last
            const unsigned m_l = mrow + (unsigned)rows_valid - 1u;
            const int n_l = (int)args.div_pq.div(m_l);
            const long long first = nhwc ? (long long)mrow * args.K + k : ((long long)n_img * args.K + k) * args.PQ + pq;
            const long long last = nhwc ? (long long)m_l * args.K + k
                                        : ((long long)n_l * args.K + k) * args.PQ + (int)(m_l - (unsigned)n_l * (unsigned)args.PQ);
            bool okb = true;
            if (args.out_mode & B2C_OUT_I32) okb = B2C_O32_OK(args.dbg, 32, args.y32 + first, 4) && B2C_O32_OK(args.dbg, 32, args.y32 + last, 4);
            if (okb && (args.out_mode & B2C_OUT_I8)) okb = B2C_O8_OK(args.dbg, 33, args.y8 + first, 1) && B2C_O8_OK(args.dbg, 33, args.y8 + last, 1);
            if (!okb) continue;
          }
#endif
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[b][i] = activate(args, acc[b][i], k);
          if (!nhwc && one_image) {
            // four consecutive pixels of one image and one channel: contiguous in NKPQ
            const long long o = ((long long)n_img * args.K + k) * args.PQ + pq;
            if (args.out_mode & B2C_OUT_I32) {
              int32_t* dst = args.y32 + o;
              if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
                *reinterpret_cast<int4*>(dst) = make_int4(acc[b][0], acc[b][1], acc[b][2], acc[b][3]);
              } else {
                dst[0] = acc[b][0]; dst[1] = acc[b][1]; dst[2] = acc[b][2]; dst[3] = acc[b][3];
              }
            }
            if (args.out_mode & B2C_OUT_I8) {
              int8_t* dst = args.y8 + o;
              const uint32_t q4 = (uint32_t)(uint8_t)requant(acc[b][0], args.shift) |
                                  ((uint32_t)(uint8_t)requant(acc[b][1], args.shift) << 8) |
                                  ((uint32_t)(uint8_t)requant(acc[b][2], args.shift) << 16) |
                                  ((uint32_t)(uint8_t)requant(acc[b][3], args.shift) << 24);
              if ((reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
                *reinterpret_cast<uint32_t*>(dst) = q4;
              } else {
                dst[0] = (int8_t)(q4 & 0xff); dst[1] = (int8_t)((q4 >> 8) & 0xff);
                dst[2] = (int8_t)((q4 >> 16) & 0xff); dst[3] = (int8_t)(q4 >> 24);
              }
            }
          } else {
            // general case: row by row (image boundary inside the group, tail rows, or NPQK)
            for (int i = 0; i < rows_valid; ++i) {
              const unsigned mi = mrow + (unsigned)i;
              long long o;
              if (nhwc) {
                o = (long long)mi * args.K + k;
              } else {
                const int ni = (int)args.div_pq.div(mi);
                o = ((long long)ni * args.K + k) * args.PQ + (int)(mi - (unsigned)ni * (unsigned)args.PQ);
              }
              if (args.out_mode & B2C_OUT_I32) args.y32[o] = acc[b][i];
              if (args.out_mode & B2C_OUT_I8) args.y8[o] = requant(acc[b][i], args.shift);
            }
          }
        }
      }
    }
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  }

  // ---------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (ctl.abort_flag) {
    // Give copies that were already issued time to land before the shared memory is released.
    if (threadIdx.x == 0) {
      const unsigned long long t0 = global_ns();
      while (global_ns() - t0 < 50000ull) __nanosleep(1000);
    }
    __syncthreads();
  }
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(args.tmem_cols * nbuf)
                 : "memory");
  }
}

// One block waits, with the same bounded wait the convolution kernel uses, on a barrier that
// nothing ever completes.  The wait gives up after its time limit, records B2C_E_TIMEOUT in
// `status` and the kernel returns normally: the context stays usable.
__global__ void bounded_wait_selftest_kernel(int* status) {
  __shared__ SharedCtl ctl;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl.full[0]), 1);
    ctl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  mbar_wait(smem_u32(&ctl.full[0]), 0u, &ctl, status);
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(int* status, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(status);
  return cudaGetLastError();
}

size_t conv_mma_smem_bytes(int amode, const ConvArgs& a) {
  size_t b = 1024 + (size_t)a.stage_region;
  if (amode == A_GATHER) b += (size_t)a.table_len * sizeof(GatherEntry);
  if (amode == A_STAGED) b += (size_t)((a.table_len * 4 + 15) & ~15) + (size_t)a.win_bytes + 16;
  return b;
}

cudaError_t launch_conv_mma(int amode, const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const ConvArgs& args,
                            cudaStream_t st) {
  const size_t smem = conv_mma_smem_bytes(amode, args);
  dim3 grid((unsigned)((args.Mg + kTileM - 1) / kTileM), (unsigned)((args.K + args.tile_n - 1) / args.tile_n),
            (unsigned)args.split_k);
  if (args.swap)
    grid = dim3((unsigned)((args.Mg + args.tile_n - 1) / args.tile_n), (unsigned)((args.K + kTileM - 1) / kTileM),
                (unsigned)args.split_k);
  if (args.persistent) {
    const int per_sm = args.persistent_blocks_per_sm > 0 ? args.persistent_blocks_per_sm : (args.persistent == 2 ? 3 : 1);
    grid = dim3((unsigned)std::min(args.num_tiles, kNumSMs * per_sm), 1, 1);
  }
  if (args.groups > 1) grid.z = (unsigned)args.groups;  // (grouped plans never split the reduction)
  cudaError_t e;
#define B2C_LAUNCH(MODE, PERS)                                                                             \
  {                                                                                                       \
    static std::atomic<unsigned long long> configured{0};                                                 \
    e = set_max_dynamic_smem_once(configured, (const void*)conv_mma_kernel<MODE, PERS>, 200 * 1024);      \
    if (e != cudaSuccess) return e;                                                                       \
    e = launch_pdl_cluster(conv_mma_kernel<MODE, PERS>, grid, dim3(kThreads), smem, st,                   \
                           args.cluster_split ? args.split_k : 1, *tmap_a, *tmap_b, args);                \
    if (e != cudaSuccess) return e;                                                                       \
  }
  if (amode == A_TILED && args.persistent == 1) B2C_LAUNCH(A_TILED, 1)
  else if (amode == A_TILED && args.persistent == 2) B2C_LAUNCH(A_TILED, 2)
  else if (amode == A_TILED) B2C_LAUNCH(A_TILED, 0)
  else if (amode == A_IM2COL_TMA && args.persistent == 1) B2C_LAUNCH(A_IM2COL_TMA, 1)
  else if (amode == A_IM2COL_TMA && args.persistent == 2) B2C_LAUNCH(A_IM2COL_TMA, 2)
  else if (amode == A_IM2COL_TMA) B2C_LAUNCH(A_IM2COL_TMA, 0)
  else if (amode == A_SHIFT) B2C_LAUNCH(A_SHIFT, 2)
  else if (amode == A_STAGED && args.persistent == 2) B2C_LAUNCH(A_STAGED, 2)
  else if (amode == A_STAGED) B2C_LAUNCH(A_STAGED, 0)
  else B2C_LAUNCH(A_GATHER, 0)
#undef B2C_LAUNCH
#undef B2C_TILE_ORIGIN
  return cudaGetLastError();
}

}  // namespace b2c
