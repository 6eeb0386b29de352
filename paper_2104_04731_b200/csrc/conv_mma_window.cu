// Stencil unroll (Table 2, rule 1) formed inside the kernel from a TMA-staged input window, for the
// low-channel shapes of Section 6.1 (ic = 1, ic = 3), where padding the channel axis to the
// intrinsic's reduction depth wastes almost all of it and only the fused (c, r, s) axis gives a
// usable reduction dimension.
//
// Tile = tile_h x tile_w output pixels of one image (tile_h * tile_w = 128, tile_w a power of two).
// The input patch those pixels read, C channels x win_h rows x win_w bytes, reaches shared memory by
// ONE tiled TMA copy of the NCHW tensor (zeros outside the image: the spatial padding is never
// materialised).  Eight builder warps then write the A operand of the tile, 128 rows of
// K_pad = pad32(C * R * S_run) bytes in the 128-byte-swizzled K-major layout the MMA descriptor
// expects: the S taps of a (c, r) run are consecutive window bytes, runs are padded to a multiple of
// 4 (S_run), so every 32-bit word of an A row is one unaligned word of the window (two aligned loads,
// of which consecutive words share one, and a byte permute).  Columns that are padding of a run or of
// the reduction axis are never cleared: the packed weights are zero there, and any int8 times zero is
// zero.  The packed weights stay resident in shared memory; one warp issues the MMAs; four epilogue
// warps drain the accumulators (activation step, shift / clip, NKPQ or NPQK stores), so that the
// operand build of tile t + 1, the MMAs of tile t and the stores of tile t - 1 overlap.
// Small images (LINEAR form): when a whole image of C x H x W bytes is a multiple of 16 bytes and a few
// KB, tiles are 128 consecutive fused (n, p, q) pixels instead, the window is the whole images those
// pixels belong to, each fetched by one bulk copy of the NCHW tensor as it is (no zero padding in
// shared memory), and the builders clear the taps that fall outside the image with per-row masks
// (a bit per filter row, a byte mask per word of a run) computed once per tile and row.
// Every wait is bounded as in the other kernels.
#include <algorithm>

#include "conv_mma_common.cuh"

namespace b2c {

namespace {

constexpr int kBuildWarps = 8;   // warps 2..9
constexpr int kEpiWarps = 4;     // warps 10..13 (one per tensor-memory lane quadrant)
constexpr int kWinThreads = 64 + 32 * (kBuildWarps + kEpiWarps);
constexpr int kWinStages = kWindowStages;  // input windows in flight
constexpr int kABufs = 2;        // A operand buffers

// Bounded wait with back-off: the roles of this kernel wait for whole tiles (a microsecond or so), and
// fourteen warps polling shared-memory barriers compete with the builders for the same memory pipe, so
// a waiting warp sleeps between polls.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, SharedCtl* ctl, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  while (true) {
    __nanosleep(100);
    if (mbar_try_wait(bar, parity)) return true;
    if (ctl->abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) {
      ctl->abort_flag = 1;
      atomicCAS(status, 0, B2C_E_TIMEOUT);
      return false;
    }
  }
}

static_assert(kWinStages <= 8, "one lane per window barrier");
struct __align__(8) WindowCtl {
  unsigned long long win_full[kWinStages];
  unsigned long long win_empty[kWinStages];
  unsigned long long a_full[kABufs];
  unsigned long long a_empty[kABufs];
  unsigned long long tmem_full[4];
  unsigned long long tmem_empty[4];
  unsigned long long w_full;
  SharedCtl base;  // abort flag and tensor-memory base (the bounded waits take this)
};

template <bool LINEAR>
__global__ void __launch_bounds__(kWinThreads, 2)
    conv_mma_window_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b,
                           const ConvArgs args) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ WindowCtl wc;
  SharedCtl* ctl = &wc.base;

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const int nkb = args.num_kb;                         // 128-byte reduction blocks of a tile
  const uint32_t a_block_bytes = kTileM * 128u;        // one reduction block of A
  const uint32_t a_buf_bytes = (uint32_t)nkb * a_block_bytes;
  const uint32_t b_block_bytes = (uint32_t)args.tile_n * 128u;
  const uint32_t win_bytes = (uint32_t)args.wn_win_bytes;  // one window buffer (multiple of 128)
  const int nbuf = args.tmem_bufs;                     // accumulator ring: 2 or 4
  const int nbuf_log2 = nbuf == 4 ? 2 : 1;

  // shared memory: [A buffers][resident weights][window ring][word table]
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_aligned = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t a_base = smem_base;
  const uint32_t b_base = a_base + kABufs * a_buf_bytes;
  const uint32_t win_base = b_base + (uint32_t)nkb * b_block_bytes;
  uint8_t* win_ptr = smem_aligned + (win_base - smem_base);
  const int32_t* s_table = reinterpret_cast<const int32_t*>(win_ptr + kWinStages * win_bytes);

  if (warp == 0) {
    if (lane < kWinStages) {
      mbar_init(smem_u32(&wc.win_full[lane]), 1);
      mbar_init(smem_u32(&wc.win_empty[lane]), kBuildWarps);
    }
    if (lane >= 8 && lane < 8 + kABufs) {
      mbar_init(smem_u32(&wc.a_full[lane - 8]), kBuildWarps);
      mbar_init(smem_u32(&wc.a_empty[lane - 8]), 1);
    }
    if (lane >= 12 && lane < 16) {
      mbar_init(smem_u32(&wc.tmem_full[lane - 12]), 1);
      mbar_init(smem_u32(&wc.tmem_empty[lane - 12]), kEpiWarps);
    }
    if (lane == 16) {
      mbar_init(smem_u32(&wc.w_full), 1);
      ctl->abort_flag = 0;
    }
    if (lane == 17) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    if (lane == 18) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_b) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(args.tmem_cols * nbuf)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // word table: reduction word -> byte offset inside the window (plan constant, not written by any kernel)
  {
    int32_t* t = reinterpret_cast<int32_t*>(win_ptr + kWinStages * win_bytes);
    for (int i = threadIdx.x; i < args.table_len; i += kWinThreads) t[i] = args.table32[i];
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = __shfl_sync(0xffffffffu, ctl->tmem_base, 0);
  pdl_wait();
  pdl_launch_dependents();

  const int tile_first = (int)blockIdx.x, tile_step = (int)gridDim.x, tile_end = args.num_tiles;
  const int tiles_per_image = args.sh_tiles_h * args.sh_tiles_w;
  const int tw_log2 = 31 - __clz(args.wn_tile_w);
  const int tile_h = kTileM >> tw_log2;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    const uint32_t leader = elect_one() ? 1u : 0u;
    // resident weights: one box [128 bytes x tile_n rows] per reduction block
    mbar_arrive_expect_tx(smem_u32(&wc.w_full), (uint32_t)nkb * b_block_bytes, leader);
    for (int kb = 0; kb < nkb; ++kb)
      tma_load_2d(b_base + (uint32_t)kb * b_block_bytes, &tmap_b, kb * 128, 0, smem_u32(&wc.w_full), leader);
    int s = 0;
    uint32_t ph = 0;
    for (int t = tile_first; t < tile_end; t += tile_step) {
      if (!__all_sync(0xffffffffu, mbar_wait_relaxed(smem_u32(&wc.win_empty[s]), ph ^ 1u, ctl, args.status))) break;
      const uint32_t full = smem_u32(&wc.win_full[s]);
      if (LINEAR) {
        // the whole images of the tile's 128 pixels, one bulk copy each, behind the window's margin
        const int m0 = t * kTileM;
        const int n_a = (int)args.div_pq.div((uint32_t)m0);
        const int n_b = (int)args.div_pq.div((uint32_t)min(m0 + kTileM - 1, args.Mg - 1));
        const uint32_t img_bytes = (uint32_t)args.wn_box_bytes;
        int copies = n_b - n_a + 1;
#ifdef B2C_DEBUG_BOUNDS
        for (int n = n_a; n <= n_b; ++n)
          if (!B2C_X_OK(args.dbg, 50, args.x + (size_t)n * img_bytes, img_bytes)) --copies;  // refused below: not expected
#endif
        mbar_arrive_expect_tx(full, (uint32_t)copies * img_bytes, leader);
        for (int n = n_a; n <= n_b; ++n) {
          if (!B2C_X_OK(args.dbg, 50, args.x + (size_t)n * img_bytes, img_bytes)) continue;
          const uint32_t dst = win_base + (uint32_t)s * win_bytes + (uint32_t)args.wn_left + (uint32_t)(n - n_a) * img_bytes;
          asm volatile(
              "{\n.reg .pred q;\nsetp.ne.b32 q, %4, 0;\n"
              "@q cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n}" ::"r"(dst),
              "l"(args.x + (size_t)n * img_bytes), "r"(img_bytes), "r"(full), "r"(leader)
              : "memory");
        }
      } else {
        const int img = (int)args.div_tiles_hw.div((uint32_t)t);
        const int rem = t - img * tiles_per_image;
        const int ty = (int)args.div_tiles_w.div((uint32_t)rem), tx = rem - ty * args.sh_tiles_w;
        mbar_arrive_expect_tx(full, (uint32_t)args.wn_box_bytes, leader);
        // (the first column is a multiple of 16 bytes below the tile's first input column)
        tma_load_tiled_4d(win_base + (uint32_t)s * win_bytes, &tmap_x, tx * args.wn_tile_w * args.stride_w - args.wn_left,
                          ty * tile_h * args.stride_h - args.pad_h, 0, img, full, leader);
      }
      if (++s == kWinStages) {
        s = 0;
        ph ^= 1u;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    const uint32_t idesc = make_idesc_i8(args.tile_n);
    const uint32_t leader = elect_one() ? 1u : 0u;
    const uint64_t a_kb_step = a_block_bytes >> 4, b_kb_step = b_block_bytes >> 4;
    bool alive = __all_sync(0xffffffffu, mbar_wait(smem_u32(&wc.w_full), 0u, ctl, args.status));
    int ti = 0;
    for (int t = tile_first; t < tile_end && alive; t += tile_step, ++ti) {
      const int ab = ti & (kABufs - 1);
      const uint32_t a_use = (uint32_t)(ti / kABufs);
      const int tb = ti & (nbuf - 1);
      const uint32_t t_use = (uint32_t)(ti >> nbuf_log2);
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&wc.tmem_empty[tb]), (t_use & 1u) ^ 1u, ctl, args.status))) break;
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&wc.a_full[ab]), a_use & 1u, ctl, args.status))) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t d_tmem = tmem_acc + (uint32_t)(tb * args.tmem_cols);
      uint64_t adesc = make_smem_desc(a_base + (uint32_t)ab * a_buf_bytes, 128);
      uint64_t bdesc = make_smem_desc(b_base, 128);
      for (int kb = 0; kb < nkb; ++kb) {
        mma_i8_block(d_tmem, adesc, bdesc, idesc, kb ? 1u : 0u, leader, kb == nkb - 1 ? args.ksteps_last : 4);
        adesc += a_kb_step;
        bdesc += b_kb_step;
      }
      mma_commit(smem_u32(&wc.a_empty[ab]), leader);
      mma_commit(smem_u32(&wc.tmem_full[tb]), leader);
    }
    __syncwarp();
  } else if (warp < 2 + kBuildWarps) {
    // ---------------------------------------------------------------- operand builders
    const int tid = (int)threadIdx.x - 64;
    const int row = tid & (kTileM - 1);
    const int half = tid >> 7;  // warps 2-5 take the even 16-byte chunks of a row, warps 6-9 the odd ones
    const int ti_row = row >> tw_log2, tj = row & (args.wn_tile_w - 1);
    // byte offset of this row's first tap inside a window, and the permute selector of its alignment
    // (two-dimensional tiles: the same for every tile; linear tiles: set per tile below)
    int tbase = ti_row * args.stride_h * args.wn_win_w + tj * args.stride_w + args.wn_off0;
    uint32_t sel = 0x3210u + 0x1111u * ((uint32_t)tbase & 3u);
    int tbase4 = tbase & ~3;
    uint32_t rbits = 0, hm0 = 0, hm1 = 0;  // linear tiles: valid filter rows, byte masks of the two words of a run
    const uint32_t xr = (uint32_t)(row & 7);
    const uint32_t row_off = (uint32_t)row * 128u;
    const int nchunks = args.wn_chunks;  // 16-byte chunks of a row (K_pad / 16)
    int s = 0, ti = 0;
    uint32_t ph = 0;
    bool ok = true;
    for (int t = tile_first; t < tile_end && ok; t += tile_step, ++ti) {
      const int ab = ti & (kABufs - 1);
      const uint32_t a_use = (uint32_t)(ti / kABufs);
      ok = mbar_wait_relaxed(smem_u32(&wc.a_empty[ab]), (a_use & 1u) ^ 1u, ctl, args.status);
      if (ok) ok = mbar_wait_relaxed(smem_u32(&wc.win_full[s]), ph, ctl, args.status);
      if (!ok) break;
      if (LINEAR) {
        // this row's pixel (n, p, q); rows past the last pixel build from the window's first image (never stored)
        const unsigned m = (unsigned)t * kTileM + (unsigned)row;
        const int n_a = (int)args.div_pq.div((uint32_t)t * kTileM);
        int part = 0, p = 0, q = 0;
        if (m < (unsigned)args.Mg) {
          const int n = (int)args.div_pq.div(m);
          const int pq = (int)(m - (unsigned)n * (unsigned)args.PQ);
          p = (int)args.div_q.div((uint32_t)pq);
          q = pq - p * args.Q;
          part = n - n_a;
        }
        const int h0 = p * args.stride_h - args.pad_h, w0 = q * args.stride_w - args.pad_w;
        tbase = args.wn_left + part * args.wn_box_bytes + h0 * args.W + w0;
        sel = 0x3210u + 0x1111u * ((uint32_t)tbase & 3u);
        tbase4 = tbase & ~3;
        rbits = 0;
        for (int r = 0; r < args.sh_R; ++r)
          if ((unsigned)(h0 + r * args.dil_h) < (unsigned)args.H) rbits |= 1u << r;
        hm0 = hm1 = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          if ((unsigned)(w0 + b) < (unsigned)args.W) hm0 |= 0xFFu << (8 * b);
          if ((unsigned)(w0 + 4 + b) < (unsigned)args.W) hm1 |= 0xFFu << (8 * b);
        }
      }
      const uint8_t* wslot = win_ptr + (size_t)s * win_bytes;
      const uint8_t* win = wslot + tbase4;
      const uint32_t a_row = a_base + (uint32_t)ab * a_buf_bytes + row_off;
      if (LINEAR) {
        for (int ch = half; ch < nchunks; ch += 2) {
          // table entry of a word: window offset (16 bits), filter row (8 bits), word of the run (8 bits)
          const int4 e = *reinterpret_cast<const int4*>(s_table + ch * 4);
          const int ev[4] = {e.x, e.y, e.z, e.w};
          uint32_t wv[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int off = ev[i] & 0xFFFF, r = (ev[i] >> 16) & 0xFF, wi = ev[i] >> 24;
            // (image rows are not multiples of 4 bytes here: the word's alignment depends on its offset too)
            const int addr = tbase + off;
            const uint8_t* src = wslot + (addr & ~3);
            const uint32_t lo = *reinterpret_cast<const uint32_t*>(src);
            const uint32_t hi = *reinterpret_cast<const uint32_t*>(src + 4);
            const uint32_t mask = ((rbits >> r) & 1u) ? (wi ? hm1 : hm0) : 0u;
            wv[i] = __byte_perm(lo, hi, 0x3210u + 0x1111u * ((uint32_t)addr & 3u)) & mask;
          }
          const uint32_t dst = a_row + (uint32_t)(ch >> 3) * a_block_bytes + ((((uint32_t)ch & 7u) ^ xr) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(wv[0]), "r"(wv[1]), "r"(wv[2]), "r"(wv[3]));
        }
      } else {
        // 32-bit shared-memory addresses and explicit ld.shared: no generic-pointer arithmetic in the loop.
        // The table gives each chunk's four word offsets; the low two bits of the first say how they lie:
        // 0 = one run of 16 consecutive bytes (five aligned loads), 1 = two runs of 8 (three loads each),
        // 2 = four separate words.
        const uint32_t win_s = win_base + (uint32_t)s * win_bytes + (uint32_t)tbase4;
        const uint32_t tab_s = win_base + kWinStages * win_bytes;
        for (int ch = half; ch < nchunks; ch += 2) {
          uint32_t o0, o1, o2, o3;
          asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(o0), "=r"(o1), "=r"(o2), "=r"(o3) : "r"(tab_s + (uint32_t)ch * 16u));
          const uint32_t kind = o0 & 3u;
          const uint32_t a0 = win_s + (o0 & ~3u);
          uint32_t w0, w1, w2, w3;
          if (kind == 0u) {
            uint32_t v0, v1, v2, v3, v4;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v0) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(v1) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+8];" : "=r"(v2) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+12];" : "=r"(v3) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+16];" : "=r"(v4) : "r"(a0));
            w0 = __byte_perm(v0, v1, sel);
            w1 = __byte_perm(v1, v2, sel);
            w2 = __byte_perm(v2, v3, sel);
            w3 = __byte_perm(v3, v4, sel);
          } else if (kind == 1u) {
            const uint32_t a2 = win_s + o2;
            uint32_t v0, v1, v2, u0, u1, u2;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v0) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(v1) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+8];" : "=r"(v2) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(u0) : "r"(a2));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(u1) : "r"(a2));
            asm volatile("ld.shared.b32 %0, [%1+8];" : "=r"(u2) : "r"(a2));
            w0 = __byte_perm(v0, v1, sel);
            w1 = __byte_perm(v1, v2, sel);
            w2 = __byte_perm(u0, u1, sel);
            w3 = __byte_perm(u1, u2, sel);
          } else {
            const uint32_t a1 = win_s + o1, a2 = win_s + o2, a3 = win_s + o3;
            uint32_t l0, h0, l1, h1, l2, h2, l3, h3;
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(l0) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(h0) : "r"(a0));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(l1) : "r"(a1));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(h1) : "r"(a1));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(l2) : "r"(a2));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(h2) : "r"(a2));
            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(l3) : "r"(a3));
            asm volatile("ld.shared.b32 %0, [%1+4];" : "=r"(h3) : "r"(a3));
            w0 = __byte_perm(l0, h0, sel);
            w1 = __byte_perm(l1, h1, sel);
            w2 = __byte_perm(l2, h2, sel);
            w3 = __byte_perm(l3, h3, sel);
          }
          const uint32_t dst = a_row + (uint32_t)(ch >> 3) * a_block_bytes + ((((uint32_t)ch & 7u) ^ xr) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3));
        }
      }
      // the window has been read; the A rows are visible to the tensor core's async proxy
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&wc.win_empty[s]));
        mbar_arrive(smem_u32(&wc.a_full[ab]));
      }
      if (++s == kWinStages) {
        s = 0;
        ph ^= 1u;
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue warps
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int ti_row = row >> tw_log2, tj = row & (args.wn_tile_w - 1);
    bool ok = true;
    int ti = 0;
    for (int t = tile_first; t < tile_end && ok; t += tile_step, ++ti) {
      int img, out_pq;
      bool row_valid;
      if (LINEAR) {
        const unsigned m = (unsigned)t * kTileM + (unsigned)row;
        row_valid = m < (unsigned)args.Mg;
        img = row_valid ? (int)args.div_pq.div(m) : 0;
        out_pq = row_valid ? (int)(m - (unsigned)img * (unsigned)args.PQ) : 0;
      } else {
        img = (int)args.div_tiles_hw.div((uint32_t)t);
        const int rem = t - img * tiles_per_image;
        const int ty = (int)args.div_tiles_w.div((uint32_t)rem), tx = rem - ty * args.sh_tiles_w;
        const int po = ty * tile_h + ti_row, qo = tx * args.wn_tile_w + tj;
        row_valid = po < args.out_P && qo < args.out_Q;
        out_pq = po * args.out_Q + qo;
      }
      const int tb = ti & (nbuf - 1);
      const uint32_t t_use = (uint32_t)(ti >> nbuf_log2);
      ok = mbar_wait_relaxed(smem_u32(&wc.tmem_full[tb]), t_use & 1u, ctl, args.status);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (!ok) break;
      const long long base_nkpq = (long long)img * args.y_stride_n + out_pq;
      const long long base_npqk = ((long long)img * args.out_PQ + out_pq) * args.K;
      const uint32_t taddr = tmem_acc + ((uint32_t)(quad * 32) << 16) + (uint32_t)(tb * args.tmem_cols);
      if ((args.tile_n & 31) == 0) {
        for (int c = 0; c < args.tile_n; c += 32)
          epilogue_columns<32>(args, taddr + (uint32_t)c, c, row_valid, base_nkpq, base_npqk, 0u);
      } else {
        epilogue_columns<16>(args, taddr, 0, row_valid, base_nkpq, base_npqk, 0u);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&wc.tmem_empty[tb]));
    }
  }

  // ---------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (ctl->abort_flag) {
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

}  // namespace

size_t conv_mma_window_smem_bytes(const ConvArgs& a) {
  const size_t a_buf = (size_t)a.num_kb * kTileM * 128, b_buf = (size_t)a.num_kb * a.tile_n * 128;
  return 1024 + kABufs * a_buf + b_buf + (size_t)kWinStages * a.wn_win_bytes + (((size_t)a.table_len * 4 + 127) & ~(size_t)127) + 128;
}

cudaError_t launch_conv_mma_window(const CUtensorMap* tmap_x, const CUtensorMap* tmap_b, const ConvArgs& args,
                                   cudaStream_t st) {
  const size_t smem = conv_mma_window_smem_bytes(args);
  static std::atomic<unsigned long long> configured{0}, configured_linear{0};
  cudaError_t e = args.wn_linear
                      ? set_max_dynamic_smem_once(configured_linear, (const void*)conv_mma_window_kernel<true>, 226 * 1024)
                      : set_max_dynamic_smem_once(configured, (const void*)conv_mma_window_kernel<false>, 226 * 1024);
  if (e != cudaSuccess) return e;
  // blocks per SM by shared memory (at most two); the grid is one wave of resident blocks walking the tiles
  const int per_sm = smem * 2 + 4096 <= 227 * 1024 ? 2 : 1;
  const dim3 grid((unsigned)std::min(args.num_tiles, kNumSMs * per_sm), 1, 1);
  if (args.wn_linear)
    e = launch_pdl(conv_mma_window_kernel<true>, grid, dim3(kWinThreads), smem, st, *tmap_x, *tmap_b, args);
  else
    e = launch_pdl(conv_mma_window_kernel<false>, grid, dim3(kWinThreads), smem, st, *tmap_x, *tmap_b, args);
  if (e != cudaSuccess) return e;
  return cudaGetLastError();
}

}  // namespace b2c
