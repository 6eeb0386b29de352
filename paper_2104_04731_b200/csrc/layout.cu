// Data-layout rewrites of Table 2 as CUDA kernels: Pad + Reorder of the activations
// (NCHW -> NHWC with the channel axis zero-padded to the intrinsic's block), the weight packs
// (reduction index made contiguous, Section 5.1: the B operand is held transposed), the
// explicit Stencil Unroll (im2col matrix, formed by direct indexing rather than the index-list
// gather the paper found slow in Section 6.1), and the finish pass of a split reduction.
#include <algorithm>

#include "b2c_internal.h"

namespace b2c {

namespace {

constexpr int kPackThreads = 256;
constexpr int kPackMaxC = 128;  // channels per tile (64 when the padded channel count is below 128)
constexpr int kPackMaxP = 256;  // pixels per tile
constexpr int kPackSmem = kPackMaxC * (kPackMaxP + 4) + (kPackMaxC / 16) * 16;

// One block moves a [CT channels] x [PT pixels] tile of one image through shared memory.
// Reads run along the pixel axis of NCHW in VEC-byte vectors (VEC = 16 or 4 when H*W allows the
// alignment, else 1) with many loads in flight per thread; the tile is kept as rows of `pitch`
// bytes (pitch/4 odd) with each group of 16 rows skewed by 16 bytes, which makes the transposing
// reads below conflict free.  Writes run along the channel axis of NHWC: a thread takes 16
// channels of 4 consecutive pixels as 16 words, transposes them in registers with byte permutes
// and stores four 16-byte vectors; the 8 (or 4) threads of one pixel cover 128 (or 64) contiguous
// bytes.  Channels >= C are written as zeros.
template <int VEC>
__global__ void __launch_bounds__(kPackThreads) pack_activations_kernel(const int8_t* __restrict__ x,
                                                                        int8_t* __restrict__ out, int C, int HW,
                                                                        int C_pad, int hw_tiles, int CT, int PT, Dbg dbg) {
  __shared__ __align__(16) uint8_t tile[kPackSmem];
  const int n = blockIdx.x / hw_tiles;
  const int c0 = blockIdx.y * CT;
  const int hw0 = (blockIdx.x - n * hw_tiles) * PT;
  const int t = threadIdx.x;
  const int pitch = PT + 4;
  const int8_t* xin = x + ((size_t)n * C + c0) * HW + hw0;
  const int rows = min(CT, C - c0);  // channels that exist; the rest of the tile is zero padding
  pdl_wait();

  // ---- load ----
  if constexpr (VEC >= 4) {
    constexpr int NW = VEC / 4;  // words per vector
    const int wpr = PT >> 2;     // words per row
    const int vecs = CT * wpr / NW;
#pragma unroll 8
    for (int i = t; i < vecs; i += kPackThreads) {
      const int wi = i * NW;
      const int row = wi / wpr;
      const int hw = (wi - row * wpr) * 4;
      uint32_t v[NW];
#pragma unroll
      for (int k = 0; k < NW; ++k) v[k] = 0;
      if (row < rows) {
        const int8_t* src = xin + (size_t)row * HW + hw;
        if (hw0 + hw + VEC <= HW && B2C_X_OK(dbg, 1, src, VEC)) {
          if constexpr (VEC == 16) {
            const uint4 q = *reinterpret_cast<const uint4*>(src);
            v[0] = q.x;
            v[NW - 3] = q.y;
            v[NW - 2] = q.z;
            v[NW - 1] = q.w;
          } else {
            v[0] = *reinterpret_cast<const uint32_t*>(src);
          }
        } else {
          for (int b = 0; b < VEC; ++b)
            if (hw0 + hw + b < HW && B2C_X_OK(dbg, 1, src + b, 1)) v[b >> 2] |= (uint32_t)(uint8_t)src[b] << (8 * (b & 3));
        }
      }
      uint32_t* dst = reinterpret_cast<uint32_t*>(&tile[row * pitch + (row >> 4) * 16 + hw]);
#pragma unroll
      for (int k = 0; k < NW; ++k) dst[k] = v[k];
    }
  } else {
    const int total = CT * PT;
#pragma unroll 8
    for (int i = t; i < total; i += kPackThreads) {
      const int row = i / PT;
      const int hw = i - row * PT;
      uint8_t v = 0;
      if (row < rows && hw0 + hw < HW && B2C_X_OK(dbg, 1, xin + (size_t)row * HW + hw, 1)) v = (uint8_t)xin[(size_t)row * HW + hw];
      tile[row * pitch + (row >> 4) * 16 + hw] = v;
    }
  }
  __syncthreads();
  pdl_launch_dependents();  // after the loads: an earlier start would only take shared memory from this grid

  // ---- transpose in registers and store ----
  const int chunks = CT >> 4;            // 16-channel chunks per pixel in this tile
  const int items = (PT >> 2) * chunks;  // (group of 4 pixels, chunk)
  for (int it = t; it < items; it += kPackThreads) {
    const int ch = it % chunks;
    const int pg = it / chunks;
    const int hw = hw0 + pg * 4;
    if (hw >= HW || c0 + ch * 16 >= C_pad) continue;
    uint32_t w[16];
    const uint8_t* src = &tile[(ch * 16) * pitch + ch * 16 + pg * 4];
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = *reinterpret_cast<const uint32_t*>(src + i * pitch);
    int8_t* dst = out + ((size_t)n * HW + hw) * C_pad + c0 + ch * 16;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (hw + j < HW) {
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t lo = __byte_perm(w[4 * k], w[4 * k + 1], j | ((4 + j) << 4));
          const uint32_t hi = __byte_perm(w[4 * k + 2], w[4 * k + 3], j | ((4 + j) << 4));
          o[k] = __byte_perm(lo, hi, 0x5410);
        }
        if (B2C_WS_OK(dbg, 2, dst + (size_t)j * C_pad, 16))
          *reinterpret_cast<uint4*>(dst + (size_t)j * C_pad) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// Bulk-copy variant of the activation pack for the common aligned cases.  The tile's rows reach
// shared memory by asynchronous bulk copies (cp.async.bulk) that complete on an mbarrier, so the
// load phase costs no per-byte instructions and keeps whole tiles in flight:
//   group mode (kRowMode = false): the tile spans all H*W pixels of 16-channel groups, and every
//     group (16*H*W contiguous bytes of NCHW) is fetched by one copy;
//   row mode (kRowMode = true): H*W is a multiple of 16 and every channel row segment of PT pixels
//     is fetched by one copy.
// Groups of 16 rows are spaced 16 bytes further apart than their size, which makes the
// transposing word reads of the store phase conflict free.  The store phase is the same register
// transpose as in pack_activations_kernel.
constexpr unsigned long long kPackWaitLimitNs = 1000ull * 1000ull * 1000ull;  // 1 s, as in the MMA kernel
__device__ __forceinline__ unsigned long long pack_global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool pack_bar_try_wait(uint32_t bar) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar)
      : "memory");
  return ok != 0;
}

__device__ __forceinline__ bool pack_wait_bounded(uint32_t bar, int* status, bool reporter) {
  bool done = false;
  for (int tries = 0; tries < 64 && !done; ++tries) done = pack_bar_try_wait(bar);
  if (!done) {
    const unsigned long long t0 = pack_global_ns();
    while (!(done = pack_bar_try_wait(bar)) && pack_global_ns() - t0 < kPackWaitLimitNs) {
    }
  }
  if (!done) {
    if (reporter && status != nullptr) atomicCAS(status, 0, B2C_E_TIMEOUT);
    const unsigned long long t1 = pack_global_ns();
    while (pack_global_ns() - t1 < 50000ull) __nanosleep(1000);
  }
  return done;
}

// One block waits, with the bounded wait of the bulk-copy pack kernel, on a barrier that expects
// bytes no copy delivers; the wait gives up after its limit and reports through `status`.
__global__ void pack_wait_selftest_kernel(int* status) {
  __shared__ __align__(8) unsigned long long bar;
  const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&bar);
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(16u) : "memory");
  }
  __syncthreads();
  pack_wait_bounded(bar_a, status, threadIdx.x == 0);
}

template <bool kRowMode>
__global__ void __launch_bounds__(kPackThreads) pack_activations_bulk_kernel(const int8_t* __restrict__ x,
                                                                             int8_t* __restrict__ out, int C, int HW,
                                                                             int C_pad, int hw_tiles, int CT, int PT,
                                                                             int* status, Dbg dbg) {
  extern __shared__ __align__(128) uint8_t btile[];
  __shared__ __align__(8) unsigned long long bar;
  const int n = blockIdx.x / hw_tiles;
  const int c0 = blockIdx.y * CT;
  const int hw0 = (blockIdx.x - n * hw_tiles) * PT;
  const int t = threadIdx.x;
  const int npx = min(PT, HW - hw0);        // pixels of this tile
  const int rows = max(0, min(CT, C - c0));  // channels that exist (a multiple of 16)
  const int rp = kRowMode ? PT : HW;         // row pitch in shared memory
  const int gs = 16 * rp + 16;               // group stride
  const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&bar);
  const uint32_t tile_a = (uint32_t)__cvta_generic_to_shared(btile);
  if (t == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const uint32_t bytes = (uint32_t)rows * (uint32_t)npx;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
  }
  __syncthreads();
  pdl_wait();
  const int8_t* xin = x + ((size_t)n * C + c0) * HW + hw0;
  if (kRowMode) {
    if (t < rows && B2C_X_OK(dbg, 3, xin + (size_t)t * HW, npx)) {
      const uint32_t dst = tile_a + (uint32_t)((t >> 4) * gs + (t & 15) * rp);
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
          "l"(xin + (size_t)t * HW), "r"((uint32_t)npx), "r"(bar_a)
          : "memory");
    }
#ifdef B2C_DEBUG_BOUNDS
    else if (t < rows)  // a refused copy: account for its bytes so that the barrier still completes
      asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar_a), "r"((uint32_t)npx) : "memory");
#endif
  } else {
    if (t < (rows >> 4) && B2C_X_OK(dbg, 3, xin + (size_t)t * 16 * HW, 16 * HW)) {
      const uint32_t dst = tile_a + (uint32_t)(t * gs);
      asm volatile(
          "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
          "l"(xin + (size_t)t * 16 * HW), "r"((uint32_t)(16 * HW)), "r"(bar_a)
          : "memory");
    }
#ifdef B2C_DEBUG_BOUNDS
    else if (t < (rows >> 4))
      asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar_a), "r"((uint32_t)(16 * HW)) : "memory");
#endif
  }
  // Bounded wait for the copies (every thread polls the barrier).  On expiry the block records
  // B2C_E_TIMEOUT in the status word (when the caller gave one), leaves the copies that were issued
  // some time to land before its shared memory is released, and returns; its part of the output
  // stays unwritten.
  if (!pack_wait_bounded(bar_a, status, t == 0)) return;
  // The next kernel may start its set-up once every block of this one has its tile in shared
  // memory (earlier, its resident blocks would only take shared memory away from this grid).
  pdl_launch_dependents();

  const int chunks = CT >> 4;
  const int items = ((npx + 3) >> 2) * chunks;
  for (int it = t; it < items; it += kPackThreads) {
    const int ch = it % chunks;
    const int pg = it / chunks;
    const int hw = hw0 + pg * 4;
    if (c0 + ch * 16 >= C_pad) continue;
    uint32_t w[16];
    if (ch * 16 < rows) {
      const uint8_t* src = btile + ch * gs + pg * 4;
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i] = *reinterpret_cast<const uint32_t*>(src + i * rp);
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i] = 0;
    }
    int8_t* dst = out + ((size_t)n * HW + hw) * C_pad + c0 + ch * 16;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (hw + j < HW) {
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t lo = __byte_perm(w[4 * k], w[4 * k + 1], j | ((4 + j) << 4));
          const uint32_t hi = __byte_perm(w[4 * k + 2], w[4 * k + 3], j | ((4 + j) << 4));
          o[k] = __byte_perm(lo, hi, 0x5410);
        }
        if (B2C_WS_OK(dbg, 2, dst + (size_t)j * C_pad, 16))
          *reinterpret_cast<uint4*>(dst + (size_t)j * C_pad) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// Activation pack for large batches of small images whose channels all fit one tile (C a multiple of 16,
// at most 64; H*W a multiple of 4, at most 256): the images of a batch tensor are then contiguous, so one
// block fetches `ipb` whole images with ONE bulk copy (several KB in flight per block instead of one
// 16-channel group) and transposes them as the kernels above do.  Channels C .. C_pad-1 are written as zeros.
__global__ void __launch_bounds__(kPackThreads) pack_small_images_kernel(const int8_t* __restrict__ x,
                                                                        int8_t* __restrict__ out, int N, int C, int HW,
                                                                        int C_pad, int ipb, int* status, Dbg dbg) {
  extern __shared__ __align__(128) uint8_t btile[];
  __shared__ __align__(8) unsigned long long bar;
  const int t = threadIdx.x;
  const int n0 = blockIdx.x * ipb;
  const int nimg = min(ipb, N - n0);
  const int img_bytes = C * HW;
  const uint32_t bar_a = (uint32_t)__cvta_generic_to_shared(&bar);
  const uint32_t tile_a = (uint32_t)__cvta_generic_to_shared(btile);
  const int8_t* xin = x + (size_t)n0 * img_bytes;
  if (t == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_a) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  pdl_wait();
  if (t == 0) {
    const uint32_t bytes = (uint32_t)(nimg * img_bytes);
    if (B2C_X_OK(dbg, 17, xin, bytes)) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_a), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(tile_a),
                   "l"(xin), "r"(bytes), "r"(bar_a)
                   : "memory");
    } else {
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_a) : "memory");  // refused (debug build): nothing to wait for
    }
  }
  if (!pack_wait_bounded(bar_a, status, t == 0)) return;
  pdl_launch_dependents();
  const int chunks = C_pad >> 4;            // 16-channel chunks of an output pixel
  const int pgs = (HW + 3) >> 2;            // groups of 4 pixels of an image
  const int items = nimg * pgs * chunks;
  for (int it = t; it < items; it += kPackThreads) {
    const int ch = it % chunks;
    const int r = it / chunks;
    const int pg = r % pgs;
    const int i = r / pgs;
    uint32_t w[16];
    if (ch * 16 < C) {
      const uint8_t* src = btile + (size_t)i * img_bytes + (ch * 16) * HW + pg * 4;
#pragma unroll
      for (int k = 0; k < 16; ++k) w[k] = *reinterpret_cast<const uint32_t*>(src + k * HW);
    } else {
#pragma unroll
      for (int k = 0; k < 16; ++k) w[k] = 0;
    }
    int8_t* dst = out + ((size_t)(n0 + i) * HW + pg * 4) * C_pad + ch * 16;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (pg * 4 + j < HW) {
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint32_t lo = __byte_perm(w[4 * k], w[4 * k + 1], j | ((4 + j) << 4));
          const uint32_t hi = __byte_perm(w[4 * k + 2], w[4 * k + 3], j | ((4 + j) << 4));
          o[k] = __byte_perm(lo, hi, 0x5410);
        }
        if (B2C_WS_OK(dbg, 18, dst + (size_t)j * C_pad, 16))
          *reinterpret_cast<uint4*>(dst + (size_t)j * C_pad) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// Channel-pack weights: out[k][(r*S + s)][c_pad] = w[k][c][r][s], zeros for c >= C.
__global__ void pack_weights_cp_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ out, int K, int C, int RS,
                                       int C_pad) {
  const long long total = (long long)K * RS * C_pad;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(i % C_pad);
    const long long kt = i / C_pad;
    const int tap = (int)(kt % RS);
    const long long k = kt / RS;
    out[i] = c < C ? w[(k * C + c) * RS + tap] : (int8_t)0;
  }
}

// Table-driven weight pack for the rewritten maps: out[k][j] = w[k][table[j]], zero where table[j] < 0.
__global__ void pack_weights_table_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ out, int K, int Kg, int cols,
                                          const int32_t* __restrict__ table) {
  const long long total = (long long)K * cols;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(i % cols);
    const long long k = i / cols;
    const int src = table[j];
    out[i] = src >= 0 ? w[k * Kg + src] : (int8_t)0;
  }
}

// Stencil-unroll weights: rows of w[k][(c,r,s)] with every (c, r) run of S taps padded with zeros
// to S_run entries (S_run = S for the plain unroll), then the row zero-padded to K_pad.
__global__ void pack_weights_rows_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ out, int K, int Kg,
                                         int K_pad, int S, int S_run) {
  const long long total = (long long)K * K_pad;
  const int runs = Kg / S;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(i % K_pad);
    const long long k = i / K_pad;
    const int run = j / S_run, s = j - run * S_run;
    out[i] = (run < runs && s < S) ? w[k * Kg + run * S + s] : (int8_t)0;
  }
}

// Explicit stencil unroll.  One thread produces 16 consecutive reduction entries of one output
// pixel's row and stores them as one 16-byte vector; the window geometry comes from a lookup
// table indexed by the reduction position, so no per-element division is needed.
__global__ void __launch_bounds__(256) im2col_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a,
                                                     const GatherEntry* __restrict__ table, long long Mg, int PQ, int Q,
                                                     int H, int W, int stride_h, int stride_w, int pad_h, int pad_w,
                                                     long long x_stride_n, int x_stride_h, int x_stride_w, int K_pad,
                                                     Dbg dbg) {
  const int chunks = K_pad >> 4;
  const long long total = Mg * chunks;
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long m = i / chunks;
    const int ck = (int)(i - m * chunks);
    const int n = (int)(m / PQ);
    const int pq = (int)(m - (long long)n * PQ);
    const int p = pq / Q, q = pq - p * Q;
    const int h0 = p * stride_h - pad_h, w0 = q * stride_w - pad_w;
    const int8_t* base = x + n * x_stride_n + (long long)h0 * x_stride_h + (long long)w0 * x_stride_w;
    uint32_t wv[4] = {0, 0, 0, 0};
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const GatherEntry g = table[ck * 16 + e];
      const int h = h0 + g.dh, ww = w0 + g.dw;
      uint32_t v = 0;
      if (g.off >= 0 && (unsigned)h < (unsigned)H && (unsigned)ww < (unsigned)W && B2C_X_OK(dbg, 4, base + g.off, 1))
        v = (uint8_t)base[g.off];
      wv[e >> 2] |= v << (8 * (e & 3));
    }
    if (B2C_WS_OK(dbg, 5, a + m * K_pad + ck * 16, 16))
      *reinterpret_cast<uint4*>(a + m * K_pad + ck * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
  pdl_launch_dependents();
}

// Image Pack of a dilated convolution: sub-image (n, a, b) holds phase (a, b) of image n,
// out[n'][hs][ws][c] = x[n][c][hs*dh + a][ws*dw + b] with n' = (n*dh + a)*dw + b, zeros past the
// image and in the padded channels; NHWC with C_pad channels.  One thread writes 16 channels of one
// sub-image pixel as a 16-byte vector.
__global__ void __launch_bounds__(256) phase_split_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ out, int N,
                                                          int C, int H, int W, int dh, int dw, int Hs, int Ws, int C_pad,
                                                          long long stride_n, long long stride_c, int stride_h,
                                                          int stride_w, Dbg dbg) {
  const int chunks = C_pad >> 4;
  const long long total = (long long)N * dh * dw * Hs * Ws * chunks;
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long pix = i / chunks;
    const int ck = (int)(i - pix * chunks);
    const int ws = (int)(pix % Ws);
    const long long t = pix / Ws;
    const int hs = (int)(t % Hs);
    const long long nsub = t / Hs;
    const int b = (int)(nsub % dw);
    const int a = (int)((nsub / dw) % dh);
    const long long n = nsub / ((long long)dw * dh);
    const int h = hs * dh + a, w = ws * dw + b;
    uint32_t wv[4] = {0, 0, 0, 0};
    if (h < H && w < W) {
      const int8_t* src = x + n * stride_n + (long long)h * stride_h + (long long)w * stride_w;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int c = ck * 16 + e;
        if (c < C && B2C_X_OK(dbg, 6, src + c * stride_c, 1)) wv[e >> 2] |= (uint32_t)(uint8_t)src[c * stride_c] << (8 * (e & 3));
      }
    }
    if (B2C_WS_OK(dbg, 7, out + pix * C_pad + ck * 16, 16))
      *reinterpret_cast<uint4*>(out + pix * C_pad + ck * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
  pdl_launch_dependents();
}

// Image Pack of a strided convolution (space to depth): scratch pixel (n, hs, ws) holds the
// stride_h x stride_w phases of every channel, out[n][hs][ws][(c*stride_h + dh)*stride_w + dw] =
// x[n][c][hs*stride_h + dh - pad_h][ws*stride_w + dw - pad_w], zeros outside the image and in the
// padded channels.  One thread forms 16 consecutive scratch channels of one pixel by direct indexing
// (running (c, dh, dw) counters, no lookup table) and stores them as one 16-byte vector.
__global__ void __launch_bounds__(256) space_to_depth_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ out,
                                                             unsigned total, FastDiv div_chunks, FastDiv div_ws,
                                                             FastDiv div_hs, int C, int H, int W, int sh, int sw,
                                                             int pad_h, int pad_w, int C_pad, int pack,
                                                             long long stride_n, int stride_c, int stride_h,
                                                             int stride_w, Dbg dbg) {
  // (32-bit indices and multiply-shift divisions: a 64-bit division costs more than the 16 bytes moved)
  const int chunks = (int)div_chunks.d, Ws = (int)div_ws.d, Hs = (int)div_hs.d;
  const int creal = pack * C * sh * sw;  // a column's own phases plus those of its pack - 1 right neighbours
  pdl_wait();
  for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const unsigned pix = div_chunks.div(i);
    const int ck = (int)(i - pix * (unsigned)chunks);
    uint32_t wv[4] = {0, 0, 0, 0};
    const int j0 = ck * 16;
    if (j0 < creal) {
      const unsigned t = div_ws.div(pix);
      const int ws = (int)(pix - t * (unsigned)Ws);
      const unsigned n = div_hs.div(t);
      const int hs = (int)(t - n * (unsigned)Hs);
      const int h0 = hs * sh - pad_h, w0 = ws * sw - pad_w;
      // scratch channel j = ((c*sh + dh)*pack + ui)*sw + dw: the pack*sw bytes of one (c, dh) are
      // consecutive input bytes of one row
      const int run_len = pack * sw;
      const int run = j0 / run_len;
      int within = j0 - run * run_len;
      int c = run / sh, dh = run - c * sh;
      const int8_t* base = x + (long long)n * stride_n;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int h = h0 + dh, w = w0 + within;
        if (c < C && (unsigned)h < (unsigned)H && (unsigned)w < (unsigned)W &&
            B2C_X_OK(dbg, 8, base + c * stride_c + h * stride_h + w * stride_w, 1))
          wv[e >> 2] |= (uint32_t)(uint8_t)base[c * stride_c + h * stride_h + w * stride_w] << (8 * (e & 3));
        if (++within == run_len) {
          within = 0;
          if (++dh == sh) {
            dh = 0;
            ++c;
          }
        }
      }
    }
    if (B2C_WS_OK(dbg, 9, out + (size_t)i * 16, 16))
      *reinterpret_cast<uint4*>(out + (size_t)i * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
  pdl_launch_dependents();
}

// Space to depth for NCHW input whose rows are multiples of 16 bytes: one block forms kS2dTile
// consecutive scratch pixels of one scratch row.  The C*stride_h input row segments those pixels
// read are first copied to shared memory with aligned 16-byte loads (zeros outside the image), then
// each thread assembles the bytes of its pixel from shared memory and stores 16-byte vectors.
constexpr int kS2dTile = 128;
__global__ void __launch_bounds__(kS2dTile) space_to_depth_rows_kernel(const int8_t* __restrict__ x,
                                                                       int8_t* __restrict__ out, int Hs, int Ws, int C,
                                                                       int H, int W, int sh, int sw, int pad_h,
                                                                       int pad_w, int C_pad, int pack, int seg,
                                                                       int ws_tiles, Dbg dbg) {
  extern __shared__ __align__(16) uint8_t s2d_rows[];
  const int tile = blockIdx.x % ws_tiles;
  const int rowi = blockIdx.x / ws_tiles;  // (n, hs)
  const int n = rowi / Hs, hs = rowi - n * Hs;
  const int ws0 = tile * kS2dTile;
  const int wbeg = ws0 * sw - pad_w;        // first input column of the tile
  const int walign = wbeg & ~15;            // (two's complement: rounds toward minus infinity)
  const int rows = C * sh;
  const int vecs = seg >> 4;
  pdl_wait();
  for (int i = threadIdx.x; i < rows * vecs; i += kS2dTile) {
    const int r = i / vecs, v = i - r * vecs;
    const int c = r / sh, dh = r - c * sh;
    const int h = hs * sh + dh - pad_h;
    const int w = walign + v * 16;
    uint4 val = make_uint4(0, 0, 0, 0);
    if ((unsigned)h < (unsigned)H && w >= 0 && w + 16 <= W) {
      if (B2C_X_OK(dbg, 10, x + (((size_t)n * C + c) * H + h) * W + w, 16))
        val = __ldg(reinterpret_cast<const uint4*>(x + (((size_t)n * C + c) * H + h) * W + w));
    } else if ((unsigned)h < (unsigned)H && w + 16 > 0 && w < W) {
      uint32_t wv[4] = {0, 0, 0, 0};
      const int8_t* src = x + (((size_t)n * C + c) * H + h) * W;
      for (int b = 0; b < 16; ++b)
        if ((unsigned)(w + b) < (unsigned)W && B2C_X_OK(dbg, 10, src + w + b, 1)) wv[b >> 2] |= (uint32_t)(uint8_t)src[w + b] << (8 * (b & 3));
      val = make_uint4(wv[0], wv[1], wv[2], wv[3]);
    }
    *reinterpret_cast<uint4*>(s2d_rows + (size_t)r * seg + v * 16) = val;
  }
  __syncthreads();
  pdl_launch_dependents();
  const int ws = ws0 + threadIdx.x;
  if (ws >= Ws) return;
  const int off0 = threadIdx.x * sw + (wbeg - walign);
  // scratch channel j = ((c*sh + dh)*pack + ui)*sw + dw: the run of pack*sw bytes of one (c, dh) is
  // pack*sw consecutive bytes of one staged row.  Runs that are whole words are copied word by word
  // (an unaligned word = two aligned loads and a byte permute), others byte by byte.
  const int run_len = pack * sw;
  const int creal = C * sh * run_len;
  int8_t* dst = out + (((size_t)n * Hs + hs) * Ws + ws) * C_pad;
  int run = 0, within = 0;
  for (int j0 = 0; j0 < C_pad; j0 += 16) {
    uint32_t wv[4] = {0, 0, 0, 0};
    if (j0 < creal) {
      if ((run_len & 3) == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (j0 + 4 * k < creal) {
            const int src = run * seg + off0 + within;
            const uint32_t lo = *reinterpret_cast<const uint32_t*>(s2d_rows + (src & ~3));
            const uint32_t hi = *reinterpret_cast<const uint32_t*>(s2d_rows + (src & ~3) + 4);
            wv[k] = __byte_perm(lo, hi, 0x3210u + 0x1111u * (uint32_t)(src & 3));
          }
          within += 4;
          if (within == run_len) {
            within = 0;
            ++run;
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          if (j0 + e < creal) wv[e >> 2] |= (uint32_t)s2d_rows[run * seg + off0 + within] << (8 * (e & 3));
          if (++within == run_len) {
            within = 0;
            ++run;
          }
        }
      }
    }
    if (B2C_WS_OK(dbg, 11, dst + j0, 16)) *reinterpret_cast<uint4*>(dst + j0) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
}

// Row-phase unroll: scratch pixel (n, hs, q) holds, for every vertical stride phase dh, tap s and
// channel c, out[n][hs][q][(dh*S + s)*C + c] = x[n][c][hs*stride_h + dh - pad_h][q*stride_w - pad_w + s*dil_w]
// (zeros outside the image and in the padded channels).  One block forms kS2dTile consecutive pixels
// of one scratch row: the C*stride_h input row segments they read are staged in shared memory
// (aligned 16-byte loads where the layout allows, byte loads otherwise), then each thread assembles
// its pixel's bytes from there and stores 16-byte vectors.
__global__ void __launch_bounds__(kS2dTile) row_phase_unroll_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ out,
                                                                    int Hs, int Q, int C, int H, int W, int S, int sh,
                                                                    int sw, int pad_h, int pad_w, int dil_w, int C_pad,
                                                                    int seg, int q_tiles, long long stride_n,
                                                                    long long stride_c, int stride_h, int stride_w,
                                                                    int vec_ok, Dbg dbg) {
  extern __shared__ __align__(16) uint8_t rp_rows[];
  const int tile = blockIdx.x % q_tiles;
  const int rowi = blockIdx.x / q_tiles;  // (n, hs)
  const int n = rowi / Hs, hs = rowi - n * Hs;
  const int q0 = tile * kS2dTile;
  const int wbeg = q0 * sw - pad_w;  // first input column the tile reads
  const int walign = wbeg & ~15;     // rounds toward minus infinity
  const int rows = C * sh;
  const int8_t* xn = x + (size_t)n * stride_n;
  pdl_wait();
  if (vec_ok) {
    const int vecs = seg >> 4;
    for (int i = threadIdx.x; i < rows * vecs; i += kS2dTile) {
      const int r = i / vecs, v = i - r * vecs;
      const int c = r / sh, dh = r - c * sh;
      const int h = hs * sh + dh - pad_h;
      const int w = walign + v * 16;
      uint4 val = make_uint4(0, 0, 0, 0);
      if ((unsigned)h < (unsigned)H && w >= 0 && w + 16 <= W) {
        if (B2C_X_OK(dbg, 12, xn + c * stride_c + (long long)h * stride_h + w, 16))
          val = __ldg(reinterpret_cast<const uint4*>(xn + c * stride_c + (long long)h * stride_h + w));
      } else if ((unsigned)h < (unsigned)H && w + 16 > 0 && w < W) {
        uint32_t wv[4] = {0, 0, 0, 0};
        const int8_t* src = xn + c * stride_c + (long long)h * stride_h;
        for (int b = 0; b < 16; ++b)
          if ((unsigned)(w + b) < (unsigned)W && B2C_X_OK(dbg, 12, src + w + b, 1)) wv[b >> 2] |= (uint32_t)(uint8_t)src[w + b] << (8 * (b & 3));
        val = make_uint4(wv[0], wv[1], wv[2], wv[3]);
      }
      *reinterpret_cast<uint4*>(rp_rows + (size_t)r * seg + v * 16) = val;
    }
  } else {
    for (int i = threadIdx.x; i < rows * seg; i += kS2dTile) {
      const int r = i / seg, b = i - r * seg;
      const int c = r / sh, dh = r - c * sh;
      const int h = hs * sh + dh - pad_h;
      const int w = walign + b;
      uint8_t val = 0;
      if ((unsigned)h < (unsigned)H && (unsigned)w < (unsigned)W &&
          B2C_X_OK(dbg, 12, xn + c * stride_c + (long long)h * stride_h + (long long)w * stride_w, 1))
        val = (uint8_t)xn[c * stride_c + (long long)h * stride_h + (long long)w * stride_w];
      rp_rows[(size_t)r * seg + b] = val;
    }
  }
  __syncthreads();
  pdl_launch_dependents();
  const int q = q0 + threadIdx.x;
  if (q >= Q) return;
  const int off0 = threadIdx.x * sw + (wbeg - walign);
  const int creal = sh * S * C;
  int8_t* dst = out + (((size_t)n * Hs + hs) * Q + q) * C_pad;
  int dh = 0, s = 0, c = 0;
  for (int j0 = 0; j0 < C_pad; j0 += 16) {
    uint32_t wv[4] = {0, 0, 0, 0};
    if (j0 < creal) {
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        if (dh < sh) wv[e >> 2] |= (uint32_t)rp_rows[(c * sh + dh) * seg + off0 + s * dil_w] << (8 * (e & 3));
        if (++c == C) {
          c = 0;
          if (++s == S) {
            s = 0;
            ++dh;
          }
        }
      }
    }
    if (B2C_WS_OK(dbg, 13, dst + j0, 16)) *reinterpret_cast<uint4*>(dst + j0) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
}

// Finish of a split reduction: the int32 sums are complete in `acc`; copy them out and/or apply
// the shift-and-clip requantisation (arithmetic shift = floor division by 2^shift).
__global__ void splitk_finish_kernel(const int32_t* __restrict__ acc, int32_t* __restrict__ y32,
                                     int8_t* __restrict__ y8, long long elems, int shift, int out_mode,
                                     const int32_t* __restrict__ bias, int relu, int K, int PQ, int nhwc, Dbg dbg) {
  pdl_wait();
  pdl_launch_dependents();
  const bool act = bias != nullptr || relu != 0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < elems;
       i += (long long)gridDim.x * blockDim.x) {
    if (!(acc == y32 ? B2C_O32_OK(dbg, 14, acc + i, 4) : B2C_WS_OK(dbg, 14, acc + i, 4))) continue;
    int v = acc[i];
    if (bias != nullptr) v += bias[nhwc ? (int)(i % K) : (int)((i / PQ) % K)];  // output channel of element i
    if (relu) v = max(v, 0);
    if ((out_mode & B2C_OUT_I32) && (y32 != acc || act) && B2C_O32_OK(dbg, 15, y32 + i, 4)) y32[i] = v;
    if ((out_mode & B2C_OUT_I8) && B2C_O8_OK(dbg, 16, y8 + i, 1)) y8[i] = (int8_t)max(-128, min(127, v >> shift));
  }
}

int grid_for(long long total, int block) {
  long long g = (total + block - 1) / block;
  const long long cap = (long long)kNumSMs * 16;
  return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

}  // namespace

cudaError_t launch_pack_activations(const int8_t* x, int8_t* out, int N, int C, int H, int W, int C_pad,
                                    cudaStream_t st, int* status, const Dbg& dbg) {
  const int HW = H * W;
  int CT = C_pad >= 128 ? 128 : 64;
  const bool a16 = (reinterpret_cast<uintptr_t>(x) & 15) == 0;
  // large batches of small images with few channels: several whole images per block
  if (a16 && (C % 16) == 0 && C <= 64 && (HW % 4) == 0 && HW <= 256 && C * HW <= 12 * 1024 && N >= 8 * kNumSMs) {
    const int ipb = std::max(1, std::min(16, (24 * 1024) / (C * HW)));
    const size_t smem = (size_t)ipb * C * HW;
    return launch_pdl(pack_small_images_kernel, dim3((unsigned)((N + ipb - 1) / ipb)), dim3(kPackThreads), smem, st, x, out, N, C,
                      HW, C_pad, ipb, status, dbg);
  }
  // Bulk-copy kernels: channels in whole groups of 16 and either the whole image per tile
  // (H*W <= 256, a multiple of 4) or rows that are multiples of 16 bytes.
  if (a16 && (C % 16) == 0 && (HW % 4) == 0 && (HW <= 256 || (HW % 16) == 0)) {
    const bool row_mode = HW > 256;
    const int PT = row_mode ? 256 : HW;
    const int hw_tiles = (HW + PT - 1) / PT;
    // small tensors: narrower channel tiles so that the grid still covers the machine
    while (CT > 32 && (long long)hw_tiles * N * ((C_pad + CT - 1) / CT) < 2 * kNumSMs) CT >>= 1;
    const size_t smem = (size_t)(CT / 16) * (16 * PT + 16);
    dim3 grid((unsigned)hw_tiles * (unsigned)N, (C_pad + CT - 1) / CT, 1);
    if (row_mode)
      return launch_pdl(pack_activations_bulk_kernel<true>, grid, dim3(kPackThreads), smem, st, x, out, C, HW, C_pad,
                        hw_tiles, CT, PT, status, dbg);
    return launch_pdl(pack_activations_bulk_kernel<false>, grid, dim3(kPackThreads), smem, st, x, out, C, HW, C_pad,
                      hw_tiles, CT, PT, status, dbg);
  }
  const int PT = HW > 128 ? 256 : (HW > 64 ? 128 : 64);
  const int hw_tiles = (HW + PT - 1) / PT;
  dim3 grid((unsigned)hw_tiles * (unsigned)N, (C_pad + CT - 1) / CT, 1);
  if ((HW % 16) == 0 && a16)
    return launch_pdl(pack_activations_kernel<16>, grid, dim3(kPackThreads), 0, st, x, out, C, HW, C_pad, hw_tiles, CT,
                      PT, dbg);
  if ((HW % 4) == 0 && a16)
    return launch_pdl(pack_activations_kernel<4>, grid, dim3(kPackThreads), 0, st, x, out, C, HW, C_pad, hw_tiles, CT,
                      PT, dbg);
  return launch_pdl(pack_activations_kernel<1>, grid, dim3(kPackThreads), 0, st, x, out, C, HW, C_pad, hw_tiles, CT, PT, dbg);
}

cudaError_t launch_pack_wait_selftest(int* status, cudaStream_t st) {
  pack_wait_selftest_kernel<<<1, 64, 0, st>>>(status);
  return cudaGetLastError();
}

cudaError_t launch_pack_weights_cp(const int8_t* w, int8_t* out, int K, int C, int R, int S, int C_pad,
                                   cudaStream_t st) {
  const long long total = (long long)K * R * S * C_pad;
  pack_weights_cp_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, out, K, C, R * S, C_pad);
  return cudaGetLastError();
}

cudaError_t launch_pack_weights_table(const int8_t* w, int8_t* out, int K, int Kg, int cols, const int32_t* table,
                                      cudaStream_t st) {
  const long long total = (long long)K * cols;
  pack_weights_table_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, out, K, Kg, cols, table);
  return cudaGetLastError();
}

namespace {
__global__ void expand_group_weights_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ out, int K, int cg, int kg,
                                            int m, int RS) {
  pdl_wait();
  const long long row = (long long)m * cg * RS;  // elements of one expanded filter
  const long long total = (long long)K * row;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int k = (int)(i / row);
    const int rem = (int)(i - (long long)k * row);
    const int c = rem / RS, t = rem - c * RS;
    const int slot = (k / kg) % m;  // which of the merged groups filter k belongs to
    out[i] = (c / cg == slot) ? w[((long long)k * cg + (c - slot * cg)) * RS + t] : (int8_t)0;
  }
  pdl_launch_dependents();
}
}  // namespace

cudaError_t launch_expand_group_weights(const int8_t* w, int8_t* out, int K, int cg, int kg, int m, int RS, cudaStream_t st) {
  const long long total = (long long)K * m * cg * RS;
  const int blocks = (int)std::min<long long>((total + 255) / 256, 148 * 8);
  return launch_pdl(expand_group_weights_kernel, dim3((unsigned)std::max(1, blocks)), dim3(256), 0, st, w, out, K, cg, kg, m, RS);
}

cudaError_t launch_pack_weights_rows(const int8_t* w, int8_t* out, int K, int Kg, int K_pad, int S, int S_run,
                                     cudaStream_t st) {
  const long long total = (long long)K * K_pad;
  pack_weights_rows_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, out, K, Kg, K_pad, S, S_run);
  return cudaGetLastError();
}

cudaError_t launch_im2col(const int8_t* x, int8_t* a, const GatherEntry* table, long long Mg, int PQ, int Q, int H,
                          int W, int stride_h, int stride_w, int pad_h, int pad_w, long long x_stride_n,
                          int x_stride_h, int x_stride_w, int K_pad, cudaStream_t st, const Dbg& dbg) {
  const long long total = Mg * (K_pad / 16);
  return launch_pdl(im2col_kernel, dim3(grid_for(total, 256)), dim3(256), 0, st, x, a, table, Mg, PQ, Q, H, W, stride_h,
                    stride_w, pad_h, pad_w, x_stride_n, x_stride_h, x_stride_w, K_pad, dbg);
}

cudaError_t launch_space_to_depth(const int8_t* x, int8_t* out, int N, int Hs, int Ws, int C, int H, int W, int sh,
                                  int sw, int pad_h, int pad_w, int C_pad, int pack, long long stride_n,
                                  long long stride_c, int stride_h, int stride_w, cudaStream_t st, const Dbg& dbg) {
  // Fast path: NCHW rows that are multiples of 16 bytes, row segments of a tile within 48 KB.
  const int seg = ((kS2dTile * sw + pack * sw + 15 + 15) / 16) * 16;  // bytes of one input row a tile reads, from a 16-byte boundary
  const long long smem = (long long)C * sh * seg;
  const long long blocks = (long long)N * Hs * ((Ws + kS2dTile - 1) / kS2dTile);
  if (stride_w == 1 && stride_h == W && stride_c == (long long)H * W && (W % 16) == 0 &&
      (reinterpret_cast<uintptr_t>(x) & 15) == 0 && smem <= 48 * 1024 && blocks < 0x7FFFFFFFLL && Ws >= 32)
    return launch_pdl(space_to_depth_rows_kernel, dim3((unsigned)blocks), dim3(kS2dTile), (size_t)smem, st, x, out, Hs, Ws, C,
                      H, W, sh, sw, pad_h, pad_w, C_pad, pack, seg, (Ws + kS2dTile - 1) / kS2dTile, dbg);
  // total 16-byte chunks of the scratch tensor; the planner keeps N*Hs*Ws*C_pad below 2^40 and one
  // image below 2^31 bytes, and the launch below is split so that each part's chunk count fits 32 bits
  const long long per_image = (long long)Hs * Ws * (C_pad / 16);
  const int images_per_launch = (int)std::max<long long>(1, std::min<long long>(N, 0x7FFFFFFFLL / per_image));
  for (int n0 = 0; n0 < N; n0 += images_per_launch) {
    const int nn = std::min(images_per_launch, N - n0);
    const long long total = per_image * nn;
    cudaError_t e = launch_pdl(space_to_depth_kernel, dim3(grid_for(total, 256)), dim3(256), 0, st,
                               x + (long long)n0 * stride_n, out + (long long)n0 * per_image * 16, (unsigned)total,
                               make_fastdiv((uint32_t)(C_pad / 16)), make_fastdiv((uint32_t)Ws), make_fastdiv((uint32_t)Hs),
                               C, H, W, sh, sw, pad_h, pad_w, C_pad, pack, stride_n, (int)stride_c, stride_h, stride_w, dbg);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_row_phase_unroll(const int8_t* x, int8_t* out, int N, int Hs, int Q, int C, int H, int W, int S, int sh,
                                    int sw, int pad_h, int pad_w, int dil_w, int C_pad, long long stride_n,
                                    long long stride_c, int stride_h, int stride_w, cudaStream_t st, const Dbg& dbg) {
  // bytes of one input row a tile of kS2dTile pixels reads, counted from a 16-byte boundary
  static_assert(kRowPhaseTile == kS2dTile, "one pixel per thread");
  const int seg = row_phase_seg(sw, S, dil_w);
  const long long smem = (long long)C * sh * seg;
  const int q_tiles = (Q + kS2dTile - 1) / kS2dTile;
  const long long blocks = (long long)N * Hs * q_tiles;
  if (smem > kRowPhaseSmemMax || blocks >= 0x7FFFFFFFLL) return cudaErrorInvalidValue;
  const int vec_ok = (stride_w == 1 && (stride_h % 16) == 0 && (stride_c % 16) == 0 && (stride_n % 16) == 0 &&
                      (reinterpret_cast<uintptr_t>(x) & 15) == 0)
                         ? 1
                         : 0;
  static std::atomic<unsigned long long> configured{0};
  cudaError_t ea = set_max_dynamic_smem_once(configured, (const void*)row_phase_unroll_kernel, kRowPhaseSmemMax);
  if (ea != cudaSuccess) return ea;
  return launch_pdl(row_phase_unroll_kernel, dim3((unsigned)blocks), dim3(kS2dTile), (size_t)smem, st, x, out, Hs, Q, C, H,
                    W, S, sh, sw, pad_h, pad_w, dil_w, C_pad, seg, q_tiles, stride_n, stride_c, stride_h, stride_w, vec_ok, dbg);
}

cudaError_t launch_phase_split(const int8_t* x, int8_t* out, int N, int C, int H, int W, int dh, int dw, int Hs, int Ws,
                               int C_pad, long long stride_n, long long stride_c, int stride_h, int stride_w,
                               cudaStream_t st, const Dbg& dbg) {
  const long long total = (long long)N * dh * dw * Hs * Ws * (C_pad / 16);
  return launch_pdl(phase_split_kernel, dim3(grid_for(total, 256)), dim3(256), 0, st, x, out, N, C, H, W, dh, dw, Hs, Ws,
                    C_pad, stride_n, stride_c, stride_h, stride_w, dbg);
}

cudaError_t launch_splitk_finish(const int32_t* acc, int32_t* y32, int8_t* y8, long long elems, int shift,
                                 int out_mode, const int32_t* bias, int relu, int K, int PQ, int nhwc, cudaStream_t st,
                                 const Dbg& dbg) {
  return launch_pdl(splitk_finish_kernel, dim3(grid_for(elems, 256)), dim3(256), 0, st, acc, y32, y8, elems, shift,
                    out_mode, bias, relu, K, PQ, nhwc, dbg);
}

}  // namespace b2c

// ---------------------------------------------------------------------------------------------
// Stencil unroll for callers that cannot allocate device memory.
//
// b2c_im2col builds its lookup table on the host and puts it in a temporary cudaMalloc buffer.
// Some callers cannot do that: code running inside a stream capture or under a framework's
// "no allocation from here on" rule, real-time loops that must not touch the allocator, or
// processes whose memory pool was handed to another library in full.  For them the table lives in
// the fixed device array below (128 KB, resident on every GPU that loads the library until the
// process exits) and is filled by a small kernel on the caller's stream.
// ---------------------------------------------------------------------------------------------
namespace b2c {
namespace {

constexpr int kStaticTableEntries = 16384;  // largest padded reduction length C*R*S the static table can hold
static __device__ __align__(256) GatherEntry g_static_table[kStaticTableEntries];

// Writes entries [0, K_pad): (c, r, s) -> element offset and displacement; -1 past C*R*S.  Every
// entry a later im2col launch reads is rewritten here, so nothing of an earlier call survives.
__global__ void fill_static_table_kernel(GatherEntry* table, int K_pad, int Kg, int R, int S, int dil_h, int dil_w,
                                         long long stride_c, long long stride_h, long long stride_w) {
  for (int kg = blockIdx.x * blockDim.x + threadIdx.x; kg < K_pad; kg += gridDim.x * blockDim.x) {
    GatherEntry e;
    if (kg < Kg) {
      const int s = kg % S;
      const int cr = kg / S;
      const int r = cr % R;
      const int c = cr / R;
      e.off = (int32_t)(c * stride_c + (long long)r * dil_h * stride_h + (long long)s * dil_w * stride_w);
      e.dh = (int16_t)(r * dil_h);
      e.dw = (int16_t)(s * dil_w);
    } else {
      e.off = -1;
      e.dh = 0;
      e.dw = 0;
    }
    table[kg] = e;
  }
}

// Device address of g_static_table, looked up once per device.  In host code the array's name is
// only a handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress.
constexpr int kMaxDevices = 64;
GatherEntry* g_static_table_addr[kMaxDevices] = {};

int static_table_address(GatherEntry** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    set_last_cuda_error((int)(e != cudaSuccess ? e : cudaErrorInvalidDevice));
    return B2C_E_CUDA;
  }
  GatherEntry* p = __atomic_load_n(&g_static_table_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_table);
    if (e != cudaSuccess || !p) {
      set_last_cuda_error((int)e);
      return B2C_E_CUDA;
    }
    __atomic_store_n(&g_static_table_addr[dev], p, __ATOMIC_RELEASE);
  }
  *out = p;
  return B2C_OK;
}

}  // namespace
}  // namespace b2c

extern "C" int b2c_im2col_noalloc(const b2c_conv_desc* desc, const int8_t* x, int8_t* a, int K_pad, void* cuda_stream) {
  using namespace b2c;
  if (!desc || !x || !a) return B2C_E_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(a) & 15)) return B2C_E_INVALID_ARG;
  b2c_conv_desc d = *desc;
  if ((d.out_mode & 3) == 0) d.out_mode = B2C_OUT_I32;
  Geom g;
  int rc = resolve_geom(&d, &g);
  if (rc != B2C_OK) return rc;
  if (K_pad < g.Kg || (K_pad % 16) != 0) return B2C_E_INVALID_ARG;
  if (K_pad > kStaticTableEntries) return B2C_E_WORKSPACE_TOO_SMALL;
  if ((long long)(d.R - 1) * d.dil_h >= 32768 || (long long)(d.S - 1) * d.dil_w >= 32768 ||
      (long long)d.C * d.H * d.W >= 0x7FFFFFFFLL)
    return B2C_E_UNSUPPORTED;
  GatherEntry* table = nullptr;
  rc = static_table_address(&table);
  if (rc != B2C_OK) return rc;
  const bool nchw = d.in_layout == B2C_LAYOUT_NCHW;
  const long long sc = nchw ? (long long)d.H * d.W : 1;
  const long long sh = nchw ? d.W : (long long)d.W * d.C;
  const long long sw = nchw ? 1 : d.C;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  fill_static_table_kernel<<<(K_pad + 255) / 256, 256, 0, st>>>(table, K_pad, g.Kg, d.R, d.S, d.dil_h, d.dil_w, sc, sh,
                                                                 sw);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess)
    e = launch_im2col(x, a, table, g.Mg, g.PQ, g.Q, d.H, d.W, d.stride_h, d.stride_w, d.pad_h, d.pad_w,
                      (long long)d.C * d.H * d.W, (int)sh, (int)sw, K_pad, st);
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return B2C_E_CUDA;
  }
  return B2C_OK;
}

