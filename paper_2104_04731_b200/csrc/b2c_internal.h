// Internal declarations shared by the host code and the kernel launchers of libb2conv.
// Nothing here is part of the public ABI (see include/b2conv.h).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "b2conv.h"

namespace b2c {

constexpr int kTileM = 128;       // rows of one tcgen05.mma accumulator tile (cta_group::1)
constexpr int kMmaK = 32;         // reduction depth of one kind::i8 instruction (bytes per row)
constexpr int kMaxKg = 131071;    // C*R*S bound that keeps |acc| <= Kg * 2^14 inside int32
constexpr int kNumSMs = 148;

// Resolved geometry of one convolution.
struct Geom {
  b2c_conv_desc d;
  int P, Q;
  int PQ;
  long long Mg;  // N*P*Q
  int Kg;        // C*R*S
  long long x_elems, w_elems, y_elems;
};

// One entry of the stencil lookup table used by the in-kernel gather and the explicit unroll:
// reduction index kg = (c*R + r)*S + s  ->  element offset from the window's top-left input
// element and the (dh, dw) displacement used for the bounds test.  Entries past C*R*S (the
// zero padding of the reduction axis) have off = -1.
struct GatherEntry {
  int32_t off;
  int16_t dh;
  int16_t dw;
};

// Division of a non-negative 31-bit integer by a run-time constant as multiply + shift
// (round-up method: l = ceil(log2 d), m = ceil(2^(31+l) / d), n / d = (n * m) >> (31 + l) for all
// 0 <= n < 2^31).  Per-thread index arithmetic in the kernels uses it instead of the ~20
// instruction hardware-less integer division.
struct FastDiv {
  uint32_t mul;
  uint32_t shr;
  uint32_t d;
#ifdef __CUDACC__
  __host__ __device__
#endif
  inline uint32_t div(uint32_t n) const {
    return (uint32_t)(((unsigned long long)n * mul) >> shr);
  }
};
inline FastDiv make_fastdiv(uint32_t d) {
  FastDiv f;
  f.d = d;
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;
  f.shr = 31 + l;
  f.mul = (uint32_t)(((1ull << (31 + l)) + d - 1) / d);
  return f;
}

// Debug build (-DB2C_DEBUG_BOUNDS, libb2conv_debug.so): the address ranges every hand-computed global
// access of a kernel must stay inside.  A null `lo` leaves that range unchecked.  In the release build
// the struct travels along unused and every check below compiles to `true`.
struct Dbg {
  const void* x_lo = nullptr;    // the tensor the kernel reads with its own loads or bulk copies
  long long x_bytes = 0;
  const void* o32_lo = nullptr;  // int32 output
  long long o32_bytes = 0;
  const void* o8_lo = nullptr;   // int8 output
  long long o8_bytes = 0;
  const void* ws_lo = nullptr;   // scratch the kernel writes (rewritten operand, split-reduction sums, counters)
  long long ws_bytes = 0;
  int* status = nullptr;         // [0] status word, [1] site, [2..3] byte offset of the first bad access from its range start
};

enum AMode { A_TILED = 0, A_IM2COL_TMA = 1, A_GATHER = 2, A_STAGED = 3, A_SHIFT = 4, A_WINDOW = 5 };

// Everything the MMA kernel needs besides its two tensor maps.
struct ConvArgs {
  int32_t* y32;
  int8_t* y8;
  int32_t* acc;  // split-K accumulation buffer (int32, output index order), or nullptr
  int* status;
  const int8_t* x;
  const GatherEntry* table;
  const int32_t* table32;  // staged window: reduction index -> byte offset inside the window, -1 for padding
  long long x_stride_n;
  int x_stride_h, x_stride_w;
  int Mg, K, PQ, Q, H, W;
  int stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  int S;
  int num_kb;       // 128-byte (or bk-byte) reduction blocks in total
  int ksteps_full;  // MMA instructions per full block (bk / 32)
  int ksteps_last;  // MMA instructions in the last block
  int kb_per_tap;   // channel-pack map: blocks per filter tap
  int tap_cols;     // channel-pack map: columns of the packed weight matrix per tap (C_pad)
  int table_len;    // gather: entries of the lookup table (padded reduction length)
  // staged window (A_STAGED): per image part, C x win_rows rows of win_pitch bytes; image column 0
  // sits at byte win_left of a row; win_bytes covers the parts a tile can touch
  FastDiv div_pq, div_q, div_vec_per_row, div_c_rows, div_rows;  // by PQ, Q, win_pitch/16, C*win_rows, win_rows
  int C, P, win_rows, win_pitch, win_left, win_bytes, win_tap_span, win_word_mode;
  int bk;           // bytes of reduction per block: 32, 64 or 128
  int tile_n;
  int tmem_cols;
  int stages;
  int split_k;
  int shift, out_mode, out_layout;
  // persistent mode: gridDim.x blocks walk num_tiles tiles (tiles_n column tiles per row tile);
  // tmem_bufs accumulator buffers of tmem_cols columns each
  int persistent, num_tiles, tiles_n, tmem_bufs;
  FastDiv div_tiles_n;
  int stage_region;   // bytes of shared memory reserved for the stage ring (and the cluster exchange tile)
  int cluster_split;  // split_k slices form a cluster (1, 1, split_k) and reduce through shared memory
  // swapped axis map: accumulator rows = output channels (the 128-row MMA operand is the packed
  // weights), accumulator columns = tile_n fused (n, p, q) pixels (the N operand is the activations)
  int swap;
  // Output geometry.  out_PQ is the channel stride of the NKPQ tensor (always the convolution's own
  // P*Q).  remap != 0 (dilation phase pack): accumulator row m' = (n', p', q') of the phase
  // sub-image convolution belongs to image n = n' / (ph_dh*ph_dw), phase (a, b) = the remainder,
  // output pixel p = (p' - ph_pad_h)*ph_dh + a + out_pad_h (q likewise), and is dropped when that
  // pixel lies outside the out_P x out_Q output.
  int out_PQ, remap, ph_dh, ph_dw, ph_pad_h, ph_pad_w, out_pad_h, out_pad_w, out_P, out_Q;
  // Stencil as operand shift (A_SHIFT; stride-1 geometry over an NHWC tensor with padded channels).
  // Accumulator rows enumerate window origins on a grid of sh_hp x sh_wps positions per image
  // (sh_wps = padded width rounded up to 8, so that every staged image row starts on a swizzle
  // atom); a tile's 128 consecutive positions read, for tap (r, s), the 128 consecutive staged
  // pixels that start (r*dil_h*sh_wps + s*dil_w) pixels further on.  One stage holds sh_rows padded
  // image rows per channel block; the packed weights stay resident in shared memory.
  int sh_wps, sh_hp, sh_rows, sh_row_bytes, sh_ncb, sh_R, sh_cblk_bytes, sh_win_bytes, sh_w_bytes, sh_mtot;
  // two-dimensional tiles (remap == 3): tile t = (image, tile row, tile column); accumulator row m of
  // a tile is pixel (m / tile_w, m % tile_w) of it (tile_w = sh_wps); the window is one box per channel block
  int sh_tiles_h, sh_tiles_w, sh_valid_w;  // sh_valid_w: columns of a tile that are outputs (tiles advance by it)
  FastDiv div_tiles_hw, div_tiles_w;
  int persistent_blocks_per_sm;  // blocks per SM the persistent grid is sized for (0: the mode's default)
  // Two-SM schedule: a pair of blocks (cluster of two) owns a 256 x tile_n tile; num_tiles counts pair
  // tiles, every block loads its own 128 A rows and tile_n / 2 B rows per stage.
  int pair;
  // Activation pack fused into the two-SM kernel (NCHW input, channel-pack map): four extra warps of
  // every block rewrite the input into the NHWC scratch tensor that the kernel's own TMA loads read,
  // in batches of pk_ct channels x pk_pt pixels of one image (units of 16 channels), taken from a
  // global work counter in image order; pk_ctl[0] is that counter, pk_ctl[1 + n] counts the finished
  // units of image n, and a tile's loads start once all units of its images are done.
  const int8_t* pk_src;
  int8_t* pk_dst;
  int* pk_ctl;
  int pk_on, pk_N, pk_C, pk_HW, pk_Cpad, pk_ct, pk_pt, pk_hw_tiles, pk_ctiles, pk_smem;
  // Stencil unroll from a TMA-staged two-dimensional window (A_WINDOW): tiles of (128 / wn_tile_w) x
  // wn_tile_w output pixels (sh_tiles_h x sh_tiles_w tiles per image); the window of a tile is C x win_h
  // rows of wn_win_w bytes, its first byte wn_left columns left of the tile's first input column
  // (wn_off0 = wn_left - pad_w bytes before the first tap); wn_chunks 16-byte chunks per A row.
  // wn_linear: tiles are 128 consecutive fused pixels, the window holds whole images (wn_box_bytes each,
  // behind a margin of wn_left bytes), taps outside the image are masked by the builders.
  int wn_tile_w, wn_win_w, wn_win_bytes, wn_box_bytes, wn_left, wn_off0, wn_chunks, wn_linear;
  // Grouped convolution in one launch (in-kernel stencil unroll, NCHW / NKPQ): blockIdx.z is the group;
  // group g reads channels [g*C, (g+1)*C) of x (group_x_stride elements further on per group), uses rows
  // [g*K, (g+1)*K) of the packed weights and of the bias, and writes output channels [g*K, (g+1)*K).
  int groups;
  long long group_x_stride;
  Dbg dbg;  // debug build: ranges of x, the outputs and the scratch
  FastDiv div_wps, div_hp;
  // elements between consecutive images of the NKPQ output (K * P * Q, or more when this
  // convolution writes one channel group of a wider tensor)
  long long y_stride_n;
  // activation step applied to the complete sums before they are written: + bias[k] (nullptr: none),
  // then max(., 0) when relu != 0
  const int32_t* bias;
  int relu;
};

// Programmatic dependent launch: a kernel launched through launch_pdl may start while the previous
// kernel of the stream is still running; it must call pdl_wait() before its first access to global
// memory that an earlier kernel may write or still read, and calls pdl_launch_dependents() once the
// next kernel may begin its own set-up.  Every kernel of this library follows that rule, so the
// stream order of memory effects is unchanged; what overlaps is launch latency and block set-up.
#ifdef __CUDACC__
#ifdef B2C_DEBUG_BOUNDS
// True when [p, p + n) lies inside [lo, lo + bytes) (or the range is unchecked).  Otherwise the first
// offender records B2C_E_BOUNDS, its site and its byte offset from the range start in the status
// words, and the caller skips the access.
__device__ __forceinline__ bool b2c_dbg_in_range(int* status, int site, const void* lo, long long bytes, const void* p,
                                                 long long n) {
  if (lo == nullptr) return true;
  const long long off = (const char*)p - (const char*)lo;
  if (off >= 0 && off + n <= bytes) return true;
  if (status != nullptr && atomicCAS(status, 0, B2C_E_BOUNDS) == 0) {
    status[1] = site;
    status[2] = (int)(off & 0xFFFFFFFFLL);
    status[3] = (int)(off >> 32);
  }
  return false;
}
#define B2C_X_OK(d, site, p, n) b2c_dbg_in_range((d).status, site, (d).x_lo, (d).x_bytes, p, n)
#define B2C_O32_OK(d, site, p, n) b2c_dbg_in_range((d).status, site, (d).o32_lo, (d).o32_bytes, p, n)
#define B2C_O8_OK(d, site, p, n) b2c_dbg_in_range((d).status, site, (d).o8_lo, (d).o8_bytes, p, n)
#define B2C_WS_OK(d, site, p, n) b2c_dbg_in_range((d).status, site, (d).ws_lo, (d).ws_bytes, p, n)
#else
#define B2C_X_OK(d, site, p, n) true
#define B2C_O32_OK(d, site, p, n) true
#define B2C_O8_OK(d, site, p, n) true
#define B2C_WS_OK(d, site, p, n) true
#endif
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                               int cluster_z, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.numAttrs = 1;
  if (cluster_z > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = (unsigned)cluster_z;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  return launch_pdl_cluster(kernel, grid, block, smem, st, 1, static_cast<Args&&>(args)...);
}
#endif

// Opt-in to more than 48 KB of dynamic shared memory for one kernel.  The attribute belongs to the
// current device's context, so it is set once per (kernel, device): `done` holds one bit per device
// ordinal (devices past 63 set it on every launch).  Safe from concurrent host threads.
inline cudaError_t set_max_dynamic_smem_once(std::atomic<unsigned long long>& done, const void* kernel, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess && tracked) done.fetch_or(1ull << dev, std::memory_order_release);
  return e;
}

// What the im2col-mode-TMA convolution kernel is given: an NHWC int8 tensor whose channel count is
// a multiple of 32 and a filter geometry over it.  The channel-pack map uses the (padded) input
// itself; the row-unroll and space-to-depth maps first rewrite the input into a scratch tensor for
// which the remaining convolution has this simpler geometry.  In every case the output extent and
// pixel order are those of the original convolution.
struct TmaView {
  int N, C, H, W;  // NHWC tensor, C already padded
  int R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w;
  long long bytes() const { return (long long)N * H * W * C; }
};
inline bool is_tma_view_variant(int v) {
  return v == B2C_VARIANT_CP_TMA || v == B2C_VARIANT_ROW_UNROLL || v == B2C_VARIANT_SPACE_TO_DEPTH ||
         v == B2C_VARIANT_DILATION_PACK || v == B2C_VARIANT_CP_SHIFT || v == B2C_VARIANT_S2D_SHIFT ||
         v == B2C_VARIANT_ROWPHASE_SHIFT;
}
// The two shift variants execute the channel-pack and space-to-depth views (same rewrite, same
// packed weights) with the stencil as operand shifts over a staged window instead of one
// im2col-mode copy per tap.
inline bool is_shift_variant(int v) {
  return v == B2C_VARIANT_CP_SHIFT || v == B2C_VARIANT_S2D_SHIFT || v == B2C_VARIANT_ROWPHASE_SHIFT;
}
// The row-phase view has a single tap per filter row, so its tiles can be two-dimensional
// (tile_h x tile_w output pixels, tile_w a power of two from kShiftTileW to 128, tile_h = 128 / tile_w):
// the window is then one box of (tile_h + R' - 1) x tile_w pixels, tap r' the same tile read r' * tile_w
// pixels on.
constexpr int kShiftTileW = 16;
// Row-phase unroll kernel: pixels per block and bytes of one input row segment a block stages
// (counted from a 16-byte boundary); the C*stride_h segments of a block must fit in shared memory.
constexpr int kRowPhaseTile = 128;
constexpr int kRowPhaseSmemMax = 160 * 1024;
inline int row_phase_seg(int sw, int S, int dil_w) { return ((kRowPhaseTile * sw + (S - 1) * dil_w + 1 + 15 + 15) / 16) * 16; }
inline bool shift_tiles_2d(int v) { return v == B2C_VARIANT_ROWPHASE_SHIFT; }
inline int shift_base_variant(int v) {
  return v == B2C_VARIANT_CP_SHIFT ? B2C_VARIANT_CP_TMA : (v == B2C_VARIANT_S2D_SHIFT ? B2C_VARIANT_SPACE_TO_DEPTH : v);
}
constexpr int kNumVariants = 11;
// Family of a variant for the timed selection's "five best candidates": variants that share the
// kind of rewrite (a view and its shift execution; row unroll with and without the stride phases)
// count as one candidate with several schedules.
inline int variant_family(int v) {
  if (v == B2C_VARIANT_ROWPHASE_SHIFT) return B2C_VARIANT_ROW_UNROLL;
  if (v == B2C_VARIANT_IM2COL_WINDOW) return B2C_VARIANT_IM2COL_STAGED;  // both form the unroll from a staged window
  return shift_base_variant(v);
}
// Shared-memory geometry of the shift execution of a view; false if it does not apply (stride,
// more than 256 output channels, rows wider than one copy, or window + weights beyond shared memory).
struct ShiftGeom {
  int wps, hp, rows, row_bytes, ncb, cb, cblk_bytes, win_bytes, w_bytes, tile_n, stages, blocks_per_sm;
  int two_d, tiles_h, tiles_w, valid_w;  // two-dimensional tiles: pixel columns of a tile that are outputs
  long long mtot;
};
bool shift_geom(const Geom& g, const TmaView& v, ShiftGeom* sg, bool tiles_2d = false);
// Output pixels of the convolution a view describes: the original N*P*Q, except for the dilation
// phase pack, whose sub-image convolutions also produce rows that map outside the output.
long long view_rows(const Geom& g, int variant, const TmaView& v);
bool tma_view_for(const Geom& g, int variant, TmaView* v);  // false: the variant is not legal for g

// --- planner.cpp -------------------------------------------------------------------------------
int resolve_geom(const b2c_conv_desc* d, Geom* g);  // validation + derived sizes; B2C_* code
int round_up(int v, int m);
int cp_channel_pad(int C);           // channels after Pad for the channel-pack map
int cp_block_bytes(int C_pad);       // reduction bytes per block for the channel-pack map
int im2col_k_pad(int Kg);            // padded reduction length for the stencil-unroll maps
void enumerate_embeddings(const Geom& g, std::vector<b2c_embedding>* out);
int pick_by_policy(const std::vector<b2c_embedding>& all, int policy);  // index or -1
size_t workspace_bytes_for(const Geom& g, int variant, int tile_n, int split_k, bool swap = false);
inline bool is_swapped(const b2c_embedding& e) { return e.map_m == B2C_AXIS_K; }
// A split reduction of 2, 4 or 8 slices whose tile is wide enough runs as a thread-block cluster:
// the slices exchange their partial accumulators through distributed shared memory, so no scratch
// buffer, zero-fill or finish pass is needed.
// (The variants that keep a lookup table or an input window in shared memory leave room for a
// 128-column exchange tile at most.)
// Two-SM schedule (tile_m = 256): a pair of blocks shares one accumulator tile of 256 fused pixels.  It
// exists for the TMA-fed maps (operand A by im2col-mode or tiled TMA) without a split reduction, with
// column tiles of 32 to 256 channels (each block loads tile_n / 2 weight rows, at least one 16-row
// group), when the problem has more than one 128-row tile.
inline bool pair_schedule_ok(int variant, int tile_n, int split_k, bool swap, long long rows) {
  const bool tma_fed = variant == B2C_VARIANT_CP_TMA || variant == B2C_VARIANT_IM2COL_EXPLICIT ||
                       variant == B2C_VARIANT_ROW_UNROLL || variant == B2C_VARIANT_SPACE_TO_DEPTH ||
                       variant == B2C_VARIANT_DILATION_PACK;
  return tma_fed && !swap && split_k == 1 && tile_n >= 32 && rows > kTileM;
}
inline bool cluster_split_ok(int variant, int tile_n, int split_k, bool swap = false) {
  // the swapped map and the phase pack (scattered output rows) meet their partial sums in global memory
  if (swap || variant == B2C_VARIANT_DILATION_PACK || is_shift_variant(variant)) return false;
  const bool table_in_smem = variant == B2C_VARIANT_IM2COL_GATHER || variant == B2C_VARIANT_IM2COL_STAGED;
  return (split_k == 2 || split_k == 4 || split_k == 8) && tile_n >= 32 * split_k && (!table_in_smem || tile_n <= 128);
}
// Geometry of the shared-memory input window of the staged stencil unroll; false if it does not fit.
struct WindowGeom {
  int rows, pitch, left, parts, bytes;
};
bool staged_window(const Geom& g, WindowGeom* w);
// Space to depth, horizontal tap packing: when the stride phases of all channels fill at most half
// of the 32-byte channel block, each scratch pixel also carries the phases of its next pack - 1
// horizontal neighbours, and the remaining convolution has ceil(S' / pack) taps per row at a
// horizontal dilation of `pack` instead of S' (the bytes would otherwise be zero padding).
int s2d_pack_factor(const Geom& g);
// Staged stencil unroll with unit horizontal dilation: each (c, r) run of S taps is padded to a
// multiple of 4 so that the A rows are built from aligned 32-bit words of the window.
bool staged_word_mode(const Geom& g);
int staged_run_len(const Geom& g);  // taps per (c, r) run after padding
int variant_k_pad(const Geom& g, int variant);  // padded reduction length of the stencil-unroll variants

constexpr int kWindowStages = 6;  // input windows in flight per block of the window unroll kernel
// Geometry of the TMA-staged window unroll (B2C_VARIANT_IM2COL_WINDOW); false if it does not apply.
struct WindowTile {
  int tile_w, tile_h, win_w, win_h, left, off0, S_run, K_pad, tiles_h, tiles_w, box_bytes, win_bytes, tile_n, num_kb;
  int linear;      // small images: linear tiles over whole images staged by bulk copies (box_bytes = C*H*W, left = margin)
  long long mtot;  // accumulator rows issued: N * tiles_h * tiles_w * 128
  size_t smem;
};
bool window_tile_geom(const Geom& g, WindowTile* wt);

// --- tma.cpp -----------------------------------------------------------------------------------
// Tensor-map encoders obtained through cudaGetDriverEntryPoint (no link-time libcuda dependency).
int encode_tiled_2d(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                    uint32_t box_inner, uint32_t box_outer, int swizzle_bytes);
int encode_tiled_nhwc_rows(CUtensorMap* map, const void* base, int C_pad, int W, int H, int N, int box_c, int box_w,
                           int swizzle_bytes, int box_h = 1);
int encode_im2col_nhwc(CUtensorMap* map, const void* base, int C_pad, int W, int H, int N, int pad_w, int pad_h,
                       int S, int R, int dil_w, int dil_h, int stride_w, int stride_h, int channels_per_pixel,
                       int pixels_per_column, int swizzle_bytes);
int encode_tiled_nchw_window(CUtensorMap* map, const void* base, int W, int H, int C, int N, int box_w, int box_h);
void set_last_cuda_error(int e);
int get_last_cuda_error();

// --- kernel launchers (layout.cu, conv_mma.cu) -------------------------------------------------
// status: device status word that a bounded wait of the kernel reports into, or nullptr
cudaError_t launch_pack_activations(const int8_t* x, int8_t* out, int N, int C, int H, int W, int C_pad,
                                    cudaStream_t st, int* status, const Dbg& dbg = Dbg());
cudaError_t launch_pack_weights_cp(const int8_t* w, int8_t* out, int K, int C, int R, int S, int C_pad,
                                   cudaStream_t st);
cudaError_t launch_pack_weights_table(const int8_t* w, int8_t* out, int K, int Kg, int cols, const int32_t* table,
                                      cudaStream_t st);
// Filters of a grouped convolution [K][cg][RS] expanded for groups merged m at a time: [K][m * cg][RS],
// row k holds its own cg channels at channel offset ((k / kg) % m) * cg and zeros elsewhere.
cudaError_t launch_expand_group_weights(const int8_t* w, int8_t* out, int K, int cg, int kg, int m, int RS, cudaStream_t st);
cudaError_t launch_pack_weights_rows(const int8_t* w, int8_t* out, int K, int Kg, int K_pad, int S, int S_run,
                                     cudaStream_t st);
cudaError_t launch_im2col(const int8_t* x, int8_t* a, const GatherEntry* table, long long Mg, int PQ, int Q, int H,
                          int W, int stride_h, int stride_w, int pad_h, int pad_w, long long x_stride_n,
                          int x_stride_h, int x_stride_w, int K_pad, cudaStream_t st, const Dbg& dbg = Dbg());
cudaError_t launch_space_to_depth(const int8_t* x, int8_t* out, int N, int Hs, int Ws, int C, int H, int W, int sh,
                                  int sw, int pad_h, int pad_w, int C_pad, int pack, long long stride_n,
                                  long long stride_c, int stride_h, int stride_w, cudaStream_t st, const Dbg& dbg = Dbg());
cudaError_t launch_row_phase_unroll(const int8_t* x, int8_t* out, int N, int Hs, int Q, int C, int H, int W, int S, int sh,
                                    int sw, int pad_h, int pad_w, int dil_w, int C_pad, long long stride_n,
                                    long long stride_c, int stride_h, int stride_w, cudaStream_t st, const Dbg& dbg = Dbg());
cudaError_t launch_phase_split(const int8_t* x, int8_t* out, int N, int C, int H, int W, int dh, int dw, int Hs, int Ws,
                               int C_pad, long long stride_n, long long stride_c, int stride_h, int stride_w,
                               cudaStream_t st, const Dbg& dbg = Dbg());
cudaError_t launch_splitk_finish(const int32_t* acc, int32_t* y32, int8_t* y8, long long elems, int shift,
                                 int out_mode, const int32_t* bias, int relu, int K, int PQ, int nhwc, cudaStream_t st,
                                 const Dbg& dbg = Dbg());
cudaError_t launch_conv_mma(int amode, const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const ConvArgs& args,
                            cudaStream_t st);
size_t conv_mma_smem_bytes(int amode, const ConvArgs& args);
cudaError_t launch_conv_mma_pair(int amode, const CUtensorMap* tmap_a, const CUtensorMap* tmap_b, const ConvArgs& args,
                                 cudaStream_t st);
size_t conv_mma_pair_smem_bytes(const ConvArgs& args);
cudaError_t launch_conv_mma_window(const CUtensorMap* tmap_x, const CUtensorMap* tmap_b, const ConvArgs& args, cudaStream_t st);
size_t conv_mma_window_smem_bytes(const ConvArgs& args);
// Geometry of the fused activation pack; false when the tensor has no bulk-copy form.
bool fused_pack_geometry(int C, int H, int W, int C_pad, int* ct, int* pt, int* hw_tiles, int* ctiles, int* smem);
cudaError_t launch_bounded_wait_selftest(int* status, cudaStream_t st);
cudaError_t launch_pack_wait_selftest(int* status, cudaStream_t st);

}  // namespace b2c
