// C ABI of libb2conv: descriptor validation, plan objects, the run path (layout rewrite ->
// MMA kernel with fused epilogue -> optional split-reduction finish), the one-shot calls and
// the timed candidate selection.  See include/b2conv.h for the contract of each entry point.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "b2c_internal.h"

using namespace b2c;

struct b2c_plan {
  Geom g;
  b2c_embedding emb;
  int device = 0;
  int8_t* w_packed = nullptr;   // device, plan-owned
  size_t w_packed_bytes = 0;
  GatherEntry* table = nullptr;  // device, plan-owned (stencil lookup table)
  int32_t* table32 = nullptr;    // device, plan-owned (offsets into the staged window)
  WindowGeom win = {0, 0, 0, 0, 0};
  TmaView view = {};             // geometry handed to the im2col-mode-TMA kernel (TMA-view variants)
  int32_t* wtable = nullptr;     // device, plan-owned: packed weight column -> index into one filter, -1 = zero
  int table_len = 0;
  int* status = nullptr;         // device status word
  int32_t* bias_buf = nullptr;   // device, plan-owned copy of the per-channel bias (activation step)
  int32_t* bias = nullptr;       // bias_buf while a bias is set, else null
  int relu = 0;
  bool weights_set = false;
  // derived launch parameters
  int amode = 0;
  int C_pad = 0, K_pad = 0, bk = 128;
  size_t ws_layout_bytes = 0;    // bytes of the layout rewrite's output at the start of the workspace
  size_t ws_total = 0;
  ConvArgs args;
  CUtensorMap tmap_b;
  // one-shot cache extras
  void* own_ws = nullptr;
  // Grouped convolution: the plan owns one sub-plan per group (a dense convolution of C/groups
  // input and K/groups output channels that reads its channel slice of x and writes its slice of
  // y through the batch strides of the whole tensors); the group plan itself launches nothing.
  int groups = 1;
  std::vector<b2c_plan*> subs;
  int group_count = 1;  // on the sub-plan of a group plan: groups run by one launch (blockIdx.z = group)
  // Group merge (group plan): `merge` consecutive groups run as ONE group of merge x the channels with
  // block-diagonal filters (zeros between the groups), so that narrow groups fill the MMA's columns and
  // reduction depth; w_expanded holds the expanded filters [K][merge * C/groups][R][S].
  int merge = 1;
  int8_t* w_expanded = nullptr;  // device, plan-owned
  // Group plan whose one sub-plan is the DENSE convolution of the whole tensors with block-diagonal filters
  // (every group merged): it runs like any dense plan, rewrite and scratch included.
  bool dense_sub = false;
  long long x_stride_n_whole = 0, y_stride_n_whole = 0;  // sub-plans: batch strides of the whole tensors
  struct HostPipe* pipe = nullptr;  // streaming host-buffer calls: created by the first b2c_plan_run_host_async
  // The two-SM persistent channel-pack schedule can run the activation pack inside the MMA kernel
  // (NCHW input whose rows have a bulk-copy form): run then launches one kernel, preceded by a memset
  // of the work counters, which live in the workspace after the rewritten operand.
  bool fused_pack = false;
  size_t ws_ctl_offset = 0;  // bytes from the workspace start to the counters [1 + N] int
  int dbg_site = 0;          // debug build: site and byte offset of the last reported out-of-range access
  long long dbg_offset = 0;
};

// Device side of the streaming host-buffer calls: a ring of input / output buffers and three
// streams (copy in, convolve, copy out) chained by events, so that the copy of call i + 1 and the
// read-back of call i - 1 run beside the kernels of call i.
struct HostPipe {
  static constexpr int kSlots = 3;
  struct Slot {
    int8_t* x = nullptr;
    int32_t* y32 = nullptr;
    int8_t* y8 = nullptr;
    cudaEvent_t in_done = nullptr, run_done = nullptr, out_done = nullptr;
    bool used = false;
  } slot[kSlots];
  cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
  void* ws = nullptr;
  size_t x_bytes = 0, y_elems = 0;
  int next = 0;
};

namespace {

constexpr int kStatusWords = 4;     // [0] status, [1] site, [2..3] byte offset (debug build's bounds report)
#ifdef B2C_DEBUG_BOUNDS
constexpr size_t kCanaryBytes = 64;  // guard band on either side of the caller's workspace
#else
constexpr size_t kCanaryBytes = 0;
#endif
constexpr unsigned char kCanaryByte = 0xC5;
std::atomic<long long> g_dbg_shrink{0};  // test hook: bytes taken off the end of every checked range

#define CUDA_TRY(expr)                  \
  do {                                  \
    cudaError_t e__ = (expr);           \
    if (e__ != cudaSuccess) {           \
      set_last_cuda_error((int)e__);    \
      return B2C_E_CUDA;                \
    }                                   \
  } while (0)

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int tmem_cols_for(int n) {
  int c = 32;
  while (c < n) c <<= 1;
  return c;
}

// Stencil lookup table: reduction index (c, r, s) -> input offset and displacement, in the
// element strides of the activation layout.
void build_table(const Geom& g, int K_pad, std::vector<GatherEntry>* t) {
  const b2c_conv_desc& d = g.d;
  long long sc, sh, sw;
  if (d.in_layout == B2C_LAYOUT_NCHW) {
    sc = (long long)d.H * d.W;
    sh = d.W;
    sw = 1;
  } else {
    sc = 1;
    sh = (long long)d.W * d.C;
    sw = d.C;
  }
  t->assign(K_pad, GatherEntry{-1, 0, 0});
  int kg = 0;
  for (int c = 0; c < d.C; ++c)
    for (int r = 0; r < d.R; ++r)
      for (int s = 0; s < d.S; ++s, ++kg) {
        GatherEntry e;
        e.off = (int32_t)(c * sc + (long long)r * d.dil_h * sh + (long long)s * d.dil_w * sw);
        e.dh = (int16_t)(r * d.dil_h);
        e.dw = (int16_t)(s * d.dil_w);
        (*t)[kg] = e;
      }
}

bool table_variant_legal(const Geom& g) {
  const b2c_conv_desc& d = g.d;
  return (long long)(d.R - 1) * d.dil_h < 32768 && (long long)(d.S - 1) * d.dil_w < 32768 &&
         (long long)d.C * d.H * d.W < 0x7FFFFFFFLL;
}

void fill_common_args(b2c_plan* p) {
  const b2c_conv_desc& d = p->g.d;
  ConvArgs& a = p->args;
  std::memset(&a, 0, sizeof(a));
  a.status = p->status;
  a.table = p->table;
  if (d.in_layout == B2C_LAYOUT_NCHW) {
    a.x_stride_n = (long long)d.C * d.H * d.W;
    a.x_stride_h = d.W;
    a.x_stride_w = 1;
  } else {
    a.x_stride_n = (long long)d.C * d.H * d.W;
    a.x_stride_h = d.W * d.C;
    a.x_stride_w = d.C;
  }
  a.Mg = (int)p->g.Mg;
  a.K = d.K;
  a.PQ = p->g.PQ;
  a.Q = p->g.Q;
  a.H = d.H;
  a.W = d.W;
  a.stride_h = d.stride_h;
  a.stride_w = d.stride_w;
  a.pad_h = d.pad_h;
  a.pad_w = d.pad_w;
  a.dil_h = d.dil_h;
  a.dil_w = d.dil_w;
  a.S = d.S;
  a.tile_n = p->emb.tile_n;
  a.tmem_cols = tmem_cols_for(p->emb.tile_n);
  a.split_k = p->emb.split_k;
  a.shift = d.shift;
  a.out_mode = d.out_mode;
  a.out_layout = d.out_layout;
  a.table_len = p->table_len;
  a.table32 = p->table32;
  a.swap = is_swapped(p->emb) ? 1 : 0;
  a.y_stride_n = (long long)d.K * p->g.PQ;
  a.groups = p->group_count;
  a.group_x_stride = (long long)d.C * d.H * d.W;
  a.out_PQ = p->g.PQ;
  a.out_P = p->g.P;
  a.out_Q = p->g.Q;
  a.C = d.C;
  a.P = p->g.P;
  a.win_rows = p->win.rows;
  a.win_pitch = p->win.pitch;
  a.win_left = p->win.left;
  a.win_bytes = p->win.bytes;
  a.win_tap_span = (d.R - 1) * d.dil_h;
  a.div_pq = make_fastdiv((uint32_t)p->g.PQ);
  a.div_q = make_fastdiv((uint32_t)p->g.Q);
  a.div_vec_per_row = make_fastdiv((uint32_t)std::max(1, p->win.pitch / 16));
  a.div_c_rows = make_fastdiv((uint32_t)std::max(1, d.C * p->win.rows));
  a.div_rows = make_fastdiv((uint32_t)std::max(1, p->win.rows));
  a.win_word_mode = (p->emb.variant == B2C_VARIANT_IM2COL_STAGED && staged_word_mode(p->g)) ? 1 : 0;
  if (is_tma_view_variant(p->emb.variant)) {
    // the kernel walks the view's taps and channel blocks; output extent and order are unchanged
    const TmaView& v = p->view;
    p->amode = A_IM2COL_TMA;
    p->C_pad = v.C;
    p->bk = cp_block_bytes(v.C);
    a.bk = p->bk;
    a.kb_per_tap = v.C / p->bk;
    a.tap_cols = v.C;
    a.num_kb = v.R * v.S * a.kb_per_tap;
    a.ksteps_full = p->bk / kMmaK;
    a.ksteps_last = a.ksteps_full;
    a.stride_h = v.stride_h;
    a.stride_w = v.stride_w;
    a.pad_h = v.pad_h;
    a.pad_w = v.pad_w;
    a.dil_h = v.dil_h;
    a.dil_w = v.dil_w;
    a.S = v.S;
    if (is_shift_variant(p->emb.variant)) {
      ShiftGeom sg;
      shift_geom(p->g, v, &sg, shift_tiles_2d(p->emb.variant));  // legal: checked when the plan was created
      p->amode = A_SHIFT;
      a.Mg = (int)sg.mtot;
      a.sh_mtot = (int)sg.mtot;
      a.sh_wps = sg.wps;
      a.sh_hp = sg.hp;
      a.sh_rows = sg.rows;
      a.sh_row_bytes = sg.row_bytes;
      a.sh_ncb = sg.ncb;
      a.sh_R = v.R;
      a.sh_cblk_bytes = sg.cblk_bytes;
      a.sh_win_bytes = sg.win_bytes;
      a.sh_w_bytes = sg.w_bytes;
      a.div_wps = make_fastdiv((uint32_t)sg.wps);
      a.div_hp = make_fastdiv((uint32_t)sg.hp);
      a.remap = 2;
      if (sg.two_d) {
        a.remap = 3;
        a.sh_tiles_h = sg.tiles_h;
        a.sh_tiles_w = sg.tiles_w;
        a.sh_valid_w = sg.valid_w;
        a.div_tiles_hw = make_fastdiv((uint32_t)(sg.tiles_h * sg.tiles_w));
        a.div_tiles_w = make_fastdiv((uint32_t)sg.tiles_w);
      }
    }
    if (p->emb.variant == B2C_VARIANT_DILATION_PACK) {
      // the kernel's rows are the pixels of the phase sub-image convolutions
      const int Pv = v.H + 2 * v.pad_h - v.R + 1, Qv = v.W + 2 * v.pad_w - v.S + 1;
      a.Mg = (int)view_rows(p->g, p->emb.variant, v);
      a.PQ = Pv * Qv;
      a.Q = Qv;
      a.P = Pv;
      a.div_pq = make_fastdiv((uint32_t)a.PQ);
      a.div_q = make_fastdiv((uint32_t)a.Q);
      a.remap = 1;
      a.ph_dh = d.dil_h;
      a.ph_dw = d.dil_w;
      a.ph_pad_h = v.pad_h;
      a.ph_pad_w = v.pad_w;
      a.out_pad_h = d.pad_h;
      a.out_pad_w = d.pad_w;
    }
  } else if (p->emb.variant == B2C_VARIANT_IM2COL_WINDOW) {
    WindowTile wt;
    window_tile_geom(p->g, &wt);  // legal: checked when the plan was created
    p->amode = A_WINDOW;
    p->K_pad = wt.K_pad;
    p->bk = 128;
    a.bk = 128;
    a.num_kb = wt.num_kb;
    a.ksteps_full = 4;
    a.ksteps_last = (wt.K_pad - (wt.num_kb - 1) * 128) / kMmaK;
    a.Mg = (int)wt.mtot;
    a.wn_tile_w = wt.tile_w;
    a.wn_win_w = wt.win_w;
    a.wn_win_bytes = wt.win_bytes;
    a.wn_box_bytes = wt.box_bytes;
    a.wn_left = wt.left;
    a.wn_off0 = wt.off0;
    a.wn_chunks = wt.K_pad / 16;
    a.wn_linear = wt.linear;
    a.sh_R = d.R;
    a.sh_tiles_h = wt.tiles_h;
    a.sh_tiles_w = wt.tiles_w;
    a.div_tiles_hw = make_fastdiv((uint32_t)(wt.tiles_h * wt.tiles_w));
    a.div_tiles_w = make_fastdiv((uint32_t)wt.tiles_w);
    a.num_tiles = wt.linear ? (int)((wt.mtot + kTileM - 1) / kTileM) : (int)((long long)d.N * wt.tiles_h * wt.tiles_w);
    a.tiles_n = 1;
    a.persistent = 2;
    a.split_k = 1;
    a.cluster_split = 0;
    // accumulator ring: four buffers while two resident blocks' rings fit the 512 columns of tensor memory
    const int per_sm = wt.smem * 2 + 4096 <= 227 * 1024 ? 2 : 1;
    a.tmem_bufs = 4 * a.tmem_cols * per_sm <= 512 ? 4 : (2 * a.tmem_cols * per_sm <= 512 ? 2 : 1);
    if (a.tmem_bufs == 1) a.tmem_bufs = 2;  // (tile_n = 256 leaves one block per SM by shared memory: two buffers fit)
    a.stages = 3;
    a.stage_region = 0;
    return;
  } else {
    p->amode = p->emb.variant == B2C_VARIANT_IM2COL_EXPLICIT
                   ? A_TILED
                   : (p->emb.variant == B2C_VARIANT_IM2COL_STAGED ? A_STAGED : A_GATHER);
    p->K_pad = variant_k_pad(p->g, p->emb.variant);
    p->bk = 128;
    a.bk = 128;
    a.num_kb = (p->K_pad + 127) / 128;
    a.ksteps_full = 4;
    a.ksteps_last = (p->K_pad - (a.num_kb - 1) * 128) / kMmaK;
    a.kb_per_tap = 1;
  }
  // Pipeline depth: as many stages as the reduction slice has blocks, at most 6, within 196 KB (a
  // block that is alone with its tile is paced by the copies it has in flight: a fourth 48 KB stage
  // took 9 % off the 128 x 256 kernel of the 3x3 stride-2 256 -> 512 layer).
  // When the grid has more blocks than the machine has SMs, stay within 100 KB (but keep at least
  // two stages) so that two blocks are resident per SM: one block's epilogue and set-up then
  // overlap the other's main loop.
  int per_cta_kb = (a.num_kb + a.split_k - 1) / a.split_k;
  int stages = std::min(6, std::max(1, per_cta_kb));
  const long long ctas = a.swap ? ((p->g.Mg + a.tile_n - 1) / a.tile_n) * ((d.K + kTileM - 1) / kTileM) * a.split_k
                                : (((long long)a.Mg + kTileM - 1) / kTileM) * ((d.K + a.tile_n - 1) / a.tile_n) * a.split_k *
                                      p->group_count;
  // Large TMA-fed problems run persistently: one block per SM walks the tile list with two
  // accumulator buffers in tensor memory and the deepest stage ring that fits.
  const long long tiles_m = ((long long)a.Mg + kTileM - 1) / kTileM;
  const int tiles_n = (d.K + a.tile_n - 1) / a.tile_n;
  a.tiles_n = tiles_n;
  a.num_tiles = (int)std::min<long long>(tiles_m * tiles_n, 0x7FFFFFFF);
  a.div_tiles_n = make_fastdiv((uint32_t)tiles_n);
  // Wide tiles: one block per SM.  Narrow tiles have short main loops and do better with three
  // blocks per SM, each still walking several tiles (mode 2) once there are enough tiles.
  const bool tma_fed = (p->amode == A_TILED || p->amode == A_IM2COL_TMA) && a.split_k == 1 && !a.swap &&
                       tiles_m * tiles_n < 0x7FFFFFFF;
  a.persistent = 0;
  if (tma_fed && a.tile_n >= 128 && tiles_m * tiles_n > 2 * kNumSMs) a.persistent = 1;
  if (tma_fed && a.tile_n < 128 && tiles_m * tiles_n > 2 * 3 * kNumSMs) a.persistent = 2;
  // the staged-window kernel walks tiles the same way (window restaged per tile)
  if (p->amode == A_STAGED && a.split_k == 1 && tiles_m * tiles_n > 2 * 3 * kNumSMs &&
      tiles_m * tiles_n < 0x7FFFFFFF)
    a.persistent = 2;
  a.tmem_bufs = (a.persistent && 2 * a.tmem_cols <= 512) ? 2 : 1;
  a.pair = p->emb.tile_m == 2 * kTileM ? 1 : 0;
  if (a.pair) {
    // Pair tiles of 256 rows; grids beyond one wave of pairs walk the tile list with one block per SM,
    // two accumulator buffers and the deepest ring that fits; smaller grids keep two blocks per SM
    // (one accumulator each, ring within half of the shared memory) so that one block's set-up and
    // epilogue overlap the other's main loop.
    const long long tiles_m2 = ((long long)a.Mg + 2 * kTileM - 1) / (2 * kTileM);
    a.num_tiles = (int)std::min<long long>(tiles_m2 * tiles_n, 0x3FFFFFFF);
    a.persistent = tiles_m2 * tiles_n > kNumSMs / 2 ? 1 : 0;
    a.tmem_bufs = (a.persistent && 2 * a.tmem_cols <= 512) ? 2 : 1;
    a.cluster_split = 0;
    const size_t pair_stage = (size_t)(kTileM + a.tile_n / 2) * a.bk;
    size_t pair_budget = a.persistent ? 196 * 1024 : 100 * 1024;
    // activation pack inside the kernel: NCHW input of the channel-pack map, persistent grid
    a.pk_on = 0;
    p->fused_pack = false;
    if (a.persistent && p->emb.variant == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NCHW &&
        fused_pack_geometry(d.C, d.H, d.W, p->C_pad, &a.pk_ct, &a.pk_pt, &a.pk_hw_tiles, &a.pk_ctiles, &a.pk_smem) &&
        (long long)d.N * a.pk_hw_tiles * a.pk_ctiles < 0x7FFFFFFFLL) {
      p->fused_pack = true;
      a.pk_N = d.N;
      a.pk_C = d.C;
      a.pk_HW = d.H * d.W;
      a.pk_Cpad = p->C_pad;
      pair_budget = 224 * 1024 - (size_t)a.pk_smem;
    }
    int st = std::min(8, std::max(1, a.num_kb));
    while (st > 2 && (size_t)st * pair_stage > pair_budget) --st;
    a.stages = st;
    a.stage_region = (int)((size_t)st * pair_stage);
    return;
  }
  const size_t budget = a.persistent == 1 ? 196 * 1024 : (a.persistent == 2 ? 68 * 1024 : (ctas > kNumSMs ? 100 * 1024 : 196 * 1024));
  const size_t stage_bytes = (size_t)(kTileM + a.tile_n) * a.bk;
  // lookup table and staged window share the block's shared memory with the stages
  const size_t extra = p->amode == A_STAGED ? (size_t)p->win.bytes + 4 * (size_t)p->table_len + 64
                                            : (p->amode == A_GATHER ? 8 * (size_t)p->table_len : 0);
  while (stages > 2 && (size_t)stages * stage_bytes + extra > budget) --stages;
  while (stages > 1 && (size_t)stages * stage_bytes + extra > 196 * 1024) --stages;
  a.cluster_split = cluster_split_ok(p->emb.variant, a.tile_n, a.split_k, a.swap != 0) ? 1 : 0;
  if (p->amode == A_SHIFT) {
    // the window buffers form the stage ring; the resident weights follow them
    ShiftGeom sg;
    shift_geom(p->g, p->view, &sg, shift_tiles_2d(p->emb.variant));
    a.persistent = 2;
    // Accumulator ring: two buffers; four for tiles of 64 columns and more when the rings of all
    // resident blocks fit the 512 columns of tensor memory (measured: the 64-column 3x3 walk gains
    // 6 % from the deeper ring, the 16-column one loses 6 %, 32 columns are indifferent).
    a.tmem_bufs = (a.tile_n >= 64 && sg.blocks_per_sm * 4 * a.tmem_cols <= 512) ? 4 : (2 * a.tmem_cols <= 512 ? 2 : 1);
    a.tiles_n = 1;
    a.num_tiles = (int)((sg.mtot + kTileM - 1) / kTileM);
    a.div_tiles_n = make_fastdiv(1);
    a.num_kb = 1;
    a.stages = sg.stages;
    a.stage_region = sg.stages * sg.win_bytes + sg.w_bytes;
    a.persistent_blocks_per_sm = sg.blocks_per_sm;
    return;
  }
  size_t region = (size_t)stages * stage_bytes;
  // the stage buffers double as the 128 x tile_n int32 exchange tile of the cluster reduction
  if (a.cluster_split) region = std::max(region, (size_t)kTileM * a.tile_n * 4);
  a.stage_region = (int)region;
  a.stages = stages;
}

int create_plan_for(const Geom& g, const b2c_embedding& emb, b2c_plan** out, int group_count = 1) {
  b2c_plan* p = new (std::nothrow) b2c_plan();
  if (!p) return B2C_E_INVALID_ARG;
  p->g = g;
  p->emb = emb;
  p->group_count = group_count;
  cudaGetDevice(&p->device);
  const b2c_conv_desc& d = g.d;
  auto fail = [&](int code) {
    b2c_plan_destroy(p);
    return code;
  };
  if (cudaMalloc(&p->status, kStatusWords * sizeof(int)) != cudaSuccess) return fail(B2C_E_CUDA);
  if (cudaMemset(p->status, 0, kStatusWords * sizeof(int)) != cudaSuccess) return fail(B2C_E_CUDA);
  if (is_tma_view_variant(emb.variant)) {
    if (!tma_view_for(g, emb.variant, &p->view)) return fail(B2C_E_UNSUPPORTED);
    const TmaView& v = p->view;
    p->w_packed_bytes = (size_t)d.K * v.R * v.S * v.C;
    if (emb.variant != B2C_VARIANT_CP_TMA && emb.variant != B2C_VARIANT_DILATION_PACK &&
        emb.variant != B2C_VARIANT_CP_SHIFT) {
      // Lookup tables of the rewritten maps.  Activations: scratch channel j of scratch pixel
      // (n, h', w') <- input element, in the form the stencil-unroll kernel takes.  Weights: packed
      // column (tap, j) <- index into one KCRS filter.
      const long long sc = d.in_layout == B2C_LAYOUT_NCHW ? (long long)d.H * d.W : 1;
      const long long sw = d.in_layout == B2C_LAYOUT_NCHW ? 1 : d.C;
      std::vector<GatherEntry> t(v.C, GatherEntry{-1, 0, 0});
      std::vector<int32_t> wt((size_t)v.R * v.S * v.C, -1);
      if (emb.variant == B2C_VARIANT_ROWPHASE_SHIFT) {
        // scratch channel j = (dh*S + s)*C + c; packed weight column (r', j) <- filter tap r = r'*stride_h + dh
        // (the activation rewrite has a kernel of its own and needs no table)
        for (int dh = 0; dh < d.stride_h; ++dh)
          for (int s = 0; s < d.S; ++s)
            for (int c = 0; c < d.C; ++c) {
              const int j = (dh * d.S + s) * d.C + c;
              for (int rp = 0; rp < v.R; ++rp) {
                const int r = rp * d.stride_h + dh;
                if (r < d.R) wt[(size_t)rp * v.C + j] = (c * d.R + r) * d.S + s;
              }
            }
      } else if (emb.variant == B2C_VARIANT_ROW_UNROLL) {
        for (int s = 0; s < d.S; ++s)
          for (int c = 0; c < d.C; ++c) {
            const int j = s * d.C + c;
            t[j] = GatherEntry{(int32_t)(c * sc + (long long)s * d.dil_w * sw), 0, (int16_t)(s * d.dil_w)};
            for (int r = 0; r < d.R; ++r) wt[(size_t)r * v.C + j] = (c * d.R + r) * d.S + s;
          }
      } else {
        // space to depth with horizontal tap packing: scratch channel (c, dh, ui, dw) of pixel w' is phase
        // (dh, dw) of channel c at scratch column w' + ui; tap s'' of the view stands for columns
        // pack*s'' + ui (the activation rewrite has a kernel of its own and needs no table)
        const int pack = s2d_pack_factor(g);
        for (int ui = 0; ui < pack; ++ui)
          for (int c = 0; c < d.C; ++c)
            for (int dh = 0; dh < d.stride_h; ++dh)
              for (int dw = 0; dw < d.stride_w; ++dw) {
                const int j = (((c * d.stride_h + dh) * pack) + ui) * d.stride_w + dw;
                for (int rp = 0; rp < v.R; ++rp)
                  for (int sp = 0; sp < v.S; ++sp) {
                    const int r = rp * d.stride_h + dh, s = (sp * pack + ui) * d.stride_w + dw;
                    if (r < d.R && s < d.S) wt[((size_t)rp * v.S + sp) * v.C + j] = (c * d.R + r) * d.S + s;
                  }
              }
      }
      p->table_len = (int)t.size();
      if (cudaMalloc(&p->table, t.size() * sizeof(GatherEntry)) != cudaSuccess) return fail(B2C_E_CUDA);
      if (cudaMemcpy(p->table, t.data(), t.size() * sizeof(GatherEntry), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(B2C_E_CUDA);
      if (cudaMalloc(&p->wtable, wt.size() * sizeof(int32_t)) != cudaSuccess) return fail(B2C_E_CUDA);
      if (cudaMemcpy(p->wtable, wt.data(), wt.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(B2C_E_CUDA);
    }
  } else {
    int K_pad = variant_k_pad(g, emb.variant);
    p->w_packed_bytes = (size_t)d.K * K_pad * group_count;  // grouped: the filters of all groups, one block of K rows each
    std::vector<GatherEntry> t;
    build_table(g, K_pad, &t);
    p->table_len = K_pad;
    if (cudaMalloc(&p->table, t.size() * sizeof(GatherEntry)) != cudaSuccess) return fail(B2C_E_CUDA);
    if (cudaMemcpy(p->table, t.data(), t.size() * sizeof(GatherEntry), cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(B2C_E_CUDA);
    if (emb.variant == B2C_VARIANT_IM2COL_WINDOW) {
      WindowTile wt;
      if (!window_tile_geom(g, &wt)) return fail(B2C_E_UNSUPPORTED);
      // one entry per 32-bit word of an A row: byte offset of the word's first tap inside the window
      // [c][row][byte]; words of the reduction padding point at the window's start (their weights are zero)
      std::vector<int32_t> t32(K_pad / 4, 0);
      for (int wi = 0; wi < K_pad / 4; ++wi) {
        const int run = (wi * 4) / wt.S_run, s0 = (wi * 4) % wt.S_run;
        if (run >= d.C * d.R) continue;
        t32[wi] = ((run / d.R) * wt.win_h + (run % d.R) * d.dil_h) * wt.win_w + s0;
        // linear tiles: + the filter row (bits 16-23) and the word of the run (bits 24-31) for the masks
        if (wt.linear) t32[wi] |= ((run % d.R) << 16) | ((s0 >> 2) << 24);
      }
      if (!wt.linear) {
        // two-dimensional tiles: the low two bits of a chunk's first entry say how its four words lie
        // (offsets are multiples of 4): 0 = 16 consecutive bytes, 1 = two runs of 8 bytes, 2 = anything else
        for (int ch = 0; ch + 3 < (int)t32.size(); ch += 4) {
          const int o0 = t32[ch], o1 = t32[ch + 1], o2 = t32[ch + 2], o3 = t32[ch + 3];
          int kind = 2;
          if (o1 == o0 + 4 && o2 == o0 + 8 && o3 == o0 + 12) kind = 0;
          else if (o1 == o0 + 4 && o3 == o2 + 4) kind = 1;
          t32[ch] = o0 | kind;
        }
      }
      p->table_len = (int)t32.size();
      if (cudaMalloc(&p->table32, t32.size() * sizeof(int32_t)) != cudaSuccess) return fail(B2C_E_CUDA);
      if (cudaMemcpy(p->table32, t32.data(), t32.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(B2C_E_CUDA);
    }
    if (emb.variant == B2C_VARIANT_IM2COL_STAGED) {
      if (!staged_window(g, &p->win)) return fail(B2C_E_UNSUPPORTED);
      // reduction index (c, r, s) -> byte offset from the window position of the pixel's first tap
      std::vector<int32_t> t32;
      if (staged_word_mode(g)) {
        // one entry per 32-bit word of an A row: window offset of the word's first byte
        const int run = staged_run_len(g);
        t32.assign(K_pad / 4, -1);
        for (int wi = 0; wi < K_pad / 4; ++wi) {
          const int cr = (wi * 4) / run, k4 = (wi * 4) % run;
          if (cr < d.C * d.R) t32[wi] = ((cr / d.R) * p->win.rows + (cr % d.R) * d.dil_h) * p->win.pitch + k4;
        }
      } else {
        t32.assign(K_pad, -1);
        int kg = 0;
        for (int c = 0; c < d.C; ++c)
          for (int r = 0; r < d.R; ++r)
            for (int s = 0; s < d.S; ++s, ++kg)
              t32[kg] = (c * p->win.rows + r * d.dil_h) * p->win.pitch + s * d.dil_w;
      }
      p->table_len = (int)t32.size();
      if (cudaMalloc(&p->table32, t32.size() * sizeof(int32_t)) != cudaSuccess) return fail(B2C_E_CUDA);
      if (cudaMemcpy(p->table32, t32.data(), t32.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(B2C_E_CUDA);
    }
  }
  // Room for one extra box row block so that a TMA box never starts past the allocation.
  if (cudaMalloc(&p->w_packed, p->w_packed_bytes + 256) != cudaSuccess) return fail(B2C_E_CUDA);
  fill_common_args(p);
  p->ws_total = workspace_bytes_for(g, emb.variant, emb.tile_n, emb.split_k, is_swapped(emb));
  if (p->fused_pack) {
    p->ws_ctl_offset = (p->ws_total + 255) / 256 * 256;
    p->ws_total = p->ws_ctl_offset + ((size_t)(d.N + 1) * sizeof(int) + 255) / 256 * 256;
  }
  if (is_tma_view_variant(emb.variant)) {
    bool direct = shift_base_variant(emb.variant) == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NHWC && p->C_pad == d.C;
    p->ws_layout_bytes = direct ? 0 : ((size_t)p->view.bytes() + 255) / 256 * 256;
  } else if (emb.variant == B2C_VARIANT_IM2COL_EXPLICIT) {
    p->ws_layout_bytes = ((size_t)g.Mg * p->K_pad + 255) / 256 * 256;
  }
  // Tensor map of the packed weights (plan-owned memory, so it is encoded once).
  // (Swapped map: the weights are the 128-row operand, so their box is 128 rows high.)
  int rc;
  const int w_box_rows = is_swapped(emb) ? kTileM : (emb.tile_m == 2 * kTileM ? emb.tile_n / 2 : emb.tile_n);
  if (is_tma_view_variant(emb.variant)) {
    uint64_t cols = (uint64_t)p->view.R * p->view.S * p->view.C;
    rc = encode_tiled_2d(&p->tmap_b, p->w_packed, cols, d.K, cols, p->bk, w_box_rows, p->bk);
  } else {
    rc = encode_tiled_2d(&p->tmap_b, p->w_packed, p->K_pad, (uint64_t)d.K * group_count, p->K_pad, 128, w_box_rows, 128);
  }
  if (rc != B2C_OK) return fail(rc);
  *out = p;
  return B2C_OK;
}

// Device time of one run of `p`: the launches of `iters` runs are captured into a CUDA graph on a
// private stream and the graph is replayed, so that host launch cost does not mask the kernels.
// With lanes > 1 every iteration enqueues one run per lane, each lane on a stream of its own
// (forked from and joined back into the first) with its own outputs and scratch, so that kernels
// of different lanes may overlap on the GPU; *us is then the time per run at that concurrency.
constexpr int kMaxLanes = 16;
struct LaneBuffers {
  int32_t* y32;
  int8_t* y8;
  void* ws;
};
int time_plan(b2c_plan* p, const int8_t* x, const LaneBuffers* lane, int lanes, float* us) {
  const int iters = 10, replays = 5;
  cudaStream_t st[kMaxLanes] = {};
  cudaEvent_t e0 = nullptr, e1 = nullptr, fork = nullptr, join[kMaxLanes] = {};
  cudaGraph_t graph = nullptr;
  cudaGraphExec_t exec = nullptr;
  int rc = B2C_OK;
  cudaError_t e = cudaSuccess;
  for (int l = 0; l < lanes && e == cudaSuccess; ++l) e = cudaStreamCreateWithFlags(&st[l], cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&fork, cudaEventDisableTiming);
  for (int l = 1; l < lanes && e == cudaSuccess; ++l) e = cudaEventCreateWithFlags(&join[l], cudaEventDisableTiming);
  if (e == cudaSuccess) {
    // plain runs first: first-launch set-up (function attributes) must not happen under capture
    for (int i = 0; i < 2 && rc == B2C_OK; ++i)
      rc = b2c_conv2d_int8_run(p, x, lane[0].y32, lane[0].y8, lane[0].ws, st[0]);
    if (rc == B2C_OK) e = cudaStreamSynchronize(st[0]);
  }
  if (e == cudaSuccess && rc == B2C_OK) {
    e = cudaStreamBeginCapture(st[0], cudaStreamCaptureModeThreadLocal);
    if (e == cudaSuccess) {
      if (lanes > 1) {
        e = cudaEventRecord(fork, st[0]);
        for (int l = 1; l < lanes && e == cudaSuccess; ++l) e = cudaStreamWaitEvent(st[l], fork, 0);
      }
      for (int i = 0; i < iters && rc == B2C_OK && e == cudaSuccess; ++i)
        for (int l = 0; l < lanes && rc == B2C_OK; ++l)
          rc = b2c_conv2d_int8_run(p, x, lane[l].y32, lane[l].y8, lane[l].ws, st[l]);
      for (int l = 1; l < lanes && e == cudaSuccess; ++l) {
        e = cudaEventRecord(join[l], st[l]);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st[0], join[l], 0);
      }
      cudaError_t e2 = cudaStreamEndCapture(st[0], &graph);
      if (e == cudaSuccess && e2 != cudaSuccess) e = e2;
    }
  }
  if (e == cudaSuccess && rc == B2C_OK) e = cudaGraphInstantiate(&exec, graph, 0);
  if (e == cudaSuccess && rc == B2C_OK) {
    e = cudaGraphLaunch(exec, st[0]);  // warm
    // the fastest of the replays: candidates a few per cent apart are otherwise ordered by noise
    float best_ms = -1.0f;
    for (int i = 0; i < replays && e == cudaSuccess; ++i) {
      e = cudaEventRecord(e0, st[0]);
      if (e == cudaSuccess) e = cudaGraphLaunch(exec, st[0]);
      if (e == cudaSuccess) e = cudaEventRecord(e1, st[0]);
      if (e == cudaSuccess) e = cudaEventSynchronize(e1);
      float ms = 0;
      if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
      if (e == cudaSuccess && (best_ms < 0 || ms < best_ms)) best_ms = ms;
    }
    if (e == cudaSuccess) *us = best_ms * 1000.0f / (iters * lanes);
  }
  if (exec) cudaGraphExecDestroy(exec);
  if (graph) cudaGraphDestroy(graph);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (fork) cudaEventDestroy(fork);
  for (int l = 0; l < kMaxLanes; ++l) {
    if (join[l]) cudaEventDestroy(join[l]);
    if (st[l]) cudaStreamDestroy(st[l]);
  }
  if (e != cudaSuccess) {
    set_last_cuda_error((int)e);
    return B2C_E_CUDA;
  }
  if (rc == B2C_OK) {
    int32_t s = 0;
    rc = b2c_plan_device_status(p, &s);
    if (rc == B2C_OK && s != B2C_OK) rc = s;
  }
  return rc;
}

// Key of the one-shot cache: shape, output mode, device and the stream the call enqueues on.  Calls on
// one stream are ordered by the stream; calls on different streams get plans (packed weights,
// scratch, status word) of their own, so they may overlap on the GPU.
struct ShapeKey {
  int v[12];
  uintptr_t stream;
  bool operator<(const ShapeKey& o) const {
    const int c = std::memcmp(v, o.v, sizeof(v));
    return c != 0 ? c < 0 : stream < o.stream;
  }
};
std::mutex g_cache_mu;
std::map<ShapeKey, b2c_plan*> g_cache;

}  // namespace

extern "C" {

const char* b2c_status_string(int s) {
  switch (s) {
    case B2C_OK: return "ok";
    case B2C_E_INVALID_ARG: return "invalid argument";
    case B2C_E_UNSUPPORTED: return "unsupported problem";
    case B2C_E_WORKSPACE_TOO_SMALL: return "workspace too small";
    case B2C_E_CUDA: return "CUDA call failed";
    case B2C_E_TIMEOUT: return "bounded device wait expired";
    case B2C_E_NOT_READY: return "plan has no weights";
    case B2C_E_BOUNDS: return "address outside its tensor (debug build)";
    default: return "unknown status";
  }
}

int b2c_out_shape(const b2c_conv_desc* desc, int32_t* P, int32_t* Q) {
  if (!desc || !P || !Q) return B2C_E_INVALID_ARG;
  Geom g;
  int rc = resolve_geom(desc, &g);
  if (rc == B2C_E_INVALID_ARG) return rc;
  *P = g.P;
  *Q = g.Q;
  return B2C_OK;
}

int b2c_enumerate(const b2c_conv_desc* desc, b2c_embedding* out, int32_t cap, int32_t* count) {
  if (!desc || !count || cap < 0 || (cap > 0 && !out)) return B2C_E_INVALID_ARG;
  Geom g;
  int rc = resolve_geom(desc, &g);
  if (rc != B2C_OK) return rc;
  std::vector<b2c_embedding> all;
  enumerate_embeddings(g, &all);
  if (!table_variant_legal(g))
    all.erase(std::remove_if(all.begin(), all.end(), [](const b2c_embedding& e) { return e.variant != B2C_VARIANT_CP_TMA; }),
              all.end());  // every other variant goes through the stencil lookup table
  for (size_t i = 0; i < all.size(); ++i) all[i].id = (int)i;
  *count = (int32_t)all.size();
  for (int i = 0; i < cap && i < (int)all.size(); ++i) out[i] = all[i];
  return all.empty() ? B2C_E_UNSUPPORTED : B2C_OK;
}

int b2c_plan_create(const b2c_conv_desc* desc, int32_t policy_or_id, void* cuda_stream, b2c_plan** out) {
  if (!desc || !out) return B2C_E_INVALID_ARG;
  *out = nullptr;
  Geom g;
  int rc = resolve_geom(desc, &g);
  if (rc != B2C_OK) return rc;
  int32_t count = 0;
  rc = b2c_enumerate(desc, nullptr, 0, &count);
  if (rc != B2C_OK) return rc;
  std::vector<b2c_embedding> all(count);
  rc = b2c_enumerate(desc, all.data(), count, &count);
  if (rc != B2C_OK) return rc;
  if (policy_or_id < B2C_POLICY_AUTO_TIMED_CONCURRENT) return B2C_E_INVALID_ARG;
  const int lanes = policy_or_id == B2C_POLICY_AUTO_TIMED_CONCURRENT ? kMaxLanes : 1;
  if (policy_or_id != B2C_POLICY_AUTO_TIMED && policy_or_id != B2C_POLICY_AUTO_TIMED_CONCURRENT) {
    int idx = pick_by_policy(all, policy_or_id);
    if (idx < 0) return B2C_E_INVALID_ARG;
    return create_plan_for(g, all[idx], out);
  }
  // Timed selection (Section 6.1: the best candidates by the overhead metric are tuned and the
  // fastest is kept).  All schedules of the five lowest-overhead (axis map, layout variant)
  // groups are run on scratch tensors.
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // (Variants of one family count as one candidate: a view and its shift execution, the row unrolls.)
  std::vector<int> groups;
  for (const b2c_embedding& e : all)
    if (std::find(groups.begin(), groups.end(), variant_family(e.variant)) == groups.end() && groups.size() < 5)
      groups.push_back(variant_family(e.variant));
  size_t ws_max = 0;
  for (const b2c_embedding& e : all) ws_max = std::max(ws_max, (size_t)e.workspace_bytes);
  int8_t *x = nullptr, *w = nullptr;
  LaneBuffers lane[kMaxLanes] = {};
  auto cleanup = [&]() {
    cudaFree(x);
    cudaFree(w);
    for (int l = 0; l < kMaxLanes; ++l) {
      cudaFree(lane[l].y8);
      cudaFree(lane[l].y32);
      cudaFree(lane[l].ws);
    }
  };
  bool alloc_ok = cudaMalloc(&x, g.x_elems + 256) == cudaSuccess && cudaMalloc(&w, g.w_elems + 256) == cudaSuccess;
  for (int l = 0; l < lanes && alloc_ok; ++l)
    alloc_ok = cudaMalloc(&lane[l].y8, g.y_elems + 256) == cudaSuccess &&
               cudaMalloc(&lane[l].y32, g.y_elems * 4 + 256) == cudaSuccess &&
               cudaMalloc(&lane[l].ws, ws_max + 1024) == cudaSuccess;
  if (!alloc_ok) {
    set_last_cuda_error((int)cudaGetLastError());
    cleanup();
    return B2C_E_CUDA;
  }
  cudaMemsetAsync(x, 1, g.x_elems, st);
  cudaMemsetAsync(w, 1, g.w_elems, st);
  cudaStreamSynchronize(st);
  int best = -1;
  float best_us = 0;
  int first_error = B2C_OK;
  for (size_t i = 0; i < all.size(); ++i) {
    if (std::find(groups.begin(), groups.end(), variant_family(all[i].variant)) == groups.end()) continue;
    // A candidate that cannot be built or run (a tensor map the driver refuses, an allocation that
    // fails, a device wait that expires) is left out of the selection; the others are still timed.
    b2c_plan* p = nullptr;
    rc = create_plan_for(g, all[i], &p);
    if (rc == B2C_OK) rc = b2c_plan_set_weights(p, w, st);
    if (rc == B2C_OK && cudaStreamSynchronize(st) != cudaSuccess) rc = B2C_E_CUDA;
    float us = -1;
    if (rc == B2C_OK) rc = time_plan(p, x, lane, lanes, &us);
    b2c_plan_destroy(p);
    if (rc != B2C_OK) {
      if (first_error == B2C_OK) first_error = rc;
      if (cudaGetLastError() != cudaSuccess && cudaDeviceSynchronize() != cudaSuccess) break;  // the context is lost
      continue;
    }
    all[i].device_us = us;
    if (best < 0 || us < best_us) {
      best = (int)i;
      best_us = us;
    }
  }
  cleanup();
  if (best < 0) return first_error != B2C_OK ? first_error : B2C_E_UNSUPPORTED;
  return create_plan_for(g, all[best], out);
}

int b2c_plan_create_grouped(const b2c_conv_desc* desc, int32_t groups, b2c_plan** out) {
  if (!desc || !out || groups < 1) return B2C_E_INVALID_ARG;
  *out = nullptr;
  if (desc->C < 1 || desc->K < 1 || desc->C % groups != 0 || desc->K % groups != 0) return B2C_E_INVALID_ARG;
  // whole tensors are NCHW / NKPQ: a group is then a contiguous channel slice of every image
  if (desc->in_layout != B2C_LAYOUT_NCHW || desc->out_layout != B2C_LAYOUT_NCHW) return B2C_E_UNSUPPORTED;
  // Narrow groups are merged: a depth-wise layer run group by group gives every MMA one useful column and
  // nine useful reduction elements.  m consecutive groups as one group with block-diagonal filters spend m
  // times the MACs (which are idle anyway) for 1/m of the tiles: the smallest divisor m of `groups` that
  // brings a merged group to 32 output channels, within 1024 reduction elements.
  const int cg = desc->C / groups, kg = desc->K / groups;
  int merge = 1;
  for (int m = 1; m <= groups; ++m) {
    if (groups % m != 0) continue;
    if ((long long)m * cg * desc->R * desc->S > 1024 && m > 1) break;
    merge = m;
    if (m * kg >= 32) break;
  }
  b2c_conv_desc sd = *desc;
  sd.C = cg * merge;
  sd.K = kg * merge;
  Geom sg;
  int rc = resolve_geom(&sd, &sg);
  if (rc != B2C_OK) return rc;
  const int run_groups = groups / merge;
  // Embedding of every group: the lowest-overhead unsplit stencil unroll formed inside the kernel
  // (staged window where it fits, else the gather); both read their channel slice of x in place.
  std::vector<b2c_embedding> all;
  enumerate_embeddings(sg, &all);
  // (the staged window before the gather: it builds the operand from shared memory with word loads; of
  // one variant's schedules the one whose column tile holds a whole group, else the widest)
  int pick = -1;
  auto better = [&](const b2c_embedding& a, const b2c_embedding& b) {
    const bool as = a.variant == B2C_VARIANT_IM2COL_STAGED, bs = b.variant == B2C_VARIANT_IM2COL_STAGED;
    if (as != bs) return as;
    const bool af = a.tile_n >= sd.K, bf = b.tile_n >= sd.K;
    if (af != bf) return af;
    return af ? a.tile_n < b.tile_n : a.tile_n > b.tile_n;
  };
  for (size_t i = 0; i < all.size(); ++i)
    if (all[i].split_k == 1 && !is_swapped(all[i]) && all[i].tile_m == kTileM && table_variant_legal(sg) &&
        (all[i].variant == B2C_VARIANT_IM2COL_STAGED || all[i].variant == B2C_VARIANT_IM2COL_GATHER) &&
        (pick < 0 || better(all[i], all[pick])))
      pick = (int)i;
  if (pick < 0) return B2C_E_UNSUPPORTED;
  b2c_plan* p = new (std::nothrow) b2c_plan();
  if (!p) return B2C_E_INVALID_ARG;
  p->g = sg;
  p->g.d.C = desc->C;  // the group plan describes the whole convolution
  p->g.d.K = desc->K;
  p->emb = all[pick];
  p->groups = groups;
  p->merge = merge;
  cudaGetDevice(&p->device);
  if (cudaMalloc(&p->status, kStatusWords * sizeof(int)) != cudaSuccess ||
      cudaMemset(p->status, 0, kStatusWords * sizeof(int)) != cudaSuccess) {
    set_last_cuda_error((int)cudaGetLastError());
    b2c_plan_destroy(p);
    return B2C_E_CUDA;
  }
  // one sub-plan runs all groups in one launch (the group is a grid axis of the kernel)
  b2c_plan* sub = nullptr;
  rc = create_plan_for(sg, all[pick], &sub, run_groups);
  if (rc != B2C_OK) {
    b2c_plan_destroy(p);
    return rc;
  }
  if (merge > 1 &&
      cudaMalloc(&p->w_expanded, (size_t)desc->K * sd.C * desc->R * desc->S + 256) != cudaSuccess) {
    set_last_cuda_error((int)cudaGetLastError());
    b2c_plan_destroy(sub);
    b2c_plan_destroy(p);
    return B2C_E_CUDA;
  }
  sub->x_stride_n_whole = (long long)desc->C * desc->H * desc->W;
  sub->y_stride_n_whole = (long long)desc->K * sg.PQ;
  p->subs.push_back(sub);
  *out = p;
  return B2C_OK;
}

int b2c_plan_create_grouped_timed(const b2c_conv_desc* desc, int32_t groups, void* cuda_stream, b2c_plan** out) {
  if (!desc || !out) return B2C_E_INVALID_ARG;
  *out = nullptr;
  b2c_plan* inplace = nullptr;
  int rc = b2c_plan_create_grouped(desc, groups, &inplace);
  if (rc != B2C_OK) return rc;
  // The other form: every group merged, i.e. the dense convolution with block-diagonal filters through the
  // timed selection of dense plans.  It pays `groups` times the MACs and has the rewrite and the scratch
  // of its embedding; on this device it still wins for a few hundred groups.
  const long long dense_w = (long long)desc->K * desc->C * desc->R * desc->S;
  if (groups < 2 || dense_w > (16ll << 20)) {
    *out = inplace;
    return B2C_OK;
  }
  cudaStream_t st = (cudaStream_t)cuda_stream;
  b2c_plan* dense = nullptr;
  if (b2c_plan_create(desc, B2C_POLICY_AUTO_TIMED, cuda_stream, &dense) != B2C_OK || dense->emb.device_us <= 0) {
    b2c_plan_destroy(dense);
    *out = inplace;
    return B2C_OK;
  }
  // time the in-place form on scratch tensors, as the dense candidates were
  const Geom& g = dense->g;
  int8_t *x = nullptr, *w = nullptr;
  LaneBuffers lane = {};
  float us = -1;
  bool ok = cudaMalloc(&x, g.x_elems + 256) == cudaSuccess && cudaMalloc(&w, g.w_elems + 256) == cudaSuccess &&
            cudaMalloc(&lane.y8, g.y_elems + 256) == cudaSuccess && cudaMalloc(&lane.y32, g.y_elems * 4 + 256) == cudaSuccess &&
            cudaMalloc(&lane.ws, 1024) == cudaSuccess;
  if (ok) {
    cudaMemsetAsync(x, 1, g.x_elems, st);
    cudaMemsetAsync(w, 1, g.w_elems, st);  // (the grouped filter tensor is smaller than the dense one)
    ok = b2c_plan_set_weights(inplace, w, st) == B2C_OK && cudaStreamSynchronize(st) == cudaSuccess &&
         time_plan(inplace, x, &lane, 1, &us) == B2C_OK;
    inplace->weights_set = false;  // the caller's filters are still to come
  }
  cudaFree(x);
  cudaFree(w);
  cudaFree(lane.y8);
  cudaFree(lane.y32);
  cudaFree(lane.ws);
  if (!ok) (void)cudaGetLastError();
  if (!ok || us <= dense->emb.device_us) {  // (an in-place form that could not be timed is still the safe choice)
    b2c_plan_destroy(dense);
    inplace->emb.device_us = us;
    *out = inplace;
    return B2C_OK;
  }
  // wrap the dense plan: filters expanded at set_weights, everything else is the dense plan's own path
  b2c_plan* p = new (std::nothrow) b2c_plan();
  bool made = p != nullptr;
  if (made) {
    p->g = dense->g;
    p->emb = dense->emb;
    p->groups = groups;
    p->merge = groups;
    p->dense_sub = true;
    p->ws_total = dense->ws_total;
    p->ws_layout_bytes = dense->ws_layout_bytes;
    cudaGetDevice(&p->device);
    made = cudaMalloc(&p->status, kStatusWords * sizeof(int)) == cudaSuccess &&
           cudaMemset(p->status, 0, kStatusWords * sizeof(int)) == cudaSuccess &&
           cudaMalloc(&p->w_expanded, (size_t)dense_w + 256) == cudaSuccess;
  }
  if (!made) {
    set_last_cuda_error((int)cudaGetLastError());
    b2c_plan_destroy(p);
    b2c_plan_destroy(dense);
    *out = inplace;
    return B2C_OK;
  }
  p->subs.push_back(dense);
  b2c_plan_destroy(inplace);
  *out = p;
  return B2C_OK;
}

int b2c_plan_info(const b2c_plan* plan, b2c_embedding* chosen) {
  if (!plan || !chosen) return B2C_E_INVALID_ARG;
  *chosen = plan->emb;
  return B2C_OK;
}

int b2c_plan_workspace_bytes(const b2c_plan* plan, size_t* bytes) {
  if (!plan || !bytes) return B2C_E_INVALID_ARG;
  *bytes = plan->ws_total ? plan->ws_total + 2 * kCanaryBytes : 0;  // debug build: + the guard bands
  return B2C_OK;
}

static int set_weights_one(b2c_plan* p, const int8_t* w, cudaStream_t st);

int b2c_plan_set_weights(b2c_plan* p, const int8_t* w, void* cuda_stream) {
  if (!p || !w) return B2C_E_INVALID_ARG;
  if (!aligned16(w)) return B2C_E_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (!p->subs.empty()) {
    // w is [K][C/groups][R][S]: group g's filters are the g-th block of K/groups rows
    // (one pack launch: the rows of all groups have the same format)
    const int8_t* src = w;
    if (p->merge > 1) {
      const b2c_conv_desc& d = p->g.d;  // (the whole convolution)
      CUDA_TRY(launch_expand_group_weights(w, p->w_expanded, d.K, d.C / p->groups, d.K / p->groups, p->merge, d.R * d.S, st));
      src = p->w_expanded;
    }
    int rc = set_weights_one(p->subs[0], src, st);
    if (rc != B2C_OK) return rc;
    p->weights_set = true;
    return B2C_OK;
  }
  return set_weights_one(p, w, st);
}

static int set_weights_one(b2c_plan* p, const int8_t* w, cudaStream_t st) {
  const b2c_conv_desc& d = p->g.d;
  if (p->emb.variant == B2C_VARIANT_CP_TMA || p->emb.variant == B2C_VARIANT_DILATION_PACK ||
      p->emb.variant == B2C_VARIANT_CP_SHIFT)
    CUDA_TRY(launch_pack_weights_cp(w, p->w_packed, d.K, d.C, d.R, d.S, p->C_pad, st));
  else if (is_tma_view_variant(p->emb.variant))
    CUDA_TRY(launch_pack_weights_table(w, p->w_packed, d.K, p->g.Kg, p->view.R * p->view.S * p->view.C, p->wtable, st));
  else
    CUDA_TRY(launch_pack_weights_rows(w, p->w_packed, d.K * p->group_count, p->g.Kg, p->K_pad, d.S,
                                      p->emb.variant == B2C_VARIANT_IM2COL_STAGED
                                          ? staged_run_len(p->g)
                                          : (p->emb.variant == B2C_VARIANT_IM2COL_WINDOW ? round_up(d.S, 4) : d.S),
                                      st));
  p->weights_set = true;
  return B2C_OK;
}

// The two halves of the path.  run_rewrite is the layout rewrite of the activations (the paper's
// "Transf." column): it fills the start of the workspace.  run_convolve is the MMA kernel with its
// epilogue and the split-reduction finish (the "Op." column): it reads the rewritten operand from
// the workspace (or x itself when the embedding has no rewrite).
static int run_rewrite(b2c_plan* p, const int8_t* x, void* ws, cudaStream_t st) {
  const b2c_conv_desc& d = p->g.d;
  const Geom& g = p->g;
  const ConvArgs& a = p->args;
  if (!p->ws_layout_bytes) return B2C_OK;
  int8_t* scratch = static_cast<int8_t*>(ws);
  Dbg dbg;
  const long long shrink = g_dbg_shrink.load();
  dbg.x_lo = x;
  dbg.x_bytes = (long long)(d.N - 1) * a.x_stride_n + (long long)d.C * d.H * d.W - shrink;
  dbg.ws_lo = ws;
  dbg.ws_bytes = (long long)p->ws_layout_bytes - shrink;
  dbg.status = p->status;
  if (is_tma_view_variant(p->emb.variant)) {
    const TmaView& v = p->view;
    const int base_variant = shift_base_variant(p->emb.variant);
    if (base_variant == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NHWC) {
      // NHWC re-pad (Pad rule alone): the layout-generic copy kernel with one phase per axis
      CUDA_TRY(launch_phase_split(x, scratch, d.N, d.C, d.H, d.W, 1, 1, d.H, d.W, v.C, a.x_stride_n, 1, a.x_stride_h,
                                  a.x_stride_w, st, dbg));
    } else if (base_variant == B2C_VARIANT_CP_TMA) {
      CUDA_TRY(launch_pack_activations(x, scratch, d.N, d.C, d.H, d.W, p->C_pad, st, p->status, dbg));
    } else if (base_variant == B2C_VARIANT_DILATION_PACK) {
      const bool nchw = d.in_layout == B2C_LAYOUT_NCHW;
      CUDA_TRY(launch_phase_split(x, scratch, d.N, d.C, d.H, d.W, d.dil_h, d.dil_w, v.H, v.W, v.C, a.x_stride_n,
                                  nchw ? (long long)d.H * d.W : 1, a.x_stride_h, a.x_stride_w, st, dbg));
    } else if (base_variant == B2C_VARIANT_ROWPHASE_SHIFT) {
      const bool nchw = d.in_layout == B2C_LAYOUT_NCHW;
      CUDA_TRY(launch_row_phase_unroll(x, scratch, v.N, v.H, v.W, d.C, d.H, d.W, d.S, d.stride_h, d.stride_w, d.pad_h,
                                       d.pad_w, d.dil_w, v.C, a.x_stride_n, nchw ? (long long)d.H * d.W : 1,
                                       a.x_stride_h, a.x_stride_w, st, dbg));
    } else if (base_variant == B2C_VARIANT_ROW_UNROLL) {
      // scratch pixel (n, h, q): window origin (h, q*stride_w - pad_w), channels (s, c)
      CUDA_TRY(launch_im2col(x, scratch, p->table, (long long)v.N * v.H * v.W, v.H * v.W, v.W, d.H, d.W, 1,
                             d.stride_w, 0, d.pad_w, a.x_stride_n, a.x_stride_h, a.x_stride_w, v.C, st, dbg));
    } else {
      // space to depth: scratch pixel (n, h', w') holds the stride phases (c, dh, dw) of its window
      const bool nchw = d.in_layout == B2C_LAYOUT_NCHW;
      CUDA_TRY(launch_space_to_depth(x, scratch, v.N, v.H, v.W, d.C, d.H, d.W, d.stride_h, d.stride_w, d.pad_h, d.pad_w,
                                     v.C, s2d_pack_factor(g), a.x_stride_n, nchw ? (long long)d.H * d.W : 1,
                                     a.x_stride_h, a.x_stride_w, st, dbg));
    }
  } else if (p->emb.variant == B2C_VARIANT_IM2COL_EXPLICIT) {
    CUDA_TRY(launch_im2col(x, scratch, p->table, g.Mg, g.PQ, g.Q, d.H, d.W, d.stride_h, d.stride_w, d.pad_h, d.pad_w,
                           a.x_stride_n, a.x_stride_h, a.x_stride_w, p->K_pad, st, dbg));
  }
  return B2C_OK;
}

static int run_convolve(b2c_plan* p, const int8_t* x, int32_t* y32, int8_t* y8, void* ws, cudaStream_t st,
                        bool fused_pack = false) {
  const b2c_conv_desc& d = p->g.d;
  const Geom& g = p->g;
  ConvArgs a = p->args;
  a.x = x;
  a.y32 = y32;
  a.y8 = y8;
  a.bias = p->bias;
  a.relu = p->relu;
  if (p->x_stride_n_whole) a.x_stride_n = p->x_stride_n_whole;
  if (p->y_stride_n_whole) a.y_stride_n = p->y_stride_n_whole;
  const bool act = p->bias != nullptr || p->relu != 0;
  {
    const long long shrink = g_dbg_shrink.load();
    const long long y_span = (long long)(d.N - 1) * a.y_stride_n + (long long)d.K * g.PQ * a.groups;
    a.dbg.x_lo = x;
    a.dbg.x_bytes = x ? (long long)(d.N - 1) * a.x_stride_n + (long long)d.C * d.H * d.W * a.groups - shrink : 0;
    a.dbg.o32_lo = y32;
    a.dbg.o32_bytes = (y_span - shrink) * 4;
    a.dbg.o8_lo = y8;
    a.dbg.o8_bytes = y_span - shrink;
    a.dbg.ws_lo = ws;
    a.dbg.ws_bytes = (long long)p->ws_total - shrink;
    a.dbg.status = p->status;
  }
  CUtensorMap tmap_a;
  std::memset(&tmap_a, 0, sizeof(tmap_a));
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  int rc = B2C_OK;
  if (is_tma_view_variant(p->emb.variant)) {
    const TmaView& v = p->view;
    const int8_t* act = p->ws_layout_bytes ? reinterpret_cast<const int8_t*>(wsb) : x;
    if (p->amode == A_SHIFT)
      rc = encode_tiled_nhwc_rows(&tmap_a, act, v.C, v.W, v.H, v.N, p->bk, a.sh_wps, p->bk, a.remap == 3 ? a.sh_rows : 1);
    else
      rc = encode_im2col_nhwc(&tmap_a, act, v.C, v.W, v.H, v.N, v.pad_w, v.pad_h, v.S, v.R, v.dil_w, v.dil_h,
                            v.stride_w, v.stride_h, p->bk, a.swap ? a.tile_n : kTileM, p->bk);
    if (rc != B2C_OK) return rc;
  } else if (p->emb.variant == B2C_VARIANT_IM2COL_EXPLICIT) {
    rc = encode_tiled_2d(&tmap_a, wsb, p->K_pad, (uint64_t)g.Mg, p->K_pad, 128, a.swap ? a.tile_n : kTileM, 128);
    if (rc != B2C_OK) return rc;
  } else if (p->amode == A_WINDOW) {
    if (a.wn_linear) {
      tmap_a = p->tmap_b;  // the images arrive by plain bulk copies; any valid map
    } else {
      rc = encode_tiled_nchw_window(&tmap_a, x, d.W, d.H, d.C, d.N, a.wn_win_w, a.wn_box_bytes / (d.C * a.wn_win_w));
      if (rc != B2C_OK) return rc;
    }
  } else {
    tmap_a = p->tmap_b;  // unused by the gather kernel; any valid map
  }

  // ---- split reduction: partial sums meet in a zeroed int32 buffer ----
  bool need_finish = false;
  if (a.split_k > 1 && !a.cluster_split) {
    if (d.out_mode == B2C_OUT_I32) {
      a.acc = y32;           // the partial sums meet in the output itself ...
      need_finish = act;     // ... and the activation step, if any, is applied to it in place afterwards
    } else {
      a.acc = reinterpret_cast<int32_t*>(wsb + p->ws_layout_bytes);
      need_finish = true;
    }
    CUDA_TRY(cudaMemsetAsync(a.acc, 0, (size_t)g.y_elems * 4, st));
  }

  if (a.pair) {
    a.pk_on = fused_pack ? 1 : 0;
    if (fused_pack) {
      // the kernel's pack warps rewrite x into the start of the workspace; its counters start at zero
      a.pk_src = x;
      a.pk_dst = reinterpret_cast<int8_t*>(wsb);
      a.pk_ctl = reinterpret_cast<int*>(wsb + p->ws_ctl_offset);
      CUDA_TRY(cudaMemsetAsync(a.pk_ctl, 0, (size_t)(d.N + 1) * sizeof(int), st));
    }
    CUDA_TRY(launch_conv_mma_pair(p->amode, &tmap_a, &p->tmap_b, a, st));
  } else if (p->amode == A_WINDOW) {
    CUDA_TRY(launch_conv_mma_window(&tmap_a, &p->tmap_b, a, st));
  } else
    CUDA_TRY(launch_conv_mma(p->amode, &tmap_a, &p->tmap_b, a, st));
  if (need_finish)
    CUDA_TRY(launch_splitk_finish(a.acc, y32, y8, g.y_elems, d.shift, d.out_mode, p->bias, p->relu, d.K, g.PQ,
                                  d.out_layout == B2C_LAYOUT_NHWC ? 1 : 0, st, a.dbg));
  return B2C_OK;
}

static int check_run_args(b2c_plan* p, const int8_t* x, bool need_x, int32_t* y32, int8_t* y8, bool need_y, void* ws) {
  if (!p || (need_x && !x)) return B2C_E_INVALID_ARG;
  const b2c_conv_desc& d = p->g.d;
  if (need_y && !p->weights_set) return B2C_E_NOT_READY;
  if (need_y && (d.out_mode & B2C_OUT_I32) && !y32) return B2C_E_INVALID_ARG;
  if (need_y && (d.out_mode & B2C_OUT_I8) && !y8) return B2C_E_INVALID_ARG;
  if (p->ws_total > 0 && !ws) return B2C_E_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y32) || !aligned16(y8) || !aligned16(ws)) return B2C_E_INVALID_ARG;
  return B2C_OK;
}

// Debug build: the caller's workspace is [guard band][scratch][guard band]; every run repaints the
// bands and uses the middle.
static void* guard_workspace(b2c_plan* p, void* ws, cudaStream_t st, int* rc) {
  *rc = B2C_OK;
  if (kCanaryBytes == 0 || !ws || !p->ws_total) return ws;
  uint8_t* w = static_cast<uint8_t*>(ws);
  if (cudaMemsetAsync(w, kCanaryByte, kCanaryBytes, st) != cudaSuccess ||
      cudaMemsetAsync(w + kCanaryBytes + p->ws_total, kCanaryByte, kCanaryBytes, st) != cudaSuccess) {
    set_last_cuda_error((int)cudaGetLastError());
    *rc = B2C_E_CUDA;
  }
  return w + kCanaryBytes;
}

int b2c_conv2d_int8_run(b2c_plan* p, const int8_t* x, int32_t* y32, int8_t* y8, void* ws, void* cuda_stream) {
  int rc = check_run_args(p, x, true, y32, y8, true, ws);
  if (rc != B2C_OK) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  ws = guard_workspace(p, ws, st, &rc);
  if (rc != B2C_OK) return rc;
  if (!p->subs.empty() && !p->dense_sub) {
    // one launch: every group convolves its channel slice of x (NCHW) into its slice of y (NKPQ)
    return run_convolve(p->subs[0], x, y32, y8, nullptr, st);
  }
  b2c_plan* r = p->dense_sub ? p->subs[0] : p;  // (all groups merged: the dense plan's own path)
  if (r->fused_pack && aligned16(x)) return run_convolve(r, x, y32, y8, ws, st, /*fused_pack=*/true);
  rc = run_rewrite(r, x, ws, st);
  if (rc != B2C_OK) return rc;
  return run_convolve(r, x, y32, y8, ws, st);
}

int b2c_plan_rewrite_activations(b2c_plan* p, const int8_t* x, void* ws, void* cuda_stream) {
  int rc = check_run_args(p, x, true, nullptr, nullptr, false, ws);
  if (rc != B2C_OK) return rc;
  if (!p->subs.empty()) return B2C_OK;  // the group convolutions read x directly: nothing to rewrite
  ws = guard_workspace(p, ws, (cudaStream_t)cuda_stream, &rc);
  if (rc != B2C_OK) return rc;
  return run_rewrite(p, x, ws, (cudaStream_t)cuda_stream);
}

int b2c_conv2d_int8_run_rewritten(b2c_plan* p, const int8_t* x, int32_t* y32, int8_t* y8, void* ws, void* cuda_stream) {
  // x is still needed by the embeddings that have no rewrite (they read the input directly)
  int rc = check_run_args(p, x, p && p->ws_layout_bytes == 0, y32, y8, true, ws);
  if (rc != B2C_OK) return rc;
  if (!p->subs.empty()) return b2c_conv2d_int8_run(p, x, y32, y8, ws, cuda_stream);
  if (kCanaryBytes && ws && p->ws_total) ws = static_cast<uint8_t*>(ws) + kCanaryBytes;  // bands painted by the rewrite half
  return run_convolve(p, x, y32, y8, ws, (cudaStream_t)cuda_stream);
}

int b2c_plan_set_activation(b2c_plan* p, const int32_t* bias_dev, int relu, void* cuda_stream) {
  if (!p || (relu != 0 && relu != 1)) return B2C_E_INVALID_ARG;
  if (bias_dev && (reinterpret_cast<uintptr_t>(bias_dev) & 3) != 0) return B2C_E_INVALID_ARG;
  const size_t bytes = (size_t)p->g.d.K * sizeof(int32_t);
  if (bias_dev) {
    if (!p->bias_buf) CUDA_TRY(cudaMalloc(&p->bias_buf, bytes));
    CUDA_TRY(cudaMemcpyAsync(p->bias_buf, bias_dev, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream));
    p->bias = p->bias_buf;
  } else {
    p->bias = nullptr;  // the buffer is kept for a later call
  }
  p->relu = relu;
  // group plans: every group takes its own K/groups entries of the copy
  for (b2c_plan* sub : p->subs) {  // (the kernel indexes the bias by group)
    sub->bias = p->bias;
    sub->relu = relu;
  }
  return B2C_OK;
}

int b2c_plan_footprint(const b2c_plan* p, size_t* rewritten_bytes, size_t* packed_weight_bytes) {
  if (!p || !rewritten_bytes || !packed_weight_bytes) return B2C_E_INVALID_ARG;
  *rewritten_bytes = p->ws_layout_bytes;
  *packed_weight_bytes = p->w_packed_bytes;
  for (const b2c_plan* sub : p->subs) *packed_weight_bytes += sub->w_packed_bytes;
  return B2C_OK;
}

int b2c_plan_device_status(b2c_plan* p, int32_t* status) {
  if (!p || !status) return B2C_E_INVALID_ARG;
  int s = 0;
  // (a plain cudaMemcpy only orders against blocking streams; kernels of this plan may run on
  // non-blocking ones, so wait for the whole device first)
  CUDA_TRY(cudaDeviceSynchronize());
  int words[kStatusWords] = {0, 0, 0, 0};
  CUDA_TRY(cudaMemcpy(words, p->status, sizeof(words), cudaMemcpyDeviceToHost));
  s = words[0];
  if (s != 0) {
    p->dbg_site = words[1];
    p->dbg_offset = ((long long)words[3] << 32) | (unsigned int)words[2];
    CUDA_TRY(cudaMemset(p->status, 0, sizeof(words)));
  }
  for (b2c_plan* sub : p->subs) {  // a group plan reports the first sub-plan status that is set
    int32_t ss = 0;
    int rc = b2c_plan_device_status(sub, &ss);
    if (rc != B2C_OK) return rc;
    if (s == 0) s = ss;
  }
  *status = s;
  return B2C_OK;
}

int b2c_debug_build(void) {
#ifdef B2C_DEBUG_BOUNDS
  return 1;
#else
  return 0;
#endif
}

int b2c_plan_debug_info(const b2c_plan* p, int32_t* site, int64_t* byte_offset) {
  if (!p || !site || !byte_offset) return B2C_E_INVALID_ARG;
  *site = p->dbg_site;
  *byte_offset = p->dbg_offset;
  for (const b2c_plan* sub : p->subs)
    if (*site == 0 && sub->dbg_site != 0) {
      *site = sub->dbg_site;
      *byte_offset = sub->dbg_offset;
    }
  return B2C_OK;
}

int b2c_plan_check_canaries(b2c_plan* p, const void* workspace_dev, int32_t* intact) {
  if (!p || !intact) return B2C_E_INVALID_ARG;
  if (kCanaryBytes == 0) return B2C_E_UNSUPPORTED;
  *intact = 1;
  if (!p->ws_total) return B2C_OK;
  if (!workspace_dev) return B2C_E_INVALID_ARG;
  CUDA_TRY(cudaDeviceSynchronize());
  unsigned char band[2][64];
  const unsigned char* w = static_cast<const unsigned char*>(workspace_dev);
  CUDA_TRY(cudaMemcpy(band[0], w, kCanaryBytes, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(band[1], w + kCanaryBytes + p->ws_total, kCanaryBytes, cudaMemcpyDeviceToHost));
  for (int b = 0; b < 2; ++b)
    for (size_t i = 0; i < kCanaryBytes; ++i)
      if (band[b][i] != kCanaryByte) *intact = 0;
  return B2C_OK;
}

int b2c_test_shrink_checked_ranges(long long bytes) {
  if (bytes < 0) return B2C_E_INVALID_ARG;
  g_dbg_shrink.store(bytes);
  return B2C_OK;
}

int b2c_selftest_bounded_wait(b2c_plan* p, void* cuda_stream) {
  if (!p) return B2C_E_INVALID_ARG;
  CUDA_TRY(launch_bounded_wait_selftest(p->status, (cudaStream_t)cuda_stream));
  return B2C_OK;
}

int b2c_selftest_pack_wait(b2c_plan* p, void* cuda_stream) {
  if (!p) return B2C_E_INVALID_ARG;
  CUDA_TRY(launch_pack_wait_selftest(p->status, (cudaStream_t)cuda_stream));
  return B2C_OK;
}

static void destroy_pipe(HostPipe* hp) {
  if (!hp) return;
  if (hp->s_in) cudaStreamSynchronize(hp->s_in);
  if (hp->s_run) cudaStreamSynchronize(hp->s_run);
  if (hp->s_out) cudaStreamSynchronize(hp->s_out);
  for (HostPipe::Slot& sl : hp->slot) {
    cudaFree(sl.x);
    cudaFree(sl.y32);
    cudaFree(sl.y8);
    if (sl.in_done) cudaEventDestroy(sl.in_done);
    if (sl.run_done) cudaEventDestroy(sl.run_done);
    if (sl.out_done) cudaEventDestroy(sl.out_done);
  }
  cudaFree(hp->ws);
  if (hp->s_in) cudaStreamDestroy(hp->s_in);
  if (hp->s_run) cudaStreamDestroy(hp->s_run);
  if (hp->s_out) cudaStreamDestroy(hp->s_out);
  delete hp;
}

void b2c_plan_destroy(b2c_plan* p) {
  if (!p) return;
  destroy_pipe(p->pipe);
  for (b2c_plan* sub : p->subs) b2c_plan_destroy(sub);
  cudaFree(p->w_packed);
  cudaFree(p->w_expanded);
  cudaFree(p->table);
  cudaFree(p->table32);
  cudaFree(p->wtable);
  cudaFree(p->status);
  cudaFree(p->bias_buf);
  cudaFree(p->own_ws);
  delete p;
}

int b2c_conv2d_int8(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int dilation, int shift,
                    const int8_t* x, const int8_t* w, int32_t* y32, int8_t* y8, void* cuda_stream) {
  if (!x || !w || (!y32 && !y8)) return B2C_E_INVALID_ARG;
  b2c_conv_desc d;
  std::memset(&d, 0, sizeof(d));
  d.N = N; d.C = C; d.H = H; d.W = W; d.K = K; d.R = R; d.S = S;
  d.stride_h = d.stride_w = stride;
  d.pad_h = d.pad_w = pad;
  d.dil_h = d.dil_w = dilation;
  d.shift = shift;
  d.in_layout = B2C_LAYOUT_NCHW;
  d.out_layout = B2C_LAYOUT_NCHW;
  d.out_mode = (y32 ? B2C_OUT_I32 : 0) | (y8 ? B2C_OUT_I8 : 0);
  int dev = 0;
  cudaGetDevice(&dev);
  ShapeKey key = {{N, C, H, W, K, R, S, stride, pad, dilation, shift, d.out_mode * 64 + dev},
                  reinterpret_cast<uintptr_t>(cuda_stream)};
  std::lock_guard<std::mutex> lock(g_cache_mu);
  b2c_plan* p = nullptr;
  auto it = g_cache.find(key);
  if (it == g_cache.end()) {
    // first use of a shape: timed selection (allocates and synchronises once, then cached)
    int rc = b2c_plan_create(&d, B2C_POLICY_AUTO_TIMED, cuda_stream, &p);
    if (rc != B2C_OK) return rc;
    if (p->ws_total) {
      if (cudaMalloc(&p->own_ws, p->ws_total + 2 * kCanaryBytes) != cudaSuccess) {
        set_last_cuda_error((int)cudaGetLastError());
        b2c_plan_destroy(p);
        return B2C_E_CUDA;
      }
    }
    g_cache[key] = p;
  } else {
    p = it->second;
  }
  int rc = b2c_plan_set_weights(p, w, cuda_stream);
  if (rc != B2C_OK) return rc;
  return b2c_conv2d_int8_run(p, x, y32, y8, p->own_ws, cuda_stream);
}

int b2c_oneshot_status(int32_t* status) {
  if (!status) return B2C_E_INVALID_ARG;
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(g_cache_mu);
  int32_t first = B2C_OK;
  for (auto& kv : g_cache) {
    if (kv.second->device != dev) continue;
    int32_t s = B2C_OK;
    int rc = b2c_plan_device_status(kv.second, &s);
    if (rc != B2C_OK) return rc;
    if (first == B2C_OK) first = s;
  }
  *status = first;
  return B2C_OK;
}

int b2c_oneshot_cache_clear(void) {
  int dev = 0;
  cudaGetDevice(&dev);
  std::lock_guard<std::mutex> lock(g_cache_mu);
  bool synced = false;
  for (auto it = g_cache.begin(); it != g_cache.end();) {
    if (it->second->device != dev) {
      ++it;
      continue;
    }
    if (!synced) {
      CUDA_TRY(cudaDeviceSynchronize());  // work enqueued by earlier one-shot calls may still use the buffers
      synced = true;
    }
    b2c_plan_destroy(it->second);
    it = g_cache.erase(it);
  }
  return B2C_OK;
}

int b2c_conv2d_int8_host(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int dilation, int shift,
                         const int8_t* xh, const int8_t* wh, int32_t* y32h, int8_t* y8h) {
  if (!xh || !wh || (!y32h && !y8h)) return B2C_E_INVALID_ARG;
  b2c_conv_desc d;
  std::memset(&d, 0, sizeof(d));
  d.N = N; d.C = C; d.H = H; d.W = W; d.K = K; d.R = R; d.S = S;
  d.stride_h = d.stride_w = stride;
  d.pad_h = d.pad_w = pad;
  d.dil_h = d.dil_w = dilation;
  d.shift = shift;
  d.out_mode = (y32h ? B2C_OUT_I32 : 0) | (y8h ? B2C_OUT_I8 : 0);
  Geom g;
  int rc = resolve_geom(&d, &g);
  if (rc != B2C_OK) return rc;
  // Device staging buffers, grown on demand and kept for the next call (per process).
  static std::mutex mu;
  static int8_t *dx = nullptr, *dw = nullptr, *dy8 = nullptr;
  static int32_t* dy32 = nullptr;
  static size_t cx = 0, cw = 0, cy8 = 0, cy32 = 0;
  std::lock_guard<std::mutex> lock(mu);
  auto grow = [](void** p, size_t* cap, size_t need) -> bool {
    if (need <= *cap) return true;
    cudaFree(*p);
    *p = nullptr;
    *cap = 0;
    if (cudaMalloc(p, need + 256) != cudaSuccess) return false;
    *cap = need;
    return true;
  };
  bool ok = grow((void**)&dx, &cx, (size_t)g.x_elems) && grow((void**)&dw, &cw, (size_t)g.w_elems);
  if (ok && y8h) ok = grow((void**)&dy8, &cy8, (size_t)g.y_elems);
  if (ok && y32h) ok = grow((void**)&dy32, &cy32, (size_t)g.y_elems * 4);
  if (!ok) {
    set_last_cuda_error((int)cudaGetLastError());
    return B2C_E_CUDA;
  }
  cudaStream_t st = 0;
  CUDA_TRY(cudaMemcpyAsync(dx, xh, g.x_elems, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(dw, wh, g.w_elems, cudaMemcpyHostToDevice, st));
  rc = b2c_conv2d_int8(N, C, H, W, K, R, S, stride, pad, dilation, shift, dx, dw, y32h ? dy32 : nullptr,
                       y8h ? dy8 : nullptr, st);
  if (rc != B2C_OK) return rc;
  if (y32h) CUDA_TRY(cudaMemcpyAsync(y32h, dy32, g.y_elems * 4, cudaMemcpyDeviceToHost, st));
  if (y8h) CUDA_TRY(cudaMemcpyAsync(y8h, dy8, g.y_elems, cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  return B2C_OK;
}

static int create_pipe(b2c_plan* p) {
  HostPipe* hp = new (std::nothrow) HostPipe;
  if (!hp) return B2C_E_CUDA;
  p->pipe = hp;  // owned by the plan from here on: b2c_plan_destroy frees whatever was created
  const b2c_conv_desc& d = p->g.d;
  hp->x_bytes = (size_t)d.N * d.C * d.H * d.W;
  hp->y_elems = (size_t)d.N * d.K * p->g.PQ;
  CUDA_TRY(cudaStreamCreateWithFlags(&hp->s_in, cudaStreamNonBlocking));
  CUDA_TRY(cudaStreamCreateWithFlags(&hp->s_run, cudaStreamNonBlocking));
  CUDA_TRY(cudaStreamCreateWithFlags(&hp->s_out, cudaStreamNonBlocking));
  if (p->ws_total) CUDA_TRY(cudaMalloc(&hp->ws, p->ws_total + 2 * kCanaryBytes));
  for (HostPipe::Slot& sl : hp->slot) {
    CUDA_TRY(cudaMalloc((void**)&sl.x, hp->x_bytes + 256));
    if (d.out_mode & B2C_OUT_I32) CUDA_TRY(cudaMalloc((void**)&sl.y32, hp->y_elems * 4));
    if (d.out_mode & B2C_OUT_I8) CUDA_TRY(cudaMalloc((void**)&sl.y8, hp->y_elems));
    CUDA_TRY(cudaEventCreateWithFlags(&sl.in_done, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&sl.run_done, cudaEventDisableTiming));
    CUDA_TRY(cudaEventCreateWithFlags(&sl.out_done, cudaEventDisableTiming));
  }
  return B2C_OK;
}

int b2c_plan_run_host_async(b2c_plan* p, const int8_t* xh, int32_t* y32h, int8_t* y8h) {
  if (!p || !xh) return B2C_E_INVALID_ARG;
  const int mode = p->g.d.out_mode;
  if (((mode & B2C_OUT_I32) && !y32h) || ((mode & B2C_OUT_I8) && !y8h)) return B2C_E_INVALID_ARG;
  if (!p->pipe) {
    int rc = create_pipe(p);
    if (rc != B2C_OK) {
      destroy_pipe(p->pipe);
      p->pipe = nullptr;
      return rc;
    }
  }
  HostPipe* hp = p->pipe;
  HostPipe::Slot& sl = hp->slot[hp->next];
  hp->next = (hp->next + 1) % HostPipe::kSlots;
  // the slot's buffers are free once the read-back of the call that used them last has finished
  if (sl.used) CUDA_TRY(cudaEventSynchronize(sl.out_done));
  CUDA_TRY(cudaMemcpyAsync(sl.x, xh, hp->x_bytes, cudaMemcpyHostToDevice, hp->s_in));
  CUDA_TRY(cudaEventRecord(sl.in_done, hp->s_in));
  CUDA_TRY(cudaStreamWaitEvent(hp->s_run, sl.in_done, 0));
  int rc = b2c_conv2d_int8_run(p, sl.x, sl.y32, sl.y8, hp->ws, hp->s_run);
  if (rc != B2C_OK) return rc;
  CUDA_TRY(cudaEventRecord(sl.run_done, hp->s_run));
  CUDA_TRY(cudaStreamWaitEvent(hp->s_out, sl.run_done, 0));
  if (mode & B2C_OUT_I32) CUDA_TRY(cudaMemcpyAsync(y32h, sl.y32, hp->y_elems * 4, cudaMemcpyDeviceToHost, hp->s_out));
  if (mode & B2C_OUT_I8) CUDA_TRY(cudaMemcpyAsync(y8h, sl.y8, hp->y_elems, cudaMemcpyDeviceToHost, hp->s_out));
  CUDA_TRY(cudaEventRecord(sl.out_done, hp->s_out));
  sl.used = true;
  return B2C_OK;
}

int b2c_plan_host_sync(b2c_plan* p) {
  if (!p) return B2C_E_INVALID_ARG;
  if (!p->pipe) return B2C_OK;  // nothing was enqueued
  // every call ends with its read-back on the copy-out stream, which waits for the other two
  CUDA_TRY(cudaStreamSynchronize(p->pipe->s_out));
  return B2C_OK;
}

int b2c_pack_activations(const int8_t* x, int8_t* out, int N, int C, int H, int W, int C_pad, void* cuda_stream) {
  if (!x || !out || N < 1 || C < 1 || H < 1 || W < 1 || C_pad < C || (C_pad % 16) != 0) return B2C_E_INVALID_ARG;
  if (!aligned16(x) || !aligned16(out)) return B2C_E_INVALID_ARG;
  CUDA_TRY(launch_pack_activations(x, out, N, C, H, W, C_pad, (cudaStream_t)cuda_stream, nullptr));
  return B2C_OK;
}

int b2c_im2col(const b2c_conv_desc* desc, const int8_t* x, int8_t* a, int K_pad, void* cuda_stream) {
  if (!desc || !x || !a || !aligned16(x) || !aligned16(a)) return B2C_E_INVALID_ARG;
  b2c_conv_desc d = *desc;
  if ((d.out_mode & 3) == 0) d.out_mode = B2C_OUT_I32;
  Geom g;
  int rc = resolve_geom(&d, &g);
  if (rc != B2C_OK) return rc;
  if (K_pad < g.Kg || (K_pad % 16) != 0) return B2C_E_INVALID_ARG;
  if (!table_variant_legal(g)) return B2C_E_UNSUPPORTED;
  std::vector<GatherEntry> t;
  build_table(g, K_pad, &t);
  GatherEntry* dt = nullptr;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(cudaMalloc(&dt, t.size() * sizeof(GatherEntry)));
  cudaError_t e = cudaMemcpyAsync(dt, t.data(), t.size() * sizeof(GatherEntry), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);  // the host table goes out of scope below
  long long sn = (long long)d.C * d.H * d.W;
  int sh = d.in_layout == B2C_LAYOUT_NCHW ? d.W : d.W * d.C;
  int sw = d.in_layout == B2C_LAYOUT_NCHW ? 1 : d.C;
  if (e == cudaSuccess)
    e = launch_im2col(x, a, dt, g.Mg, g.PQ, g.Q, d.H, d.W, d.stride_h, d.stride_w, d.pad_h, d.pad_w, sn, sh, sw, K_pad,
                      st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(dt);
  CUDA_TRY(e);
  return B2C_OK;
}

}  // extern "C"
