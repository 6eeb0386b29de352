// Host-side embedding planner: which convolution axes feed the MMA's M / N / K dimensions, with
// which layout rewrite, tile width and reduction split.
//
// The paper finds embeddings by constraint solving over the scalar data-flow graph (Section 4)
// and derives the layout rewrites of Table 2 from the solution.  For a 2-D convolution on a
// matrix-multiply intrinsic the legal, axis-aligned, dense solutions form a small closed family
// (the hyper-rectangle and linear-access constraints of Section 4.2 leave only: feed K from the
// padded channel axis, or from the unrolled stencil), so this planner writes that family out
// directly, ranks it with the overhead terms of Section 4.4 and leaves the final choice to
// measured device time, as Section 6.1 does with its five best candidates.
#include <algorithm>
#include <cstring>

#include "b2c_internal.h"

namespace b2c {

int round_up(int v, int m) { return (v + m - 1) / m * m; }

static int out_extent(int in, int k, int stride, int pad, int dil) {
  long long span = (long long)in + 2LL * pad - (long long)dil * (k - 1) - 1;
  if (span < 0) return 0;
  return (int)(span / stride) + 1;
}

int resolve_geom(const b2c_conv_desc* d, Geom* g) {
  if (!d || !g) return B2C_E_INVALID_ARG;
  if (d->N < 1 || d->C < 1 || d->H < 1 || d->W < 1 || d->K < 1 || d->R < 1 || d->S < 1) return B2C_E_INVALID_ARG;
  if (d->stride_h < 1 || d->stride_w < 1 || d->pad_h < 0 || d->pad_w < 0 || d->dil_h < 1 || d->dil_w < 1)
    return B2C_E_INVALID_ARG;
  if (d->shift < 0 || d->shift > 31) return B2C_E_INVALID_ARG;
  if (d->in_layout != B2C_LAYOUT_NCHW && d->in_layout != B2C_LAYOUT_NHWC) return B2C_E_INVALID_ARG;
  if (d->out_layout != B2C_LAYOUT_NCHW && d->out_layout != B2C_LAYOUT_NHWC) return B2C_E_INVALID_ARG;
  if ((d->out_mode & ~3) != 0 || (d->out_mode & 3) == 0) return B2C_E_INVALID_ARG;
  g->d = *d;
  g->P = out_extent(d->H, d->R, d->stride_h, d->pad_h, d->dil_h);
  g->Q = out_extent(d->W, d->S, d->stride_w, d->pad_w, d->dil_w);
  long long kg = (long long)d->C * d->R * d->S;
  if (g->P == 0 || g->Q == 0) return B2C_E_UNSUPPORTED;
  if (kg > kMaxKg) return B2C_E_UNSUPPORTED;
  // A padding of a million pixels per side serves no convolution and would let the products below
  // leave 64 bits for extreme images; P*Q must fit 31 bits before anything is derived from it.
  if (d->pad_h > (1 << 20) || d->pad_w > (1 << 20)) return B2C_E_UNSUPPORTED;
  const long long pq = (long long)g->P * g->Q;
  if (pq > 0x7FFFFF00LL) return B2C_E_UNSUPPORTED;
  g->PQ = (int)pq;
  g->Mg = (long long)d->N * pq;
  g->Kg = (int)kg;
  g->x_elems = (long long)d->N * d->C * d->H * d->W;
  g->w_elems = (long long)d->K * kg;
  g->y_elems = g->Mg * d->K;
  // Index arithmetic in the kernels is 32-bit for rows/columns and 64-bit for byte offsets.
  if (g->Mg > 0x7FFFFF00LL || g->x_elems > (1LL << 40) || g->y_elems > (1LL << 40)) return B2C_E_UNSUPPORTED;
  if ((long long)d->H * d->W * d->C > 0x7FFFFFFFLL) return B2C_E_UNSUPPORTED;
  return B2C_OK;
}

// Pad rule (Table 2, rule 2) for the channel axis: the intrinsic consumes 32 channels per
// instruction, so C is padded to a multiple of 32.
int cp_channel_pad(int C) { return round_up(C, kMmaK); }

// Split rule (Table 2, rule 3): the padded channel axis is cut into blocks of the largest of
// 128 / 64 / 32 bytes that divides it (one shared-memory swizzle row per block).
int cp_block_bytes(int C_pad) {
  if (C_pad % 128 == 0) return 128;
  if (C_pad % 64 == 0) return 64;
  return 32;
}

int im2col_k_pad(int Kg) { return round_up(Kg, kMmaK); }

bool staged_word_mode(const Geom& g) { return g.d.dil_w == 1; }
int staged_run_len(const Geom& g) { return staged_word_mode(g) ? round_up(g.d.S, 4) : g.d.S; }
int variant_k_pad(const Geom& g, int variant) {
  if (variant == B2C_VARIANT_IM2COL_WINDOW) return round_up(g.d.C * g.d.R * round_up(g.d.S, 4), kMmaK);
  if (variant == B2C_VARIANT_IM2COL_STAGED) return round_up(g.d.C * g.d.R * staged_run_len(g), kMmaK);
  return im2col_k_pad(g.Kg);
}

size_t workspace_bytes_for(const Geom& g, int variant, int tile_n, int split_k, bool swap) {
  size_t ws = 0;
  const b2c_conv_desc& d = g.d;
  TmaView v;
  if (is_tma_view_variant(variant) && tma_view_for(g, variant, &v)) {
    bool direct = shift_base_variant(variant) == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NHWC && v.C == d.C;
    if (!direct) ws += (size_t)v.bytes();
  } else if (variant == B2C_VARIANT_IM2COL_EXPLICIT) {
    ws += (size_t)g.Mg * im2col_k_pad(g.Kg);
  }
  ws = (ws + 255) / 256 * 256;
  // A split reduction accumulates int32 partial sums in scratch unless the int32 output itself
  // can serve (int32-only output in any layout).
  if (split_k > 1 && !cluster_split_ok(variant, tile_n, split_k, swap) && (d.out_mode & B2C_OUT_I8))
    ws += (size_t)g.y_elems * 4;
  return ws;
}

// Limits of the 4-D im2col-mode tensor map: corners in [-128, 127], tap offsets in [0, 255],
// traversal strides in [1, 8].
static bool view_fits_tensor_map(const TmaView& v) {
  int up_w = v.pad_w - (v.S - 1) * v.dil_w, up_h = v.pad_h - (v.R - 1) * v.dil_h;
  if (v.pad_w > 128 || v.pad_h > 128 || up_w < -128 || up_h < -128 || up_w > 127 || up_h > 127) return false;
  if ((v.S - 1) * v.dil_w > 255 || (v.R - 1) * v.dil_h > 255) return false;
  if (v.stride_w > 8 || v.stride_h > 8) return false;
  if (v.bytes() > (1LL << 40) || (long long)v.H * v.W * v.C > 0x7FFFFFFFLL) return false;
  return true;
}

int s2d_pack_factor(const Geom& g) {
  const int cphase = g.d.C * g.d.stride_h * g.d.stride_w;
  const int Sp = (g.d.S + g.d.stride_w - 1) / g.d.stride_w;
  if (cphase > kMmaK / 2) return 1;
  return std::max(1, std::min(kMmaK / cphase, Sp));
}

bool shift_geom(const Geom& g, const TmaView& v, ShiftGeom* sg, bool tiles_2d) {
  if (v.stride_h != 1 || v.stride_w != 1 || g.d.K > 256) return false;
  sg->cb = cp_block_bytes(v.C);
  sg->ncb = v.C / sg->cb;
  sg->tiles_h = sg->tiles_w = 0;
  long long rows;
  sg->two_d = 0;
  sg->valid_w = 0;
  // Two-dimensional tiles for the multi-tap views: a tile is 128/pitch rows of `pitch` window origins
  // (pitch a power of two), its window one TMA box of the rows those origins and their taps touch.
  // Narrow rows (padded width up to 128, at most a quarter lost to rounding the pitch up): the pitch
  // covers the whole padded row and a tile is several image rows.  Wide rows (padded width >= 192):
  // one-row tiles of 128 origins of which the last (S - 1)*dil_w only serve as the taps' overhang
  // (tiles advance by the valid width).  In between, and for anything else, the window is whole
  // padded rows (below).
  const int wp_real = v.W + 2 * v.pad_w;
  const long long wp_full = round_up(wp_real, 8);
  const int overhang = (v.S - 1) * v.dil_w;
  int pitch = 16;
  while (pitch < wp_real) pitch <<= 1;
  const bool narrow_2d = !tiles_2d && pitch <= kTileM && (long long)pitch * 100 <= wp_full * 125;
  const bool wide_2d = !tiles_2d && v.S > 1 && wp_full >= 192 && overhang <= kTileM / 4;
  if (narrow_2d || wide_2d) {
    sg->two_d = 1;
    sg->wps = narrow_2d ? pitch : kTileM;
    sg->valid_w = narrow_2d ? wp_real - overhang : kTileM - overhang;
    sg->hp = v.H + 2 * v.pad_h;
    const int tile_h = kTileM / sg->wps;
    rows = tile_h + (long long)(v.R - 1) * v.dil_h + (overhang > 0 ? 1 : 0);
    if (rows > 256) return false;
    sg->tiles_h = (g.P + tile_h - 1) / tile_h;
    sg->tiles_w = (g.Q + sg->valid_w - 1) / sg->valid_w;
  } else if (tiles_2d) {
    // tiles of 128/tw x tw pixels over an unpadded view with one tap per filter row: the window is one
    // box of (128/tw + R - 1) rows of tw pixels, and a tap moves the tile by one row of tw pixels
    if (v.S != 1 || v.pad_h != 0 || v.pad_w != 0 || v.dil_h != 1) return false;
    sg->two_d = 1;
    // tile width: the widest power of two up to 128 that wastes at most 15 % of its columns on the
    // ragged right edge (wide tiles give long contiguous output runs), else 16
    int tile_w = kShiftTileW;
    for (int tw = kTileM; tw > kShiftTileW; tw >>= 1)
      if ((long long)((g.Q + tw - 1) / tw) * tw * 100 <= (long long)g.Q * 115) {
        tile_w = tw;
        break;
      }
    const int tile_h = kTileM / tile_w;
    sg->wps = tile_w;
    sg->valid_w = tile_w;
    sg->hp = v.H;
    rows = tile_h + v.R - 1;
    if (rows > 256) return false;
    sg->tiles_h = (g.P + tile_h - 1) / tile_h;
    sg->tiles_w = (g.Q + tile_w - 1) / tile_w;
  } else {
    const int wp = v.W + 2 * v.pad_w;
    sg->wps = round_up(wp, 8);
    sg->hp = v.H + 2 * v.pad_h;
    if (sg->wps > 256) return false;  // one copy per staged image row
    const long long shift_max = (long long)(v.R - 1) * v.dil_h * sg->wps + (long long)(v.S - 1) * v.dil_w;
    // a tile starts anywhere inside its first staged row and reads 128 positions plus the largest shift
    rows = (sg->wps - 1 + kTileM - 1 + shift_max) / sg->wps + 1;
    if (rows > 4096) return false;
  }
  sg->rows = (int)rows;
  sg->row_bytes = sg->wps * sg->cb;
  const long long cblk = rows * sg->row_bytes;
  const long long win = (cblk * sg->ncb + 1023) / 1024 * 1024;
  int tile_n = 16;
  while (tile_n < g.d.K) tile_n <<= 1;
  const long long wbytes = (long long)v.R * v.S * sg->ncb * tile_n * sg->cb;
  if (2 * win + wbytes + 2048 > 200 * 1024) return false;
  sg->cblk_bytes = (int)cblk;
  sg->win_bytes = (int)win;
  sg->w_bytes = (int)wbytes;
  sg->tile_n = tile_n;
  // Window buffers per block and blocks per SM: as many windows in flight per SM as fit (each block
  // at least two, at most six), preferring more resident blocks on a tie.
  sg->stages = 2;
  sg->blocks_per_sm = 1;
  for (int bps = 3; bps >= 1; --bps) {
    const long long room = (220 * 1024) / bps - wbytes - 2048;
    const int st = (int)std::min<long long>(6, std::min<long long>(room, 198 * 1024 - wbytes) / win);
    if (st >= 2 && st * bps > sg->stages * sg->blocks_per_sm) {
      sg->stages = st;
      sg->blocks_per_sm = bps;
    }
  }
  sg->mtot = sg->two_d ? (long long)v.N * sg->tiles_h * sg->tiles_w * kTileM : (long long)v.N * sg->hp * sg->wps;
  return sg->mtot <= 0x7FFFFF00LL;
}

bool tma_view_for(const Geom& g, int variant, TmaView* v) {
  const b2c_conv_desc& d = g.d;
  if (variant == B2C_VARIANT_ROWPHASE_SHIFT) {
    // Stencil Unroll along s and Image Pack of the vertical stride in one rewrite:
    // U[n][h'][q][(dh, s, c)] = x[n][c][h'*stride_h + dh - pad_h][q*stride_w - pad_w + s*dil_w], and an
    // R' x 1, stride-1, unpadded convolution over U remains (r = r'*stride_h + dh).
    if (d.dil_h != 1) return false;
    const int Rp = (d.R + d.stride_h - 1) / d.stride_h;
    const long long cq = (long long)d.stride_h * d.S * d.C;
    if (cq > 4096) return false;
    if ((long long)d.C * d.stride_h * row_phase_seg(d.stride_w, d.S, d.dil_w) > kRowPhaseSmemMax) return false;
    *v = TmaView{d.N, round_up((int)cq, kMmaK), g.P + Rp - 1, g.Q, Rp, 1, 1, 1, 0, 0, 1, 1};
    ShiftGeom sg;
    return view_fits_tensor_map(*v) && shift_geom(g, *v, &sg, true);
  }
  if (is_shift_variant(variant)) {
    ShiftGeom sg;
    return tma_view_for(g, shift_base_variant(variant), v) && shift_geom(g, *v, &sg);
  }
  if (variant == B2C_VARIANT_CP_TMA) {
    // Pad + Split + Reorder of the channel axis (Table 2).  An NHWC source with a multiple of 32
    // channels is read in place; any other NHWC source is re-padded into the scratch tensor.
    *v = TmaView{d.N, cp_channel_pad(d.C), d.H, d.W, d.R, d.S, d.stride_h, d.stride_w, d.pad_h, d.pad_w, d.dil_h, d.dil_w};
  } else if (variant == B2C_VARIANT_ROW_UNROLL) {
    // Stencil Unroll along s only: U[n][h][q][(s, c)] = x[n][c][h][q*stride_w - pad_w + s*dil_w].
    // What is left is an R x 1 convolution over U with the vertical geometry unchanged.
    if (d.S == 1) return false;  // nothing to unroll: same as the channel-pack map
    *v = TmaView{d.N, round_up(d.S * d.C, kMmaK), d.H, g.Q, d.R, 1, d.stride_h, 1, d.pad_h, 0, d.dil_h, 1};
  } else if (variant == B2C_VARIANT_SPACE_TO_DEPTH) {
    // Image Pack of a strided convolution: with hp = h + pad_h = (p + r')*stride_h + dh the stride
    // phases (dh, dw) become channels of X'[n][hp / stride_h][wp / stride_w][(c, dh, dw)], and a
    // stride-1, unpadded R' x S' convolution over X' remains (R' = ceil(R / stride_h)).
    if (d.dil_h != 1 || d.dil_w != 1 || (d.stride_h == 1 && d.stride_w == 1)) return false;
    const int Rp = (d.R + d.stride_h - 1) / d.stride_h, Sp = (d.S + d.stride_w - 1) / d.stride_w;
    // horizontal tap packing: X''[..][w'][(ui, c, dh, dw)] = X'[..][w' + ui][(c, dh, dw)], taps at w' + pack*s''
    const int pack = s2d_pack_factor(g);
    const int Sv = (Sp + pack - 1) / pack;
    *v = TmaView{d.N, round_up(pack * d.C * d.stride_h * d.stride_w, kMmaK), g.P + Rp - 1, g.Q + pack * (Sv - 1), Rp, Sv,
                 1, 1, 0, 0, 1, pack};
  } else if (variant == B2C_VARIANT_DILATION_PACK) {
    // Image Pack of a dilated convolution (Section 6.1): with h - pad_h = i*dil_h + a every tap of an
    // output pixel reads phase a of the image, X_a[j] = x[j*dil_h + a], at j = i + r.  The dil_h*dil_w
    // phase sub-images (extent ceil(H / dil_h), zeros past the image) are fused into the batch and a
    // dense, stride-1 R x S convolution with padding ceil(pad / dil) remains.
    if ((d.dil_h == 1 && d.dil_w == 1) || d.stride_h != 1 || d.stride_w != 1) return false;
    const long long n_sub = (long long)d.N * d.dil_h * d.dil_w;
    if (n_sub > 0x7FFFFFFF) return false;
    *v = TmaView{(int)n_sub, cp_channel_pad(d.C), (d.H + d.dil_h - 1) / d.dil_h, (d.W + d.dil_w - 1) / d.dil_w, d.R, d.S,
                 1, 1, (d.pad_h + d.dil_h - 1) / d.dil_h, (d.pad_w + d.dil_w - 1) / d.dil_w, 1, 1};
    const long long rows = (long long)v->N * (v->H + 2 * v->pad_h - v->R + 1) * (v->W + 2 * v->pad_w - v->S + 1);
    if (rows > 0x7FFFFF00LL) return false;
  } else {
    return false;
  }
  return view_fits_tensor_map(*v);
}

long long view_rows(const Geom& g, int variant, const TmaView& v) {
  if (is_shift_variant(variant)) {
    // window origins on the padded grid (width rounded up to 8), not only the valid output pixels
    ShiftGeom sg;
    return shift_geom(g, v, &sg, shift_tiles_2d(variant)) ? sg.mtot : g.Mg;
  }
  if (variant != B2C_VARIANT_DILATION_PACK) return g.Mg;
  return (long long)v.N * (v.H + 2 * v.pad_h - v.R + 1) * (v.W + 2 * v.pad_w - v.S + 1);
}

// The staged stencil unroll keeps, per image a tile can touch, the zero-padded input rows that
// feed the tile's 128 output pixels: C x rows x pitch bytes, with the left margin rounded up to 16
// so that aligned 16-byte copies land on aligned shared-memory addresses.
bool staged_window(const Geom& g, WindowGeom* w) {
  const b2c_conv_desc& d = g.d;
  if (d.in_layout != B2C_LAYOUT_NCHW) return false;  // the window is staged from whole NCHW rows
  const int rows_out = std::min(g.P, (kTileM - 2) / g.Q + 2);  // output rows 128 consecutive pixels can span
  const int parts = (int)std::min<long long>(d.N, (kTileM - 2) / g.PQ + 2);
  const long long rows = (long long)(rows_out - 1) * d.stride_h + (long long)(d.R - 1) * d.dil_h + 1;
  const long long left = round_up(d.pad_w, 16);
  // columns read: up to (Q-1)*stride_w - pad_w + (S-1)*dil_w
  const long long right_edge = (long long)(g.Q - 1) * d.stride_w - d.pad_w + (long long)(d.S - 1) * d.dil_w + 1;
  const long long width = std::max<long long>(d.W, right_edge);
  const long long pitch = (left + width + 15) / 16 * 16;
  const long long bytes = (long long)parts * d.C * rows * pitch;
  if (bytes > 64 * 1024 || variant_k_pad(g, B2C_VARIANT_IM2COL_STAGED) > 4096) return false;
  w->rows = (int)rows;
  w->pitch = (int)pitch;
  w->left = (int)left;
  w->parts = parts;
  w->bytes = (int)bytes;
  return true;
}

// Small images: whole images as the window, linear tiles.
static bool window_linear_geom(const Geom& g, WindowTile* wt) {
  const b2c_conv_desc& d = g.d;
  const long long chw = (long long)d.C * d.H * d.W;
  // an image is one bulk copy (16-byte multiple, a few KB); a tile of 128 consecutive pixels touches
  // at most four images; runs of at most two words; the margin in front of the window covers the
  // negative offsets of the padding (those taps are masked, but their addresses must be valid)
  if ((chw % 16) != 0 || chw > 16 * 1024 || d.S > 8 || d.R > 32 || g.PQ < 43) return false;
  if ((long long)d.pad_h * d.W + d.pad_w + 8 > 128) return false;
  const int parts = (kTileM - 2) / g.PQ + 2;
  wt->linear = 1;
  wt->tile_w = kTileM;
  wt->tile_h = 1;
  wt->win_w = d.W;
  wt->win_h = d.H;
  wt->left = 128;
  wt->off0 = 0;
  wt->tiles_h = wt->tiles_w = 1;
  wt->box_bytes = (int)chw;
  // rows below the image that masked taps may address: up to (R-1)*dil_h rows past the last output row's first tap
  const long long slack = round_up((int)((long long)(d.R - 1) * d.dil_h * d.W + d.S + 16), 128) + 128;
  const long long win = 128 + (long long)parts * chw + slack;
  if (win > 60 * 1024 || chw >= (1 << 16) || win >= (1 << 16)) return false;
  wt->win_bytes = round_up((int)win, 128);
  wt->mtot = g.Mg;
  return true;
}

bool window_tile_geom(const Geom& g, WindowTile* wt) {
  const b2c_conv_desc& d = g.d;
  // words of an A row are unaligned words of a window row: unit horizontal dilation
  if (d.in_layout != B2C_LAYOUT_NCHW || d.dil_w != 1 || d.C > 64 || d.K > 256) return false;
  wt->linear = 0;
  wt->S_run = round_up(d.S, 4);
  wt->K_pad = round_up(d.C * d.R * wt->S_run, kMmaK);
  if (wt->K_pad > 1024) return false;
  wt->num_kb = (wt->K_pad + 127) / 128;
  wt->tile_n = 16;
  while (wt->tile_n < d.K) wt->tile_n <<= 1;
  // small images: linear tiles over whole images (no padded positions at all)
  if (((d.W % 16) != 0 || g.PQ <= 1024) && window_linear_geom(g, wt)) {
    wt->smem = 1024 + 2 * (size_t)wt->num_kb * kTileM * 128 + (size_t)wt->num_kb * wt->tile_n * 128 + kWindowStages * (size_t)wt->win_bytes +
               (size_t)round_up(wt->K_pad, 128) + 256;
    return wt->mtot <= 0x7FFFFF00LL && wt->smem <= 200 * 1024;
  }
  wt->linear = 0;
  // the window is one tiled TMA box of the NCHW tensor: rows must be multiples of 16 bytes, every box
  // extent at most 256
  if ((d.W % 16) != 0) return false;
  wt->left = round_up(d.pad_w, 16);
  wt->off0 = wt->left - d.pad_w;
  long long best_tiles = -1;
  for (int tw = kTileM; tw >= 16; tw >>= 1) {
    const int th = kTileM / tw;
    // last byte a row can touch: the last pixel's last (padded) tap, plus the second word of an unaligned read
    const long long ww = round_up((int)std::min<long long>((long long)(tw - 1) * d.stride_w + wt->off0 + wt->S_run + 8, 1 << 20), 16);
    const long long wh = (long long)(th - 1) * d.stride_h + (long long)(d.R - 1) * d.dil_h + 1;
    if (ww > 256 || wh > 256 || (long long)d.C * wh * ww > 24 * 1024) continue;
    const long long tiles = (long long)((g.P + th - 1) / th) * ((g.Q + tw - 1) / tw);
    if (best_tiles < 0 || tiles < best_tiles) {
      best_tiles = tiles;
      wt->tile_w = tw;
      wt->tile_h = th;
      wt->win_w = (int)ww;
      wt->win_h = (int)wh;
    }
  }
  if (best_tiles < 0) return false;
  wt->tiles_h = (g.P + wt->tile_h - 1) / wt->tile_h;
  wt->tiles_w = (g.Q + wt->tile_w - 1) / wt->tile_w;
  wt->box_bytes = d.C * wt->win_h * wt->win_w;
  wt->win_bytes = round_up(wt->box_bytes + 32, 128);
  wt->mtot = (long long)d.N * wt->tiles_h * wt->tiles_w * kTileM;
  wt->smem = 1024 + 2 * (size_t)wt->num_kb * kTileM * 128 + (size_t)wt->num_kb * wt->tile_n * 128 + kWindowStages * (size_t)wt->win_bytes +
             (size_t)round_up(wt->K_pad, 128) + 256;
  return wt->mtot <= 0x7FFFFF00LL && wt->smem <= 200 * 1024 && (long long)d.N * wt->tiles_h * wt->tiles_w < 0x7FFFFFFFLL;
}

static void add(std::vector<b2c_embedding>* out, const Geom& g, int variant, int tile_n, int split_k,
                bool swap = false, int tile_m = kTileM) {
  const b2c_conv_desc& d = g.d;
  b2c_embedding e;
  std::memset(&e, 0, sizeof(e));
  e.map_m = swap ? B2C_AXIS_K : B2C_AXIS_NPQ;
  e.map_n = swap ? B2C_AXIS_NPQ : B2C_AXIS_K;
  e.variant = variant;
  e.tile_m = tile_m;
  e.tile_n = tile_n;
  e.split_k = split_k;
  e.device_us = -1.0f;
  long long M_pad = (g.Mg + tile_m - 1) / tile_m * tile_m;
  long long N_pad = (long long)round_up(d.K, tile_n);
  if (swap) {
    M_pad = (long long)round_up(d.K, kTileM);
    N_pad = (g.Mg + tile_n - 1) / tile_n * tile_n;
  }
  long long k_issued, moved;
  long long mac_min = g.Mg * d.K * g.Kg;
  long long data_min = g.x_elems + g.w_elems + g.y_elems;
  TmaView v;
  if (is_tma_view_variant(variant) && tma_view_for(g, variant, &v)) {
    e.map_k = (variant == B2C_VARIANT_CP_TMA || variant == B2C_VARIANT_DILATION_PACK || variant == B2C_VARIANT_CP_SHIFT)
                  ? B2C_AXIS_C
                  : ((variant == B2C_VARIANT_ROW_UNROLL || variant == B2C_VARIANT_ROWPHASE_SHIFT) ? B2C_AXIS_SC
                                                                                                  : B2C_AXIS_C_PHASES);
    if (!swap) M_pad = (view_rows(g, variant, v) + tile_m - 1) / tile_m * tile_m;
    k_issued = (long long)v.R * v.S * v.C;
    long long packed = v.bytes();
    bool direct = shift_base_variant(variant) == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NHWC && v.C == d.C;
    moved = (direct ? 0 : g.x_elems + packed) + packed + (long long)d.K * k_issued + g.y_elems;
  } else {
    e.map_k = B2C_AXIS_CRS;
    int K_pad = variant_k_pad(g, variant);
    k_issued = K_pad;
    WindowTile wt;
    if (variant == B2C_VARIANT_IM2COL_WINDOW && window_tile_geom(g, &wt)) M_pad = wt.mtot;  // whole two-dimensional tiles
    if (variant == B2C_VARIANT_IM2COL_EXPLICIT)
      moved = g.x_elems + 2 * g.Mg * K_pad + (long long)d.K * K_pad + g.y_elems;
    else if (variant == B2C_VARIANT_IM2COL_STAGED)
      moved = g.x_elems + (long long)d.K * K_pad + g.y_elems;
    else
      moved = g.x_elems + (long long)d.K * K_pad + g.y_elems;
  }
  if (split_k > 1 && !cluster_split_ok(variant, tile_n, split_k, swap)) moved += 2 * g.y_elems;  // partial sums through memory
  e.o_mac = M_pad * N_pad * k_issued - mac_min;
  e.o_data = moved - data_min;
  e.workspace_bytes = (int64_t)workspace_bytes_for(g, variant, tile_n, split_k, swap);
  // two-SM channel-pack schedule on NCHW input: room for the work counters of the pack that runs
  // inside the MMA kernel (1 + N integers after the rewritten operand)
  if (tile_m == 2 * kTileM && variant == B2C_VARIANT_CP_TMA && d.in_layout == B2C_LAYOUT_NCHW)
    e.workspace_bytes = (e.workspace_bytes + 255) / 256 * 256 + ((int64_t)(d.N + 1) * 4 + 255) / 256 * 256;
  out->push_back(e);
}

void enumerate_embeddings(const Geom& g, std::vector<b2c_embedding>* out) {
  out->clear();
  const b2c_conv_desc& d = g.d;
  // Tile widths: every MMA N extent up to the first one that covers K.
  std::vector<int> tiles;
  for (int t = 16; t <= 256; t <<= 1) {
    tiles.push_back(t);
    if (t >= d.K) break;
  }
  for (int variant = 0; variant < kNumVariants; ++variant) {
    TmaView view;
    if (is_tma_view_variant(variant) && !tma_view_for(g, variant, &view)) continue;
    const long long tiles_m =
        ((is_tma_view_variant(variant) ? view_rows(g, variant, view) : g.Mg) + kTileM - 1) / kTileM;
    WindowGeom wg;
    if (variant == B2C_VARIANT_IM2COL_STAGED && !staged_window(g, &wg)) continue;
    if (variant == B2C_VARIANT_IM2COL_WINDOW) {
      // one schedule: all output channels in one column tile (the weights are resident), no split
      WindowTile wt;
      if (window_tile_geom(g, &wt)) add(out, g, variant, wt.tile_n, 1);
      continue;
    }
    int num_kb;
    if (is_tma_view_variant(variant)) {
      num_kb = view.R * view.S * (view.C / cp_block_bytes(view.C));
    } else {
      num_kb = (variant_k_pad(g, variant) + 127) / 128;
    }
    // The in-kernel gather keeps its lookup table in shared memory.
    if (variant == B2C_VARIANT_IM2COL_GATHER && im2col_k_pad(g.Kg) > 4096) continue;
    if (is_shift_variant(variant)) {
      // one schedule: all output channels in one column tile (the weights are resident), no split
      ShiftGeom sg;
      if (shift_geom(g, view, &sg, shift_tiles_2d(variant))) add(out, g, variant, sg.tile_n, 1);
      continue;
    }
    for (int t : tiles) {
      // Skip widths that only add padding: keep t if it is the covering width or K % t == 0
      // or it wastes less than a quarter of the columns.
      int n_pad = round_up(d.K, t);
      if (t < tiles.back() && (n_pad - d.K) * 4 > n_pad) continue;
      long long ctas = tiles_m * (n_pad / t);
      for (int split = 1; split <= 32; split <<= 1) {
        if (split > num_kb) break;
        // A split reduction only helps while the grid is smaller than the machine.
        if (split > 1 && ctas * (split / 2) >= kNumSMs) break;
        add(out, g, variant, t, split);
      }
      // two-SM schedule of the same map: 256-row tiles, each block of the pair loads half of the column tile
      if (pair_schedule_ok(variant, t, 1, false, tiles_m * kTileM)) add(out, g, variant, t, 1, false, 2 * kTileM);
    }
    // Swapped axis map (M <- k, N <- fused pixels) for the TMA-fed variants: the 128 accumulator rows
    // are output channels, so it is only listed when K fills at least half of them; the pixel tile
    // widths are those that waste less than a quarter of their columns (or the covering one).
    if ((is_tma_view_variant(variant) || variant == B2C_VARIANT_IM2COL_EXPLICIT) && d.K >= kTileM / 2 &&
        variant != B2C_VARIANT_DILATION_PACK && !is_shift_variant(variant)) {
      const long long tiles_k = (d.K + kTileM - 1) / kTileM;
      for (int t = 32; t <= 256; t <<= 1) {
        const long long n_pad = (g.Mg + t - 1) / t * t;
        const bool covering = t >= g.Mg || t == 256;
        if (!covering && (n_pad - g.Mg) * 4 > n_pad) continue;
        const long long ctas = tiles_k * (n_pad / t);
        for (int split = 1; split <= 32; split <<= 1) {
          if (split > num_kb) break;
          if (split > 1 && ctas * (split / 2) >= kNumSMs) break;
          add(out, g, variant, t, split, true);
        }
        if (t >= g.Mg) break;
      }
    }
  }
  std::stable_sort(out->begin(), out->end(), [](const b2c_embedding& a, const b2c_embedding& b) {
    return a.o_mac + a.o_data < b.o_mac + b.o_data;
  });
  for (size_t i = 0; i < out->size(); ++i) (*out)[i].id = (int)i;
}

int pick_by_policy(const std::vector<b2c_embedding>& all, int policy) {
  if (all.empty()) return -1;
  if (policy >= 0) return policy < (int)all.size() ? policy : -1;
  if (policy == B2C_POLICY_MIN_WORKSPACE) {
    int best = 0;
    for (size_t i = 1; i < all.size(); ++i)
      if (all[i].workspace_bytes < all[best].workspace_bytes) best = (int)i;
    return best;
  }
  return 0;  // MIN_OVERHEAD (AUTO_TIMED is resolved by the caller)
}

}  // namespace b2c
