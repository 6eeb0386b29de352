// Data-layout rewrites of Table 2 as CUDA kernels: Pad + Reorder of the activations
// (NCHW -> NHWC with the channel axis zero-padded to the intrinsic's block), the weight packs
// (reduction index made contiguous, Section 5.1: the B operand is held transposed), the
// explicit Stencil Unroll (im2col matrix, formed by direct indexing rather than the index-list
// gather the paper found slow in Section 6.1), and the finish pass of a split reduction.
#include "b2c_internal.h"

namespace b2c {

namespace {

constexpr int kPackC = 64;   // channels per tile
constexpr int kPackHW = 64;  // pixels per tile
constexpr int kPackPitch = kPackHW + 4;

// One block moves a [64 channels] x [64 pixels] tile of one image through shared memory:
// reads run along the pixel axis of NCHW, writes along the channel axis of NHWC in 16-byte
// vectors.  Channels >= C are written as zeros.
template <bool kVec4>
__global__ void __launch_bounds__(256) pack_activations_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ out,
                                                               int C, int HW, int C_pad, int hw_tiles) {
  __shared__ __align__(16) uint8_t tile[kPackC * kPackPitch];
  const int n = blockIdx.x / hw_tiles;
  const int c0 = blockIdx.y * kPackC;
  const int hw0 = (blockIdx.x - n * hw_tiles) * kPackHW;
  const int t = threadIdx.x;
  const int8_t* xin = x + (size_t)n * C * HW;
  if (kVec4) {
    // 16 threads cover one channel row (4 pixels each), 16 rows per pass.
    const int hq = (t & 15) * 4;
#pragma unroll
    for (int pass = 0; pass < kPackC / 16; ++pass) {
      const int cl = pass * 16 + (t >> 4);
      const int c = c0 + cl;
      uint32_t v = 0;
      if (c < C) {
        const int hw = hw0 + hq;
        if (hw + 3 < HW) {
          v = *reinterpret_cast<const uint32_t*>(xin + (size_t)c * HW + hw);
        } else {
          for (int i = 0; i < 4; ++i)
            if (hw + i < HW) v |= (uint32_t)(uint8_t)xin[(size_t)c * HW + hw + i] << (8 * i);
        }
      }
      *reinterpret_cast<uint32_t*>(&tile[cl * kPackPitch + hq]) = v;
    }
  } else {
    const int hl = t & 63;
#pragma unroll
    for (int pass = 0; pass < kPackC / 4; ++pass) {
      const int cl = pass * 4 + (t >> 6);
      const int c = c0 + cl;
      uint8_t v = 0;
      if (c < C && hw0 + hl < HW) v = (uint8_t)xin[(size_t)c * HW + hw0 + hl];
      tile[cl * kPackPitch + hl] = v;
    }
  }
  __syncthreads();
  // Thread -> (pixel, 16-channel chunk); 4 chunks per pixel.
  const int pl = t >> 2;
  const int ch = (t & 3) * 16;
  const int hw = hw0 + pl;
  if (hw < HW && c0 + ch < C_pad) {
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t v = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) v |= (uint32_t)tile[(ch + j * 4 + i) * kPackPitch + pl] << (8 * i);
      w[j] = v;
    }
    uint4 o = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(out + ((size_t)n * HW + hw) * C_pad + c0 + ch) = o;
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

// Stencil-unroll weights: rows of w[k][(c,r,s)] zero-padded to K_pad.
__global__ void pack_weights_rows_kernel(const int8_t* __restrict__ w, int8_t* __restrict__ out, int K, int Kg,
                                         int K_pad) {
  const long long total = (long long)K * K_pad;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(i % K_pad);
    const long long k = i / K_pad;
    out[i] = j < Kg ? w[k * Kg + j] : (int8_t)0;
  }
}

// Explicit stencil unroll.  One thread produces 16 consecutive reduction entries of one output
// pixel's row and stores them as one 16-byte vector; the window geometry comes from a lookup
// table indexed by the reduction position, so no per-element division is needed.
__global__ void __launch_bounds__(256) im2col_kernel(const int8_t* __restrict__ x, int8_t* __restrict__ a,
                                                     const GatherEntry* __restrict__ table, long long Mg, int PQ, int Q,
                                                     int H, int W, int stride_h, int stride_w, int pad_h, int pad_w,
                                                     long long x_stride_n, int x_stride_h, int x_stride_w, int K_pad) {
  const int chunks = K_pad >> 4;
  const long long total = Mg * chunks;
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
      if (g.off >= 0 && (unsigned)h < (unsigned)H && (unsigned)ww < (unsigned)W) v = (uint8_t)base[g.off];
      wv[e >> 2] |= v << (8 * (e & 3));
    }
    *reinterpret_cast<uint4*>(a + m * K_pad + ck * 16) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
  }
}

// Finish of a split reduction: the int32 sums are complete in `acc`; copy them out and/or apply
// the shift-and-clip requantisation (arithmetic shift = floor division by 2^shift).
__global__ void splitk_finish_kernel(const int32_t* __restrict__ acc, int32_t* __restrict__ y32,
                                     int8_t* __restrict__ y8, long long elems, int shift, int out_mode) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < elems;
       i += (long long)gridDim.x * blockDim.x) {
    const int v = acc[i];
    if ((out_mode & B2C_OUT_I32) && y32 != acc) y32[i] = v;
    if (out_mode & B2C_OUT_I8) y8[i] = (int8_t)max(-128, min(127, v >> shift));
  }
}

int grid_for(long long total, int block) {
  long long g = (total + block - 1) / block;
  const long long cap = (long long)kNumSMs * 16;
  return (int)(g < 1 ? 1 : (g > cap ? cap : g));
}

}  // namespace

cudaError_t launch_pack_activations(const int8_t* x, int8_t* out, int N, int C, int H, int W, int C_pad,
                                    cudaStream_t st) {
  const int HW = H * W;
  const int hw_tiles = (HW + kPackHW - 1) / kPackHW;
  dim3 grid((unsigned)hw_tiles * (unsigned)N, (C_pad + kPackC - 1) / kPackC, 1);
  const bool vec4 = (HW % 4 == 0) && ((reinterpret_cast<uintptr_t>(x) & 3) == 0);
  if (vec4)
    pack_activations_kernel<true><<<grid, 256, 0, st>>>(x, out, C, HW, C_pad, hw_tiles);
  else
    pack_activations_kernel<false><<<grid, 256, 0, st>>>(x, out, C, HW, C_pad, hw_tiles);
  return cudaGetLastError();
}

cudaError_t launch_pack_weights_cp(const int8_t* w, int8_t* out, int K, int C, int R, int S, int C_pad,
                                   cudaStream_t st) {
  const long long total = (long long)K * R * S * C_pad;
  pack_weights_cp_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, out, K, C, R * S, C_pad);
  return cudaGetLastError();
}

cudaError_t launch_pack_weights_rows(const int8_t* w, int8_t* out, int K, int Kg, int K_pad, cudaStream_t st) {
  const long long total = (long long)K * K_pad;
  pack_weights_rows_kernel<<<grid_for(total, 256), 256, 0, st>>>(w, out, K, Kg, K_pad);
  return cudaGetLastError();
}

cudaError_t launch_im2col(const int8_t* x, int8_t* a, const GatherEntry* table, long long Mg, int PQ, int Q, int H,
                          int W, int stride_h, int stride_w, int pad_h, int pad_w, long long x_stride_n,
                          int x_stride_h, int x_stride_w, int K_pad, cudaStream_t st) {
  const long long total = Mg * (K_pad / 16);
  im2col_kernel<<<grid_for(total, 256), 256, 0, st>>>(x, a, table, Mg, PQ, Q, H, W, stride_h, stride_w, pad_h, pad_w,
                                                      x_stride_n, x_stride_h, x_stride_w, K_pad);
  return cudaGetLastError();
}

cudaError_t launch_splitk_finish(const int32_t* acc, int32_t* y32, int8_t* y8, long long elems, int shift,
                                 int out_mode, cudaStream_t st) {
  splitk_finish_kernel<<<grid_for(elems, 256), 256, 0, st>>>(acc, y32, y8, elems, shift, out_mode);
  return cudaGetLastError();
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

