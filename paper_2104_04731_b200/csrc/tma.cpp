// Tensor-map construction for the TMA loads of the MMA kernel.  The driver's encoders are
// looked up at run time through cudaGetDriverEntryPoint, so the library has no link-time
// dependency on libcuda and loads on machines without a driver.
#include <atomic>
#include <mutex>

#include "b2c_internal.h"

namespace b2c {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn g_tiled = nullptr;
static EncodeIm2colFn g_im2col = nullptr;
static std::once_flag g_once;
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }
int get_last_cuda_error() { return g_last_cuda_error; }
// Host-side fault injection for the tests: the n-th tensor-map encode from now on reports failure.
static std::atomic<int> g_fail_countdown{0};
static bool injected_failure() {
  int n = g_fail_countdown.load();
  while (n > 0) {
    if (g_fail_countdown.compare_exchange_weak(n, n - 1)) {
      if (n == 1) {
        set_last_cuda_error((int)CUDA_ERROR_INVALID_VALUE);
        return true;
      }
      return false;
    }
  }
  return false;
}


static void resolve() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    g_tiled = (EncodeTiledFn)fn;
  fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    g_im2col = (EncodeIm2colFn)fn;
}

static CUtensorMapSwizzle swizzle_of(int bytes) {
  switch (bytes) {
    case 128: return CU_TENSOR_MAP_SWIZZLE_128B;
    case 64: return CU_TENSOR_MAP_SWIZZLE_64B;
    case 32: return CU_TENSOR_MAP_SWIZZLE_32B;
    default: return CU_TENSOR_MAP_SWIZZLE_NONE;
  }
}

int encode_tiled_2d(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_bytes,
                    uint32_t box_inner, uint32_t box_outer, int swizzle_bytes) {
  std::call_once(g_once, resolve);
  if (injected_failure()) return B2C_E_CUDA;
  if (!g_tiled) {
    set_last_cuda_error((int)CUDA_ERROR_NOT_FOUND);
    return B2C_E_CUDA;
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return B2C_E_CUDA;
  }
  return B2C_OK;
}

// NHWC activation tensor with C_pad channels seen as a 4-D tensor {C, W, H, N}.  The bounding box
// of window origins runs from -pad to (extent - 1) + pad - dil*(kernel - 1) on W and H; the
// traversal strides are the convolution strides, so that `pixels_per_column` consecutive output
// pixels (q fastest, then p, then n) are fetched by one copy, and the per-tap displacement
// (s*dil_w, r*dil_h) is given with each copy.
int encode_im2col_nhwc(CUtensorMap* map, const void* base, int C_pad, int W, int H, int N, int pad_w, int pad_h,
                       int S, int R, int dil_w, int dil_h, int stride_w, int stride_h, int channels_per_pixel,
                       int pixels_per_column, int swizzle_bytes) {
  std::call_once(g_once, resolve);
  if (injected_failure()) return B2C_E_CUDA;
  if (!g_im2col) {
    set_last_cuda_error((int)CUDA_ERROR_NOT_FOUND);
    return B2C_E_CUDA;
  }
  cuuint64_t dims[4] = {(cuuint64_t)C_pad, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C_pad, (cuuint64_t)C_pad * W, (cuuint64_t)C_pad * W * H};
  int lower[2] = {-pad_w, -pad_h};
  int upper[2] = {pad_w - (S - 1) * dil_w, pad_h - (R - 1) * dil_h};
  cuuint32_t estr[4] = {1, (cuuint32_t)stride_w, (cuuint32_t)stride_h, 1};
  CUresult r = g_im2col(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, lower, upper,
                        (cuuint32_t)channels_per_pixel, (cuuint32_t)pixels_per_column, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return B2C_E_CUDA;
  }
  return B2C_OK;
}

// NHWC activation tensor with C_pad channels seen as a 4-D tensor {C, W, H, N} in tiled mode: one
// copy fetches `box_c` channel bytes of `box_w` consecutive pixels of one image row; pixels left or
// right of the row, rows above or below the image and images past the batch read as zeros.
int encode_tiled_nhwc_rows(CUtensorMap* map, const void* base, int C_pad, int W, int H, int N, int box_c, int box_w,
                           int swizzle_bytes, int box_h) {
  std::call_once(g_once, resolve);
  if (injected_failure()) return B2C_E_CUDA;
  if (!g_tiled) {
    set_last_cuda_error((int)CUDA_ERROR_NOT_FOUND);
    return B2C_E_CUDA;
  }
  cuuint64_t dims[4] = {(cuuint64_t)C_pad, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C_pad, (cuuint64_t)C_pad * W, (cuuint64_t)C_pad * W * H};
  cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = g_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_of(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return B2C_E_CUDA;
  }
  return B2C_OK;
}

// NCHW int8 activation tensor seen as a 4-D tensor {W, H, C, N} in tiled mode without swizzle: one copy
// fetches box_w bytes of box_h rows of all C channels of one image; columns left or right of the
// image, rows above or below it and images past the batch read as zeros.  W must be a multiple of 16.
int encode_tiled_nchw_window(CUtensorMap* map, const void* base, int W, int H, int C, int N, int box_w, int box_h) {
  std::call_once(g_once, resolve);
  if (injected_failure()) return B2C_E_CUDA;
  if (!g_tiled) {
    set_last_cuda_error((int)CUDA_ERROR_NOT_FOUND);
    return B2C_E_CUDA;
  }
  cuuint64_t dims[4] = {(cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)C, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)W, (cuuint64_t)W * H, (cuuint64_t)W * H * C};
  cuuint32_t box[4] = {(cuuint32_t)box_w, (cuuint32_t)box_h, (cuuint32_t)C, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = g_tiled(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error((int)r);
    return B2C_E_CUDA;
  }
  return B2C_OK;
}

}  // namespace b2c

extern "C" int b2c_last_cuda_error(void) { return b2c::get_last_cuda_error(); }

extern "C" int b2c_test_fail_nth_encode(int n) {
  if (n < 0) return B2C_E_INVALID_ARG;
  b2c::g_fail_countdown.store(n);
  return B2C_OK;
}
