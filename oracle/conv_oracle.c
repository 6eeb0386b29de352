/*
 * CPU oracle for int8 2-D convolution with int32 accumulation and shift/clip requantisation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement of what
 * the GPU library must compute.  It shares no code with the CUDA path and must never be called
 * from the product path; only the tests, the smoke check and the CPU-baseline leg of the
 * benchmark may load it.
 *
 * What it follows in the paper (Rieber et al., "Joint Program and Layout Transformations to
 * enable Convolutional Operators on Specialized Hardware based on Constraint Programming"):
 *   - Section 5.1 (Experimental Setup): the GEMM core multiplies 8-bit operands and accumulates
 *     in 32 bits, computes C_xy += A_xz * B_zy^T, and is followed by a vector unit that does
 *     the quantisation; tensors are NCHW.
 *   - Figure 5, step 1: the baseline conv2d is the seven-loop nest over n, oc, oh, ow, ic, kh, kw.
 *   - Table 2: the stencil access function is [n, i + k], i.e. cross-correlation (no kernel flip).
 *   - Section 4.2.4 (Padding): padded positions hold zeros.
 *   - Section 5 (Validation Experiments): all values are integers, so every association order
 *     of the sum gives the same result; there is exactly one correct output tensor.
 *
 * Readings taken where the paper is silent: symmetric zero padding, floor output-extent
 * formula, dilation multiplies the tap offset, requantisation is floor(acc / 2^shift) clipped
 * to [-128, 127] with no rounding offset, accumulators outside int32 are an error (neither
 * wrap nor saturate).
 *
 * All parity pins for these functions live in tests/test_oracle_pins.py; nothing here is
 * "parity unpinned".
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Output extent of one spatial axis: floor((in + 2*pad - dil*(k-1) - 1) / stride) + 1, or 0
 * when the dilated kernel does not fit.  (Paper silent; standard floor reading.) */
int oracle_out_extent(int in, int k, int stride, int pad, int dil) {
  int span = in + 2 * pad - dil * (k - 1) - 1;
  if (span < 0) return 0;
  return span / stride + 1;
}

/* floor(acc / 2^shift) clipped to int8.  Written with explicit floor division so it does not
 * depend on the implementation-defined behaviour of >> on negative values.
 * (Section 5.1: "quantization operations" after the 32-bit accumulation.) */
int8_t oracle_requant(int64_t acc, int shift) {
  int64_t d = (int64_t)1 << shift;
  int64_t q = acc / d;               /* C division truncates toward zero */
  if ((acc % d) != 0 && acc < 0) q -= 1;
  if (q < -128) q = -128;
  if (q > 127) q = 127;
  return (int8_t)q;
}

/*
 * The definition (Figure 5 step 1; Table 2 access [n, i + k]), followed by the vector unit's
 * "activation and quantization operations" (Section 5.1, which also describes the micro-benchmark that runs
 * pack -> conv -> activation -> unpack).  The paper does not say which activation; the reading
 * taken here is an optional per-output-channel int32 bias and an optional ReLU, both applied to
 * the exact sum before the outputs are written:
 *   t = acc + bias[k]   (bias == NULL: t = acc);   relu != 0: t = max(t, 0);
 *   y32 = t;   y8 = clip(floor(t / 2^shift)).
 * t outside the int32 range is reported like an accumulator overflow.
 *
 * Grouped convolution (Section 6.1 names depth-wise convolutions as the same low-channel problem):
 * with `groups` > 1 the input channels and the filters are cut into that many equal groups, filter
 * k (of group k / (K/groups)) has C/groups channels, w is [K][C/groups][R][S], and output channel k
 * sums over the input channels of its own group only; groups = C = K is the depth-wise case.
 *
 * The convolution itself:
 *   y[n][k][p][q] = sum_{c,r,s} x[n][c][p*stride_h - pad_h + r*dil_h][q*stride_w - pad_w + s*dil_w]
 *                               * w[k][c][r][s]        (terms outside the image are zero)
 * x is NCHW, w is KCRS, y32/y8 are NKPQ; either output pointer may be NULL.
 * Returns 0, or 1 if some accumulator left the int32 range (outputs then undefined there).
 * `threads` > 0 sets the OpenMP team size used over the (n, k) loops; <= 0 keeps the default.
 */
int oracle_conv2d_int8_grouped(const int8_t* x, const int8_t* w, const int32_t* bias, int relu, int groups,
                               int N, int C, int H, int W, int K, int R, int S,
                               int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                               int shift, int32_t* y32, int8_t* y8, int threads) {
  const int P = oracle_out_extent(H, R, stride_h, pad_h, dil_h);
  const int Q = oracle_out_extent(W, S, stride_w, pad_w, dil_w);
  const int Cg = C / groups, Kg = K / groups; /* channels per group; the caller checks divisibility */
  int overflow = 0;
#ifdef _OPENMP
  if (threads > 0) omp_set_num_threads(threads);
#else
  (void)threads;
#endif
#pragma omp parallel for collapse(2) schedule(static) reduction(| : overflow)
  for (int n = 0; n < N; ++n) {
    for (int k = 0; k < K; ++k) {
      for (int p = 0; p < P; ++p) {
        for (int q = 0; q < Q; ++q) {
          int64_t acc = 0;
          const int c0 = (k / Kg) * Cg; /* first input channel of output channel k's group */
          for (int c = 0; c < Cg; ++c) {
            for (int r = 0; r < R; ++r) {
              for (int s = 0; s < S; ++s) {
                int h = p * stride_h - pad_h + r * dil_h;
                int ww = q * stride_w - pad_w + s * dil_w;
                if (h >= 0 && h < H && ww >= 0 && ww < W) {
                  int xv = x[(((size_t)n * C + c0 + c) * H + h) * W + ww];
                  int wv = w[(((size_t)k * Cg + c) * R + r) * S + s];
                  acc += (int64_t)(xv * wv);
                }
              }
            }
          }
          if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
          if (bias) acc += (int64_t)bias[k];
          if (relu && acc < 0) acc = 0;
          if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
          size_t o = (((size_t)n * K + k) * P + p) * Q + q;
          if (y32) y32[o] = (int32_t)acc;
          if (y8) y8[o] = oracle_requant(acc, shift);
        }
      }
    }
  }
  return overflow;
}

/* Dense convolution (one group) with the activation step. */
int oracle_conv2d_int8_act(const int8_t* x, const int8_t* w, const int32_t* bias, int relu,
                           int N, int C, int H, int W, int K, int R, int S,
                           int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                           int shift, int32_t* y32, int8_t* y8, int threads) {
  return oracle_conv2d_int8_grouped(x, w, bias, relu, 1, N, C, H, W, K, R, S, stride_h, stride_w, pad_h, pad_w, dil_h,
                                    dil_w, shift, y32, y8, threads);
}

/* The convolution with the plain quantisation step only (no bias, no ReLU). */
int oracle_conv2d_int8(const int8_t* x, const int8_t* w,
                       int N, int C, int H, int W, int K, int R, int S,
                       int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                       int shift, int32_t* y32, int8_t* y8, int threads) {
  return oracle_conv2d_int8_act(x, w, NULL, 0, N, C, H, W, K, R, S, stride_h, stride_w, pad_h, pad_w, dil_h, dil_w,
                                shift, y32, y8, threads);
}

/*
 * Stencil unroll (Table 2, rule 1): data layout [N, I] => [N, I, K], access [n, i + k] => [n, i, k].
 * Writes the explicit matrix A[(n,p,q)][(c,r,s)] with row length C*R*S, zeros where the tap
 * falls outside the image.  This is the "im2col" the paper names as the popular alternative
 * strategy (Section 6.2).
 */
void oracle_im2col(const int8_t* x, int N, int C, int H, int W, int R, int S,
                   int stride_h, int stride_w, int pad_h, int pad_w, int dil_h, int dil_w,
                   int8_t* A) {
  const int P = oracle_out_extent(H, R, stride_h, pad_h, dil_h);
  const int Q = oracle_out_extent(W, S, stride_w, pad_w, dil_w);
  const size_t Kg = (size_t)C * R * S;
  for (int n = 0; n < N; ++n)
    for (int p = 0; p < P; ++p)
      for (int q = 0; q < Q; ++q) {
        int8_t* row = A + (((size_t)n * P + p) * Q + q) * Kg;
        for (int c = 0; c < C; ++c)
          for (int r = 0; r < R; ++r)
            for (int s = 0; s < S; ++s) {
              int h = p * stride_h - pad_h + r * dil_h;
              int ww = q * stride_w - pad_w + s * dil_w;
              int8_t v = 0;
              if (h >= 0 && h < H && ww >= 0 && ww < W) v = x[(((size_t)n * C + c) * H + h) * W + ww];
              row[((size_t)c * R + r) * S + s] = v;
            }
      }
}

/* The intrinsic of Section 5.1 written out for whole matrices: D[m][j] = sum_z A[m][z] * B[j][z]
 * (B is held transposed, reduction index contiguous in both operands).  int64 result so the
 * caller can range-check. */
void oracle_gemm_abt(const int8_t* A, const int8_t* B, int64_t M, int64_t Nn, int64_t Kg, int64_t* D) {
  for (int64_t m = 0; m < M; ++m)
    for (int64_t j = 0; j < Nn; ++j) {
      int64_t acc = 0;
      for (int64_t z = 0; z < Kg; ++z) acc += (int64_t)((int)A[m * Kg + z] * (int)B[j * Kg + z]);
      D[m * Nn + j] = acc;
    }
}

/* Pad + Reorder (Table 2, rules 2 and 4) for the activation tensor: NCHW => NHWC with the
 * channel axis zero-padded to C_pad. */
void oracle_pack_nhwc_cpad(const int8_t* x, int N, int C, int H, int W, int C_pad, int8_t* out) {
  for (int n = 0; n < N; ++n)
    for (int h = 0; h < H; ++h)
      for (int ww = 0; ww < W; ++ww)
        for (int c = 0; c < C_pad; ++c) {
          int8_t v = 0;
          if (c < C) v = x[(((size_t)n * C + c) * H + h) * W + ww];
          out[(((size_t)n * H + h) * W + ww) * C_pad + c] = v;
        }
}
