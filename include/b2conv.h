/*
 * b2conv — int8 2-D convolution embedded into the Blackwell dense MMA intrinsic.
 *
 * C ABI of the library.  Every entry point is `extern "C"`, takes plain integers, structs of
 * integers and raw pointers, and never throws, aborts or prints.  Unless a parameter says
 * otherwise, pointers named *_dev are DEVICE pointers (global memory of the current CUDA
 * device) and must be 16-byte aligned; all other pointers are HOST pointers.  `cuda_stream`
 * is a `cudaStream_t` passed as `void*` (NULL = the legacy default stream).
 *
 * The operation follows Rieber, Acosta, Froening, "Joint Program and Layout Transformations to
 * enable Convolutional Operators on Specialized Hardware based on Constraint Programming"
 * (2021): a convolution is executed on a fixed matrix-multiply intrinsic (Section 5.1: 8-bit
 * operands, 32-bit accumulation, C_xy += A_xz * B_zy^T, followed by a quantisation step) by
 * choosing which convolution axes feed the intrinsic's x/y/z dimensions and rewriting the data
 * layout to match (Table 2: stencil unroll, image pack, pad, split, reorder, fuse).  Here the
 * intrinsic is `tcgen05.mma.kind::i8` (M = 128 rows, N = 16..256 columns, K = 32 per
 * instruction, int32 accumulators in tensor memory).
 *
 * All calls return 0 (B2C_OK) or a negative B2C_E_* code.
 */
#ifndef B2CONV_H_
#define B2CONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes --------------------------------------------------------------------------- */
#define B2C_OK 0
#define B2C_E_INVALID_ARG (-1)         /* null pointer, misaligned pointer, value out of range   */
#define B2C_E_UNSUPPORTED (-2)         /* valid request this library does not execute            */
#define B2C_E_WORKSPACE_TOO_SMALL (-3) /* fixed-size scratch cannot hold this problem            */
#define B2C_E_CUDA (-4)                /* a CUDA runtime/driver call failed; see b2c_last_cuda_error */
#define B2C_E_TIMEOUT (-5)             /* a bounded device-side wait expired (device status word) */
#define B2C_E_NOT_READY (-6)           /* plan has no weights yet                                */
#define B2C_E_BOUNDS (-7)              /* debug build only: a kernel computed an address outside its tensor (device status word) */

/* ---- problem description -------------------------------------------------------------------- */
/* Convolution y[n][k][p][q] = sum_{c,r,s} x[n][c][p*stride_h - pad_h + r*dil_h][q*stride_w - pad_w + s*dil_w] * w[k][c][r][s]
 * (Figure 5 step 1 and the access function [n, i + k] of Table 2: cross-correlation, zero
 * padding per Section 4.2.4), int8 operands, exact int32 sums (Section 5.1).
 * P = floor((H + 2*pad_h - dil_h*(R-1) - 1)/stride_h) + 1, Q likewise. */
typedef struct {
  int32_t N, C, H, W; /* input: batch, channels, height, width (all >= 1)                        */
  int32_t K, R, S;    /* weights: output channels, kernel height, kernel width (all >= 1)        */
  int32_t stride_h, stride_w; /* >= 1                                                            */
  int32_t pad_h, pad_w;       /* >= 0, zeros on both sides                                       */
  int32_t dil_h, dil_w;       /* >= 1                                                            */
  int32_t shift;      /* 0..31: int8 output = clip(floor(acc / 2^shift), -128, 127)              */
  int32_t in_layout;  /* B2C_LAYOUT_NCHW or B2C_LAYOUT_NHWC; tensors are dense, no strides       */
  int32_t out_layout; /* B2C_LAYOUT_NCHW (= NKPQ) or B2C_LAYOUT_NHWC (= NPQK)                    */
  int32_t out_mode;   /* bit 0: write int32 accumulators; bit 1: write requantised int8          */
} b2c_conv_desc;

#define B2C_LAYOUT_NCHW 0
#define B2C_LAYOUT_NHWC 1
#define B2C_OUT_I32 1
#define B2C_OUT_I8 2

/* ---- embeddings ------------------------------------------------------------------------------ */
/* An embedding says which convolution axes feed the intrinsic's M / N / K dimensions and which
 * layout rewrite makes that possible (Section 5.1 for the reference map n->x, oc->y, ic->z;
 * Table 2 for the rewrites; Section 6 for the relaxed family). */
#define B2C_AXIS_NPQ 1 /* fused batch and output pixels (Fuse rule)                              */
#define B2C_AXIS_K 2   /* output channels                                                        */
#define B2C_AXIS_C 3   /* input channels, padded to the intrinsic block (Pad + Split); r, s sequential */
#define B2C_AXIS_CRS 4 /* fused (c, r, s) (Stencil Unroll + Fuse), padded to the K block         */
#define B2C_AXIS_SC 5  /* fused (s, c) padded to the K block, r sequential (partial Stencil Unroll) */
#define B2C_AXIS_C_PHASES 6 /* channels x stride phases (Image Pack of a strided conv), padded; r', s' sequential */

#define B2C_VARIANT_CP_TMA 0         /* channel pack: NHWC C-padded activations, im2col-mode TMA */
#define B2C_VARIANT_IM2COL_EXPLICIT 1 /* stencil unroll materialised as a matrix in scratch memory */
#define B2C_VARIANT_IM2COL_GATHER 2  /* stencil unroll formed in shared memory inside the conv kernel */
#define B2C_VARIANT_IM2COL_STAGED 3  /* same, from a zero-padded input window staged in shared memory (low-channel shapes) */
#define B2C_VARIANT_ROW_UNROLL 4     /* stencil unroll along the kernel row only: scratch tensor [N][H][Q][(s,c)], im2col-mode TMA over r */
#define B2C_VARIANT_SPACE_TO_DEPTH 5 /* image pack: stride phases folded into channels, then a stride-1 channel-pack conv */
#define B2C_VARIANT_DILATION_PACK 6  /* image pack of a dilated conv (Section 6.1): the dil_h*dil_w phase sub-images are fused
                                      * into the batch, convolved densely, and the epilogue interleaves the results back */

#define B2C_VARIANT_CP_SHIFT 7       /* channel pack with the stencil as operand shifts (stride 1): every tile stages the padded
                                      * image rows it needs once, tap (r, s) is the same shared-memory tile read (r*dil_h rows +
                                      * s*dil_w pixels) further on, and the packed weights stay resident in shared memory */
#define B2C_VARIANT_S2D_SHIFT 8      /* image pack (space to depth) of a strided conv, then the stride-1 remainder as operand shifts */
#define B2C_VARIANT_ROWPHASE_SHIFT 9 /* low-channel shapes: the kernel row is unrolled into channels together with the vertical
                                      * stride phases (scratch [N][P + R' - 1][Q][(dh, s, c)], R' = ceil(R / stride_h)); what remains
                                      * is an R' x 1 stride-1 convolution, executed as operand shifts over 8 x 16-pixel tiles */

#define B2C_VARIANT_IM2COL_WINDOW 10  /* low-channel shapes: stencil unroll formed in shared memory from a two-dimensional input
                                      * window that one tiled TMA copy of the NCHW tensor stages per tile of tile_h x tile_w output
                                      * pixels (zeros outside the image); builder warps write the swizzled A rows word by word,
                                      * separate epilogue warps drain the accumulators; weights resident; needs NCHW input with
                                      * rows that are multiples of 16 bytes and unit horizontal dilation */

typedef struct {
  int32_t id;       /* index in the enumeration for this descriptor; pass to b2c_plan_create      */
  int32_t map_m, map_n, map_k; /* B2C_AXIS_*                                                      */
  int32_t variant;  /* B2C_VARIANT_*                                                              */
  int32_t tile_m, tile_n; /* accumulator tile of one thread block                                */
  int32_t split_k;  /* number of thread blocks sharing one output tile's reduction                */
  int64_t o_mac;    /* MACs issued to the intrinsic minus N*K*P*Q*C*R*S (Section 4.4)             */
  int64_t o_data;   /* tensor elements moved minus (|x| + |w| + |y|) (Section 4.4)                */
  int64_t workspace_bytes; /* scratch the caller passes to run                                    */
  float device_us;  /* measured device time per run, or -1 if this candidate was not timed        */
} b2c_embedding;

#define B2C_POLICY_AUTO_TIMED (-1)   /* time the 5 lowest-overhead candidates, keep the fastest (Section 6.1) */
#define B2C_POLICY_MIN_OVERHEAD (-2) /* lowest |[o_mac, o_data] . [1, 1]| without timing (Section 4.4)        */
#define B2C_POLICY_MIN_WORKSPACE (-3) /* smallest scratch footprint (Table 4)                                 */
#define B2C_POLICY_AUTO_TIMED_CONCURRENT (-4) /* as AUTO_TIMED, but every candidate is timed as sixteen independent
                                        * runs on sixteen streams at once and the highest throughput wins: for callers
                                        * that keep several independent convolutions in flight, where a schedule
                                        * with fewer, wider tiles beats the one with the shortest single-run time */

typedef struct b2c_plan b2c_plan; /* opaque, library-owned */

/* Output extent (host only).  *P or *Q is 0 when the dilated kernel does not fit; that is
 * reported as B2C_E_UNSUPPORTED by the calls below.  INVALID_ARG on null or bad fields. */
int b2c_out_shape(const b2c_conv_desc* desc, int32_t* P, int32_t* Q);

/* Lists every legal embedding of `desc` (host only, no CUDA call), sorted by increasing
 * o_mac + o_data.  Writes at most `cap` records to `out` (may be NULL when cap == 0) and the
 * total number to *count.  UNSUPPORTED when C*R*S > 131071 (an int32 accumulator could
 * overflow) or the output is empty. */
int b2c_enumerate(const b2c_conv_desc* desc, b2c_embedding* out, int32_t cap, int32_t* count);

/* Creates a plan for `desc` on the current device.  `policy_or_id` is a B2C_POLICY_* value or
 * an embedding id from b2c_enumerate.  AUTO_TIMED (and AUTO_TIMED_CONCURRENT, with sixteen sets of
 * output and scratch buffers) allocates temporary device buffers, captures
 * each candidate's launches in a CUDA graph on a private stream, replays it and keeps the
 * fastest; it synchronises with the device and must not be called while a stream of the calling
 * thread is being captured.  `cuda_stream` is used for the buffer initialisation only.  The plan
 * owns its packed weights, lookup tables and a device status word; free it with b2c_plan_destroy. */
int b2c_plan_create(const b2c_conv_desc* desc, int32_t policy_or_id, void* cuda_stream, b2c_plan** out);

/* Grouped convolution (Section 6.1 names depth-wise convolutions as the same low-channel problem as
 * the low-channel layers, without evaluating them).  `desc` describes the whole convolution: C input
 * and K output channels, both multiples of `groups`; filter k belongs to group k / (K / groups), has
 * C / groups channels and sums over the input channels of its own group only; the weight tensor
 * given to b2c_plan_set_weights is int8 [K][C / groups][R][S]; groups == C == K is depth-wise.
 * desc.in_layout and desc.out_layout must be B2C_LAYOUT_NCHW (UNSUPPORTED otherwise; INVALID_ARG when
 * groups < 1 or does not divide C and K).  The plan runs all groups in ONE launch of the MMA kernel
 * (the group is a grid axis: every block convolves its group's channel slice of x into that
 * group's slice of y in place, with the filters of all groups packed once into one matrix; no
 * scratch: b2c_plan_workspace_bytes is 0), with a stencil unroll formed inside the kernel (the
 * staged window where it fits, else the gather); b2c_plan_info reports that embedding.
 * Narrow groups are merged: m consecutive groups (m the smallest divisor of `groups` that brings a
 * merged group to 32 output channels, within 1024 reduction elements) run as one group of m times
 * the channels with block-diagonal filters; b2c_plan_set_weights expands the filters into a buffer
 * the plan owns (zeros between the groups) before it packs them.  Results are those of the grouped
 * convolution; only the number of tiles and the idle share of each MMA change.
 * All other plan calls (set_weights, set_activation with K bias values, run, device_status, destroy)
 * apply as to any plan; the rewrite / run_rewritten halves are no-op and run respectively. */
int b2c_plan_create_grouped(const b2c_conv_desc* desc, int32_t groups, b2c_plan** out);

/* Grouped convolution with the form chosen by timing (Section 6.1's timed choice among candidates, applied
 * to the merge factor).  Two forms are built and run on scratch tensors: the in-place form of
 * b2c_plan_create_grouped, and the full merge: the dense convolution of the whole tensors with
 * block-diagonal filters (all other filter elements zero), itself chosen by B2C_POLICY_AUTO_TIMED.  The
 * full merge spends `groups` times the MACs and may need scratch (b2c_plan_workspace_bytes is then that of
 * its embedding, and run takes the workspace like any dense plan); it is considered when the expanded
 * filters [K][C][R][S] are at most 16 MB.  The faster form is returned; b2c_plan_info reports its
 * embedding with the measured device_us.  Weights, activation, run and results are as for
 * b2c_plan_create_grouped.  Allocates temporary device buffers and synchronises with the device like
 * B2C_POLICY_AUTO_TIMED; `cuda_stream` is used for buffer initialisation.  Errors as
 * b2c_plan_create_grouped; when the full merge cannot be built or timed the in-place form is returned. */
int b2c_plan_create_grouped_timed(const b2c_conv_desc* desc, int32_t groups, void* cuda_stream, b2c_plan** out);

/* Copies the chosen embedding (with device_us if it was timed) to *chosen. */
int b2c_plan_info(const b2c_plan* plan, b2c_embedding* chosen);

/* Bytes of scratch `run` needs (0 for embeddings that need none). */
int b2c_plan_workspace_bytes(const b2c_plan* plan, size_t* bytes);

/* Weight pack (Section 5.1: the B operand is held transposed, reduction index contiguous):
 * reads w_kcrs_dev (int8 [K][C][R][S], device) and writes the plan's own packed copy,
 * asynchronously on `cuda_stream`.  Call once per weight tensor, before run. */
int b2c_plan_set_weights(b2c_plan* plan, const int8_t* w_kcrs_dev, void* cuda_stream);

/* Activation step between accumulation and output (Section 5.1: the vector unit after the GEMM core
 * performs "activation and quantization"; the paper does not name the activation, the reading here
 * is bias + ReLU).  With a plan so configured every complete sum becomes
 *   t = acc + bias[k]  (bias_dev != NULL),  then  t = max(t, 0)  (relu == 1),
 * the int32 output is t and the int8 output clip(floor(t / 2^shift)).  bias_dev: K int32 values in
 * device memory (4-byte aligned), copied into the plan asynchronously on `cuda_stream`; NULL removes
 * the bias.  relu: 0 or 1.  The caller keeps acc + bias inside int32 (|acc| <= C*R*S*2^14); the
 * addition wraps otherwise.  Applies to later b2c_conv2d_int8_run / run_rewritten calls of this
 * plan; a new plan has no bias and no ReLU.  INVALID_ARG on a null plan, misaligned bias or relu
 * outside {0, 1}; B2C_E_CUDA if the copy or its buffer fails. */
int b2c_plan_set_activation(b2c_plan* plan, const int32_t* bias_dev, int relu, void* cuda_stream);

/* Enqueues the whole path on `cuda_stream` and returns without waiting: activation layout
 * rewrite (if the embedding has one), the MMA kernel with fused shift/clip epilogue, stores in
 * desc.out_layout.  x_dev: int8 input in desc.in_layout.  y_i32_dev / y_i8_dev: outputs
 * selected by desc.out_mode (a selected output must be non-null; an unselected one is ignored).
 * workspace_dev: at least b2c_plan_workspace_bytes bytes (may be NULL when that is 0); its
 * contents are scratch.  The caller owns all four buffers and must keep them alive until the
 * stream has run the work.  A plan must not be used from two threads at once. */
int b2c_conv2d_int8_run(b2c_plan* plan, const int8_t* x_dev, int32_t* y_i32_dev, int8_t* y_i8_dev,
                        void* workspace_dev, void* cuda_stream);

/* The two halves of b2c_conv2d_int8_run on their own, matching the "Transf." and "Op." columns of
 * Tables 3 to 5: b2c_plan_rewrite_activations enqueues only the layout rewrite of x into the start
 * of workspace_dev (nothing is enqueued for embeddings without a rewrite), and
 * b2c_conv2d_int8_run_rewritten enqueues only the MMA kernel, epilogue and split finish on a
 * workspace an earlier b2c_plan_rewrite_activations (or b2c_conv2d_int8_run) of the same plan filled,
 * e.g. to convolve one rewritten input again after b2c_plan_set_weights.  x_dev may be NULL in
 * run_rewritten when the plan has a rewrite; embeddings without one read x_dev there.  Same
 * argument rules, stream semantics and error codes as b2c_conv2d_int8_run. */
int b2c_plan_rewrite_activations(b2c_plan* plan, const int8_t* x_dev, void* workspace_dev, void* cuda_stream);
int b2c_conv2d_int8_run_rewritten(b2c_plan* plan, const int8_t* x_dev, int32_t* y_i32_dev, int8_t* y_i8_dev,
                                  void* workspace_dev, void* cuda_stream);

/* Memory footprint of the chosen embedding (the "Memory" columns of Tables 3 to 5): bytes of the
 * rewritten activation operand in the workspace (0 without a rewrite) and of the plan's packed
 * weights.  Host only. */
int b2c_plan_footprint(const b2c_plan* plan, size_t* rewritten_bytes, size_t* packed_weight_bytes);

/* One-shot form of the paper's problem statement: NCHW int8 input, KCRS int8 weights, NKPQ
 * outputs (either may be NULL, not both), symmetric stride / pad / dilation.  All four tensor
 * pointers are DEVICE pointers.  Keeps plans and scratch in a library-owned cache keyed by
 * (shape, output mode, device, cuda_stream): the first call for a key picks the embedding by
 * timed selection (it allocates and synchronises with the device, so make it outside any stream
 * capture); later calls only re-pack the weights and enqueue on `cuda_stream`.
 * Ordering: every call re-packs w into its cached plan's weight buffer and runs in that plan's
 * scratch.  Calls with the same key are ordered by their stream, so one call's buffers are never
 * rewritten under another; calls on different streams use different cached plans and may overlap
 * on the GPU.  Two host threads may call concurrently (the enqueue is serialised inside).
 * A bounded device wait that expired inside a one-shot call is reported by b2c_oneshot_status. */
int b2c_conv2d_int8(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int dilation,
                    int shift, const int8_t* x_dev, const int8_t* w_dev, int32_t* y_i32_dev,
                    int8_t* y_i8_dev, void* cuda_stream);

/* Device status of the one-shot cache on the current device: *status is B2C_OK, or B2C_E_TIMEOUT if a
 * kernel enqueued by b2c_conv2d_int8 / b2c_conv2d_int8_host gave up on a bounded wait since the last
 * query (the words are then cleared).  Waits for the device to be idle first. */
int b2c_oneshot_status(int32_t* status);

/* Frees every cached one-shot plan of the current device (packed weights, scratch, status words)
 * after waiting for the device to be idle.  The next one-shot call of a shape selects again. */
int b2c_oneshot_cache_clear(void);

/* Same operation with HOST tensors: copies x and w to the device, runs, copies the requested
 * outputs back and synchronises.  Convenience for callers without device memory of their own. */
int b2c_conv2d_int8_host(int N, int C, int H, int W, int K, int R, int S, int stride, int pad, int dilation,
                         int shift, const int8_t* x_host, const int8_t* w_host, int32_t* y_i32_host,
                         int8_t* y_i8_host);

/* Streaming form for HOST tensors (the micro-benchmark of Section 5.1 runs packing, convolution,
 * activation and unpacking on tensors that start and end in host memory; this is that loop with the
 * copies across the host link pipelined around the path): the plan keeps its weights, and each call enqueues, without waiting, the copy of one
 * input batch to the device, the whole path of b2c_conv2d_int8_run on it and the copy of the
 * outputs desc.out_mode selects back to the host.  The three steps run on three library-owned
 * streams chained by events over a ring of three device buffer sets, so the copy of the next input
 * and the read-back of the previous output overlap the kernels of the current call; a fourth call
 * in flight blocks the host until the oldest one has finished.  x_host: int8 input in
 * desc.in_layout; y_i32_host / y_i8_host: outputs in desc.out_layout (a selected output must be
 * non-null, an unselected one is ignored).  The caller owns the host buffers, keeps them unchanged
 * (x) and unread (y) until b2c_plan_host_sync returns, and should allocate them page-locked:
 * pageable buffers give correct results but the copies then do not overlap.  Weights, bias and
 * ReLU flag set on another stream must have completed before the first call.  The first call
 * allocates the ring and a workspace (B2C_E_CUDA if that fails; nothing is then enqueued);
 * b2c_plan_destroy frees them.  INVALID_ARG on null plan / x / selected output; NOT_READY without
 * weights.  Not to be mixed with b2c_conv2d_int8_run on the same plan while calls are in flight. */
int b2c_plan_run_host_async(b2c_plan* plan, const int8_t* x_host, int32_t* y_i32_host, int8_t* y_i8_host);

/* Blocks until every b2c_plan_run_host_async of this plan has delivered its outputs to the host
 * buffers.  B2C_OK when nothing is in flight; B2C_E_CUDA if a copy or kernel failed. */
int b2c_plan_host_sync(b2c_plan* plan);

/* Reads the plan's device status word after waiting for ALL work on the current device to finish
 * (cudaDeviceSynchronize: the plan does not know which streams its kernels were enqueued on).
 * *status is B2C_OK or B2C_E_TIMEOUT if a kernel of this plan gave up on a bounded wait; the word is
 * then cleared.  Not to be called while a stream is being captured. */
int b2c_plan_device_status(b2c_plan* plan, int32_t* status);

/* Failure-detection self-test (no counterpart in the paper): enqueues a one-block kernel that
 * waits, with the bounded wait every kernel of this library uses, on a barrier nothing completes.
 * After the wait's limit (about one second) the kernel records B2C_E_TIMEOUT in the plan's status
 * word and returns normally; b2c_plan_device_status then reports it and the plan stays usable. */
int b2c_selftest_bounded_wait(b2c_plan* plan, void* cuda_stream);

/* The same self-test for the activation-pack kernel's wait on its bulk copies (no counterpart in the
 * paper): one block waits for bytes that no copy delivers, gives up after about one second, records
 * B2C_E_TIMEOUT in the plan's status word and returns normally. */
int b2c_selftest_pack_wait(b2c_plan* plan, void* cuda_stream);

void b2c_plan_destroy(b2c_plan* plan);

/* Layout rewrites on their own (the Pad / Reorder / Stencil Unroll rules of Table 2), exposed so
 * they can be checked and timed separately.  b2c_pack_activations is asynchronous on
 * `cuda_stream` (called on its own it has no status word: a block whose bounded wait for its
 * bulk copies expires leaves its part of the output unwritten; inside a plan's run the same
 * kernel records B2C_E_TIMEOUT in the plan's status word); b2c_im2col builds a temporary lookup
 * table and synchronises the stream.
 * b2c_pack_activations: int8 NCHW [N][C][H][W] -> NHWC [N][H][W][C_pad], channels >= C zero;
 *   C_pad must be a multiple of 16 and >= C.
 * b2c_im2col: int8 input in desc.in_layout -> A[N*P*Q][K_pad], row m = (n, p, q), column
 *   (c*R + r)*S + s, zeros for taps outside the image and for columns >= C*R*S; K_pad must be a
 *   multiple of 16 and >= C*R*S. */
int b2c_pack_activations(const int8_t* x_nchw_dev, int8_t* out_dev, int N, int C, int H, int W, int C_pad,
                         void* cuda_stream);
int b2c_im2col(const b2c_conv_desc* desc, const int8_t* x_dev, int8_t* a_dev, int K_pad, void* cuda_stream);

/* b2c_im2col for callers that cannot allocate device memory (the paper has no counterpart; this
 * is a property of the library, not of the method).  b2c_im2col puts its lookup table in a
 * temporary cudaMalloc buffer; code that runs where allocation is forbidden or impossible - inside
 * a region a framework has frozen against allocation, in a latency-critical loop that must stay
 * off the allocator, or in a process that has given all device memory to another pool - can call
 * this instead.  Same arguments, same output, but the table lives in a fixed 128 KB device array
 * inside the library (held by every GPU that loads it, until the process exits) and is filled by
 * a small kernel on `cuda_stream`; the call makes no cudaMalloc / cudaFree and does not
 * synchronise.  Limits and rules:
 *   - K_pad <= 16384, else B2C_E_WORKSPACE_TOO_SMALL (nothing is launched);
 *   - the first call on a device looks up the array's device address (cudaGetSymbolAddress):
 *     make that first call outside any stream capture;
 *   - all calls on a device share the one array and each call rewrites the part it uses, so two
 *     calls whose kernels can overlap on the GPU (different streams, no ordering) race: order
 *     them on one stream or with events. */
int b2c_im2col_noalloc(const b2c_conv_desc* desc, const int8_t* x_dev, int8_t* a_dev, int K_pad, void* cuda_stream);

/* Peak of the intrinsic itself on this device (Section 5.1: the GEMM core is the unit whose
 * utilisation decides the operator time; this measures that unit alone).  Launches one block per SM
 * that issues `mmas_per_block` (a multiple of 4, at most 2^22) tcgen05.mma.kind::i8 instructions of
 * shape 128 x tile_n x 32 back to back on operands resident in shared memory, on `cuda_stream`, and
 * waits for it.  *device_us: CUDA-event time of the launch (all SMs busy), so that
 * 148 * mmas_per_block * 2*128*tile_n*32 / device_us is the device's int8 issue rate;
 * *cycles_per_mma: median over the SMs of SM clock cycles per instruction.  tile_n in
 * {16, 32, 64, 128, 256}.  Allocates a few KB and synchronises: not for use under stream capture.
 * INVALID_ARG on bad arguments, B2C_E_CUDA / B2C_E_TIMEOUT on failure. */
int b2c_measure_mma_rate(int tile_n, int mmas_per_block, float* device_us, float* cycles_per_mma, void* cuda_stream);

/* The same for the two-SM form (tcgen05.mma.cta_group::2.kind::i8, 256 x tile_n x 32 per instruction,
 * issued by the leader of each of the device's 74 block pairs; every block holds 128 rows of A and
 * tile_n / 2 rows of B and its tensor core reads the other half of B from its peer's shared memory):
 * 74 * mmas_per_pair * 2*256*tile_n*32 / device_us is the issue rate of the two-SM schedule, the
 * ceiling of the kernel that uses it.  tile_n in {64, 128, 256}; *cycles_per_mma: median over the
 * pairs.  Same allocation, synchronisation and error behaviour as b2c_measure_mma_rate. */
int b2c_measure_mma_rate_pair(int tile_n, int mmas_per_pair, float* device_us, float* cycles_per_mma, void* cuda_stream);

/* ---- debug build (no counterpart in the paper) ---------------------------------------------------
 * libb2conv_debug.so is the same library compiled with -DB2C_DEBUG_BOUNDS.  In it every address a
 * kernel computes by hand (loads of x, stores and atomics to the outputs and to the scratch; TMA
 * copies are clipped by their tensor maps and need no check) is tested against the range of its
 * tensor; the first access outside records B2C_E_BOUNDS, a site number and the byte offset from the
 * range start in the plan's device status words and is skipped, later ones are only skipped.  The
 * workspace gains a 64-byte guard band on either side (b2c_plan_workspace_bytes includes them; run
 * repaints them and uses the middle).  It stands in for a memory checker where none can be run.
 * b2c_debug_build: 1 in that library, 0 in the release one.
 * b2c_plan_debug_info: site and byte offset of the report b2c_plan_device_status last returned.
 * b2c_plan_check_canaries: waits for the device, reads the guard bands of `workspace_dev` (the
 *   pointer given to run) and sets *intact to 0 if a byte changed; UNSUPPORTED in the release build.
 * b2c_test_shrink_checked_ranges: test hook; every checked range is declared `bytes` shorter than it
 *   is, so that in-range accesses near a tensor's end are reported and skipped (nothing out of range
 *   is ever touched); 0 restores.  No effect in the release build. */
int b2c_debug_build(void);
int b2c_plan_debug_info(const b2c_plan* plan, int32_t* site, int64_t* byte_offset);
int b2c_plan_check_canaries(b2c_plan* plan, const void* workspace_dev, int32_t* intact);
int b2c_test_shrink_checked_ranges(long long bytes);

/* Host-side fault injection for tests (no counterpart in the paper): the n-th tensor-map encode
 * from now on, counted over all threads, fails as if the driver had refused it (the call that
 * needed it returns B2C_E_CUDA); n = 0 disarms.  Nothing on the device is touched. */
int b2c_test_fail_nth_encode(int n);

const char* b2c_status_string(int status);

/* The last CUDA error code (cudaError_t or CUresult as int) seen by this thread's failing call. */
int b2c_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* B2CONV_H_ */
