// Issue-rate measurement of the intrinsic itself: tcgen05.mma.kind::i8 (M = 128, N = tile_n, K = 32)
// issued back to back by one thread per block on operands that already sit in shared memory, one
// block per SM.  No loads, no epilogue: what is timed is the tensor pipe alone, which gives the
// second denominator of the roofline (the first is twice the measured bf16 GEMM throughput).
// Section 5.1's GEMM core is the unit whose utilisation the paper reasons about; this is the
// measurement of that unit's peak on the device at hand.
#include <algorithm>

#include "conv_mma_common.cuh"

namespace b2c {

namespace {

constexpr int kRateThreads = 64;

__global__ void __launch_bounds__(kRateThreads, 1) mma_rate_kernel(int tile_n, int tmem_cols, int blocks_of_four,
                                                                   unsigned long long* cycles, int* status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedCtl ctl;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t a_base = smem_base, b_base = smem_base + kTileM * 128;
  // operands: zeros (any bytes would do; the products are never read back)
  uint8_t* p = smem_raw + (smem_base - smem_u32(smem_raw));
  for (int i = threadIdx.x * 16; i < (kTileM + tile_n) * 128; i += kRateThreads * 16)
    *reinterpret_cast<uint4*>(p + i) = make_uint4(0, 0, 0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctl.full[0]), 1);
    ctl.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = __shfl_sync(0xffffffffu, ctl.tmem_base, 0);
  if (warp == 0) {
    const uint32_t idesc = make_idesc_i8(tile_n);
    const uint64_t adesc = make_smem_desc(a_base, 128), bdesc = make_smem_desc(b_base, 128);
    const uint32_t leader = elect_one() ? 1u : 0u;
    const long long t0 = clock64();
    for (int i = 0; i < blocks_of_four; ++i) mma_i8_block(tmem_acc, adesc, bdesc, idesc, i ? 1u : 0u, leader, 4);
    mma_commit(smem_u32(&ctl.full[0]), leader);
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&ctl.full[0]), 0u, &ctl, status));
    const long long t1 = clock64();
    if (lane == 0) cycles[blockIdx.x] = ok ? (unsigned long long)(t1 - t0) : 0ull;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

}  // namespace b2c

extern "C" int b2c_measure_mma_rate(int tile_n, int mmas_per_block, float* device_us, float* cycles_per_mma, void* cuda_stream) {
  using namespace b2c;
  if (!device_us || !cycles_per_mma || mmas_per_block < 4 || mmas_per_block > (1 << 22)) return B2C_E_INVALID_ARG;
  if (tile_n != 16 && tile_n != 32 && tile_n != 64 && tile_n != 128 && tile_n != 256) return B2C_E_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int tmem_cols = 32;
  while (tmem_cols < tile_n) tmem_cols <<= 1;
  const int blocks = kNumSMs;
  unsigned long long* cyc = nullptr;
  int* status = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  auto fail = [&](cudaError_t e) {
    set_last_cuda_error((int)e);
    cudaFree(cyc);
    cudaFree(status);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    return B2C_E_CUDA;
  };
  cudaError_t e = cudaMalloc(&cyc, blocks * sizeof(unsigned long long));
  if (e == cudaSuccess) e = cudaMalloc(&status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  if (e != cudaSuccess) return fail(e);
  // more than half of the shared memory per block: exactly one block per SM
  const size_t smem = 120 * 1024;
  static std::atomic<unsigned long long> configured{0};
  e = set_max_dynamic_smem_once(configured, (const void*)mma_rate_kernel, 200 * 1024);
  if (e != cudaSuccess) return fail(e);
  const int fours = mmas_per_block / 4;
  for (int rep = 0; rep < 2 && e == cudaSuccess; ++rep) {  // the first launch warms up
    e = cudaEventRecord(e0, st);
    if (e == cudaSuccess) {
      mma_rate_kernel<<<blocks, kRateThreads, smem, st>>>(tile_n, tmem_cols, fours, cyc, status);
      e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
  }
  if (e != cudaSuccess) return fail(e);
  float ms = 0;
  std::vector<unsigned long long> h(blocks);
  int hs = 0;
  e = cudaEventElapsedTime(&ms, e0, e1);
  if (e == cudaSuccess) e = cudaMemcpy(h.data(), cyc, blocks * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(&hs, status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail(e);
  cudaFree(cyc);
  cudaFree(status);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (hs != 0) return hs;
  std::sort(h.begin(), h.end());
  if (h[0] == 0) return B2C_E_TIMEOUT;
  *device_us = ms * 1000.0f;
  *cycles_per_mma = (float)((double)h[blocks / 2] / (double)(fours * 4));  // median over the SMs
  return B2C_OK;
}
