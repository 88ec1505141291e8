// Developer microbenchmark: cycles per tcgen05.mma (TF32, M = 128) as a function of N, with A in
// tensor memory or shared memory.  One block; operands are whatever the memories hold.
#include "../../include/swila.h"
#include "swila_umma.cuh"

namespace {
using namespace swila::umma;

template <int N, bool A_TMEM>
__global__ void __launch_bounds__(128) umma_rate_kernel(int reps, long long *cycles) {
  extern __shared__ __align__(128) float sm[];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  if (warp == 0) tmem_alloc(&tmem_base_s, 512);
  if (tid == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
  for (int i = tid; i < 16384; i += 128) sm[i] = 1.0f;
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tb = tmem_base_s;
  if (tid == 0) {
    constexpr uint32_t id = idesc_tf32(128, N);
    const uint64_t b0 = smem_desc_kmajor(smem_u32(sm), N * 16, 128);
    const uint64_t a0 = smem_desc_kmajor(smem_u32(sm) + 32768, 128 * 16, 128);
    const long long t0 = clock64();
    for (int r = 0; r < reps; ++r) {
      // 4 independent accumulators, 16-deep K loop each round
#pragma unroll 1
      for (int ks = 0; ks < 16; ++ks) {
        const int acc = ks & 3;
        if (A_TMEM) mma_tf32_ts(tb + 256 + acc * 64, tb + ks * 8, b0 + (uint64_t)(ks * 2 * N), id, true);
        else mma_tf32_ss(tb + 256 + acc * 64, a0 + (uint64_t)(ks * 2 * 128), b0 + (uint64_t)(ks * 2 * N), id, true);
      }
    }
    mma_commit(&bar);
    const bool ok = mbar_wait(&bar, 0);
    const long long t1 = clock64();
    cycles[0] = ok ? (t1 - t0) : -1;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tb, 512);
}
}  // namespace

extern "C" int swila_bench_tf32_mma_rate(int N, int a_in_tmem, int reps, long long *cycles_dev, void *stream) {
  cudaStream_t st = (cudaStream_t)stream;
  const int smem = 131072;
#define RUN(NN, AT)                                                                                        \
  {                                                                                                        \
    cudaFuncSetAttribute(umma_rate_kernel<NN, AT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);     \
    umma_rate_kernel<NN, AT><<<1, 128, smem, st>>>(reps, cycles_dev);                                     \
  }
  if (a_in_tmem) {
    if (N == 16) RUN(16, true) else if (N == 32) RUN(32, true) else if (N == 64) RUN(64, true)
    else if (N == 128) RUN(128, true) else if (N == 256) RUN(256, true) else return SWILA_ERR_UNSUPPORTED;
  } else {
    if (N == 16) RUN(16, false) else if (N == 32) RUN(32, false) else if (N == 64) RUN(64, false)
    else if (N == 128) RUN(128, false) else if (N == 256) RUN(256, false) else return SWILA_ERR_UNSUPPORTED;
  }
  return cudaGetLastError() == cudaSuccess ? SWILA_OK : SWILA_ERR_CUDA;
}
