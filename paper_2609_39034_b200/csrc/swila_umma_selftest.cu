// Self-test of the tcgen05 plumbing used by the chunked kernel: D[128 x N] = A[128 x K] * B[N x K]^T
// in TF32 with A placed in tensor memory by the threads, B in shared memory (K-major, no
// swizzle), the result read back from tensor memory.  One block of 128 threads.
#include "../../include/swila_dev.h"
#include "swila_umma.cuh"

namespace {
using namespace swila::umma;

template <int N, int K>
__global__ void __launch_bounds__(128) umma_selftest_kernel(const float *A, const float *B, float *D, int *status) {
  __shared__ __align__(128) float sB[N * K];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  constexpr uint32_t TM_COLS = 256;  // A: K columns at 0, D: N columns at 128

  if (warp == 0) tmem_alloc(&tmem_base_s, TM_COLS);
  if (tid == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  // B [N][K] -> shared, K-major tile: 16-byte unit (row n, k-chunk c) at (c*N + n)*16
  for (int i = tid; i < N * (K / 4); i += 128) {
    const int n = i % N, c = i / N;
    const float4 v = *reinterpret_cast<const float4 *>(B + (size_t)n * K + c * 4);
    *reinterpret_cast<float4 *>(sB + (size_t)(c * N + n) * 4) = v;
  }
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tbase = tmem_base_s;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;

  // A row `tid` -> TMEM lane tid, columns 0..K-1
#pragma unroll
  for (int c = 0; c < K / 16; ++c) {
    float v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = A[(size_t)tid * K + c * 16 + i];
    tmem_st16(tbase + lane_base + c * 16, v);
  }
  tmem_st_wait();
  tc_fence_before_sync();
  __syncthreads();

  if (tid == 0) {
    tc_fence_after_sync();
    constexpr uint32_t idesc = idesc_tf32(128, N);
#pragma unroll
    for (int ks = 0; ks < K / 8; ++ks) {
      const uint64_t bdesc = smem_desc_kmajor(smem_u32(sB) + ks * 2 * (N * 16), N * 16, 128);
      mma_tf32_ts(tbase + 128, tbase + ks * 8, bdesc, idesc, ks > 0);
    }
    mma_commit(&bar);
  }
  const bool ok = mbar_wait(&bar, 0);
  tc_fence_after_sync();
  if (ok) {
#pragma unroll
    for (int c = 0; c < N / 16; ++c) {
      float v[16];
      tmem_ld16(tbase + lane_base + 128 + c * 16, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) D[(size_t)tid * N + c * 16 + i] = v[i];
    }
  } else if (tid == 0) {
    *status = 1;  // the MMA never signalled completion
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tbase, TM_COLS);
}

// round-to-nearest-even bf16 bits of an fp32 value (finite inputs)
__device__ __forceinline__ uint32_t bf16_bits(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

// Same product with BF16 operands (K = 16 per instruction).  AMODE 0: A from tensor memory, two K
// elements per 32-bit column; AMODE 1: A from shared memory in the same K-major layout as B (16-byte
// unit = 8 elements).
template <int N, int K, int AMODE>
__global__ void __launch_bounds__(128) umma_selftest_bf16_kernel(const float *A, const float *B, float *D, int *status) {
  __shared__ __align__(128) uint16_t sB[N * K];
  __shared__ __align__(128) uint16_t sA[AMODE ? 128 * K : 8];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  constexpr uint32_t TM_COLS = 256;  // A: K/2 columns at 0, D: N columns at 128

  if (warp == 0) tmem_alloc(&tmem_base_s, TM_COLS);
  if (tid == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  // B [N][K] -> shared, K-major tile: 16-byte unit (row n, k-chunk c of 8 elements) at (c*N + n)*16
  for (int i = tid; i < N * K; i += 128) {
    const int n = i / K, k = i % K;
    sB[((k / 8) * N + n) * 8 + (k % 8)] = (uint16_t)bf16_bits(B[(size_t)n * K + k]);
  }
  if (AMODE) {
    for (int i = tid; i < 128 * K; i += 128) {
      const int m = i / K, k = i % K;
      sA[((k / 8) * 128 + m) * 8 + (k % 8)] = (uint16_t)bf16_bits(A[(size_t)m * K + k]);
    }
  }
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tbase = tmem_base_s;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;

  if (!AMODE) {  // A row `tid` -> TMEM lane tid, columns 0..K/2-1
#pragma unroll
    for (int c = 0; c < K / 8; ++c) {
      uint32_t v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i)
        v[i] = bf16_bits(A[(size_t)tid * K + c * 8 + 2 * i]) | (bf16_bits(A[(size_t)tid * K + c * 8 + 2 * i + 1]) << 16);
      tmem_st4(tbase + lane_base + c * 4, v);
    }
    tmem_st_wait();
  }
  tc_fence_before_sync();
  __syncthreads();

  if (tid == 0) {
    tc_fence_after_sync();
    constexpr uint32_t idesc = idesc_bf16(128, N);
#pragma unroll
    for (int ks = 0; ks < K / 16; ++ks) {
      const uint64_t bdesc = smem_desc_kmajor(smem_u32(sB) + ks * 2 * (N * 16), N * 16, 128);
      if (AMODE) {
        const uint64_t adesc = smem_desc_kmajor(smem_u32(sA) + ks * 2 * (128 * 16), 128 * 16, 128);
        mma_bf16_ss(tbase + 128, adesc, bdesc, idesc, ks > 0);
      } else {
        mma_bf16_ts(tbase + 128, tbase + ks * 8, bdesc, idesc, ks > 0);
      }
    }
    mma_commit(&bar);
  }
  const bool ok = mbar_wait(&bar, 0);
  tc_fence_after_sync();
  if (ok) {
#pragma unroll
    for (int c = 0; c < N / 16; ++c) {
      float v[16];
      tmem_ld16(tbase + lane_base + 128 + c * 16, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) D[(size_t)tid * N + c * 16 + i] = v[i];
    }
  } else if (tid == 0) {
    *status = 1;  // the MMA never signalled completion
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tbase, TM_COLS);
}

// Both operands in shared memory in the 128-byte-swizzle K-major layout (K = 64 per tile): D[128 x N] = A B^T.
template <int N>
__global__ void __launch_bounds__(128) umma_selftest_sw128_kernel(const float *A, const float *B, float *D, int *status) {
  constexpr int K = 64;
  __shared__ __align__(1024) uint16_t sA[128 * K];
  __shared__ __align__(1024) uint16_t sB[N * K];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  constexpr uint32_t TM_COLS = 256;

  if (warp == 0) tmem_alloc(&tmem_base_s, TM_COLS);
  if (tid == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  // element (row, k) -> row*64 + ((k/8) ^ (row & 7))*8 + k%8
  for (int i = tid; i < N * K; i += 128) {
    const int n = i / K, k = i % K;
    sB[n * K + (((k >> 3) ^ (n & 7)) << 3) + (k & 7)] = (uint16_t)bf16_bits(B[(size_t)n * K + k]);
  }
  for (int i = tid; i < 128 * K; i += 128) {
    const int m = i / K, k = i % K;
    sA[m * K + (((k >> 3) ^ (m & 7)) << 3) + (k & 7)] = (uint16_t)bf16_bits(A[(size_t)m * K + k]);
  }
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tbase = tmem_base_s;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  if (tid == 0) {
    constexpr uint32_t idesc = idesc_bf16(128, N);
#pragma unroll
    for (int ks = 0; ks < K / 16; ++ks)
      mma_bf16_ss(tbase + 128, smem_desc_sw128(smem_u32(sA) + ks * 32, 1024), smem_desc_sw128(smem_u32(sB) + ks * 32, 1024),
                  idesc, ks > 0);
    mma_commit(&bar);
  }
  const bool ok = mbar_wait(&bar, 0);
  tc_fence_after_sync();
  if (ok) {
#pragma unroll
    for (int c = 0; c < N / 16; ++c) {
      float v[16];
      tmem_ld16(tbase + lane_base + 128 + c * 16, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) D[(size_t)tid * N + c * 16 + i] = v[i];
    }
  } else if (tid == 0) {
    *status = 1;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tbase, TM_COLS);
}

// A through tensor memory (two K elements per column), B [N = 128][K = 32] stored MN-major with the 128-byte
// swizzle: rows = K index, 128 bytes = 64 consecutive N per row, two blocks of 64 N.
__global__ void __launch_bounds__(128) umma_selftest_bmn_kernel(const float *A, const float *B, float *D, int *status) {
  constexpr int N = 128, K = 32, BLOCK = K * 128;  // bytes of one block of 64 N
  __shared__ __align__(1024) unsigned char sB[2 * BLOCK];
  __shared__ __align__(8) uint64_t bar;
  __shared__ uint32_t tmem_base_s;
  const int tid = threadIdx.x, warp = tid >> 5;
  constexpr uint32_t TM_COLS = 256;

  if (warp == 0) tmem_alloc(&tmem_base_s, TM_COLS);
  if (tid == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  for (int i = tid; i < N * K; i += 128) {
    const int n = i / K, k = i % K;
    const int off = (n >> 6) * BLOCK + k * 128 + ((((n & 63) >> 3) ^ (k & 7)) << 4) + (n & 7) * 2;
    *reinterpret_cast<uint16_t *>(sB + off) = (uint16_t)bf16_bits(B[(size_t)n * K + k]);
  }
  fence_async_smem();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tbase = tmem_base_s;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
#pragma unroll
  for (int c = 0; c < K / 8; ++c) {
    uint32_t v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      v[i] = bf16_bits(A[(size_t)tid * K + c * 8 + 2 * i]) | (bf16_bits(A[(size_t)tid * K + c * 8 + 2 * i + 1]) << 16);
    tmem_st4(tbase + lane_base + c * 4, v);
  }
  tmem_st_wait();
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0) {
    tc_fence_after_sync();
    constexpr uint32_t idesc = idesc_bf16_bmn(128, N);
#pragma unroll
    for (int ks = 0; ks < K / 16; ++ks) {  // 16 K indices = 16 rows of 128 bytes
      const uint64_t bdesc = smem_desc_sw128_mn(smem_u32(sB) + ks * 16 * 128, BLOCK, 1024);
      mma_bf16_ts(tbase + 128, tbase + ks * 8, bdesc, idesc, ks > 0);
    }
    mma_commit(&bar);
  }
  const bool ok = mbar_wait(&bar, 0);
  tc_fence_after_sync();
  if (ok) {
#pragma unroll
    for (int c = 0; c < N / 16; ++c) {
      float v[16];
      tmem_ld16(tbase + lane_base + 128 + c * 16, v);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) D[(size_t)tid * N + c * 16 + i] = v[i];
    }
  } else if (tid == 0) {
    *status = 1;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tbase, TM_COLS);
}
}  // namespace

extern "C" int swila_selftest_tf32_mma(const float *A, const float *B, float *D, int N, int K, int *status,
                                       void *stream) {
  if (!A || !B || !D || !status) return SWILA_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (N == 32 && K == 32) umma_selftest_kernel<32, 32><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 128 && K == 32) umma_selftest_kernel<128, 32><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 32 && K == 128) umma_selftest_kernel<32, 128><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 64 && K == 128) umma_selftest_kernel<64, 128><<<1, 128, 0, st>>>(A, B, D, status);
  else return SWILA_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? SWILA_OK : SWILA_ERR_CUDA;
}

extern "C" int swila_selftest_bf16_mma(const float *A, const float *B, float *D, int N, int K, int a_in_smem,
                                       int *status, void *stream) {
  if (!A || !B || !D || !status) return SWILA_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (N == 64 && K == 128 && !a_in_smem) umma_selftest_bf16_kernel<64, 128, 0><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 128 && K == 32 && !a_in_smem) umma_selftest_bf16_kernel<128, 32, 0><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 32 && K == 32 && !a_in_smem) umma_selftest_bf16_kernel<32, 32, 0><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 64 && K == 64 && a_in_smem == 1) umma_selftest_bf16_kernel<64, 64, 1><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 64 && K == 64 && a_in_smem == 2) umma_selftest_sw128_kernel<64><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 32 && K == 64 && a_in_smem == 2) umma_selftest_sw128_kernel<32><<<1, 128, 0, st>>>(A, B, D, status);
  else if (N == 128 && K == 32 && a_in_smem == 3) umma_selftest_bmn_kernel<<<1, 128, 0, st>>>(A, B, D, status);
  else return SWILA_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? SWILA_OK : SWILA_ERR_CUDA;
}
