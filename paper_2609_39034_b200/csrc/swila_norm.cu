// RMSNorm of the layer output (App. D.1), in place: a memory-bound pass over o [B,H,T,Dv].
//
// A lane holds 16-byte vectors of a row (8 bf16 or 4 fp32 values).  Rows up to 32 vectors wide (Dv <= 256 in bf16,
// <= 128 in fp32) are shared by the lanes of a warp, several rows per warp in flight, read once and kept in
// registers between the mean and the scaling; wider rows take one warp each and are read twice (the second time
// from L1/L2).  Traffic is one read and one write of o: the roofline is the HBM copy bandwidth.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/swila.h"

namespace swila {

template <bool BF16>
__device__ __forceinline__ void unpack(const uint4 &u, float (&x)[8]) {
  if constexpr (BF16) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  } else {
    x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y); x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    x[4] = x[5] = x[6] = x[7] = 0.f;
  }
}

template <bool BF16>
__device__ __forceinline__ uint4 pack(const float (&x)[8]) {
  uint4 u;
  if constexpr (BF16) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
    const __nv_bfloat162 c = __floats2bfloat162_rn(x[4], x[5]), d = __floats2bfloat162_rn(x[6], x[7]);
    u.x = *reinterpret_cast<const uint32_t *>(&a); u.y = *reinterpret_cast<const uint32_t *>(&b);
    u.z = *reinterpret_cast<const uint32_t *>(&c); u.w = *reinterpret_cast<const uint32_t *>(&d);
  } else {
    u.x = __float_as_uint(x[0]); u.y = __float_as_uint(x[1]); u.z = __float_as_uint(x[2]); u.w = __float_as_uint(x[3]);
  }
  return u;
}

// Rows of at most 32 vectors: LPR lanes per row (the power of two that covers the row), 32 / LPR rows per warp at
// a time and U such groups in flight per warp, so that enough bytes are outstanding to cover the memory latency
// (one 256-byte row per warp at a time reached a third of the copy bandwidth).
template <bool BF16, int LPR>
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(uint4 *o, const float *weight, size_t rows, int Dv, float eps) {
  constexpr int EPV = BF16 ? 8 : 4, RPW = 32 / LPR, U = 4;
  const int lane = threadIdx.x & 31, c = lane % LPR, sub = lane / LPR;
  const size_t warp0 = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const size_t nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  const int nvec = Dv / EPV;
  const bool c_ok = c < nvec;
  const float inv_dv = 1.0f / (float)Dv;
  float wv[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) wv[i] = (weight && c_ok && i < EPV) ? __ldg(weight + c * EPV + i) : 1.0f;
  for (size_t row0 = warp0 * (RPW * U); row0 < rows; row0 += nwarps * (RPW * U)) {
    uint4 u[U];
    bool ok[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      const size_t row = row0 + k * RPW + sub;
      ok[k] = c_ok && row < rows;
      u[k] = ok[k] ? __ldcs(o + row * nvec + c) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
      float x[8];
      unpack<BF16>(u[k], x);
      float ss = 0.f;
#pragma unroll
      for (int i = 0; i < EPV; ++i) ss = fmaf(x[i], x[i], ss);
#pragma unroll
      for (int off = 1; off < LPR; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const float scale = rsqrtf(fmaf(ss, inv_dv, eps));
#pragma unroll
      for (int i = 0; i < EPV; ++i) x[i] *= scale * wv[i];
      if (ok[k]) __stcs(o + (row0 + k * RPW + sub) * nvec + c, pack<BF16>(x));
    }
  }
}

// Any row width: one warp per row, the row read twice when it is wider than 32 vectors.
template <bool BF16>
__global__ void __launch_bounds__(256) rmsnorm_kernel(uint4 *o, const float *weight, size_t rows, int Dv, float eps) {
  constexpr int EPV = BF16 ? 8 : 4;  // elements per 16-byte vector
  const int lane = threadIdx.x & 31;
  const size_t warp0 = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const size_t nwarps = ((size_t)gridDim.x * blockDim.x) >> 5;
  const int nvec = Dv / EPV;
  const float inv_dv = 1.0f / (float)Dv;
  for (size_t row = warp0; row < rows; row += nwarps) {
    uint4 *base = o + row * nvec;
    uint4 held = make_uint4(0, 0, 0, 0);
    float ss = 0.f;
    for (int c = lane; c < nvec; c += 32) {
      const uint4 u = __ldcs(base + c);
      if (c == lane) held = u;
      float x[8];
      unpack<BF16>(u, x);
#pragma unroll
      for (int i = 0; i < EPV; ++i) ss = fmaf(x[i], x[i], ss);
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float scale = rsqrtf(fmaf(ss, inv_dv, eps));
    for (int c = lane; c < nvec; c += 32) {
      const uint4 u = (c == lane) ? held : base[c];
      float x[8];
      unpack<BF16>(u, x);
#pragma unroll
      for (int i = 0; i < EPV; ++i) x[i] *= weight ? scale * __ldg(weight + c * EPV + i) : scale;
      __stcs(base + c, pack<BF16>(x));
    }
  }
}

template <bool BF16>
static void launch_rmsnorm(uint4 *o, const float *weight, size_t rows, int Dv, float eps, int sms, cudaStream_t st) {
  const int nvec = Dv / (BF16 ? 8 : 4);
  // 8 warps per block; as many blocks as are resident at once (the kernels stride over the rows), fewer for few rows
  auto grid_for = [&](auto kern, size_t rows_per_warp) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 256, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    const size_t want = (rows + 8 * rows_per_warp - 1) / (8 * rows_per_warp), cap = (size_t)sms * per_sm;
    return (unsigned)(want < cap ? want : cap);
  };
#define SWILA_NORM_CASE(LPR)                                                                                   \
  if (nvec <= LPR) {                                                                                           \
    auto kern = rmsnorm_rows_kernel<BF16, LPR>;                                                                \
    kern<<<grid_for(kern, 4 * 32 / LPR), 256, 0, st>>>(o, weight, rows, Dv, eps);                               \
    return;                                                                                                    \
  }
  SWILA_NORM_CASE(2) SWILA_NORM_CASE(4) SWILA_NORM_CASE(8) SWILA_NORM_CASE(16) SWILA_NORM_CASE(32)
#undef SWILA_NORM_CASE
  auto kern = rmsnorm_kernel<BF16>;
  kern<<<grid_for(kern, 1), 256, 0, st>>>(o, weight, rows, Dv, eps);
}

}  // namespace swila

extern "C" int swila_output_norm(const swila_shape_t *s, void *o, const float *weight, float eps, void *stream) {
  if (!s || !o) return SWILA_ERR_NULL;
  if (s->B <= 0 || s->H <= 0 || s->T < 0 || s->Dv <= 0 || s->Dv % 8 != 0 || !(eps >= 0.f)) return SWILA_ERR_SHAPE;
  if (s->io_dtype != SWILA_IO_FP32 && s->io_dtype != SWILA_IO_BF16) return SWILA_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(o) & 15u) return SWILA_ERR_ALIGN;
  const size_t rows = (size_t)s->B * s->H * (size_t)s->T;
  if (rows == 0) return SWILA_OK;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SWILA_ERR_CUDA;
  if (s->io_dtype == SWILA_IO_BF16)
    swila::launch_rmsnorm<true>((uint4 *)o, weight, rows, s->Dv, eps, sms, (cudaStream_t)stream);
  else
    swila::launch_rmsnorm<false>((uint4 *)o, weight, rows, s->Dv, eps, sms, (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? SWILA_OK : SWILA_ERR_CUDA;
}
