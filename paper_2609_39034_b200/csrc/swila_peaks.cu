// Microbenchmarks that measure the denominators of the scan kernel's roofline on the
// device at hand: the FP32 FMA rate of plain and packed (f32x2) FMAs with register-resident
// operands.  Not part of the recurrence; used by the benchmark harness only.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/swila_dev.h"

namespace {

// Each thread owns CH independent accumulator pairs and applies `iters` rounds of
// acc = acc * a + b to all of them.  PACKED uses one f32x2 FMA per pair, otherwise two
// scalar FMAs.  2 * CH FMAs per thread per round.
template <int CH, bool PACKED>
__global__ void __launch_bounds__(256) fma_chain_kernel(float *out, int iters, float a0, float b0) {
  float2 acc[CH];
#pragma unroll
  for (int i = 0; i < CH; ++i) acc[i] = make_float2(threadIdx.x * 1e-6f + i, blockIdx.x * 1e-7f - i);
  float2 a = make_float2(a0, a0 * 0.999f), b = make_float2(b0, -b0);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < CH; ++i) {
      if constexpr (PACKED) {
        acc[i] = __ffma2_rn(acc[i], a, b);
      } else {
        acc[i].x = fmaf(acc[i].x, a.x, b.x);
        acc[i].y = fmaf(acc[i].y, a.y, b.y);
      }
    }
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < CH; ++i) s += acc[i].x + acc[i].y;
  if (s == 123.456f) out[0] = s;  // keeps the chains alive; practically never true
}

template <int CH, bool PACKED>
int launch(float *out, int blocks, int iters, cudaStream_t st) {
  fma_chain_kernel<CH, PACKED><<<blocks, 256, 0, st>>>(out, iters, 0.9999f, 1e-3f);
  return (int)cudaGetLastError();
}

}  // namespace

extern "C" int swila_bench_fma_chain(int packed, int chains, int blocks, int iters, float *scratch_out,
                                     double *fma_per_launch, void *stream) {
  if (!scratch_out || !fma_per_launch || blocks <= 0 || iters <= 0) return SWILA_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  int rc;
  switch (chains) {
    case 4: rc = packed ? launch<4, true>(scratch_out, blocks, iters, st) : launch<4, false>(scratch_out, blocks, iters, st); break;
    case 8: rc = packed ? launch<8, true>(scratch_out, blocks, iters, st) : launch<8, false>(scratch_out, blocks, iters, st); break;
    case 16: rc = packed ? launch<16, true>(scratch_out, blocks, iters, st) : launch<16, false>(scratch_out, blocks, iters, st); break;
    default: return SWILA_ERR_UNSUPPORTED;
  }
  if (rc != 0) return SWILA_ERR_CUDA;
  *fma_per_launch = 2.0 * chains * 256.0 * (double)blocks * (double)iters;
  return SWILA_OK;
}
