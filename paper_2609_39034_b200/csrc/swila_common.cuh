// Shared declarations of the SwiLA CUDA library: launch parameter block, small device
// helpers (approximate transcendental units, packed FP32 FMA, cp.async staging).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/swila.h"

namespace swila {

// One launch of the recurrence; filled by the C-ABI entry points after validation.
struct ScanParams {
  int B, H, T, Dv;
  int temporal;     // 0/1
  int gran;         // SWILA_GATE_*
  const void *q, *k, *v;
  const void *beta_logit, *pik_logit, *piq_logit;
  const void *gk_logit, *gq_logit;
  const float *alpha;
  const float *W_in, *r_in, *rho_in;  // may be null: zero state / uniform distributions
  float *W_out, *r_out, *rho_out;     // may be null: state discarded
  void *o;
  float *r_debug;                     // may be null
  int qkv_act;                        // 0/1: SiLU on q, k, v and L2 normalisation of q, k inside the kernel
  int post;                           // 0/1: post-decay form (Eq. 3.7) of the gated variants
  // Gated rows in the chunked kernel: a word written by the guard pass that looks at the decays first.  The chunked
  // kernel returns at once when it is non-zero, the scan kernel launched behind it when it is zero (null: no guard).
  const unsigned *guard;
  int guard_runs_scan;                // scan kernel: 1 = run only if *guard != 0
  float *r_sum, *r_ent, *rho_sum, *rho_ent;  // sums over time of the mixture weights; each may be null
};

// epsilon under the root of the in-kernel L2 normalisation of q and k
constexpr float kL2Eps = 1e-6f;

struct LaunchArgs {
  ScanParams p;
  int Dk, J, io_dtype, gate_mode /*0 none, 1 per-key, 2 per-row, 3 per-element*/, post, algo;
  cudaStream_t stream;
};

// Dispatch entry of one translation unit (one key dimension, one gate mode).
// Returns SWILA_OK, SWILA_ERR_UNSUPPORTED or SWILA_ERR_CUDA.
template <int DK, int GATE, bool POST>
int scan_dispatch(const LaunchArgs &a);

// ---------------------------------------------------------------------------------------
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kHalfLog2e = 0.7213475204444817f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sigmoid_approx(float x) {
  return rcp_approx(1.0f + ex2_approx(-kLog2e * x));
}

// SiLU(x) = x sigmoid(x) (App. B.2)
__device__ __forceinline__ float silu_approx(float x) { return x * sigmoid_approx(x); }

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float &dst, float x) { dst = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 &dst, float x) { dst = __float2bfloat16_rn(x); }

// 16-byte asynchronous global->shared copy, L2 only; src_bytes == 0 zero-fills.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src, int src_bytes) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem_src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Two FP32 FMAs / multiplies on a register pair.  SWILA_SCALAR_FMA selects plain scalar
// instructions instead of the packed f32x2 forms.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
#ifdef SWILA_SCALAR_FMA
  return make_float2(fmaf(a.x, b.x, c.x), fmaf(a.y, b.y, c.y));
#else
  return __ffma2_rn(a, b, c);
#endif
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
#ifdef SWILA_SCALAR_FMA
  return make_float2(a.x * b.x, a.y * b.y);
#else
  return __fmul2_rn(a, b);
#endif
}

// J consecutive floats from shared memory with the widest aligned loads.
template <int J>
__device__ __forceinline__ void lds_vec(const float *p, float (&out)[J]) {
  if constexpr (J % 4 == 0) {
#pragma unroll
    for (int i = 0; i < J / 4; ++i) {
      float4 t = reinterpret_cast<const float4 *>(p)[i];
      out[4 * i] = t.x; out[4 * i + 1] = t.y; out[4 * i + 2] = t.z; out[4 * i + 3] = t.w;
    }
  } else if constexpr (J == 2) {
    float2 t = *reinterpret_cast<const float2 *>(p);
    out[0] = t.x; out[1] = t.y;
  } else {
#pragma unroll
    for (int i = 0; i < J; ++i) out[i] = p[i];
  }
}

}  // namespace swila
