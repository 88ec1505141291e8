// Gated SwiLA (Sec. 3.4) with one decay per state row -- alpha_tjd (Eqs. 3.7 / 3.8 as printed; "Diag(alpha_tj) W" in
// App. B.4) or one per component -- in the chunked tensor-core kernel: its instantiations, and the guard pass that
// decides whether a call may take that kernel.
//
// Inside a chunk the kernel works in units of the state at the chunk's start: coefficients are divided by the running
// product A_t of the row's decays.  That is exact while A_t stays a normal number of moderate size; a product of 32
// decays below 2^-40 (a row wiped out within one chunk) could overflow those quotients.  The guard pass reads the
// decays first and raises a flag if any (row, chunk) is that small; the chunked kernel then returns at once and the
// scan kernel, launched right behind it, evaluates the call instead (it returns at once when the flag is clear).
#include <atomic>

#include "../../include/swila.h"
#include "swila_chunk.cuh"

namespace swila {

constexpr int kGuardSlots = 8;
static __device__ unsigned g_gate_guard[kGuardSlots];

// One thread per (batch-head, chunk, component, group of V columns) -- V = 4 with one decay per output dimension (Dv
// is a multiple of 8, rows are 16-byte aligned), V = 1 with one per component -- multiplies the decays of the chunk's
// tokens.  per = decays per (token, component): Dv or 1.
template <int V>
__global__ void __launch_bounds__(256) swila_gate_guard_kernel(const float *__restrict__ alpha, long long nbh, int T, int J,
                                                              int per, int C, unsigned *flag) {
  const long long nch = (T + C - 1) / C;
  const int groups = per / V;
  const long long total = nbh * nch * J * groups;
  bool bad = false;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int g = (int)(i % groups);
    const int j = (int)((i / groups) % J);
    const long long c = (i / ((long long)groups * J)) % nch;
    const long long bh = i / ((long long)groups * J * nch);
    const float *a0 = alpha + ((bh * T + c * C) * J + j) * (size_t)per + (size_t)g * V;
    const size_t tstride = (size_t)J * per;
    const int nt = min(C, T - (int)c * C);
    float prod[V];
#pragma unroll
    for (int v = 0; v < V; ++v) prod[v] = 1.0f;
#pragma unroll 1
    for (int t = 0; t < nt; t += 8) {
      float x[8][V];  // the loads of a trip are all in flight together
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if constexpr (V == 4) {
          const float4 q = (t + u < nt) ? __ldg(reinterpret_cast<const float4 *>(a0 + (size_t)(t + u) * tstride)) : make_float4(1.f, 1.f, 1.f, 1.f);
          x[u][0] = q.x; x[u][1] = q.y; x[u][2] = q.z; x[u][3] = q.w;
        } else {
          x[u][0] = (t + u < nt) ? __ldg(a0 + (size_t)(t + u) * tstride) : 1.0f;
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
#pragma unroll
        for (int v = 0; v < V; ++v) prod[v] *= x[u][v];
      }
    }
#pragma unroll
    for (int v = 0; v < V; ++v) bad = bad || !(prod[v] >= 9.094947e-13f && prod[v] <= 1.0000001f);  // 2^-40; NaN and decays above 1 too
  }
  if (__any_sync(0xffffffffu, bad) && (threadIdx.x & 31) == 0) atomicOr(flag, 1u);
}

// Returns a cudaError_t value (>= 0), or -1000 when the combination is not compiled.  On success a.p.guard points at
// the flag the caller must hand to the scan kernel it launches behind this one.
int chunk_gated_dispatch(LaunchArgs &a) {
  if (a.io_dtype != SWILA_IO_BF16 || a.gate_mode != 2 || a.p.qkv_act) return -1000;
  if (a.p.temporal && a.Dk != 64) return -1000;  // Temporal with row gates fits shared memory at Dk = 64 only
  if (a.p.gran != SWILA_GATE_PER_OUT && a.p.gran != SWILA_GATE_SCALAR) return -1000;
  // (J = 8 at Dk = 128 does not fit shared memory with the decay products beside the wider gate stages)
  if (!((a.J == 4 && (a.Dk == 64 || a.Dk == 128)) || (a.J == 8 && a.Dk == 64))) return -1000;
  if (a.p.r_debug || a.p.r_sum || a.p.r_ent || a.p.rho_sum || a.p.rho_ent) return -1000;
  static std::atomic<unsigned> counter{0};
  unsigned *flags = nullptr;
  cudaError_t e = cudaGetSymbolAddress((void **)&flags, g_gate_guard);
  if (e != cudaSuccess) return (int)e;
  unsigned *flag = flags + (counter++ % kGuardSlots);
  e = cudaMemsetAsync(flag, 0, sizeof(unsigned), a.stream);
  if (e != cudaSuccess) return (int)e;
  const int per = a.p.gran == SWILA_GATE_PER_OUT ? a.p.Dv : 1;
  const long long nbh = (long long)a.p.B * a.p.H, nch = (a.p.T + 31) / 32;
  const long long total = nbh * nch * a.J * (per == 1 ? 1 : per / 4);
  const unsigned grid = (unsigned)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
  if (per == 1) swila_gate_guard_kernel<1><<<grid, 256, 0, a.stream>>>(a.p.alpha, nbh, a.p.T, a.J, per, 32, flag);
  else swila_gate_guard_kernel<4><<<grid, 256, 0, a.stream>>>(a.p.alpha, nbh, a.p.T, a.J, per, 32, flag);
  e = cudaGetLastError();
  if (e != cudaSuccess) return (int)e;
  a.p.guard = flag;
  a.p.guard_runs_scan = 0;
  if (a.p.temporal) return a.J == 4 ? launch_chunk<4, 64, true, true>(a) : launch_chunk<8, 64, true, true>(a);
  if (a.J == 4) return a.Dk == 128 ? launch_chunk<4, 128, false, true>(a) : launch_chunk<4, 64, false, true>(a);
  return launch_chunk<8, 64, false, true>(a);
}

// Reads (and clears) this translation unit's copy of the device-side error word; synchronises.
int chunk_gated_error_fetch(int *flag) {
  int zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(flag, umma::g_chunk_error, sizeof(int));
  if (e == cudaSuccess && *flag) e = cudaMemcpyToSymbol(umma::g_chunk_error, &zero, sizeof(int));
  return (int)e;
}

}  // namespace swila
