// Instantiations and dispatch of the chunked tensor-core kernel (bf16 io, ungated, plain or Temporal,
// J in {4, 8}, and 16 at Dk = 64: with fewer components a block covers more columns and its shared-memory tiles do
// not fit).
#include "../../include/swila_dev.h"
#include "swila_chunk.cuh"

namespace swila {

// Returns a cudaError_t value (>= 0), or -1000 when the combination is not compiled.
int chunk_dispatch(const LaunchArgs &a) {
  if (a.io_dtype != SWILA_IO_BF16 || a.gate_mode != 0 || a.p.qkv_act) return -1000;
#define SWILA_CHUNK_CASE(JJ)                                                                   \
  case JJ:                                                                                     \
    if (a.Dk == 128) return a.p.temporal ? launch_chunk<JJ, 128, true>(a) : launch_chunk<JJ, 128>(a); \
    if (a.Dk == 64) return a.p.temporal ? launch_chunk<JJ, 64, true>(a) : launch_chunk<JJ, 64>(a);   \
    return -1000;
  switch (a.J) {
    SWILA_CHUNK_CASE(4)
    SWILA_CHUNK_CASE(8)
    case 16:  // the component-count ablation of Sec. 5; only Dk = 64 fits shared memory
      if (a.Dk == 64) return a.p.temporal ? launch_chunk<16, 64, true>(a) : launch_chunk<16, 64>(a);
      return -1000;
    default: return -1000;
  }
}

// Reads (and clears) the device-side error flag of the current device; synchronises.
int chunk_error_fetch(int *flag) {
  int zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(flag, umma::g_chunk_error, sizeof(int));
  if (e == cudaSuccess && *flag) e = cudaMemcpyToSymbol(umma::g_chunk_error, &zero, sizeof(int));
  return (int)e;
}

}  // namespace swila

namespace swila {
// One block, one barrier that nothing ever arrives at: the bounded wait must give up, leave its code in the error word
// and let the kernel end normally (no trap, no fault: the context stays usable).
__global__ void swila_wait_timeout_kernel(int *gave_up) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    umma::mbar_init(&bar, 1);
    umma::mbar_fence_init();
  }
  __syncthreads();
  const bool ok = umma::mbar_wait(&bar, 0);
  if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}
}  // namespace swila

extern "C" int swila_selftest_wait_timeout(int *gave_up, void *stream) {
  if (!gave_up) return SWILA_ERR_NULL;
  swila::swila_wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(gave_up);
  return cudaGetLastError() == cudaSuccess ? SWILA_OK : SWILA_ERR_CUDA;
}

// Host-only probes of the chunked kernel's work distribution (no GPU call): what the CPU tests check.
extern "C" int swila_chunk_plan(int B, int H, int T, int Dv, int J, int sm_count, int has_state_out, long long out[6]) {
  if (!out) return SWILA_ERR_NULL;
  if (B <= 0 || H <= 0 || T <= 0 || Dv <= 0 || sm_count <= 0) return SWILA_ERR_SHAPE;
  if (J != 4 && J != 8 && J != 16) return SWILA_ERR_UNSUPPORTED;
  const long long cols = 128 / J, nslice = (Dv + cols - 1) / cols, nch = (T + 31) / 32;
  const swila::ChunkPlan pl =
      swila::chunk_plan((long long)B * H, nslice, nch, sm_count, has_state_out != 0, swila::kChunkFlagTiles);
  out[0] = pl.split; out[1] = pl.gang; out[2] = pl.nch; out[3] = pl.per; out[4] = pl.units; out[5] = pl.grid;
  return SWILA_OK;
}

extern "C" int swila_chunk_run_pieces(long long units, int nch, int per, long long run, int *pieces, int capacity) {
  if (units <= 0 || nch <= 0 || per <= 0 || run < 0) return SWILA_ERR_SHAPE;
  const int n = swila::chunk_run_pieces(units, nch, per, run);
  if (n > capacity) return SWILA_ERR_SIZE;
  if (n > 0 && !pieces) return SWILA_ERR_NULL;
  for (int i = 0; i < n; ++i) {
    const swila::ChunkPiece pc = swila::chunk_run_piece(units, nch, per, run, i);
    pieces[3 * i] = pc.unit; pieces[3 * i + 1] = pc.cb; pieces[3 * i + 2] = pc.ce;
  }
  return n;
}
