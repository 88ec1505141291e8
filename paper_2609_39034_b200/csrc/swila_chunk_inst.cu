// Instantiations and dispatch of the chunked tensor-core kernel (bf16 io, ungated, non-temporal,
// J in {4, 8}: with fewer components a block covers more columns and its shared-memory tiles do not fit).
#include "swila_chunk.cuh"

namespace swila {

// Returns a cudaError_t value (>= 0), or -1000 when the combination is not compiled.
int chunk_dispatch(const LaunchArgs &a) {
  if (a.io_dtype != SWILA_IO_BF16 || a.gate_mode != 0 || a.p.temporal) return -1000;
#define SWILA_CHUNK_CASE(JJ)                         \
  case JJ:                                           \
    if (a.Dk == 128) return launch_chunk<JJ, 128>(a); \
    if (a.Dk == 64) return launch_chunk<JJ, 64>(a);   \
    return -1000;
  switch (a.J) {
    SWILA_CHUNK_CASE(4)
    SWILA_CHUNK_CASE(8)
    default: return -1000;
  }
}

// Reads (and clears) the device-side error flag of the current device; synchronises.
int chunk_error_fetch(int *flag) {
  int zero = 0;
  cudaError_t e = cudaMemcpyFromSymbol(flag, g_chunk_error, sizeof(int));
  if (e == cudaSuccess && *flag) e = cudaMemcpyToSymbol(g_chunk_error, &zero, sizeof(int));
  return (int)e;
}

}  // namespace swila

#ifdef SWILA_CHUNK_PROFILE
// Developer build only: per-phase cycle counters of block 0, 8 per warp role (rows, helpers, ...).
extern "C" int swila_chunk_profile(long long *out32) {
  return cudaMemcpyFromSymbol(out32, swila::g_chunk_prof, 32 * sizeof(long long)) == cudaSuccess ? 0 : -1;
}
// Developer build only: per block (first 1024) total cycles, SM id and start time in ns.
extern "C" int swila_chunk_blocks(long long *out3072) {
  return cudaMemcpyFromSymbol(out3072, swila::g_chunk_blk, 3 * 1024 * sizeof(long long)) == cudaSuccess ? 0 : -1;
}
#endif
