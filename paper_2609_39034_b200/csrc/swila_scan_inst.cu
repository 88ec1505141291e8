// One translation unit per (key dimension, decay mode): compiled several times with
// -DSWILA_DK=<16|64|128> -DSWILA_GATE=<0|1|2> -DSWILA_POST=<0|1>, so that the many
// register-resident instantiations build in parallel.
#include "swila_scan.cuh"

#ifndef SWILA_DK
#error "compile with -DSWILA_DK, -DSWILA_GATE, -DSWILA_POST"
#endif

namespace swila {

namespace {
template <typename IO, int J>
int pick(const LaunchArgs &a) {
  constexpr int DK = SWILA_DK;
  constexpr int GATE = SWILA_GATE;
  constexpr bool POST = SWILA_POST != 0;
  // tokens per staged block: fp32 rows are twice as wide, and per-key gates at Dk = 128 add 2 KB of fp32 per token;
  // keep two blocks per SM resident (8-token blocks of gates would leave room for one only)
  constexpr int TB = (sizeof(IO) == 2 && !(GATE == 1 && DK == 128)) ? 8 : 4;
  if constexpr (DK == 16) {
    return launch_scan<ScanCfg<IO, J, DK, 32, TB, GATE>, POST>(a);
  } else {
    if (a.algo == SWILA_ALGO_SCAN_WIDE) {
      if constexpr (GATE == 0 && DK == 128) return launch_scan<ScanCfg<IO, J, DK, 256, TB, GATE>, POST>(a);
      return -1000;
    }
    if (a.algo == SWILA_ALGO_SCAN_NARROW) {
      if constexpr (GATE == 0 && DK == 128 && J >= 4) return launch_scan<ScanCfg<IO, J, DK, 128, TB, GATE, 16>, POST>(a);
      return -1000;
    }
    // a decode step stages and prepares one token: blocks of one token (same arithmetic per token, so the bits
    // of a prefill and of the decode steps that continue it still agree)
    if (a.p.T == 1) return launch_scan<ScanCfg<IO, J, DK, 128, 1, GATE>, POST>(a);
    return launch_scan<ScanCfg<IO, J, DK, 128, TB, GATE>, POST>(a);
  }
}
template <typename IO>
int pick_j(const LaunchArgs &a) {
  switch (a.J) {
    case 1: return pick<IO, 1>(a);
    case 2: return pick<IO, 2>(a);
    case 4: return pick<IO, 4>(a);
    case 8: return pick<IO, 8>(a);
    case 16: return pick<IO, 16>(a);
    default: return -1000;
  }
}
}  // namespace

// Returns a cudaError_t value (>= 0), or -1000 when the combination is not compiled.
template <>
int scan_dispatch<SWILA_DK, SWILA_GATE, (SWILA_POST != 0)>(const LaunchArgs &a) {
  return a.io_dtype == SWILA_IO_BF16 ? pick_j<__nv_bfloat16>(a) : pick_j<float>(a);
}

}  // namespace swila
