// Work distribution of the chunked kernel, as plain integer arithmetic shared by the kernel, the launch code
// and a host-only probe that the CPU tests call.
//
// The units x nch chunks of a launch (unit after unit; a unit is a tile, or a (batch, head) when the blocks
// come in gangs of column slices) are cut into equal runs of `per` chunks.  A run falls into pieces
// (unit, first chunk, end chunk).  Within a run the piece that ends in the middle of a unit (a head, whose
// state the owner of the next run waits for) comes first, whole units next, and the piece that starts in
// the middle of a unit (a tail, which needs the state left by the previous run's head) comes last.  With
// per >= nch a head is shorter than a run, so it is finished before the owner of the tail gets there.
#pragma once

#if defined(__CUDACC__)
#define SWILA_HD __host__ __device__
#else
#define SWILA_HD
#endif

namespace swila {

struct ChunkPiece {
  int unit, cb, ce;  // chunks [cb, ce) of `unit`
};

// Number of pieces of run `run` (0 when the run lies past the end of the work).
SWILA_HD inline int chunk_run_pieces(long long units, int nch, int per, long long run) {
  const long long run0 = run * per, total = units * nch;
  const long long run1 = run0 + per < total ? run0 + per : total;
  if (run1 <= run0) return 0;
  return (int)((run1 - 1) / nch) - (int)(run0 / nch) + 1;
}

// The pi-th piece of run `run` in processing order (0 <= pi < chunk_run_pieces(...)).
SWILA_HD inline ChunkPiece chunk_run_piece(long long units, int nch, int per, long long run, int pi) {
  const long long run0 = run * per, total = units * nch;
  const long long run1 = run0 + per < total ? run0 + per : total;
  const int unit_first = (int)(run0 / nch), chunk_first = (int)(run0 % nch);
  const int npieces = (int)((run1 - 1) / nch) - unit_first + 1;
  const bool has_tail = chunk_first > 0;
  const bool has_head = run1 % nch != 0 && !(npieces == 1 && has_tail);
  int ps;  // position of the piece inside the run, in unit order
  if (has_head && pi == 0) {
    ps = npieces - 1;
  } else {
    const int k = pi - (has_head ? 1 : 0);
    const int mid = npieces - (has_head ? 1 : 0) - (has_tail ? 1 : 0);
    ps = k < mid ? k + (has_tail ? 1 : 0) : 0;
  }
  ChunkPiece pc;
  pc.unit = unit_first + ps;
  pc.cb = ps == 0 ? chunk_first : 0;
  const long long end = run1 - (long long)pc.unit * nch;
  pc.ce = end < nch ? (int)end : nch;
  return pc;
}

// How a launch is laid out.  split == 0: one tile per block, nothing is handed over.  split == 1: `gangs` runs of
// `per` chunks over the (batch, head) units, each walked by a gang of `gang` blocks (one column slice each).
struct ChunkPlan {
  int split, gang, nch, per;
  long long units, grid;
};

// nbh = B*H, nslice = column slices per (batch, head), nsm = SMs (one block per SM), max_flags = tiles the
// hand-over flags can cover.  The split is taken when there are more (batch, head) units than gangs, the state
// output exists (it carries the state of a split tile), and it shortens the longest block by at least 3 %.
inline ChunkPlan chunk_plan(long long nbh, long long nslice, long long nch, int nsm, bool has_state_out, long long max_flags) {
  ChunkPlan pl;
  const long long ntiles = nbh * nslice;
  pl.split = 0; pl.gang = 1; pl.nch = (int)nch; pl.per = (int)nch; pl.units = ntiles; pl.grid = ntiles;
  const long long gangs = nslice > 0 ? nsm / nslice : 0;
  if (gangs <= 0 || !has_state_out || nbh <= gangs || ntiles > max_flags || nch < 16) return pl;
  const long long total = nbh * nch;
  const long long per = (total + gangs - 1) / gangs;
  const long long plain = ((ntiles + nsm - 1) / nsm) * nch;
  if (per < nch || per * 100 > plain * 97) return pl;
  pl.split = 1; pl.gang = (int)nslice; pl.per = (int)per; pl.units = nbh;
  pl.grid = ((total + per - 1) / per) * nslice;
  return pl;
}

}  // namespace swila
