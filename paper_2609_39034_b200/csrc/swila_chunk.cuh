// Chunked tensor-core kernel of the SwiLA recurrence (Sec. 3.2, Eqs. 3.3-3.5) for sm_100a.
//
// The recurrence is nonlinear only through the scalar coefficient c_tjd = beta r delta that
// multiplies the rank-one update k_t; the state enters a token only through two dot products.
// Over a chunk of C tokens starting from state W0, for every row (j, d):
//
//   pred_t = w_0 . k_t + sum_{s<t}  c_s (k_s . k_t)        -> delta_t = v_t - pred_t   (Eq. 3.3 text)
//   r_t    = E-step over j of (lk_t - delta_t^2 / 2)                                   (Eq. 3.4)
//   c_t    = beta_t r_t delta_t
//   w_t.q_t = w_0 . q_t + sum_{s<=t} c_s (k_s . q_t)       -> o_t = sum_j pi^q_j w_t.q_t (Eq. 3.5)
//   w_C    = w_0 + sum_s c_s k_s                                                        (Eq. 3.3)
//
// This is the same recurrence, token by token and exact (no Newton iteration): only the order
// of the floating-point additions differs from the scan.  The dense contractions
//   P0 = W0 K^T, Q0 = W0 Q^T  (M x Dk x C),   W += Cmat K  (M x C x Dk),   the Gram matrices
// run on the tcgen05 tensor cores with BF16 operands (K = 16 per instruction) and FP32
// accumulation in tensor memory.  k and q are bf16 inputs, hence exact operands; every FP32
// operand (the state, the update coefficients, Gram matrices used as operands) is split as
// x = hi + lo with hi = bf16(x), lo = bf16(x - hi) and both parts are multiplied (lo x lo is
// dropped), which keeps 16 significant bits of the operand: a relative error of 4e-6 per product,
// unbiased, against a parity tolerance of 1e-4.  The update coefficients of W += Cmat K alone get
// a third part (24 bits): their rounding is the one error that is added to the state and carried
// along the sequence, and from a zero state with near-uniform gates, where the components separate
// only through the E-step's feedback, 16 bits left the state 2e-4 off after 8192 tokens.  The
// triangular part (the sums over s inside the chunk) and the E-step stay on the FP32 ALUs, one
// thread per row.
//
// Across chunks the products of the state with the next chunk's keys and queries are taken off
// the serial path: with W_{n+1} = W_n + Cmat_n K_n,
//   W_{n+1} [K;Q]_{n+1}^T = W_n [K;Q]_{n+1}^T  +  Cmat_n (K_n [K;Q]_{n+1}^T),
// the first term only needs the state BEFORE chunk n's update, so it runs while chunk n is still
// being processed; of the small second term (K = 32) the half of the chunk's first 16 tokens is
// issued as soon as their coefficients are final, the other half remains after the chunk.
//
// One block owns 128 rows = COLS = 128/J output columns of one (batch, head) and is split into
// three roles that run concurrently and meet on mbarriers:
//   row warps 0-3    thread r serves row (d = r / J, j = r % J), which is also its tensor-memory
//                    lane; the J components of a column sit in adjacent lanes, so the E-step
//                    normalisation is a few shuffles.  They run the sequential part of a chunk.
//   helper warps 4-7 turn gate logits into gates, move Gram matrices from tensor memory to shared
//                    memory (plain rows for the row warps, hi / lo operand tiles for the MMAs),
//                    split the state into its operand parts after each update, and form the
//                    outputs of the previous chunk.  One of their threads issues the tensor copies
//                    (TMA) that stage a chunk: k and q straight into the tensor cores' swizzled
//                    operand tile, v and the gate logits into a raw stage.
//   warp 8, lane 0   issues every tcgen05.mma and commits them to the barriers.
//
// When the tiles of a launch do not fill a whole number of waves, the chunk sequence is cut into
// equal runs per gang of blocks and split tiles hand their state over between blocks (ChunkSched).
//
// Instantiations: J = 4, 8 at Dk = 64, 128 and J = 16 at Dk = 64; plain, Temporal (App. B.3: the key-side prior
// mixes in the row's previous responsibility on the serial chain, the readout weights are a running average the
// helper warps form with the outputs), and an auxiliary one (plain, J <= 8) that also writes the responsibilities
// and the sums over time behind the load-balancing loss of Sec. 3.5.
#pragma once

#include <cuda.h>  // CUtensorMap and its enums (types only; the encoder is fetched through the runtime)
#include <cuda_bf16.h>

#include <atomic>
#include <type_traits>

#include "swila_chunk_sched.h"
#include "swila_common.cuh"
#include "swila_umma.cuh"

namespace swila {


// How the (tile, chunk) work items are spread over the blocks of a launch.  The ntiles * nch chunks, tile
// after tile, are cut into equal runs of `per` chunks, one run per block; within a run the piece that
// ends in the middle of a tile comes first and the piece that starts in the middle of a tile comes last.  The block that owns
// the head of a split tile leaves the state in the state output and releases flags[tile] = epoch; the
// block that owns the tail acquires it before loading that state.  With per == nch every block owns
// exactly one tile and no block ever waits.
// `gang` > 1: the blocks come in gangs of `gang` = column slices per (batch, head); the schedule above is then
// laid over (batch, head) units and the blocks of a gang walk it in step, one column slice each, so that the
// slices of one (batch, head) -- which share every 128-byte line of the gate tensors and all of k and q --
// are fetched at the same time and meet in L2 (without this the DRAM read traffic doubles).
struct ChunkSched {
  int ntiles, nch, per, gang;
  unsigned epoch;
  unsigned *flags;
};
constexpr int kChunkFlagSlots = 8, kChunkFlagTiles = 4096;
static __device__ unsigned g_chunk_flags[kChunkFlagSlots][kChunkFlagTiles];

// TEMPORAL_: Temporal SwiLA (App. B.3): two more streamed inputs (the temporal gate logits), the key-side prior
// normalised by the helpers (it enters a convex combination), and two carried distributions per row.
// GATED_: Gated SwiLA (Sec. 3.4) with one decay value per state ROW and token: alpha_tjd (Eq. 3.7 / 3.8 as printed,
// "Diag(alpha_tj) W" of App. B.4) or one per component.  A row's state is then a scalar multiple of an undecayed
// one, w_t = A_t (w_0 + sum_{s<=t} (c_s / A_s) k_s) with A_t the product of the row's decays since the chunk began,
// so the Gram matrices stay shared by all rows and the decay enters as per-row scalars on the FP32 ALUs.
template <int J_, int DK_, bool TEMPORAL_ = false, bool GATED_ = false>
struct ChunkCfg {
  static constexpr int J = J_, DK = DK_;
  static constexpr bool TEMPORAL = TEMPORAL_, GATED = GATED_;
  static constexpr int C = 32;            // tokens per chunk
  static constexpr int WIN = 24;          // tokens ahead (incl. its own trip) that a token's pushes reach on the ALUs;
                                          // the pushes of tokens 0-7 into tokens 24-31 go through the tensor cores
  static constexpr int GT = 8;            // tokens per trip of the rolled loops (keeps the hot code inside the instruction cache)
  static constexpr int NROW = 128;        // row threads = rows of the tile
  static constexpr int NT = GATED_ ? 320 : 288;  // 4 row warps + 4 helper warps + 1 MMA warp (+ 1 decay warp when Gated)
  static constexpr int COLS = NROW / J;   // output columns per block
  static constexpr int ES = 2;            // bf16 io
  // tensor-memory columns.  W: the state (FP32 accumulator); WHI / WLO: its bf16 operand parts, two key
  // dims per column; PQ: [P0 | Q0] = state x [K;Q] of the next chunk to run; QD: the query-side readouts
  // of a chunk (double-buffered); G: Gram matrices as they leave the tensor cores; FAR: what the first 8 tokens of
  // the chunk add to the predictions of its last 16 (only the last 8 are non-zero); CHI / CLO / CL3: the bf16 parts of the
  // chunk's update coefficients, two tokens per column (the third part is an operand of the state update only)
  static constexpr int TM_W = 0, TM_WHI = DK, TM_WLO = DK + DK / 2, TM_PQ = 2 * DK, TM_QD = TM_PQ + 2 * C,
                       TM_G = TM_QD + 2 * C, TM_FAR = TM_G + 2 * C, TM_CHI = TM_FAR + C / 2, TM_CLO = TM_CHI + C / 2,
                       TM_CL3 = TM_CLO + C / 2, TM_USED = TM_CL3 + C / 2;
  static constexpr int TM_ALLOC = 512;
  static_assert(TM_USED <= TM_ALLOC, "tensor memory budget");
  static_assert(J == 4 || J == 8 || (J == 16 && DK == 64),
                "J = 4, 8: outputs by in-group transposition; J = 16: by shuffle sums, and only Dk = 64 fits shared memory");
  // K/Q operand tile (bf16, K-major, 128-byte swizzle): per half of 64 key dims, 128 rows of 128 bytes, rows
  // [K_even ; Q_even ; K_odd ; Q_odd]: the chunks of both parities side by side, so that one 128-row A operand
  // covers the keys of two consecutive chunks.  Key dim d of row r sits at
  //   (d / 64) * TILE_HALF + r * 128 + (((d / 8) % 8) ^ (r % 8)) * 16 + (d % 8) * 2,
  // which is what a tensor copy with the 128-byte swizzle mode writes: k and q go straight from global memory
  // into the tile, 4 KB per copy.
  static constexpr int TILE_HALF = 4 * C * 128;
  static constexpr int TILE_BYTES = (DK / 64) * TILE_HALF;
  // A second copy of a chunk's keys for the update MMA, which reads them MN-major (tokens = K index) after the
  // chunk, when the tile rows are already being refilled: 3-deep ring of [DK/64][C rows][128 bytes], same swizzle.
  // The ring is laid out [half of 64 key dims][slot][token row]: the slots of two consecutive chunks are then
  // adjacent rows of one K-major operand (except when the ring wraps), which is what the Gram batch reads.
  // A fourth slot mirrors slot 0 (a chunk that goes to slot 0 is copied there too), so that the pair is adjacent
  // also when the ring wraps: (slot 2, slot 3).  Not in the Temporal kernel at Dk = 128, which is not bound by its
  // MMA count and measured 1 % slower with the extra copies (two MMAs per K step on those chunks there).
  static constexpr bool KU_MIRROR = !((TEMPORAL || GATED) && DK == 128);
  static constexpr int KU_HALF = C * 128;        // one slot of one half
  static constexpr int KU_HSTRIDE = (KU_MIRROR ? 4 : 3) * KU_HALF;  // distance between the halves
  static constexpr int KU_BYTES = (DK / 64) * KU_HALF;
  // raw stages (2-deep ring): v [C][COLS] bf16; beta logits [C][J][COLS] bf16, overwritten in place by the
  // helpers with beta = sigmoid(.) as fp32 [C][NROW] (hence the fp32-sized slot); pik logits [C][J][COLS]
  // bf16.  The query-prior logits piq [C][J][COLS] live in their own 3-deep ring because the outputs of
  // chunk n are formed while chunk n+2 is being fetched; chunk n+3 is staged into the slot of chunk n by the helper
  // thread that has just passed the barrier that ends the forming of chunk n's outputs.
  // Gate rows are fetched 8 columns wider than the slice (GROW = COLS + 8, the extra columns are never read):
  // the 16-byte skew between rows spreads the J lanes of a column over different banks.
  static constexpr int GROW = COLS + 8;
  static constexpr int R_V = 0;
  static constexpr int R_B = R_V + C * COLS * ES;
  static constexpr int R_PK = R_B + C * NROW * 4;
  // Temporal: the pik logits are overwritten in place by the normalised prior as fp32 [C][NROW] (like beta), and
  // the key-side temporal gate logits gk [C][COLS] bf16 follow; the query-side ones gq [C][COLS] follow the piq
  // logits in their ring.
  static constexpr int R_GK = R_PK + (TEMPORAL ? C * NROW * 4 : C * J * GROW * ES);
  static constexpr int RAW_BYTES = R_GK + (TEMPORAL ? C * COLS * ES : 0);
  static constexpr int RQ_GQ = C * J * GROW * ES;
  static constexpr int RPQ_BYTES = RQ_GQ + (TEMPORAL ? C * COLS * ES : 0);
  // bytes one chunk's tensor copies deliver: k and q into the operand tile, v, three gate tensors (+ gk, gq)
  static constexpr int STAGE_TX_BYTES = 3 * C * DK * ES + C * COLS * ES + 3 * C * J * GROW * ES + (TEMPORAL ? 2 * C * COLS * ES : 0);
  static_assert(C * J * GROW * ES <= C * NROW * 4, "the beta logits must fit the slot their gates overwrite");
  static constexpr int C_K = DK * ES / 16, C_V = COLS * ES / 16;  // 16-byte units per token row / column slice
  // operand tiles written by the helpers (bf16, same unit layout, 8 tokens per unit)
  static constexpr int BQ_LBO = C * 16;            // masked (K Q^T)^T: rows = later token, K index = earlier token
  static constexpr int BQ_TILE = (C / 8) * BQ_LBO;
  static constexpr int GX_LBO = 2 * C * 16;        // ([K;Q]_{n+1} K_n^T): rows = token of the next chunk
  static constexpr int GX_TILE = (C / 8) * GX_LBO;
  // shared memory map (bytes)
  static constexpr int OFF_TILE = 0;
  static constexpr int OFF_KU = OFF_TILE + TILE_BYTES;
  static constexpr int OFF_RAW = OFF_KU + (DK / 64) * KU_HSTRIDE;
  static constexpr int OFF_RPQ = OFF_RAW + 2 * RAW_BYTES;
  static constexpr int OFF_G = OFF_RPQ + 3 * RPQ_BYTES;             // 2 x Gkk [C][C] fp32 (-K K^T, for the row warps)
  static constexpr int OFF_BQ = OFF_G + 2 * C * C * 4;        // 2 x { hi, lo } readout operand tiles
  static constexpr int OFF_GX = OFF_BQ + 2 * 2 * BQ_TILE;     // { hi, lo } cross-chunk operand tiles
  static constexpr int OFF_OST = OFF_GX + 2 * GX_TILE;        // 2 x [C][COLS] bf16 output staging
  static constexpr int FAR_LBO = (C / 2) * 16;     // far-push operand: rows = tokens 16..31, K index = tokens 0..15
  static constexpr int FAR_TILE = 2 * FAR_LBO;
  static constexpr int OFF_FAR = OFF_OST + 2 * C * COLS * ES;  // 2 x { hi, lo }
  static constexpr int OFF_P0 = OFF_FAR + 2 * 2 * FAR_TILE;  // [C/4][NROW] float4: a chunk's P0 rows, kept for the rare redo
  static constexpr int OFF_RP = OFF_P0 + C * NROW * 4;  // Temporal: [NROW] fp32, a piece's initial r_prev, helpers -> row warps
  static constexpr int OFF_OS = OFF_RP + (TEMPORAL ? NROW * 4 : 0);  // J = 16: [C][COLS][J] fp32, a chunk's readouts regrouped by output
  // Gated: 2 x [C + 1][NROW] fp32, the running products of a chunk's decays per row: entry t + 1 holds A_t, entry 0
  // is 1 (the pre-decay form of Eq. 3.8 predicts with A_t, the post-decay form of Eq. 3.7 with A_{t-1})
  static constexpr int OFF_A = OFF_OS + (J > 8 ? C * NROW * 4 : 0);
  static constexpr int A_STAGE = (C + 1) * NROW * 4;
  // entry of row (column dl, component j) inside a token's NROW products: component-major, the column index XORed
  // with 8 j so that the J lanes of a column (adjacent row threads) fall into different banks; four consecutive
  // columns of one component stay four consecutive words, which is what the decay warp stores
  __host__ __device__ static constexpr int a_slot(int dl, int j) { return j * COLS + (dl ^ ((8 * j) & (COLS - 1))); }
  static constexpr int OFF_BAR = OFF_A + (GATED ? 2 * A_STAGE : 0);
  static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;  // barriers and three words; + 1024: the kernel aligns its window to 1024 bytes
  static_assert(R_GK % 128 == 0 && RQ_GQ % 128 == 0, "temporal gate rows start 128-byte aligned");
  static_assert(RAW_BYTES % 128 == 0 && RPQ_BYTES % 128 == 0 && R_B % 128 == 0 && R_PK % 128 == 0 && OFF_RAW % 128 == 0 &&
                    OFF_RPQ % 128 == 0 && OFF_TILE % 1024 == 0 && OFF_KU % 1024 == 0 && KU_BYTES % 1024 == 0 && DK % 64 == 0 && (COLS * ES) % 16 == 0 && (GROW * ES) % 16 == 0,
                "destinations of the tensor copies are 128-byte aligned, their rows multiples of 16 bytes");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

// barrier slots.  Committed by the MMA thread: E (state x [K;Q] of a chunk complete), G (Gram batch), U (update of W),
// QD (readouts), FAR (far pushes of a chunk's first 8 tokens).  Completed by the tensor copies: KQ0 / KQ1 (everything
// staged for an even / odd chunk has landed).  Arrived by threads: WP (operand parts of W refreshed, 128 helpers), GS
// (Gram batch spilled, 2 helper warps), C (chunk finished, 128 rows), PQF ([P0|Q0] taken out of tensor memory, 128
// rows), BE (gates of a chunk ready, 128 helpers), OD (outputs of a chunk formed, 128 helpers), T0 (update
// coefficients of a chunk's first 8 tokens stored, 128 rows).
// Gated only: A (running decay products of a chunk in place, 32 lanes of the decay warp).
enum { B_E = 0, B_G, B_U, B_QD, B_KQ0, B_KQ1, B_WP, B_GS, B_C, B_PQF, B_BE, B_OD, B_T0, B_FAR, B_A, B_COUNT };

// bf16 split of FP32 values: hi = bf16(x) (nearest), lo = bf16(x - hi); pairs packed with the first
// value in the low half, which is where the tensor cores expect the even K index.
__device__ __forceinline__ void bf16_split2(float x0, float x1, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  const float r0 = x0 - __uint_as_float(hi << 16), r1 = x1 - __uint_as_float(hi & 0xffff0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(r0, r1);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}
// Three parts (24 bits of the value): for operands whose rounding would otherwise accumulate in the state.
__device__ __forceinline__ void bf16_split3(float x0, float x1, uint32_t &hi, uint32_t &mid, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  const float r0 = x0 - __uint_as_float(hi << 16), r1 = x1 - __uint_as_float(hi & 0xffff0000u);
  const __nv_bfloat162 m = __floats2bfloat162_rn(r0, r1);
  mid = *reinterpret_cast<const uint32_t *>(&m);
  const float s0 = r0 - __uint_as_float(mid << 16), s1 = r1 - __uint_as_float(mid & 0xffff0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(s0, s1);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

// Tensor maps of the six streamed inputs (built by the host for every launch), see chunk_make_maps.
struct ChunkMaps {
  CUtensorMap k, q, v, be, pk, pq;
  CUtensorMap gk, gq;  // Temporal only
};

// Staging of chunk m of a piece by ONE thread: tiled bulk tensor copies (TMA) straight into the operand tile (k, q:
// 64 key dims x 32 tokens per copy, 128-byte swizzle) and into the raw stage (v, gate logits).  Tokens past the end
// of the sequence and columns past Dv are filled with zeros by the copy engine.  Everything lands on `bar`.
template <class Cf>
__device__ __forceinline__ void chunk_stage(const ChunkMaps &maps, unsigned char *tile, unsigned char *ku, unsigned char *raw,
                                            unsigned char *rawpq, int bh, int tok, int col0, int m, uint64_t *bar,
                                            unsigned char *ku_mirror) {
  using namespace umma;
  constexpr int DK = Cf::DK, C = Cf::C;
  fence_async_smem();  // the buffers were last read through ordinary loads
  mbar_arrive_expect_tx(bar, Cf::STAGE_TX_BYTES + (ku_mirror ? C * DK * Cf::ES : 0));
  unsigned char *trow = tile + (m & 1) * 2 * C * 128;  // this chunk's 2C rows of the operand tile
#pragma unroll
  for (int hf = 0; hf < DK / 64; ++hf) {
    tma_load_3d(trow + hf * Cf::TILE_HALF, &maps.k, hf * 64, tok, bh, bar);
    tma_load_3d(trow + hf * Cf::TILE_HALF + C * 128, &maps.q, hf * 64, tok, bh, bar);
    tma_load_3d(ku + hf * Cf::KU_HSTRIDE, &maps.k, hf * 64, tok, bh, bar);
    if (ku_mirror) tma_load_3d(ku_mirror + hf * Cf::KU_HSTRIDE, &maps.k, hf * 64, tok, bh, bar);
  }
  tma_load_3d(raw + Cf::R_V, &maps.v, col0, tok, bh, bar);
  tma_load_4d(raw + Cf::R_B, &maps.be, col0, 0, tok, bh, bar);
  tma_load_4d(raw + Cf::R_PK, &maps.pk, col0, 0, tok, bh, bar);
  tma_load_4d(rawpq, &maps.pq, col0, 0, tok, bh, bar);
  if constexpr (Cf::TEMPORAL) {
    tma_load_3d(raw + Cf::R_GK, &maps.gk, col0, tok, bh, bar);
    tma_load_3d(rawpq + Cf::RQ_GQ, &maps.gq, col0, tok, bh, bar);
  }
}

// RDEBUG: the auxiliary instantiation, which also writes the responsibilities (p.r_debug) and / or adds the sums
// over time of the mixture weights (Sec. 3.5) to p.r_sum, p.r_ent, p.rho_sum, p.rho_ent; each pointer is tested at
// run time there, none of it is in the plain instantiation.
template <class Cf, bool RDEBUG>
__global__ void __launch_bounds__(Cf::NT, 1) swila_chunk_kernel(const __grid_constant__ ScanParams p,
                                                                     const __grid_constant__ ChunkSched sched,
                                                                     const __grid_constant__ ChunkMaps maps) {
  using namespace umma;
  constexpr int J = Cf::J, DK = Cf::DK, C = Cf::C, NROW = Cf::NROW, COLS = Cf::COLS;
  static_assert(!(RDEBUG && J > 8), "the auxiliary outputs for J = 16 come from the scan kernel");
  static_assert(!(RDEBUG && Cf::GATED), "the auxiliary outputs of the Gated variant come from the scan kernel");
  static_assert(!(Cf::GATED && J > 8), "gated rows: J <= 8");
  // Gated: a guard pass has looked at the decays first; if the product over some chunk is so small that quantities
  // taken relative to the chunk's start would overflow, the scan kernel runs this call instead
  if constexpr (Cf::GATED) {
    if (p.guard && *p.guard != 0u) return;
  }
  constexpr bool kOdWaitAtTop = DK == 128;  // where the row warps wait for the helpers' outputs of an earlier chunk
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // the swizzled operand tile needs a 1024-byte aligned shared-memory address
  unsigned char *smem = smem_raw + ((1024u - (umma::smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char *tile = smem + Cf::OFF_TILE;
  float *G_all = reinterpret_cast<float *>(smem + Cf::OFF_G);
  unsigned char *BQ_all = smem + Cf::OFF_BQ;
  unsigned char *GX_all = smem + Cf::OFF_GX;
  __nv_bfloat16 *ostage = reinterpret_cast<__nv_bfloat16 *>(smem + Cf::OFF_OST);
  float4 *p0s = reinterpret_cast<float4 *>(smem + Cf::OFF_P0);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + Cf::OFF_BAR);
  uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + B_COUNT);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nslice = (p.Dv + COLS - 1) / COLS;
  uint32_t *fail_s = tmem_base_s + 1;  // set by any thread whose bounded wait expired: no further piece is started
  // set by a row warp that redid a chunk with the exact E-step: the part of the cross-chunk term that was issued
  // while the chunk still ran used the fast pass's coefficients and is issued again (read and cleared by the MMA thread)
  volatile uint32_t *redo_s = tmem_base_s + 2;
  // this block's run of chunks and the pieces (tile, first chunk, end chunk) it falls into
  const int gang_slice = (int)(blockIdx.x % sched.gang);
  const long long run = blockIdx.x / sched.gang;
  const int npieces = chunk_run_pieces(sched.ntiles, sched.nch, sched.per, run);
  if (warp == 8) tmem_alloc(tmem_base_s, Cf::TM_ALLOC);
  if (tid == 0) { *fail_s = 0; *redo_s = 0; }
  const uint32_t tb_lane = ((uint32_t)((warp & 3) * 32) << 16);  // this warp's lane quarter
  // row served by this thread in either 128-thread role
  const int r = tid & 127;
  const int dl = r / J, j = r % J;
  [[maybe_unused]] const int a_slot = Cf::a_slot(dl, j);  // Gated: this row's entry in a token's decay products

#pragma unroll 1
  for (int pi = 0; pi < npieces; ++pi) {
    // the piece being processed (uniform over the block); the order of a run's pieces is chunk_run_piece's
    const ChunkPiece piece = chunk_run_piece(sched.ntiles, sched.nch, sched.per, run, pi);
    const int tl = piece.unit, cb = piece.cb, ce = piece.ce;
    const int bh = sched.gang > 1 ? tl : tl / nslice;
    const int col0 = (sched.gang > 1 ? gang_slice : tl - bh * nslice) * COLS;
    const int nchunks = ce - cb;
    const int Tseg = min(p.T, ce * C) - cb * C;
    const size_t tok0 = (size_t)bh * p.T + (size_t)cb * C;
    const int tseg0 = cb * C;  // first token of the piece inside its sequence
    const bool from_flag = cb > 0, to_flag = ce < sched.nch;  // state handed over from / to another block
    unsigned *const flag = sched.flags + (sched.gang > 1 ? tl * sched.gang + gang_slice : tl);
    const int col = col0 + dl;
    const bool col_ok = col < p.Dv;
    bool failed = false;
    // the same for a warp that is in nobody's way as long as it does not compete for issue slots: it sleeps between polls
    [[maybe_unused]] auto bwait_idle = [&](int b, uint32_t parity) -> bool {
      const unsigned long long t_begin = global_timer_ns();
      while (!mbar_try_wait(&bars[b], parity)) {
        if (global_timer_ns() - t_begin > 2000000000ull) {
          atomicCAS(&g_chunk_error, 0, (int)((warp + 1) * 65536 + (smem_u32(&bars[b]) & 0xffffu)));
          return false;
        }
        __nanosleep(200);
      }
      return true;
    };
  if (pi > 0) {  // every barrier of the previous piece is quiescent: all its phases were waited for
    __syncthreads();
    if (tid == 0) {
      for (int b = 0; b < B_COUNT; ++b) mbar_inval(&bars[b]);
    }
  }
  if (tid == 0) {
    mbar_init(&bars[B_E], 1);
    mbar_init(&bars[B_G], 1);
    mbar_init(&bars[B_U], 1);
    mbar_init(&bars[B_QD], 1);
    mbar_init(&bars[B_KQ0], 1);  // the thread that issues the tensor copies
    mbar_init(&bars[B_KQ1], 1);
    mbar_init(&bars[B_WP], 128);
    mbar_init(&bars[B_GS], 64);
    mbar_init(&bars[B_C], 128);
    mbar_init(&bars[B_PQF], 128);
    mbar_init(&bars[B_BE], 128);
    mbar_init(&bars[B_OD], 128);
    mbar_init(&bars[B_T0], 128);
    mbar_init(&bars[B_FAR], 1);
    mbar_init(&bars[B_A], 32);
    mbar_fence_init();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (*fail_s) break;
  const uint32_t tb0 = *tmem_base_s;
  const uint32_t tb = tb0 + tb_lane;

  // outputs of one chunk (Eq. 3.5): o_td = sum_j pi^q_j (w_t.q_t)_j, pi^q = softmax over the J
  // components of a column
  [[maybe_unused]] float rho_run = 1.0f / J;  // helper lanes, Temporal: running average of the query-side prior (App. B.3)
  [[maybe_unused]] float sq_sum[J], sq_ent = 0.f;  // helper lanes, auxiliary instantiation: slot c = component j ^ pattern(c)
#pragma unroll
  for (int c = 0; c < J; ++c) sq_sum[c] = 0.f;
  auto write_outputs = [&](int n) {
    const int t0 = n * C;
    const int nvalid = min(C, Tseg - t0);
    const __nv_bfloat16 *rpq = reinterpret_cast<const __nv_bfloat16 *>(smem + Cf::OFF_RPQ + (n % 3) * Cf::RPQ_BYTES);
    __nv_bfloat16 *ost = ostage + (n & 1) * C * COLS;
    tc_fence_after_sync();
#pragma unroll 1
    for (int tg = 0; tg < C; tg += 8) {  // rolled: the loop body stays resident in the instruction cache
      // This lane's readouts of 8 tokens (own component j) are transposed inside the J-lane group of the
      // column, one exchange round per bit of j, so that the lane ends up with all J components of 8/J
      // tokens and forms their outputs without any further exchange.
      constexpr int LJ = (J == 4) ? 2 : 3;
      float hq[8];
      tmem_ld8(tb + Cf::TM_QD + (n & 1) * C + tg, hq);
      tmem_ld_wait();
      if constexpr (Cf::GATED) {
        // the readouts were accumulated in units of the chunk's start: w_t.q_t = A_t (w_0.q_t + sum_{s<=t} (c_s / A_s) k_s.q_t)
        const float *As = reinterpret_cast<const float *>(smem + Cf::OFF_A + (n & 1) * Cf::A_STAGE);
#pragma unroll
        for (int i = 0; i < 8; ++i) hq[i] *= As[(tg + i + 1) * NROW + a_slot];
      }
      if constexpr (Cf::TEMPORAL) {
        // readout weight of this lane's own component: rho_t = (1 - g) rho_{t-1} + g pi^q_t, g = sigmoid(gq logit),
        // a running average along the tokens, so it is applied before the transposition
        const __nv_bfloat16 *rgq = reinterpret_cast<const __nv_bfloat16 *>(reinterpret_cast<const unsigned char *>(rpq) + Cf::RQ_GQ);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int t = tg + i;
          float x[J], mx = -3.0e38f;
#pragma unroll
          for (int jj = 0; jj < J; ++jj) {
            x[jj] = __bfloat162float(rpq[(t * J + jj) * Cf::GROW + dl]) * kLog2e;
            mx = fmaxf(mx, x[jj]);
          }
          const float own = __bfloat162float(rpq[(t * J + j) * Cf::GROW + dl]) * kLog2e;
          const float eo = ex2_approx(own - mx);
          float se = eo;
#pragma unroll
          for (int off = 1; off < J; off <<= 1) se += __shfl_xor_sync(0xffffffffu, se, off);
          const float pq = eo * rcp_approx(se);
          const float gq = sigmoid_approx(__bfloat162float(rgq[t * COLS + dl]));
          if (t < nvalid) rho_run = fmaf(gq, pq - rho_run, rho_run);
          hq[i] *= rho_run;
          if constexpr (RDEBUG) {
            // sums over time of the readout weights (this lane: its own component) and of their entropy over the
            // components (bits; summed over the J lanes of the column, kept by every lane, added once at the end)
            float hb = rho_run > 0.f ? rho_run * lg2_approx(rho_run) : 0.f;
#pragma unroll
            for (int off = 1; off < J; off <<= 1) hb += __shfl_xor_sync(0xffffffffu, hb, off);
            if (t < nvalid) {
              sq_sum[0] += rho_run;
              sq_ent -= hb;
            }
          }
        }
      }
      if constexpr (J > 8) {
        // More components than tokens in a trip: no transposition inside the lane group.  The readouts (Temporal:
        // already weighted) go to shared memory grouped by output, [token][column][component]: a warp's 32 lanes
        // (2 columns x 16 components) write 32 consecutive floats per token; the outputs are formed below.
        float *os = reinterpret_cast<float *>(smem + Cf::OFF_OS);
#pragma unroll
        for (int i = 0; i < 8; ++i) os[((tg + i) * COLS + dl) * J + j] = hq[i];
        continue;
      }
#pragma unroll
      for (int rd = 0; rd < LJ; ++rd) {
        const int nrem = 3 - rd;              // token bits still in the index
        const int m = J >> (rd + 1);          // partner lane distance
        const bool mybit = (j & m) != 0;
        float g[8];
#pragma unroll
        for (int c = 0; c < (1 << rd); ++c) {
#pragma unroll
          for (int rest = 0; rest < (1 << (nrem - 1)); ++rest) {
            const float lo = hq[(c << nrem) | rest], hi = hq[(c << nrem) | (1 << (nrem - 1)) | rest];
            const float keep = mybit ? hi : lo, send = mybit ? lo : hi;
            const float recv = __shfl_xor_sync(0xffffffffu, send, m);
            g[(((c << 1) | 0) << (nrem - 1)) | rest] = keep;
            g[(((c << 1) | 1) << (nrem - 1)) | rest] = recv;
          }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) hq[i] = g[i];
      }
      // hq[(c << (3 - LJ)) | rest]: token tg + (j << (3 - LJ)) + rest, component j ^ pattern(c), where bit
      // (LJ - 1 - rd) of c says whether the value came from the partner of round rd
#pragma unroll
      for (int rest = 0; rest < (8 >> LJ); ++rest) {
        const int tl = tg + (j << (3 - LJ)) + rest;
        if constexpr (Cf::TEMPORAL) {  // the readouts arrive weighted: the output is their plain sum over the components
          float so = 0.f;
#pragma unroll
          for (int c = 0; c < J; ++c) so += hq[(c << (3 - LJ)) | rest];
          ost[tl * COLS + dl] = __float2bfloat16_rn(so);
          continue;
        }
        float x[J];
        [[maybe_unused]] float ex[J];
        float mx = -3.0e38f;
#pragma unroll
        for (int c = 0; c < J; ++c) {
          int pat = 0;
#pragma unroll
          for (int rd = 0; rd < LJ; ++rd) pat |= ((c >> (LJ - 1 - rd)) & 1) ? (J >> (rd + 1)) : 0;
          x[c] = __bfloat162float(rpq[(tl * J + (j ^ pat)) * Cf::GROW + dl]) * kLog2e;
          mx = fmaxf(mx, x[c]);
        }
        float se = 0.f, so = 0.f;
#pragma unroll
        for (int c = 0; c < J; ++c) {
          const float e = ex2_approx(x[c] - mx);
          if constexpr (RDEBUG) ex[c] = e;
          se += e;
          so = fmaf(e, hq[(c << (3 - LJ)) | rest], so);
        }
        const float ise = rcp_approx(se);
        ost[tl * COLS + dl] = __float2bfloat16_rn(so * ise);
        if constexpr (RDEBUG) {
          // sums over time of the readout weights and of their entropy (bits): log2 p_c = x_c - mx - log2(se)
          if (tl < nvalid) {
            float hb = 0.f;
#pragma unroll
            for (int c = 0; c < J; ++c) {
              const float pc = ex[c] * ise;
              sq_sum[c] += pc;
              if (pc > 0.f) hb = fmaf(pc, x[c] - mx, hb);
            }
            sq_ent += lg2_approx(se) - hb;
          }
        }
      }
    }
    if constexpr (J > 8) {
      // one thread per output (C x COLS = 256 of them): its J readouts are 4 vector loads, the softmax over the
      // components of Eq. 3.5 is local (shuffle sums over 16 lanes cost several times as much)
      named_bar_sync(2, 128);
      const float *os = reinterpret_cast<const float *>(smem + Cf::OFF_OS);
      for (int e = r; e < C * COLS; e += 128) {
        const int t = e / COLS, d = e - t * COLS;
        float val[J];
#pragma unroll
        for (int c4 = 0; c4 < J / 4; ++c4) {
          const float4 v4 = *reinterpret_cast<const float4 *>(os + e * J + c4 * 4);
          val[4 * c4] = v4.x; val[4 * c4 + 1] = v4.y; val[4 * c4 + 2] = v4.z; val[4 * c4 + 3] = v4.w;
        }
        float out = 0.f;
        if constexpr (Cf::TEMPORAL) {
#pragma unroll
          for (int jj = 0; jj < J; ++jj) out += val[jj];
        } else {
          float x[J], mx = -3.0e38f;
#pragma unroll
          for (int jj = 0; jj < J; ++jj) {
            x[jj] = __bfloat162float(rpq[(t * J + jj) * Cf::GROW + d]) * kLog2e;
            mx = fmaxf(mx, x[jj]);
          }
          float se = 0.f;
#pragma unroll
          for (int jj = 0; jj < J; ++jj) {
            const float ex = ex2_approx(x[jj] - mx);
            se += ex;
            out = fmaf(ex, val[jj], out);
          }
          out *= rcp_approx(se);
        }
        ost[t * COLS + d] = __float2bfloat16_rn(out);
      }
    }
    tc_fence_before_sync();
    named_bar_sync(2, 128);
    constexpr int GROUPS = COLS / 8;  // 8 outputs = 16 bytes per store
    for (int e = r; e < C * GROUPS; e += 128) {
      const int t = e / GROUPS, g8 = e - t * GROUPS;
      if (t < nvalid && col0 + g8 * 8 < p.Dv)
        *reinterpret_cast<uint4 *>((__nv_bfloat16 *)p.o + (tok0 + (size_t)(t0 + t)) * p.Dv + col0 + g8 * 8) =
            *reinterpret_cast<const uint4 *>(ost + t * COLS + g8 * 8);
    }
  };

  if (warp < 4) {
    // =============================== row warps ===============================================
    const int jbase = lane - j;
    [[maybe_unused]] float st_r = 0.f, st_h = 0.f;  // auxiliary instantiation: this piece's sums over time
    if (!mbar_wait(&bars[B_BE], 0) || !mbar_wait(&bars[B_GS], 0)) failed = true;
    [[maybe_unused]] float rprev = 1.0f / J;  // Temporal: this row's previous responsibility r_{t-1} (App. B.3)
    // Gated: the product of this row's decays over the previous chunk of the piece.  What the tensor cores hand over
    // for a chunk, W_n [K;Q]^T + Cmat'_{n-1} (K_{n-1} [K;Q]^T), is in units of the state at the START of chunk n-1.
    [[maybe_unused]] float acarry = 1.0f;
    [[maybe_unused]] const int a_off = p.post ? 0 : 1;  // entry of the running products that a token's prediction uses
    if constexpr (Cf::TEMPORAL) rprev = reinterpret_cast<const float *>(smem + Cf::OFF_RP)[r];
#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const int t0 = n * C;
      const int nvalid = min(C, Tseg - t0);
      const unsigned char *raw = smem + Cf::OFF_RAW + (n & 1) * Cf::RAW_BYTES;
      const __nv_bfloat16 *rv = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_V);
      const float *bes = reinterpret_cast<const float *>(raw + Cf::R_B);
      const __nv_bfloat16 *rpk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_PK);
      [[maybe_unused]] const float *pks = reinterpret_cast<const float *>(raw + Cf::R_PK);            // Temporal: normalised prior
      [[maybe_unused]] const __nv_bfloat16 *rgk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_GK);  // Temporal: gate logits
      const float *Gkk = G_all + (n & 1) * C * C;
      [[maybe_unused]] const float *As = reinterpret_cast<const float *>(smem + Cf::OFF_A + (n & 1) * Cf::A_STAGE);

      if (!mbar_wait(&bars[B_E], n & 1)) { failed = true; break; }
      tc_fence_after_sync();
      // the readout buffer this chunk seeds below was last read by the helpers for the outputs of chunk n-2.  At
      // Dk = 128 they finish those about when chunk n-1 ends, so the wait sits here, where it has long been met; at
      // Dk = 64 they are early and the wait is cheaper at the hand-over below (both placements measured)
      if constexpr (kOdWaitAtTop) {
        if (n >= 2 && !mbar_wait(&bars[B_OD], n & 1)) { failed = true; break; }
      }
      // [P0 | Q0] out of tensor memory: P0 to registers, Q0 seeds the readout accumulator of this chunk;
      // then the tensor cores may overwrite the region with the next chunk's products
      float pred0[C];
#pragma unroll
      for (int cc = 0; cc < C / 16; ++cc) {
        float a[16], b[16];
        tmem_ld16(tb + Cf::TM_PQ + cc * 16, a);
        tmem_ld16(tb + Cf::TM_PQ + C + cc * 16, b);
        tmem_ld_wait();
        if constexpr (Cf::GATED) {
#pragma unroll
          for (int i = 0; i < 16; ++i) { a[i] *= acarry; b[i] *= acarry; }
        }
        tmem_st16(tb + Cf::TM_QD + (n & 1) * C + cc * 16, b);
#pragma unroll
        for (int i = 0; i < 16; ++i) pred0[cc * 16 + i] = a[i];
#pragma unroll
        for (int i = 0; i < 4; ++i)  // copy for the redo path, so that the values need not stay in registers
          p0s[((cc * 4 + i) * NROW + r)] = make_float4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&bars[B_PQF]);

      // ---- sequential part of the chunk: E-step and the triangular key-side corrections.  Only one FMA
      //      of a token's push (into the next token's prediction) sits on the serial chain; the rest is
      //      deferred into the shuffle latency of the next token's E-step.
      //      FAST: exponentials are taken without subtracting the per-token maximum; the pass reports whether
      //      any normaliser left the safe range (all components > ~13 standard deviations off, or extreme
      //      prior logits), in which case the chunk is redone with the maximum subtracted. ----
      [[maybe_unused]] float chunk_r = 0.f, chunk_h = 0.f;  // written by the pass whose results stand
      [[maybe_unused]] float chunk_rp = 0.f;                 // Temporal: r of the chunk's last token, likewise
      auto sequential = [&](auto exact_tag, [[maybe_unused]] const float rp_in) -> bool {
        constexpr bool EXACT = decltype(exact_tag)::value;
        [[maybe_unused]] float rp = rp_in;
        constexpr int GT = Cf::GT;
        bool bad = false;
        [[maybe_unused]] float cr = 0.f, ch = 0.f;  // auxiliary instantiation: this chunk's sums of r and of r log2 r
        // P(i): v - prediction (the prediction error so far) of token tg + i of the current trip, for the WINS
        // tokens that the pushes of a token reach on the ALUs (slots past the chunk end are dead weight that keeps the
        // trip's code independent of tg); the Gram rows are stored negated, so a push is one FMA and the error of
        // the next token is ready without a subtraction on the serial chain.  The fast pass reaches WIN = 24 tokens:
        // the pushes of tokens 0-7 into tokens 24-31 come from the tensor cores (FAR) when token 24 is reached.
        // The redo pass does everything itself.
        constexpr int WINS = EXACT ? C : Cf::WIN;
        // (held as pairs: the deferred pushes below are packed two-wide FMAs, half the instructions)
        float2 pred2[WINS / 2];
        auto P = [&](int k) -> float & { return (k & 1) ? pred2[k >> 1].y : pred2[k >> 1].x; };
#pragma unroll
        for (int t = 0; t < WINS; ++t) {
          // Gated: the window holds minus the prediction in units of the chunk's start; the decay and v enter per token
          if constexpr (Cf::GATED) P(t) = -pred0[t];
          else P(t) = __bfloat162float(rv[t * COLS + dl]) - pred0[t];
        }
        [[maybe_unused]] float p0late[C - Cf::WIN];
        if constexpr (!EXACT) {
#pragma unroll
          for (int t = 0; t < C - Cf::WIN; ++t) {
            if constexpr (Cf::GATED) p0late[t] = -pred0[Cf::WIN + t];
            else p0late[t] = __bfloat162float(rv[(Cf::WIN + t) * COLS + dl]) - pred0[Cf::WIN + t];
          }
        }
        float c_prev = 0.f;
#pragma unroll 1
        for (int tg = 0; tg < C; tg += GT) {
          if constexpr (!EXACT) {
            if (tg == Cf::WIN) {  // far pushes of tokens 0-6 into tokens 24-31
              if (!mbar_wait(&bars[B_FAR], n & 1)) failed = true;
              tc_fence_after_sync();
              float far[8];
              tmem_ld8(tb + Cf::TM_FAR + Cf::WIN - C / 2, far);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) P(i) -= far[i];
            }
          }
          float cs[GT];
#pragma unroll
          for (int i = 0; i < GT; ++i) {
            const int t = tg + i;
            const float be = bes[t * NROW + r];
            // serial chain: prediction error -> responsibilities (Eq. 3.4) -> update coefficient (Eq. 3.3)
            // Gated: delta = v - A (w_0.k + sum_s (c_s / A_s) k_s.k), A = the row's decay product up to this token
            // (pre-decay, Eq. 3.8) or up to the previous one (post-decay, Eq. 3.7); beta arrives divided by A_t, so
            // that the coefficient below is already c_t / A_t
            float delta;
            if constexpr (Cf::GATED) delta = fmaf(As[(t + a_off) * NROW + a_slot], P(i), __bfloat162float(rv[t * COLS + dl]));
            else delta = P(i);
            float a;
            if constexpr (Cf::TEMPORAL) {
              // key-side prior (1 - g) r_{t-1} + g pi^k with g = sigmoid(gk logit) (App. B.3): a convex combination of
              // two distributions over j, so it needs no further normalisation
              const float gk = sigmoid_approx(__bfloat162float(rgk[t * COLS + dl]));
              const float prior = fmaf(gk, pks[t * NROW + r] - rp, rp);
              a = fmaf(-kHalfLog2e * delta, delta, lg2_approx(prior));
            } else {
              a = fmaf(-kHalfLog2e * delta, delta, __bfloat162float(rpk[(t * J + j) * Cf::GROW + dl]) * kLog2e);
            }
            float e, sum;
            if constexpr (EXACT) {
              float all[J];
#pragma unroll
              for (int jj = 0; jj < J; ++jj) all[jj] = __shfl_sync(0xffffffffu, a, jbase + jj);
              float m = all[0];
#pragma unroll
              for (int jj = 1; jj < J; ++jj) m = fmaxf(m, all[jj]);
              sum = 0.f;
#pragma unroll
              for (int jj = 0; jj < J; ++jj) sum += ex2_approx(all[jj] - m);
              e = ex2_approx(a - m);
            } else {
              e = ex2_approx(a);
              if constexpr (J <= 8) {
                float part[J];  // the other components' terms arrive together: add them as a tree
                part[0] = e;
#pragma unroll
                for (int jj = 1; jj < J; ++jj) part[jj] = __shfl_sync(0xffffffffu, e, jbase + ((j + jj) & (J - 1)));
#pragma unroll
                for (int w = J / 2; w >= 1; w /= 2) {
#pragma unroll
                  for (int jj = 0; jj < w; ++jj) part[jj] += part[jj + w];
                }
                sum = part[0];
              } else {  // 15 shuffles per token cost more than the latency of 4 dependent rounds
                sum = e;
#pragma unroll
                for (int off = 1; off < J; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
              }
              bad = bad || !(sum > 1e-30f && sum < 1e30f);
            }
            {  // deferred push of token t-1 into the predictions of tokens t+1 .. (slots i+1 ..)
              const float4 *gp = reinterpret_cast<const float4 *>(Gkk + max(t - 1, 0) * C + tg);
#pragma unroll
              for (int u4 = (i + 1) / 4; u4 < WINS / 4; ++u4) {
                const float4 g = gp[u4];
                const float2 cc = make_float2(c_prev, c_prev);
                if (4 * u4 + 0 > i) pred2[2 * u4] = __ffma2_rn(cc, make_float2(g.x, g.y), pred2[2 * u4]);
                else if (4 * u4 + 1 > i) pred2[2 * u4].y = fmaf(c_prev, g.y, pred2[2 * u4].y);
                if (4 * u4 + 2 > i) pred2[2 * u4 + 1] = __ffma2_rn(cc, make_float2(g.z, g.w), pred2[2 * u4 + 1]);
                else if (4 * u4 + 3 > i) pred2[2 * u4 + 1].y = fmaf(c_prev, g.w, pred2[2 * u4 + 1].y);
              }
            }
            const float rs = rcp_approx(sum);
            float c = ((be * delta) * e) * rs;  // beta r delta with one multiplication after the reciprocal
            if constexpr (Cf::TEMPORAL) {
              if (t < nvalid) rp = e * rs;
            }
            // (padding tokens of the last chunk have beta = 0 and leave the state alone)
            cs[i] = c;
            if constexpr (RDEBUG) {
              const float rr = e * rs;
              if (p.r_debug && col_ok && t < nvalid) p.r_debug[((tok0 + (size_t)(t0 + t)) * J + j) * p.Dv + col] = rr;
              if (t < nvalid) {  // log2 r = log2 e - log2(sum); a component whose responsibility underflowed adds nothing
                cr += rr;
                if (rr > 0.f) ch = fmaf(rr, lg2_approx(e) - lg2_approx(sum), ch);
              }
            }
            P(i + 1) = fmaf(c, Gkk[t * C + t + 1], P(i + 1));  // the push the next token waits for
            c_prev = c;
          }
          // the coefficient columns are still operands of the previous chunk's update and readout MMAs until
          // those complete (normally long before the first trip ends)
          if (tg == 0 && n > 0) {
            if (!mbar_wait(&bars[B_QD], (n - 1) & 1)) failed = true;
          }
          {  // GT update coefficients complete: park their bf16 parts in tensor memory, two tokens per column
            uint32_t hi[GT / 2], lo[GT / 2], l3[GT / 2];
#pragma unroll
            for (int i = 0; i < GT / 2; ++i) bf16_split3(cs[2 * i], cs[2 * i + 1], hi[i], lo[i], l3[i]);
            tmem_st4(tb + Cf::TM_CHI + tg / 2, hi);
            tmem_st4(tb + Cf::TM_CLO + tg / 2, lo);
            tmem_st4(tb + Cf::TM_CL3 + tg / 2, l3);
          }
          if constexpr (!EXACT) {
            // the coefficients of tokens 0-15 are in place: the far pushes (of tokens 0-7, needed at token 24) and the
            // first half of the cross-chunk term may be issued
            if (tg == GT) {
              tmem_st_wait();
              tc_fence_before_sync();
              mbar_arrive(&bars[B_T0]);
            }
          }
#pragma unroll
          for (int i = 0; i + GT < WINS; i += 2) pred2[i / 2] = pred2[(i + GT) / 2];
#pragma unroll
          for (int i = 0; i < GT; ++i) {  // the slots that enter the window: tokens 24-31 after the first trip, dead later
            if constexpr (EXACT) {
              P(WINS - GT + i) = 0.f;
            } else {
              P(WINS - GT + i) = p0late[i];
              p0late[i] = 0.f;
            }
          }
        }
        if constexpr (RDEBUG) { chunk_r = cr; chunk_h = ch; }
        if constexpr (Cf::TEMPORAL) chunk_rp = rp;
        return bad;
      };
      const bool unsafe = sequential(std::false_type{}, rprev);
      if (__any_sync(0xffffffffu, unsafe)) {
        if (lane == 0) *redo_s = 1;
        tmem_st_wait();
#pragma unroll
        for (int i = 0; i < C / 4; ++i) {  // P0 again, from the copy in shared memory
          const float4 v4 = p0s[i * NROW + r];
          pred0[4 * i] = v4.x; pred0[4 * i + 1] = v4.y; pred0[4 * i + 2] = v4.z; pred0[4 * i + 3] = v4.w;
        }
        sequential(std::true_type{}, rprev);
      }
      if constexpr (Cf::TEMPORAL) rprev = chunk_rp;
      if constexpr (Cf::GATED) acarry = As[C * NROW + a_slot];
      if constexpr (RDEBUG) { st_r += chunk_r; st_h += chunk_h; }
      tmem_st_wait();
      tc_fence_before_sync();
      // what the next steps rely on must be in place before this chunk is handed over (this also keeps every
      // barrier at most one phase ahead of its waiters): gates and Gram rows of chunk n+1
      if (n + 1 < nchunks && (!mbar_wait(&bars[B_BE], (n + 1) & 1) || !mbar_wait(&bars[B_GS], (n + 1) & 1))) failed = true;
      if constexpr (!kOdWaitAtTop) {
        if (n > 0 && !mbar_wait(&bars[B_OD], (n - 1) & 1)) failed = true;
      }
      mbar_arrive(&bars[B_C]);
    }
    // ---- final state row -> global ----
    if (!failed && !mbar_wait(&bars[B_U], (nchunks - 1) & 1)) failed = true;
    if (!failed && p.W_out && col_ok) {
      tc_fence_after_sync();
      float *dst = p.W_out + (((size_t)bh * J + j) * p.Dv + col) * DK;
#pragma unroll
      for (int cc = 0; cc < DK / 16; ++cc) {
        float w[16];
        tmem_ld16(tb + Cf::TM_W + cc * 16, w);
        tmem_ld_wait();
        if constexpr (Cf::GATED) {  // the last update left the state in units of the last chunk's start
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] *= acarry;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
          __stcs(reinterpret_cast<float4 *>(dst + cc * 16 + i * 4), make_float4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]));
      }
    }
    if constexpr (RDEBUG) {
      if (!failed && col_ok) {  // other pieces of the tile may run in other blocks: atomic additions
        constexpr float kLn2 = 0.6931471805599453f;
        if (p.r_sum) atomicAdd(p.r_sum + ((size_t)bh * J + j) * p.Dv + col, st_r);
        if (p.r_ent) atomicAdd(p.r_ent + (size_t)bh * p.Dv + col, -st_h * kLn2);
      }
    }
    if constexpr (Cf::TEMPORAL) {
      if (!failed && p.r_out && col_ok) p.r_out[((size_t)bh * J + j) * p.Dv + col] = rprev;
    }
    if (to_flag) {  // the rest of this tile belongs to another block: publish the state
      __threadfence();
      if constexpr (Cf::TEMPORAL) named_bar_sync(5, 256);  // ... the helpers' part of it included
      else named_bar_sync(4, 128);
      if (r == 0 && !failed) st_release_gpu(flag, sched.epoch);
    }
  } else if (warp < 8) {
    // =============================== helper warps ============================================
    const int h = r;
    // beta = sigmoid(logit) of this helper's row for every token of a raw stage (App. B.2), written over the
    // logits, 8 tokens per pass (rolled: less code in the instruction cache), last tokens first: a token's FP32
    // row (512 bytes) lies further into the region than its logits (at most 384 bytes), so a pass overwrites only
    // logits of its own tokens -- which every helper has read by the barrier -- and of later, finished ones
    // Tokens past the end of the sequence (the last chunk's padding) get beta = 0: their update coefficient is then
    // zero by itself and the row warps need no test on their serial chain.
    auto cook_be = [&](unsigned char *raw, const int nvalid, [[maybe_unused]] const float *As) {
      const __nv_bfloat16 *rb = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_B);
      float *bes = reinterpret_cast<float *>(raw + Cf::R_B);
      static_assert(J * Cf::GROW * Cf::ES <= NROW * 4, "a token's logits end before its FP32 row does");
#pragma unroll 1
      for (int t8 = C - 8; t8 >= 0; t8 -= 8) {
        float be[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          be[i] = sigmoid_approx(__bfloat162float(rb[((t8 + i) * J + j) * Cf::GROW + dl]));
          // Gated: beta / A_t, so that the row warps' coefficient is c_t / A_t without a further operation
          if constexpr (Cf::GATED) be[i] *= rcp_approx(As[(t8 + i + 1) * NROW + a_slot]);
          if (t8 + i >= nvalid) be[i] = 0.f;
        }
        named_bar_sync(3, 128);
#pragma unroll
        for (int i = 0; i < 8; ++i) bes[(t8 + i) * NROW + h] = be[i];
      }
    };
    // Temporal: the key-side prior pi^k = softmax over the J components (App. B.2), written over the logits as fp32
    // [C][NROW] in the same rolled, last-tokens-first passes as beta.  The J lanes of a column share the work by
    // token: a lane takes the whole softmax of 8 / J tokens of the pass and writes all J values of each (one or two
    // 16-byte stores), instead of every lane taking one exponential of every token plus a shuffle sum.
    [[maybe_unused]] auto cook_pk = [&](unsigned char *raw) {
      const __nv_bfloat16 *rk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_PK);
      float *pks = reinterpret_cast<float *>(raw + Cf::R_PK);
      constexpr int TPL = (J <= 8) ? 8 / J : 1;  // tokens per lane and pass (J = 16: lanes 8..15 of a column idle)
#pragma unroll 1
      for (int t8 = C - 8; t8 >= 0; t8 -= 8) {
        float pk[TPL][J];
#pragma unroll
        for (int i = 0; i < TPL; ++i) {
          const int t = t8 + (j * TPL + i) % 8;
          float mx = -3.0e38f;
#pragma unroll
          for (int jj = 0; jj < J; ++jj) {
            pk[i][jj] = __bfloat162float(rk[(t * J + jj) * Cf::GROW + dl]) * kLog2e;
            mx = fmaxf(mx, pk[i][jj]);
          }
          float se = 0.f;
#pragma unroll
          for (int jj = 0; jj < J; ++jj) {
            pk[i][jj] = ex2_approx(pk[i][jj] - mx);
            se += pk[i][jj];
          }
          const float inv = rcp_approx(se);
#pragma unroll
          for (int jj = 0; jj < J; ++jj) pk[i][jj] *= inv;
        }
        named_bar_sync(3, 128);
        if (J <= 8 || j < 8) {
#pragma unroll
          for (int i = 0; i < TPL; ++i) {
            const int t = t8 + (j * TPL + i) % 8;
#pragma unroll
            for (int c4 = 0; c4 < J / 4; ++c4)
              *reinterpret_cast<float4 *>(pks + t * NROW + dl * J + c4 * 4) =
                  make_float4(pk[i][4 * c4], pk[i][4 * c4 + 1], pk[i][4 * c4 + 2], pk[i][4 * c4 + 3]);
          }
        }
      }
    };
    // operand parts of W after an update, this helper's tensor-memory lane
    auto refresh_parts = [&]([[maybe_unused]] const float decay) {
#pragma unroll 2
      for (int cc = 0; cc < DK / 16; ++cc) {
        float w[16];
        uint32_t hi[8], lo[8];
        tmem_ld16(tb + Cf::TM_W + cc * 16, w);
        tmem_ld_wait();
        if constexpr (Cf::GATED) {  // the update was taken in units of the chunk's start: now the chunk's decay
#pragma unroll
          for (int i = 0; i < 16; ++i) w[i] *= decay;
          tmem_st16(tb + Cf::TM_W + cc * 16, w);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) bf16_split2(w[2 * i], w[2 * i + 1], hi[i], lo[i]);
        tmem_st8(tb + Cf::TM_WHI + cc * 8, reinterpret_cast<const float(&)[8]>(hi));
        tmem_st8(tb + Cf::TM_WLO + cc * 8, reinterpret_cast<const float(&)[8]>(lo));
      }
      tmem_st_wait();
      tc_fence_before_sync();
    };
    // 32 FP32 values of this lane's Gram row -> bf16 hi / lo operand units (row `row` of a tile with `lbo`)
    auto store_parts = [&](const float (&x)[C], unsigned char *thi, unsigned char *tlo, int lbo, int row) {
#pragma unroll
      for (int c = 0; c < C / 8; ++c) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) bf16_split2(x[8 * c + 2 * i], x[8 * c + 2 * i + 1], hi[i], lo[i]);
        *reinterpret_cast<uint4 *>(thi + c * lbo + row * 16) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        *reinterpret_cast<uint4 *>(tlo + c * lbo + row * 16) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    };
    // The Gram batch of chunk m is [K_e;Q_e;K_o;Q_o] x [K_{m-1} | K_m]^T (in that order in tensor memory); the two helper warps whose
    // tensor-memory lanes hold the rows of chunk m's keys and queries spill it:
    //   key rows   (lane s):  -K_m K_m^T as plain FP32 rows for the row warps (negated: they track v - prediction);
    //   query rows (lane t):  Q_m K_m^T, causally masked (s <= t), as the hi / lo operand of the readout MMA;
    //   both:                 [K_m;Q_m] K_{m-1}^T as the hi / lo operand of the cross-chunk MMA.
    auto spill_gram = [&](int m) {
      const bool qrows = (warp & 1) != 0;
      float a[C];
#pragma unroll
      for (int cc = 0; cc < C / 16; ++cc) tmem_ld16(tb + Cf::TM_G + C + cc * 16, reinterpret_cast<float(&)[16]>(a[cc * 16]));
      tmem_ld_wait();
      if (!qrows) {
        float *Gkk = G_all + (m & 1) * C * C;
#pragma unroll
        for (int i = 0; i < C / 4; ++i)
          *reinterpret_cast<float4 *>(Gkk + lane * C + i * 4) = make_float4(-a[4 * i], -a[4 * i + 1], -a[4 * i + 2], -a[4 * i + 3]);
        // far-push operand: row = token u = lane (16..31), K index = tokens 0..7 (K K^T is symmetric, so this lane's
        // row holds k_s.k_u).  Through the tensor cores go the pushes of tokens s = 0..6 into tokens u >= WIN: the row
        // warps push token s into tokens s+1 .. 23 while they are in the first trip, and token 7, whose deferred push
        // runs in the second trip, reaches token 31 there.  Everything else in the operand is zero.
        if (lane >= C / 2) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const bool use = lane >= Cf::WIN;
            bf16_split2(use ? a[2 * i] : 0.f, (use && 2 * i + 1 < Cf::GT - 1) ? a[2 * i + 1] : 0.f, hi[i], lo[i]);
          }
          unsigned char *ft = smem + Cf::OFF_FAR + (m & 1) * 2 * Cf::FAR_TILE;
          *reinterpret_cast<uint4 *>(ft + (lane - C / 2) * 16) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4 *>(ft + Cf::FAR_TILE + (lane - C / 2) * 16) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      } else {
#pragma unroll
        for (int s = 0; s < C; ++s) a[s] = (s <= lane) ? a[s] : 0.f;
        unsigned char *bq = BQ_all + (m & 1) * 2 * Cf::BQ_TILE;
        store_parts(a, bq, bq + Cf::BQ_TILE, Cf::BQ_LBO, lane);
      }
      if (m > 0) {
#pragma unroll
        for (int cc = 0; cc < C / 16; ++cc)
          tmem_ld16(tb + Cf::TM_G + cc * 16, reinterpret_cast<float(&)[16]>(a[cc * 16]));
        tmem_ld_wait();
        store_parts(a, GX_all, GX_all + Cf::GX_TILE, Cf::GX_LBO, (qrows ? C : 0) + lane);
      }
      tc_fence_before_sync();
      fence_async_smem();
    };
    const bool spill_mine[2] = {warp < 6, warp >= 6};  // which parity of chunks this warp's lanes hold

    // ---- prologue: stage chunks 0 and 1, state row -> tensor memory, operands of chunk 0 ----
    // stage chunk m of this piece (one thread; the buffers it overwrites were last read through ordinary loads,
    // hence the proxy fence)
    auto stage = [&](int m) {
      chunk_stage<Cf>(maps, tile, smem + Cf::OFF_KU + (m % 3) * Cf::KU_HALF, smem + Cf::OFF_RAW + (m & 1) * Cf::RAW_BYTES, smem + Cf::OFF_RPQ + (m % 3) * Cf::RPQ_BYTES, bh,
                      tseg0 + m * C, col0, m, &bars[B_KQ0 + (m & 1)],
                      (Cf::KU_MIRROR && m > 0 && m % 3 == 0) ? smem + Cf::OFF_KU + 3 * Cf::KU_HALF : nullptr);
    };
    // everything staged for chunk m has landed (the barrier of m's parity completes once per chunk of that parity)
    auto staged = [&](int m) { return mbar_wait(&bars[B_KQ0 + (m & 1)], (m >> 1) & 1); };
    if (h == 0) {
      stage(0);
      if (nchunks > 1) stage(1);
    }
    if (from_flag) {  // the head of this tile was processed by another block: wait for its state
      if (h == 0) {
        bool seen = false;
        const unsigned long long t_begin = global_timer_ns();
        while (!seen) {  // bounded by wall time (about two seconds)
          seen = ld_acquire_gpu(flag) == sched.epoch;
          if (!seen) {
            if (global_timer_ns() - t_begin > 2000000000ull) break;
            __nanosleep(100);
          }
        }
        if (!seen) *fail_s = 1;
        // A flag has one producer and one consumer per launch.  The consumer clears it, so that a launch that is
        // replayed with the SAME epoch (a captured CUDA graph) waits again instead of finding last time's value.
        else st_release_gpu(flag, 0u);
      }
      named_bar_sync(1, 128);
      if (*fail_s) failed = true;
    }
    if constexpr (Cf::TEMPORAL) {
      // carried distributions of this helper's row (App. B.3): r_prev goes to the row warps through shared memory
      // (published with the first gates, barrier BE), rho_prev stays here
      const float *r_src = from_flag ? p.r_out : p.r_in, *q_src = from_flag ? p.rho_out : p.rho_in;
      float rp = 1.0f / J;
      rho_run = 1.0f / J;
      if (col_ok && !failed) {
        const size_t idx = ((size_t)bh * J + j) * p.Dv + col;
        if (r_src) rp = __ldcg(r_src + idx);
        if (q_src) rho_run = __ldcg(q_src + idx);
      }
      reinterpret_cast<float *>(smem + Cf::OFF_RP)[h] = rp;
    }
    {
      const float *w_src = from_flag ? p.W_out : p.W_in;
      const float *src = (w_src && col_ok && !failed) ? w_src + (((size_t)bh * J + j) * p.Dv + col) * DK : nullptr;
#pragma unroll
      for (int cc = 0; cc < DK / 16; ++cc) {
        float w[16];
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
          if (src) t = __ldcg(reinterpret_cast<const float4 *>(src + cc * 16 + i * 4));
          w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) bf16_split2(w[2 * i], w[2 * i + 1], hi[i], lo[i]);
        tmem_st16(tb + Cf::TM_W + cc * 16, w);
        tmem_st8(tb + Cf::TM_WHI + cc * 8, reinterpret_cast<const float(&)[8]>(hi));
        tmem_st8(tb + Cf::TM_WLO + cc * 8, reinterpret_cast<const float(&)[8]>(lo));
      }
      {  // coefficient columns: finite from the start (see below); ordered before the row warps' first store by WP -> E
        const uint32_t z[4] = {0u, 0u, 0u, 0u};
#pragma unroll
        for (int cc = 0; cc < C / 8; ++cc) {
          tmem_st4(tb + Cf::TM_CHI + cc * 4, z);
          tmem_st4(tb + Cf::TM_CLO + cc * 4, z);
        }
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&bars[B_WP]);
    }
    // the far-push MMA spans 16 tokens of coefficients and of its operand, of which only the first 8 count: the
    // operand's other half stays zero, and the coefficient columns must at least be finite from the start
    for (int e = h; e < 4 * (C / 2); e += 128)
      *reinterpret_cast<uint4 *>(smem + Cf::OFF_FAR + (e / (C / 2)) * Cf::FAR_TILE + Cf::FAR_LBO + (e % (C / 2)) * 16) = make_uint4(0, 0, 0, 0);
    if (nchunks == 1) {  // the odd half of the operand tile is read (as don't-care rows) by the Gram batch: make it finite
      for (int e = h; e < (DK / 64) * 2 * C * 8; e += 128)
        *reinterpret_cast<uint4 *>(tile + (e / (2 * C * 8)) * Cf::TILE_HALF + 2 * C * 128 + (e % (2 * C * 8)) * 16) = make_uint4(0, 0, 0, 0);
    }
    if (!staged(0)) failed = true;
    {
      const float *As0 = nullptr;
      if constexpr (Cf::GATED) {  // the decay warp has the running products of chunk 0 in place
        if (!mbar_wait(&bars[B_A], 0)) failed = true;
        As0 = reinterpret_cast<const float *>(smem + Cf::OFF_A);
      }
      cook_be(smem + Cf::OFF_RAW, min(C, Tseg), As0);
    }
    if constexpr (Cf::TEMPORAL) cook_pk(smem + Cf::OFF_RAW);
    mbar_arrive(&bars[B_BE]);
    if (spill_mine[0]) {
      if (!mbar_wait(&bars[B_G], 0)) failed = true;
      tc_fence_after_sync();
      if (!failed) spill_gram(0);
      mbar_arrive(&bars[B_GS]);
    }

    // Per chunk n, in the order of what the other roles wait for first.
#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const bool more = n + 1 < nchunks;
      // (2) outputs of chunk n-1, whose readouts completed shortly after chunk n started.  The row warps wait for
      // OD(n-2) at the top of chunk n, and OD must not complete another phase before they have: in every iteration
      // but the last the Gram batch spilled in (1) was issued after the row warps passed that point (PQF(n)); in the
      // last one, and in the Gated kernel, the same barrier is waited for here.
      auto outputs_of_previous = [&]() -> bool {
        if (n == 0) return true;
        if ((!more || Cf::GATED) && !mbar_wait(&bars[B_PQF], n & 1)) return false;
        if (!mbar_wait(&bars[B_QD], (n - 1) & 1)) return false;
        write_outputs(n - 1);
        mbar_arrive(&bars[B_OD]);
        return true;
      };
      if constexpr (Cf::GATED) {
        // the outputs of chunk n-1 take the running products of its decays from the stage that the decay warp fills
        // for chunk n+1 once these outputs are formed (it waits for OD): outputs first here
        if (!outputs_of_previous()) { failed = true; break; }
      }
      if (more) {
        // (1) gates of chunk n+1 for the row warps, then its Gram batch
        if (!staged(n + 1)) { failed = true; break; }
        const float *As1 = nullptr;
        if constexpr (Cf::GATED) {
          if (!mbar_wait(&bars[B_A], (n + 1) & 1)) { failed = true; break; }
          As1 = reinterpret_cast<const float *>(smem + Cf::OFF_A + ((n + 1) & 1) * Cf::A_STAGE);
        }
        cook_be(smem + Cf::OFF_RAW + ((n + 1) & 1) * Cf::RAW_BYTES, min(C, Tseg - (n + 1) * C), As1);
        if constexpr (Cf::TEMPORAL) cook_pk(smem + Cf::OFF_RAW + ((n + 1) & 1) * Cf::RAW_BYTES);
        mbar_arrive(&bars[B_BE]);
        if (spill_mine[(n + 1) & 1]) {
          if (!mbar_wait(&bars[B_G], (n + 1) & 1)) failed = true;
          tc_fence_after_sync();
          if (!failed) spill_gram(n + 1);
          mbar_arrive(&bars[B_GS]);
        }
      }
      if constexpr (!Cf::GATED) {
        if (!outputs_of_previous()) { failed = true; break; }
      }
      // (3) chunk n is finished by the row warps: stage chunk n+2 into the buffers chunk n used
      if (!mbar_wait(&bars[B_C], n & 1)) { failed = true; break; }
      if (n + 2 < nchunks && h == 0) stage(n + 2);
      // (4) W has been updated with chunk n: split it into operand parts again
      if (!mbar_wait(&bars[B_U], n & 1)) { failed = true; break; }
      if (more) {
        tc_fence_after_sync();
        float decay = 1.0f;
        if constexpr (Cf::GATED) decay = reinterpret_cast<const float *>(smem + Cf::OFF_A + (n & 1) * Cf::A_STAGE)[C * NROW + a_slot];
        refresh_parts(decay);
        mbar_arrive(&bars[B_WP]);
      }
    }
    if (!failed && !mbar_wait(&bars[B_QD], (nchunks - 1) & 1)) failed = true;
    if (!failed) write_outputs(nchunks - 1);
    if constexpr (Cf::TEMPORAL) {
      if (!failed && p.rho_out && col_ok) p.rho_out[((size_t)bh * J + j) * p.Dv + col] = rho_run;
      if (to_flag) {  // the row warps publish the hand-over flag once both roles have stored their carried state
        __threadfence();
        named_bar_sync(5, 256);
      }
    }
    if constexpr (RDEBUG) {
      // this piece's sums of the readout weights: the J lanes of a column hold disjoint tokens, and other pieces of
      // the tile may run in other blocks, hence atomic additions
      constexpr float kLn2 = 0.6931471805599453f;
      if constexpr (Cf::TEMPORAL) {
        if (!failed && col_ok) {
          if (p.rho_sum) atomicAdd(p.rho_sum + ((size_t)bh * J + j) * p.Dv + col, sq_sum[0]);
          if (p.rho_ent && j == 0) atomicAdd(p.rho_ent + (size_t)bh * p.Dv + col, sq_ent * kLn2);
        }
      } else if (!failed && col_ok) {
        constexpr int LJ = (J == 4) ? 2 : 3;
#pragma unroll
        for (int c = 0; c < J; ++c) {
          int pat = 0;
#pragma unroll
          for (int rd = 0; rd < LJ; ++rd) pat |= ((c >> (LJ - 1 - rd)) & 1) ? (J >> (rd + 1)) : 0;
          if (p.rho_sum) atomicAdd(p.rho_sum + ((size_t)bh * J + (j ^ pat)) * p.Dv + col, sq_sum[c]);
        }
        if (p.rho_ent) atomicAdd(p.rho_ent + (size_t)bh * p.Dv + col, sq_ent * kLn2);
      }
    }
  } else if (warp == 9) {
    // =============================== decay warp (Gated only) =================================
    // Lane L serves component L / (COLS / 4) and four consecutive columns of the tile.  Per chunk: their decays straight
    // from global memory (one 16-byte load per token, or one value when there is one decay per component; a warp of
    // its own, so that the load latency stalls nobody else, and few instructions, because every issue slot it takes
    // on its scheduler is taken from a row warp), their running products A_t since the chunk began into the stage of
    // the chunk's parity: entry t + 1 = A_t, entry 0 = 1.  Tokens past the end of the sequence and columns past Dv
    // decay by 1.  A stage is refilled once the outputs of the chunk two back are formed.
    if constexpr (Cf::GATED) {
      const int gj = lane / (COLS / 4), gc = 4 * (lane % (COLS / 4));
      const bool per_out = p.gran == SWILA_GATE_PER_OUT;
      const bool cols_ok = col0 + gc < p.Dv;  // Dv is a multiple of 8: four columns are inside or outside together
      const float *src = per_out ? p.alpha + (tok0 * J + gj) * (size_t)p.Dv + col0 + gc : p.alpha + tok0 * J + gj;
      const size_t tstride = per_out ? (size_t)J * p.Dv : (size_t)J;
      const int slot4 = Cf::a_slot(gc, gj) / 4;
#pragma unroll 1
      for (int m = 0; m < nchunks && !failed; ++m) {
        const int nv = min(C, Tseg - m * C);
        float4 *As = reinterpret_cast<float4 *>(smem + Cf::OFF_A + (m & 1) * Cf::A_STAGE);
        // the chunk's decays and their running products into registers, a whole chunk ahead of their use
        float4 prod[C];
        if (per_out) {
#pragma unroll
          for (int t = 0; t < C; ++t)
            prod[t] = (t < nv && cols_ok) ? __ldg(reinterpret_cast<const float4 *>(src + t * tstride)) : make_float4(1.f, 1.f, 1.f, 1.f);
        } else {
#pragma unroll
          for (int t = 0; t < C; ++t) {
            const float a1 = (t < nv && cols_ok) ? __ldg(src + t * tstride) : 1.0f;
            prod[t] = make_float4(a1, a1, a1, a1);
          }
        }
        src += C * tstride;
#pragma unroll
        for (int t = 1; t < C; ++t) {
          prod[t].x *= prod[t - 1].x; prod[t].y *= prod[t - 1].y; prod[t].z *= prod[t - 1].z; prod[t].w *= prod[t - 1].w;
        }
        // ... then the stage must be free: the outputs of the chunk two back are formed
        if (m >= 2 && !bwait_idle(B_OD, (m - 2) & 1)) { failed = true; break; }
        As[slot4] = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
        for (int t = 0; t < C; ++t) As[(t + 1) * (NROW / 4) + slot4] = prod[t];
        // A must never run two phases ahead of its waiters (the helpers): for m >= 2 the wait above implies that they
        // have taken chunk m-1's products; chunk 1's must not be announced before they have taken chunk 0's, which
        // the first gates (BE) tell -- a piece that waits for its state to be handed over gets there late
        if (m == 1 && !bwait_idle(B_BE, 0)) failed = true;
        mbar_arrive(&bars[B_A]);
      }
    }
  } else if (warp == 8 && lane == 0) {
    // =============================== MMA issuer ==============================================
    constexpr uint32_t idE = idesc_bf16(128, 2 * C);  // N = 2C: [P0 | Q0], Gram batch, cross-chunk term
    constexpr uint32_t idU = idesc_bf16_bmn(128, DK);  // B (the keys) is read MN-major
    constexpr uint32_t idQ = idesc_bf16(128, C);
    // operand of the tile starting at row `row0`, K step ks (16 key dims = 32 bytes inside a 128-byte row; four
    // steps per half of 64 key dims)
    const uint32_t tile_addr = smem_u32(tile);
    auto tile_desc = [&](int row0, int ks) {
      return smem_desc_sw128(tile_addr + (ks >> 2) * Cf::TILE_HALF + row0 * 128 + (ks & 3) * 32, 1024);
    };
    const uint64_t gx_hi = smem_desc_kmajor(smem_u32(GX_all), Cf::GX_LBO, 128);
    const uint64_t gx_lo = smem_desc_kmajor(smem_u32(GX_all + Cf::GX_TILE), Cf::GX_LBO, 128);
    // Gram batch of chunk m: every row of the tile against the keys of chunk m and against the keys of chunk m-1
    // The keys come from the ring of key copies: when the slots of chunks m-1 and m are adjacent (always with the
    // mirror slot, else two times out of three) they are one operand of 64 rows and one MMA per K step gives
    // [Tile K_{m-1}^T | Tile K_m^T].
    const uint32_t ku_addr = smem_u32(smem + Cf::OFF_KU);
    auto ku_desc = [&](int slot, int ks) {
      return smem_desc_sw128(ku_addr + (ks >> 2) * Cf::KU_HSTRIDE + slot * Cf::KU_HALF + (ks & 3) * 32, 1024);
    };
    auto gram = [&](int m) {
      const int so = m % 3, sp = (m + 2) % 3;
      if (m > 0 && (sp + 1 == so || Cf::KU_MIRROR)) {  // (slot 2, mirror of slot 0) when the ring wraps
#pragma unroll 1
        for (int ks = 0; ks < DK / 16; ++ks) mma_bf16_ss(tb0 + Cf::TM_G, tile_desc(0, ks), ku_desc(sp, ks), idE, ks > 0);
      } else {
#pragma unroll 1
        for (int ks = 0; ks < DK / 16; ++ks) mma_bf16_ss(tb0 + Cf::TM_G + C, tile_desc(0, ks), ku_desc(so, ks), idQ, ks > 0);
        if (m > 0) {
#pragma unroll 1
          for (int ks = 0; ks < DK / 16; ++ks) mma_bf16_ss(tb0 + Cf::TM_G, tile_desc(0, ks), ku_desc(sp, ks), idQ, ks > 0);
        }
      }
      mma_commit(&bars[B_G]);
    };
    // [P0 | Q0] of chunk m from the state as it is now (hi and lo parts)
    auto w_times_kq = [&](int m) {
#pragma unroll 1
      for (int ks = 0; ks < DK / 16; ++ks)
        mma_bf16_ts(tb0 + Cf::TM_PQ, tb0 + Cf::TM_WHI + ks * 8, tile_desc((m & 1) * 2 * C, ks), idE, ks > 0);
#pragma unroll 1
      for (int ks = 0; ks < DK / 16; ++ks)
        mma_bf16_ts(tb0 + Cf::TM_PQ, tb0 + Cf::TM_WLO + ks * 8, tile_desc((m & 1) * 2 * C, ks), idE, true);
    };
    // + Cmat (K_prev [K;Q]^T): the update of the chunk that just finished, seen by the next chunk's products
    // (16 tokens of the chunk per call)
    auto cross = [&](int ks) {
      const uint64_t adv = (uint64_t)(ks * 2 * (Cf::GX_LBO / 16));
      mma_bf16_ts(tb0 + Cf::TM_PQ, tb0 + Cf::TM_CHI + ks * 8, gx_hi + adv, idE, true);
      mma_bf16_ts(tb0 + Cf::TM_PQ, tb0 + Cf::TM_CLO + ks * 8, gx_hi + adv, idE, true);
      mma_bf16_ts(tb0 + Cf::TM_PQ, tb0 + Cf::TM_CHI + ks * 8, gx_lo + adv, idE, true);
    };
    // readouts of chunk n: QD += Cmat (K Q^T masked)  -- c_hi B_hi + c_lo B_hi + c_hi B_lo
    auto readout = [&](int n) {
      const uint64_t bh0 = smem_desc_kmajor(smem_u32(BQ_all + (n & 1) * 2 * Cf::BQ_TILE), Cf::BQ_LBO, 128);
      const uint64_t bl0 = smem_desc_kmajor(smem_u32(BQ_all + (n & 1) * 2 * Cf::BQ_TILE + Cf::BQ_TILE), Cf::BQ_LBO, 128);
      const uint32_t d = tb0 + Cf::TM_QD + (n & 1) * C;
#pragma unroll 1
      for (int ks = 0; ks < C / 16; ++ks) {
        const uint64_t adv = (uint64_t)(ks * 2 * (Cf::BQ_LBO / 16));
        mma_bf16_ts(d, tb0 + Cf::TM_CHI + ks * 8, bh0 + adv, idQ, true);
        mma_bf16_ts(d, tb0 + Cf::TM_CLO + ks * 8, bh0 + adv, idQ, true);
        mma_bf16_ts(d, tb0 + Cf::TM_CHI + ks * 8, bl0 + adv, idQ, true);
      }
      mma_commit(&bars[B_QD]);
    };
    if (!mbar_wait(&bars[B_KQ0], 0) || !mbar_wait(&bars[B_WP], 0)) failed = true;
    tc_fence_after_sync();
    if (!failed) {
      gram(0);
      w_times_kq(0);
      mma_commit(&bars[B_E]);
    }
#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const bool more = n + 1 < nchunks;
      if (more) {
        // ahead of the serial path: Gram batch and state x [K;Q] of chunk n+1 with the state before chunk n's
        // update (W is final up to chunk n-1 and split into parts; [P0|Q0] of chunk n has been taken out)
        if (!mbar_wait(&bars[B_KQ0 + ((n + 1) & 1)], ((n + 1) >> 1) & 1) || !mbar_wait(&bars[B_PQF], n & 1)) { failed = true; break; }
        if (n > 0 && !mbar_wait(&bars[B_WP], n & 1)) { failed = true; break; }
        tc_fence_after_sync();
        gram(n + 1);
      }
      {
        // far pushes of chunk n: what its first 8 tokens add to the predictions of its last 8, needed when the row
        // warps reach token 24.  A = the coefficient columns of tokens 0..15 (8..15 are stale but finite and meet
        // zero rows of the operand), B = rows 16..31 of K K^T against tokens 0..7.
        if (!mbar_wait(&bars[B_T0], n & 1)) { failed = true; break; }
        tc_fence_after_sync();
        const uint32_t fa = smem_u32(smem + Cf::OFF_FAR + (n & 1) * 2 * Cf::FAR_TILE);
        const uint64_t f_hi = smem_desc_kmajor(fa, Cf::FAR_LBO, 128), f_lo = smem_desc_kmajor(fa + Cf::FAR_TILE, Cf::FAR_LBO, 128);
        constexpr uint32_t idF = idesc_bf16(128, C / 2);
        mma_bf16_ts(tb0 + Cf::TM_FAR, tb0 + Cf::TM_CHI, f_hi, idF, false);
        mma_bf16_ts(tb0 + Cf::TM_FAR, tb0 + Cf::TM_CLO, f_hi, idF, true);
        mma_bf16_ts(tb0 + Cf::TM_FAR, tb0 + Cf::TM_CHI, f_lo, idF, true);
        mma_commit(&bars[B_FAR]);
      }
      if (more) {
        w_times_kq(n + 1);
        // first half of the cross-chunk term (tokens 0-15 of chunk n, whose coefficients T0 released), while the
        // chunk still runs
        if (!mbar_wait(&bars[B_GS], (n + 1) & 1)) { failed = true; break; }
        tc_fence_after_sync();
        cross(0);
      }
      if (!mbar_wait(&bars[B_C], n & 1)) { failed = true; break; }
      tc_fence_after_sync();
      const bool redone = *redo_s != 0;  // ordered by the barrier: set before the row warps arrived
      if (redone) *redo_s = 0;
      if (more) {
        if (redone) {  // rare: a row warp replaced the coefficients that the first half was formed from
          w_times_kq(n + 1);
          cross(0);
        }
        cross(1);  // -> E(n+1): the only tensor work left between two chunks of the row warps
        mma_commit(&bars[B_E]);
      }
      if constexpr (Cf::GATED) {
        // the helpers wrote the decayed state back over W after the previous update: that must be complete (in
        // every iteration but the last it has been waited for above already)
        if (n > 0 && !mbar_wait(&bars[B_WP], n & 1)) { failed = true; break; }
        tc_fence_after_sync();
      }
#pragma unroll 1
      for (int ks = 0; ks < C / 16; ++ks) {  // W += Cmat K (Eq. 3.3 summed over the chunk)
        // B = the second copy of the chunk's keys, read MN-major: 16 tokens per step = 16 rows of 128 bytes, the
        // halves of 64 key dims KU_HSTRIDE apart
        const uint64_t bt = smem_desc_sw128_mn(smem_u32(smem + Cf::OFF_KU + (n % 3) * Cf::KU_HALF) + ks * 16 * 128, Cf::KU_HSTRIDE, 1024);
        mma_bf16_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CHI + ks * 8, bt, idU, true);
        mma_bf16_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CLO + ks * 8, bt, idU, true);
        mma_bf16_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CL3 + ks * 8, bt, idU, true);
      }
      mma_commit(&bars[B_U]);
      readout(n);
    }
  }
  if (failed) {
    atomicCAS(&g_chunk_error, 0, 1);  // (a wait that gave up has left its own code already)
    *fail_s = 1;
  }
  }  // pieces
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 8) tmem_dealloc(*tmem_base_s, Cf::TM_ALLOC);
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link against the driver.
typedef CUresult (*ChunkEncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                       const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                       CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline ChunkEncodeTiledFn chunk_encode_fn() {
  static ChunkEncodeTiledFn fn = [] {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      sym = nullptr;
    return (ChunkEncodeTiledFn)sym;
  }();
  return fn;
}

// One bf16 tensor map: `rank` dimensions (innermost first) of sizes `dims` with byte strides `strides` (for dimensions
// 1 .. rank-1) and a copy box of `box` elements; no swizzle, out-of-range elements read as zero.
inline bool chunk_encode(CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides,
                         const cuuint32_t *box, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE) {
  ChunkEncodeTiledFn fn = chunk_encode_fn();
  if (!fn) return false;
  const cuuint32_t ones[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, ones,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor maps of one launch.  k, q [BH][T][DK] as (DK, T, BH) with a box of 64 key dims x 32 tokens and the 128-byte
// swizzle, which is how the operand tile stores them; v [BH][T][Dv] as (Dv, T, BH); the gate
// logits [BH][T][J][Dv] as (Dv, J, T, BH) with a box of GROW columns, all J components, 32 tokens.
template <class Cf>
bool chunk_make_maps(const ScanParams &p, ChunkMaps *m) {
  const cuuint64_t BH = (cuuint64_t)p.B * p.H, T = (cuuint64_t)p.T, Dv = (cuuint64_t)p.Dv, J = Cf::J, DK = Cf::DK;
  {
    const cuuint64_t dims[3] = {DK, T, BH};
    const cuuint64_t strides[2] = {DK * 2, T * DK * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)Cf::C, 1};
    if (!chunk_encode(&m->k, p.k, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !chunk_encode(&m->q, p.q, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
      return false;
  }
  {
    const cuuint64_t dims[3] = {Dv, T, BH};
    const cuuint64_t strides[2] = {Dv * 2, T * Dv * 2};
    const cuuint32_t box[3] = {(cuuint32_t)Cf::COLS, (cuuint32_t)Cf::C, 1};
    if (!chunk_encode(&m->v, p.v, 3, dims, strides, box)) return false;
    if constexpr (Cf::TEMPORAL) {
      if (!chunk_encode(&m->gk, p.gk_logit, 3, dims, strides, box) || !chunk_encode(&m->gq, p.gq_logit, 3, dims, strides, box))
        return false;
    }
  }
  {
    const cuuint64_t dims[4] = {Dv, J, T, BH};
    const cuuint64_t strides[3] = {Dv * 2, J * Dv * 2, T * J * Dv * 2};
    const cuuint32_t box[4] = {(cuuint32_t)Cf::GROW, (cuuint32_t)Cf::J, (cuuint32_t)Cf::C, 1};
    if (!chunk_encode(&m->be, p.beta_logit, 4, dims, strides, box) || !chunk_encode(&m->pk, p.pik_logit, 4, dims, strides, box) ||
        !chunk_encode(&m->pq, p.piq_logit, 4, dims, strides, box))
      return false;
  }
  return true;
}

// Number of SMs of the current device (one block is resident per SM).
inline int chunk_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return n;
}

// Launch counter shared by every instantiation: the value a launch publishes in the hand-over flags
// (never 0, the flags' initial value).
inline unsigned chunk_next_epoch() {
  static std::atomic<unsigned> counter{0};
  unsigned e = ++counter;
  if (e == 0) e = ++counter;
  return e;
}

template <int J, int DK, bool TEMPORAL = false, bool GATED = false>
int launch_chunk(const LaunchArgs &a) {
  using Cf = ChunkCfg<J, DK, TEMPORAL, GATED>;
  const bool aux = a.p.r_debug || a.p.r_sum || a.p.r_ent || a.p.rho_sum || a.p.rho_ent;
  if (J > 8 && aux) return -1000;     // likewise for J = 16
  if (GATED && aux) return -1000;     // and for the Gated variant
  auto kern = swila_chunk_kernel<Cf, false>;
  if constexpr (!GATED && J <= 8) {
    if (aux) kern = swila_chunk_kernel<Cf, true>;
  }
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cf::SMEM_BYTES);
  if (e != cudaSuccess) return (int)e;
  const long long nslice = (a.p.Dv + Cf::COLS - 1) / Cf::COLS;
  const long long ntiles = nslice * a.p.B * a.p.H;
  const long long nch = (a.p.T + Cf::C - 1) / Cf::C;
  if (ntiles <= 0 || ntiles > 0x7fffffffLL || nch <= 0 || nch > 0x7fffffffLL) return (int)cudaErrorInvalidConfiguration;
  ChunkSched sc{(int)ntiles, (int)nch, (int)nch, 1, 0u, nullptr};
  ScanParams prm = a.p;
  ChunkMaps maps;
  if (!chunk_make_maps<Cf>(a.p, &maps)) return (int)cudaErrorInvalidValue;

  // More tiles than SMs, not a whole number of waves: cut the chunk sequence into equal runs instead of whole
  // tiles, so that the last wave is not half empty (chunk_plan).  The state of a split tile travels through the
  // state output, hence only when that is given; blocks of such a launch wait for each other, hence the
  // cooperative launch (all blocks resident or no launch at all).
  const ChunkPlan pl = chunk_plan((long long)a.p.B * a.p.H, nslice, nch, chunk_sm_count(),
                                   a.p.W_out != nullptr && (!TEMPORAL || (a.p.r_out && a.p.rho_out)), kChunkFlagTiles);
  if (pl.split) {
    unsigned *flags = nullptr;
    if (cudaGetSymbolAddress((void **)&flags, g_chunk_flags) == cudaSuccess) {
      const unsigned epoch = chunk_next_epoch();
      ChunkSched ss{(int)pl.units, pl.nch, pl.per, pl.gang, epoch, flags + (size_t)(epoch % kChunkFlagSlots) * kChunkFlagTiles};
      void *args[] = {(void *)&prm, (void *)&ss, (void *)&maps};
      // The launch starts from cleared flags: a consumer whose wait expired leaves its flag set, and a captured
      // launch is replayed with the epoch of its capture, which its own earlier run has already published.
      e = cudaMemsetAsync(ss.flags, 0, (size_t)pl.units * pl.gang * sizeof(unsigned), a.stream);
      if (e == cudaSuccess)
      e = cudaLaunchCooperativeKernel((const void *)kern, dim3((unsigned)pl.grid), dim3(Cf::NT), args, Cf::SMEM_BYTES, a.stream);
      if (e == cudaSuccess) return (int)cudaGetLastError();
      (void)cudaGetLastError();  // not launched (e.g. the blocks cannot all be resident): fall back to whole tiles
    }
  }
  kern<<<(unsigned)ntiles, Cf::NT, Cf::SMEM_BYTES, a.stream>>>(prm, sc, maps);
  return (int)cudaGetLastError();
}

}  // namespace swila
