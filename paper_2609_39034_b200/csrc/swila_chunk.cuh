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
// of the floating-point additions differs from the scan.  The three dense contractions
//   P0 = W0 K^T, Q0 = W0 Q^T  (M x Dk x C)      and      W += Cmat K  (M x C x Dk)
// plus the two Gram matrices K K^T, K Q^T run on the tcgen05 tensor cores in TF32 with FP32
// accumulation in tensor memory; FP32 operands are split as x = hi + lo (hi = the 19 leading
// bits the hardware keeps, lo = the remainder) and both parts are multiplied, so products carry
// ~22 significant bits.  bf16 inputs k, q are exact in TF32.  The triangular part (the sums over
// s inside the chunk) and the E-step stay on the FP32 ALUs, one thread per row.
//
// One block owns 128 rows = COLS = 128/J output columns of one (batch, head) and is split into
// three roles that run concurrently and meet on mbarriers:
//   row warps 0-3    thread r serves row (d = r / J, j = r % J), which is also its tensor-memory
//                    lane; the J components of a column sit in adjacent lanes, so the E-step
//                    normalisation is a few shuffles.  They run the sequential part of a chunk.
//   helper warps 4-7 stage the next chunk (cp.async), convert K and Q into the tensor cores'
//                    shared-memory operand layout, move the Gram matrices from tensor memory to
//                    shared memory, refresh the low part of W after each update, and write the
//                    chunk's outputs -- all while the row warps are busy.
//   warp 8, lane 0   issues every tcgen05.mma and commits them to the barriers.
#pragma once

#include <type_traits>

#include "swila_common.cuh"
#include "swila_umma.cuh"

namespace swila {

// Set when a bounded wait on a completion barrier expires (never expected).
static __device__ int g_chunk_error = 0;
#ifdef SWILA_CHUNK_PROFILE
// Developer build only: cycle counters per phase, kept in registers by the first thread of each warp
// role of block 0 and written out at the end; per-block totals for every block.
static __device__ long long g_chunk_prof[4 * 8];
static __device__ long long g_chunk_blk[3 * 1024];  // per block: cycles, SM id, start time (ns)
#define PROF_ADD(i, who) do { long long now_ = clock64(); prof_acc[i] += now_ - prof_t; prof_t = now_; } while (0)
#else
#define PROF_ADD(i, who) do {} while (0)
#endif

template <int J_, int DK_>
struct ChunkCfg {
  static constexpr int J = J_, DK = DK_;
  static constexpr int C = 32;            // tokens per chunk
  static constexpr int GT = 8;            // tokens per trip of the row warps' rolled serial loop
  static constexpr int NROW = 128;        // row threads = rows of the tile
  static constexpr int NT = 288;          // 4 row warps + 4 helper warps + 1 MMA warp
  static constexpr int COLS = NROW / J;   // output columns per block
  static constexpr int ES = 2;            // bf16 io
  // tensor-memory columns
  // W, W_lo: the state and its low part; PQ: [P0 | Q0] of the current chunk; QD: the query-side
  // readouts w_t.q_t of a chunk (double-buffered: the outputs of chunk n are formed while chunk
  // n+1 runs); G: [K K^T | K Q^T]; CHI / CLO: the update coefficients of the chunk
  static constexpr int TM_W = 0, TM_WLO = DK, TM_PQ = 2 * DK, TM_QD = TM_PQ + 2 * C, TM_G = TM_QD + 2 * C,
                       TM_CHI = TM_G + 2 * C, TM_CLO = TM_CHI + C, TM_USED = TM_CLO + C;
  static constexpr int TM_ALLOC = 512;
  static_assert(TM_USED <= TM_ALLOC, "tensor memory budget");
  static_assert(J == 4 || J == 8, "the output transposition assumes that J divides 8");
  // raw stages (bytes), all bf16.  Main part: k, q [C][DK], v [C][COLS], beta/pik [C][J][COLS] (2-deep
  // ring); the query-prior logits piq [C][J][COLS] live in their own 3-deep ring because the helper
  // warps still need them for the outputs of chunk n while chunk n+2 is being fetched.
  static constexpr int R_K = 0;
  static constexpr int R_Q = R_K + C * DK * ES;
  static constexpr int R_V = R_Q + C * DK * ES;
  static constexpr int R_B = R_V + C * COLS * ES;   // beta logits; the helpers overwrite them in place with
                                                    // beta = sigmoid(.) as fp32 [C][NROW], hence the fp32-sized slot
  static constexpr int R_PK = R_B + C * NROW * 4;
  static constexpr int RAW_BYTES = R_PK + C * J * COLS * ES;
  static constexpr int RPQ_BYTES = C * J * COLS * ES;
  static constexpr int BQ_LBO = C * 16 + 16;        // padded K-chunk stride of the readout operand tiles (bank spread)
  static constexpr int BQ_TILE = (C / 4) * BQ_LBO;
  static constexpr int C_K = DK * ES / 16, C_V = COLS * ES / 16;  // 16-byte units per token row / column slice
  // shared memory map (bytes)
  static constexpr int OFF_RAW = 0;
  static constexpr int OFF_RPQ = OFF_RAW + 2 * RAW_BYTES;  // 4-deep ring of query-prior logits
  static constexpr int OFF_KQ = OFF_RPQ + 4 * RPQ_BYTES;   // 2 x [DK/4][2C][4] fp32: rows 0..C-1 = K, C..2C-1 = Q tokens
  static constexpr int OFF_KT = OFF_KQ + 2 * 2 * C * DK * 4;  // [C/4][DK][4] fp32: K transposed (rows = key dims)
  static constexpr int OFF_G = OFF_KT + C * DK * 4;        // 2 x Gkk [C][C] fp32 (K K^T, for the row warps)
  static constexpr int OFF_BQ = OFF_G + 2 * C * C * 4;     // 2 x { hi, lo } masked (K Q^T)^T operand tiles
  static constexpr int OFF_OST = OFF_BQ + 2 * 2 * BQ_TILE; // 2 x [C][COLS] bf16 output staging
  static constexpr int OFF_BAR = OFF_OST + 2 * C * COLS * ES;
  static constexpr int SMEM_BYTES = OFF_BAR + 128;
  static_assert(RAW_BYTES % 16 == 0 && RPQ_BYTES % 16 == 0 && (COLS * ES) % 16 == 0, "alignment");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

// barrier slots
enum { B_E = 0, B_G, B_U, B_QD, B_KQ, B_KT, B_WLO, B_GS, B_C, B_COUNT };

// hi/lo split of an FP32 value for TF32 operands: hi keeps the bits the tensor core reads
// (it ignores the 13 low mantissa bits), lo is the exact remainder.
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

// cp.async staging of one chunk by the 128 helper threads (h = 0..127)
template <class Cf>
__device__ __forceinline__ void chunk_issue_raw(const ScanParams &p, unsigned char *raw, unsigned char *rawpq,
                                                size_t tok0, int t0, int col0, int h) {
  constexpr int J = Cf::J, DK = Cf::DK, C = Cf::C, ES = Cf::ES, C_K = Cf::C_K, C_V = Cf::C_V;
  const int nvalid = min(C, p.T - t0);
  const size_t tokb = tok0 + (size_t)t0;
  const char *kb = (const char *)p.k + tokb * DK * ES;
  const char *qb = (const char *)p.q + tokb * DK * ES;
#pragma unroll
  for (int u = h; u < C * C_K; u += 128) {  // k and q rows of the chunk are contiguous in global memory
    const bool valid = (u / C_K) < nvalid;
    cp_async16(raw + Cf::R_K + u * 16, valid ? kb + u * 16 : (const char *)p.k, valid ? 16 : 0);
    cp_async16(raw + Cf::R_Q + u * 16, valid ? qb + u * 16 : (const char *)p.k, valid ? 16 : 0);
  }
#pragma unroll
  for (int u = h; u < C * C_V; u += 128) {
    const int tok = u / C_V, cu = u % C_V;
    const int col = col0 + cu * 8;
    const bool valid = tok < nvalid && col < p.Dv;
    cp_async16(raw + Cf::R_V + u * 16, valid ? (const char *)p.v + ((tokb + tok) * p.Dv + col) * ES : (const char *)p.k,
               valid ? 16 : 0);
  }
#pragma unroll
  for (int u = h; u < C * J * C_V; u += 128) {
    const int cu = u % C_V, jj = (u / C_V) % J, tok = u / (C_V * J);
    const int col = col0 + cu * 8;
    const bool valid = tok < nvalid && col < p.Dv;
    const size_t off = (((tokb + tok) * J + jj) * (size_t)p.Dv + col) * ES;
    cp_async16(raw + Cf::R_B + u * 16, valid ? (const char *)p.beta_logit + off : (const char *)p.k, valid ? 16 : 0);
    cp_async16(raw + Cf::R_PK + u * 16, valid ? (const char *)p.pik_logit + off : (const char *)p.k, valid ? 16 : 0);
    cp_async16(rawpq + u * 16, valid ? (const char *)p.piq_logit + off : (const char *)p.k, valid ? 16 : 0);
  }
}

template <class Cf, bool RDEBUG>
__global__ void __launch_bounds__(Cf::NT, 1) swila_chunk_kernel(const __grid_constant__ ScanParams p) {
  using namespace umma;
  constexpr int J = Cf::J, DK = Cf::DK, C = Cf::C, NROW = Cf::NROW, COLS = Cf::COLS;
  extern __shared__ __align__(128) unsigned char smem[];
  float *KQ_all = reinterpret_cast<float *>(smem + Cf::OFF_KQ);
  float *Kt = reinterpret_cast<float *>(smem + Cf::OFF_KT);
  float *G_all = reinterpret_cast<float *>(smem + Cf::OFF_G);
  unsigned char *BQ_all = smem + Cf::OFF_BQ;
  __nv_bfloat16 *ostage = reinterpret_cast<__nv_bfloat16 *>(smem + Cf::OFF_OST);
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + Cf::OFF_BAR);
  uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bars + B_COUNT);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nslice = (p.Dv + COLS - 1) / COLS;
  const int bh = blockIdx.x / nslice;
  const int col0 = (blockIdx.x - bh * nslice) * COLS;
  const size_t tok0 = (size_t)bh * p.T;
  const int nchunks = (p.T + C - 1) / C;

  if (warp == 8) tmem_alloc(tmem_base_s, Cf::TM_ALLOC);
  if (tid == 0) {
    mbar_init(&bars[B_E], 1);
    mbar_init(&bars[B_G], 1);
    mbar_init(&bars[B_U], 1);
    mbar_init(&bars[B_QD], 1);
    mbar_init(&bars[B_KQ], 128);
    mbar_init(&bars[B_KT], 128);
    mbar_init(&bars[B_WLO], 128);
    mbar_init(&bars[B_GS], 32);
    mbar_init(&bars[B_C], 128);
    mbar_fence_init();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tb0 = *tmem_base_s;
  const uint32_t tb = tb0 + ((uint32_t)((warp & 3) * 32) << 16);  // this warp's lane quarter
  bool failed = false;
#ifdef SWILA_CHUNK_PROFILE
  long long prof_t = clock64();
  const long long prof_t0 = prof_t;
  long long prof_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  if (tid == 0 && blockIdx.x < 1024) {
    unsigned smid;
    unsigned long long ns;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
    g_chunk_blk[1024 + blockIdx.x] = smid;
    g_chunk_blk[2048 + blockIdx.x] = (long long)ns;
  }
#endif

  if (warp < 4) {
    // =============================== row warps ===============================================
    const int r = tid;
    const int dl = r / J, j = r % J;
    const int col = col0 + dl;
    const bool col_ok = col < p.Dv;
    const int jbase = lane - j;
    if (!mbar_wait(&bars[B_KQ], 0) || !mbar_wait(&bars[B_GS], 0)) failed = true;
    // outputs of one chunk (Eq. 3.5): o_td = sum_j pi^q_j (w_t.q_t)_j, pi^q = softmax over the J lanes
    // of a column; eight tokens at a time so that the shuffles of different tokens overlap
    auto write_outputs = [&](int n) {
      const int t0 = n * C;
      const int nvalid = min(C, p.T - t0);
      const __nv_bfloat16 *rpq = reinterpret_cast<const __nv_bfloat16 *>(smem + Cf::OFF_RPQ + (n & 3) * Cf::RPQ_BYTES);
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
          float x[J];
          float mx = -3.0e38f;
#pragma unroll
          for (int c = 0; c < J; ++c) {
            int pat = 0;
#pragma unroll
            for (int rd = 0; rd < LJ; ++rd) pat |= ((c >> (LJ - 1 - rd)) & 1) ? (J >> (rd + 1)) : 0;
            x[c] = __bfloat162float(rpq[(tl * J + (j ^ pat)) * COLS + dl]) * kLog2e;
            mx = fmaxf(mx, x[c]);
          }
          float se = 0.f, so = 0.f;
#pragma unroll
          for (int c = 0; c < J; ++c) {
            const float e = ex2_approx(x[c] - mx);
            se += e;
            so = fmaf(e, hq[(c << (3 - LJ)) | rest], so);
          }
          ost[tl * COLS + dl] = __float2bfloat16_rn(so * rcp_approx(se));
        }
      }
      tc_fence_before_sync();
      PROF_ADD(4, 0);
      named_bar_sync(2, 128);
      PROF_ADD(5, 0);
      constexpr int GROUPS = COLS / 8;  // 8 outputs = 16 bytes per store
      for (int e = r; e < C * GROUPS; e += 128) {
        const int t = e / GROUPS, g8 = e - t * GROUPS;
        if (t < nvalid && col0 + g8 * 8 < p.Dv)
          *reinterpret_cast<uint4 *>((__nv_bfloat16 *)p.o + (tok0 + (size_t)(t0 + t)) * p.Dv + col0 + g8 * 8) =
              *reinterpret_cast<const uint4 *>(ost + t * COLS + g8 * 8);
      }
      PROF_ADD(6, 0);
    };

#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const int t0 = n * C;
      const int nvalid = min(C, p.T - t0);
      const unsigned char *raw = smem + Cf::OFF_RAW + (n & 1) * Cf::RAW_BYTES;
      const __nv_bfloat16 *rv = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_V);
      const __nv_bfloat16 *rpk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_PK);
      const float *Gkk = G_all + (n & 1) * C * C;
      const float *bes = reinterpret_cast<const float *>(raw + Cf::R_B);

      PROF_ADD(0, 0);
      if (!mbar_wait(&bars[B_E], n & 1)) { failed = true; break; }
      tc_fence_after_sync();
      PROF_ADD(1, 0);
      // ---- sequential part of the chunk: E-step and the triangular key-side corrections.  Only one FMA
      //      of a token's push (into the next token's prediction) sits on the serial chain; the rest is
      //      deferred into the shuffle latency of the next token's E-step.
      //      FAST: exponentials are taken without subtracting the per-token maximum; the pass reports whether
      //      any normaliser left the safe range (all components > ~13 standard deviations off, or extreme
      //      prior logits), in which case the chunk is redone with the maximum subtracted. ----
      auto sequential = [&](auto exact_tag) -> bool {
        constexpr bool EXACT = decltype(exact_tag)::value;
        constexpr int GT = Cf::GT;
        bool bad = false;
        // pred[i]: prediction of token tg + i of the current trip (slots past the chunk end are dead weight that
        // keeps the trip's code independent of tg); slot C takes the last token's push
        float pred[C + 1];
#pragma unroll
        for (int cc = 0; cc < C / 16; ++cc) {
          float a[16];
          tmem_ld16(tb + Cf::TM_PQ + cc * 16, a);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) pred[cc * 16 + i] = a[i];
        }
        pred[C] = 0.f;
        float c_prev = 0.f;
#pragma unroll 1
        for (int tg = 0; tg < C; tg += GT) {  // rolled: GT tokens of straight-line code stay in the instruction cache
          float cs[GT];
#pragma unroll
          for (int i = 0; i < GT; ++i) {
            const int t = tg + i;
            const float v = __bfloat162float(rv[t * COLS + dl]);
            const float be = bes[t * NROW + r];
            // serial chain: prediction error -> responsibilities (Eq. 3.4) -> update coefficient (Eq. 3.3)
            const float delta = v - pred[i];
            const float a = fmaf(-kHalfLog2e * delta, delta, __bfloat162float(rpk[(t * J + j) * COLS + dl]) * kLog2e);
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
              sum = e;
#pragma unroll
              for (int jj = 1; jj < J; ++jj) sum += __shfl_sync(0xffffffffu, e, jbase + ((j + jj) & (J - 1)));
              bad = bad || !(sum > 1e-30f && sum < 1e30f);
            }
#ifndef SWILA_EXP_NOPUSH
            {  // deferred push of token t-1 into the predictions of tokens t+1 .. (slots i+1 ..)
              const float4 *gp = reinterpret_cast<const float4 *>(Gkk + max(t - 1, 0) * C + tg);
#pragma unroll
              for (int u4 = (i + 1) / 4; u4 < C / 4; ++u4) {
                const float4 g = gp[u4];
                if (4 * u4 + 0 > i) pred[4 * u4 + 0] = fmaf(c_prev, g.x, pred[4 * u4 + 0]);
                if (4 * u4 + 1 > i) pred[4 * u4 + 1] = fmaf(c_prev, g.y, pred[4 * u4 + 1]);
                if (4 * u4 + 2 > i) pred[4 * u4 + 2] = fmaf(c_prev, g.z, pred[4 * u4 + 2]);
                if (4 * u4 + 3 > i) pred[4 * u4 + 3] = fmaf(c_prev, g.w, pred[4 * u4 + 3]);
              }
            }
#endif
            const float rr = e * rcp_approx(sum);
            float c = (be * delta) * rr;
            if (t >= nvalid) c = 0.f;  // padding tokens of the last chunk leave the state alone
            cs[i] = c;
            if constexpr (RDEBUG) {
              if (col_ok && t < nvalid) p.r_debug[((tok0 + (size_t)(t0 + t)) * J + j) * p.Dv + col] = rr;
            }
            pred[i + 1] = fmaf(c, Gkk[t * C + t + 1], pred[i + 1]);  // the push the next token waits for
            c_prev = c;
          }
          {  // GT update coefficients complete: park them in tensor memory (hi / lo)
            float hi[GT], lo[GT];
#pragma unroll
            for (int i = 0; i < GT; ++i) { hi[i] = tf32_hi(cs[i]); lo[i] = cs[i] - hi[i]; }
            if constexpr (GT == 8) {
              tmem_st8(tb + Cf::TM_CHI + tg, hi);
              tmem_st8(tb + Cf::TM_CLO + tg, lo);
            } else {
              tmem_st16(tb + Cf::TM_CHI + tg, hi);
              tmem_st16(tb + Cf::TM_CLO + tg, lo);
            }
          }
#pragma unroll
          for (int i = 0; i + GT <= C; ++i) pred[i] = pred[i + GT];
#pragma unroll
          for (int i = C - GT + 1; i <= C; ++i) pred[i] = 0.f;
        }
        return bad;
      };
      {  // Q0 seeds the readout accumulator of this chunk
#pragma unroll
        for (int cc = 0; cc < C / 16; ++cc) {
          float b[16];
          tmem_ld16(tb + Cf::TM_PQ + C + cc * 16, b);
          tmem_ld_wait();
          tmem_st16(tb + Cf::TM_QD + (n & 1) * C + cc * 16, b);
        }
      }
      const bool underflow = sequential(std::false_type{});
      if (__any_sync(0xffffffffu, underflow)) {
        tmem_st_wait();
        sequential(std::true_type{});
      }
      tmem_st_wait();
      tc_fence_before_sync();
      PROF_ADD(2, 0);
      // the next chunk's operands, and the previous chunk's readouts, must be in place before this
      // chunk is handed over (keeps every barrier at most one phase ahead of its waiters)
      if (n + 1 < nchunks && (!mbar_wait(&bars[B_KQ], (n + 1) & 1) || !mbar_wait(&bars[B_GS], (n + 1) & 1))) failed = true;
      if (n > 0 && !mbar_wait(&bars[B_QD], (n - 1) & 1)) failed = true;
      mbar_arrive(&bars[B_C]);
      PROF_ADD(3, 0);
      // outputs of the previous chunk, in the shadow of the tensor-core work for chunk n+1
      if (n > 0 && !failed) write_outputs(n - 1);
    }
    if (!failed && !mbar_wait(&bars[B_QD], (nchunks - 1) & 1)) failed = true;
    if (!failed) write_outputs(nchunks - 1);
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
#pragma unroll
        for (int i = 0; i < 4; ++i)
          __stcs(reinterpret_cast<float4 *>(dst + cc * 16 + i * 4), make_float4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]));
      }
    }
  } else if (warp < 8) {
    // =============================== helper warps ============================================
    const int h = tid - 128;
    const int dl = h / J, j = h % J;
    const int col = col0 + dl;
    const bool col_ok = col < p.Dv;

    // K, Q of a raw stage -> stacked fp32 operand tile (16-byte unit (row, k-chunk c) at (c*2C + row)*16)
    auto cook_kq = [&](const unsigned char *raw, float *KQ) {
      const __nv_bfloat16 *rk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_K);
      const __nv_bfloat16 *rq = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_Q);
      // diagonal walk over 8-token x 16-chunk blocks: conflict-free 8-byte reads and 16-byte writes
      constexpr int NBLK = (C / 8) * (DK / 4 / 16);
#pragma unroll 2
      for (int blk = 0; blk < NBLK; ++blk) {
        const int tb8 = blk % (C / 8), cb16 = blk / (C / 8);
        const int s = h >> 4, u = h & 15;
        const int t = tb8 * 8 + ((u + s) & 7), c = cb16 * 16 + u;
        const uint2 kr = *reinterpret_cast<const uint2 *>(rk + t * DK + c * 4);
        const uint2 qr = *reinterpret_cast<const uint2 *>(rq + t * DK + c * 4);
        float4 kf, qf;
        kf.x = __uint_as_float(kr.x << 16); kf.y = __uint_as_float(kr.x & 0xffff0000u);
        kf.z = __uint_as_float(kr.y << 16); kf.w = __uint_as_float(kr.y & 0xffff0000u);
        qf.x = __uint_as_float(qr.x << 16); qf.y = __uint_as_float(qr.x & 0xffff0000u);
        qf.z = __uint_as_float(qr.y << 16); qf.w = __uint_as_float(qr.y & 0xffff0000u);
        *reinterpret_cast<float4 *>(KQ + (c * 2 * C + t) * 4) = kf;
        *reinterpret_cast<float4 *>(KQ + (c * 2 * C + C + t) * 4) = qf;
      }
    };
    // K of a raw stage, transposed: unit (row d', k-chunk c4) holds K[4 c4 .. 4 c4 + 3][d']
    auto cook_kt = [&](const unsigned char *raw) {
      const __nv_bfloat16 *rk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_K);
#pragma unroll 2
      for (int e = h; e < (C / 4) * DK; e += 128) {
        const int dd = e % DK, c4 = e / DK;
        float4 f;
        f.x = __bfloat162float(rk[(4 * c4 + 0) * DK + dd]);
        f.y = __bfloat162float(rk[(4 * c4 + 1) * DK + dd]);
        f.z = __bfloat162float(rk[(4 * c4 + 2) * DK + dd]);
        f.w = __bfloat162float(rk[(4 * c4 + 3) * DK + dd]);
        *reinterpret_cast<float4 *>(Kt + (c4 * DK + dd) * 4) = f;
      }
    };
    // beta = sigmoid(logit) of this helper's row for every token of a raw stage (App. B.2), written over the
    // logits: all helpers read their logits first, then all write
    auto cook_be = [&](unsigned char *raw) {
      const __nv_bfloat16 *rb = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_B);
      float *bes = reinterpret_cast<float *>(raw + Cf::R_B);
      float be[C];
#pragma unroll
      for (int t = 0; t < C; ++t) be[t] = sigmoid_approx(__bfloat162float(rb[(t * J + j) * COLS + dl]));
      named_bar_sync(3, 128);
#pragma unroll
      for (int t = 0; t < C; ++t) bes[t * NROW + h] = be[t];
    };
    // low part of W after an update: W_lo = W - hi(W), this helper's tensor-memory lane
    auto refresh_wlo = [&]() {
#pragma unroll
      for (int half = 0; half < DK / 64; ++half) {
        float w[4][16];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) tmem_ld16(tb + Cf::TM_W + half * 64 + cc * 16, w[cc]);
        tmem_ld_wait();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
#pragma unroll
          for (int i = 0; i < 16; ++i) w[cc][i] = w[cc][i] - tf32_hi(w[cc][i]);
          tmem_st16(tb + Cf::TM_WLO + half * 64 + cc * 16, w[cc]);
        }
      }
      tmem_st_wait();
      tc_fence_before_sync();
    };
    // Gram rows (tensor-memory lanes 0..C-1, helper warp 4 only) -> shared memory: K K^T row-major for the
    // row warps; K Q^T as the B operand of the readout MMA -- transposed (rows = later token t, K index
    // = earlier token s = this lane), causally masked (s <= t), split into hi / lo TF32 parts
    auto spill_gram = [&](int n) {
      float *Gkk = G_all + (n & 1) * C * C;
      float *Bhi = reinterpret_cast<float *>(BQ_all + (n & 1) * 2 * Cf::BQ_TILE);
      float *Blo = reinterpret_cast<float *>(BQ_all + (n & 1) * 2 * Cf::BQ_TILE + Cf::BQ_TILE);
#pragma unroll
      for (int cc = 0; cc < C / 16; ++cc) {
        float a[16], b[16];
        tmem_ld16(tb + Cf::TM_G + cc * 16, a);
        tmem_ld16(tb + Cf::TM_G + C + cc * 16, b);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<float4 *>(Gkk + lane * C + cc * 16 + i * 4) = make_float4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int t = cc * 16 + i;
          const float val = (lane <= t) ? b[i] : 0.f;
          const float hi = tf32_hi(val);
          const int idx = (lane >> 2) * (Cf::BQ_LBO / 4) + t * 4 + (lane & 3);
          Bhi[idx] = hi;
          Blo[idx] = val - hi;
        }
      }
      tc_fence_before_sync();
      fence_async_smem();
    };

    // ---- prologue: stage chunks 0 and 1, state row -> tensor memory, operands of chunk 0 ----
    chunk_issue_raw<Cf>(p, smem + Cf::OFF_RAW, smem + Cf::OFF_RPQ, tok0, 0, col0, h);
    cp_async_commit();
    if (nchunks > 1)
      chunk_issue_raw<Cf>(p, smem + Cf::OFF_RAW + Cf::RAW_BYTES, smem + Cf::OFF_RPQ + Cf::RPQ_BYTES, tok0, C, col0, h);
    cp_async_commit();
    {
      const float *src = (p.W_in && col_ok) ? p.W_in + (((size_t)bh * J + j) * p.Dv + col) * DK : nullptr;
#pragma unroll
      for (int cc = 0; cc < DK / 16; ++cc) {
        float w[16], lo[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
          if (src) t = __ldcs(reinterpret_cast<const float4 *>(src + cc * 16 + i * 4));
          w[4 * i] = t.x; w[4 * i + 1] = t.y; w[4 * i + 2] = t.z; w[4 * i + 3] = t.w;
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) lo[i] = w[i] - tf32_hi(w[i]);
        tmem_st16(tb + Cf::TM_W + cc * 16, w);
        tmem_st16(tb + Cf::TM_WLO + cc * 16, lo);
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&bars[B_WLO]);
    }
    cp_async_wait<1>();
    named_bar_sync(1, 128);  // every helper's copies of chunk 0 have landed
    cook_kq(smem + Cf::OFF_RAW, KQ_all);
    cook_be(smem + Cf::OFF_RAW);
    fence_async_smem();
    mbar_arrive(&bars[B_KQ]);
    cook_kt(smem + Cf::OFF_RAW);
    fence_async_smem();
    mbar_arrive(&bars[B_KT]);
    if (warp == 4) {
      if (!mbar_wait(&bars[B_G], 0)) failed = true;
      tc_fence_after_sync();
      if (!failed) spill_gram(0);
      mbar_arrive(&bars[B_GS]);
    }

#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const bool more = n + 1 < nchunks;
      unsigned char *raw_next = smem + Cf::OFF_RAW + ((n + 1) & 1) * Cf::RAW_BYTES;
      // (1) operands of chunk n+1: its raw stage has landed, and the K/Q tile it goes to was last read by
      //     the MMAs of chunk n-1, which completed before the update of chunk n-1 this warp waited for
      cp_async_wait<0>();
      named_bar_sync(1, 128);
      if (more) {
        cook_kq(raw_next, KQ_all + ((n + 1) & 1) * 2 * C * DK);
        cook_be(raw_next);
        fence_async_smem();
        mbar_arrive(&bars[B_KQ]);
        if (warp == 4) {  // Gram matrices of chunk n+1
          if (!mbar_wait(&bars[B_G], (n + 1) & 1)) { failed = true; }
          tc_fence_after_sync();
          if (!failed) spill_gram(n + 1);
          mbar_arrive(&bars[B_GS]);
        }
      }
      
      
      // (3) chunk n is finished by the row warps: stage chunk n+2 into the buffers chunk n used
      if (!mbar_wait(&bars[B_C], n & 1)) { failed = true; break; }
      
      
      if (n + 2 < nchunks)
        chunk_issue_raw<Cf>(p, smem + Cf::OFF_RAW + (n & 1) * Cf::RAW_BYTES, smem + Cf::OFF_RPQ + ((n + 2) & 3) * Cf::RPQ_BYTES,
                            tok0, (n + 2) * C, col0, h);
      cp_async_commit();
      // (4) W has been updated with chunk n: refresh its low part, then the transposed K of chunk n+1
      if (more) {
        if (!mbar_wait(&bars[B_U], n & 1)) { failed = true; break; }
        tc_fence_after_sync();
        refresh_wlo();
        mbar_arrive(&bars[B_WLO]);
        cook_kt(raw_next);
        fence_async_smem();
        mbar_arrive(&bars[B_KT]);
      }
      
      
    }
    cp_async_wait<0>();
  } else if (lane == 0) {
    // =============================== MMA issuer ==============================================
    constexpr uint32_t idE = idesc_tf32(128, 2 * C);  // [P0 | Q0] and [Gkk | Gkq]: N = 2C
    constexpr uint32_t idU = idesc_tf32(128, DK);
    const uint64_t kq_desc[2] = {smem_desc_kmajor(smem_u32(KQ_all), 2 * C * 16, 128),
                                 smem_desc_kmajor(smem_u32(KQ_all + 2 * C * DK), 2 * C * 16, 128)};
    const uint64_t kt0 = smem_desc_kmajor(smem_u32(Kt), DK * 16, 128);
    auto gram = [&](int chunk) {
      const uint64_t kq0 = kq_desc[chunk & 1];
#pragma unroll 1
      for (int ks = 0; ks < DK / 8; ++ks) {
        const uint64_t d = kq0 + (uint64_t)(ks * 2 * 2 * C);  // start address advances in 16-byte units
        mma_tf32_ss(tb0 + Cf::TM_G, d, d, idE, ks > 0);        // rows >= C of the A tile are don't-care
      }
      mma_commit(&bars[B_G]);
    };
    auto w_times_kq = [&](int chunk, int w_col, bool first) {
      const uint64_t kq0 = kq_desc[chunk & 1];
#pragma unroll 1
      for (int ks = 0; ks < DK / 8; ++ks)
        mma_tf32_ts(tb0 + Cf::TM_PQ, tb0 + w_col + ks * 8, kq0 + (uint64_t)(ks * 2 * 2 * C), idE, !(first && ks == 0));
    };
    constexpr uint32_t idQ = idesc_tf32(128, C);
    // readouts of chunk n: QD += Cmat (K Q^T masked)  -- c_hi B_hi + c_lo B_hi + c_hi B_lo
    auto readout = [&](int n) {
      const uint64_t bh0 = smem_desc_kmajor(smem_u32(BQ_all + (n & 1) * 2 * Cf::BQ_TILE), Cf::BQ_LBO, 128);
      const uint64_t bl0 = smem_desc_kmajor(smem_u32(BQ_all + (n & 1) * 2 * Cf::BQ_TILE + Cf::BQ_TILE), Cf::BQ_LBO, 128);
      const uint32_t d = tb0 + Cf::TM_QD + (n & 1) * C;
#pragma unroll 1
      for (int ks = 0; ks < C / 8; ++ks) {
        const uint64_t adv = (uint64_t)(ks * 2 * (Cf::BQ_LBO / 16));
        mma_tf32_ts(d, tb0 + Cf::TM_CHI + ks * 8, bh0 + adv, idQ, true);
        mma_tf32_ts(d, tb0 + Cf::TM_CLO + ks * 8, bh0 + adv, idQ, true);
        mma_tf32_ts(d, tb0 + Cf::TM_CHI + ks * 8, bl0 + adv, idQ, true);
      }
      mma_commit(&bars[B_QD]);
    };
    if (!mbar_wait(&bars[B_KQ], 0)) failed = true;
    tc_fence_after_sync();
    if (!failed) gram(0);
    if (!failed && !mbar_wait(&bars[B_WLO], 0)) failed = true;
    tc_fence_after_sync();
    if (!failed) {
      w_times_kq(0, Cf::TM_W, true);
      w_times_kq(0, Cf::TM_WLO, false);
      mma_commit(&bars[B_E]);
    }
#pragma unroll 1
    for (int n = 0; n < nchunks && !failed; ++n) {
      const bool more = n + 1 < nchunks;
      if (more) {
        if (!mbar_wait(&bars[B_KQ], (n + 1) & 1)) { failed = true; break; }
        tc_fence_after_sync();
        gram(n + 1);
      }
      if (!mbar_wait(&bars[B_C], n & 1) || !mbar_wait(&bars[B_KT], n & 1)) { failed = true; break; }
      tc_fence_after_sync();
#pragma unroll 1
      for (int ks = 0; ks < C / 8; ++ks) {  // W += Cmat K (Eq. 3.3 summed over the chunk)
        const uint64_t bt = kt0 + (uint64_t)(ks * 2 * DK);
        mma_tf32_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CHI + ks * 8, bt, idU, true);
        mma_tf32_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CLO + ks * 8, bt, idU, true);
      }
      mma_commit(&bars[B_U]);
      if (more) {
        w_times_kq(n + 1, Cf::TM_W, true);  // executes after the update: MMAs of one thread run in order
        if (!mbar_wait(&bars[B_WLO], (n + 1) & 1)) { failed = true; break; }
        tc_fence_after_sync();
        w_times_kq(n + 1, Cf::TM_WLO, false);
        mma_commit(&bars[B_E]);
      }
      readout(n);  // not needed before the outputs are formed one chunk later: off the critical path
    }
  }
  if (failed) atomicExch(&g_chunk_error, 1);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 8) tmem_dealloc(tb0, Cf::TM_ALLOC);
#ifdef SWILA_CHUNK_PROFILE
  if (tid == 0 && blockIdx.x < 1024) g_chunk_blk[blockIdx.x] = clock64() - prof_t0;
  if (blockIdx.x == 0 && (tid & 127) == 0 && tid < 512) {
    for (int i = 0; i < 8; ++i) g_chunk_prof[(tid >> 7) * 8 + i] = prof_acc[i];
  }
#endif
}

template <int J, int DK>
int launch_chunk(const LaunchArgs &a) {
  using Cf = ChunkCfg<J, DK>;
  auto kern = a.p.r_debug ? swila_chunk_kernel<Cf, true> : swila_chunk_kernel<Cf, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cf::SMEM_BYTES);
  if (e != cudaSuccess) return (int)e;
  const long long nslice = (a.p.Dv + Cf::COLS - 1) / Cf::COLS;
  const long long grid = nslice * a.p.B * a.p.H;
  if (grid <= 0 || grid > 0x7fffffffLL) return (int)cudaErrorInvalidConfiguration;
  kern<<<(unsigned)grid, Cf::NT, Cf::SMEM_BYTES, a.stream>>>(a.p);
  return (int)cudaGetLastError();
}

}  // namespace swila
