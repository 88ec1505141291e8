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
// One block = 128 threads = 128 rows = COLS = 128/J output columns of one (batch, head); thread r
// serves row (d = r / J, j = r % J), which is also its tensor-memory lane, so the J components
// of a column sit in adjacent lanes of one warp and the E-step normalisation is a few shuffles.
#pragma once

#include "swila_common.cuh"
#include "swila_umma.cuh"

namespace swila {

// Set when a bounded wait on a tensor-core completion barrier expires (never expected).
static __device__ int g_chunk_error = 0;

template <int J_, int DK_>
struct ChunkCfg {
  static constexpr int J = J_, DK = DK_;
  static constexpr int C = 32;           // tokens per chunk
  static constexpr int NT = 128;         // threads = rows
  static constexpr int COLS = NT / J;    // output columns per block
  static constexpr int ES = 2;           // bf16 io
  // tensor-memory columns
  static constexpr int TM_W = 0, TM_WLO = DK, TM_P0 = 2 * DK, TM_Q0 = TM_P0 + C, TM_GKK = TM_Q0 + C,
                       TM_GKQ = TM_GKK + C, TM_CHI = TM_GKQ + C, TM_CLO = TM_CHI + C, TM_USED = TM_CLO + C;
  static constexpr int TM_ALLOC = 512;
  static_assert(TM_USED <= TM_ALLOC, "tensor memory budget");
  // raw stage (bytes): k, q [C][DK], v [C][COLS], beta/pik/piq [C][J][COLS], all bf16
  static constexpr int R_K = 0;
  static constexpr int R_Q = R_K + C * DK * ES;
  static constexpr int R_V = R_Q + C * DK * ES;
  static constexpr int R_B = R_V + C * COLS * ES;
  static constexpr int R_PK = R_B + C * J * COLS * ES;
  static constexpr int R_PQ = R_PK + C * J * COLS * ES;
  static constexpr int RAW_BYTES = R_PQ + C * J * COLS * ES;
  static constexpr int C_K = DK * ES / 16, C_V = COLS * ES / 16;
  static constexpr int CH = 2 * C_K + C_V + 3 * J * C_V;  // 16-byte copies per token
  // shared memory map (bytes)
  static constexpr int OFF_RAW = 0;
  static constexpr int OFF_KB = OFF_RAW + 2 * RAW_BYTES;  // [DK/4][C][4] fp32: K, K-major, rows = tokens
  static constexpr int OFF_QB = OFF_KB + C * DK * 4;      // same for Q
  static constexpr int OFF_KT = OFF_QB + C * DK * 4;      // [C/4][DK][4] fp32: K transposed, rows = key dims
  static constexpr int OFF_BS = OFF_KT + C * DK * 4;      // [C][NT] fp32 beta
  static constexpr int OFF_LK = OFF_BS + C * NT * 4;      // [C][NT] fp32 base-2 key-prior logits
  static constexpr int OFF_PQ = OFF_LK + C * NT * 4;      // [C][NT] fp32 query prior
  static constexpr int OFF_PR = OFF_PQ + C * NT * 4;      // [C][NT] fp32 prior-weighted readouts
  static constexpr int OFF_G = OFF_PR + C * NT * 4;       // Gkk [C][C], Gkq [C][C] fp32
  static constexpr int OFF_MISC = OFF_G + 2 * C * C * 4;  // barriers, tensor-memory base
  static constexpr int SMEM_BYTES = OFF_MISC + 64;
  static_assert(RAW_BYTES % 16 == 0 && (COLS * ES) % 16 == 0, "alignment");
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

template <class Cf>
__device__ __forceinline__ void chunk_issue_raw(const ScanParams &p, unsigned char *raw, size_t tok0, int t0, int col0,
                                                int tid) {
  constexpr int J = Cf::J, DK = Cf::DK, C = Cf::C, COLS = Cf::COLS, ES = Cf::ES, CH = Cf::CH;
  const int nvalid = min(C, p.T - t0);
  for (int c = tid; c < C * CH; c += Cf::NT) {
    const int s = c / CH;
    int cc = c - s * CH;
    const size_t tok = tok0 + (size_t)(t0 + s);
    bool valid = s < nvalid;
    const char *src;
    unsigned char *dst;
    if (cc < 2 * Cf::C_K) {
      const bool isq = cc >= Cf::C_K;
      if (isq) cc -= Cf::C_K;
      src = (const char *)(isq ? p.q : p.k) + (tok * DK) * ES + cc * 16;
      dst = raw + (isq ? Cf::R_Q : Cf::R_K) + s * DK * ES + cc * 16;
    } else {
      cc -= 2 * Cf::C_K;
      if (cc < Cf::C_V) {
        const int col = col0 + cc * (16 / ES);
        valid = valid && col < p.Dv;
        src = (const char *)p.v + (tok * p.Dv + col) * ES;
        dst = raw + Cf::R_V + s * COLS * ES + cc * 16;
      } else {
        cc -= Cf::C_V;
        const int which = cc / (J * Cf::C_V);
        cc -= which * (J * Cf::C_V);
        const int j = cc / Cf::C_V;
        cc -= j * Cf::C_V;
        const int col = col0 + cc * (16 / ES);
        valid = valid && col < p.Dv;
        const void *base = which == 0 ? p.beta_logit : (which == 1 ? p.pik_logit : p.piq_logit);
        src = (const char *)base + ((tok * J + j) * (size_t)p.Dv + col) * ES;
        dst = raw + (which == 0 ? Cf::R_B : (which == 1 ? Cf::R_PK : Cf::R_PQ)) + ((s * J + j) * COLS) * ES + cc * 16;
      }
    }
    cp_async16(dst, valid ? (const void *)src : (const void *)p.k, valid ? 16 : 0);
  }
}

// hi/lo split of an FP32 value for TF32 operands: hi keeps the bits the tensor core reads
// (it ignores the 13 low mantissa bits), lo is the exact remainder.
__device__ __forceinline__ float tf32_hi(float x) { return __uint_as_float(__float_as_uint(x) & 0xffffe000u); }

template <class Cf>
__global__ void __launch_bounds__(Cf::NT, 1) swila_chunk_kernel(const __grid_constant__ ScanParams p) {
  using namespace umma;
  constexpr int J = Cf::J, DK = Cf::DK, C = Cf::C, NT = Cf::NT, COLS = Cf::COLS;
  extern __shared__ __align__(128) unsigned char smem[];
  float *Kb = reinterpret_cast<float *>(smem + Cf::OFF_KB);
  float *Qb = reinterpret_cast<float *>(smem + Cf::OFF_QB);
  float *Kt = reinterpret_cast<float *>(smem + Cf::OFF_KT);
  float *bs = reinterpret_cast<float *>(smem + Cf::OFF_BS);
  float *lks = reinterpret_cast<float *>(smem + Cf::OFF_LK);
  float *pqs = reinterpret_cast<float *>(smem + Cf::OFF_PQ);
  float *prs = reinterpret_cast<float *>(smem + Cf::OFF_PR);
  float *Gkk = reinterpret_cast<float *>(smem + Cf::OFF_G);
  float *Gkq = Gkk + C * C;
  uint64_t *bar1 = reinterpret_cast<uint64_t *>(smem + Cf::OFF_MISC);
  uint64_t *bar2 = bar1 + 1;
  uint32_t *tmem_base_s = reinterpret_cast<uint32_t *>(bar2 + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nslice = (p.Dv + COLS - 1) / COLS;
  const int bh = blockIdx.x / nslice;
  const int col0 = (blockIdx.x - bh * nslice) * COLS;
  const int dl = tid / J, j = tid % J;
  const int col = col0 + dl;
  const bool col_ok = col < p.Dv;
  const size_t tok0 = (size_t)bh * p.T;
  const int jbase = lane - j;  // first lane of this column's J-lane group

  if (warp == 0) tmem_alloc(tmem_base_s, Cf::TM_ALLOC);
  if (tid == 0) {
    mbar_init(bar1, 1);
    mbar_init(bar2, 1);
    mbar_fence_init();
  }
  const int nchunks = (p.T + C - 1) / C;
  chunk_issue_raw<Cf>(p, smem + Cf::OFF_RAW, tok0, 0, col0, tid);
  cp_async_commit();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tb = *tmem_base_s + ((uint32_t)(warp * 32) << 16);  // this warp's lane quarter
  const uint32_t tb0 = *tmem_base_s;

  // ---- initial state row -> tensor memory (W and its low part) ----
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
  }

  bool failed = false;
  for (int n = 0; n < nchunks && !failed; ++n) {
    const int t0 = n * C;
    const int nvalid = min(C, p.T - t0);
    unsigned char *raw = smem + Cf::OFF_RAW + (n & 1) * Cf::RAW_BYTES;
    cp_async_wait<0>();
    __syncthreads();  // raw chunk n landed for everyone; previous chunk fully consumed
    if (n + 1 < nchunks) chunk_issue_raw<Cf>(p, smem + Cf::OFF_RAW + ((n + 1) & 1) * Cf::RAW_BYTES, tok0, t0 + C, col0, tid);
    cp_async_commit();

    // ---- cook: K, Q -> fp32 K-major operand tiles (16-byte unit (row, k-chunk c) at (c*rows + row)*16) ----
    {
      const __nv_bfloat16 *rk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_K);
      const __nv_bfloat16 *rq = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_Q);
      // diagonal walk over 8-token x 16-chunk blocks: conflict-free 8-byte reads and 16-byte writes
      constexpr int NBLK = (C / 8) * (DK / 4 / 16);
#pragma unroll 2
      for (int blk = 0; blk < NBLK; ++blk) {
        const int tb8 = blk % (C / 8), cb16 = blk / (C / 8);
        const int s = tid >> 4, u = tid & 15;
        const int t = tb8 * 8 + ((u + s) & 7), c = cb16 * 16 + u;
        const uint2 kr = *reinterpret_cast<const uint2 *>(rk + t * DK + c * 4);
        const uint2 qr = *reinterpret_cast<const uint2 *>(rq + t * DK + c * 4);
        float4 kf, qf;
        kf.x = __uint_as_float(kr.x << 16); kf.y = __uint_as_float(kr.x & 0xffff0000u);
        kf.z = __uint_as_float(kr.y << 16); kf.w = __uint_as_float(kr.y & 0xffff0000u);
        qf.x = __uint_as_float(qr.x << 16); qf.y = __uint_as_float(qr.x & 0xffff0000u);
        qf.z = __uint_as_float(qr.y << 16); qf.w = __uint_as_float(qr.y & 0xffff0000u);
        *reinterpret_cast<float4 *>(Kb + (c * C + t) * 4) = kf;
        *reinterpret_cast<float4 *>(Qb + (c * C + t) * 4) = qf;
      }
      // K transposed: unit (row d', k-chunk c4) holds K[4 c4 .. 4 c4 + 3][d']
      for (int e = tid; e < (C / 4) * DK; e += NT) {
        const int dd = e % DK, c4 = e / DK;
        float4 f;
        f.x = __bfloat162float(rk[(4 * c4 + 0) * DK + dd]);
        f.y = __bfloat162float(rk[(4 * c4 + 1) * DK + dd]);
        f.z = __bfloat162float(rk[(4 * c4 + 2) * DK + dd]);
        f.w = __bfloat162float(rk[(4 * c4 + 3) * DK + dd]);
        *reinterpret_cast<float4 *>(Kt + (c4 * DK + dd) * 4) = f;
      }
      // this row's gate activations for the chunk (App. B.2): beta = sigmoid, priors = softmax over j
      const __nv_bfloat16 *rb = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_B);
      const __nv_bfloat16 *rpk = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_PK);
      const __nv_bfloat16 *rpq = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_PQ);
#pragma unroll 4
      for (int t = 0; t < C; ++t) {
        const int gi = (t * J + j) * COLS + dl;
        const float be = sigmoid_approx(__bfloat162float(rb[gi]));
        const float lk = __bfloat162float(rpk[gi]) * kLog2e;
        const float x = __bfloat162float(rpq[gi]) * kLog2e;
        float m = x;
#pragma unroll
        for (int off = 1; off < J; off <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
        const float e = ex2_approx(x - m);
        float sum = e;
#pragma unroll
        for (int off = 1; off < J; off <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        bs[t * NT + tid] = be;
        lks[t * NT + tid] = lk;
        pqs[t * NT + tid] = e * rcp_approx(sum);
      }
    }
    fence_async_smem();
    tc_fence_before_sync();
    __syncthreads();

    // ---- tensor cores: P0 = W K^T, Q0 = W Q^T (hi and lo parts of W), Gram matrices ----
    if (tid == 0) {
      tc_fence_after_sync();
      constexpr uint32_t idC = idesc_tf32(128, C);
      const uint64_t bk0 = smem_desc_kmajor(smem_u32(Kb), C * 16, 128);
      const uint64_t bq0 = smem_desc_kmajor(smem_u32(Qb), C * 16, 128);
#pragma unroll 1
      for (int ks = 0; ks < DK / 8; ++ks) {
        const uint64_t bk = bk0 + (uint64_t)(ks * 2 * C);  // start address advances in 16-byte units
        const uint64_t bq = bq0 + (uint64_t)(ks * 2 * C);
        mma_tf32_ts(tb0 + Cf::TM_P0, tb0 + Cf::TM_W + ks * 8, bk, idC, ks > 0);
        mma_tf32_ts(tb0 + Cf::TM_Q0, tb0 + Cf::TM_W + ks * 8, bq, idC, ks > 0);
        mma_tf32_ts(tb0 + Cf::TM_P0, tb0 + Cf::TM_WLO + ks * 8, bk, idC, true);
        mma_tf32_ts(tb0 + Cf::TM_Q0, tb0 + Cf::TM_WLO + ks * 8, bq, idC, true);
        mma_tf32_ss(tb0 + Cf::TM_GKK, bk, bk, idC, ks > 0);  // rows >= C of the A tile are don't-care
        mma_tf32_ss(tb0 + Cf::TM_GKQ, bk, bq, idC, ks > 0);
      }
      mma_commit(bar1);
    }
    failed = !mbar_wait(bar1, n & 1);
    failed = __syncthreads_or(failed);
    if (failed) break;
    tc_fence_after_sync();

    float pred[C], qd[C], cs[16];
#pragma unroll
    for (int cc = 0; cc < C / 16; ++cc) {
      float a[16], b[16];
      tmem_ld16(tb + Cf::TM_P0 + cc * 16, a);
      tmem_ld16(tb + Cf::TM_Q0 + cc * 16, b);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) { pred[cc * 16 + i] = a[i]; qd[cc * 16 + i] = b[i]; }
    }
    if (warp == 0) {  // lanes 0..C-1 hold the Gram rows: spill them to shared memory for everyone
#pragma unroll
      for (int cc = 0; cc < C / 16; ++cc) {
        float a[16], b[16];
        tmem_ld16(tb + Cf::TM_GKK + cc * 16, a);
        tmem_ld16(tb + Cf::TM_GKQ + cc * 16, b);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          *reinterpret_cast<float4 *>(Gkk + lane * C + cc * 16 + i * 4) = make_float4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
          *reinterpret_cast<float4 *>(Gkq + lane * C + cc * 16 + i * 4) = make_float4(b[4 * i], b[4 * i + 1], b[4 * i + 2], b[4 * i + 3]);
        }
      }
    }
    tc_fence_before_sync();
    __syncthreads();

    // ---- sequential part of the chunk: E-step and the triangular corrections, one row per thread ----
    const __nv_bfloat16 *rv = reinterpret_cast<const __nv_bfloat16 *>(raw + Cf::R_V);
#pragma unroll
    for (int t = 0; t < C; ++t) {
      const float v = __bfloat162float(rv[t * COLS + dl]);
      const float delta = v - pred[t];
      const float a = fmaf(-kHalfLog2e * delta, delta, lks[t * NT + tid]);
      float all[J];
#pragma unroll
      for (int jj = 0; jj < J; ++jj) all[jj] = __shfl_sync(0xffffffffu, a, jbase + jj);
      float m = all[0];
#pragma unroll
      for (int jj = 1; jj < J; ++jj) m = fmaxf(m, all[jj]);
      float sum = 0.f;
#pragma unroll
      for (int jj = 0; jj < J; ++jj) sum += ex2_approx(all[jj] - m);
      const float r = ex2_approx(a - m) * rcp_approx(sum);
      float c = bs[t * NT + tid] * r * delta;
      if (t >= nvalid) c = 0.f;  // padding tokens of the last chunk leave the state alone
      cs[t & 15] = c;
      if (p.r_debug != nullptr && col_ok && t < nvalid)
        p.r_debug[((tok0 + (size_t)(t0 + t)) * J + j) * p.Dv + col] = r;
      // push this token's update into the later predictions / readouts of the chunk
#pragma unroll
      for (int u = t + 1; u < C; ++u) pred[u] = fmaf(c, Gkk[t * C + u], pred[u]);
#pragma unroll
      for (int u = t; u < C; ++u) qd[u] = fmaf(c, Gkq[t * C + u], qd[u]);
      prs[t * NT + tid] = pqs[t * NT + tid] * qd[t];
      if ((t & 15) == 15) {  // 16 update coefficients complete: park them in tensor memory (hi / lo)
        float hi[16], lo[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) { hi[i] = tf32_hi(cs[i]); lo[i] = cs[i] - hi[i]; }
        tmem_st16(tb + Cf::TM_CHI + (t - 15), hi);
        tmem_st16(tb + Cf::TM_CLO + (t - 15), lo);
      }
    }

    // ---- W += Cmat K on the tensor cores ----
    tmem_st_wait();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      constexpr uint32_t idD = idesc_tf32(128, DK);
      const uint64_t bt0 = smem_desc_kmajor(smem_u32(Kt), DK * 16, 128);
#pragma unroll 1
      for (int ks = 0; ks < C / 8; ++ks) {
        const uint64_t bt = bt0 + (uint64_t)(ks * 2 * DK);
        mma_tf32_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CHI + ks * 8, bt, idD, true);
        mma_tf32_ts(tb0 + Cf::TM_W, tb0 + Cf::TM_CLO + ks * 8, bt, idD, true);
      }
      mma_commit(bar2);
    }

    // ---- outputs of the chunk (overlaps the update MMAs): o_td = sum_j of the weighted readouts ----
    {
      constexpr int GROUPS = COLS / 8;  // 8 outputs = 16 bytes per store
      for (int e = tid; e < C * GROUPS; e += NT) {
        const int t = e / GROUPS, g8 = e - t * GROUPS;
        if (t < nvalid && col0 + g8 * 8 < p.Dv) {
          __align__(16) __nv_bfloat16 out[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            float o = 0.f;
#pragma unroll
            for (int jj = 0; jj < J; ++jj) o += prs[t * NT + (g8 * 8 + i) * J + jj];
            out[i] = __float2bfloat16_rn(o);
          }
          *reinterpret_cast<uint4 *>((__nv_bfloat16 *)p.o + (tok0 + (size_t)(t0 + t)) * p.Dv + col0 + g8 * 8) =
              *reinterpret_cast<const uint4 *>(out);
        }
      }
    }

    failed = !mbar_wait(bar2, n & 1);
    failed = __syncthreads_or(failed);
    if (failed) break;
    tc_fence_after_sync();
    // ---- refresh the low part of W ----
#pragma unroll
    for (int cc = 0; cc < DK / 16; ++cc) {
      float w[16];
      tmem_ld16(tb + Cf::TM_W + cc * 16, w);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i] = w[i] - tf32_hi(w[i]);
      tmem_st16(tb + Cf::TM_WLO + cc * 16, w);
    }
    tmem_st_wait();
  }
  cp_async_wait<0>();
  if (failed && tid == 0) atomicExch(&g_chunk_error, 1);

  // ---- final state row -> global ----
  if (!failed && p.W_out && col_ok) {
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
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(*tmem_base_s, Cf::TM_ALLOC);
}

template <int J, int DK>
int launch_chunk(const LaunchArgs &a) {
  using Cf = ChunkCfg<J, DK>;
  auto kern = swila_chunk_kernel<Cf>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cf::SMEM_BYTES);
  if (e != cudaSuccess) return (int)e;
  const long long nslice = (a.p.Dv + Cf::COLS - 1) / Cf::COLS;
  const long long grid = nslice * a.p.B * a.p.H;
  if (grid <= 0 || grid > 0x7fffffffLL) return (int)cudaErrorInvalidConfiguration;
  kern<<<(unsigned)grid, Cf::NT, Cf::SMEM_BYTES, a.stream>>>(a.p);
  return (int)cudaGetLastError();
}

}  // namespace swila
