// Sequential-scan kernel of the SwiLA recurrence (Sec. 3.2, Eqs. 3.3-3.5) for sm_100a.
//
// Parallel decomposition.  Every output dimension d of every (batch, head) is an
// independent recurrence over t with a J x Dk state (Sec. 3.1: each output dimension
// selects its own component), so the grid is (B*H) x (Dv / COLS) thread blocks and a
// block owns COLS output columns of one head for the whole sequence.  A column is served
// by G = Dk / L adjacent lanes; each lane keeps L key dimensions of all J components in
// registers (J*L <= 128 floats) for the whole call.  Key dimensions are dealt to the G
// lanes in interleaved groups of four, so that state loads/stores and the shared-memory
// reads of k and q are 16-byte vectors whose addresses are contiguous across the G lanes.
//
// Per token: pass A forms the J predictions w_jd . k_t (packed FP32 FMAs, then log2(G)
// xor-shuffles), the E-step is evaluated redundantly by the G lanes (bitwise identical
// inputs), pass B applies the rank-one update and accumulates w_jd . q_t on the UPDATED
// state, and a second shuffle reduction yields o_td.
//
// Staging.  Per-token inputs arrive through a 3-stage cp.async ring of TB-token blocks
// ("raw", io dtype).  Once per block all threads "cook" the next block into fp32 shared
// memory: k, q, v converted, beta = sigmoid(logit), the query prior softmaxed, the key
// prior scaled to base-2 logits (or softmaxed when TEMPORAL) -- each activation computed
// once per block instead of once per lane.  One __syncthreads per token block.
//
// The single-token decode step is this same kernel with T = 1, so prefill and decode share
// every instruction of the token update and agree bit for bit.
#pragma once

#include "swila_common.cuh"

namespace swila {

template <typename IO_, int J_, int DK_, int NT_, int TB_, int GATE_, int LCAP_ = 64>
struct ScanCfg {
  using IO = IO_;
  static constexpr int J = J_, DK = DK_, NT = NT_, TB = TB_, GATE = GATE_;
  static constexpr int L0 = (J * DK >= 128) ? (128 / J) : DK;
  static constexpr int L = L0 > LCAP_ ? LCAP_ : L0;           // key dims per lane (J*L <= 128 state registers)
  static constexpr int G = DK / L;                            // lanes per output column
  static constexpr int COLS = NT / G;                         // output columns per block
  static constexpr int ES = (int)sizeof(IO);
  static constexpr int S = 3;                                 // raw ring depth
  // resident blocks per SM the register budget is sized for
  static constexpr int MIN_BLOCKS = (NT <= 128) ? ((J * L <= 64 && NT * 4 <= 512) ? 4 : 2) : 1;
  static_assert(L >= 4 && L % 4 == 0 && G >= 1 && G <= 32 && (G & (G - 1)) == 0, "lane split");
  static_assert((COLS * ES) % 16 == 0, "column slice must be a whole number of 16-byte chunks");

  // ---- raw stage (bytes) ----
  static constexpr int R_K = 0;
  static constexpr int R_Q = R_K + TB * DK * ES;
  static constexpr int R_V = R_Q + TB * DK * ES;
  static constexpr int R_B = R_V + TB * COLS * ES;
  static constexpr int R_PK = R_B + TB * J * COLS * ES;
  static constexpr int R_PQ = R_PK + TB * J * COLS * ES;
  static constexpr int R_GK = R_PQ + TB * J * COLS * ES;
  static constexpr int R_GQ = R_GK + TB * COLS * ES;
  static constexpr int R_A = R_GQ + TB * COLS * ES;
  // decays staged with the block: one per key dimension [TB][J][DK], or (GATE == 2) one per output dimension, the
  // block's column slice [TB][J][COLS]; one per component is read in place (J values per token)
  static constexpr int RAW_BYTES = R_A + (GATE == 1 ? TB * J * DK * 4 : (GATE == 2 ? TB * J * COLS * 4 : 0));
  // 16-byte chunks per token of each segment
  static constexpr int C_K = DK * ES / 16;
  static constexpr int C_V = COLS * ES / 16;
  static constexpr int C_A = (GATE == 1) ? J * DK * 4 / 16 : ((GATE == 2) ? J * COLS * 4 / 16 : 0);
  static constexpr int CH_BASE = 2 * C_K + C_V + 3 * J * C_V;  // k q v beta pik piq
  static constexpr int CH_TEMP = 2 * C_V;
  // ---- cooked stage (floats) ----
  static constexpr int K_K = 0;
  static constexpr int K_Q = K_K + TB * DK;
  static constexpr int K_V = K_Q + TB * DK;
  static constexpr int K_B = K_V + TB * COLS;
  static constexpr int K_LK = K_B + TB * COLS * J;
  static constexpr int K_PQ = K_LK + TB * COLS * J;
  static constexpr int K_GK = K_PQ + TB * COLS * J;
  static constexpr int K_GQ = K_GK + TB * COLS;
  static constexpr int K_AR = K_GQ + TB * COLS;
  static constexpr int COOKED_FLOATS = K_AR + (GATE == 2 ? TB * COLS * J : 0);
  static constexpr int O_BYTES = TB * COLS * ES;
  static constexpr int OFF_COOKED = S * RAW_BYTES;
  static constexpr int OFF_O = OFF_COOKED + 2 * COOKED_FLOATS * 4;
  static constexpr int SMEM_BYTES = OFF_O + 2 * O_BYTES;
  static_assert(RAW_BYTES % 16 == 0 && (COOKED_FLOATS * 4) % 16 == 0, "alignment");
};

// ---- issue the cp.async copies of one token block into a raw stage ---------------------
template <class C>
__device__ __forceinline__ void issue_block(const ScanParams &p, unsigned char *raw, size_t tok0, int t0,
                                            int col0, int tid) {
  using IO = typename C::IO;
  constexpr int J = C::J, DK = C::DK, NT = C::NT, TB = C::TB, GATE = C::GATE;
  (void)J; (void)DK; (void)NT; (void)TB; (void)GATE;
  constexpr int ES = C::ES, COLS = C::COLS;
  const int nvalid = min(TB, p.T - t0);
  // chunks per token; both candidates are compile-time constants so the divisions below
  // become multiply-shifts
  constexpr int CH_N = C::CH_BASE + C::C_A, CH_T = CH_N + C::CH_TEMP;
  const int CH = p.temporal ? CH_T : CH_N;
  const int total = TB * CH;
  for (int c = tid; c < total; c += NT) {
    const int s = p.temporal ? c / CH_T : c / CH_N;
    int cc = c - s * CH;
    const size_t tok = tok0 + (size_t)(t0 + s);
    const bool tvalid = s < nvalid;
    const char *src;
    unsigned char *dst;
    bool valid = tvalid;
    if (cc < 2 * C::C_K) {  // k, q rows
      const bool isq = cc >= C::C_K;
      if (isq) cc -= C::C_K;
      src = (const char *)(isq ? p.q : p.k) + (tok * DK) * ES + cc * 16;
      dst = raw + (isq ? C::R_Q : C::R_K) + s * DK * ES + cc * 16;
    } else {
      cc -= 2 * C::C_K;
      if (cc < C::C_V) {  // v slice
        const int col = col0 + cc * (16 / ES);
        valid = valid && col < p.Dv;
        src = (const char *)p.v + (tok * p.Dv + col) * ES;
        dst = raw + C::R_V + s * COLS * ES + cc * 16;
      } else {
        cc -= C::C_V;
        if (cc < 3 * J * C::C_V) {  // beta / pik / piq slices, one row per component
          const int which = cc / (J * C::C_V);
          cc -= which * (J * C::C_V);
          const int j = cc / C::C_V;
          cc -= j * C::C_V;
          const int col = col0 + cc * (16 / ES);
          valid = valid && col < p.Dv;
          const void *base = which == 0 ? p.beta_logit : (which == 1 ? p.pik_logit : p.piq_logit);
          src = (const char *)base + ((tok * J + j) * (size_t)p.Dv + col) * ES;
          dst = raw + (which == 0 ? C::R_B : (which == 1 ? C::R_PK : C::R_PQ)) + ((s * J + j) * COLS) * ES + cc * 16;
        } else {
          cc -= 3 * J * C::C_V;
          if (p.temporal && cc < C::CH_TEMP) {  // temporal gate logits
            const bool isq = cc >= C::C_V;
            if (isq) cc -= C::C_V;
            const int col = col0 + cc * (16 / ES);
            valid = valid && col < p.Dv;
            src = (const char *)(isq ? p.gq_logit : p.gk_logit) + (tok * p.Dv + col) * ES;
            dst = raw + (isq ? C::R_GQ : C::R_GK) + s * COLS * ES + cc * 16;
          } else if constexpr (GATE == 2) {  // decay per output dimension: this block's columns, fp32 [J][COLS] per token
            if (p.temporal) cc -= C::CH_TEMP;
            const int j = cc / (COLS / 4), c4 = cc - j * (COLS / 4);
            const int col = col0 + c4 * 4;
            valid = valid && col < p.Dv && p.gran == SWILA_GATE_PER_OUT;
            src = (const char *)p.alpha + ((tok * J + j) * (size_t)p.Dv + col) * 4;
            dst = raw + C::R_A + ((s * J + j) * COLS + c4 * 4) * 4;
          } else {  // per-key decay, fp32 [J][DK] per token
            if (p.temporal) cc -= C::CH_TEMP;
            src = (const char *)p.alpha + (tok * J * DK) * 4 + cc * 16;
            dst = raw + C::R_A + s * J * DK * 4 + cc * 16;
          }
        }
      }
    }
    cp_async16(dst, valid ? (const void *)src : (const void *)p.k, valid ? 16 : 0);
  }
}

// ---- cook one raw block into fp32 operands ---------------------------------------------
template <class C>
__device__ __forceinline__ void cook_block(const ScanParams &p, const unsigned char *raw, float *ck, size_t tok0,
                                           int t0, int col0, int tid) {
  using IO = typename C::IO;
  constexpr int J = C::J, DK = C::DK, NT = C::NT, TB = C::TB, GATE = C::GATE;
  (void)J; (void)DK; (void)NT; (void)TB; (void)GATE;
  constexpr int COLS = C::COLS;
  const int nvalid = min(TB, p.T - t0);
  const IO *rk = reinterpret_cast<const IO *>(raw + C::R_K);
  const IO *rq = reinterpret_cast<const IO *>(raw + C::R_Q);
  if (!p.qkv_act) {
    // k, q: straight conversion
    for (int i = tid; i < nvalid * DK / 4; i += NT) {
      float4 a, b;
      a.x = to_f32(rk[4 * i]); a.y = to_f32(rk[4 * i + 1]); a.z = to_f32(rk[4 * i + 2]); a.w = to_f32(rk[4 * i + 3]);
      b.x = to_f32(rq[4 * i]); b.y = to_f32(rq[4 * i + 1]); b.z = to_f32(rq[4 * i + 2]); b.w = to_f32(rq[4 * i + 3]);
      reinterpret_cast<float4 *>(ck + C::K_K)[i] = a;
      reinterpret_cast<float4 *>(ck + C::K_Q)[i] = b;
    }
  } else {
    // raw projections: SiLU, then division by the L2 norm over the key dimension (App. B.2, App. D.1).  A token's
    // DK / 4 work items sit in adjacent lanes of one warp (DK / 4 divides 32 and NT is a multiple of 32), so the
    // sums of squares are xor-shuffles; every thread runs every trip of the loop.
    constexpr int LPT = DK / 4;
    static_assert(LPT <= 32 && 32 % LPT == 0 && NT % 32 == 0, "a token's lanes must share a warp");
    const int items = nvalid * LPT;
    for (int i0 = 0; i0 < items; i0 += NT) {
      const int i = i0 + tid;
      const bool on = i < items;
      float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
      if (on) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { a[e] = silu_approx(to_f32(rk[4 * i + e])); b[e] = silu_approx(to_f32(rq[4 * i + e])); }
      }
      float sa = a[0] * a[0] + a[1] * a[1] + a[2] * a[2] + a[3] * a[3];
      float sb = b[0] * b[0] + b[1] * b[1] + b[2] * b[2] + b[3] * b[3];
#pragma unroll
      for (int off = 1; off < LPT; off <<= 1) {
        sa += __shfl_xor_sync(0xffffffffu, sa, off);
        sb += __shfl_xor_sync(0xffffffffu, sb, off);
      }
      const float ia = rsqrtf(sa + kL2Eps), ib = rsqrtf(sb + kL2Eps);
      if (on) {
        reinterpret_cast<float4 *>(ck + C::K_K)[i] = make_float4(a[0] * ia, a[1] * ia, a[2] * ia, a[3] * ia);
        reinterpret_cast<float4 *>(ck + C::K_Q)[i] = make_float4(b[0] * ib, b[1] * ib, b[2] * ib, b[3] * ib);
      }
    }
  }
  // per (token, column): v and the gate activations
  const IO *rv = reinterpret_cast<const IO *>(raw + C::R_V);
  const IO *rb = reinterpret_cast<const IO *>(raw + C::R_B);
  const IO *rpk = reinterpret_cast<const IO *>(raw + C::R_PK);
  const IO *rpq = reinterpret_cast<const IO *>(raw + C::R_PQ);
  const IO *rgk = reinterpret_cast<const IO *>(raw + C::R_GK);
  const IO *rgq = reinterpret_cast<const IO *>(raw + C::R_GQ);
  for (int i = tid; i < nvalid * COLS; i += NT) {
    const int s = i / COLS, c = i - s * COLS;
    ck[C::K_V + i] = p.qkv_act ? silu_approx(to_f32(rv[i])) : to_f32(rv[i]);
    float be[J], lk[J], pq[J];
#pragma unroll
    for (int j = 0; j < J; ++j) {
      be[j] = sigmoid_approx(to_f32(rb[(s * J + j) * COLS + c]));
      lk[j] = to_f32(rpk[(s * J + j) * COLS + c]) * kLog2e;
      pq[j] = to_f32(rpq[(s * J + j) * COLS + c]) * kLog2e;
    }
    // query-side prior: softmax over j (App. B.2)
    float m = pq[0];
#pragma unroll
    for (int j = 1; j < J; ++j) m = fmaxf(m, pq[j]);
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < J; ++j) { pq[j] = ex2_approx(pq[j] - m); sum += pq[j]; }
    float inv = rcp_approx(sum);
#pragma unroll
    for (int j = 0; j < J; ++j) pq[j] *= inv;
    if (p.temporal) {
      // the key-side prior enters a convex combination (App. B.3): it must be normalised
      float mk = lk[0];
#pragma unroll
      for (int j = 1; j < J; ++j) mk = fmaxf(mk, lk[j]);
      float sk = 0.f;
#pragma unroll
      for (int j = 0; j < J; ++j) { lk[j] = ex2_approx(lk[j] - mk); sk += lk[j]; }
      float invk = rcp_approx(sk);
#pragma unroll
      for (int j = 0; j < J; ++j) lk[j] *= invk;
      ck[C::K_GK + i] = sigmoid_approx(to_f32(rgk[i]));
      ck[C::K_GQ + i] = sigmoid_approx(to_f32(rgq[i]));
    }
#pragma unroll
    for (int j = 0; j < J; ++j) {
      ck[C::K_B + i * J + j] = be[j];
      ck[C::K_LK + i * J + j] = lk[j];
      ck[C::K_PQ + i * J + j] = pq[j];
    }
    if constexpr (GATE == 2) {
      // one decay value per (component, output column), staged with the block -- or per component, read in place
      const size_t tok = tok0 + (size_t)(t0 + s);
      const int col = col0 + c;
#pragma unroll
      for (int j = 0; j < J; ++j) {
        float a = 1.f;
        if (col < p.Dv)
          a = (p.gran == SWILA_GATE_PER_OUT) ? reinterpret_cast<const float *>(raw + C::R_A)[(s * J + j) * COLS + c]
                                             : __ldg(p.alpha + tok * J + j);
        ck[C::K_AR + i * J + j] = a;
      }
    }
  }
}

// ---- write a finished block of outputs ---------------------------------------------------
template <class C>
__device__ __forceinline__ void flush_o(const ScanParams &p, const unsigned char *ob, size_t tok0, int t0, int col0,
                                        int tid) {
  using IO = typename C::IO;
  constexpr int J = C::J, DK = C::DK, NT = C::NT, TB = C::TB, GATE = C::GATE;
  (void)J; (void)DK; (void)NT; (void)TB; (void)GATE;
  const int nvalid = min(TB, p.T - t0);
  for (int c = tid; c < nvalid * C::C_V; c += NT) {
    const int s = c / C::C_V, cc = c - s * C::C_V;
    const int col = col0 + cc * (16 / C::ES);
    if (col < p.Dv) {
      const uint4 val = *reinterpret_cast<const uint4 *>(ob + s * C::COLS * C::ES + cc * 16);
      *reinterpret_cast<uint4 *>((char *)p.o + ((tok0 + (size_t)(t0 + s)) * p.Dv + col) * C::ES) = val;
    }
  }
}

// ---- the kernel ---------------------------------------------------------------------------
// AUX: the instantiation that also writes the responsibilities (r_debug) and / or forms the sums over time of the
// mixture weights (Sec. 3.5); run-time tests of those pointers stay out of the plain instantiation's serial chain.
template <class C, bool POST, bool AUX>
__global__ void __launch_bounds__(C::NT, C::MIN_BLOCKS) swila_scan_kernel(const __grid_constant__ ScanParams p) {
  using IO = typename C::IO;
  constexpr int J = C::J, DK = C::DK, NT = C::NT, TB = C::TB, GATE = C::GATE;
  (void)J; (void)DK; (void)NT; (void)TB; (void)GATE;
  constexpr int L = C::L, G = C::G, COLS = C::COLS, S = C::S;
  if (p.guard && p.guard_runs_scan && *p.guard == 0u) return;  // the chunked kernel took this call
  extern __shared__ __align__(16) unsigned char smem[];
  float *cooked = reinterpret_cast<float *>(smem + C::OFF_COOKED);
  unsigned char *obuf = smem + C::OFF_O;

  const int tid = threadIdx.x;
  const int nslice = (p.Dv + COLS - 1) / COLS;
  const int bh = blockIdx.x / nslice;
  const int col0 = (blockIdx.x - bh * nslice) * COLS;
  const int lcol = tid / G, g = tid % G;
  const int col = col0 + lcol;
  const bool col_ok = col < p.Dv;
  const size_t tok0 = (size_t)bh * p.T;
  const bool temporal = p.temporal != 0;

  // ---- state slice -> registers: lane g holds key dims (i*G + g)*4 .. +3, i = 0..L/4-1 ----
  float2 w[J][L / 2];
  float rprev[J], rho[J];
  [[maybe_unused]] float st_r[J], st_q[J], st_re = 0.f, st_qe = 0.f;  // AUX: sums over time, entropies in bits
#pragma unroll
  for (int j = 0; j < J; ++j) st_r[j] = st_q[j] = 0.f;
#pragma unroll
  for (int j = 0; j < J; ++j) {
    const float *src = p.W_in ? p.W_in + (((size_t)bh * J + j) * p.Dv + col) * DK : nullptr;
#pragma unroll
    for (int i = 0; i < L / 4; ++i) {
      float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
      if (src && col_ok) t = __ldcs(reinterpret_cast<const float4 *>(src + (i * G + g) * 4));
      w[j][2 * i] = make_float2(t.x, t.y);
      w[j][2 * i + 1] = make_float2(t.z, t.w);
    }
    rprev[j] = rho[j] = 1.0f / J;
    if (temporal && col_ok) {
      if (p.r_in) rprev[j] = p.r_in[((size_t)bh * J + j) * p.Dv + col];
      if (p.rho_in) rho[j] = p.rho_in[((size_t)bh * J + j) * p.Dv + col];
    }
  }

  const int nblocks = (p.T + TB - 1) / TB;
  // prologue: fill the ring, cook block 0
#pragma unroll
  for (int b = 0; b < S - 1; ++b) {
    if (b < nblocks) issue_block<C>(p, smem + b * C::RAW_BYTES, tok0, b * TB, col0, tid);
    cp_async_commit();
  }
  cp_async_wait<S - 2>();
  __syncthreads();
  if (nblocks > 0) cook_block<C>(p, smem, cooked, tok0, 0, col0, tid);

  for (int nb = 0; nb < nblocks; ++nb) {
    const int t0 = nb * TB;
    cp_async_wait<S - 3>();  // block nb+1 has landed (this thread's copies)
    __syncthreads();         // ... everyone's; cooked[nb&1] visible; block nb-1 fully consumed
    if (nb + S - 1 < nblocks)
      issue_block<C>(p, smem + ((nb + S - 1) % S) * C::RAW_BYTES, tok0, (nb + S - 1) * TB, col0, tid);
    cp_async_commit();
    if (nb > 0) flush_o<C>(p, obuf + ((nb - 1) & 1) * C::O_BYTES, tok0, t0 - TB, col0, tid);
    if (nb + 1 < nblocks)
      cook_block<C>(p, smem + ((nb + 1) % S) * C::RAW_BYTES, cooked + ((nb + 1) & 1) * C::COOKED_FLOATS,
                                          tok0, t0 + TB, col0, tid);

    const float *ck = cooked + (nb & 1) * C::COOKED_FLOATS;
    const float *araw = reinterpret_cast<const float *>(smem + (nb % S) * C::RAW_BYTES + C::R_A);
    IO *ob = reinterpret_cast<IO *>(obuf + (nb & 1) * C::O_BYTES);
    const int nvalid = min(TB, p.T - t0);

    for (int s = 0; s < nvalid; ++s) {
      const float *kt = ck + C::K_K + s * DK;
      const float *qt = ck + C::K_Q + s * DK;
      const float v = ck[C::K_V + s * COLS + lcol];
      float be[J], lk[J], pq[J], arow[J];
      lds_vec<J>(ck + C::K_B + (s * COLS + lcol) * J, be);
      lds_vec<J>(ck + C::K_LK + (s * COLS + lcol) * J, lk);
      lds_vec<J>(ck + C::K_PQ + (s * COLS + lcol) * J, pq);
      if constexpr (GATE == 2) lds_vec<J>(ck + C::K_AR + (s * COLS + lcol) * J, arow);
      // one decay value per state element (App. B.4, the general form): this thread's elements of token t are read
      // where they are used, straight from global memory (the tensor is J*Dv*Dk values per token: no staging helps)
      [[maybe_unused]] const float *ael = nullptr;
      if constexpr (GATE == 3) ael = p.alpha + (((tok0 + (size_t)(t0 + s)) * J) * p.Dv + min(col, p.Dv - 1)) * DK;

      // ---- pass A: predictions w_jd . k_t (on the decayed state when pre-decay, Eq. 3.8) ----
      float2 acc[J];
#pragma unroll
      for (int j = 0; j < J; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < L / 4; ++i) {
        const float4 k4 = *reinterpret_cast<const float4 *>(kt + (i * G + g) * 4);
        const float2 klo = make_float2(k4.x, k4.y), khi = make_float2(k4.z, k4.w);
#pragma unroll
        for (int j = 0; j < J; ++j) {
          if constexpr (GATE == 1 && !POST) {
            const float4 a4 = *reinterpret_cast<const float4 *>(araw + (s * J + j) * DK + (i * G + g) * 4);
            w[j][2 * i] = mul2(w[j][2 * i], make_float2(a4.x, a4.y));
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], make_float2(a4.z, a4.w));
          }
          if constexpr (GATE == 2 && !POST) {
            const float2 a2 = make_float2(arow[j], arow[j]);
            w[j][2 * i] = mul2(w[j][2 * i], a2);
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], a2);
          }
          if constexpr (GATE == 3 && !POST) {
            const float4 a4 = __ldg(reinterpret_cast<const float4 *>(ael + (size_t)j * p.Dv * DK + (i * G + g) * 4));
            w[j][2 * i] = mul2(w[j][2 * i], make_float2(a4.x, a4.y));
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], make_float2(a4.z, a4.w));
          }
          acc[j] = fma2(w[j][2 * i], klo, acc[j]);
          acc[j] = fma2(w[j][2 * i + 1], khi, acc[j]);
        }
      }
      float delta[J];
#pragma unroll
      for (int j = 0; j < J; ++j) {
        float pk = acc[j].x + acc[j].y;
#pragma unroll
        for (int off = 1; off < G; off <<= 1) pk += __shfl_xor_sync(0xffffffffu, pk, off);
        delta[j] = v - pk;
      }

      // ---- E-step (Eq. 3.4) as a base-2 softmax over j of log2(prior) - delta^2 log2(e)/2 ----
      float a[J], rr[J];
      if (temporal) {
        const float gk = ck[C::K_GK + s * COLS + lcol];
#pragma unroll
        for (int j = 0; j < J; ++j) {
          const float prior = fmaf(gk, lk[j] - rprev[j], rprev[j]);  // (1-g) r_{t-1} + g pi^k
          a[j] = fmaf(-kHalfLog2e * delta[j], delta[j], lg2_approx(prior));
        }
      } else {
#pragma unroll
        for (int j = 0; j < J; ++j) a[j] = fmaf(-kHalfLog2e * delta[j], delta[j], lk[j]);
      }
      float m = a[0];
#pragma unroll
      for (int j = 1; j < J; ++j) m = fmaxf(m, a[j]);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < J; ++j) { rr[j] = ex2_approx(a[j] - m); sum += rr[j]; }
      const float inv = rcp_approx(sum);
      float2 c2[J];
#pragma unroll
      for (int j = 0; j < J; ++j) {
        rr[j] *= inv;
        const float c = be[j] * rr[j] * delta[j];
        c2[j] = make_float2(c, c);
      }
      if (temporal) {
        const float gq = ck[C::K_GQ + s * COLS + lcol];
#pragma unroll
        for (int j = 0; j < J; ++j) {
          rprev[j] = rr[j];
          rho[j] = fmaf(gq, pq[j] - rho[j], rho[j]);  // (1-g) rhobar_{t-1} + g pi^q
          pq[j] = rho[j];
        }
      }
      if constexpr (AUX) {  // compile-time: a run-time test here would sit on every token's serial chain
        if (p.r_debug && g == 0 && col_ok) {
#pragma unroll
          for (int j = 0; j < J; ++j) p.r_debug[((tok0 + (size_t)(t0 + s)) * J + j) * p.Dv + col] = rr[j];
        }
        // sums over time (Sec. 3.5).  log2 r_j = a_j - m - log2(sum) and sum_j r_j = 1, so the entropy in bits is
        // log2(sum) - sum_j r_j (a_j - m); a component whose responsibility underflowed adds nothing
        float hk = 0.f, hq = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
          st_r[j] += rr[j];
          st_q[j] += pq[j];
          if (rr[j] > 0.f) hk = fmaf(rr[j], a[j] - m, hk);
          if (pq[j] > 0.f) hq = fmaf(pq[j], lg2_approx(pq[j]), hq);
        }
        st_re += lg2_approx(sum) - hk;
        st_qe -= hq;
      }

      // ---- pass B: M-step (Eq. 3.3 / 3.7) and readout on the updated state (Eq. 3.5) ----
#pragma unroll
      for (int j = 0; j < J; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < L / 4; ++i) {
        const float4 k4 = *reinterpret_cast<const float4 *>(kt + (i * G + g) * 4);
        const float4 q4 = *reinterpret_cast<const float4 *>(qt + (i * G + g) * 4);
        const float2 klo = make_float2(k4.x, k4.y), khi = make_float2(k4.z, k4.w);
        const float2 qlo = make_float2(q4.x, q4.y), qhi = make_float2(q4.z, q4.w);
#pragma unroll
        for (int j = 0; j < J; ++j) {
          if constexpr (GATE == 1 && POST) {
            const float4 a4 = *reinterpret_cast<const float4 *>(araw + (s * J + j) * DK + (i * G + g) * 4);
            w[j][2 * i] = mul2(w[j][2 * i], make_float2(a4.x, a4.y));
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], make_float2(a4.z, a4.w));
          }
          if constexpr (GATE == 2 && POST) {
            const float2 a2 = make_float2(arow[j], arow[j]);
            w[j][2 * i] = mul2(w[j][2 * i], a2);
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], a2);
          }
          if constexpr (GATE == 3 && POST) {
            const float4 a4 = __ldg(reinterpret_cast<const float4 *>(ael + (size_t)j * p.Dv * DK + (i * G + g) * 4));
            w[j][2 * i] = mul2(w[j][2 * i], make_float2(a4.x, a4.y));
            w[j][2 * i + 1] = mul2(w[j][2 * i + 1], make_float2(a4.z, a4.w));
          }
          w[j][2 * i] = fma2(c2[j], klo, w[j][2 * i]);
          w[j][2 * i + 1] = fma2(c2[j], khi, w[j][2 * i + 1]);
          acc[j] = fma2(w[j][2 * i], qlo, acc[j]);
          acc[j] = fma2(w[j][2 * i + 1], qhi, acc[j]);
        }
      }
      float o = 0.f;
#pragma unroll
      for (int j = 0; j < J; ++j) o = fmaf(pq[j], acc[j].x + acc[j].y, o);
#pragma unroll
      for (int off = 1; off < G; off <<= 1) o += __shfl_xor_sync(0xffffffffu, o, off);
      if (g == 0) from_f32(ob[s * COLS + lcol], o);
    }
  }
  __syncthreads();
  if (nblocks > 0) flush_o<C>(p, obuf + ((nblocks - 1) & 1) * C::O_BYTES, tok0, (nblocks - 1) * TB, col0, tid);

  // ---- registers -> state slice ----
  if (p.W_out && col_ok) {
#pragma unroll
    for (int j = 0; j < J; ++j) {
      float *dst = p.W_out + (((size_t)bh * J + j) * p.Dv + col) * DK;
#pragma unroll
      for (int i = 0; i < L / 4; ++i)
        __stcs(reinterpret_cast<float4 *>(dst + (i * G + g) * 4),
               make_float4(w[j][2 * i].x, w[j][2 * i].y, w[j][2 * i + 1].x, w[j][2 * i + 1].y));
    }
  }
  if constexpr (AUX) {
    if (col_ok && g == 0) {  // each element belongs to one thread of one block: plain read-modify-write
      constexpr float kLn2 = 0.6931471805599453f;
#pragma unroll
      for (int j = 0; j < J; ++j) {
        if (p.r_sum) p.r_sum[((size_t)bh * J + j) * p.Dv + col] += st_r[j];
        if (p.rho_sum) p.rho_sum[((size_t)bh * J + j) * p.Dv + col] += st_q[j];
      }
      if (p.r_ent) p.r_ent[(size_t)bh * p.Dv + col] += st_re * kLn2;
      if (p.rho_ent) p.rho_ent[(size_t)bh * p.Dv + col] += st_qe * kLn2;
    }
  }
  if (temporal && col_ok && g == 0) {
#pragma unroll
    for (int j = 0; j < J; ++j) {
      if (p.r_out) p.r_out[((size_t)bh * J + j) * p.Dv + col] = rprev[j];
      if (p.rho_out) p.rho_out[((size_t)bh * J + j) * p.Dv + col] = rho[j];
    }
  }
}

// ---- host-side launch of one instantiation -----------------------------------------------
template <class C, bool POST>
int launch_scan(const LaunchArgs &a) {
  using IO = typename C::IO;
  constexpr int J = C::J, DK = C::DK, NT = C::NT, TB = C::TB, GATE = C::GATE;
  (void)J; (void)DK; (void)NT; (void)TB; (void)GATE;
  const bool aux = a.p.r_debug || a.p.r_sum || a.p.r_ent || a.p.rho_sum || a.p.rho_ent;
  auto kern = aux ? swila_scan_kernel<C, POST, true> : swila_scan_kernel<C, POST, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES);
  if (e != cudaSuccess) return (int)e;
  const long long nslice = (a.p.Dv + C::COLS - 1) / C::COLS;
  const long long grid = nslice * a.p.B * a.p.H;
  if (grid <= 0 || grid > 0x7fffffffLL) return (int)cudaErrorInvalidConfiguration;
  kern<<<(unsigned)grid, NT, C::SMEM_BYTES, a.stream>>>(a.p);
  return (int)cudaGetLastError();
}

}  // namespace swila
