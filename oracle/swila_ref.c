/*
 * CPU oracle for the Switching Linear Attention (SwiLA) recurrence -- TEST
 * INFRASTRUCTURE ONLY.  Plain fp64, one scalar loop nest, no blocking, no fusion,
 * no reordering beyond what the equations state.  It shares no code with the CUDA
 * path and must never be called from it; only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference arm execute it.
 *
 * What it computes, per (batch b, head h), per token t, for every output dimension d
 * and mixture component j (Sec. 3.2):
 *
 *   delta_tjd = v_td - w_{t-1,jd}^T k_t                         (text below Eq. 3.3)
 *   r_tjd     = pi^k_jd exp(-delta^2/2) / sum_j' pi^k_j'd exp(-delta_j'^2/2)   (Eq. 3.4, E-step)
 *   w_tjd     = w_{t-1,jd} + beta_tjd r_tjd delta_tjd k_t       (Eq. 3.3, M-step)
 *   o_td      = sum_j pi^q_jd  w_tjd^T q_t                      (Eq. 3.5, readout on the UPDATED state)
 *
 * with beta = sigmoid(beta_logit) and pi^k, pi^q = softmax over j of their logits
 * (App. B.2).  The E-step is evaluated as a softmax over j of log(prior_j) - delta_j^2/2
 * with the maximum subtracted: identical in exact arithmetic to Eq. 3.4, and free of
 * 0/0 when every Gaussian factor underflows.
 *
 * Variants:
 *   TEMPORAL (App. B.3): rbar_tjd = (1-g^k_td) r_{t-1,jd} + g^k_td pi^k_jd replaces the
 *     key-side prior; rhobar_tjd = (1-g^q_td) rhobar_{t-1,jd} + g^q_td pi^q_jd replaces the
 *     query-side prior; g = sigmoid(logit).  r_{t-1} (the previous posterior) and
 *     rhobar_{t-1} are carried state.
 *   GATED (Sec. 3.4): pre-decay (Eq. 3.8, default): the state is decayed first and
 *     delta, r and the update all use the decayed state; post-decay (Eq. 3.7): delta and r
 *     from the undecayed state, then w = alpha*w + beta r delta k.  Granularity of
 *     alpha (App. B.4): 1 = one gate per key dimension [B,H,T,J,Dk], 2 = per output
 *     dimension [B,H,T,J,Dv], 3 = scalar per component [B,H,T,J], 4 = one gate per state
 *     element [B,H,T,J,Dv,Dk] (the general form, of which 1-3 are restrictions).
 *
 * Layouts (row-major, last index fastest): q,k [B,H,T,Dk]; v,o [B,H,T,Dv];
 * gate logits [B,H,T,J,Dv]; temporal gate logits [B,H,T,Dv]; W [B,H,J,Dv,Dk] (rows =
 * output dims, columns = key dims, App. B.4); r_prev, rho_prev [B,H,J,Dv].
 * Parity status: every function here is pinned by the CPU tests (reductions, closed
 * forms, a hand-worked example, brute force); nothing is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define REF_TEMPORAL 1
#define REF_GATED 2
#define REF_POST_DECAY 4

static double sigmoid_(double x) { return 1.0 / (1.0 + exp(-x)); }

/* softmax over j of x[j*stride], written to out[j] */
static void softmax_(int J, const double *x, size_t stride, double *out) {
  double m = x[0];
  for (int j = 1; j < J; ++j)
    if (x[(size_t)j * stride] > m) m = x[(size_t)j * stride];
  double s = 0.0;
  for (int j = 0; j < J; ++j) {
    out[j] = exp(x[(size_t)j * stride] - m);
    s += out[j];
  }
  for (int j = 0; j < J; ++j) out[j] /= s;
}

/* decay alpha_{t,j,d,c} of state element (component j, output dim d, key dim c) at token `tok`, by granularity
 * (App. B.4, "Granularity of the gate"): 4 = one value per element (the general form), 1 = per key dimension
 * (W Diag(a_tj)), 2 = per output dimension (Diag(alpha_tj) W), 3 = one scalar per component */
static double decay_(const double *alpha, int gran, size_t tok, int j, int d, int c, int J, int Dv, int Dk) {
  switch (gran) {
    case 1: return alpha[(tok * J + j) * (size_t)Dk + c];
    case 2: return alpha[(tok * J + j) * (size_t)Dv + d];
    case 3: return alpha[tok * J + j];
    default: return alpha[((tok * J + j) * (size_t)Dv + d) * (size_t)Dk + c];
  }
}

int swila_ref_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Returns 0 on success, -1 on bad arguments.  W, r_prev, rho_prev are updated in place
 * (they hold the initial state on entry and the final state on return). */
int swila_ref_forward(int B, int H, int T, int Dk, int Dv, int J, int flags, int gran,
                      const double *q, const double *k, const double *v,
                      const double *beta_logit, const double *pik_logit, const double *piq_logit,
                      const double *gk_logit, const double *gq_logit, const double *alpha,
                      double *W, double *r_prev, double *rho_prev, double *o, double *r_out) {
  if (B <= 0 || H <= 0 || T < 0 || Dk <= 0 || Dv <= 0 || J <= 0) return -1;
  const int temporal = (flags & REF_TEMPORAL) != 0;
  const int gated = (flags & REF_GATED) != 0;
  const int post = (flags & REF_POST_DECAY) != 0;
  if (temporal && (!gk_logit || !gq_logit || !r_prev || !rho_prev)) return -1;
  if (gated && (!alpha || gran < 1 || gran > 4)) return -1;
  if (J > 64) return -1;

  const long rows = (long)B * H * Dv;
#pragma omp parallel for schedule(dynamic, 1)
  for (long row = 0; row < rows; ++row) {
    const int d = (int)(row % Dv);
    const size_t bh = (size_t)(row / Dv);
    double pik[64], piq[64], prior[64], rho[64], delta[64], a[64], r[64], wq[64];
    for (int t = 0; t < T; ++t) {
      const size_t tok = bh * (size_t)T + (size_t)t;
      const double *kt = k + tok * Dk;
      const double *qt = q + tok * Dk;
      const double vt = v[tok * Dv + d];
      const size_t g0 = tok * (size_t)J * Dv + d; /* gate logit (t, j=0, d); stride Dv over j */

      /* decay applied before the prediction (pre-decay, Eq. 3.8) */
      if (gated && !post) {
        for (int j = 0; j < J; ++j) {
          double *w = W + ((bh * J + j) * (size_t)Dv + d) * Dk;
          for (int c = 0; c < Dk; ++c) {
            w[c] *= decay_(alpha, gran, tok, j, d, c, J, Dv, Dk);
          }
        }
      }

      /* prediction errors */
      for (int j = 0; j < J; ++j) {
        const double *w = W + ((bh * J + j) * (size_t)Dv + d) * Dk;
        double pred = 0.0;
        for (int c = 0; c < Dk; ++c) pred += w[c] * kt[c];
        delta[j] = vt - pred;
      }

      /* key-side prior */
      softmax_(J, pik_logit + g0, (size_t)Dv, pik);
      if (temporal) {
        const double gk = sigmoid_(gk_logit[tok * Dv + d]);
        for (int j = 0; j < J; ++j)
          prior[j] = (1.0 - gk) * r_prev[(bh * J + j) * (size_t)Dv + d] + gk * pik[j];
      } else {
        for (int j = 0; j < J; ++j) prior[j] = pik[j];
      }

      /* E-step (Eq. 3.4): r = softmax_j(log prior_j - delta_j^2 / 2) */
      double m = -INFINITY;
      for (int j = 0; j < J; ++j) {
        a[j] = log(prior[j]) - 0.5 * delta[j] * delta[j];
        if (a[j] > m) m = a[j];
      }
      double s = 0.0;
      for (int j = 0; j < J; ++j) {
        r[j] = exp(a[j] - m);
        s += r[j];
      }
      for (int j = 0; j < J; ++j) r[j] /= s;
      if (r_out)
        for (int j = 0; j < J; ++j) r_out[g0 + (size_t)j * Dv] = r[j];
      if (temporal)
        for (int j = 0; j < J; ++j) r_prev[(bh * J + j) * (size_t)Dv + d] = r[j];

      /* M-step (Eq. 3.3; Eq. 3.7 when the decay comes after the responsibilities) */
      for (int j = 0; j < J; ++j) {
        double *w = W + ((bh * J + j) * (size_t)Dv + d) * Dk;
        const double beta = sigmoid_(beta_logit[g0 + (size_t)j * Dv]);
        const double coef = beta * r[j] * delta[j];
        for (int c = 0; c < Dk; ++c) {
          double wc = w[c];
          if (gated && post) {
            wc *= decay_(alpha, gran, tok, j, d, c, J, Dv, Dk);
          }
          w[c] = wc + coef * kt[c];
        }
      }

      /* readout on the updated state (Eq. 3.5) */
      softmax_(J, piq_logit + g0, (size_t)Dv, piq);
      if (temporal) {
        const double gq = sigmoid_(gq_logit[tok * Dv + d]);
        for (int j = 0; j < J; ++j) {
          rho[j] = (1.0 - gq) * rho_prev[(bh * J + j) * (size_t)Dv + d] + gq * piq[j];
          rho_prev[(bh * J + j) * (size_t)Dv + d] = rho[j];
        }
      } else {
        for (int j = 0; j < J; ++j) rho[j] = piq[j];
      }
      double out = 0.0;
      for (int j = 0; j < J; ++j) {
        const double *w = W + ((bh * J + j) * (size_t)Dv + d) * Dk;
        wq[j] = 0.0;
        for (int c = 0; c < Dk; ++c) wq[j] += w[c] * qt[c];
        out += rho[j] * wq[j];
      }
      o[tok * Dv + d] = out;
    }
  }
  return 0;
}
