"""Literal, loop-by-loop evaluation of the SwiLA equations for tiny inputs -- a second,
separately written implementation used only to pin the C oracle (test infrastructure).

Differences from the C oracle on purpose: pure Python floats and lists, explicit
mixture densities pi_j * exp(-delta_j^2 / 2) divided by their sum exactly as Eq. 3.4
prints it (no log-sum-exp), state held as nested lists per (j, d) row, the history
kept token by token.  Use only for T <= 8 or so."""
from __future__ import annotations

import math
from typing import List, Optional


def _softmax(xs: List[float]) -> List[float]:
    es = [math.exp(x) for x in xs]
    z = sum(es)
    return [e / z for e in es]


def swila_one_head(q, k, v, beta_logit, pik_logit, piq_logit, W0, *, gk_logit=None, gq_logit=None,
                   r0=None, rho0=None, alpha=None, gran: int = 0, post_decay: bool = False):
    """One (batch, head).  q,k: T x Dk; v: T x Dv; logits: T x J x Dv; W0: J x Dv x Dk;
    gk/gq logits: T x Dv; r0, rho0: J x Dv; alpha: by granularity (1: T x J x Dk,
    2: T x J x Dv, 3: T x J, 4: T x J x Dv x Dk).  Returns (o [T][Dv], W [J][Dv][Dk], r [T][J][Dv], r_prev, rho_prev)."""
    T, Dk, Dv, J = len(q), len(q[0]) if len(q) else 0, len(v[0]) if len(v) else 0, len(W0)
    W = [[[float(x) for x in row] for row in comp] for comp in W0]
    temporal = gk_logit is not None
    r_prev = [[float(x) for x in row] for row in r0] if temporal else None
    rho_prev = [[float(x) for x in row] for row in rho0] if temporal else None
    o_all, r_all = [], []

    def decay(t, j, d, c):
        if alpha is None:
            return 1.0
        if gran == 1:
            return float(alpha[t][j][c])
        if gran == 2:
            return float(alpha[t][j][d])
        if gran == 4:  # one value per state element (App. B.4, the general form)
            return float(alpha[t][j][d][c])
        return float(alpha[t][j])

    for t in range(T):
        o_t = [0.0] * Dv
        r_t = [[0.0] * Dv for _ in range(J)]
        for d in range(Dv):
            if alpha is not None and not post_decay:  # Eq. 3.8: decay first
                for j in range(J):
                    for c in range(Dk):
                        W[j][d][c] *= decay(t, j, d, c)
            pik = _softmax([float(pik_logit[t][j][d]) for j in range(J)])
            if temporal:
                gk = 1.0 / (1.0 + math.exp(-float(gk_logit[t][d])))
                prior = [(1.0 - gk) * r_prev[j][d] + gk * pik[j] for j in range(J)]
            else:
                prior = pik
            delta = [float(v[t][d]) - sum(W[j][d][c] * float(k[t][c]) for c in range(Dk)) for j in range(J)]
            dens = [prior[j] * math.exp(-0.5 * delta[j] ** 2) for j in range(J)]
            Z = sum(dens)
            r = [dens[j] / Z for j in range(J)]
            for j in range(J):
                r_t[j][d] = r[j]
                beta = 1.0 / (1.0 + math.exp(-float(beta_logit[t][j][d])))
                for c in range(Dk):
                    a = decay(t, j, d, c) if (alpha is not None and post_decay) else 1.0
                    W[j][d][c] = a * W[j][d][c] + beta * r[j] * delta[j] * float(k[t][c])
            piq = _softmax([float(piq_logit[t][j][d]) for j in range(J)])
            if temporal:
                gq = 1.0 / (1.0 + math.exp(-float(gq_logit[t][d])))
                rho = [(1.0 - gq) * rho_prev[j][d] + gq * piq[j] for j in range(J)]
                for j in range(J):
                    r_prev[j][d] = r[j]
                    rho_prev[j][d] = rho[j]
            else:
                rho = piq
            o_t[d] = sum(rho[j] * sum(W[j][d][c] * float(q[t][c]) for c in range(Dk)) for j in range(J))
        o_all.append(o_t)
        r_all.append(r_t)
    return o_all, W, r_all, r_prev, rho_prev
