"""fp64 numpy oracle of the steps either side of the recurrence: test infrastructure only.

Nothing here is used by the product path.  Three plain definitions, each a few numpy lines:

* ``qkv_activation``  -- how the paper's models make q, k, v from their projections (App. B.2 and the
  model description of App. D.1): SiLU on all three, then L2 normalisation of q and k over the key
  dimension.  The paper gives no epsilon for the normalisation; the reading taken is
  x / sqrt(sum x^2 + eps) with eps = 1e-6.
* ``readout_weights`` -- the weights the readout (Eq. 3.5) mixes the components with: the query-side
  prior pi^q = softmax over the components, or its running average rho-bar when Temporal (App. B.3).
* ``responsibility_stats`` -- the sums over time from which the mutual-information load-balancing loss
  (Sec. 3.5: entropy of the time-averaged responsibilities minus the mean per-token entropy) and the
  router diagnostics of App. D.5 are formed: per (batch, head, component, column) the sum over tokens of the
  responsibilities, per (batch, head, column) the sum over tokens of their entropy over the components (nats).
* ``output_rmsnorm``  -- RMSNorm on the layer output (App. D.1), over the value dimension of each
  (batch, head, token): y = x / sqrt(mean x^2 + eps) * weight.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

L2_EPS = 1e-6


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").double().numpy()
    return np.asarray(x, dtype=np.float64)


def silu(x) -> np.ndarray:
    """SiLU(x) = x * sigmoid(x) (App. B.2)."""
    x = _f64(x)
    return x / (1.0 + np.exp(-x))


def qkv_activation(q, k, v, eps: float = L2_EPS):
    """SiLU on q, k, v; then q and k divided by sqrt(sum of squares over the key dimension + eps)."""
    def l2n(x):
        return x / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + eps)
    return l2n(silu(q)), l2n(silu(k)), silu(v)


def _softmax_j(logit: np.ndarray) -> np.ndarray:
    z = logit - logit.max(axis=3, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=3, keepdims=True)


def readout_weights(piq_logit, gq_logit=None, rho0=None) -> np.ndarray:
    """[B,H,T,J,Dv] weights of Eq. 3.5: softmax over J of the query-side logits; when gq_logit is
    given (Temporal), rho_t = (1 - g) rho_{t-1} + g pi^q_t with g = sigmoid(gq_logit) per (t, d)
    and rho_0 = rho0 (uniform 1/J if None)."""
    pq = _softmax_j(_f64(piq_logit))
    if gq_logit is None:
        return pq
    B, H, T, J, Dv = pq.shape
    g = 1.0 / (1.0 + np.exp(-_f64(gq_logit)))  # [B,H,T,Dv]
    rho = np.full((B, H, J, Dv), 1.0 / J) if rho0 is None else _f64(rho0).copy()
    out = np.empty_like(pq)
    for t in range(T):
        gt = g[:, :, t, None, :]
        rho = (1.0 - gt) * rho + gt * pq[:, :, t]
        out[:, :, t] = rho
    return out


def _entropy_j(p: np.ndarray) -> np.ndarray:
    """-sum_j p ln p over axis 3 with 0 ln 0 = 0."""
    with np.errstate(divide="ignore", invalid="ignore"):
        term = np.where(p > 0.0, p * np.log(p), 0.0)
    return -term.sum(axis=3)


def responsibility_stats(r, rho) -> Dict[str, np.ndarray]:
    """r, rho: [B,H,T,J,Dv] key-side responsibilities (Eq. 3.4) and readout weights.
    Returns r_sum, rho_sum [B,H,J,Dv] (sums over t) and r_ent, rho_ent [B,H,Dv] (sums over t of
    the entropy over j, in nats)."""
    r, rho = _f64(r), _f64(rho)
    return {"r_sum": r.sum(axis=2), "r_ent": _entropy_j(r).sum(axis=2),
            "rho_sum": rho.sum(axis=2), "rho_ent": _entropy_j(rho).sum(axis=2)}


def mutual_information(p_sum: np.ndarray, ent_sum: np.ndarray, T: int) -> np.ndarray:
    """I(token; component) per (batch, head, column) from the sums above (Sec. 3.5):
    entropy of the time-averaged distribution minus the mean per-token entropy."""
    avg = _f64(p_sum) / T  # [B,H,J,Dv]
    with np.errstate(divide="ignore", invalid="ignore"):
        h_marg = -np.where(avg > 0.0, avg * np.log(avg), 0.0).sum(axis=2)
    return h_marg - _f64(ent_sum) / T


def output_rmsnorm(o, weight: Optional[np.ndarray] = None, eps: float = 1e-6) -> np.ndarray:
    """y = o / sqrt(mean over the last axis of o^2 + eps) * weight (weight [Dv], ones if None)."""
    o = _f64(o)
    y = o / np.sqrt(np.mean(o * o, axis=-1, keepdims=True) + eps)
    return y if weight is None else y * _f64(weight)
