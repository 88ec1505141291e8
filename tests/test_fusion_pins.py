"""Pins of the oracle's definitions either side of the recurrence (oracle/swila_fusions.py): q/k/v
activation (App. B.2, App. D.1), readout weights (Eq. 3.5, App. B.3), responsibility statistics
(Sec. 3.5, App. D.5) and the output RMSNorm (App. D.1).  Each is checked against something other than
itself: a library routine that computes the same textbook quantity, a closed form, or an invariant."""
import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

from oracle import swila_fusions as fus
from oracle import swila_oracle as oracle
from paper_2609_39034_b200 import workloads as wl


def _rng(seed):
    return np.random.default_rng(seed)


def test_silu_and_l2_norm_against_library_routines():
    g = _rng(1)
    q, k, v = g.normal(size=(2, 3, 5, 16)), 3.0 * g.normal(size=(2, 3, 5, 16)), g.normal(size=(2, 3, 5, 8))
    qa, ka, va = fus.qkv_activation(q, k, v)
    silu = lambda x: torch.nn.functional.silu(torch.from_numpy(x)).numpy()  # noqa: E731
    np.testing.assert_allclose(va, silu(v), rtol=1e-14, atol=0)
    # expit is the logistic function: SiLU(x) = x expit(x)
    np.testing.assert_allclose(va, v * scipy.special.expit(v), rtol=1e-14, atol=0)
    for got, raw in ((qa, q), (ka, k)):
        s = silu(raw)
        lib = torch.nn.functional.normalize(torch.from_numpy(s), p=2.0, dim=-1, eps=0.0).numpy()
        # eps = 1e-6 under the root changes a vector of squared norm n by the factor sqrt(n / (n + eps))
        n2 = (s * s).sum(-1, keepdims=True)
        np.testing.assert_allclose(got, lib * np.sqrt(n2 / (n2 + fus.L2_EPS)), rtol=1e-13, atol=0)
        np.testing.assert_allclose((got * got).sum(-1), (n2 / (n2 + fus.L2_EPS))[..., 0], rtol=1e-13)


def test_l2_norm_is_scale_invariant_and_safe_at_zero():
    g = _rng(2)
    x = g.normal(size=(1, 1, 4, 64))
    a, _, _ = fus.qkv_activation(x, x, x[..., :8])
    # SiLU is not homogeneous, so scale the activated vector instead: normalising s and 7 s agree
    s = fus.silu(x)
    l2 = lambda y: y / np.sqrt((y * y).sum(-1, keepdims=True) + fus.L2_EPS)  # noqa: E731
    np.testing.assert_allclose(l2(7.0 * s), a, rtol=1e-6)
    z, _, _ = fus.qkv_activation(np.zeros((1, 1, 1, 16)), np.zeros((1, 1, 1, 16)), np.zeros((1, 1, 1, 8)))
    assert np.all(z == 0.0)


def test_readout_weights_softmax_and_running_average():
    g = _rng(3)
    B, H, T, J, Dv = 1, 2, 9, 4, 8
    lq = 2.0 * g.normal(size=(B, H, T, J, Dv))
    pq = fus.readout_weights(lq)
    np.testing.assert_allclose(pq, scipy.special.softmax(lq, axis=3), rtol=1e-13)
    # Temporal: a gate of 1 (logit +40) forgets the past, a gate of 0 (logit -40) keeps the initial value
    np.testing.assert_allclose(fus.readout_weights(lq, np.full((B, H, T, Dv), 40.0)), pq, rtol=1e-12)
    rho0 = scipy.special.softmax(g.normal(size=(B, H, J, Dv)), axis=2)
    kept = fus.readout_weights(lq, np.full((B, H, T, Dv), -40.0), rho0)
    np.testing.assert_allclose(kept, np.broadcast_to(rho0[:, :, None], kept.shape), atol=1e-15)
    # a constant gate g gives the closed form rho_t = (1-g)^(t+1) rho_0 + g sum_s (1-g)^(t-s) pi_s
    gl = 0.3
    gv = 1.0 / (1.0 + np.exp(-gl))
    rho = fus.readout_weights(lq, np.full((B, H, T, Dv), gl), rho0)
    for t in (0, 4, 8):
        want = (1 - gv) ** (t + 1) * rho0 + sum(gv * (1 - gv) ** (t - s) * pq[:, :, s] for s in range(t + 1))
        np.testing.assert_allclose(rho[:, :, t], want, rtol=1e-12)
    np.testing.assert_allclose(rho.sum(axis=3), 1.0, rtol=1e-12)


def test_temporal_readout_weights_match_the_recurrence_oracle():
    """The C oracle carries rho-bar as state (App. B.3): after T tokens its rho_prev must be the last
    row of the numpy running average, two independent codings of the same recursion."""
    w = wl.CONFIGS[0].variant(temporal=True)
    inp = wl.make_inputs(w, stress=True)
    ref = oracle.forward_inputs(inp, flags=1)
    rho = fus.readout_weights(inp["piq_logit"], inp["gq_logit"], inp["rho0"])
    np.testing.assert_allclose(rho[:, :, -1], ref["rho_prev"], rtol=1e-12, atol=1e-15)


def test_statistics_against_scipy_entropy_and_invariants():
    g = _rng(4)
    B, H, T, J, Dv = 2, 2, 33, 4, 8
    r = scipy.special.softmax(3.0 * g.normal(size=(B, H, T, J, Dv)), axis=3)
    rho = scipy.special.softmax(g.normal(size=(B, H, T, J, Dv)), axis=3)
    r[0, 0, 5, 1, :] = 0.0  # exact zeros must count as 0 ln 0 = 0
    r[0, 0, 5] /= r[0, 0, 5].sum(axis=0, keepdims=True)
    st = fus.responsibility_stats(r, rho)
    np.testing.assert_allclose(st["r_ent"], scipy.stats.entropy(r, axis=3).sum(axis=2), rtol=1e-12)
    np.testing.assert_allclose(st["rho_ent"], scipy.stats.entropy(rho, axis=3).sum(axis=2), rtol=1e-12)
    # the components' sums add up to the number of tokens; entropies lie in [0, T ln J]
    np.testing.assert_allclose(st["r_sum"].sum(axis=2), T, rtol=1e-12)
    np.testing.assert_allclose(st["rho_sum"].sum(axis=2), T, rtol=1e-12)
    assert np.all(st["r_ent"] >= 0) and np.all(st["r_ent"] <= T * np.log(J) + 1e-9)
    # mutual information is non-negative (entropy is concave) ...
    mi = fus.mutual_information(st["r_sum"], st["r_ent"], T)
    assert np.all(mi > -1e-12)
    # ... zero when every token has the same distribution, ln J when tokens are one-hot and balanced
    same = np.broadcast_to(r[:, :, :1], r.shape)
    s2 = fus.responsibility_stats(same, same)
    np.testing.assert_allclose(fus.mutual_information(s2["r_sum"], s2["r_ent"], T), 0.0, atol=1e-12)
    hot = np.zeros((1, 1, 8, J, 8))
    for t in range(8):
        hot[0, 0, t, t % J, :] = 1.0
    s3 = fus.responsibility_stats(hot, hot)
    np.testing.assert_allclose(fus.mutual_information(s3["r_sum"], s3["r_ent"], 8), np.log(J), rtol=1e-12)


def test_statistics_of_the_recurrence_uniform_case():
    """Identical components (zero state, equal prior logits across j): every responsibility is 1/J
    (Eq. 3.4 with equal likelihoods), so r_sum = T/J and the entropy sum is T ln J exactly."""
    w = wl.CONFIGS[0]
    inp = wl.make_inputs(w)
    for name in ("beta_logit", "pik_logit", "piq_logit"):
        inp[name] = inp[name][:, :, :, :1].expand_as(inp[name]).contiguous()
    ref = oracle.forward_inputs(inp, want_r=True)
    st = fus.responsibility_stats(ref["r"], fus.readout_weights(inp["piq_logit"]))
    np.testing.assert_allclose(st["r_sum"], w.T / w.J, rtol=1e-12)
    np.testing.assert_allclose(st["r_ent"], w.T * np.log(w.J), rtol=1e-12)
    np.testing.assert_allclose(st["rho_ent"], w.T * np.log(w.J), rtol=1e-12)


def test_output_rmsnorm_against_torch():
    g = _rng(5)
    o = g.normal(size=(2, 3, 7, 32)) * np.exp(g.normal(size=(2, 3, 7, 1)))
    wgt = 1.0 + 0.1 * g.normal(size=32)
    got = fus.output_rmsnorm(o, wgt, eps=1e-6)
    lib = torch.nn.functional.rms_norm(torch.from_numpy(o), (32,), torch.from_numpy(wgt), eps=1e-6).numpy()
    np.testing.assert_allclose(got, lib, rtol=1e-13)
    plain = fus.output_rmsnorm(o)
    np.testing.assert_allclose((plain * plain).mean(-1), (o * o).mean(-1) / ((o * o).mean(-1) + 1e-6), rtol=1e-12)


@pytest.mark.parametrize("scale", [1e-3, 1.0, 1e3])
def test_output_rmsnorm_scale_invariance(scale):
    g = _rng(6)
    o = g.normal(size=(1, 1, 3, 16))
    np.testing.assert_allclose(fus.output_rmsnorm(scale * o, eps=0.0), fus.output_rmsnorm(o, eps=0.0), rtol=1e-12)
