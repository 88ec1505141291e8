"""Pins for the fp64 CPU oracle: everything here checks the oracle against something
other than itself -- closed forms, stated reductions, invariants, a hand-worked
example, and a separately written brute-force evaluation.  No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2609_39034_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_problem(seed, B=2, H=2, T=12, Dk=8, Dv=6, J=3, temporal=False, gran=0, logit_std=1.0, w_std=1.0):
    g = np.random.default_rng(seed)
    k = g.standard_normal((B, H, T, Dk))
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    q = g.standard_normal((B, H, T, Dk))
    q /= np.linalg.norm(q, axis=-1, keepdims=True)
    p = dict(q=q, k=k, v=g.standard_normal((B, H, T, Dv)),
             beta_logit=logit_std * g.standard_normal((B, H, T, J, Dv)),
             pik_logit=logit_std * g.standard_normal((B, H, T, J, Dv)),
             piq_logit=logit_std * g.standard_normal((B, H, T, J, Dv)),
             W0=w_std * g.standard_normal((B, H, J, Dv, Dk)))
    if temporal:
        p["gk_logit"] = g.standard_normal((B, H, T, Dv))
        p["gq_logit"] = g.standard_normal((B, H, T, Dv))
        r0 = g.random((B, H, J, Dv)); p["r0"] = r0 / r0.sum(2, keepdims=True)
        rho0 = g.random((B, H, J, Dv)); p["rho0"] = rho0 / rho0.sum(2, keepdims=True)
    if gran:
        shape = {1: (B, H, T, J, Dk), 2: (B, H, T, J, Dv), 3: (B, H, T, J), 4: (B, H, T, J, Dv, Dk)}[gran]
        p["alpha"] = 0.5 + 0.5 * g.random(shape)
    return p


def _run(oracle, p, flags=0, gran=0, want_r=False):
    return oracle.forward(p["q"], p["k"], p["v"], p["beta_logit"], p["pik_logit"], p["piq_logit"],
                          gk_logit=p.get("gk_logit"), gq_logit=p.get("gq_logit"), alpha=p.get("alpha"),
                          W0=p.get("W0"), r0=p.get("r0"), rho0=p.get("rho0"), flags=flags, gran=gran, want_r=want_r)


# ---- invariants: responsibilities are a posterior (Eq. 3.4) ------------------------------
@pytest.mark.parametrize("flags,gran", [(0, 0), (1, 0), (2, 1), (3, 1), (6, 2)])
def test_responsibilities_on_simplex(oracle, flags, gran):
    p = _rand_problem(1, temporal=bool(flags & 1), gran=gran, T=20)
    out = _run(oracle, p, flags, gran, want_r=True)
    r = out["r"]
    assert (r >= 0).all()
    np.testing.assert_allclose(r.sum(axis=3), 1.0, atol=1e-14)
    if flags & 1:  # carried distributions stay distributions (App. B.3: convex combinations)
        np.testing.assert_allclose(out["r_prev"].sum(axis=2), 1.0, atol=1e-14)
        np.testing.assert_allclose(out["rho_prev"].sum(axis=2), 1.0, atol=1e-13)
        np.testing.assert_allclose(out["r_prev"], r[:, :, -1], atol=0)


# ---- J = 1 is the delta rule (Eqs. 4.1-4.2), with a per-output-dimension learning rate ------
def test_single_component_is_deltanet(oracle):
    p = _rand_problem(2, J=1, T=16, Dk=8, Dv=5)
    out = _run(oracle, p)
    B, H, T, Dk = p["q"].shape
    Dv = p["v"].shape[-1]
    beta = 1.0 / (1.0 + np.exp(-p["beta_logit"][:, :, :, 0, :]))
    for b in range(B):
        for h in range(H):
            W = p["W0"][b, h, 0].copy()  # [Dv, Dk]
            for t in range(T):
                kt, qt, vt = p["k"][b, h, t], p["q"][b, h, t], p["v"][b, h, t]
                W = W + np.outer(beta[b, h, t] * (vt - W @ kt), kt)  # matrix form of Eq. 4.1
                np.testing.assert_allclose(out["o"][b, h, t], W @ qt, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(out["W"][b, h, 0], W, rtol=1e-12, atol=1e-13)


# ---- J = 1, beta = 1, orthonormal keys, zero state: plain linear attention -----------------
def test_orthonormal_keys_give_linear_attention(oracle):
    g = np.random.default_rng(3)
    Dk, Dv, T = 8, 4, 8
    Q, _ = np.linalg.qr(g.standard_normal((Dk, Dk)))
    k = Q[:T][None, None]  # orthonormal rows
    q = g.standard_normal((1, 1, T, Dk))
    v = g.standard_normal((1, 1, T, Dv))
    big = np.full((1, 1, T, 1, Dv), 60.0)  # sigmoid(60) == 1 to fp64 precision
    z = np.zeros((1, 1, T, 1, Dv))
    out = oracle.forward(q, k, v, big, z, z)
    expect = np.tril(q[0, 0] @ k[0, 0].T) @ v[0, 0]  # o_t = sum_{i<=t} (k_i . q_t) v_i
    np.testing.assert_allclose(out["o"][0, 0], expect, rtol=1e-12, atol=1e-13)


# ---- identical components stay identical: reduces to J = 1 with beta / J ----------------
def test_symmetric_components_reduce_to_one(oracle):
    g = np.random.default_rng(4)
    B, H, T, Dk, Dv, J = 1, 2, 24, 8, 4, 4
    p = _rand_problem(4, B=B, H=H, T=T, Dk=Dk, Dv=Dv, J=J)
    p["W0"] = np.zeros_like(p["W0"])
    p["pik_logit"][:] = 0.0
    p["piq_logit"][:] = 0.0
    beta = 0.1 + 0.8 * g.random((B, H, T, 1, Dv))
    p["beta_logit"] = np.broadcast_to(np.log(beta / (1 - beta)), (B, H, T, J, Dv)).copy()
    out = _run(oracle, p, want_r=True)
    np.testing.assert_allclose(out["r"], 1.0 / J, atol=1e-15)
    b1 = beta / J
    p1 = dict(p, beta_logit=np.log(b1 / (1 - b1)), pik_logit=np.zeros((B, H, T, 1, Dv)),
              piq_logit=np.zeros((B, H, T, 1, Dv)), W0=np.zeros((B, H, 1, Dv, Dk)))
    out1 = _run(oracle, p1)
    np.testing.assert_allclose(out["o"], out1["o"], rtol=1e-12, atol=1e-14)
    for j in range(J):
        np.testing.assert_allclose(out["W"][:, :, j], out1["W"][:, :, 0], rtol=1e-12, atol=1e-14)


# ---- first token from a zero state, in closed form ---------------------------------------
def test_first_token_closed_form(oracle):
    p = _rand_problem(5, T=1, J=3)
    p["W0"][:] = 0.0
    out = _run(oracle, p, want_r=True)
    sm = lambda x: np.exp(x) / np.exp(x).sum(axis=3, keepdims=True)
    pik, piq = sm(p["pik_logit"]), sm(p["piq_logit"])
    beta = 1 / (1 + np.exp(-p["beta_logit"]))
    np.testing.assert_allclose(out["r"], pik, rtol=1e-13)  # delta_j = v for all j: r = pi^k
    kq = (p["k"] * p["q"]).sum(-1)[..., None]  # [B,H,1,1]
    expect = p["v"] * kq * (piq * beta * pik).sum(axis=3)
    np.testing.assert_allclose(out["o"], expect, rtol=1e-12, atol=1e-15)
    # state: w_jd = beta_jd pi^k_jd v_d k
    expW = np.einsum("bhjd,bhc->bhjdc", (beta * pik)[:, :, 0] * p["v"][:, :, 0][:, :, None, :], p["k"][:, :, 0])
    np.testing.assert_allclose(out["W"], expW, rtol=1e-12, atol=1e-15)


# ---- hand-worked two-token example (fixture + its closed forms) --------------------------
def test_worked_example(oracle):
    rows = [list(map(float, ln.split())) for ln in open(os.path.join(GOLDEN, "worked_example_two_tokens.txt"))
            if ln.strip() and not ln.startswith("#")]
    # the fixture itself against the closed forms it states
    r1 = 1.0 / (1.0 + math.exp(0.5))
    assert abs(rows[0][3] - r1) < 1e-9 and abs(rows[0][7] - (r1 + 1) / 2) < 1e-9
    e = [math.exp(-0.5 * r1 * r1), math.exp(-0.5)]
    r2 = [e[0] / sum(e), e[1] / sum(e)]
    w2 = [r1 + 0.5 * r2[0] * (-r1), 1 + 0.5 * r2[1] * (-1.0)]
    assert abs(rows[1][3] - r2[0]) < 1e-9 and abs(rows[1][5] - w2[0]) < 1e-9 and abs(rows[1][6] - w2[1]) < 1e-9
    assert abs(rows[1][7] - 2 * (0.25 * w2[0] + 0.75 * w2[1])) < 1e-9
    # the oracle against the fixture
    k = np.array([1.0, 1.0]).reshape(1, 1, 2, 1)
    v = np.array([1.0, 0.0]).reshape(1, 1, 2, 1)
    q = np.array([1.0, 2.0]).reshape(1, 1, 2, 1)
    beta_logit = np.array([[60.0, 60.0], [0.0, 0.0]]).reshape(1, 1, 2, 2, 1)
    pik_logit = np.zeros((1, 1, 2, 2, 1))
    piq_logit = np.array([[0.0, 0.0], [0.0, math.log(3.0)]]).reshape(1, 1, 2, 2, 1)
    W0 = np.array([0.0, 1.0]).reshape(1, 1, 2, 1, 1)
    out = oracle.forward(q, k, v, beta_logit, pik_logit, piq_logit, W0=W0, want_r=True)
    for t in range(2):
        np.testing.assert_allclose(out["r"][0, 0, t, :, 0], rows[t][3:5], atol=2e-9)
        np.testing.assert_allclose(out["o"][0, 0, t, 0], rows[t][7], atol=2e-9)
    np.testing.assert_allclose(out["W"][0, 0, :, 0, 0], rows[1][5:7], atol=2e-9)
    # and token 1 alone
    out1 = oracle.forward(q[:, :, :1], k[:, :, :1], v[:, :, :1], beta_logit[:, :, :1], pik_logit[:, :, :1],
                          piq_logit[:, :, :1], W0=W0)
    np.testing.assert_allclose(out1["W"][0, 0, :, 0, 0], rows[0][5:7], atol=2e-9)


# ---- permuting the components changes nothing ---------------------------------------------
@pytest.mark.parametrize("flags,gran", [(0, 0), (3, 1)])
def test_component_permutation_invariance(oracle, flags, gran):
    p = _rand_problem(6, J=4, temporal=bool(flags & 1), gran=gran)
    perm = np.array([2, 0, 3, 1])
    pp = dict(p)
    for name in ("beta_logit", "pik_logit", "piq_logit"):
        pp[name] = p[name][:, :, :, perm]
    pp["W0"] = p["W0"][:, :, perm]
    if flags & 1:
        pp["r0"], pp["rho0"] = p["r0"][:, :, perm], p["rho0"][:, :, perm]
    if gran:
        pp["alpha"] = p["alpha"][:, :, :, perm]
    a, b = _run(oracle, p, flags, gran), _run(oracle, pp, flags, gran)
    np.testing.assert_allclose(a["o"], b["o"], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(a["W"][:, :, perm], b["W"], rtol=1e-11, atol=1e-13)


# ---- output dimensions are independent recurrences (Sec. 3.1) ---------------------------
def test_column_independence(oracle):
    p = _rand_problem(7, temporal=True, gran=2)
    a = _run(oracle, p, flags=3, gran=2)
    pp = {n: (x.copy() if x is not None else None) for n, x in p.items()}
    d0 = 2
    pp["v"][..., d0] += 1.0
    pp["beta_logit"][..., d0] -= 0.5
    pp["pik_logit"][..., 0, d0] += 1.0
    b = _run(oracle, pp, flags=3, gran=2)
    keep = [d for d in range(p["v"].shape[-1]) if d != d0]
    assert np.array_equal(a["o"][..., keep], b["o"][..., keep])
    assert np.array_equal(a["W"][:, :, :, keep], b["W"][:, :, :, keep])
    assert not np.allclose(a["o"][..., d0], b["o"][..., d0])
    # and a column subset is itself a valid problem with the same answers
    cols = torch.tensor([0, 3])
    sub = wl.slice_rows({n: (torch.from_numpy(x) if x is not None else None) for n, x in p.items()},
                        torch.arange(4), cols, gran=2)
    c = oracle.forward_inputs(sub, flags=3, gran=2)
    np.testing.assert_array_equal(c["o"].reshape(2, 2, -1, 2), a["o"][..., [0, 3]])


# ---- hard prior: one component takes every update, the others freeze --------------------
def test_hard_prior_limit(oracle):
    p = _rand_problem(8, J=3, T=10)
    p["pik_logit"][:] = 0.0
    p["pik_logit"][:, :, :, 1] = 800.0  # pi^k one-hot to fp64 precision; exp(-800) underflows harmlessly
    out = _run(oracle, p, want_r=True)
    np.testing.assert_allclose(out["r"][:, :, :, 1], 1.0, atol=0)
    np.testing.assert_array_equal(out["W"][:, :, 0], p["W0"][:, :, 0])
    np.testing.assert_array_equal(out["W"][:, :, 2], p["W0"][:, :, 2])
    # component 1 follows the delta rule on its own
    p1 = dict(p, beta_logit=p["beta_logit"][:, :, :, 1:2], pik_logit=np.zeros_like(p["pik_logit"][:, :, :, :1]),
              piq_logit=np.zeros_like(p["piq_logit"][:, :, :, :1]), W0=p["W0"][:, :, 1:2])
    np.testing.assert_allclose(out["W"][:, :, 1], _run(oracle, p1)["W"][:, :, 0], rtol=1e-13)


# ---- continuity: carrying the state across calls equals one long call --------------------
@pytest.mark.parametrize("flags,gran", [(0, 0), (1, 0), (2, 1), (7, 3)])
def test_split_sequence_continuity(oracle, flags, gran):
    p = _rand_problem(9, T=13, temporal=bool(flags & 1), gran=gran)
    full = _run(oracle, p, flags, gran)
    st = dict(W=p["W0"], r_prev=p.get("r0"), rho_prev=p.get("rho0"))
    outs = []
    for (a, b) in [(0, 5), (5, 6), (6, 13)]:
        part = {n: (x[:, :, a:b] if (x is not None and n not in ("W0", "r0", "rho0")) else x) for n, x in p.items()}
        part.update(W0=st["W"], r0=st.get("r_prev"), rho0=st.get("rho_prev"))
        st = _run(oracle, part, flags, gran)
        outs.append(st["o"])
    assert np.array_equal(np.concatenate(outs, axis=2), full["o"])
    assert np.array_equal(st["W"], full["W"])


# ---- brute force on tiny inputs -------------------------------------------------------------
@pytest.mark.parametrize("flags,gran", [(0, 0), (1, 0), (2, 1), (2, 2), (2, 3), (6, 1), (6, 2), (3, 1), (7, 3), (2, 4), (6, 4), (3, 4)])
def test_brute_force(oracle, flags, gran):
    from oracle import brute_force

    p = _rand_problem(10 + flags + 10 * gran, B=1, H=2, T=7, Dk=5, Dv=3, J=3, temporal=bool(flags & 1), gran=gran)
    out = _run(oracle, p, flags, gran, want_r=True)
    for h in range(2):
        g = lambda n: (p[n][0, h].tolist() if p.get(n) is not None else None)
        o, W, r, rp, rh = brute_force.swila_one_head(
            g("q"), g("k"), g("v"), g("beta_logit"), g("pik_logit"), g("piq_logit"), g("W0"),
            gk_logit=g("gk_logit"), gq_logit=g("gq_logit"), r0=g("r0"), rho0=g("rho0"),
            alpha=g("alpha"), gran=gran, post_decay=bool(flags & 4))
        np.testing.assert_allclose(out["o"][0, h], np.array(o), rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(out["W"][0, h], np.array(W), rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(out["r"][0, h], np.array(r), rtol=1e-12, atol=1e-14)
        if flags & 1:
            np.testing.assert_allclose(out["rho_prev"][0, h], np.array(rh), rtol=1e-12)


# ---- gated and temporal reductions ---------------------------------------------------------
def test_gating_reductions(oracle):
    # alpha == 1 is the ungated layer; g^k = g^q = 1 makes the temporal layer memoryless
    p = _rand_problem(11, temporal=True, gran=1)
    base = _run(oracle, p)
    p["alpha"][:] = 1.0
    for fl in (2, 6):
        np.testing.assert_array_equal(_run(oracle, p, fl, 1)["o"], base["o"])
    p["gk_logit"][:] = 60.0
    p["gq_logit"][:] = 60.0
    np.testing.assert_allclose(_run(oracle, p, 1)["o"], base["o"], rtol=1e-12, atol=1e-14)


def test_pre_post_decay_coincide_for_one_component(oracle):
    # App. B.4: with J = 1 the two gated forms agree under (alpha, beta, v) -> (alpha, beta/alpha, alpha v)
    g = np.random.default_rng(12)
    B, H, T, Dk, Dv = 1, 2, 9, 6, 4
    p = _rand_problem(12, B=B, H=H, T=T, Dk=Dk, Dv=Dv, J=1, gran=2)
    alpha = 0.6 + 0.4 * g.random((B, H, T, 1, Dv))
    beta_post = 0.05 + 0.5 * g.random((B, H, T, 1, Dv))
    p["alpha"] = alpha
    p["beta_logit"] = np.log(beta_post / (1 - beta_post))
    post = _run(oracle, p, flags=6, gran=2)
    beta_pre = beta_post / alpha
    assert (beta_pre < 1).all()
    pp = dict(p, beta_logit=np.log(beta_pre / (1 - beta_pre)), v=p["v"] * alpha[:, :, :, 0])
    pre = _run(oracle, pp, flags=2, gran=2)
    np.testing.assert_allclose(pre["W"], post["W"], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(pre["o"], post["o"], rtol=1e-11, atol=1e-13)


def test_decay_granularities_agree_when_tied(oracle):
    # per-key, per-output and scalar gates are restrictions of one elementwise gate (App. B.4)
    p = _rand_problem(13, gran=3, J=2)
    B, H, T, J = p["alpha"].shape
    Dk, Dv = p["q"].shape[-1], p["v"].shape[-1]
    for fl in (2, 6):
        s = _run(oracle, p, fl, 3)
        pk = dict(p, alpha=np.broadcast_to(p["alpha"][..., None], (B, H, T, J, Dk)).copy())
        po = dict(p, alpha=np.broadcast_to(p["alpha"][..., None], (B, H, T, J, Dv)).copy())
        pe = dict(p, alpha=np.broadcast_to(p["alpha"][..., None, None], (B, H, T, J, Dv, Dk)).copy())
        np.testing.assert_array_equal(_run(oracle, pk, fl, 1)["o"], s["o"])
        np.testing.assert_array_equal(_run(oracle, po, fl, 2)["o"], s["o"])
        np.testing.assert_array_equal(_run(oracle, pe, fl, 4)["o"], s["o"])


@pytest.mark.parametrize("gran", [1, 2])
def test_elementwise_gate_restricts_to_the_coarser_ones(oracle, gran):
    # Eq. (gate-elementwise) of App. B.4 with alpha_{tjdd'} constant along the output index d is W Diag(a_tj)
    # (one gate per key dimension); constant along the key index d' it is Diag(alpha_tj) W (one per output
    # dimension).  Dk != Dv here, so an elementwise gate indexed [d'][d] instead of [d][d'] cannot pass.
    p = _rand_problem(15, gran=gran, J=3, temporal=True)
    B, H, T, J = p["alpha"].shape[:4]
    Dk, Dv = p["q"].shape[-1], p["v"].shape[-1]
    assert Dk != Dv
    full = p["alpha"][..., None, :] if gran == 1 else p["alpha"][..., :, None]
    pe = dict(p, alpha=np.broadcast_to(full, (B, H, T, J, Dv, Dk)).copy())
    for fl in (2, 6, 3):
        a, b = _run(oracle, p, fl, gran), _run(oracle, pe, fl, 4)
        np.testing.assert_array_equal(a["o"], b["o"])
        np.testing.assert_array_equal(a["W"], b["W"])


# ---- own-block Jacobian of the update (Eqs. C.4-C.5) by finite differences ---------------
def test_update_jacobian(oracle):
    g = np.random.default_rng(14)
    Dk, J = 5, 3
    p = _rand_problem(14, B=1, H=1, T=1, Dk=Dk, Dv=1, J=J)
    out = _run(oracle, p, want_r=True)
    k = p["k"][0, 0, 0]
    beta = 1 / (1 + np.exp(-p["beta_logit"][0, 0, 0, :, 0]))
    r = out["r"][0, 0, 0, :, 0]
    delta = p["v"][0, 0, 0, 0] - p["W0"][0, 0, :, 0] @ k
    for j in range(J):
        gcoef = beta[j] * r[j] * (1 - delta[j] ** 2 * (1 - r[j]))
        expect = np.eye(Dk) - gcoef * np.outer(k, k)
        num = np.zeros((Dk, Dk))
        eps = 1e-6
        for c in range(Dk):
            for sgn in (+1, -1):
                pp = dict(p, W0=p["W0"].copy())
                pp["W0"][0, 0, j, 0, c] += sgn * eps
                num[:, c] += sgn * _run(oracle, pp)["W"][0, 0, j, 0] / (2 * eps)
        np.testing.assert_allclose(num, expect, atol=5e-9)


# ---- test power: a mutant without the -delta^2/2 term must be told apart -----------------
def test_stress_inputs_expose_a_broken_estep(oracle):
    w = wl.CONFIGS[0].with_(T=64)
    calm, hot = wl.make_inputs(w), wl.make_inputs(w, stress=True)

    def mutant(inp):
        # prior-only routing: what a kernel that dropped the Gaussian factor would compute.
        big = {n: (x.double().numpy() if x is not None else None) for n, x in inp.items()}
        B, H, T, J, Dv = big["pik_logit"].shape
        W = big["W0"].copy()
        o = np.zeros((B, H, T, Dv))
        sm = lambda x: np.exp(x - x.max(2, keepdims=True)) / np.exp(x - x.max(2, keepdims=True)).sum(2, keepdims=True)
        for t in range(T):
            kt, qt, vt = big["k"][:, :, t], big["q"][:, :, t], big["v"][:, :, t]
            delta = vt[:, :, None, :] - np.einsum("bhjdc,bhc->bhjd", W, kt)
            r = sm(big["pik_logit"][:, :, t])
            beta = 1 / (1 + np.exp(-big["beta_logit"][:, :, t]))
            W = W + np.einsum("bhjd,bhc->bhjdc", beta * r * delta, kt)
            o[:, :, t] = (sm(big["piq_logit"][:, :, t]) * np.einsum("bhjdc,bhc->bhjd", W, qt)).sum(2)
        return o

    e_hot = wl.rel_err(torch.from_numpy(mutant(hot)), torch.from_numpy(oracle.forward_inputs(hot)["o"]))
    e_calm = wl.rel_err(torch.from_numpy(mutant(calm)), torch.from_numpy(oracle.forward_inputs(calm)["o"]))
    assert e_hot > 0.2, e_hot      # far above the 2e-2 bf16 tolerance: the stress set has power
    assert e_calm < e_hot          # the plain benchmark inputs are much less sensitive
