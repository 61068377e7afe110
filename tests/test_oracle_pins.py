"""Pins for the CPU oracle: it is checked against what the paper and the mathematics
fix, never against itself or the CUDA path.  All CPU, fp64, seconds."""
import os

import numpy as np
import pytest

import oracle
from oracle import chunkwise as cw

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_problem(seed, T, dk, dv, B=1, H=1, mu_zero=False, beta_zero=False, unit_k=True,
                 eta_one=False, stable=False):
    r = np.random.default_rng(seed)
    q = r.standard_normal((B, T, H, dk))
    k = r.standard_normal((B, T, H, dk))
    if unit_k:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = r.standard_normal((B, T, H, dv))
    alpha = r.uniform(0.3, 0.99, (B, T, H))
    mu = r.uniform(0.4, 0.99, (B, T, H))
    beta = r.uniform(0.05, 0.9, (B, T, H))
    if stable:
        beta = np.minimum(beta, 1 - alpha)
    eta = np.ones((B, T, H)) if eta_one else r.uniform(0.2, 1.8, (B, T, H))
    f = np.float32
    la = np.log(alpha).astype(f)
    lm = np.full((B, T, H), -np.inf, dtype=f) if mu_zero else np.log(mu).astype(f)
    be = np.zeros((B, T, H), dtype=f) if beta_zero else beta.astype(f)
    S0 = r.standard_normal((B, H, dk, dv)).astype(f)
    M0 = r.standard_normal((B, H, dk, dv)).astype(f)
    return dict(q=q.astype(f), k=k.astype(f), v=v.astype(f), beta=be, log_alpha=la, log_mu=lm,
                eta=eta.astype(f), S0=S0, M0=M0)


def run(p, scale=1.0, **kw):
    return oracle.stepwise(p["q"], p["k"], p["v"], p["beta"], p["log_alpha"], p["log_mu"], p["eta"],
                           scale=scale, S0=p.get("S0"), M0=p.get("M0"), **kw)


def d64(x):
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------- hand example
def test_hand_computed_scalar_example():
    rows = np.loadtxt(os.path.join(GOLDEN, "scalar_two_steps.txt"))
    al, mu, be, et, k, v, q, o_exp, S_exp, M_exp = rows.T
    sh = (1, 2, 1)
    o, S, M = oracle.stepwise(q.reshape(sh + (1,)), k.reshape(sh + (1,)), v.reshape(sh + (1,)),
                              be.reshape(sh), np.log(al).reshape(sh), np.log(mu).reshape(sh),
                              et.reshape(sh), scale=1.0, S0=np.ones((1, 1, 1, 1)), M0=np.ones((1, 1, 1, 1)))
    assert np.allclose(o.ravel(), o_exp, atol=1e-6)
    assert abs(S.item() - S_exp[-1]) < 1e-6 and abs(M.item() - M_exp[-1]) < 1e-6
    # first step alone
    o1, S1, M1 = oracle.stepwise(q[:1].reshape(1, 1, 1, 1), k[:1].reshape(1, 1, 1, 1), v[:1].reshape(1, 1, 1, 1),
                                 be[:1].reshape(1, 1, 1), np.log(al[:1]).reshape(1, 1, 1),
                                 np.log(mu[:1]).reshape(1, 1, 1), et[:1].reshape(1, 1, 1),
                                 S0=np.ones((1, 1, 1, 1)), M0=np.ones((1, 1, 1, 1)))
    assert abs(S1.item() - S_exp[0]) < 1e-6 and abs(M1.item() - M_exp[0]) < 1e-6


# --------------------------------------------------------------------------- special cases
def test_mu_zero_is_gated_delta_rule():
    """mu=0, eta=1, M0=0: S_t = alpha_t (I - beta_t k k^T) S_{t-1} + beta_t k v^T (Section 2.3)."""
    p = rand_problem(1, T=40, dk=6, dv=5, mu_zero=True, eta_one=True)
    p["M0"] = None
    o, S, M = run(p, scale=0.7)
    Sg = d64(p["S0"][0, 0])
    for t in range(40):
        a = np.exp(d64(p["log_alpha"][0, t, 0])); b = d64(p["beta"][0, t, 0])
        k = d64(p["k"][0, t, 0]); v = d64(p["v"][0, t, 0]); q = d64(p["q"][0, t, 0])
        Sg = a * (np.eye(6) - b * np.outer(k, k)) @ Sg + b * np.outer(k, v)
        assert np.allclose(o[0, t, 0], 0.7 * Sg.T @ q, atol=1e-12)
    assert np.allclose(S[0, 0], Sg, atol=1e-12)


def test_alpha_one_is_deltanet():
    """additionally alpha=1 (so p=k): S_t = (I - beta k k^T) S_{t-1} + beta k v^T (Table 1)."""
    p = rand_problem(2, T=30, dk=5, dv=4, mu_zero=True, eta_one=True)
    p["log_alpha"][:] = 0.0
    p["M0"] = None
    o, S, _ = run(p)
    Sd = d64(p["S0"][0, 0])
    for t in range(30):
        b = d64(p["beta"][0, t, 0]); k = d64(p["k"][0, t, 0]); v = d64(p["v"][0, t, 0])
        Sd = (np.eye(5) - b * np.outer(k, k)) @ Sd + b * np.outer(k, v)
    assert np.allclose(S[0, 0], Sd, atol=1e-12)


def test_beta_zero_leaves_purely_decayed_state():
    p = rand_problem(3, T=50, dk=4, dv=3, beta_zero=True)
    o, S, M = run(p, scale=1.0)
    abar = np.exp(np.cumsum(d64(p["log_alpha"][0, :, 0])))
    S0 = d64(p["S0"][0, 0])
    assert np.allclose(S[0, 0], abar[-1] * S0, rtol=0, atol=1e-14)
    for t in range(50):
        assert np.allclose(o[0, t, 0], abar[t] * S0.T @ d64(p["q"][0, t, 0]), atol=1e-14)
    assert not np.allclose(M[0, 0], d64(p["M0"][0, 0]))          # M still evolves


def test_zero_keys_give_closed_form_decay_of_S0_and_M0():
    """k=0: M_t = mubar_t M0, S_t = abar_t S0 - b_t M0 with b_t = abar_t sum_i beta_i mubar_i/abar_i (Eq. 10)."""
    p = rand_problem(4, T=33, dk=3, dv=2)
    p["k"][:] = 0
    _, S, M = run(p)
    al = np.exp(d64(p["log_alpha"][0, :, 0])); mu = np.exp(d64(p["log_mu"][0, :, 0]))
    be = d64(p["beta"][0, :, 0])
    abar, mubar = np.cumprod(al), np.cumprod(mu)
    b_T = abar[-1] * np.sum(be * mubar / abar)
    assert np.allclose(M[0, 0], mubar[-1] * d64(p["M0"][0, 0]), atol=1e-13)
    assert np.allclose(S[0, 0], abar[-1] * d64(p["S0"][0, 0]) - b_T * d64(p["M0"][0, 0]), atol=1e-13)


# --------------------------------------------------------------------------- brute force
def brute_force_closed_form(p, scale):
    """Unrolled closed forms of Appendix C for one head, written with explicit sums:
    M_t = mubar_t M0 - sum_i (mubar_t/mubar_i) eta_i k_i v~_i^T,
    S_t = abar_t S0 - b_t M0 + sum_i gamma_{t,i} eta_i k_i v~_i^T,
    gamma_{t,i} = abar_t/mubar_i (c_t - c_{i-1}), c_t = sum_{i<=t} beta_i mubar_i/abar_i,
    v~_t = v_t - alpha_t k_t^T S_{t-1}."""
    q, k, v = d64(p["q"][0, :, 0]), d64(p["k"][0, :, 0]), d64(p["v"][0, :, 0])
    al = np.exp(d64(p["log_alpha"][0, :, 0])); mu = np.exp(d64(p["log_mu"][0, :, 0]))
    be = d64(p["beta"][0, :, 0]); et = d64(p["eta"][0, :, 0])
    S0, M0 = d64(p["S0"][0, 0]), d64(p["M0"][0, 0])
    T = len(al)
    abar = [np.prod(al[:t + 1]) for t in range(T)]
    mubar = [np.prod(mu[:t + 1]) for t in range(T)]
    c = [sum(be[i] * mubar[i] / abar[i] for i in range(t + 1)) for t in range(T)]

    def gamma(t, i):
        return abar[t] / mubar[i] * (c[t] - (c[i - 1] if i > 0 else 0.0))

    def S_at(t, vt):      # state after token t (t = -1: initial)
        if t < 0:
            return S0
        return abar[t] * S0 - abar[t] * c[t] * M0 + sum(gamma(t, i) * et[i] * np.outer(k[i], vt[i]) for i in range(t + 1))

    vt, o = [], []
    for t in range(T):
        vt.append(v[t] - al[t] * (S_at(t - 1, vt).T @ k[t]))
        o.append(scale * S_at(t, vt).T @ q[t])
    S_T = S_at(T - 1, vt)
    M_T = mubar[-1] * M0 - sum(mubar[-1] / mubar[i] * et[i] * np.outer(k[i], vt[i]) for i in range(T))
    return np.array(o), S_T, M_T


@pytest.mark.parametrize("T", [1, 2, 7, 16])
def test_brute_force_unrolled_closed_form(T):
    p = rand_problem(10 + T, T=T, dk=4, dv=3)
    o, S, M = run(p, scale=0.5)
    o_b, S_b, M_b = brute_force_closed_form(p, 0.5)
    assert np.allclose(o[0, :, 0], o_b, atol=1e-10)
    assert np.allclose(S[0, 0], S_b, atol=1e-10)
    assert np.allclose(M[0, 0], M_b, atol=1e-10)


def test_second_order_two_step_form():
    """Table 1 footnote: S_t = (a~ I - alpha_t beta_t eta_t k k^T) S_{t-1} - g~ S_{t-2} + beta_t eta_t k v^T
    with a~ = alpha_t + mu_t beta_t/beta_{t-1}, g~ = alpha_{t-1} mu_t beta_t/beta_{t-1}
    (the k k^T coefficient carries alpha_t, as in the block form of Appendix F)."""
    T = 9
    p = rand_problem(21, T=T, dk=4, dv=3)
    states = [d64(p["S0"][0, 0])]
    for t in range(1, T + 1):
        sub = {n: (x[:, :t] if n not in ("S0", "M0") else x) for n, x in p.items()}
        states.append(run(sub)[1][0, 0])
    al = np.exp(d64(p["log_alpha"][0, :, 0])); mu = np.exp(d64(p["log_mu"][0, :, 0]))
    be = d64(p["beta"][0, :, 0]); et = d64(p["eta"][0, :, 0])
    for t in range(1, T):          # token index t (0-based) needs beta_{t-1}
        k = d64(p["k"][0, t, 0]); v = d64(p["v"][0, t, 0])
        a_t = al[t] + mu[t] * be[t] / be[t - 1]
        g_t = al[t - 1] * mu[t] * be[t] / be[t - 1]
        rhs = (a_t * np.eye(4) - al[t] * be[t] * et[t] * np.outer(k, k)) @ states[t] - g_t * states[t - 1] \
            + be[t] * et[t] * np.outer(k, v)
        assert np.allclose(states[t + 1], rhs, atol=1e-11)


# --------------------------------------------------------------------------- reordering identity
def test_summation_reordering_identity():
    r = np.random.default_rng(5)
    a, b = r.standard_normal(13), r.standard_normal(13)
    lhs = sum(a[i] * b[j] for i in range(13) for j in range(i + 1))
    mid = sum(a[i] * b[j] for j in range(13) for i in range(j, 13))
    rhs = sum(a[j] * b[i] for i in range(13) for j in range(i, 13))
    assert abs(lhs - mid) < 1e-12 and abs(lhs - rhs) < 1e-12


def test_coefficients_reordered_equal_nested_sums():
    """Eq. 10 (after reordering) == the nested sums before it; also the log-domain route."""
    r = np.random.default_rng(6)
    for C in (4, 16, 64):
        la = np.log(r.uniform(0.5, 0.999, C)); lm = np.log(r.uniform(0.4, 0.999, C))
        be = r.uniform(0.01, 0.9, C)
        abar, mubar, c, b, G = cw.coefficients(la, lm, be)
        abar2, mubar2, b2, G2, Mm = cw.coefficients_by_products(la, lm, be)
        assert np.allclose(abar, abar2, rtol=1e-12) and np.allclose(mubar, mubar2, rtol=1e-12)
        assert np.allclose(b, b2, rtol=1e-10, atol=1e-14)
        assert np.allclose(G, G2, rtol=1e-9, atol=1e-13)
        assert np.allclose(np.diag(G), be, rtol=1e-12)                # gamma_{i,i} = beta_i
        assert np.allclose(np.tril(mubar[:, None] / mubar[None, :]), Mm, rtol=1e-10)
        _, _, c3, b3, G3 = cw.coefficients_log_domain(la, lm, be, eps=0.0)
        assert np.allclose(b, b3, rtol=1e-10) and np.allclose(G, G3, rtol=1e-8, atol=1e-12)


# --------------------------------------------------------------------------- chunkwise == stepwise
@pytest.mark.parametrize("C,T", [(4, 37), (8, 37), (16, 50), (64, 150), (64, 64), (64, 1)])
@pytest.mark.parametrize("log_domain", [False, True])
def test_chunkwise_equals_stepwise(C, T, log_domain):
    p = rand_problem(30 + C + T, T=T, dk=6, dv=5, stable=True)
    o, S, M = run(p, scale=0.4)
    oc, Sc, Mc = cw.chunk_forward(p["q"][0, :, 0], p["k"][0, :, 0], p["v"][0, :, 0], p["beta"][0, :, 0],
                                  p["log_alpha"][0, :, 0], p["log_mu"][0, :, 0], p["eta"][0, :, 0],
                                  scale=0.4, S0=p["S0"][0, 0], M0=p["M0"][0, 0], chunk=C,
                                  log_domain=log_domain)
    tol = 1e-9
    assert np.allclose(o[0, :, 0], oc, atol=tol)
    assert np.allclose(S[0, 0], Sc, atol=tol) and np.allclose(M[0, 0], Mc, atol=tol)


def test_printed_epsilon_makes_chunk_form_inexact():
    """With the printed 1e-6 added to beta the chunk form drifts at the 1e-6 level: the
    reason the oracle (and the CUDA path) use beta as given."""
    p = rand_problem(77, T=64, dk=6, dv=5, stable=True)
    o, _, _ = run(p)
    oc, _, _ = cw.chunk_forward(p["q"][0, :, 0], p["k"][0, :, 0], p["v"][0, :, 0], p["beta"][0, :, 0],
                                p["log_alpha"][0, :, 0], p["log_mu"][0, :, 0], p["eta"][0, :, 0],
                                S0=p["S0"][0, 0], M0=p["M0"][0, 0], chunk=16, log_domain=True, eps=1e-6)
    err = np.abs(o[0, :, 0] - oc).max()
    assert 1e-9 < err < 1e-3


# --------------------------------------------------------------------------- spectrum / one step vs block matrix
def block_matrix(alpha, mu, beta, eta, k):
    d = len(k)
    kk = np.outer(k, k)
    I = np.eye(d)
    return np.block([[alpha * I - alpha * beta * eta * kk, -beta * mu * I],
                     [alpha * eta * kk, mu * I]])


def test_one_step_equals_block_transition_matrix():
    """One oracle step is [S;M] <- A [S;M] + [beta eta k v^T; -eta k v^T] (Appendix F)."""
    p = rand_problem(40, T=1, dk=5, dv=3)
    _, S, M = run(p)
    al = np.exp(d64(p["log_alpha"][0, 0, 0])); mu = np.exp(d64(p["log_mu"][0, 0, 0]))
    be = d64(p["beta"][0, 0, 0]); et = d64(p["eta"][0, 0, 0])
    k = d64(p["k"][0, 0, 0]); v = d64(p["v"][0, 0, 0])
    A = block_matrix(al, mu, be, et, k)
    x = A @ np.vstack([d64(p["S0"][0, 0]), d64(p["M0"][0, 0])]) + np.vstack([be * et * np.outer(k, v), -et * np.outer(k, v)])
    assert np.allclose(S[0, 0], x[:5], atol=1e-13) and np.allclose(M[0, 0], x[5:], atol=1e-13)


def test_spectrum_closed_form_and_stable_region():
    import mdn_workloads as wl
    beta, la, lm, eta = wl.draw_gates((500,), seed=3, preset="F", dk=1)   # tau = 1: widest eta spread
    r = np.random.default_rng(8)
    worst_abs, min_re = 0.0, 1.0
    for i in range(500):
        al, mu, be, et = np.exp(float(la[i])), np.exp(float(lm[i])), float(beta[i]), float(eta[i])
        assert be <= 1 - al + 1e-7 and np.exp(-1) - 1e-7 <= mu < 1
        k = r.standard_normal(4); k /= np.linalg.norm(k)
        ev = np.linalg.eigvals(block_matrix(al, mu, be, et, k))
        tr = al + mu - al * be * et
        disc = np.sqrt(complex(tr * tr - 4 * al * mu))
        expected = np.array([al] * 3 + [mu] * 3 + [(tr + disc) / 2, (tr - disc) / 2], dtype=complex)
        for lam in expected:                       # every closed-form root is an eigenvalue
            assert np.abs(ev - lam).min() < 1e-6
        worst_abs = max(worst_abs, np.abs(ev).max()); min_re = min(min_re, ev.real.min())
    assert worst_abs < 1.0 and min_re > 0.0


# --------------------------------------------------------------------------- hand-off, packing, chains
def test_state_handoff_two_calls_equal_one():
    p = rand_problem(50, T=41, dk=5, dv=4, B=2, H=3)
    o, S, M = run(p, scale=0.3)
    a = {n: (x[:, :17] if n not in ("S0", "M0") else x) for n, x in p.items()}
    o1, S1, M1 = run(a, scale=0.3)
    b = {n: (x[:, 17:] if n not in ("S0", "M0") else x) for n, x in p.items()}
    b["S0"], b["M0"] = S1, M1                      # float64 -> float32 cast inside: compare loosely
    o2, S2, M2 = run(b, scale=0.3)
    assert np.allclose(o[:, :17], o1, atol=1e-12)
    assert np.allclose(o[:, 17:], o2, atol=1e-5) and np.allclose(S, S2, atol=1e-5) and np.allclose(M, M2, atol=1e-5)


def test_packed_sequences_equal_separate_calls_and_chain_subset():
    p = rand_problem(60, T=60, dk=4, dv=3, B=1, H=2)
    lens = np.array([13, 1, 46]); starts = np.array([0, 13, 14])
    S0 = np.random.default_rng(1).standard_normal((3, 2, 4, 3)).astype(np.float32)
    M0 = np.random.default_rng(2).standard_normal((3, 2, 4, 3)).astype(np.float32)
    o, S, M = oracle.stepwise(p["q"], p["k"], p["v"], p["beta"], p["log_alpha"], p["log_mu"], p["eta"],
                              S0=S0, M0=M0, seq_start=starts, seq_len=lens)
    for n in range(3):
        sl = slice(starts[n], starts[n] + lens[n])
        on, Sn, Mn = oracle.stepwise(p["q"][:, sl], p["k"][:, sl], p["v"][:, sl], p["beta"][:, sl],
                                     p["log_alpha"][:, sl], p["log_mu"][:, sl], p["eta"][:, sl],
                                     S0=S0[n:n + 1], M0=M0[n:n + 1])
        assert np.array_equal(o[:, sl], on) and np.array_equal(S[n], Sn[0]) and np.array_equal(M[n], Mn[0])
    osub, Ssub, _ = oracle.stepwise(p["q"], p["k"], p["v"], p["beta"], p["log_alpha"], p["log_mu"], p["eta"],
                                    S0=S0, M0=M0, seq_start=starts, seq_len=lens, chains=[5])
    assert np.array_equal(osub[0, 14:, 1], o[0, 14:, 1]) and np.isnan(osub[0, :14]).all()
    assert np.array_equal(Ssub[2, 1], S[2, 1]) and np.isnan(Ssub[0]).all()
