"""Pins for the backward oracle (oracle/mdn_stepwise_bwd.c): its gradients are checked against central finite
differences of the FORWARD oracle (the definition of a gradient), against a closed form, and against linearity.
All CPU, fp64, seconds."""
import numpy as np
import pytest

import oracle


def problem(seed, B=1, T=11, H=2, dk=5, dv=4, with_eta=True, with_state=True, ragged=False):
    r = np.random.default_rng(seed)
    f = np.float32
    p = dict(q=r.standard_normal((B, T, H, dk)).astype(f), k=r.standard_normal((B, T, H, dk)).astype(f),
             v=r.standard_normal((B, T, H, dv)).astype(f), beta=r.uniform(0.05, 0.6, (B, T, H)).astype(f),
             log_alpha=np.log(r.uniform(0.5, 0.99, (B, T, H))).astype(f),
             log_mu=np.log(r.uniform(0.4, 0.95, (B, T, H))).astype(f),
             eta=r.uniform(0.3, 1.6, (B, T, H)).astype(f) if with_eta else None)
    p["k"] /= np.linalg.norm(p["k"], axis=-1, keepdims=True)
    N = B
    p["seq_start"], p["seq_len"] = None, None
    if ragged:                      # B = 1: three packed sequences, one of them a single token
        lens = np.array([T - 5, 1, 4]); assert B == 1
        p["seq_start"], p["seq_len"] = np.concatenate([[0], np.cumsum(lens)[:-1]]), lens
        N = 3
    p["S0"] = (0.3 * r.standard_normal((N, H, dk, dv))).astype(f) if with_state else None
    p["M0"] = (0.3 * r.standard_normal((N, H, dk, dv))).astype(f) if with_state else None
    p["w_o"] = r.standard_normal((B, T, H, dv)).astype(f)          # loss = <w_o, o> + <w_S, S_T> + <w_M, M_T>
    p["w_S"] = r.standard_normal((N, H, dk, dv)).astype(f)
    p["w_M"] = r.standard_normal((N, H, dk, dv)).astype(f)
    p["scale"] = 0.7
    return p


def loss(p, **override):
    a = dict(p); a.update(override)
    o, S, M = oracle.stepwise(a["q"], a["k"], a["v"], a["beta"], a["log_alpha"], a["log_mu"], a["eta"],
                              scale=a["scale"], S0=a["S0"], M0=a["M0"], seq_start=a["seq_start"], seq_len=a["seq_len"])
    return float((p["w_o"] * o).sum() + (p["w_S"] * S).sum() + (p["w_M"] * M).sum())


def grads(p):
    return oracle.stepwise_bwd(p["q"], p["k"], p["v"], p["beta"], p["log_alpha"], p["log_mu"], p["eta"], p["w_o"],
                               scale=p["scale"], S0=p["S0"], M0=p["M0"], dS_final=p["w_S"], dM_final=p["w_M"],
                               seq_start=p["seq_start"], seq_len=p["seq_len"])


def fd(p, name, idx, h):
    """Central difference of the loss w.r.t. one entry; the forward oracle takes float32 inputs, so the step is
    chosen exactly representable around the entry (x +- h evaluated in float32, difference divided by the real gap)."""
    x = p[name].astype(np.float32)
    xp, xm = x.copy(), x.copy()
    xp[idx] = np.float32(x[idx] + h); xm[idx] = np.float32(x[idx] - h)
    return (loss(p, **{name: xp}) - loss(p, **{name: xm})) / (float(xp[idx]) - float(xm[idx]))


PAIRS = [("q", "dq"), ("k", "dk"), ("v", "dv"), ("beta", "dbeta"), ("log_alpha", "dlog_alpha"), ("log_mu", "dlog_mu"),
         ("eta", "deta"), ("S0", "dS0"), ("M0", "dM0")]


@pytest.mark.parametrize("ragged", [False, True])
def test_gradients_equal_finite_differences(ragged):
    p = problem(1, ragged=ragged)
    g = grads(p)
    r = np.random.default_rng(7)
    for name, gname in PAIRS:
        x = p[name]
        for _ in range(6):
            idx = tuple(int(r.integers(0, s)) for s in x.shape)
            num = fd(p, name, idx, 2.0 ** -7)
            # the loss is a polynomial of low degree in any single q, v, beta, eta, S0, M0 entry and smooth in the
            # others; a 2^-7 step leaves a relative truncation error well below 1e-4
            assert abs(num - g[gname][idx]) <= 2e-4 * max(1.0, abs(num)), (name, idx, num, g[gname][idx])


def test_crossing_a_checkpoint_boundary_changes_nothing():
    """T = 150 spans three 64-token recomputation segments; spot-check entries in each and at the seams."""
    p = problem(2, T=150, H=1, dk=4, dv=3)
    g = grads(p)
    for name, gname in PAIRS[:7]:
        for t in (0, 63, 64, 65, 127, 128, 149):
            idx = (0, t, 0) + ((1,) if p[name].ndim == 4 else ())
            num = fd(p, name, idx, 2.0 ** -7)
            assert abs(num - g[gname][idx]) <= 2e-4 * max(1.0, abs(num)), (name, t, num, g[gname][idx])


def test_single_token_closed_form():
    """T = 1 from zero state: M_1 = -eta k v^T, S_1 = beta eta k v^T, o = scale beta eta (k.q) v."""
    p = problem(3, T=1, H=1, with_state=False)
    p["w_S"][:] = 0; p["w_M"][:] = 0
    g = grads(p)
    q, k, v, w = (p[n][0, 0, 0].astype(np.float64) for n in ("q", "k", "v", "w_o"))
    be, et, sc = float(p["beta"][0, 0, 0]), float(p["eta"][0, 0, 0]), p["scale"]
    kq, wv = k @ q, w @ v
    assert np.allclose(g["dq"][0, 0, 0], sc * be * et * wv * k)
    assert np.allclose(g["dk"][0, 0, 0], sc * be * et * wv * q)
    assert np.allclose(g["dv"][0, 0, 0], sc * be * et * kq * w)
    assert np.isclose(g["dbeta"][0, 0, 0], sc * et * kq * wv) and np.isclose(g["deta"][0, 0, 0], sc * be * kq * wv)
    assert np.isclose(g["dlog_alpha"][0, 0, 0], 0.0) and np.isclose(g["dlog_mu"][0, 0, 0], 0.0)   # zero start state


def test_gradients_are_linear_in_the_upstream_gradient_and_eta_none():
    p = problem(4, with_eta=False)
    g1 = grads(p)
    assert g1["deta"] is None
    p2 = dict(p, w_o=2 * p["w_o"], w_S=2 * p["w_S"], w_M=2 * p["w_M"])
    g2 = grads(p2)
    for name in ("dq", "dk", "dv", "dbeta", "dlog_alpha", "dlog_mu", "dS0", "dM0"):
        assert np.allclose(g2[name], 2 * g1[name], rtol=1e-12, atol=1e-14)
    # eta = None is eta = 1
    g3 = grads(dict(p, eta=np.ones_like(p["beta"])))
    for name in ("dq", "dk", "dv", "dbeta", "dlog_alpha", "dlog_mu", "dS0", "dM0"):
        assert np.array_equal(g3[name], g1[name])


def test_chain_subset_matches_full():
    p = problem(5, B=2, H=3)
    full = grads(p)
    sub = oracle.stepwise_bwd(p["q"], p["k"], p["v"], p["beta"], p["log_alpha"], p["log_mu"], p["eta"], p["w_o"],
                              scale=p["scale"], S0=p["S0"], M0=p["M0"], dS_final=p["w_S"], dM_final=p["w_M"],
                              chains=[1, 5])
    for name in ("dq", "dk", "dv", "dbeta"):
        assert np.array_equal(sub[name][0, :, 1], full[name][0, :, 1])
        assert np.array_equal(sub[name][1, :, 2], full[name][1, :, 2])
        assert np.isnan(sub[name][0, :, 0]).all()


@pytest.mark.parametrize("T,chunk", [(64, 64), (150, 64), (37, 16)])
def test_chunk_form_backward_equals_stepwise_backward(T, chunk):
    """oracle/chunkwise_bwd.py differentiates the chunkwise algorithm matrix by matrix (adjoint state recurrence,
    dA = -tril(dR V~^T, -1) through the inverse, coefficient adjoints, scans in reverse); it must give the gradients of
    the token-by-token backward, which finite differences pin above.  Several chunks, a ragged last chunk."""
    from oracle import chunkwise_bwd as cb
    p = problem(11, T=T, H=2, dk=6, dv=5)
    ref = grads(p)
    for h in range(2):
        g = cb.chain_backward(p["q"][0, :, h], p["k"][0, :, h], p["v"][0, :, h], p["beta"][0, :, h],
                              p["log_alpha"][0, :, h], p["log_mu"][0, :, h], p["eta"][0, :, h], p["w_o"][0, :, h],
                              scale=p["scale"], S0=p["S0"][0, h], M0=p["M0"][0, h], dS_final=p["w_S"][0, h],
                              dM_final=p["w_M"][0, h], chunk=chunk)
        for name in ("dq", "dk", "dv", "dbeta", "dlog_alpha", "dlog_mu", "deta"):
            r = ref[name][0, :, h]
            assert np.allclose(g[name], r, rtol=1e-9, atol=1e-11 * max(1.0, np.abs(r).max())), (name, h)
        assert np.allclose(g["dS0"], ref["dS0"][0, h], rtol=1e-9, atol=1e-12)
        assert np.allclose(g["dM0"], ref["dM0"][0, h], rtol=1e-9, atol=1e-12)
