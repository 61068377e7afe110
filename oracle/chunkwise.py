"""TEST INFRASTRUCTURE, NOT THE PRODUCT: fp64 numpy walk through the paper's
chunkwise algorithm (Section 3.1 "Coefficient Chunkwise" and "Chunkwise Algorithm",
Appendix C and D), one (sequence, head) at a time, in the paper's order and notation.

It exists to (a) pin the stepwise oracle through the paper's central claim that the
chunkwise form equals the recurrence exactly, and (b) give per-stage expected values
(coefficients, Gamma, T, V~) for the tests of the individual CUDA kernels.  It shares
no code with the CUDA path.

Readings of the paper taken here (each is checked by a pin):
 * b = abar * c (Eq. 10); the chunk formula "exp(mu^log + c^log)" is a typo for
   exp(abar^log + c^log).
 * Gamma^- is Gamma shifted down one row: (Gamma^-)[r,i] = gamma[r-1,i] for i < r
   (Appendix C substitutes S_{t-1}, hence gamma_{t-1,i}); it is not the strictly
   lower part of Gamma itself.
 * abar^{0->C-1}, b^{0->C-1} are the shifted vectors (abar_{r-1}, b_{r-1}) with
   abar_{-1} = 1, b_{-1} = 0.
 * eta is absorbed into k everywhere (P K^T, Q K^T, both state updates) except in
   p = alpha * k, which uses the raw k.
 * no epsilon is added to beta (the printed 1e-6 only serves the log of beta and
   makes the chunk form inexact); a short last chunk is padded with exact no-ops.
"""
from __future__ import annotations

import numpy as np


def coefficients(log_alpha, log_mu, beta):
    """Eq. 10 inside one chunk (requires mu > 0): returns abar, mubar, c, b [C] and
    Gamma [C,C] (lower triangular, diagonal included, gamma[r,i] for i <= r)."""
    la = np.asarray(log_alpha, dtype=np.float64)
    lm = np.asarray(log_mu, dtype=np.float64)
    be = np.asarray(beta, dtype=np.float64)
    abar = np.exp(np.cumsum(la))
    mubar = np.exp(np.cumsum(lm))
    c = np.cumsum(be * mubar / abar)
    b = abar * c
    c_prev = np.concatenate([[0.0], c[:-1]])
    Gamma = np.tril((abar[:, None] / mubar[None, :]) * (c[:, None] - c_prev[None, :]))
    return abar, mubar, c, b, Gamma


def coefficients_log_domain(log_alpha, log_mu, beta, eps=0.0):
    """The log-domain route of Section 3.1 / Appendix D (Algorithm 1 for log c):
    cumsum of the log gates, a masked row-wise log-sum-exp for log c, then
    Gamma = exp(A~) * (1 - exp(S)).  Same outputs as `coefficients`."""
    la = np.asarray(log_alpha, dtype=np.float64)
    lm = np.asarray(log_mu, dtype=np.float64)
    be = np.asarray(beta, dtype=np.float64)
    C = len(la)
    abar_log = np.cumsum(la)
    mubar_log = np.cumsum(lm)
    with np.errstate(divide="ignore"):
        term = np.log(be + eps) + mubar_log - abar_log          # log(beta_i mubar_i / abar_i)
    idx = np.arange(C)
    L = np.where(idx[:, None] >= idx[None, :], term[None, :], -np.inf)
    rmax = L.max(axis=1)
    c_log = np.log(np.exp(L - rmax[:, None]).sum(axis=1)) + rmax   # Algorithm 1
    b = np.exp(abar_log + c_log)
    c_log_prev = np.concatenate([[-np.inf], c_log[:-1]])
    A_tilde = (abar_log + c_log)[:, None] - mubar_log[None, :]
    S_log = c_log_prev[None, :] - c_log[:, None]
    Gamma = np.tril(np.exp(A_tilde) * (1.0 - np.exp(np.minimum(S_log, 0.0))))
    return np.exp(abar_log), np.exp(mubar_log), np.exp(c_log), b, Gamma


def coefficients_by_products(log_alpha, log_mu, beta):
    """The same coefficients straight from the unrolled recurrence *before* the
    summation reordering (the nested sum that precedes Eq. 7): the weight of
    k_i v~_i^T in S_r is  sum_{j=i..r} beta_j * prod_{l=j+1..r} alpha_l * prod_{l=i+1..j} mu_l,
    and the weight of -M_0 is  sum_{j<=r} beta_j * prod_{l=j+1..r} alpha_l * prod_{l<=j} mu_l.
    Division-free, so it also covers mu = 0.  Returns abar, mubar, b, Gamma, Mmask
    where Mmask[r,i] = prod_{l=i+1..r} mu_l is the weight of -k_i v~_i^T in M_r."""
    al = np.exp(np.asarray(log_alpha, dtype=np.float64))
    mu = np.exp(np.asarray(log_mu, dtype=np.float64))
    be = np.asarray(beta, dtype=np.float64)
    C = len(al)
    abar = np.array([np.prod(al[: r + 1]) for r in range(C)])
    mubar = np.array([np.prod(mu[: r + 1]) for r in range(C)])
    Gamma = np.zeros((C, C))
    Mmask = np.zeros((C, C))
    b = np.zeros(C)
    for r in range(C):
        for i in range(r + 1):
            Mmask[r, i] = np.prod(mu[i + 1: r + 1])
            Gamma[r, i] = sum(be[j] * np.prod(al[j + 1: r + 1]) * np.prod(mu[i + 1: j + 1])
                              for j in range(i, r + 1))
        b[r] = sum(be[j] * np.prod(al[j + 1: r + 1]) * np.prod(mu[: j + 1]) for j in range(r + 1))
    return abar, mubar, b, Gamma, Mmask


def shift_rows_down(G):
    """Gamma^-: row r holds row r-1 of Gamma (row 0 is zero), strictly lower part."""
    Gm = np.zeros_like(G)
    Gm[1:, :] = G[:-1, :]
    return np.tril(Gm, -1)


def chunk_forward(q, k, v, beta, log_alpha, log_mu, eta=None, *, scale=1.0, S0=None, M0=None,
                  chunk=64, eps=0.0, log_domain=False, return_stages=False):
    """Chunkwise forward for ONE (sequence, head).

    q,k: [T,dk]; v: [T,dv]; gates: [T].  Returns (o [T,dv], S [dk,dv], M [dk,dv]) and,
    with return_stages, a list of per-chunk dicts (abar, mubar, b, Gamma, T, Vtil, n).
    """
    q = np.asarray(q, dtype=np.float64); k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T_len, dk = q.shape
    dv = v.shape[1]
    be = np.asarray(beta, dtype=np.float64)
    la = np.asarray(log_alpha, dtype=np.float64)
    lm = np.asarray(log_mu, dtype=np.float64)
    et = np.ones(T_len) if eta is None else np.asarray(eta, dtype=np.float64)
    C = chunk
    S = np.zeros((dk, dv)) if S0 is None else np.array(S0, dtype=np.float64)
    M = np.zeros((dk, dv)) if M0 is None else np.array(M0, dtype=np.float64)
    o = np.zeros((T_len, dv))
    stages = []
    for t0 in range(0, T_len, C):
        n = min(C, T_len - t0)
        pad = C - n

        def padded(x, fill=0.0):
            blk = x[t0:t0 + n]
            if pad == 0:
                return blk
            shape = (pad,) + blk.shape[1:]
            return np.concatenate([blk, np.full(shape, fill)], axis=0)

        Q, K, V = padded(q), padded(k), padded(v)
        la_c, lm_c, be_c, et_c = padded(la), padded(lm), padded(be), padded(et)

        # -- coefficients (Eq. 10)
        if log_domain:
            abar, mubar, c, b, Gamma = coefficients_log_domain(la_c, lm_c, be_c, eps)
        else:
            abar, mubar, c, b, Gamma = coefficients(la_c, lm_c, be_c)
        Gamma_minus = shift_rows_down(Gamma)
        abar_minus = np.concatenate([[1.0], abar[:-1]])
        b_minus = np.concatenate([[0.0], b[:-1]])

        # -- operands: p = alpha k (raw k), eta absorbed into k
        P = np.exp(la_c)[:, None] * K
        Ke = et_c[:, None] * K

        # -- T = (I + (P K^T) .* Gamma^-)^{-1}, unit lower triangular
        A = (P @ Ke.T) * Gamma_minus
        Tm = np.linalg.inv(np.eye(C) + A)

        # -- U, Y, Z and the correction values
        U = Tm @ V
        Y = Tm @ (abar_minus[:, None] * P)
        Z = Tm @ (b_minus[:, None] * P)
        Vtil = U - Y @ S + Z @ M

        # -- output: inter-chunk + intra-chunk
        O = abar[:, None] * (Q @ S) - b[:, None] * (Q @ M) + ((Q @ Ke.T) * Gamma) @ Vtil
        o[t0:t0 + n] = scale * O[:n]

        # -- state hand-over (last row of Gamma, last entries of abar, b, mubar)
        S_next = abar[-1] * S - b[-1] * M + (Gamma[-1][:, None] * Ke).T @ Vtil
        M_next = mubar[-1] * M - ((mubar[-1] / mubar)[:, None] * Ke).T @ Vtil
        if return_stages:
            stages.append(dict(abar=abar, mubar=mubar, b=b, Gamma=Gamma, A=A, T=Tm, Vtil=Vtil,
                               n=n, S_in=S, M_in=M))
        S, M = S_next, M_next
    if return_stages:
        return o, S, M, stages
    return o, S, M
