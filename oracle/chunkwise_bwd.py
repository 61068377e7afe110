"""fp64 chunk-form backward of the MDN recurrence (TEST INFRASTRUCTURE ONLY; numpy, one chain at a time).

The stepwise backward oracle (mdn_stepwise_bwd.c) differentiates the recurrence token by token.  This module
differentiates the CHUNKWISE algorithm of Section 3.1 instead, matrix by matrix, in the "lean" form

    X = K S,  Y = K M,  R = V - abar.X + p.Y,  V~ = T R,  T = (I + A)^-1,  A = G^- o (K K^T),  W = scale Geta o (Q K^T)
    O = scale (abar.(Q S) - b.(Q M)) + W V~,   S' = abar_C S - b_C M + K^T (g_S.V~),   M' = mubar_C M - K^T (g_M.V~)

(`.` scales rows by a vector, `o` is the element-wise product), so that a chunk-parallel CUDA backward has a
reference for every intermediate: the adjoint state recurrence (dS, dM), dV = dR, dQ, dK, and the gate gradients
through the adjoints of the coefficient vectors and of the two masks, followed by the coefficient scans in reverse.
Both oracles must give the same gradients (tests/test_oracle_bwd_pins.py); nothing here is shared with the CUDA path.
"""
import numpy as np


def chunk_coefficients(alpha, mu, beta, eta):
    """Coefficient vectors and masks of one chunk (n tokens) by the plain recurrences of Eq. 10."""
    n = len(alpha)
    abar, mubar = np.cumprod(alpha), np.cumprod(mu)
    gam = np.zeros((n, n))      # gamma[r, i], i <= r
    mm = np.zeros((n, n))       # m[r, i] = prod_{i < l <= r} mu_l
    for i in range(n):
        m, g = 1.0, 0.0
        for r in range(i, n):
            if r > i:
                m *= mu[r]
            g = alpha[r] * g + beta[r] * m
            gam[r, i], mm[r, i] = g, m
    b = np.zeros(n)
    prev = 0.0
    for r in range(n):
        prev = alpha[r] * prev + beta[r] * mubar[r]
        b[r] = prev
    b_prev = np.concatenate([[0.0], b[:-1]])
    Gm = np.zeros((n, n))       # G^-[r, i] = alpha_r gamma[r-1, i] eta_i, i < r
    for r in range(1, n):
        Gm[r, :r] = alpha[r] * gam[r - 1, :r] * eta[:r]
    Geta = np.tril(gam * eta[None, :])
    return dict(abar=abar, mubar=mubar, b=b, b_prev=b_prev, p=alpha * b_prev, gam=gam, mm=mm, Gm=Gm, Geta=Geta,
                gS=gam[-1] * eta, gM=mm[-1] * eta)


def chunk_forward(Q, K, V, S, M, co, scale):
    X, Y = K @ S, K @ M
    A = co["Gm"] * (K @ K.T)
    T = np.linalg.inv(np.eye(len(Q)) + A)
    W = scale * co["Geta"] * (Q @ K.T)
    R = V - co["abar"][:, None] * X + co["p"][:, None] * Y
    Vt = T @ R
    O = scale * (co["abar"][:, None] * (Q @ S) - co["b"][:, None] * (Q @ M)) + W @ Vt
    S1 = co["abar"][-1] * S - co["b"][-1] * M + K.T @ (co["gS"][:, None] * Vt)
    M1 = co["mubar"][-1] * M - K.T @ (co["gM"][:, None] * Vt)
    return dict(X=X, Y=Y, T=T, W=W, R=R, Vt=Vt, O=O, S1=S1, M1=M1)


def chunk_backward(Q, K, S, M, co, fw, dO, dS1, dM1, alpha, mu, beta, eta, scale):
    """Adjoints of one chunk.  Returns dS, dM (start state), dQ, dK, dV and d(log alpha), d(log mu), dbeta, deta."""
    n = len(Q)
    abar, b, p, gS, gM = co["abar"], co["b"], co["p"], co["gS"], co["gM"]
    T, Vt, X, Y = fw["T"], fw["Vt"], fw["X"], fw["Y"]
    KdS, KdM = K @ dS1, K @ dM1
    dVt = fw["W"].T @ dO + gS[:, None] * KdS - gM[:, None] * KdM
    dR = T.T @ dVt
    dS = abar[-1] * dS1 - K.T @ (abar[:, None] * dR) + scale * Q.T @ (abar[:, None] * dO)
    dM = -b[-1] * dS1 + co["mubar"][-1] * dM1 + K.T @ (p[:, None] * dR) - scale * Q.T @ (b[:, None] * dO)
    dOVt = np.tril(dO @ Vt.T)
    DW = scale * co["Geta"] * dOVt
    dA = -np.tril(dR @ Vt.T, -1)
    DA = co["Gm"] * dA
    dQ = scale * (abar[:, None] * (dO @ S.T) - b[:, None] * (dO @ M.T)) + DW @ K
    dK = (-(abar[:, None] * dR) @ S.T + (p[:, None] * dR) @ M.T + gS[:, None] * (Vt @ dS1.T) - gM[:, None] * (Vt @ dM1.T)
          + DW.T @ Q + (DA + DA.T) @ K)
    # ---- adjoints of the coefficient vectors and masks
    QS, QM = Q @ S, Q @ M
    d_abar = -np.sum(dR * X, 1) + scale * np.sum(dO * QS, 1)
    d_b = -scale * np.sum(dO * QM, 1)
    d_p = np.sum(dR * Y, 1)
    d_gS = np.sum(Vt * KdS, 1)
    d_gM = -np.sum(Vt * KdM, 1)
    d_abar[-1] += np.sum(dS1 * S)
    d_b[-1] -= np.sum(dS1 * M)
    d_mubar = np.zeros(n)
    d_mubar[-1] += np.sum(dM1 * M)
    d_Geta = scale * dOVt * (Q @ K.T)          # adjoint of Geta[r, i], i <= r
    d_Gm = dA * (K @ K.T)                      # adjoint of G^-[r, i], i < r
    # ---- the scans of Eq. 10 in reverse
    gam, mm = co["gam"], co["mm"]
    d_alpha, d_mu, d_beta, d_eta = np.zeros(n), np.zeros(n), np.zeros(n), np.zeros(n)
    d_gam = d_Geta * eta[None, :]
    d_eta += np.sum(d_Geta * gam, 0)
    d_mm = np.zeros((n, n))
    d_gam[-1] += d_gS * eta
    d_mm[-1] += d_gM * eta
    d_eta += d_gS * gam[-1] + d_gM * mm[-1]
    for r in range(1, n):                      # G^-[r, i] = alpha_r gamma[r-1, i] eta_i
        d_gam[r - 1, :r] += d_Gm[r, :r] * alpha[r] * eta[:r]
        d_alpha[r] += np.sum(d_Gm[r, :r] * gam[r - 1, :r] * eta[:r])
        d_eta[:r] += d_Gm[r, :r] * alpha[r] * gam[r - 1, :r]
    for i in range(n):                         # column recurrences, last row first
        for r in range(n - 1, i - 1, -1):
            g_prev = gam[r - 1, i] if r > i else 0.0
            d_alpha[r] += d_gam[r, i] * g_prev
            d_beta[r] += d_gam[r, i] * mm[r, i]
            d_mm[r, i] += d_gam[r, i] * beta[r]
            if r > i:
                d_gam[r - 1, i] += d_gam[r, i] * alpha[r]
                d_mu[r] += d_mm[r, i] * mm[r - 1, i]
                d_mm[r - 1, i] += d_mm[r, i] * mu[r]
    b_prev = co["b_prev"]
    for r in range(n):                         # p_r = alpha_r b_{r-1}
        d_alpha[r] += d_p[r] * b_prev[r]
        if r > 0:
            d_b[r - 1] += d_p[r] * alpha[r]
    for r in range(n - 1, -1, -1):             # b_r = alpha_r b_{r-1} + beta_r mubar_r
        d_alpha[r] += d_b[r] * b_prev[r]
        d_beta[r] += d_b[r] * co["mubar"][r]
        d_mubar[r] += d_b[r] * beta[r]
        if r > 0:
            d_b[r - 1] += d_b[r] * alpha[r]
    for r in range(n - 1, -1, -1):             # abar_r = alpha_r abar_{r-1},  mubar_r = mu_r mubar_{r-1}
        a_prev = abar[r - 1] if r > 0 else 1.0
        m_prev = co["mubar"][r - 1] if r > 0 else 1.0
        d_alpha[r] += d_abar[r] * a_prev
        d_mu[r] += d_mubar[r] * m_prev
        if r > 0:
            d_abar[r - 1] += d_abar[r] * alpha[r]
            d_mubar[r - 1] += d_mubar[r] * mu[r]
    return dict(dS=dS, dM=dM, dQ=dQ, dK=dK, dV=dR, dlog_alpha=alpha * d_alpha, dlog_mu=mu * d_mu, dbeta=d_beta,
                deta=d_eta)


def chain_backward(q, k, v, beta, log_alpha, log_mu, eta, d_o, scale=1.0, S0=None, M0=None, dS_final=None,
                   dM_final=None, chunk=64):
    """One (sequence, head): q, k [T, dk]; v, d_o [T, dv]; gates [T].  Forward chunk by chunk keeping every chunk's
    start state, then the chunks in reverse.  Returns the same dict of gradients as oracle.stepwise_bwd (one chain)."""
    f8 = np.float64
    q, k, v, d_o = (np.asarray(x, dtype=f8) for x in (q, k, v, d_o))
    T_, dk = q.shape
    dv = v.shape[1]
    alpha, mu = np.exp(np.asarray(log_alpha, dtype=f8)), np.exp(np.asarray(log_mu, dtype=f8))
    beta = np.asarray(beta, dtype=f8)
    eta = np.ones(T_) if eta is None else np.asarray(eta, dtype=f8)
    S = np.zeros((dk, dv)) if S0 is None else np.asarray(S0, dtype=f8)
    M = np.zeros((dk, dv)) if M0 is None else np.asarray(M0, dtype=f8)
    saved = []
    for t0 in range(0, T_, chunk):
        sl = slice(t0, min(T_, t0 + chunk))
        co = chunk_coefficients(alpha[sl], mu[sl], beta[sl], eta[sl])
        fw = chunk_forward(q[sl], k[sl], v[sl], S, M, co, scale)
        saved.append((sl, S, M, co, fw))
        S, M = fw["S1"], fw["M1"]
    dS = np.zeros((dk, dv)) if dS_final is None else np.asarray(dS_final, dtype=f8)
    dM = np.zeros((dk, dv)) if dM_final is None else np.asarray(dM_final, dtype=f8)
    out = dict(dq=np.zeros((T_, dk)), dk=np.zeros((T_, dk)), dv=np.zeros((T_, dv)), dbeta=np.zeros(T_),
               dlog_alpha=np.zeros(T_), dlog_mu=np.zeros(T_), deta=np.zeros(T_))
    adj_end = []                # (dS', dM') at the END of every chunk, last chunk first
    for sl, S_c, M_c, co, fw in reversed(saved):
        adj_end.append((dS, dM))
        g = chunk_backward(q[sl], k[sl], S_c, M_c, co, fw, d_o[sl], dS, dM, alpha[sl], mu[sl], beta[sl], eta[sl], scale)
        out["dq"][sl], out["dk"][sl], out["dv"][sl] = g["dQ"], g["dK"], g["dV"]
        for name in ("dbeta", "dlog_alpha", "dlog_mu", "deta"):
            out[name][sl] = g[name]
        dS, dM = g["dS"], g["dM"]
    out["dS0"], out["dM0"] = dS, dM
    out["adj_end"] = adj_end[::-1]      # indexed by chunk
    return out
