"""Independent fp64 restatements of the gated delta rule -- TEST INFRASTRUCTURE ONLY.

Each function works on ONE (sequence, value head): q,k [T,dk], v [T,dv], g,beta [T],
S0 [dv,dk], all float64, and returns (out [T,dv], S_T [dv,dk]).  None of them is
used by the C oracle; the pin tests require all of them to agree with it.
"""
from __future__ import annotations

import numpy as np


def paper_form(q, k, v, g, beta, S0):
    """The recurrence exactly as the paper's Section 3.2 writes it: state held K x V,
    multiplicative gate, output taken from the *decayed old* state plus a scalar
    correction, out = q^T(gS) + delta (q^T k), so the new state is never re-read."""
    T, dk = k.shape
    S = np.array(S0, dtype=np.float64).T.copy()  # K x V
    out = np.zeros((T, v.shape[1]))
    for t in range(T):
        gate = np.exp(g[t])
        gS = gate * S
        old_v = k[t] @ gS
        delta = beta[t] * (v[t] - old_v)
        out[t] = q[t] @ gS + delta * (q[t] @ k[t])
        S = gS + np.outer(k[t], delta)
    return out, S.T.copy()


def explicit_product(q, k, v, g, beta, S0):
    """Brute force with dense transition matrices: M_t = alpha_t (I - beta_t k_t k_t^T),
    S_t = S0 M_1..M_t + sum_j beta_j v_j k_j^T M_{j+1}..M_t, o_t = S_t q_t."""
    T, dk = k.shape
    I = np.eye(dk)
    M = [np.exp(g[t]) * (I - beta[t] * np.outer(k[t], k[t])) for t in range(T)]
    out = np.zeros((T, v.shape[1]))
    S_t = np.array(S0, dtype=np.float64)
    for t in range(T):
        prod = I.copy()
        for s in range(t + 1):
            prod = prod @ M[s]
        S_t = np.array(S0, dtype=np.float64) @ prod
        for j in range(t + 1):
            tail = I.copy()
            for s in range(j + 1, t + 1):
                tail = tail @ M[s]
            S_t = S_t + beta[j] * np.outer(v[j], k[j]) @ tail
        out[t] = S_t @ q[t]
    return out, S_t


def chunked(q, k, v, g, beta, S0, C=64):
    """Chunked WY / UT-transform form.  Per chunk of L <= C tokens with incoming state S:
        gamma = cumsum(g), Gamma = exp(gamma), D_ij = exp(gamma_i - gamma_j) [j <= i]
        A = strict_lower(diag(beta) (K K^T o D)),  Tm = (I + A)^{-1}
        U = Tm diag(beta) V,  W = Tm diag(beta o Gamma) K
        Delta = U - W S^T
        O = diag(Gamma) Q S^T + ((Q K^T) o D) Delta
        S <- Gamma_L S + Delta^T diag(exp(gamma_L - gamma)) K
    The differences gamma_i - gamma_j are formed before exp and masked before exp."""
    T, dk = k.shape
    dv = v.shape[1]
    S = np.array(S0, dtype=np.float64)
    out = np.zeros((T, dv))
    for c0 in range(0, T, C):
        sl = slice(c0, min(T, c0 + C))
        K, Q, V, b = k[sl], q[sl], v[sl], beta[sl]
        L = K.shape[0]
        gam = np.cumsum(g[sl])
        diff = gam[:, None] - gam[None, :]
        low = np.tril(np.ones((L, L), dtype=bool))
        D = np.where(low, np.exp(np.where(low, diff, 0.0)), 0.0)
        A = np.tril(b[:, None] * (K @ K.T) * D, -1)
        Tm = np.linalg.solve(np.eye(L) + A, np.eye(L))
        U = Tm @ (b[:, None] * V)
        W = Tm @ ((b * np.exp(gam))[:, None] * K)
        Delta = U - W @ S.T
        out[sl] = np.exp(gam)[:, None] * (Q @ S.T) + ((Q @ K.T) * D) @ Delta
        S = np.exp(gam[-1]) * S + Delta.T @ (np.exp(gam[-1] - gam)[:, None] * K)
    return out, S


def orthogonal_keys_closed_form(q, k, v, g, beta, S0):
    """Valid only when the keys are pairwise orthogonal with unit norm (K K^T = I).
    Then the triangular system vanishes and the sequence is gated linear attention:
        Delta = diag(beta) (V - diag(Gamma) K S0^T)
        O = diag(Gamma) Q S0^T + ((Q K^T) o D) Delta
        S_T = Gamma_T S0 + Delta^T diag(exp(gamma_T - gamma)) K
    with gamma the cumulative log-gate over the whole sequence."""
    gam = np.cumsum(g)
    T = k.shape[0]
    low = np.tril(np.ones((T, T), dtype=bool))
    D = np.where(low, np.exp(np.where(low, gam[:, None] - gam[None, :], 0.0)), 0.0)
    Delta = beta[:, None] * (v - np.exp(gam)[:, None] * (k @ S0.T))
    out = np.exp(gam)[:, None] * (q @ S0.T) + ((q @ k.T) * D) @ Delta
    S = np.exp(gam[-1]) * S0 + Delta.T @ (np.exp(gam[-1] - gam)[:, None] * k)
    return out, S
