"""Independent restatements of published rules, used only to pin the oracle.

Nothing here is imported by the oracle or by the CUDA path.  Each function is a
direct transcription of a different passage of the paper than the one the
oracle follows, in the paper's own orientation S in R^{d_v x d_k}.
"""
import numpy as np


def gated_delta_rule(q, k, v, beta, alpha, S0=None):
    """GatedDeltaNet, Eq. 3 (alpha = 1 gives DeltaNet, Eq. 2): one sequence.

    q,k [T,dk], v [T,dv]; returns (o [T,dv], S_T [dv,dk]) with o_t = S_t q_t."""
    T, dk = k.shape
    dv = v.shape[1]
    S = np.zeros((dv, dk)) if S0 is None else np.array(S0, np.float64)
    o = np.zeros((T, dv))
    I = np.eye(dk)
    for t in range(T):
        S = S @ (alpha[t] * (I - beta[t] * np.outer(k[t], k[t]))) + beta[t] * np.outer(v[t], k[t])
        o[t] = S @ q[t]
    return o, S


def qdelta_error_form(S, q, k, v, beta, lam):
    """Ungated rule as first printed (error-driven form, Section 3.3.1)."""
    v_hat = S @ k
    o_hat = S @ q
    return S + beta * np.outer(v - v_hat - lam * o_hat, k)


def qdelta_linear_form(S, q, k, v, beta, lam):
    """Ungated rule in its 'equivalent linear form' (Section 3.3.1)."""
    dk = k.shape[0]
    return S @ (np.eye(dk) - beta * (np.outer(k, k) + lam * np.outer(q, k))) + beta * np.outer(v, k)


def qdelta_gated_form(S, q, k, v, beta, alpha, lam):
    """Final rule with forget gate (Section 3.3.1) / Table 1 row."""
    dk = k.shape[0]
    return alpha * S @ (np.eye(dk) - beta * (np.outer(k, k) + lam * np.outer(q, k))) + beta * np.outer(v, k)


def chunk_expansion_bruteforce(S0, q, k, v, beta, alpha, lam):
    """State after r steps from the chunk-expansion equation (Section 3.3.2):
    S^r = S F^r + G^r with explicit products of alpha_i P_i.  Returns list of S^r."""
    T, dk = k.shape
    I = np.eye(dk)
    Pm = [alpha[i] * (I - beta[i] * np.outer(k[i] + lam[i] * q[i], k[i])) for i in range(T)]
    out = []
    for r in range(1, T + 1):
        F = I.copy()
        for i in range(r):
            F = F @ Pm[i]
        G = np.zeros_like(S0)
        for i in range(r):
            tail = I.copy()
            for j in range(i + 1, r):
                tail = tail @ Pm[j]
            G = G + beta[i] * np.outer(v[i], k[i]) @ tail
        out.append(S0 @ F + G)
    return out


def value_span_state(q, k, v, beta, alpha, lam):
    """Value-span decomposition (Section 3.1): S_t = sum_tau v_tau b_{tau,t}^T with
    b_{tau,t} = P_t^T b_{tau,t-1}, b_{t,t} = eta_t k_t; S_0 = 0.  Returns list of S_t."""
    T, dk = k.shape
    I = np.eye(dk)
    b = []
    out = []
    for t in range(T):
        P = alpha[t] * (I - beta[t] * np.outer(k[t] + lam[t] * q[t], k[t]))
        b = [P.T @ bb for bb in b]
        b.append(beta[t] * k[t])
        out.append(sum(np.outer(v[tau], b[tau]) for tau in range(t + 1)))
    return out


def wy_vectors(q, k, beta, lam):
    """Extended WY recursion for w^r (Section 3.3.2): returns W [C,dk] (rows w^r)."""
    C, dk = k.shape
    X = k + lam[:, None] * q
    W = np.zeros((C, dk))
    for r in range(C):
        acc = X[r].copy()
        for i in range(r):
            acc -= W[i] * (k[i] @ X[r])
        W[r] = beta[r] * acc
    return W
