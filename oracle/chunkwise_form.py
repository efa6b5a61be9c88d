"""Separately written numpy fp64 chunkwise-parallel form of Q-Delta.

TEST INFRASTRUCTURE ONLY.  It exists to cross-check the recurrence oracle
(``oracle.recurrence``): the two are written independently and must agree to
rounding for every chunk size that divides T.

Forward follows Section 3.3.2: chunk expansion S^r = gamma^r S P^r + G^r, the
extended WY vectors w^r and u~^r, their UT-transform matrix form (Eq. for U~
and W), and the chunk-level state update / output equations, with these
readings where the printed text is inconsistent:

* state held transposed, h = S^T (d_k x d_v);
* "U~ - W<- S" is read as  U~ - W<- S^T  (the printed product does not conform);
* Q<- = diag(gamma) Q (never defined in the text; forced by the expansion of
  S^r applied at every r);
* the intra-chunk output term carries the decay ratio: (Gamma o Q K^T o M) with
  Gamma_ri = gamma^r / gamma^i and M the causal mask INCLUDING the diagonal
  (read-out uses the post-update state);
* the Gram matrix inside the UT transform is X K^T (entry (r,i) = x_r . k_i), as
  in the main text and in the appendix's own row formula;
* W<- = diag(gamma) W is obtained from ONE inverse:
  diag(gamma)(I+A0)^-1 = (I+A)^-1 diag(gamma) because A = diag(gamma) A0 diag(gamma)^-1.

The backward is the hand-derived gradient of exactly these chunk equations
(the paper gives none); it is a third form next to the recurrence reverse pass.
"""
import numpy as np


def _chunk_quantities(Q, K, V, beta, alpha, lam):
    """Per-chunk, state-independent quantities.  Q,K [C,dk], V [C,dv]."""
    C = Q.shape[0]
    g = np.cumsum(np.log(alpha))                      # g_r = log gamma^r
    gam = np.exp(g)
    r = np.arange(C)
    diff = g[:, None] - g[None, :]
    low_i = r[:, None] >= r[None, :]                  # causal incl. diagonal
    low_s = r[:, None] > r[None, :]                   # strictly lower
    Gam = np.where(low_i, np.exp(np.where(low_i, diff, 0.0)), 0.0)
    X = K + lam[:, None] * Q
    XK = X @ K.T
    A = np.where(low_s, beta[:, None] * Gam * XK, 0.0)
    M = np.linalg.solve(np.eye(C) + A, np.eye(C))     # (I + A)^-1
    Tm = M * beta[None, :]                            # M diag(beta)
    U = Tm @ V                                        # U~
    W = Tm @ (gam[:, None] * X)                       # W<-
    P = np.where(low_i, Gam * (Q @ K.T), 0.0)
    Kt = np.exp(g[-1] - g)[:, None] * K               # K-> rows scaled by gamma^C/gamma^r
    return dict(g=g, gam=gam, Gam=Gam, X=X, XK=XK, A=A, M=M, T=Tm, U=U, W=W, P=P, Kt=Kt,
                low_i=low_i, low_s=low_s)


def forward(q, k, v, beta, alpha=None, lam=None, h0=None, chunk=64, return_states=False):
    """Chunkwise forward.  Shapes as in ``oracle.recurrence.forward``."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    assert T % chunk == 0
    beta = np.asarray(beta, np.float64)
    alpha = np.ones((B, T, H)) if alpha is None else np.asarray(alpha, np.float64)
    lam = np.zeros((B, T, H)) if lam is None else np.asarray(lam, np.float64)
    o = np.zeros((B, T, H, dv))
    hT = np.zeros((B, H, dk, dv))
    states = np.zeros((B, H, T // chunk, dk, dv))
    for b in range(B):
        for hh in range(H):
            h = np.zeros((dk, dv)) if h0 is None else np.array(h0[b, hh], np.float64)
            for n in range(T // chunk):
                s = slice(n * chunk, (n + 1) * chunk)
                c = _chunk_quantities(q[b, s, hh], k[b, s, hh], v[b, s, hh],
                                      beta[b, s, hh], alpha[b, s, hh], lam[b, s, hh])
                states[b, hh, n] = h
                D = c["U"] - c["W"] @ h                                   # rows = delta_r
                o[b, s, hh] = (c["gam"][:, None] * q[b, s, hh]) @ h + c["P"] @ D
                h = c["gam"][-1] * h + c["Kt"].T @ D
            hT[b, hh] = h
    if return_states:
        return o, hT, states
    return o, hT


def backward(q, k, v, beta, alpha, lam, h0, dO, dhT=None, chunk=64):
    """Gradient of ``forward`` chunk by chunk (reverse over chunks)."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    beta = np.asarray(beta, np.float64)
    alpha = np.ones((B, T, H)) if alpha is None else np.asarray(alpha, np.float64)
    lam = np.zeros((B, T, H)) if lam is None else np.asarray(lam, np.float64)
    dO = np.asarray(dO, np.float64)
    _, _, states = forward(q, k, v, beta, alpha, lam, h0, chunk, return_states=True)
    out = dict(dq=np.zeros_like(q), dk=np.zeros_like(k), dv=np.zeros_like(v),
               dbeta=np.zeros((B, T, H)), dalpha=np.zeros((B, T, H)), dlam=np.zeros((B, T, H)),
               dh0=np.zeros((B, H, dk, dv)))
    for b in range(B):
        for hh in range(H):
            dh = np.zeros((dk, dv)) if dhT is None else np.array(dhT[b, hh], np.float64)
            for n in reversed(range(T // chunk)):
                s = slice(n * chunk, (n + 1) * chunk)
                Q, K, V = q[b, s, hh], k[b, s, hh], v[b, s, hh]
                bt, al, lm = beta[b, s, hh], alpha[b, s, hh], lam[b, s, hh]
                c = _chunk_quantities(Q, K, V, bt, al, lm)
                h = states[b, hh, n]
                gam, Gam, X, M, Tm, W, P, Kt = (c[x] for x in
                                                ("gam", "Gam", "X", "M", "T", "W", "P", "Kt"))
                D = c["U"] - W @ h
                dOc = dO[b, s, hh]
                # h_out = gam_C h + Kt^T D ;  O = gamQ h + P D
                Kdh = Kt @ dh
                dD = P.T @ dOc + Kdh
                dP = np.where(c["low_i"], dOc @ D.T, 0.0)
                dPG = dP * Gam
                dQ1 = gam[:, None] * (dOc @ h.T)
                dQ = dQ1 + dPG @ K
                dK = dPG.T @ Q + np.exp(c["g"][-1] - c["g"])[:, None] * (D @ dh.T)
                dW = -dD @ h.T
                dh_in = gam[-1] * dh + (gam[:, None] * Q).T @ dOc - W.T @ dD
                # U = T V ; W = T (gam X)
                gX = gam[:, None] * X
                dT = dD @ V.T + dW @ gX.T
                dV = Tm.T @ dD
                dXg = Tm.T @ dW
                dX = gam[:, None] * dXg
                # T = M diag(beta) ; M = (I+A)^-1
                dbt = np.sum(dT * M, axis=0)
                dM = dT * bt[None, :]
                dA = np.where(c["low_s"], -(M.T @ dM @ M.T), 0.0)
                # A_ri = beta_r Gam_ri XK_ri
                dbt = dbt + np.sum(dA * Gam * c["XK"], axis=1)
                dXK = dA * bt[:, None] * Gam
                dX = dX + dXK @ K
                dK = dK + dXK.T @ X
                # X = K + lam Q
                dK = dK + dX
                dQ = dQ + lm[:, None] * dX
                dlm = np.sum(dX * Q, axis=1)
                # log-decay: every place g enters
                dPP = dP * P
                dAA = dA * c["A"]
                dg = (np.sum(dQ1 * Q, axis=1)
                      + dPP.sum(axis=1) - dPP.sum(axis=0)
                      + np.sum(dXg * gX, axis=1)
                      + dAA.sum(axis=1) - dAA.sum(axis=0)
                      - np.sum(Kdh * D, axis=1))
                dg[-1] += gam[-1] * np.sum(dh * h) + np.sum(Kdh * D)
                dlog = np.cumsum(dg[::-1])[::-1]          # g_r = sum_{i<=r} log alpha_i
                out["dq"][b, s, hh] = dQ
                out["dk"][b, s, hh] = dK
                out["dv"][b, s, hh] = dV
                out["dbeta"][b, s, hh] = dbt
                out["dlam"][b, s, hh] = dlm
                out["dalpha"][b, s, hh] = dlog / al
                dh = dh_in
            out["dh0"][b, hh] = dh
    return out
