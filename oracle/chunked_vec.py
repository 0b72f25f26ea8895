"""Chunkwise fp64 formulation of the backward with PER-CHANNEL gates in numpy -- TEST INFRASTRUCTURE ONLY.

Second rung of the oracle ladder (paper Section 4.5) for the general recurrence of Eq. 1 with gate
vectors: g_t, b_t in R^{d_k}, w_t in R^{d_v}.  The channel-wise decay cannot be pulled out of the
chunk-local contractions as a token-token matrix; it "folds inside" them (Appendix A, last paragraph):
every token-token quantity is a contraction over the channel r with the factor
exp(gam_i[r] - gam_j[r]), which is evaluated for j <= i only (non-positive exponent).

Notation for one chunk with C rows, incoming state h (d_k x d_v), gam_i = sum_{j<=i} g_j in R^{d_k}:
    Gam_i = exp(gam_i),  E_ij[r] = exp(gam_i[r] - gam_j[r]) (j <= i),  e_j = exp(gam_{C-1} - gam_j)
    A_ij = sum_r b_i[r] k_i[r] k_j[r] E_ij[r]  (j < i)        the paper's M (Section 4.2, K#2)
    T  = (I + A)^-1
    Xk_i = Gam_i . b_i . k_i,   Xv_i = w_i . v_i               ("." = elementwise)
    W  = T Xk,  Ut = T Xv,  U = Ut - W h
    P_ij = sum_r q_i[r] k_j[r] E_ij[r]  (j <= i),  O = scale ((Gam . Q) h + P U)
    Kb_j = e_j . k_j,   h' = Diag(Gam_{C-1}) h + Kb^T U
Backward, given dO and dh' (gradient w.r.t. h'):
    dU = scale P^T dO + Kb dh' ;   dh = Diag(Gam_{C-1}) dh' + scale (Gam . Q)^T dO - W^T dU       (K#1)
    dP = scale tril(dO U^T) ;  dW = -dU h^T ;  dXk = T^T dW ;  dXv = T^T dU ;  dA = -stril(dXk W^T + dXv Ut^T)
    dq_i = scale Gam_i . (h dO_i) + sum_{j<=i} dP_ij E_ij . k_j
    dk_i = [b_i . (sum_{j<i} dA_ij E_ij . k_j + Gam_i . dXk_i)]                       (row role of k_i)
         + [sum_{j>=i} dP_ji E_ji . q_j + sum_{j>i} dA_ji E_ji . b_j . k_j + e_i . (dh' U_i)]   (column role)
    db_i = k_i . (sum_{j<i} dA_ij E_ij . k_j + Gam_i . dXk_i) ;  dv_i = w_i . dXv_i ;  dw_i = v_i . dXv_i
    dgam_i = q_i . dq_i + k_i . dk_i^row - k_i . dk_i^col   (channel by channel: gam_i[r] enters as
             exp(+gam_i[r]) attached to q_i[r] or to the row role of k_i[r], as exp(-gam_i[r]) attached to the
             column role), and the last row adds  sum_j k_j . (e_j . (dh' U_j)) + Gam_{C-1} . rowdot(dh', h)
    dg_j = sum_{i>=j} dgam_i within the chunk
"""
from __future__ import annotations

import numpy as np


def chain_bwd(q, k, v, g, b, w, dO, h0, dhT, scale=1.0, C=64, keep=False):
    """One (sequence, head) chain.  q,k,g,b [L,dk]; v,w,dO [L,dv]; h0,dhT [dk,dv] or None.
    A ragged tail is identity padding: q = k = v = dO = 0, b = w = 0, g = 0 for the missing rows."""
    L, dk = q.shape
    dv = v.shape[1]
    nC = (L + C - 1) // C
    Lp = nC * C

    def pad(a):
        a = np.asarray(a, dtype=np.float64)
        if a.shape[0] == Lp:
            return a
        z = np.zeros((Lp,) + a.shape[1:])
        z[:L] = a
        return z

    q, k, v, dO, g, b, w = (pad(a) for a in (q, k, v, dO, g, b, w))
    h = np.zeros((dk, dv)) if h0 is None else np.array(h0, dtype=np.float64)
    low = np.tril(np.ones((C, C), dtype=bool))
    F, hs = [], []
    o = np.zeros((Lp, dv))
    for c in range(nC):
        s = slice(c * C, (c + 1) * C)
        Q, K, V = q[s], k[s], v[s]
        gam = np.cumsum(g[s], axis=0)                                        # [C, dk]
        Gam = np.exp(gam)
        diff = gam[:, None, :] - gam[None, :, :]                             # [i, j, r]
        E = np.where(low[:, :, None], np.exp(np.where(low[:, :, None], diff, 0.0)), 0.0)
        A = np.tril(np.einsum("ir,jr,ijr->ij", b[s] * K, K, E), -1)
        T = np.tril(np.linalg.inv(np.eye(C) + A))
        Xk = Gam * b[s] * K
        Xv = w[s] * V
        W = T @ Xk
        Ut = T @ Xv
        P = np.tril(np.einsum("ir,jr,ijr->ij", Q, K, E))
        e = np.exp(gam[-1][None, :] - gam)                                   # [C, dk]
        Kb = e * K
        f = dict(gam=gam, Gam=Gam, E=E, A=A, T=T, W=W, Ut=Ut, P=P, e=e, Kb=Kb)
        hs.append(h.copy())
        U = Ut - W @ h
        o[s] = scale * ((Gam * Q) @ h + P @ U)
        h = Gam[-1][:, None] * h + Kb.T @ U
        F.append(f)
    hT = h

    dq = np.zeros((Lp, dk)); dkk = np.zeros((Lp, dk)); dvv = np.zeros((Lp, dv))
    dgam = np.zeros((Lp, dk)); db = np.zeros((Lp, dk)); dw = np.zeros((Lp, dv))
    dh = np.zeros((dk, dv)) if dhT is None else np.array(dhT, dtype=np.float64)
    for c in range(nC - 1, -1, -1):
        s = slice(c * C, (c + 1) * C)
        f = F[c]; h = hs[c]
        Q, K, V, dOc = q[s], k[s], v[s], dO[s]
        Gam, E, T, W, Ut, P, e, Kb = f["Gam"], f["E"], f["T"], f["W"], f["Ut"], f["P"], f["e"], f["Kb"]
        dh_next = dh
        U = Ut - W @ h
        dU = scale * P.T @ dOc + Kb @ dh_next
        dh = Gam[-1][:, None] * dh_next + scale * (Gam * Q).T @ dOc - W.T @ dU
        dP = scale * np.tril(dOc @ U.T)
        dW = -dU @ h.T
        dXk = T.T @ dW
        dXv = T.T @ dU
        dA = -np.tril(dXk @ W.T + dXv @ Ut.T, -1)
        dQ = scale * Gam * (dOc @ h.T) + np.einsum("ij,ijr,jr->ir", dP, E, K)
        row = np.einsum("ij,ijr,jr->ir", dA, E, K) + Gam * dXk               # what multiplies b_i . k_i
        dK_row = b[s] * row
        UdH = U @ dh_next.T                                                  # [C, dk]
        dK_col = (np.einsum("ji,jir,jr->ir", dP, E, Q) + np.einsum("ji,jir,jr->ir", dA, E, b[s] * K) + e * UdH)
        db[s] = K * row
        dvv[s] = w[s] * dXv
        dw[s] = V * dXv
        dgc = Q * dQ + K * dK_row - K * dK_col
        dgc[-1] += np.sum(K * e * UdH, axis=0) + Gam[-1] * np.sum(dh_next * h, axis=1)
        dgam[s] = dgc
        dq[s], dkk[s] = dQ, dK_row + dK_col
        if keep:
            f.update(U=U, dU=dU, dP=dP, dXk=dXk, dXv=dXv, dA=dA, dW=dW)
    dg = np.zeros((Lp, dk))
    for c in range(nC):
        s = slice(c * C, (c + 1) * C)
        dg[s] = np.cumsum(dgam[s][::-1], axis=0)[::-1]
    out = dict(o=o[:L], hT=hT, dq=dq[:L], dk=dkk[:L], dv=dvv[:L], dg=dg[:L], db=db[:L], dw=dw[:L], dh0=dh)
    if keep:
        out["chunks"] = F
        out["h_c"] = hs
    return out


def bwd(q, k, v, g, b, w, dO, *, cu_seqlens, scale=1.0, h0=None, dhT=None, C=64):
    """Same interface and result layout as the token-serial per-channel oracle's vec_bwd()."""
    q, k, v, g, b, w, dO = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g, b, w, dO))
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu_seqlens) - 1
    out = dict(o=np.zeros((Tt, H, dv)), hT=np.zeros((N, H, dk, dv)), dq=np.zeros((Tt, H, dk)),
               dk=np.zeros((Tt, H, dk)), dv=np.zeros((Tt, H, dv)), dg=np.zeros((Tt, H, dk)), db=np.zeros((Tt, H, dk)),
               dw=np.zeros((Tt, H, dv)), dh0=np.zeros((N, H, dk, dv)))
    for n in range(N):
        a, e = int(cu_seqlens[n]), int(cu_seqlens[n + 1])
        for hd in range(H):
            r = chain_bwd(q[a:e, hd], k[a:e, hd], v[a:e, hd], g[a:e, hd], b[a:e, hd], w[a:e, hd], dO[a:e, hd],
                          None if h0 is None else h0[n, hd], None if dhT is None else dhT[n, hd], scale=scale, C=C)
            for name in ("o", "dq", "dk", "dv", "dg", "db", "dw"):
                out[name][a:e, hd] = r[name]
            out["hT"][n, hd] = r["hT"]
            out["dh0"][n, hd] = r["dh0"]
    return out
