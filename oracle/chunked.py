"""Chunkwise fp64 formulation of the GDN backward in numpy -- TEST INFRASTRUCTURE ONLY.

Second rung of the oracle ladder (paper Section 4.5: token-serial oracle -> chunkwise reference ->
kernels).  It re-associates the token recurrence of Eq. 1 into chunks of C tokens: everything inside
a chunk becomes small dense products, and only a d_k x d_v state crosses chunk borders (Section 4.2:
"parallel inside chunks, short sequential carry between chunks, backward runs it in reverse").
The tests require it to agree with the token-serial C oracle to ~1e-12, for several chunk sizes;
it is also what the CUDA kernels are compared with stage by stage when localising a bug.

Notation for one chunk with C rows (tokens), incoming state h (d_k x d_v):
    gam_i = sum_{j<=i} g_j,  Gam = exp(gam),  gam_e = gam_{C-1},  D_ij = exp(gam_i - gam_j) for j<=i
    A  = stril(Diag(b) (K K^T . D))               the paper's M (Section 4.2, K#2)
    T  = (I + A)^-1                               unit lower triangular
    W  = T Diag(b Gam) K,   Ut = T Diag(w) V,     U = Ut - W h
    P  = tril(Q K^T . D),   O = scale (Diag(Gam) Q h + P U)
    Kb = Diag(exp(gam_e - gam)) K,   h' = Gam_e h + Kb^T U
The chain step can be written with chunk-local matrices only (used by the CUDA scans):
    Nm = Kb^T W,  Bf = Kb^T Ut        =>  h'  = Gam_e h  - Nm h    + Bf
    E  = scale (Diag(Gam)Q - P W)^T dO =>  dh  = Gam_e dh' - Nm^T dh' + E
"""
from __future__ import annotations

import numpy as np


def _chunk_fwd_factors(Q, K, V, g, b, w, scale):
    C = K.shape[0]
    gam = np.cumsum(g)
    Gam = np.exp(gam)
    diff = gam[:, None] - gam[None, :]
    low = np.tril(np.ones((C, C), dtype=bool))
    D = np.where(low, np.exp(np.where(low, diff, 0.0)), 0.0)   # mask before exponentiating
    KK = K @ K.T
    A = np.tril(b[:, None] * KK * D, -1)
    T = np.linalg.inv(np.eye(C) + A)
    T = np.tril(T)
    W = T @ ((b * Gam)[:, None] * K)
    Ut = T @ (w[:, None] * V)
    P = np.tril((Q @ K.T) * D)
    e = np.exp(gam[-1] - gam)
    Kb = e[:, None] * K
    return dict(gam=gam, Gam=Gam, D=D, KK=KK, A=A, T=T, W=W, Ut=Ut, P=P, e=e, Kb=Kb)


def chain_bwd(q, k, v, g, b, w, dO, h0, dhT, scale=1.0, C=64, keep=False):
    """One (sequence, head) chain.  q,k [L,dk]; v,dO [L,dv]; g,b,w [L]; h0,dhT [dk,dv] or None.

    Returns dict(o, hT, dq, dk, dv, dg, db, dw, dh0) (+ per-chunk intermediates when keep=True).
    A ragged tail is handled by identity padding: q=k=v=dO=0, b=w=0, g=0 for the missing rows.
    """
    L, dk = q.shape
    dv = v.shape[1]
    nC = (L + C - 1) // C
    Lp = nC * C

    def pad(a):
        if a.shape[0] == Lp:
            return np.asarray(a, dtype=np.float64)
        z = np.zeros((Lp,) + a.shape[1:])
        z[:L] = a
        return z

    q, k, v, dO, g, b, w = (pad(np.asarray(a, dtype=np.float64)) for a in (q, k, v, dO, g, b, w))
    h = np.zeros((dk, dv)) if h0 is None else np.array(h0, dtype=np.float64)
    F, hs = [], []
    o = np.zeros((Lp, dv))
    # forward: chunk-local factors, then the carry h' = Gam_e h - Nm h + Bf
    for c in range(nC):
        s = slice(c * C, (c + 1) * C)
        f = _chunk_fwd_factors(q[s], k[s], v[s], g[s], b[s], w[s], scale)
        f["Nm"] = f["Kb"].T @ f["W"]
        f["Bf"] = f["Kb"].T @ f["Ut"]
        f["Qg"] = f["Gam"][:, None] * q[s]
        f["E"] = scale * (f["Qg"] - f["P"] @ f["W"]).T @ dO[s]
        hs.append(h.copy())
        U = f["Ut"] - f["W"] @ h
        o[s] = scale * (f["Qg"] @ h + f["P"] @ U)
        h_next = f["Gam"][-1] * h - f["Nm"] @ h + f["Bf"]
        # the two-step form must agree with the affine form
        assert np.allclose(h_next, f["Gam"][-1] * h + f["Kb"].T @ U, rtol=1e-10, atol=1e-12)
        h = h_next
        F.append(f)
    hT = h

    dq = np.zeros((Lp, dk)); dkk = np.zeros((Lp, dk)); dvv = np.zeros((Lp, dv))
    dgam = np.zeros(Lp); db = np.zeros(Lp); dw = np.zeros(Lp)
    dh = np.zeros((dk, dv)) if dhT is None else np.array(dhT, dtype=np.float64)
    dhs = [None] * nC
    for c in range(nC - 1, -1, -1):
        s = slice(c * C, (c + 1) * C)
        f = F[c]; h = hs[c]
        Q, K, V, dOc = q[s], k[s], v[s], dO[s]
        Gam, D, T, W, Ut, P, e, Kb, A = f["Gam"], f["D"], f["T"], f["W"], f["Ut"], f["P"], f["e"], f["Kb"], f["A"]
        dh_next = dh
        dhs[c] = dh_next.copy()
        U = Ut - W @ h
        # gradient w.r.t. U: through the output and through the state write
        KbdH = Kb @ dh_next
        dU = scale * P.T @ dOc + KbdH
        # reverse-state step (K#1)
        dh = Gam[-1] * dh_next - f["Nm"].T @ dh_next + f["E"]
        assert np.allclose(dh, Gam[-1] * dh_next + scale * f["Qg"].T @ dOc - W.T @ dU, rtol=1e-10, atol=1e-12)
        # intra-chunk gradients
        dP = scale * np.tril(dOc @ U.T)
        dPD = dP * D
        dOh = dOc @ h.T                                  # [C, dk]
        dQ = scale * Gam[:, None] * dOh + dPD @ K
        dK = dPD.T @ Q + e[:, None] * (U @ dh_next.T)
        # WY / triangular-inverse VJP (K#2): reuse T, never re-invert
        dW = -dU @ h.T
        dXk = T.T @ dW
        dXv = T.T @ dU
        dA = -np.tril(dXk @ W.T + dXv @ Ut.T, -1)
        G = dA * D
        bG = b[s][:, None] * G
        dK += bG @ K + bG.T @ K + (b[s] * Gam)[:, None] * dXk
        dV = w[s][:, None] * dXv
        db[s] = np.sum(G * f["KK"], axis=1) + Gam * np.sum(dXk * K, axis=1)
        dw[s] = np.sum(dXv * V, axis=1)
        r = np.sum(KbdH * U, axis=1)
        dAA = dA * A
        dPP = dP * P
        dgc = (dAA.sum(1) - dAA.sum(0) + dPP.sum(1) - dPP.sum(0)
               + b[s] * Gam * np.sum(dXk * K, axis=1) + scale * Gam * np.sum(Q * dOh, axis=1) - r)
        dgc[-1] += r.sum() + Gam[-1] * np.sum(dh_next * h)
        dgam[s] = dgc
        dq[s], dkk[s], dvv[s] = dQ, dK, dV
        if keep:
            f.update(U=U, dU=dU, dP=dP, dXk=dXk, dXv=dXv, dA=dA, dW=dW, dgam=dgc.copy())
    # gam_i = sum_{j<=i} g_j inside a chunk  =>  dg_j = sum_{i>=j} dgam_i (reverse cumulative sum)
    dg = np.zeros(Lp)
    for c in range(nC):
        s = slice(c * C, (c + 1) * C)
        dg[s] = np.cumsum(dgam[s][::-1])[::-1]
    out = dict(o=o[:L], hT=hT, dq=dq[:L], dk=dkk[:L], dv=dvv[:L], dg=dg[:L], db=db[:L], dw=dw[:L], dh0=dh)
    if keep:
        out["chunks"] = F
        out["h_c"] = hs
        out["dh_next"] = dhs
    return out


def bwd(q, k, v, g, b, w, dO, *, cu_seqlens, scale=1.0, h0=None, dhT=None, C=64):
    """Same interface and result layout as the token-serial oracle's bwd()."""
    q, k, v, g, b, w, dO = (np.asarray(a, dtype=np.float64) for a in (q, k, v, g, b, w, dO))
    Tt, H, dk = q.shape
    dv = v.shape[-1]
    N = len(cu_seqlens) - 1
    out = dict(o=np.zeros((Tt, H, dv)), hT=np.zeros((N, H, dk, dv)), dq=np.zeros((Tt, H, dk)),
               dk=np.zeros((Tt, H, dk)), dv=np.zeros((Tt, H, dv)), dg=np.zeros((Tt, H)), db=np.zeros((Tt, H)),
               dw=np.zeros((Tt, H)), dh0=np.zeros((N, H, dk, dv)))
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
