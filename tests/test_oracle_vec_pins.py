"""Pins for the per-channel CPU oracle (Eq. 1 with gate vectors): everything here is fixed by the definition,
by mathematics, or by the independently pinned scalar-gate oracle -- never by the CUDA path.  No GPU needed."""
import numpy as np
import pytest

import oracle
from oracle import chunked_vec


def rel(a, b):
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def draw(seed, lengths, H, dk, dv, states=True):
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    Tt, N = int(cu[-1]), len(lengths)
    q = rng.standard_normal((Tt, H, dk)); q /= np.linalg.norm(q, axis=-1, keepdims=True)
    k = rng.standard_normal((Tt, H, dk)); k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((Tt, H, dv))
    dO = rng.standard_normal((Tt, H, dv))
    g = -0.1 * np.logaddexp(0, rng.standard_normal((Tt, H, dk)))
    b = 1 / (1 + np.exp(-rng.standard_normal((Tt, H, dk))))
    w = 1 / (1 + np.exp(-rng.standard_normal((Tt, H, dv))))
    h0 = 0.3 * rng.standard_normal((N, H, dk, dv)) if states else None
    dhT = 0.3 * rng.standard_normal((N, H, dk, dv)) if states else None
    return dict(q=q, k=k, v=v, g=g, b=b, w=w, dO=dO, h0=h0, dhT=dhT, cu=cu)


def run_bwd(x, scale=1.0):
    return oracle.vec_bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=scale,
                          h0=x["h0"], dhT=x["dhT"])


def loss(x, scale):
    o, hT = oracle.vec_fwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], cu_seqlens=x["cu"], scale=scale, h0=x["h0"])
    L = np.sum(o * x["dO"])
    if x["dhT"] is not None:
        L += np.sum(hT * x["dhT"])
    return L


# ---- central finite differences of the scalar loss pin the adjoint to the forward ----
@pytest.mark.parametrize("seed,lengths", [(0, [37]), (1, [5, 70])])
def test_finite_differences(seed, lengths):
    scale = 0.8
    x = draw(seed, lengths, H=2, dk=5, dv=4)
    gr = run_bwd(x, scale)
    rng = np.random.default_rng(99)
    eps = 1e-6
    for name, gname in dict(q="dq", k="dk", v="dv", g="dg", b="db", w="dw", h0="dh0").items():
        flat = x[name].reshape(-1)
        idx = rng.choice(flat.size, size=min(25, flat.size), replace=False)
        num = np.zeros(len(idx)); ana = gr[gname].reshape(-1)[idx]
        for n, i in enumerate(idx):
            old = flat[i]
            flat[i] = old + eps; lp = loss(x, scale)
            flat[i] = old - eps; lm = loss(x, scale)
            flat[i] = old
            num[n] = (lp - lm) / (2 * eps)
        assert rel(ana, num) < 1e-7, (name, rel(ana, num))


# ---- the forward against Eq. 1 written with explicit matrices, token by token ----
def test_forward_is_eq1_in_matrix_form():
    x = draw(3, [9], H=1, dk=6, dv=5)
    scale = 1.3
    o, hT = oracle.vec_fwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], cu_seqlens=x["cu"], scale=scale, h0=x["h0"])
    S = x["h0"][0, 0].copy()
    I = np.eye(6)
    for t in range(9):
        q, k, v, g, b, w = (x[n][t, 0] for n in ("q", "k", "v", "g", "b", "w"))
        # S_t = (I - k (b . k)^T) Diag(e^g) S_{t-1} + k (w . v)^T ;  o_t = S_t^T q_t
        S = (I - np.outer(k, b * k)) @ np.diag(np.exp(g)) @ S + np.outer(k, w * v)
        assert np.allclose(o[t, 0], scale * (S.T @ q), rtol=1e-12, atol=1e-13)
    assert np.allclose(hT[0, 0], S, rtol=1e-12, atol=1e-13)


# ---- b = w = beta reduces Eq. 1 to the KDA row of Table 2 (Section 4.1: pinned at 1e-12) ----
def test_equal_erase_and_write_gate_is_kda():
    x = draw(4, [40], H=2, dk=7, dv=5)
    rng = np.random.default_rng(5)
    beta = 1 / (1 + np.exp(-rng.standard_normal((40, 2))))
    b = np.repeat(beta[:, :, None], 7, axis=2)
    w = np.repeat(beta[:, :, None], 5, axis=2)
    o, hT = oracle.vec_fwd(x["q"], x["k"], x["v"], x["g"], b, w, cu_seqlens=x["cu"], h0=x["h0"])
    for hd in range(2):
        S = x["h0"][0, hd].copy()
        for t in range(40):
            k, v, g, bt = x["k"][t, hd], x["v"][t, hd], x["g"][t, hd], beta[t, hd]
            # KDA: S_t = (I - beta k k^T) Diag(e^g) S_{t-1} + beta k v^T, contracted in this order
            S = np.exp(g)[:, None] * S
            S = S - bt * np.outer(k, k @ S) + bt * np.outer(k, v)
            assert rel(o[t, hd], S.T @ x["q"][t, hd]) < 1e-12
        assert rel(hT[0, hd], S) < 1e-12


# ---- gate vectors with equal entries reproduce the scalar-gate oracle; its gate gradients are channel sums ----
def test_equal_entries_reproduce_the_scalar_oracle():
    x = draw(6, [33, 70], H=2, dk=6, dv=5)
    gs, bs, ws = x["g"][:, :, 0].copy(), x["b"][:, :, 0].copy(), x["w"][:, :, 0].copy()
    x["g"] = np.repeat(gs[:, :, None], 6, axis=2)
    x["b"] = np.repeat(bs[:, :, None], 6, axis=2)
    x["w"] = np.repeat(ws[:, :, None], 5, axis=2)
    vec = run_bwd(x, scale=0.7)
    sca = oracle.bwd(x["q"], x["k"], x["v"], gs, bs, ws, x["dO"], cu_seqlens=x["cu"], scale=0.7, h0=x["h0"], dhT=x["dhT"])
    for name in ("o", "hT", "dq", "dk", "dv", "dh0"):
        assert rel(vec[name], sca[name]) < 1e-13, name
    # Appendix A: the scalar path recovers only channel sums of the gate gradients
    assert rel(vec["dg"].sum(-1), sca["dg"]) < 1e-12
    assert rel(vec["db"].sum(-1), sca["db"]) < 1e-12
    assert rel(vec["dw"].sum(-1), sca["dw"]) < 1e-12


# ---- b = 0, w = 1: gated linear attention with per-channel decay (Table 2, GLA row) as a masked contraction ----
def test_erase_off_is_gated_linear_attention():
    x = draw(7, [50], H=2, dk=7, dv=5, states=False)
    x["b"] = np.zeros_like(x["b"]); x["w"] = np.ones_like(x["w"])
    gr = run_bwd(x)
    for hd in range(2):
        Q, K, V, dO = (x[n][:, hd] for n in ("q", "k", "v", "dO"))
        cs = np.cumsum(x["g"][:, hd], axis=0)                       # [T, dk]
        low = np.tril(np.ones((50, 50), dtype=bool))
        E = np.where(low[:, :, None], np.exp(np.where(low[:, :, None], cs[:, None, :] - cs[None, :, :], 0.0)), 0.0)
        S = np.einsum("tr,sr,tsr->ts", Q, K, E)                     # o_t = sum_{s<=t} (q_t . e^{cs_t - cs_s} . k_s) v_s
        assert np.allclose(gr["o"][:, hd], S @ V, rtol=1e-11, atol=1e-12)
        assert np.allclose(gr["hT"][0, hd], (np.exp(cs[-1][None, :] - cs) * K).T @ V, rtol=1e-11, atol=1e-12)
        dS = np.tril(dO @ V.T)
        assert np.allclose(gr["dv"][:, hd], S.T @ dO, rtol=1e-10, atol=1e-11)
        assert np.allclose(gr["dq"][:, hd], np.einsum("ts,tsr,sr->tr", dS, E, K), rtol=1e-10, atol=1e-11)
        assert np.allclose(gr["dk"][:, hd], np.einsum("ts,tsr,tr->sr", dS, E, Q), rtol=1e-10, atol=1e-11)
        M = np.einsum("ts,tr,sr,tsr->tsr", dS, Q, K, E)             # dL / d(cs_t[r] - cs_s[r])
        dcs = M.sum(1) - M.sum(0)
        assert np.allclose(gr["dg"][:, hd], np.cumsum(dcs[::-1], axis=0)[::-1], rtol=1e-9, atol=1e-10)


# ---- linearity (Euler) identities ----
def test_linearity_identities():
    x = draw(8, [33, 20], H=2, dk=6, dv=5)
    gr = run_bwd(x, scale=0.9)
    L = np.sum(gr["o"] * x["dO"]) + np.sum(gr["hT"] * x["dhT"])
    assert np.isclose(np.sum(gr["dv"] * x["v"]) + np.sum(gr["dh0"] * x["h0"]), L, rtol=1e-11)
    assert np.isclose(np.sum(gr["dq"] * x["q"]), np.sum(gr["o"] * x["dO"]), rtol=1e-11)
    assert np.isclose(np.sum(gr["dw"] * x["w"]) + np.sum(gr["dh0"] * x["h0"]), L, rtol=1e-11)


# ---- chunked formulation == token-serial oracle, independent of the chunk size; b = 0 => T = I ----
@pytest.mark.parametrize("C", [16, 64, 150])
def test_chunked_equals_sequential(C):
    x = draw(9, [150, 64, 1], H=2, dk=8, dv=6)
    a = run_bwd(x, scale=0.7)
    c = chunked_vec.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=0.7,
                        h0=x["h0"], dhT=x["dhT"], C=C)
    for name in a:
        assert rel(c[name], a[name]) < 1e-9, (name, rel(c[name], a[name]))


def test_erase_gate_zero_makes_the_solve_vanish():
    x = draw(10, [64], H=1, dk=8, dv=6)
    r = chunked_vec.chain_bwd(x["q"][:, 0], x["k"][:, 0], x["v"][:, 0], x["g"][:, 0], np.zeros((64, 8)), x["w"][:, 0],
                              x["dO"][:, 0], None, None, keep=True)
    assert np.array_equal(r["chunks"][0]["T"], np.eye(64))
    assert np.array_equal(r["chunks"][0]["W"], np.zeros((64, 8)))


# ---- packing and thread count ----
def test_packing_and_threads():
    x = draw(11, [30, 0, 45], H=2, dk=6, dv=5)
    packed = run_bwd(x)
    for n in range(3):
        a, e = x["cu"][n], x["cu"][n + 1]
        s = slice(a, e)
        one = oracle.vec_bwd(x["q"][s], x["k"][s], x["v"][s], x["g"][s], x["b"][s], x["w"][s], x["dO"][s],
                             cu_seqlens=[0, e - a], h0=x["h0"][n:n + 1], dhT=x["dhT"][n:n + 1], n_threads=1)
        for name in ("dq", "dk", "dv", "dg", "db", "dw", "o"):
            assert np.array_equal(one[name], packed[name][s]), name
        assert np.array_equal(one["dh0"][0], packed["dh0"][n])
    assert np.array_equal(packed["dh0"][1], x["dhT"][1])
