"""Pins for the CPU oracle: everything here is fixed by the definition (Eq. 1) or by mathematics,
never by the oracle itself and never by the CUDA path.  No GPU needed."""
import numpy as np
import pytest

import oracle
from oracle import chunked


def rel(a, b):
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def draw(seed, lengths, H, dk, dv, states=True, unit_k=True):
    rng = np.random.default_rng(seed)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    Tt, N = int(cu[-1]), len(lengths)
    q = rng.standard_normal((Tt, H, dk))
    k = rng.standard_normal((Tt, H, dk))
    if unit_k:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
    v = rng.standard_normal((Tt, H, dv))
    dO = rng.standard_normal((Tt, H, dv))
    g = -0.1 * np.logaddexp(0, rng.standard_normal((Tt, H)))
    b = 1 / (1 + np.exp(-rng.standard_normal((Tt, H))))
    w = 1 / (1 + np.exp(-rng.standard_normal((Tt, H))))
    h0 = 0.3 * rng.standard_normal((N, H, dk, dv)) if states else None
    dhT = 0.3 * rng.standard_normal((N, H, dk, dv)) if states else None
    return dict(q=q, k=k, v=v, g=g, b=b, w=w, dO=dO, h0=h0, dhT=dhT, cu=cu)


def loss(x, scale):
    o, hT = oracle.fwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], cu_seqlens=x["cu"], scale=scale, h0=x["h0"])
    L = np.sum(o * x["dO"])
    if x["dhT"] is not None:
        L += np.sum(hT * x["dhT"])
    return L


# ---- P1: central finite differences of the scalar loss pin the adjoint to the forward ----
@pytest.mark.parametrize("seed,lengths", [(0, [37]), (1, [5, 70])])
def test_finite_differences(seed, lengths):
    scale = 0.8
    x = draw(seed, lengths, H=2, dk=5, dv=4)
    gr = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=scale,
                    h0=x["h0"], dhT=x["dhT"])
    rng = np.random.default_rng(99)
    eps = 1e-6
    names = dict(q="dq", k="dk", v="dv", g="dg", b="db", w="dw", h0="dh0")
    for name, gname in names.items():
        a = x[name]
        flat = a.reshape(-1)
        idx = rng.choice(flat.size, size=min(25, flat.size), replace=False)
        num = np.zeros(len(idx)); ana = gr[gname].reshape(-1)[idx]
        for n, i in enumerate(idx):
            old = flat[i]
            flat[i] = old + eps; lp = loss(x, scale)
            flat[i] = old - eps; lm = loss(x, scale)
            flat[i] = old
            num[n] = (lp - lm) / (2 * eps)
        assert rel(ana, num) < 1e-7, (name, rel(ana, num))


# ---- P2: one token, closed form from Eq. 1 ----
def test_single_token_closed_form():
    x = draw(3, [1], H=1, dk=6, dv=5)
    scale = 1.3
    o, hT = oracle.fwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], cu_seqlens=x["cu"], scale=scale, h0=x["h0"])
    q, k, v, h0 = x["q"][0, 0], x["k"][0, 0], x["v"][0, 0], x["h0"][0, 0]
    a, b, w = np.exp(x["g"][0, 0]), x["b"][0, 0], x["w"][0, 0]
    # S_1 = (I - b k k^T) a S_0 + k (w v)^T ;  o = S_1^T q
    S1 = (np.eye(6) - b * np.outer(k, k)) @ (a * h0) + np.outer(k, w * v)
    assert np.allclose(hT[0, 0], S1, rtol=1e-13, atol=1e-14)
    assert np.allclose(o[0, 0], scale * (S1.T @ q), rtol=1e-13, atol=1e-14)
    # the expanded form: o = scale [a h0^T q + (k.q)(w v - a b h0^T k)]
    o2 = scale * (a * h0.T @ q + (k @ q) * (w * v - a * b * (h0.T @ k)))
    assert np.allclose(o[0, 0], o2, rtol=1e-13, atol=1e-14)


# ---- P3: erase gate off, write gate one => (gated) linear attention as one masked matrix product ----
@pytest.mark.parametrize("gated", [True, False])
def test_reduces_to_linear_attention(gated):
    x = draw(4, [50], H=2, dk=7, dv=5, states=False)
    Tt = 50
    x["b"] = np.zeros_like(x["b"]); x["w"] = np.ones_like(x["w"])
    if not gated:
        x["g"] = np.zeros_like(x["g"])
    o, hT = oracle.fwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], cu_seqlens=x["cu"])
    for hd in range(2):
        cs = np.cumsum(x["g"][:, hd])
        Dfull = np.tril(np.exp(cs[:, None] - cs[None, :]))     # exp(sum_{s<r<=t} g_r), diagonal = 1
        ref = ((x["q"][:, hd] @ x["k"][:, hd].T) * Dfull) @ x["v"][:, hd]
        assert np.allclose(o[:, hd], ref, rtol=1e-12, atol=1e-13)
        refS = (x["k"][:, hd] * np.exp(cs[-1] - cs)[:, None]).T @ x["v"][:, hd]
        assert np.allclose(hT[0, hd], refS, rtol=1e-12, atol=1e-13)
    # and the gradients of that masked product, by the textbook matmul rules
    gr = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"])
    for hd in range(2):
        cs = np.cumsum(x["g"][:, hd])
        Dfull = np.tril(np.exp(cs[:, None] - cs[None, :]))
        Q, K, V, dO = x["q"][:, hd], x["k"][:, hd], x["v"][:, hd], x["dO"][:, hd]
        S = (Q @ K.T) * Dfull
        dS = (dO @ V.T) * Dfull
        assert np.allclose(gr["dv"][:, hd], S.T @ dO, rtol=1e-11, atol=1e-12)
        assert np.allclose(gr["dq"][:, hd], dS @ K, rtol=1e-11, atol=1e-12)
        assert np.allclose(gr["dk"][:, hd], dS.T @ Q, rtol=1e-11, atol=1e-12)
        if gated:
            M = (dO @ V.T) * S                    # dL/d(log D_ts) for t >= s
            dcs = M.sum(1) - M.sum(0)             # D_ts = exp(cs_t - cs_s)
            dg = np.cumsum(dcs[::-1])[::-1]
            assert np.allclose(gr["dg"][:, hd], dg, rtol=1e-10, atol=1e-11)


# ---- P4: delta-rule write invariant ----
def test_delta_rule_stores_the_value():
    x = draw(5, [40], H=1, dk=8, dv=6)
    x["b"] = np.ones_like(x["b"]); x["w"] = np.ones_like(x["w"])
    for t in range(1, 41):   # after writing token t with unit key and b = w = 1, h_t^T k_t = v_t
        o, hT = oracle.fwd(x["q"][:t], x["k"][:t], x["v"][:t], x["g"][:t], x["b"][:t], x["w"][:t],
                           cu_seqlens=np.array([0, t], dtype=np.int32), h0=x["h0"])
        assert np.allclose(hT[0, 0].T @ x["k"][t - 1, 0], x["v"][t - 1, 0], rtol=1e-11, atol=1e-12)


def test_orthonormal_keys_are_recalled_exactly():
    rng = np.random.default_rng(6)
    dk, dv, T = 8, 5, 8
    Kmat, _ = np.linalg.qr(rng.standard_normal((dk, dk)))
    k = Kmat.T[:T, None, :].copy()
    v = rng.standard_normal((T, 1, dv))
    z = np.zeros((T, 1)); one = np.ones((T, 1))
    for s in range(T):
        q = np.repeat(k[s][None], T, axis=0)
        o, _ = oracle.fwd(q, k, v, z, one, one, cu_seqlens=np.array([0, T], dtype=np.int32))
        assert np.allclose(o[T - 1, 0], v[s, 0], atol=1e-12)


# ---- P5: linearity (Euler) identities, no differencing ----
def test_linearity_identities():
    x = draw(7, [33, 20], H=2, dk=6, dv=5)
    scale = 0.9
    gr = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=scale,
                    h0=x["h0"], dhT=x["dhT"])
    L = np.sum(gr["o"] * x["dO"]) + np.sum(gr["hT"] * x["dhT"])
    # L is jointly linear in (v, h0)
    assert np.isclose(np.sum(gr["dv"] * x["v"]) + np.sum(gr["dh0"] * x["h0"]), L, rtol=1e-11)
    # o is linear in q
    assert np.isclose(np.sum(gr["dq"] * x["q"]), np.sum(gr["o"] * x["dO"]), rtol=1e-11)
    # L is linear in the write gate w jointly with h0:  <dw, w> + <dh0, h0> = L
    assert np.isclose(np.sum(gr["dw"] * x["w"]) + np.sum(gr["dh0"] * x["h0"]), L, rtol=1e-11)


# ---- P6: chunked formulation == token-serial oracle, independent of the chunk size; b = 0 => T = I ----
@pytest.mark.parametrize("C", [16, 32, 64, 150])
def test_chunked_equals_sequential(C):
    x = draw(8, [150, 64, 1], H=2, dk=8, dv=6)
    a = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=0.7,
                   h0=x["h0"], dhT=x["dhT"])
    c = chunked.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], scale=0.7,
                    h0=x["h0"], dhT=x["dhT"], C=C)
    for name in a:
        assert rel(c[name], a[name]) < 1e-9, (name, rel(c[name], a[name]))


def test_erase_gate_zero_makes_the_solve_vanish():
    x = draw(9, [64], H=1, dk=8, dv=6)
    r = chunked.chain_bwd(x["q"][:, 0], x["k"][:, 0], x["v"][:, 0], x["g"][:, 0], np.zeros(64), x["w"][:, 0],
                          x["dO"][:, 0], None, None, keep=True)
    assert np.array_equal(r["chunks"][0]["T"], np.eye(64))      # bitwise: M = 0 => T = I
    assert np.array_equal(r["chunks"][0]["W"], np.zeros((64, 8)))


def test_short_form_of_the_triangular_solve_vjp():
    """The kernels take K#2 in a shorter form than its definition (dW = -dU h^T, dXk = T^T dW, dXv = T^T dU,
    dA = -stril(dXk W^T + dXv U~^T)): dXk = -dXv h^T and dA = -stril(dXv U^T) with U = U~ - W h.  Checked here on the
    intermediates of the chunkwise rung, which follows the definition and is itself pinned to the token-serial oracle."""
    x = draw(12, [200], H=1, dk=8, dv=6)
    r = chunked.chain_bwd(x["q"][:, 0], x["k"][:, 0], x["v"][:, 0], x["g"][:, 0], x["b"][:, 0], x["w"][:, 0], x["dO"][:, 0],
                          x["h0"][0, 0], x["dhT"][0, 0], scale=0.7, keep=True)
    assert len(r["chunks"]) == 4
    for f, h in zip(r["chunks"], r["h_c"]):
        assert np.linalg.norm(f["dXk"]) > 0 and np.linalg.norm(f["dA"]) > 0
        assert rel(-f["dXv"] @ h.T, f["dXk"]) < 1e-12
        assert rel(-np.tril(f["dXv"] @ f["U"].T, -1), f["dA"]) < 1e-12


# ---- P7: split and packing consistency ----
def test_split_consistency():
    x = draw(10, [90], H=2, dk=6, dv=5)
    args = lambda s: (x["q"][s], x["k"][s], x["v"][s], x["g"][s], x["b"][s], x["w"][s], x["dO"][s])
    full = oracle.bwd(*args(slice(0, 90)), cu_seqlens=[0, 90], h0=x["h0"], dhT=x["dhT"])
    T1 = 41
    first_f = oracle.fwd(*args(slice(0, T1))[:6], cu_seqlens=[0, T1], h0=x["h0"])
    second = oracle.bwd(*args(slice(T1, 90)), cu_seqlens=[0, 90 - T1], h0=first_f[1], dhT=x["dhT"])
    first = oracle.bwd(*args(slice(0, T1)), cu_seqlens=[0, T1], h0=x["h0"], dhT=second["dh0"])
    for name in ("dq", "dk", "dv", "dg", "db", "dw", "o"):
        joined = np.concatenate([first[name], second[name]])
        assert rel(joined, full[name]) < 1e-12, name
    assert rel(first["dh0"], full["dh0"]) < 1e-12
    assert rel(second["hT"], full["hT"]) < 1e-12


def test_packing_equals_separate_calls():
    x = draw(11, [30, 0, 45], H=2, dk=6, dv=5)
    packed = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"],
                        h0=x["h0"], dhT=x["dhT"])
    for n in range(3):
        a, e = x["cu"][n], x["cu"][n + 1]
        s = slice(a, e)
        one = oracle.bwd(x["q"][s], x["k"][s], x["v"][s], x["g"][s], x["b"][s], x["w"][s], x["dO"][s],
                         cu_seqlens=[0, e - a], h0=x["h0"][n:n + 1], dhT=x["dhT"][n:n + 1])
        for name in ("dq", "dk", "dv", "dg", "db", "dw", "o"):
            assert np.array_equal(one[name], packed[name][s]), name
        assert np.array_equal(one["dh0"][0], packed["dh0"][n])
    # an empty sequence passes its terminal gradient straight through
    assert np.array_equal(packed["dh0"][1], x["dhT"][1])
    assert np.array_equal(packed["hT"][1], x["h0"][1])


# ---- P8: identity padding (g = 0, b = w = 0, q = k = v = dO = 0) changes nothing ----
def test_padding_equivalence():
    x = draw(12, [50], H=1, dk=6, dv=5)
    pad = 14
    z = lambda a: np.concatenate([a, np.zeros((pad,) + a.shape[1:])])
    a = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=[0, 50], h0=x["h0"], dhT=x["dhT"])
    p = oracle.bwd(z(x["q"]), z(x["k"]), z(x["v"]), z(x["g"]), z(x["b"]), z(x["w"]), z(x["dO"]), cu_seqlens=[0, 64],
                   h0=x["h0"], dhT=x["dhT"])
    for name in ("dq", "dk", "dv", "dg", "db", "dw"):
        assert rel(p[name][:50], a[name]) < 1e-13, name
    assert rel(p["dh0"], a["dh0"]) < 1e-13


# ---- P9: degenerate cases ----
def test_degenerate_cases():
    x = draw(13, [70], H=2, dk=6, dv=5)
    z = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], np.zeros_like(x["dO"]), cu_seqlens=x["cu"], h0=x["h0"])
    for name in ("dq", "dk", "dv", "dg", "db", "dw", "dh0"):
        assert not np.any(z[name]), name
    o, hT = oracle.fwd(x["q"], x["k"], x["v"], x["g"], np.zeros_like(x["b"]), np.zeros_like(x["w"]), cu_seqlens=x["cu"])
    assert not np.any(o) and not np.any(hT)            # nothing is ever written
    o, hT = oracle.fwd(x["q"], x["k"], np.zeros_like(x["v"]), x["g"], x["b"], x["w"], cu_seqlens=x["cu"])
    assert not np.any(o) and not np.any(hT)


def test_threads_do_not_change_the_result():
    x = draw(14, [40, 41, 42], H=3, dk=6, dv=5)
    a = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], h0=x["h0"], dhT=x["dhT"], n_threads=1)
    b = oracle.bwd(x["q"], x["k"], x["v"], x["g"], x["b"], x["w"], x["dO"], cu_seqlens=x["cu"], h0=x["h0"], dhT=x["dhT"], n_threads=7)
    for name in a:
        assert np.array_equal(a[name], b[name]), name


# ---- the workload wrapper every GPU parity test goes through: its gate mapping and dbeta = db + dw ----
def _tiny_workload(delta_rule, seed):
    from paper_2608_12700_b200 import synth
    return synth.make_workload("pin_wrapper", dtype="f32", lengths=[23, 70], H=2, d_k=6, d_v=5, seed=seed,
                               delta_rule=delta_rule, states=True, scale=0.7)


def _workload_loss(wl, beta):
    """L as a function of beta itself: one array feeds both the erase and the write gate (Table 2, GDN row)."""
    o, hT = oracle.fwd(wl.q, wl.k, wl.v, wl.g, beta, beta, cu_seqlens=wl.cu_seqlens, scale=wl.scale, h0=wl.h0)
    return np.sum(o * wl.dO.astype(np.float64)) + np.sum(hT * wl.dhT.astype(np.float64))


def test_workload_wrapper_dbeta_is_the_derivative_with_respect_to_beta():
    wl = _tiny_workload(1, seed=70)
    out = oracle.bwd_workload(wl)
    beta = wl.beta.astype(np.float64)
    rng = np.random.default_rng(71)
    idx = rng.choice(beta.size, size=40, replace=False)
    eps = 1e-6
    num = np.zeros(len(idx))
    for n, i in enumerate(idx):
        bp = beta.copy().reshape(-1); bm = beta.copy().reshape(-1)
        bp[i] += eps; bm[i] -= eps
        num[n] = (_workload_loss(wl, bp.reshape(beta.shape)) - _workload_loss(wl, bm.reshape(beta.shape))) / (2 * eps)
    assert rel(out["dbeta"].reshape(-1)[idx], num) < 1e-7
    # and it is not the gradient of either gate alone
    assert rel(out["db"].reshape(-1)[idx], num) > 1e-2 and rel(out["dw"].reshape(-1)[idx], num) > 1e-2


def test_workload_wrapper_delta_rule_off_is_erase_zero_write_one():
    wl = _tiny_workload(0, seed=72)
    out = oracle.bwd_workload(wl)
    assert "dbeta" not in out
    zero, one = np.zeros_like(wl.g, dtype=np.float64), np.ones_like(wl.g, dtype=np.float64)
    direct = oracle.bwd(wl.q, wl.k, wl.v, wl.g, zero, one, wl.dO, cu_seqlens=wl.cu_seqlens, scale=wl.scale,
                        h0=wl.h0, dhT=wl.dhT)
    for n in ("o", "hT", "dq", "dk", "dv", "dg", "dh0"):
        assert np.array_equal(out[n], direct[n]), n
    # the same thing as one masked matrix product per (sequence, head) (Table 2, the scalar-decay row):
    # o = scale [ (Q K^T . D) V + Diag(Gam) Q h0 ],  D_ts = exp(cs_t - cs_s) for s <= t, Gam_t = exp(cs_t)
    cu = wl.cu_seqlens
    for n in range(wl.N):
        s = slice(cu[n], cu[n + 1])
        for hd in range(wl.H):
            Q, K, V = (a[s, hd].astype(np.float64) for a in (wl.q, wl.k, wl.v))
            dO = wl.dO[s, hd].astype(np.float64)
            cs = np.cumsum(wl.g[s, hd].astype(np.float64))
            Dm = np.tril(np.exp(cs[:, None] - cs[None, :]))
            h0 = wl.h0[n, hd].astype(np.float64)
            S = (Q @ K.T) * Dm
            o = wl.scale * (S @ V + np.exp(cs)[:, None] * (Q @ h0))
            assert np.allclose(out["o"][s, hd], o, rtol=1e-11, atol=1e-12)
            # textbook gradient of that product with respect to V, plus the path through the final state
            e = np.exp(cs[-1] - cs)
            dv = wl.scale * (S.T @ dO) + e[:, None] * (K @ wl.dhT[n, hd].astype(np.float64))
            assert np.allclose(out["dv"][s, hd], dv, rtol=1e-10, atol=1e-11)
