"""Pins for the oracle's expert, combine and backward functions (CPU only)."""
import math

import numpy as np
import pytest

from oracle import c2r_oracle as O
from paper_2504_01337_b200 import inputs as G


def _tiny(seed=0, N=8, d=16, E=4, I=8, K=2, T=2, shared=True):
    X = G.normal(seed, G.S_X, (N, d)).astype(np.float64)
    Wg = G.normal(seed, G.S_WG, (E, d), 0.5).astype(np.float64)
    W1 = G.normal(seed, G.S_W1, (E, I, d), 0.3).astype(np.float64)
    W3 = G.normal(seed, G.S_W3, (E, I, d), 0.3).astype(np.float64)
    W2 = G.normal(seed, G.S_W2, (E, d, I), 0.3).astype(np.float64)
    sh = wsg = None
    if shared:
        sh = tuple(G.normal(seed, s, shp, 0.3).astype(np.float64)
                   for s, shp in ((G.S_WS1, (2 * I, d)), (G.S_WS3, (2 * I, d)), (G.S_WS2, (d, 2 * I))))
        wsg = G.normal(seed, G.S_WSG, (d,), 0.5).astype(np.float64)
    rng = np.random.default_rng(seed)
    I_T = np.stack([rng.permutation([j for j in range(E) if j != i])[:T] for i in range(E)])
    return X, Wg, W1, W3, W2, sh, wsg, I_T, K


def test_dense_swiglu_triple_loop():
    n, d, I = 3, 5, 4
    X = G.normal(1, G.S_X, (n, d)).astype(np.float64)
    W1 = G.normal(1, G.S_W1, (I, d)).astype(np.float64)
    W3 = G.normal(1, G.S_W3, (I, d)).astype(np.float64)
    W2 = G.normal(1, G.S_W2, (d, I)).astype(np.float64)
    Y = np.zeros((n, d))
    for t in range(n):
        h = []
        for i in range(I):
            a = sum(X[t, c] * W1[i, c] for c in range(d))
            b = sum(X[t, c] * W3[i, c] for c in range(d))
            h.append(a / (1.0 + math.exp(-a)) * b)
        for o in range(d):
            Y[t, o] = sum(h[i] * W2[o, i] for i in range(I))
    assert np.allclose(O.dense_swiglu(X, W1, W3, W2)[3], Y, atol=1e-13)
    # E = 1, K = 1 grouped form reduces to the dense MLP
    A, B, H, Yp = O.swiglu_fwd(X, np.array([n]), np.array([0, n]), W1[None], W3[None], W2[None])
    assert np.allclose(Yp, Y, atol=1e-13)


def test_layer_is_weighted_sum_of_selected_experts():
    X, Wg, W1, W3, W2, sh, wsg, I_T, K = _tiny(2)
    for align in (1, 4):
        rank = np.array([2, 0, 3, 1])
        f = O.layer_fwd(X, Wg, W1, W3, W2, I_T, K, expert_rank=rank, row_align=align, shared=sh, wsg=wsg)
        Y = np.zeros_like(X)
        for t in range(X.shape[0]):
            for k in range(K):
                e = f["idx"][t, k]
                Y[t] += f["w"][t, k] * O.dense_swiglu(X[t:t + 1], W1[e], W3[e], W2[e])[3][0]
            Y[t] += 1.0 / (1.0 + math.exp(-float(X[t] @ wsg))) * O.dense_swiglu(X[t:t + 1], *sh)[3][0]
        assert np.allclose(f["Y"], Y, atol=1e-12)
    # identical experts + renormalised weights -> the layer equals that one dense expert
    W1s, W3s, W2s = (np.repeat(w[:1], 4, axis=0) for w in (W1, W3, W2))
    f = O.layer_fwd(X, Wg, W1s, W3s, W2s, I_T, K)
    assert np.allclose(f["Y"], O.dense_swiglu(X, W1[0], W3[0], W2[0])[3], atol=1e-12)


def _loss(params, names, base, Gy, frozen):
    p = dict(base); p.update(dict(zip(names, params)))
    sh = (p["Ws1"], p["Ws3"], p["Ws2"]) if p.get("Ws1") is not None else None
    # routing frozen: evaluate with the recorded selection
    L = O.gate_logits(p["X"], p["Wg"])
    w = O.route_weights(L, frozen["idx"])
    Xp = O.permute(p["X"], frozen["slot_of_row"], frozen["idx"].shape[1])
    Yp = O.swiglu_fwd(Xp, frozen["counts"], frozen["offsets"], p["W1"], p["W3"], p["W2"])[3]
    if sh is not None:
        Ys = O.dense_swiglu(p["X"], *sh)[3]
        Y = O.combine(Yp, w, frozen["row_of_slot"], Ys, p["X"] @ p["wsg"])
    else:
        Y = O.combine(Yp, w, frozen["row_of_slot"])
    return float((Y * Gy).sum())


@pytest.mark.parametrize("shared", [False, True])
def test_backward_matches_central_differences(shared):
    X, Wg, W1, W3, W2, sh, wsg, I_T, K = _tiny(3, shared=shared)
    f = O.layer_fwd(X, Wg, W1, W3, W2, I_T, K, row_align=2, shared=sh, wsg=wsg)
    Gy = G.normal(3, G.S_DY, X.shape).astype(np.float64)
    b = O.layer_bwd(X, Wg, W1, W3, W2, f, Gy, shared=sh, wsg=wsg)
    base = dict(X=X, Wg=Wg, W1=W1, W3=W3, W2=W2, Ws1=None)
    pairs = [("X", "dX"), ("Wg", "dWg"), ("W1", "dW1"), ("W3", "dW3"), ("W2", "dW2")]
    if shared:
        base.update(Ws1=sh[0], Ws3=sh[1], Ws2=sh[2], wsg=wsg)
        pairs += [("Ws1", "dWs1"), ("Ws3", "dWs3"), ("Ws2", "dWs2"), ("wsg", "dwsg")]
    rng = np.random.default_rng(0)
    h = 1e-5
    for name, gname in pairs:
        P0 = base[name]
        g = b[gname]
        assert g.shape == P0.shape
        for _ in range(12):
            pos = tuple(int(rng.integers(0, s)) for s in P0.shape)
            Pp = P0.copy(); Pp[pos] += h
            Pm = P0.copy(); Pm[pos] -= h
            fd = (_loss([Pp], [name], base, Gy, f) - _loss([Pm], [name], base, Gy, f)) / (2 * h)
            assert abs(fd - g[pos]) <= 1e-6 * max(1.0, abs(fd)), (name, pos, fd, g[pos])


def test_wgrad_sums_to_dense_when_experts_share_weights():
    X, Wg, W1, W3, W2, _, _, I_T, K = _tiny(4, shared=False)
    W1s, W3s, W2s = (np.repeat(w[:1], 4, axis=0) for w in (W1, W3, W2))
    f = O.layer_fwd(X, Wg, W1s, W3s, W2s, I_T, K)
    Gy = G.normal(4, G.S_DY, X.shape).astype(np.float64)
    b = O.layer_bwd(X, Wg, W1s, W3s, W2s, f, Gy)
    A, B, H, Y = O.dense_swiglu(X, W1[0], W3[0], W2[0])
    _, d1, d3, d2 = O.dense_swiglu_bwd(X, W1[0], W3[0], W2[0], A, B, Gy)   # weights sum to 1 per token
    assert np.allclose(b["dW1"].sum(axis=0), d1, atol=1e-11)
    assert np.allclose(b["dW3"].sum(axis=0), d3, atol=1e-11)
    assert np.allclose(b["dW2"].sum(axis=0), d2, atol=1e-11)


def test_route_bwd_without_renorm_matches_differences():
    E, K = 6, 2
    L = G.random_logits(5, 5, E).astype(np.float64)
    idx, w = O.topk_route(L, K, renorm=False)
    dw = G.normal(5, G.S_DY, (5, K)).astype(np.float64)
    dL = O.route_bwd(idx, w, dw, E, renorm=False, L=L)
    h = 1e-6
    for t in range(5):
        for e in range(E):
            Lp = L.copy(); Lp[t, e] += h
            Lm = L.copy(); Lm[t, e] -= h
            fd = ((O.route_weights(Lp, idx, False) - O.route_weights(Lm, idx, False)) * dw).sum() / (2 * h)
            assert abs(fd - dL[t, e]) < 1e-8
