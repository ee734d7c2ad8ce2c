"""Pins of the oracle's backward pass: central finite differences of the (separately
pinned) forward, and gradient identities that follow from Eq. 7 in closed form."""
import numpy as np
import pytest

from oracle import lococo_oracle as orc


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def loss(Q, K, V, G, B, PO, PK, PV, bias=None, eps=1e-6):
    O, Kc, Vc, c, _ = orc.process_sequence(Q, K, V, G, B, bias=bias, eps=eps)
    return (PO * O).sum() + (PK * Kc).sum() + (PV * Vc).sum()


def finite_difference(f, x, idx, h=1e-6):
    xp, xm = x.copy(), x.copy()
    xp[idx] += h
    xm[idx] -= h
    return (f(xp) - f(xm)) / (2 * h)


@pytest.mark.parametrize("L,B,M,c_mult,with_bias", [(20, 5, 6, 1, False), (18, 4, 5, 2, True), (12, 12, 4, 1, False),
                                                    (15, 4, 16, 1, False), (17, 5, 7, 2, False)])
def test_gradients_match_finite_differences(L, B, M, c_mult, with_bias):
    r = rng(100 + L + M)
    d, k = 3, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, c_mult * d, k))
    bias = 0.1 * r.standard_normal(M) if with_bias else None
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    dQ, dK, dV, dG, db = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV, bias=bias)
    checks = [("Q", Q, dQ, lambda x: loss(x, K, V, G, B, PO, PK, PV, bias)),
              ("K", K, dK, lambda x: loss(Q, x, V, G, B, PO, PK, PV, bias)),
              ("V", V, dV, lambda x: loss(Q, K, x, G, B, PO, PK, PV, bias)),
              ("G", G, dG, lambda x: loss(Q, K, V, x, B, PO, PK, PV, bias))]
    if with_bias:
        checks.append(("bias", bias, db, lambda x: loss(Q, K, V, G, B, PO, PK, PV, x)))
    for name, x, g, f in checks:
        flat = r.permutation(x.size)[:12]
        for fi in flat:
            idx = np.unravel_index(fi, x.shape)
            fd = finite_difference(f, x, idx)
            assert abs(fd - g[idx]) <= 2e-6 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


def test_weight_gradient_is_orthogonal_to_weights():
    # Eq. 7 is invariant under G -> aG (a > 0) when eps = 0 and there is no bias,
    # so d loss / d a = <G, dG> = 0.
    r = rng(7)
    L, B, M, d, k = 24, 6, 6, 4, 5
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    dQ, dK, dV, dG, _ = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV, eps=0.0)
    assert abs((G * dG).sum()) <= 1e-10 * np.abs(G * dG).sum()
    assert np.abs(dG).max() > 1e-3


def test_short_sequence_gradient_is_attention_gradient():
    # L <= M: no compression happens, so dG = 0 and dQ, dK, dV are those of Eq. 1 on the
    # full sequence (checked against a numpy softmax-attention backward) plus the loss's
    # direct terms on the final cache.
    r = rng(8)
    L, B, M, d, k = 10, 4, 12, 3, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    dQ, dK, dV, dG, _ = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV)
    assert np.all(dG == 0)
    sc = 1 / np.sqrt(d)
    lg = np.where(np.tril(np.ones((L, L), bool)), Q @ K.T * sc, -np.inf)
    P = np.exp(lg - lg.max(1, keepdims=True))
    P /= P.sum(1, keepdims=True)
    dP = PO @ V.T
    dS = P * (dP - (dP * P).sum(1, keepdims=True)) * sc
    np.testing.assert_allclose(dQ, dS @ K, atol=1e-12)
    np.testing.assert_allclose(dK, dS.T @ Q + PK[:L], atol=1e-12)
    np.testing.assert_allclose(dV, P.T @ PO + PV[:L], atol=1e-12)


def test_batch_gradient_sums_shared_weights():
    r = rng(9)
    Bt, H, L, d, M, k, B = 2, 2, 14, 3, 5, 3, 4
    Q, K, V, PO = (r.standard_normal((Bt, H, L, d)) for _ in range(4))
    PK, PV = r.standard_normal((Bt, H, M, d)), r.standard_normal((Bt, H, M, d))
    G = r.standard_normal((1, M, d, k))
    dQ, dK, dV, dG, _ = orc.grad_batch(Q, K, V, G, B, PO, PK, PV)
    acc = np.zeros((M, d, k))
    for bi in range(Bt):
        for h in range(H):
            q, kk, v, g, _ = orc.process_sequence_grad(Q[bi, h], K[bi, h], V[bi, h], G[0], B, PO[bi, h], PK[bi, h],
                                                       PV[bi, h])
            np.testing.assert_allclose(dQ[bi, h], q, atol=1e-13)
            np.testing.assert_allclose(dK[bi, h], kk, atol=1e-13)
            acc += g
    np.testing.assert_allclose(dG[0], acc, atol=1e-12)


def loss_from(cache, Q, K, V, G, B, PO, PK, PV):
    O, Kc, Vc, c, _ = orc.process_sequence(Q, K, V, G, B, cache=cache)
    return (PO * O).sum() + (PK * Kc).sum() + (PV * Vc).sum()


@pytest.mark.parametrize("c0,M,B,L", [(6, 6, 4, 14), (3, 7, 3, 11), (5, 5, 9, 9)])
def test_gradient_with_respect_to_the_initial_cache_matches_finite_differences(c0, M, B, L):
    # the loop started from a given cache (full, or partly filled with fill steps still to come): the cache
    # gradient against central differences of the forward; rows beyond the fill count get no gradient
    r = rng(300 + c0 + M)
    d, k = 3, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    Kc0, Vc0 = r.standard_normal((M, d)), r.standard_normal((M, d))
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    dQ, dK, dV, dG, _, dKc, dVc = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV, cache=(Kc0, Vc0, c0))
    assert np.all(dKc[c0:] == 0) and np.all(dVc[c0:] == 0)
    checks = [("Kc", Kc0, dKc, lambda x: loss_from((x, Vc0, c0), Q, K, V, G, B, PO, PK, PV)),
              ("Vc", Vc0, dVc, lambda x: loss_from((Kc0, x, c0), Q, K, V, G, B, PO, PK, PV)),
              ("K", K, dK, lambda x: loss_from((Kc0, Vc0, c0), Q, x, V, G, B, PO, PK, PV)),
              ("G", G, dG, lambda x: loss_from((Kc0, Vc0, c0), Q, K, V, x, B, PO, PK, PV))]
    for name, x, g, f in checks:
        rows = c0 if name in ("Kc", "Vc") else x.shape[0]
        for fi in r.permutation(rows * x[0].size)[:12]:
            idx = np.unravel_index(fi, (rows,) + x.shape[1:])
            fd = finite_difference(f, x, idx)
            assert abs(fd - g[idx]) <= 2e-6 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


@pytest.mark.parametrize("cut", [8, 10, 16])
def test_backward_over_two_calls_equals_backward_over_one(cut):
    # Algorithm 2 run in two calls (tokens [0, cut) then [cut, L), the cache handed over) and differentiated
    # last call first, the cache gradient handed back: the same gradients as one call over all tokens.
    # cut = 8: on a chunk boundary; 10: the first call ends with a short chunk; 16: two whole chunks each
    r = rng(400 + cut)
    L, B, M, d, k = 32 if cut == 16 else 24, 8, 6, 3, 5
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, 2 * d, k))
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    if cut % B == 0:
        one = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV)
    _, Kc1, Vc1, c1, _ = orc.process_sequence(Q[:cut], K[:cut], V[:cut], G, B)
    q2, k2, v2, g2, _, dKc, dVc = orc.process_sequence_grad(Q[cut:], K[cut:], V[cut:], G, B, PO[cut:], PK, PV,
                                                            cache=(Kc1, Vc1, c1))
    q1, k1, v1, g1, _ = orc.process_sequence_grad(Q[:cut], K[:cut], V[:cut], G, B, PO[:cut], dKc, dVc)
    if cut % B == 0:
        np.testing.assert_allclose(np.concatenate([q1, q2]), one[0], atol=1e-11)
        np.testing.assert_allclose(np.concatenate([k1, k2]), one[1], atol=1e-11)
        np.testing.assert_allclose(np.concatenate([v1, v2]), one[2], atol=1e-11)
        np.testing.assert_allclose(g1 + g2, one[3], atol=1e-10)
    else:
        # the chunking differs from any single call's: check the chained gradient against finite differences
        def f(x):
            _, a, b, c, _ = orc.process_sequence(Q[:cut], x, V[:cut], G, B)
            O2, Kf, Vf, _, _ = orc.process_sequence(Q[cut:], K[cut:], V[cut:], G, B, cache=(a, b, c))
            O1 = orc.process_sequence(Q[:cut], x, V[:cut], G, B)[0]
            return (PO[:cut] * O1).sum() + (PO[cut:] * O2).sum() + (PK * Kf).sum() + (PV * Vf).sum()
        for fi in r.permutation(cut * d)[:10]:
            idx = np.unravel_index(fi, (cut, d))
            fd = finite_difference(f, K[:cut], idx)
            assert abs(fd - k1[idx]) <= 2e-6 * max(1.0, abs(fd)), (idx, fd, k1[idx])
