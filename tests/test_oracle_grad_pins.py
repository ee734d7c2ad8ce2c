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
