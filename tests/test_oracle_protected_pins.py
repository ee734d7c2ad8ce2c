"""Pins of the oracle's protected slots (Section 5.2, Table 6: the compressor used next to an
eviction policy that always keeps some tokens): what the reading fixes independently of the
oracle's own arithmetic."""
import numpy as np
import pytest

from oracle import lococo_oracle as orc


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def weights_by_hand(XK, XV, G, eps, protected):
    """Eq. 6 -> ReLU -> Eq. 7 written as index loops, with unit rows for the protected slots."""
    S, d = XK.shape
    M, C, k = G.shape
    p = (k - 1) // 2
    Z = np.concatenate([XK, XV], axis=1)[:, :C]
    w = np.zeros((M, S))
    for i in range(M):
        if i < protected:
            w[i, i] = 1.0
            continue
        for j in range(S):
            a = 0.0
            for t in range(k):
                if 0 <= j + t - p < S:
                    a += float(G[i, :, t] @ Z[j + t - p])
            w[i, j] = max(a, 0.0)
        w[i] /= w[i].sum() + eps
    return w


@pytest.mark.parametrize("c_mult,protected", [(1, 1), (2, 3), (1, 5)])
def test_compress_against_index_loops(c_mult, protected):
    r = rng(40 + protected)
    S, d, M, k = 13, 4, 5, 3
    XK, XV = r.standard_normal((S, d)), r.standard_normal((S, d))
    G = r.standard_normal((M, c_mult * d, k))
    Kn, Vn, w, _, s = orc.compress(XK, XV, G, want_weights=True, protected=protected)
    wh = weights_by_hand(XK, XV, G, 1e-6, protected)
    np.testing.assert_allclose(w, wh, rtol=0, atol=1e-13)
    np.testing.assert_allclose(Kn, wh @ XK, rtol=0, atol=1e-13)
    np.testing.assert_allclose(Vn, wh @ XV, rtol=0, atol=1e-13)
    assert (s[:protected] == 1.0).all()


def test_protected_slots_keep_the_first_tokens_exactly():
    # the first M tokens fill the cache as they are, so slot i < s holds token i from then on,
    # whatever happens to the other slots and however the sequence is cut into chunks
    r = rng(3)
    L, d, M, k, s = 61, 4, 8, 5, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    for B in (1, 4, 7, 20, 61):
        _, Kc, Vc, c, _ = orc.process_sequence(Q, K, V, G, B, protected=s)
        assert c == M
        assert (Kc[:s] == K[:s]).all() and (Vc[:s] == V[:s]).all()
        assert not np.allclose(Kc[s:], K[s:M])


def test_all_slots_protected_is_a_frozen_cache():
    r = rng(4)
    L, d, M, k = 30, 3, 6, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    _, Kc, Vc, _, _ = orc.process_sequence(Q, K, V, G, 5, protected=M)
    assert (Kc == K[:M]).all() and (Vc == V[:M]).all()


def test_one_step_other_rows_are_the_plain_method():
    # the conv reads every entry either way, so in ONE compress step rows i >= s are those of the
    # plain method (pinned elsewhere); zero protected slots is the plain method
    r = rng(5)
    S, d, M, k, s = 19, 4, 6, 5, 2
    XK, XV = r.standard_normal((S, d)), r.standard_normal((S, d))
    G = r.standard_normal((M, 2 * d, k))
    K0, V0 = orc.compress(XK, XV, G)
    K1, V1 = orc.compress(XK, XV, G, protected=s)
    assert (K1[s:] == K0[s:]).all() and (V1[s:] == V0[s:]).all()
    assert (K1[:s] == XK[:s]).all() and (V1[:s] == XV[:s]).all()
    K2, V2 = orc.compress(XK, XV, G, protected=0)
    assert (K2 == K0).all() and (V2 == V0).all()


def test_attention_sees_the_protected_tokens():
    # with every slot protected the model is attention over the first M tokens plus the causal chunk
    r = rng(6)
    L, d, M, k, B = 24, 4, 4, 3, 6
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    O, *_ = orc.process_sequence(Q, K, V, G, B, protected=M)
    scale = 1 / np.sqrt(d)
    for t in (13, 23):
        n0 = (t // B) * B
        keys = list(range(M)) + list(range(n0, t + 1))
        lg = scale * K[keys] @ Q[t]
        p = np.exp(lg - lg.max())
        np.testing.assert_allclose(O[t], (p / p.sum()) @ V[keys], rtol=0, atol=1e-12)


def loss(Q, K, V, G, B, PO, PK, PV, s):
    O, Kc, Vc, _, _ = orc.process_sequence(Q, K, V, G, B, protected=s)
    return (PO * O).sum() + (PK * Kc).sum() + (PV * Vc).sum()


@pytest.mark.parametrize("L,B,M,c_mult,s", [(20, 5, 6, 1, 2), (17, 4, 5, 2, 1), (15, 6, 4, 1, 4)])
def test_gradients_match_finite_differences(L, B, M, c_mult, s):
    r = rng(200 + L + s)
    d, k = 3, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, c_mult * d, k))
    PO, PK, PV = r.standard_normal((L, d)), r.standard_normal((M, d)), r.standard_normal((M, d))
    dQ, dK, dV, dG, _ = orc.process_sequence_grad(Q, K, V, G, B, PO, PK, PV, protected=s)
    assert (dG[:s] == 0).all()          # protected rows have no weights in play
    if s < M:
        assert np.abs(dG[s:]).max() > 1e-4
    checks = [("Q", Q, dQ, lambda x: loss(x, K, V, G, B, PO, PK, PV, s)),
              ("K", K, dK, lambda x: loss(Q, x, V, G, B, PO, PK, PV, s)),
              ("V", V, dV, lambda x: loss(Q, K, x, G, B, PO, PK, PV, s)),
              ("G", G, dG, lambda x: loss(Q, K, V, x, B, PO, PK, PV, s))]
    h = 1e-6
    for name, x, g, f in checks:
        for fi in r.permutation(x.size)[:12]:
            idx = np.unravel_index(fi, x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            fd = (f(xp) - f(xm)) / (2 * h)
            assert abs(fd - g[idx]) <= 2e-6 * max(1.0, abs(fd)), (name, idx, fd, g[idx])
    # the final-cache gradient of a protected slot lands on its token unchanged
    dQ2, dK2, dV2, _, _ = orc.process_sequence_grad(Q, K, V, G, B, 0 * PO, PK, 0 * PV, protected=M)
    np.testing.assert_allclose(dK2[:M], PK, rtol=0, atol=1e-14)
    assert (dK2[M:] == 0).all() and (dV2 == 0).all()
