"""Pins of the float64 CPU oracle against things other than itself: textbook
library routines, hand-worked fixtures, closed forms and invariants that the
paper's equations fix.  CPU only."""
import json
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

from oracle import lococo_oracle as orc

GOLDEN = Path(__file__).resolve().parent / "golden"


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


# ----------------------------------------------------------------------------- Eq. 6
def correlate_reference(Z, G, bias=None):
    """Eq. 6 through numpy's textbook 1-D correlation, one (out, in) channel pair at a time."""
    S, C = Z.shape
    M, _, k = G.shape
    p = (k - 1) // 2
    A = np.zeros((M, S))
    for i in range(M):
        for ch in range(C):
            zp = np.concatenate([np.zeros(p), Z[:, ch], np.zeros(p)])
            A[i] += np.correlate(zp, G[i, ch], mode="valid")
        if bias is not None:
            A[i] += bias[i]
    return A


@pytest.mark.parametrize("S,C,M,k", [(7, 3, 4, 3), (32, 8, 5, 5), (13, 2, 3, 21), (40, 6, 7, 1)])
def test_conv_is_textbook_correlation(S, C, M, k):
    r = rng(S * 100 + k)
    Z, G, bias = r.standard_normal((S, C)), r.standard_normal((M, C, k)), r.standard_normal(M)
    np.testing.assert_allclose(orc.conv_logits(Z, G), correlate_reference(Z, G), atol=1e-12)
    np.testing.assert_allclose(orc.conv_logits(Z, G, bias), correlate_reference(Z, G, bias), atol=1e-12)


def test_conv_matches_scipy_correlate():
    from scipy.signal import correlate
    r = rng(5)
    Z, G = r.standard_normal((19, 4)), r.standard_normal((3, 4, 7))
    A = orc.conv_logits(Z, G)
    for i in range(3):
        ref = sum(correlate(Z[:, ch], G[i, ch], mode="same") for ch in range(4))
        np.testing.assert_allclose(A[i], ref, atol=1e-12)


def test_conv_shift_equivariance_away_from_borders():
    # Stationarity (Section 3.2.1): logits of a shifted input are the shifted logits.
    r = rng(11)
    S, C, M, k, sh = 60, 3, 4, 9, 7
    p = (k - 1) // 2
    Z, G = r.standard_normal((S, C)), r.standard_normal((M, C, k))
    Zs = np.roll(Z, sh, axis=0)
    A, As = orc.conv_logits(Z, G), orc.conv_logits(Zs, G)
    lo, hi = p, S - p - sh
    np.testing.assert_allclose(As[:, lo + sh:hi + sh], A[:, lo:hi], atol=1e-12)


# ----------------------------------------------------------------------------- worked fixtures
def test_compress_worked_example():
    fx = json.loads((GOLDEN / "compress_worked.json").read_text())
    XK, XV, G = np.array(fx["XK"]), np.array(fx["XV"]), np.array(fx["G"])
    Kn, Vn, w, A, s = orc.compress(XK, XV, G, eps=0.0, want_weights=True)
    np.testing.assert_allclose(A, np.array(fx["A"]), atol=1e-15)
    w_exp = np.array([[float(Fraction(n, fx["w_den"][i])) for n in row] for i, row in enumerate(fx["w_num"])])
    np.testing.assert_allclose(w, w_exp, atol=1e-15)
    np.testing.assert_allclose(Kn[:, 0], [float(Fraction(n, d)) for n, d in zip(fx["K_new_num"], fx["K_new_den"])],
                               atol=1e-15)
    np.testing.assert_allclose(Vn[:, 0], [float(Fraction(n, d)) for n, d in zip(fx["V_new_num"], fx["V_new_den"])],
                               atol=1e-15)


def test_attention_worked_example():
    fx = json.loads((GOLDEN / "attention_worked.json").read_text())
    Q, XV = np.array(fx["Q"]), np.array(fx["XV"])
    XK = np.log(np.array(fx["XK_exp"]))[:, None]
    O, lse = orc.attention(Q, XK, XV, fx["c"], scale=1.0)
    np.testing.assert_allclose(O[:, 0], [float(Fraction(n, d)) for n, d in zip(fx["O_num"], fx["O_den"])], atol=1e-14)
    np.testing.assert_allclose(lse, np.log(np.array(fx["lse_exp"])), atol=1e-14)


# ----------------------------------------------------------------------------- Eq. 7, Eq. 4-5 invariants
@pytest.mark.parametrize("c_mult", [1, 2])
def test_weights_normalised_nonnegative_and_hull(c_mult):
    r = rng(21 + c_mult)
    S, d, M, k = 23, 6, 5, 5
    XK, XV = r.standard_normal((S, d)), r.standard_normal((S, d))
    G = r.standard_normal((M, c_mult * d, k))
    Kn, Vn, w, A, s = orc.compress(XK, XV, G, eps=0.0, want_weights=True)
    assert (w >= 0).all()
    np.testing.assert_allclose(w.sum(1), 1.0, atol=1e-13)
    # a convex combination stays inside the per-channel hull of its inputs
    assert (Kn <= XK.max(0) + 1e-12).all() and (Kn >= XK.min(0) - 1e-12).all()
    assert (Vn <= XV.max(0) + 1e-12).all() and (Vn >= XV.min(0) - 1e-12).all()
    # Eq. 4 / Eq. 5 as plain matrix products with the returned weights
    np.testing.assert_allclose(Kn, w @ XK, atol=1e-13)
    np.testing.assert_allclose(Vn, w @ XV, atol=1e-13)
    # Eq. 7 from the returned logits
    R = np.maximum(A, 0)
    np.testing.assert_allclose(w, R / R.sum(1, keepdims=True), atol=1e-13)


def test_eps_enters_denominator_only():
    r = rng(3)
    XK, XV, G = r.standard_normal((9, 4)), r.standard_normal((9, 4)), r.standard_normal((3, 4, 3))
    eps = 0.5
    _, _, w, A, s = orc.compress(XK, XV, G, eps=eps, want_weights=True)
    R = np.maximum(A, 0)
    np.testing.assert_allclose(s, R.sum(1) + eps, atol=1e-14)
    np.testing.assert_allclose(w.sum(1), 1 - eps / s, atol=1e-14)


def test_dead_row_gives_zero_slot():
    # all logits of a row <= 0: ReLU kills the row, the eps keeps the division finite
    XK = np.abs(rng(4).standard_normal((8, 3)))
    XV = rng(5).standard_normal((8, 3))
    G = -np.abs(rng(6).standard_normal((2, 3, 3)))
    Kn, Vn = orc.compress(XK, XV, G, eps=1e-6)
    assert np.all(Kn == 0) and np.all(Vn == 0)


def test_shared_weights_for_keys_and_values():
    # Eq. 4 and Eq. 5 use the same w: with keys-only conv input, swapping the value
    # buffer changes only the value slots, and V'=w@XV for any XV
    r = rng(8)
    XK, XV, XV2 = r.standard_normal((12, 4)), r.standard_normal((12, 4)), r.standard_normal((12, 4))
    G = r.standard_normal((3, 4, 5))
    K1, V1, w1, _, _ = orc.compress(XK, XV, G, want_weights=True)
    K2, V2, w2, _, _ = orc.compress(XK, XV2, G, want_weights=True)
    np.testing.assert_array_equal(K1, K2)
    np.testing.assert_array_equal(w1, w2)
    np.testing.assert_allclose(V2, w1 @ XV2, atol=1e-13)


def test_scale_invariances_closed_form():
    r = rng(9)
    S, d, M, k = 17, 5, 4, 7
    XK, XV, G = r.standard_normal((S, d)), r.standard_normal((S, d)), r.standard_normal((M, d, k))
    K0, V0, w0, _, _ = orc.compress(XK, XV, G, eps=0.0, want_weights=True)
    K1, V1, w1, _, _ = orc.compress(XK, XV, 3.7 * G, eps=0.0, want_weights=True)
    np.testing.assert_allclose(w1, w0, atol=1e-13)          # G -> aG leaves w unchanged
    K2, V2, w2, _, _ = orc.compress(2.5 * XK, XV, G, eps=0.0, want_weights=True)
    np.testing.assert_allclose(w2, w0, atol=1e-13)          # K -> aK leaves w unchanged (keys-only input)
    np.testing.assert_allclose(K2, 2.5 * K0, atol=1e-12)
    K3, V3 = orc.compress(XK, -1.5 * XV, G, eps=0.0)
    np.testing.assert_allclose(V3, -1.5 * V0, atol=1e-12)
    np.testing.assert_allclose(K3, K0, atol=1e-13)


# ----------------------------------------------------------------------------- token dropping, averaging
@pytest.mark.parametrize("c_mult", [1, 2])
def test_one_hot_kernels_reduce_to_gather(c_mult):
    # Token dropping is a special case of the compression operator (Section 3.2.3):
    # indicator channels + one-hot kernels make R a 0/1 selection matrix.
    r = rng(31)
    S, d, M, k = 20, 8, 6, 5
    p = (k - 1) // 2
    C = c_mult * d
    XK, XV = r.standard_normal((S, d)), r.standard_normal((S, d))
    pairs = [(ch, t) for ch in range(C) for t in range(k)]
    pick = r.permutation(len(pairs))[:M]
    G = np.zeros((M, C, k))
    expect = []
    used_ch = {}
    # one indicator channel per slot; distinct channels so that indicators do not interfere
    chans = r.permutation(C)[:M]
    for i in range(M):
        ch, t = int(chans[i]), int(pairs[pick[i]][1])
        pos = int(r.integers(p, S - p))          # indicator position pi(i)
        col = np.zeros(S)
        col[pos] = 1.0
        if ch < d:
            XK[:, ch] = col
        else:
            XV[:, ch - d] = col
        G[i, ch, t] = 1.0
        expect.append(pos - (t - p))              # R[i,j] = 1 iff j + t - p = pos
    Kn, Vn, w, _, _ = orc.compress(XK, XV, G, eps=0.0, want_weights=True)
    sel = np.zeros((M, S))
    sel[np.arange(M), expect] = 1.0
    np.testing.assert_array_equal(w, sel)
    np.testing.assert_array_equal(Kn, XK[expect])
    np.testing.assert_array_equal(Vn, XV[expect])


def test_uniform_weights_give_the_mean():
    # a channel that is constant 1 and a centre-tap one-hot kernel give R = 1 everywhere
    r = rng(32)
    S, d, M, k = 15, 4, 3, 5
    XK, XV = r.standard_normal((S, d)), r.standard_normal((S, d))
    XK[:, 2] = 1.0
    G = np.zeros((M, d, k))
    G[:, 2, (k - 1) // 2] = 1.0
    Kn, Vn = orc.compress(XK, XV, G, eps=0.0)
    np.testing.assert_allclose(Kn, np.tile(XK.mean(0), (M, 1)), atol=1e-14)
    np.testing.assert_allclose(Vn, np.tile(XV.mean(0), (M, 1)), atol=1e-14)


def test_parameter_count_of_the_paper():
    # Section 4.1: 22 million added parameters for 32 layers, 256-dimensional KV states,
    # memory size 128, kernel 21 => weights [M, 2d, k] per layer, shared by the heads.
    layers, d, M, k = 32, 128, 128, 21
    assert layers * M * (2 * d) * k == 22_020_096


# ----------------------------------------------------------------------------- Eq. 1 / Algorithm 1, 2
def full_causal_attention(Q, K, V, scale):
    """Eq. 1 for a whole sequence with numpy matrix ops."""
    L = Q.shape[0]
    logits = (Q @ K.T) * scale
    logits = np.where(np.tril(np.ones((L, L), dtype=bool)), logits, -np.inf)
    logits -= logits.max(1, keepdims=True)
    P = np.exp(logits)
    P /= P.sum(1, keepdims=True)
    return P @ V


@pytest.mark.parametrize("B", [1, 3, 8, 24, 50])
def test_short_sequence_is_exact_full_attention(B):
    # L <= M: only the fill branch of Algorithm 2 runs, which is Algorithm 1, which is Eq. 1.
    r = rng(41)
    L, d, M, k = 24, 8, 24, 5
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    O, Kc, Vc, c, lse = orc.process_sequence(Q, K, V, G, B)
    np.testing.assert_allclose(O, full_causal_attention(Q, K, V, 1 / np.sqrt(d)), atol=1e-12)
    assert c == L
    np.testing.assert_array_equal(Kc[:L], K)
    np.testing.assert_array_equal(Vc[:L], V)


def test_single_token_chunks_equal_single_query_attention():
    # B = 1 is autoregressive decoding (Section 3.1)
    r = rng(42)
    c, d = 9, 4
    XK, XV = r.standard_normal((c + 1, d)), r.standard_normal((c + 1, d))
    q = r.standard_normal((1, d))
    O, lse = orc.attention(q, XK, XV, c)
    logits = (XK @ q[0]) / np.sqrt(d)
    pr = np.exp(logits - logits.max())
    pr /= pr.sum()
    np.testing.assert_allclose(O[0], pr @ XV, atol=1e-13)
    np.testing.assert_allclose(lse[0], np.log(np.exp(logits).sum()), atol=1e-13)


def test_attention_cache_permutation_invariance():
    r = rng(43)
    c, b, d = 7, 5, 4
    Q, XK, XV = r.standard_normal((b, d)), r.standard_normal((c + b, d)), r.standard_normal((c + b, d))
    perm = np.concatenate([r.permutation(c), np.arange(c, c + b)])
    O1, l1 = orc.attention(Q, XK, XV, c)
    O2, l2 = orc.attention(Q, XK[perm], XV[perm], c)
    np.testing.assert_allclose(O1, O2, atol=1e-13)
    np.testing.assert_allclose(l1, l2, atol=1e-13)


def test_attention_mask_blocks_future_chunk_tokens():
    r = rng(44)
    c, b, d = 3, 6, 4
    Q, XK, XV = r.standard_normal((b, d)), r.standard_normal((c + b, d)), r.standard_normal((c + b, d))
    O1, _, P = orc.attention(Q, XK, XV, c, want_prob=True)
    for q in range(b):
        assert np.all(P[q, c + q + 1:] == 0) and np.all(P[q, :c + q + 1] > 0)
        np.testing.assert_allclose(P[q].sum(), 1.0, atol=1e-13)
    XK2, XV2 = XK.copy(), XV.copy()
    XK2[c + 3:], XV2[c + 3:] = 99.0, -99.0          # the future of queries 0..2
    O2, _ = orc.attention(Q, XK2, XV2, c)
    np.testing.assert_array_equal(O1[:3], O2[:3])


def algorithm2_numpy(Q, K, V, G, B, M, eps, c_mult=1, chunk_first=False):
    """Algorithm 2 restated with numpy matrix ops and the correlation reference above:
    a second evaluator with a different structure from the C loops."""
    L, d = Q.shape
    Kc, Vc = np.zeros((0, d)), np.zeros((0, d))
    O = np.zeros((L, d))
    for t0 in range(0, L, B):
        Qn, Kn, Vn = Q[t0:t0 + B], K[t0:t0 + B], V[t0:t0 + B]
        b, c = len(Qn), len(Kc)
        XK, XV = np.vstack([Kc, Kn]), np.vstack([Vc, Vn])
        lg = (Qn @ XK.T) / np.sqrt(d)
        vis = np.arange(c + b)[None, :] <= (c + np.arange(b))[:, None]
        lg = np.where(vis, lg, -np.inf)
        pr = np.exp(lg - lg.max(1, keepdims=True))
        O[t0:t0 + b] = (pr / pr.sum(1, keepdims=True)) @ XV
        if c + b <= M:
            Kc, Vc = XK, XV
        else:
            if chunk_first:
                XK, XV = np.vstack([Kn, Kc]), np.vstack([Vn, Vc])
            Z = XK if c_mult == 1 else np.hstack([XK, XV])
            R = np.maximum(correlate_reference(Z, G), 0)
            w = R / (R.sum(1, keepdims=True) + eps)
            Kc, Vc = w @ XK, w @ XV
    return O, Kc, Vc


@pytest.mark.parametrize("L,B,M,c_mult,flags", [(40, 8, 8, 1, 0), (37, 5, 8, 2, 0), (30, 7, 10, 1, 0),
                                                (26, 6, 9, 1, orc.CHUNK_FIRST), (21, 21, 4, 2, 0)])
def test_algorithm2_against_numpy_restatement(L, B, M, c_mult, flags):
    r = rng(50 + L)
    d, k = 4, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, c_mult * d, k))
    O, Kc, Vc, c, _ = orc.process_sequence(Q, K, V, G, B, eps=1e-6, flags=flags)
    O2, Kc2, Vc2 = algorithm2_numpy(Q, K, V, G, B, M, 1e-6, c_mult, bool(flags & orc.CHUNK_FIRST))
    np.testing.assert_allclose(O, O2, atol=1e-11)
    np.testing.assert_allclose(Kc[:c], Kc2, atol=1e-11)
    np.testing.assert_allclose(Vc[:c], Vc2, atol=1e-11)


def test_attention_precedes_update_no_future_leak():
    # Algorithm 2 runs Step 3 with the OLD cache: outputs of chunk n must not depend on
    # later tokens, not even through the compressed slots.
    r = rng(61)
    L, B, M, d, k = 32, 8, 8, 4, 3
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    O1 = orc.process_sequence(Q, K, V, G, B)[0]
    K2, V2 = K.copy(), V.copy()
    K2[21:], V2[21:] = r.standard_normal((L - 21, d)), r.standard_normal((L - 21, d))
    O2 = orc.process_sequence(Q, K2, V2, G, B)[0]
    np.testing.assert_array_equal(O1[:21], O2[:21])
    assert np.abs(O1[21:] - O2[21:]).max() > 1e-3


def test_first_compress_with_partly_filled_cache_sees_only_real_entries():
    r = rng(62)
    d, M, k = 4, 8, 3
    Kc, Vc = np.zeros((M, d)), np.zeros((M, d))
    Kc[:3], Vc[:3] = r.standard_normal((3, d)), r.standard_normal((3, d))
    Kn, Vn = r.standard_normal((7, d)), r.standard_normal((7, d))
    G = r.standard_normal((M, d, k))
    K1, V1, c1 = orc.update_cache(Kc, Vc, 3, Kn, Vn, G)
    K2, V2 = orc.compress(np.vstack([Kc[:3], Kn]), np.vstack([Vc[:3], Vn]), G)
    assert c1 == M
    np.testing.assert_array_equal(K1, K2)
    np.testing.assert_array_equal(V1, V2)


def test_suspend_and_resume_is_identical():
    r = rng(63)
    L, B, M, d, k = 48, 8, 8, 4, 5
    Q, K, V = r.standard_normal((L, d)), r.standard_normal((L, d)), r.standard_normal((L, d))
    G = r.standard_normal((M, d, k))
    O, Kc, Vc, c, _ = orc.process_sequence(Q, K, V, G, B)
    Oa, Ka, Va, ca, _ = orc.process_sequence(Q[:24], K[:24], V[:24], G, B)
    Ob, Kb, Vb, cb, _ = orc.process_sequence(Q[24:], K[24:], V[24:], G, B, cache=(Ka, Va, ca))
    np.testing.assert_array_equal(O, np.vstack([Oa, Ob]))
    np.testing.assert_array_equal(Kc, Kb)
    np.testing.assert_array_equal(Vc, Vb)


def test_relu_on_input_reading_flag():
    r = rng(64)
    XK, XV, G = r.standard_normal((11, 4)), r.standard_normal((11, 4)), r.standard_normal((3, 4, 3))
    Kn, Vn, w, A, s = orc.compress(XK, XV, G, eps=0.0, flags=orc.RELU_ON_INPUT, want_weights=True)
    A_ref = correlate_reference(np.maximum(XK, 0), G)
    np.testing.assert_allclose(A, A_ref, atol=1e-13)
    np.testing.assert_allclose(w, A_ref / A_ref.sum(1, keepdims=True), atol=1e-11)
    np.testing.assert_allclose(Kn, w @ XK, atol=1e-12)


def test_batch_driver_equals_per_unit_calls():
    r = rng(65)
    Bt, H, L, d, M, k, B = 2, 3, 20, 4, 6, 3, 5
    Q, K, V = (r.standard_normal((Bt, H, L, d)) for _ in range(3))
    for Hg in (1, H):
        G = r.standard_normal((Hg, M, d, k))
        O, Kc, Vc, c, lse = orc.process_batch(Q, K, V, G, B)
        for bi in range(Bt):
            for h in range(H):
                o, kc, vc, cc, ls = orc.process_sequence(Q[bi, h], K[bi, h], V[bi, h], G[h % Hg], B)
                np.testing.assert_array_equal(O[bi, h], o)
                np.testing.assert_array_equal(Kc[bi, h], kc)
                np.testing.assert_array_equal(lse[bi, h], ls)
                assert c[bi, h] == cc
