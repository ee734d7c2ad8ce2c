"""ctypes front end of the float64 CPU oracle (oracle/lococo_oracle.c).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU
baseline may import this module; the CUDA library and its Python binding never
do, and this module never touches them.

All arrays are float64 numpy, row-major, positions as rows ([tokens, d]).
Each function names the passage of the paper it evaluates.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "lococo_oracle.c"
_LIB = _HERE / "liblococo_oracle.so"

CHUNK_FIRST = 1      # Eq. 6's operand order [chunk, cache] instead of Eq. 3's [cache, chunk]
RELU_ON_INPUT = 2    # ReLU on the conv input instead of its output


def build(force: bool = False) -> Path:
    """Compile the C source with gcc (OpenMP across units only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(tmp),
                               str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("M", ctypes.c_int32), ("k", ctypes.c_int32),
                ("c_in", ctypes.c_int32), ("flags", ctypes.c_int32), ("protected_slots", ctypes.c_int32),
                ("eps", ctypes.c_double), ("scale", ctypes.c_double)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.lococo_oracle_threads.restype = ctypes.c_int
        _lib.lococo_oracle_process_sequence_grad.restype = ctypes.c_int
        _lib.lococo_oracle_process_sequence_grad_from.restype = ctypes.c_int
        _lib.lococo_oracle_grad_batch.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().lococo_oracle_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _params(d, M, k, c_in, eps, scale, flags, protected=0):
    if scale is None or scale == 0:
        scale = 1.0 / np.sqrt(d)
    assert 0 <= protected <= M and not (protected and flags & 1)   # Section 5.2 reading: cache-first order only
    return _Params(d, M, k, c_in, flags, int(protected), float(eps), float(scale))


def conv_logits(Z, G, bias=None):
    """Eq. 6: logits A [M,S] of the 1-D multi-channel convolution of Z [S,C] with G [M,C,k]."""
    Z, G = _f64(Z), _f64(G)
    S, C = Z.shape
    M, C2, k = G.shape
    assert C == C2 and k % 2 == 1
    b = None if bias is None else _f64(bias)
    A = np.empty((M, S))
    _load().lococo_oracle_conv_logits(_p(Z), S, C, _p(G), _p(b), M, k, _p(A))
    return A


def compress(XK, XV, G, bias=None, eps=1e-6, flags=0, want_weights=False, protected=0):
    """Eq. 6 -> ReLU -> Eq. 7 -> Eq. 4, Eq. 5: XK, XV [S,d] -> new cache K, V [M,d]."""
    XK, XV, G = _f64(XK), _f64(XV), _f64(G)
    S, d = XK.shape
    M, C, k = G.shape
    assert XV.shape == (S, d) and C in (d, 2 * d) and k % 2 == 1
    b = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, None, flags, protected)
    Kn, Vn = np.empty((M, d)), np.empty((M, d))
    w = np.empty((M, S)) if want_weights else None
    A = np.empty((M, S)) if want_weights else None
    s = np.empty(M) if want_weights else None
    _load().lococo_oracle_compress(ctypes.byref(P), _p(XK), _p(XV), S, _p(G), _p(b), _p(Kn), _p(Vn),
                                   _p(w), _p(A), _p(s))
    if want_weights:
        return Kn, Vn, w, A, s
    return Kn, Vn


def attention(Q, XK, XV, c, scale=None, want_prob=False):
    """Eq. 1 / Algorithm 2 Step 3: Q [b,d] over [cache (c rows); chunk (b rows)] -> O [b,d], lse [b]."""
    Q, XK, XV = _f64(Q), _f64(XK), _f64(XV)
    b, d = Q.shape
    assert XK.shape == (c + b, d) and XV.shape == (c + b, d)
    if scale is None or scale == 0:
        scale = 1.0 / np.sqrt(d)
    O, lse = np.empty((b, d)), np.empty(b)
    prob = np.empty((b, c + b)) if want_prob else None
    _load().lococo_oracle_attention(_p(Q), b, _p(XK), _p(XV), c, d, ctypes.c_double(scale), _p(O), _p(lse), _p(prob))
    return (O, lse, prob) if want_prob else (O, lse)


def update_cache(Kc, Vc, c, Kn, Vn, G, bias=None, eps=1e-6, flags=0, protected=0):
    """Algorithm 2's if/else after Step 3: returns the new (Kc [M,d], Vc [M,d], c)."""
    G = _f64(G)
    M, C, k = G.shape
    Kc, Vc = _f64(Kc).copy(), _f64(Vc).copy()
    Kn, Vn = _f64(Kn), _f64(Vn)
    b, d = Kn.shape
    assert Kc.shape == (M, d)
    bb = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, None, flags, protected)
    cc = ctypes.c_int(c)
    _load().lococo_oracle_update_cache(ctypes.byref(P), _p(Kc), _p(Vc), ctypes.byref(cc), _p(Kn), _p(Vn), b,
                                       _p(G), _p(bb))
    return Kc, Vc, cc.value


def process_sequence(Q, K, V, G, B, bias=None, eps=1e-6, scale=None, flags=0, cache=None, want_snapshots=False, protected=0):
    """Algorithm 2 for one unit: Q, K, V [L,d] -> O [L,d], final cache (Kc, Vc [M,d], c), lse [L]."""
    Q, K, V, G = _f64(Q), _f64(K), _f64(V), _f64(G)
    L, d = Q.shape
    M, C, k = G.shape
    bb = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, scale, flags, protected)
    if cache is None:
        Kc, Vc, c = np.zeros((M, d)), np.zeros((M, d)), 0
    else:
        Kc, Vc, c = _f64(cache[0]).copy(), _f64(cache[1]).copy(), int(cache[2])
    O, lse = np.empty((L, d)), np.empty(L)
    N = -(-L // B)
    sK = np.zeros((N, M, d)) if want_snapshots else None
    sV = np.zeros((N, M, d)) if want_snapshots else None
    sc = np.zeros(N, dtype=np.int32) if want_snapshots else None
    cc = ctypes.c_int(c)
    _load().lococo_oracle_process_sequence(ctypes.byref(P), _p(Q), _p(K), _p(V), L, B, _p(G), _p(bb), _p(O),
                                           _p(Kc), _p(Vc), ctypes.byref(cc), _p(lse), _p(sK), _p(sV), _p(sc))
    out = (O, Kc, Vc, cc.value, lse)
    return out + (sK, sV, sc) if want_snapshots else out


def process_sequence_grad(Q, K, V, G, B, dO, dKc_final, dVc_final, bias=None, eps=1e-6, scale=None, protected=0,
                          cache=None):
    """Gradients of <dO,O> + <dKc_final,Kc_final> + <dVc_final,Vc_final> through Algorithm 2:
    returns dQ, dK, dV [L,d], dG [M,C,k], dbias [M] or None.  With cache = (Kc [M,d], Vc [M,d], c) the loop
    starts from that cache instead of an empty one and the gradients w.r.t. it, dKc_in and dVc_in [M,d], are
    returned as well (the training use of a sequence processed in several calls, last call first)."""
    Q, K, V, G = _f64(Q), _f64(K), _f64(V), _f64(G)
    L, d = Q.shape
    M, C, k = G.shape
    bb = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, scale, 0, protected)
    dO, dKf, dVf = _f64(dO), _f64(dKc_final), _f64(dVc_final)
    dQ, dK, dV = np.zeros((L, d)), np.zeros((L, d)), np.zeros((L, d))
    dG = np.zeros((M, C, k))
    db = np.zeros(M) if bias is not None else None
    if cache is None:
        rc = _load().lococo_oracle_process_sequence_grad(ctypes.byref(P), _p(Q), _p(K), _p(V), L, B, _p(G), _p(bb),
                                                         _p(dO), _p(dKf), _p(dVf), _p(dQ), _p(dK), _p(dV), _p(dG), _p(db))
        assert rc == 0
        return dQ, dK, dV, dG, db
    Kc, Vc, c = _f64(cache[0]), _f64(cache[1]), int(cache[2])
    assert Kc.shape == (M, d) and Vc.shape == (M, d) and 0 <= c <= M
    dKc, dVc = np.zeros((M, d)), np.zeros((M, d))
    rc = _load().lococo_oracle_process_sequence_grad_from(ctypes.byref(P), _p(Q), _p(K), _p(V), L, B, _p(G), _p(bb),
                                                          _p(Kc), _p(Vc), c, _p(dO), _p(dKf), _p(dVf), _p(dQ), _p(dK),
                                                          _p(dV), _p(dG), _p(db), _p(dKc), _p(dVc))
    assert rc == 0
    return dQ, dK, dV, dG, db, dKc, dVc


def process_batch(Q, K, V, G, B, bias=None, eps=1e-6, scale=None, flags=0, protected=0):
    """Algorithm 2 for [batch, heads, L, d] inputs; G [heads|1, M, C, k].  OpenMP across units.
    Returns O [batch,heads,L,d], Kc, Vc [batch,heads,M,d], c [batch,heads], lse [batch,heads,L]."""
    Q, K, V, G = _f64(Q), _f64(K), _f64(V), _f64(G)
    Bt, H, L, d = Q.shape
    Hg, M, C, k = G.shape
    assert Hg in (1, H)
    bb = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, scale, flags, protected)
    units = Bt * H
    O = np.empty((Bt, H, L, d))
    Kc, Vc = np.zeros((Bt, H, M, d)), np.zeros((Bt, H, M, d))
    c = np.zeros((Bt, H), dtype=np.int32)
    lse = np.empty((Bt, H, L))
    gs = 0 if Hg == 1 else M * C * k
    bs = 0 if Hg == 1 else M
    _load().lococo_oracle_process_batch(ctypes.byref(P), units, H, _p(Q), _p(K), _p(V), L, B, _p(G),
                                        ctypes.c_long(gs), _p(bb), ctypes.c_long(bs), _p(O), _p(Kc), _p(Vc),
                                        _p(c), _p(lse))
    return O, Kc, Vc, c, lse


def grad_batch(Q, K, V, G, B, dO, dKc_final, dVc_final, bias=None, eps=1e-6, scale=None, protected=0):
    """Batched process_sequence_grad; dG is summed over the units sharing a weight set."""
    Q, K, V, G = _f64(Q), _f64(K), _f64(V), _f64(G)
    Bt, H, L, d = Q.shape
    Hg, M, C, k = G.shape
    bb = None if bias is None else _f64(bias)
    P = _params(d, M, k, C, eps, scale, 0, protected)
    dO, dKf, dVf = _f64(dO), _f64(dKc_final), _f64(dVc_final)
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(Q), np.zeros_like(Q)
    dG = np.zeros_like(G)
    db = np.zeros((Hg, M)) if bias is not None else None
    gs = 0 if Hg == 1 else M * C * k
    bs = 0 if Hg == 1 else M
    rc = _load().lococo_oracle_grad_batch(ctypes.byref(P), Bt * H, H, _p(Q), _p(K), _p(V), L, B, _p(G),
                                          ctypes.c_long(gs), _p(bb), ctypes.c_long(bs), _p(dO), _p(dKf), _p(dVf),
                                          _p(dQ), _p(dK), _p(dV), _p(dG), _p(db))
    assert rc == 0
    return dQ, dK, dV, dG, db
