"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py
times (tensor-core path, side stream, repeated calls so that the CUDA-graph replay is what runs).
Where the oracle cannot finish the whole problem in seconds it checks whole (sequence, head) units
taken out of the full run, sampled cache slots, and properties that hold at any size."""
import time

import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, to_device, to_host

pytestmark = pytest.mark.gpu


def run_full(api, w, repeats=3, path=0, keep_inputs=False):
    """process_sequence on the whole workload, `repeats` identical calls on a side stream."""
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in,
                     weights_per_head=w.weights_per_head, path=path)
    G, _ = wl.make_weights(w)
    ctx.set_weights(to_device(G, "bf16"))
    Qh, Kh, Vh = wl.make_qkv(w)
    Q, K, V = (to_device(x, "bf16") for x in (Qh, Kh, Vh))
    O = torch.empty_like(Q)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(repeats):
        with torch.cuda.stream(side):
            c = ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK and c == w.M
    inputs = (Qh, Kh, Vh, G) if keep_inputs else None
    return O, Kc, Vc, inputs


def test_cfg2_full_size_against_the_oracle():
    # the benchmark workload itself: 32 heads, 4096 tokens, 8 chunks, per-head weights
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    w = wl.CONFIGS["cfg2"]
    O, Kc, Vc, (Q, K, V, G) = run_full(api, w, keep_inputs=True)
    Or, Kr, Vr, cr, _ = orc.process_batch(Q, K, V, G, w.B)
    assert (cr == w.M).all()
    assert_close(to_host(O), Or, "bf16", "cfg2 full O")
    assert_close(to_host(Kc), Kr, "bf16", "cfg2 full K cache")
    assert_close(to_host(Vc), Vr, "bf16", "cfg2 full V cache")


def test_cfg3_full_size_units_against_the_oracle():
    # streaming batch at full size: 16 sequences x 32 heads x 8192 tokens, 128 chunks of 64.
    # The oracle recomputes whole units picked out of the full run (units are independent).
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    w = wl.CONFIGS["cfg3"]
    O, Kc, Vc, (Q, K, V, G) = run_full(api, w, repeats=2, keep_inputs=True)
    picks = [(0, 0), (7, 13), (15, 31)]
    sel_q = np.stack([Q[n, h] for n, h in picks])[None]
    sel_k = np.stack([K[n, h] for n, h in picks])[None]
    sel_v = np.stack([V[n, h] for n, h in picks])[None]
    Or, Kr, Vr, cr, _ = orc.process_batch(sel_q, sel_k, sel_v, G, w.B)      # shared weights
    for i, (n, h) in enumerate(picks):
        assert_close(to_host(O[n, h]), Or[0, i], "bf16", f"cfg3 unit {n},{h} O")
        assert_close(to_host(Kc[n, h]), Kr[0, i], "bf16", f"cfg3 unit {n},{h} K cache")
        assert_close(to_host(Vc[n, h]), Vr[0, i], "bf16", f"cfg3 unit {n},{h} V cache")
    # every slot of every unit is a convex combination (Eq. 7): inside the hull of the unit's keys
    kmax = torch.from_numpy(K.max(axis=2, keepdims=True)).cuda()
    kmin = torch.from_numpy(K.min(axis=2, keepdims=True)).cuda()
    assert bool(((Kc.float() <= kmax + 2e-2) & (Kc.float() >= kmin - 2e-2)).all())
    assert bool(torch.isfinite(O.float()).all())


def test_cfg4_full_size_against_the_oracle():
    # fine-tuning shape at full size: 32 heads, M=512, B=4096, 32768 tokens (8 compress steps).
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    w = wl.CONFIGS["cfg4"]
    O, Kc, Vc, (Q, K, V, G) = run_full(api, w, repeats=2, keep_inputs=True)
    assert bool(torch.isfinite(O.float()).all()) and bool(torch.isfinite(Kc.float()).all())
    # (1) first chunk, sampled slots: a slot depends only on its own weight rows, so the oracle is
    #     run with those rows only (S = 4096 positions, c = 0)
    w1 = w.slice(L=w.B)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in, weights_per_head=False)
    ctx.set_weights(to_device(G, "bf16"))
    dK, dV = to_device(K[:, :, :w.B], "bf16"), to_device(V[:, :, :w.B], "bf16")
    K1 = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda")
    V1 = torch.zeros_like(K1)
    assert ctx.compress_step(K1, V1, 0, dK, dV) == w.M
    torch.cuda.synchronize()
    slots = [0, 1, 77, 255, 256, 300, 511]
    for h in (0, 19, 31):
        Kr, Vr = orc.compress(K[0, h, :w.B], V[0, h, :w.B], G[0][slots])
        assert_close(to_host(K1[0, h, slots]), Kr, "bf16", f"cfg4 head {h} sampled K slots")
        assert_close(to_host(V1[0, h, slots]), Vr, "bf16", f"cfg4 head {h} sampled V slots")
    # (2) first chunk, first 640 queries (c = 0: plain causal attention, Eq. 1)
    dQ = to_device(Q[:, :, :640], "bf16")
    O1 = torch.empty_like(dQ)
    ctx.chunk_attention(dQ, K1, V1, 0, dK[:, :, :640], dV[:, :, :640], O1)
    torch.cuda.synchronize()
    for h in (0, 31):
        Or, _ = orc.attention(Q[0, h, :640], K[0, h, :640], V[0, h, :640], 0)
        assert_close(to_host(O1[0, h]), Or, "bf16", f"cfg4 head {h} first queries")
        assert_close(to_host(O[0, h, :640]), Or, "bf16", f"cfg4 head {h} first queries (full run)")
    # (3) the whole 8-step recurrence (Algorithm 2 at M = 512, B = 4096, heavy-tailed keys) against the
    #     oracle: two whole heads taken out of the full run, every output element
    t0 = time.time()
    for h in (0, 19):
        Or, Kr, Vr, cr, _ = orc.process_sequence(Q[0, h], K[0, h], V[0, h], G[0], w.B)
        assert cr == w.M
        assert_close(to_host(O[0, h]), Or, "bf16", f"cfg4 head {h} O, all 8 chunks")
        assert_close(to_host(Kc[0, h]), Kr, "bf16", f"cfg4 head {h} final K cache")
        assert_close(to_host(Vc[0, h]), Vr, "bf16", f"cfg4 head {h} final V cache")
    print(f"cfg4: oracle, 2 heads x 8 chunks: {time.time() - t0:.1f} s on {orc.threads()} threads")
    # (4) the other heads: tensor-core path against the CUDA-core path, same bar
    O2, Kc2, Vc2, _ = run_full(api, w, repeats=1, path=api.PATH_SIMT)
    assert_close(to_host(O[0, :4]), to_host(O2[0, :4]), "bf16", "cfg4 O, tensor vs CUDA-core path")
    assert_close(to_host(Kc), to_host(Kc2), "bf16", "cfg4 K cache, tensor vs CUDA-core path")
    assert_close(to_host(Vc), to_host(Vc2), "bf16", "cfg4 V cache, tensor vs CUDA-core path")


def test_cfg5_full_shape_one_head_gradients_against_the_oracle():
    # the fine-tuning step at its real shape (M = 512, B = 4096, 32768 tokens, 8 compress steps, heavy-tailed
    # keys) on the one-head slice: dQ, dK, dV and the conv-weight gradient through all 8 steps against the
    # float64 oracle's, every element
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    from tests.test_gpu_backward import run_backward, check_gradients
    w = wl.CONFIGS["cfg5"].slice(heads=1)
    got, (Q, K, V, G, bvec, PO, PK, PV) = run_backward(api, w)
    t0 = time.time()
    rQ, rK, rV, rG, _ = orc.grad_batch(Q, K, V, G, w.B, PO, PK, PV)
    print(f"cfg5: oracle gradients, 1 head x 8 chunks: {time.time() - t0:.1f} s on {orc.threads()} threads")
    check_gradients(w, got, dict(dQ=rQ, dK=rK, dV=rV, dG=rG))
