"""Parity of the CUDA backward pass (gradients through all chunk steps of Algorithm 2) with
the float64 oracle's gradients, on the same seeded inputs and loss projections."""
import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, errors, to_device, to_host, torch_dtype

pytestmark = pytest.mark.gpu


def run_backward(api, w, bias=False, path=0):
    tdt = torch_dtype(w.dtype)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=tdt, c_in=w.c_in, weights_per_head=w.weights_per_head,
                     path=path)
    G, bvec = wl.make_weights(w, with_bias=bias)
    ctx.set_weights(to_device(G, w.dtype), None if bvec is None else to_device(bvec, w.dtype))
    Q, K, V = wl.make_qkv(w)
    PO, PK, PV = wl.make_loss_projections(w)
    dQ_, dK_, dV_, dPO, dPK, dPV = (to_device(x, w.dtype) for x in (Q, K, V, PO, PK, PV))
    O = torch.empty_like(dQ_)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=tdt, device="cuda")
    Vc = torch.zeros_like(Kc)
    saved = torch.empty(ctx.saved_bytes(w.L, w.B), dtype=torch.uint8, device="cuda")
    ctx.process_sequence(dQ_, dK_, dV_, w.B, O, Kc, Vc, 0, saved)
    gQ, gK, gV = torch.empty_like(dQ_), torch.empty_like(dQ_), torch.empty_like(dQ_)
    gG = torch.zeros(G.shape, dtype=torch.float32, device="cuda")
    gB = torch.zeros(bvec.shape, dtype=torch.float32, device="cuda") if bias else None
    scratch = torch.empty(ctx.backward_scratch_bytes(w.L, w.B), dtype=torch.uint8, device="cuda")
    ctx.process_sequence_backward(dQ_, dK_, dV_, O, w.B, saved, dPO, dPK, dPV, gQ, gK, gV, gG, gB, scratch)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    got = dict(dQ=to_host(gQ), dK=to_host(gK), dV=to_host(gV), dG=to_host(gG))
    if bias:
        got["dbias"] = to_host(gB)
    return got, (Q, K, V, G, bvec, PO, PK, PV)


def check_gradients(w, got, ref):
    """The parity bar for gradients. fp32 storage: max|g-o| <= 1e-4 max|o|. bf16 storage: mean|g-o| <= 5e-3 mean|o|
    and max|g-o| <= 2e-2 * max(1, max|o|): the absolute bar of the forward outputs where the gradient's entries
    are of order one or less, and the same bar relative to the largest entry where they are larger (a bf16 value
    near 4 is already 1.6e-2 away from its neighbour, so an absolute 2e-2 cannot be asked of a stored gradient
    of that size; the weight gradient, summed over thousands of positions, has entries in the hundreds)."""
    for name, g in got.items():
        max_abs, mean_rel, rel = errors(g, ref[name])
        top = np.abs(ref[name]).max()
        print(f"{w.name} {name}: max|o| {top:.3g}, max|g-o| {max_abs:.3g}, mean rel {mean_rel:.3g}")
        assert np.isfinite(g).all(), (w.name, name)
        if w.dtype == "f32":
            assert_close(g, ref[name], "f32", f"{w.name} {name}")
        else:
            assert max_abs <= 2e-2 * max(1.0, top) and mean_rel <= 5e-3, (w.name, name, top, max_abs, mean_rel)


def check_backward(w, bias=False, path=0):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    got, (Q, K, V, G, bvec, PO, PK, PV) = run_backward(api, w, bias, path)
    rQ, rK, rV, rG, rB = orc.grad_batch(Q, K, V, G, w.B, PO, PK, PV, bias=bvec)
    check_gradients(w, got, dict(dQ=rQ, dK=rK, dV=rV, dG=rG, dbias=rB))


def test_backward_cfg1_fp32():
    check_backward(wl.CONFIGS["cfg1"])


def test_backward_ragged_fp32_bias_per_head_stacked_input():
    w = wl.Workload("bwd_ragged", 31, batch=2, heads=2, d=64, M=24, B=19, k=7, L=100, dtype="f32",
                    weights_per_head=True, qkv_scale=1.0, g_std=0.05, c_in_mult=2)
    check_backward(w, bias=True)


def test_backward_fill_only_fp32():
    # L <= M: no compress step, dG stays zero, gradients are those of plain causal attention
    w = wl.Workload("bwd_fill", 32, batch=1, heads=2, d=64, M=64, B=16, k=5, L=60, dtype="f32",
                    weights_per_head=False, qkv_scale=1.0)
    check_backward(w)


@pytest.mark.parametrize("path", [0, 1])
def test_backward_cfg2_slice_bf16(path):
    check_backward(wl.CONFIGS["cfg2"].slice(heads=2, L=2048), path=path)


def test_backward_cfg5_shape_slice_bf16():
    # fine-tuning shape (M=512, shared weights, heavy-tailed keys), shortened chunks: 2 heads, 3 steps
    check_backward(wl.CONFIGS["cfg5"].slice(heads=2, B=512, L=1536))


def test_backward_shared_weights_fp32_batch():
    w = wl.Workload("bwd_shared", 33, batch=3, heads=2, d=128, M=32, B=40, k=9, L=130, dtype="f32",
                    weights_per_head=False, qkv_scale=0.5, g_std=0.05)
    check_backward(w)


def test_backward_bf16_tensor_path_shared_weights_batch_stacked_input_ragged():
    # tensor-core backward: several sequences share one weight set (the weight gradient sums over all
    # units), keys stacked on values as the conv input (c_in = 2d), chunk length not a multiple of 64
    w = wl.Workload("bwd_tc_shared", 34, batch=2, heads=3, d=128, M=128, B=200, k=7, L=700, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.3, g_std=0.05, c_in_mult=2)
    check_backward(w)


def test_backward_bf16_tensor_path_per_head_fill_then_partial_cache_bias():
    # tensor-core backward: per-head weights with a batch, two fill steps, a first compress step on a
    # partly filled cache (c = 192 < M), ragged last chunk, bias gradient
    w = wl.Workload("bwd_tc_fill", 35, batch=2, heads=2, d=128, M=256, B=96, k=5, L=420, dtype="bf16",
                    weights_per_head=True, qkv_scale=0.0884, g_std=0.02)
    check_backward(w, bias=True)


def test_backward_bf16_tensor_path_per_head_stacked_input():
    # tensor-core backward: one weight set per head AND keys stacked on values as the conv input
    # (the weight gradient's column index runs over taps and both 128-channel halves)
    w = wl.Workload("bwd_tc_ph2d", 36, batch=2, heads=2, d=128, M=128, B=160, k=5, L=480, dtype="bf16",
                    weights_per_head=True, qkv_scale=0.0884, g_std=0.02, c_in_mult=2)
    check_backward(w)


@pytest.mark.parametrize("name,path,cut", [("cfg1", 0, 128), ("cfg2s", 0, 1024), ("cfg2s", 1, 1024), ("fill", 0, 40)])
def test_backward_over_two_calls_equals_backward_over_one_call(name, path, cut):
    # A sequence processed in two calls of the loop (the cache handed over) and differentiated last call first, the
    # cache gradient of the second call handed back as the first call's final-cache gradient: the oracle's
    # gradients of the whole sequence. ("fill": the second call starts from a partly filled cache.)
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    w = {"cfg1": wl.CONFIGS["cfg1"],
         "cfg2s": wl.CONFIGS["cfg2"].slice(heads=2, L=2048),
         "fill": wl.Workload("bwd_fill2", 37, batch=1, heads=2, d=64, M=64, B=20, k=5, L=160, dtype="f32",
                             weights_per_head=False, qkv_scale=1.0)}[name]
    tdt = torch_dtype(w.dtype)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=tdt, c_in=w.c_in, weights_per_head=w.weights_per_head, path=path)
    G, _ = wl.make_weights(w)
    ctx.set_weights(to_device(G, w.dtype))
    Q, K, V = wl.make_qkv(w)
    PO, PK, PV = wl.make_loss_projections(w)
    dQ_, dK_, dV_, dPO, dPK, dPV = (to_device(x, w.dtype) for x in (Q, K, V, PO, PK, PV))
    O = torch.empty_like(dQ_)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=tdt, device="cuda")
    Vc = torch.zeros_like(Kc)
    parts = [(0, cut), (cut, w.L)]
    saved, c_in = [], []
    c = 0
    for a, b in parts:                                  # forward, call by call
        sv = torch.empty(ctx.saved_bytes(b - a, w.B), dtype=torch.uint8, device="cuda")
        c_in.append(c)
        c = ctx.process_sequence(dQ_[:, :, a:b], dK_[:, :, a:b], dV_[:, :, a:b], w.B, O[:, :, a:b], Kc, Vc, c, sv)
        saved.append(sv)
    gQ, gK, gV = torch.empty_like(dQ_), torch.empty_like(dQ_), torch.empty_like(dQ_)
    gG = torch.zeros(G.shape, dtype=torch.float32, device="cuda")
    gKc, gVc = dPK, dPV                                 # the loss's own terms on the final cache
    for (a, b), sv, c0 in reversed(list(zip(parts, saved, c_in))):   # backward, last call first
        scratch = torch.empty(ctx.backward_scratch_bytes(b - a, w.B), dtype=torch.uint8, device="cuda")
        gKc_in, gVc_in = torch.full_like(Kc, 7.0), torch.full_like(Kc, 7.0)
        ctx.process_sequence_backward(dQ_[:, :, a:b], dK_[:, :, a:b], dV_[:, :, a:b], O[:, :, a:b], w.B, sv,
                                      dPO[:, :, a:b], gKc, gVc, gQ[:, :, a:b], gK[:, :, a:b], gV[:, :, a:b], gG, None,
                                      scratch, cache_len_in=c0, dK_cache_in=gKc_in, dV_cache_in=gVc_in)
        torch.cuda.synchronize()
        assert not to_host(gKc_in)[:, :, c0:].any() and not to_host(gVc_in)[:, :, c0:].any()
        gKc, gVc = gKc_in, gVc_in
    assert ctx.device_status() == api.OK
    # the oracle: the same two calls chained in float64 (when the cut is on a chunk boundary this is the
    # one-call gradient, which its own pins show)
    refs = []
    rKc, rVc = PK, PV
    caches = [None]
    Or_, Kr_, Vr_, cr_, _ = orc.process_batch(Q[:, :, :cut], K[:, :, :cut], V[:, :, :cut], G, w.B)
    rQ, rK, rV = np.zeros_like(Q, dtype=np.float64), np.zeros_like(Q, dtype=np.float64), np.zeros_like(Q, dtype=np.float64)
    rG = np.zeros(G.shape)
    for n in range(w.batch):
        for h in range(w.heads):
            g = G[h if w.weights_per_head else 0]
            q2, k2, v2, g2, _, dKc, dVc = orc.process_sequence_grad(
                Q[n, h, cut:], K[n, h, cut:], V[n, h, cut:], g, w.B, PO[n, h, cut:], PK[n, h], PV[n, h],
                cache=(Kr_[n, h], Vr_[n, h], int(cr_[n, h])))
            q1, k1, v1, g1, _ = orc.process_sequence_grad(Q[n, h, :cut], K[n, h, :cut], V[n, h, :cut], g, w.B,
                                                          PO[n, h, :cut], dKc, dVc)
            rQ[n, h], rK[n, h], rV[n, h] = np.concatenate([q1, q2]), np.concatenate([k1, k2]), np.concatenate([v1, v2])
            rG[h if w.weights_per_head else 0] += g1 + g2
    if cut % w.B == 0:
        one = orc.grad_batch(Q, K, V, G, w.B, PO, PK, PV)
        for got, ref in zip((rQ, rK, rV, rG), one[:4]):
            np.testing.assert_allclose(got, ref, atol=1e-9 * max(1.0, np.abs(ref).max()))
    check_gradients(w, dict(dQ=to_host(gQ), dK=to_host(gK), dV=to_host(gV), dG=to_host(gG)),
                    dict(dQ=rQ, dK=rK, dV=rV, dG=rG))
