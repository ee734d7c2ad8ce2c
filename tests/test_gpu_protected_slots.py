"""Protected slots (Section 5.2: the compressor next to an eviction policy that always keeps some
tokens) on the GPU against the float64 oracle: forward on both kernel families, the kept tokens
bit for bit, and the backward pass."""
import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, to_device, to_host, torch_dtype
from tests.test_gpu_backward import check_gradients

pytestmark = pytest.mark.gpu


def run_forward(api, w, slots, path=0, bias=False, saved=False):
    tdt = torch_dtype(w.dtype)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=tdt, c_in=w.c_in, weights_per_head=w.weights_per_head,
                     path=path)
    G, bvec = wl.make_weights(w, with_bias=bias)
    ctx.set_weights(to_device(G, w.dtype), None if bvec is None else to_device(bvec, w.dtype))
    ctx.set_protected_slots(slots)
    Q, K, V = wl.make_qkv(w)
    dev = [to_device(x, w.dtype) for x in (Q, K, V)]
    O = torch.empty_like(dev[0])
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=tdt, device="cuda")
    Vc = torch.zeros_like(Kc)
    sv = torch.empty(ctx.saved_bytes(w.L, w.B), dtype=torch.uint8, device="cuda") if saved else None
    c = ctx.process_sequence(*dev, w.B, O, Kc, Vc, 0, sv) if saved else ctx.process_sequence(*dev, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    return ctx, (Q, K, V, G, bvec), dev, (O, Kc, Vc, c), sv


def check_forward(w, slots, path=0, bias=False):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    _, (Q, K, V, G, bvec), dev, (O, Kc, Vc, c), _ = run_forward(api, w, slots, path, bias)
    Or, Kr, Vr, cr, _ = orc.process_batch(Q, K, V, G, w.B, bias=bvec, protected=slots)
    assert (cr == c).all() and c == w.M
    assert_close(to_host(O), Or, w.dtype, f"{w.name} O")
    assert_close(to_host(Kc), Kr, w.dtype, f"{w.name} K cache")
    assert_close(to_host(Vc), Vr, w.dtype, f"{w.name} V cache")
    # the kept tokens are copies, not blends: equal bit for bit to the first tokens of the sequence
    assert torch.equal(Kc[:, :, :slots], dev[1][:, :, :slots]) and torch.equal(Vc[:, :, :slots], dev[2][:, :, :slots])
    # and the run differs from the plain method where it should
    _, _, _, (O0, Kc0, _, _), _ = run_forward(api, w, 0, path, bias)
    assert not torch.equal(Kc0[:, :, :slots], Kc[:, :, :slots])


@pytest.mark.parametrize("path", [0, 1])
def test_forward_bf16_both_kernel_families(path):
    # tensor-core path (0) and CUDA-core path (1): 4 sink slots, ragged chunks, a first compress step on a
    # partly filled cache, split position tiles (few units) on the tensor path
    w = wl.Workload("prot_bf16", 51, batch=1, heads=2, d=128, M=128, B=200, k=21, L=1100, dtype="bf16",
                    weights_per_head=True, qkv_scale=0.0884, g_std=0.02)
    check_forward(w, 4, path)


def test_forward_bf16_tensor_path_direct_cache_write_and_bias():
    # many units: every compress CTA sees all positions of its slots and normalises by itself;
    # 37 protected slots straddle the 32-row groups of the accumulator
    w = wl.Workload("prot_direct", 52, batch=3, heads=2, d=128, M=128, B=100, k=9, L=900, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02, c_in_mult=2)
    check_forward(w, 37, 0, bias=True)


def test_forward_fp32_and_larger_cache():
    w = wl.Workload("prot_f32", 53, batch=1, heads=2, d=64, M=48, B=40, k=5, L=333, dtype="f32",
                    weights_per_head=True, qkv_scale=0.3, g_std=0.1)
    check_forward(w, 5)
    w = wl.Workload("prot_m256", 54, batch=1, heads=3, d=128, M=256, B=512, k=21, L=2048, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02)
    check_forward(w, 130)   # more than one block of 128 slots: the second block is partly protected


def test_persistent_loop_gives_the_same_bits():
    from paper_2406_05317_b200 import api
    w = wl.Workload("prot_persist", 55, batch=2, heads=4, d=128, M=128, B=256, k=21, L=1536, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02)
    _, _, _, (O2, K2, V2, _), _ = run_forward(api, w, 8, api.PATH_TENSOR)
    _, _, _, (O3, K3, V3, _), _ = run_forward(api, w, 8, api.PATH_TENSOR_PERSISTENT)
    assert torch.equal(O2, O3) and torch.equal(K2, K3) and torch.equal(V2, V3)


def test_changing_the_count_between_calls_takes_effect():
    # the chunk loop is cached as a graph per call shape: a new count must not replay the old launches
    from paper_2406_05317_b200 import api
    w = wl.Workload("prot_switch", 56, batch=1, heads=2, d=128, M=128, B=256, k=9, L=1024, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02)
    ctx, _, dev, (O, Kc, Vc, _), _ = run_forward(api, w, 0)
    outs = []
    for slots in (0, 0, 6, 6, 0):
        ctx.set_protected_slots(slots)
        Kc.zero_(), Vc.zero_()
        ctx.process_sequence(*dev, w.B, O, Kc, Vc, 0)
        torch.cuda.synchronize()
        outs.append(Kc.clone())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[2], outs[3]) and torch.equal(outs[0], outs[4])
    assert torch.equal(outs[2][:, :, :6], dev[1][:, :, :6]) and not torch.equal(outs[0][:, :, :6], dev[1][:, :, :6])
    with pytest.raises(Exception):
        ctx.set_protected_slots(w.M + 1)


def check_backward(w, slots, bias=False, path=0):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    ctx, (Q, K, V, G, bvec), dev, (O, Kc, Vc, c), saved = run_forward(api, w, slots, path, bias, saved=True)
    PO, PK, PV = wl.make_loss_projections(w)
    dPO, dPK, dPV = (to_device(x, w.dtype) for x in (PO, PK, PV))
    gQ, gK, gV = (torch.empty_like(dev[0]) for _ in range(3))
    gG = torch.zeros(G.shape, dtype=torch.float32, device="cuda")
    gB = torch.zeros(bvec.shape, dtype=torch.float32, device="cuda") if bias else None
    scratch = torch.empty(ctx.backward_scratch_bytes(w.L, w.B), dtype=torch.uint8, device="cuda")
    ctx.process_sequence_backward(*dev, O, w.B, saved, dPO, dPK, dPV, gQ, gK, gV, gG, gB, scratch)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    rQ, rK, rV, rG, rB = orc.grad_batch(Q, K, V, G, w.B, PO, PK, PV, bias=bvec, protected=slots)
    got = dict(dQ=to_host(gQ), dK=to_host(gK), dV=to_host(gV), dG=to_host(gG))
    ref = dict(dQ=rQ, dK=rK, dV=rV, dG=rG, dbias=rB)
    if bias:
        got["dbias"] = to_host(gB)
    assert (got["dG"][:, :slots] == 0).all()      # unit rows: nothing reaches their conv weights
    if bias:
        assert (got["dbias"][:, :slots] == 0).all()
    assert np.abs(got["dG"][:, slots:]).max() > 0
    check_gradients(w, got, ref)


def test_backward_fp32():
    w = wl.Workload("prot_bwd_f32", 57, batch=1, heads=2, d=64, M=32, B=24, k=5, L=150, dtype="f32",
                    weights_per_head=True, qkv_scale=0.3, g_std=0.1)
    check_backward(w, 3, bias=True)


@pytest.mark.parametrize("path", [0, 1])
def test_backward_bf16(path):
    w = wl.Workload("prot_bwd_bf16", 58, batch=1, heads=4, d=128, M=128, B=256, k=9, L=1024, dtype="bf16",
                    weights_per_head=True, qkv_scale=0.0884, g_std=0.02)
    check_backward(w, 4, path=path)
