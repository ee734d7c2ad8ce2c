"""The allocation-free compress entry point (scratch in a fixed array inside the library,
for callers that are not allowed to call cudaMalloc) against the regular entry point and
against the CPU oracle.
Collected last on purpose: a failure here cannot hide one elsewhere."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, to_device, to_host, torch_dtype

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,d,M,k,c,b,c_mult,per_head,bias", [
    ("bf16", 128, 128, 21, 128, 512, 1, True, False),
    ("f32", 64, 40, 7, 33, 90, 2, False, True),
])
def test_static_scratch_compress_matches_workspace_compress(dtype, d, M, k, c, b, c_mult, per_head, bias):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    w = wl.Workload("noalloc", 21, batch=1, heads=3, d=d, M=M, B=b, k=k, L=b, dtype=dtype, weights_per_head=per_head,
                    qkv_scale=1.0, c_in_mult=c_mult)
    G, bvec = wl.make_weights(w, with_bias=bias)
    dG = to_device(G, dtype)
    dB = None if bvec is None else to_device(bvec, dtype)
    ref = api.Lococo(w.batch, w.heads, d, M, k, b, dtype=torch_dtype(dtype), c_in=w.c_in, weights_per_head=per_head,
                     path=api.PATH_SIMT)
    ref.set_weights(dG, dB)
    cfg = api.Config(w.batch, w.heads, d, M, k, w.c_in, int(per_head), api.BF16 if dtype == "bf16" else api.F32,
                     0.0, 1e-6, b, api.PATH_AUTO)
    for call in range(2):            # two calls in a row share the array; the second uses new inputs
        ws = w.slice(seed0=500 + call)
        _, Kn, Vn = wl.make_qkv(ws)
        _, Kc, Vc = wl.make_qkv(ws.slice(L=M, seed0=900 + call))
        dKc, dVc, dKn, dVn = (to_device(x, dtype) for x in (Kc, Vc, Kn, Vn))
        Ko_ref, Vo_ref = torch.zeros_like(dKc), torch.zeros_like(dVc)
        ref.compress_step(dKc, dVc, c, dKn, dVn, Ko_ref, Vo_ref)
        Ko, Vo = torch.zeros_like(dKc), torch.zeros_like(dVc)
        api.compress_step_static(cfg, dG, dB, dKc, dVc, c, dKn, dVn, Ko, Vo)
        torch.cuda.synchronize()
        assert_close(to_host(Ko), to_host(Ko_ref), dtype, f"K slots, call {call}")
        assert_close(to_host(Vo), to_host(Vo_ref), dtype, f"V slots, call {call}")
        assert to_host(Ko).any()
        # and against the float64 oracle (Eq. 6 -> ReLU -> Eq. 7 -> Eq. 4-5), unit by unit
        for h in range(w.heads):
            XK = np.concatenate([Kc[0, h, :c], Kn[0, h]])
            XV = np.concatenate([Vc[0, h, :c], Vn[0, h]])
            Kr, Vr = orc.compress(XK, XV, G[h if per_head else 0], bias=None if bvec is None else bvec[h if per_head else 0])
            assert_close(to_host(Ko)[0, h], Kr, dtype, f"K slots vs oracle, call {call}, head {h}")
            assert_close(to_host(Vo)[0, h], Vr, dtype, f"V slots vs oracle, call {call}, head {h}")


def test_static_scratch_in_place_and_just_under_the_limit():
    # the cache updated in place (outputs = cache inputs), on a problem that takes nearly all of the array:
    # 13 heads x M=128 x S=978 fp32 logits = 6.2 MiB; with the packed weights, sums and blends 4 KiB short of 8 MiB
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    heads, d, M, k, c, b = 13, 128, 128, 5, 128, 850
    need = M * d * k * 2 + M * 4 + heads * M * 4 + 2 * heads * M * d * 4 + heads * M * (c + b) * 4
    assert 0.99 * api.static_scratch_limit() < need <= api.static_scratch_limit()
    w = wl.Workload("noalloc_big", 22, batch=1, heads=heads, d=d, M=M, B=b, k=k, L=b, dtype="bf16",
                    weights_per_head=False, qkv_scale=1.0)
    G, _ = wl.make_weights(w)
    _, Kn, Vn = wl.make_qkv(w)
    _, Kc, Vc = wl.make_qkv(w.slice(L=M, seed0=77))
    dKc, dVc, dKn, dVn = (to_device(x, "bf16") for x in (Kc, Vc, Kn, Vn))
    cfg = api.Config(1, heads, d, M, k, d, 0, api.BF16, 0.0, 1e-6, b, api.PATH_AUTO)
    api.compress_step_static(cfg, to_device(G, "bf16"), None, dKc, dVc, c, dKn, dVn, dKc, dVc)
    torch.cuda.synchronize()
    for h in (0, 7, 12):
        Kr, Vr = orc.compress(np.concatenate([Kc[0, h], Kn[0, h]]), np.concatenate([Vc[0, h], Vn[0, h]]), G[0])
        assert_close(to_host(dKc)[0, h], Kr, "bf16", f"in place, K slots, head {h}")
        assert_close(to_host(dVc)[0, h], Vr, "bf16", f"in place, V slots, head {h}")


def test_static_scratch_rejects_what_does_not_fit():
    from paper_2406_05317_b200 import api
    limit = api.static_scratch_limit()
    assert limit == 8 << 20
    # 32 heads x M=128 x S=640 fp32 logits alone are 10 MiB
    cfg = api.Config(1, 32, 128, 128, 21, 128, 0, api.BF16, 0.0, 1e-6, 512, api.PATH_AUTO)
    G = torch.zeros(1, 128, 128, 21, dtype=torch.bfloat16, device="cuda")
    Kc = torch.zeros(1, 32, 128, 128, dtype=torch.bfloat16, device="cuda")
    Kn = torch.zeros(1, 32, 512, 128, dtype=torch.bfloat16, device="cuda")
    Ko, Vo = torch.ones_like(Kc), torch.ones_like(Kc)
    with pytest.raises(api.LococoError) as e:
        api.compress_step_static(cfg, G, None, Kc, Kc.clone(), 128, Kn, Kn.clone(), Ko, Vo)
    assert e.value.status == api.ERR_WORKSPACE
    with pytest.raises(api.LococoError) as e:       # the fill branch is not served here
        api.compress_step_static(cfg, G, None, Kc, Kc.clone(), 0, Kn[:, :, :64], Kn[:, :, :64].clone(), Ko, Vo)
    assert e.value.status == api.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert (Ko == 1).all() and (Vo == 1).all()      # nothing was launched
