"""The failure path of the device code, exercised without hanging anything: a bounded wait is made to run
out (a test-only kernel waits, with a poll limit of a few thousand, on an mbarrier nobody arrives at), and
the library must report it, refuse to hand out further work in the persistent kernel, and recover when the
workspace is handed over again."""
import ctypes

import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def probe():
    from paper_2406_05317_b200 import build
    lib = ctypes.CDLL(str(build.build_test_probe()))
    lib.wait_probe_run.argtypes = [ctypes.c_void_p, ctypes.c_uint, ctypes.c_void_p, ctypes.c_void_p]
    lib.wait_probe_run.restype = ctypes.c_int
    return lib


def run_sequence(ctx, w, Q, K, V, sentinel=None):
    O = torch.empty_like(Q) if sentinel is None else torch.full_like(Q, sentinel)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
    Vc = torch.zeros_like(Kc)
    c = ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    return O, Kc, Vc, c


def test_probe_refuses_long_waits(probe):
    buf = torch.zeros(8, dtype=torch.int64, device="cuda")
    assert probe.wait_probe_run(buf.data_ptr(), 1 << 20, buf.data_ptr(), None) == -1


@pytest.mark.parametrize("path", ["TENSOR", "TENSOR_PERSISTENT"])
def test_expired_wait_is_reported_and_cleared_by_a_new_workspace(probe, path):
    from paper_2406_05317_b200 import api
    w = wl.CONFIGS["cfg2"].slice(heads=2, L=1024)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in,
                     weights_per_head=w.weights_per_head, path=getattr(api, "PATH_" + path))
    G, _ = wl.make_weights(w)
    dG = to_device(G, "bf16")
    ctx.set_weights(dG)
    Q, K, V = (to_device(x, "bf16") for x in wl.make_qkv(w))
    good = run_sequence(ctx, w, Q, K, V)
    assert ctx.device_status() == api.OK

    # a wait that nobody ends: it gives up after `limit` polls and writes the status word of this handle
    # (the first word of its workspace)
    out = torch.zeros(5, dtype=torch.int64, device="cuda")
    assert probe.wait_probe_run(ctx._ws_ptr, 2048, out.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    ok1, ok2, cycles1, cycles2, failed = out.tolist()
    assert ok1 == 0 and ok2 == 0 and failed == 1
    assert cycles2 * 8 < cycles1, (cycles1, cycles2)          # 64 polls against 2048
    assert ctx.device_status() == api.ERR_TIMEOUT
    assert ctx.device_status() == api.ERR_TIMEOUT             # the word stays set

    if path == "TENSOR_PERSISTENT":
        # the persistent kernel hands out no work once the status word is set: nothing is written
        O, Kc, Vc, _ = run_sequence(ctx, w, Q, K, V, sentinel=3.0)
        assert bool((O == 3.0).all()) and not bool(Kc.any())
        assert ctx.device_status() == api.ERR_TIMEOUT

    # handing the workspace over again clears the word; with the weights set again the handle works as before
    st = torch.cuda.current_stream().cuda_stream
    assert api.raw().lococo_set_workspace(ctx.handle, ctx._ws_ptr, ctx.workspace_bytes, st) == api.OK
    assert ctx.device_status() == api.OK
    with pytest.raises(api.LococoError) as e:                 # the weights went with the old hand-over
        run_sequence(ctx, w, Q, K, V)
    assert e.value.status == api.ERR_WORKSPACE
    ctx.set_weights(dG)
    again = run_sequence(ctx, w, Q, K, V)
    assert ctx.device_status() == api.OK
    for a, b in zip(good[:3], again[:3]):
        assert torch.equal(a, b)
