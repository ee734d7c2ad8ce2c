"""Cases in which the method's result is known exactly, run on the GPU through the C ABI on both
kernel families:
  - one-hot conv kernels turn the compression into token dropping (Section 3.2.3): every new slot
    is one row of [cache; chunk], bit for bit;
  - a constant channel with a centre-tap kernel gives uniform weights: every slot is the mean;
  - a row whose logits are all <= 0 gives a zero slot (Eq. 7 with the epsilon in the denominator).
The picked rows are placed on the first and last position of every position tile, in the halo rows
next to the tile borders and on both sides of the cache / chunk seam, with every tap in use."""
import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, to_device, to_host

pytestmark = pytest.mark.gpu

M, D, K_W, B = 128, 128, 21, 512
PAD = (K_W - 1) // 2


def _targets(rng, S, c):
    """M row indices of [cache; chunk] to pick: tile borders of every tile width the planner uses,
    halo rows, the seam, the ends, and random rows for the rest (with repeats allowed)."""
    fixed = [0, 1, PAD - 1, PAD, S - 1, S - 2, S - PAD, S - PAD - 1, c - 1, c, c + 1, c - PAD, c + PAD]
    for tile in (64, 96, 128, 160, 192, 224):
        for edge in range(tile, S, tile):
            fixed += [edge - 1, edge, edge - PAD, edge + PAD - 1]
    fixed = [j for j in dict.fromkeys(fixed) if 0 <= j < S][:M]
    rest = rng.integers(0, S, size=M - len(fixed))
    return np.concatenate([np.array(fixed, dtype=np.int64), rest])


def _one_hot_problem(rng, units, S, c, c_in_mult):
    """Keys whose channel i is an indicator of one position, one-hot kernels (channel i, tap t_i):
    logit row i is 1 at exactly one position j*_i and 0 elsewhere."""
    taps = rng.permutation(np.arange(M) % K_W)                  # every tap, in random slots
    G = np.zeros((1, M, c_in_mult * D, K_W), dtype=np.float32)
    G[0, np.arange(M), np.arange(M), taps] = 1.0
    XK = np.zeros((units, S, D), dtype=np.float32)
    XV = wl.round_to_bf16(rng.standard_normal((units, S, D)).astype(np.float32))
    picks = np.zeros((units, M), dtype=np.int64)
    for u in range(units):
        want = _targets(rng, S, c)
        # the indicator of slot i sits at pi = j* + t_i - pad and must itself lie inside [0, S)
        pi = np.clip(want + taps - PAD, 0, S - 1)
        picks[u] = pi - taps + PAD
        XK[u, pi, np.arange(M)] = 1.0
    return G, XK, XV, picks


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("c_in_mult", [1, 2])
def test_one_hot_kernels_gather_rows_bit_for_bit(path, c_in_mult):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    rng = np.random.default_rng(77 + c_in_mult)
    heads, c, S = 3, M, M + B
    G, XK, XV, picks = _one_hot_problem(rng, heads, S, c, c_in_mult)
    if c_in_mult == 2:
        # the value channels of the conv input must not fire: their kernel entries are all zero
        assert not G[0, :, D:, :].any()
    ctx = api.Lococo(1, heads, D, M, K_W, B, dtype=torch.bfloat16, c_in=c_in_mult * D, weights_per_head=False,
                     norm_eps=0.0, path=path)
    ctx.set_weights(to_device(G, "bf16"))
    dXK, dXV = to_device(XK[None], "bf16"), to_device(XV[None], "bf16")
    want_k = np.stack([XK[u, picks[u]] for u in range(heads)])[None]
    want_v = np.stack([XV[u, picks[u]] for u in range(heads)])[None]
    # (1) the stand-alone compress step (partial blends + finalize pass on the tensor path)
    Kc, Vc = dXK[:, :, :c].contiguous(), dXV[:, :, :c].contiguous()
    Ko, Vo = torch.zeros_like(Kc), torch.zeros_like(Vc)
    assert ctx.compress_step(Kc, Vc, c, dXK[:, :, c:], dXV[:, :, c:], Ko, Vo) == M
    torch.cuda.synchronize()
    assert np.array_equal(to_host(Ko), want_k), "stand-alone step: K slots are not the picked rows"
    assert np.array_equal(to_host(Vo), want_v), "stand-alone step: V slots are not the picked rows"
    # (2) the same step inside the chunk loop (one launch per chunk, partial sets merged in the kernel)
    Q = torch.zeros(1, heads, B, D, dtype=torch.bfloat16, device="cuda")
    O = torch.empty_like(Q)
    Kc2, Vc2 = dXK[:, :, :c].contiguous(), dXV[:, :, :c].contiguous()
    assert ctx.process_sequence(Q, dXK[:, :, c:].contiguous(), dXV[:, :, c:].contiguous(), B, O, Kc2, Vc2, c) == M
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    assert np.array_equal(to_host(Kc2), want_k), "chunk loop: K slots are not the picked rows"
    assert np.array_equal(to_host(Vc2), want_v), "chunk loop: V slots are not the picked rows"
    # the oracle says the same (it is pinned to this case on the CPU)
    for u in range(heads):
        Kr, Vr = orc.compress(XK[u], XV[u], G[0], eps=0.0)
        assert np.array_equal(Kr, want_k[0, u]) and np.array_equal(Vr, want_v[0, u])


@pytest.mark.parametrize("path", [0, 1])
def test_one_hot_kernels_first_compress_from_an_empty_cache(path):
    # c = 0: the step compresses the chunk alone (S = B), the first tile has no cache rows
    from paper_2406_05317_b200 import api
    rng = np.random.default_rng(91)
    heads, c, S = 2, 0, B
    G, XK, XV, picks = _one_hot_problem(rng, heads, S, c, 1)
    ctx = api.Lococo(1, heads, D, M, K_W, B, dtype=torch.bfloat16, weights_per_head=False, norm_eps=0.0, path=path)
    ctx.set_weights(to_device(G, "bf16"))
    dXK, dXV = to_device(XK[None], "bf16"), to_device(XV[None], "bf16")
    Q = torch.zeros(1, heads, B, D, dtype=torch.bfloat16, device="cuda")
    O = torch.empty_like(Q)
    Kc = torch.zeros(1, heads, M, D, dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    assert ctx.process_sequence(Q, dXK, dXV, B, O, Kc, Vc, 0) == M
    torch.cuda.synchronize()
    assert np.array_equal(to_host(Kc)[0], np.stack([XK[u, picks[u]] for u in range(heads)]))
    assert np.array_equal(to_host(Vc)[0], np.stack([XV[u, picks[u]] for u in range(heads)]))


@pytest.mark.parametrize("path", [0, 1])
def test_constant_channel_gives_the_mean_of_all_entries(path):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    rng = np.random.default_rng(5)
    heads, c, S = 2, M, M + B
    XK = wl.round_to_bf16(rng.standard_normal((heads, S, D)).astype(np.float32))
    XV = wl.round_to_bf16(rng.standard_normal((heads, S, D)).astype(np.float32))
    XK[:, :, 0] = 1.0
    G = np.zeros((1, M, D, K_W), dtype=np.float32)
    G[0, :, 0, PAD] = 1.0                      # logit[i, j] = key channel 0 at position j = 1
    ctx = api.Lococo(1, heads, D, M, K_W, B, dtype=torch.bfloat16, weights_per_head=False, norm_eps=0.0, path=path)
    ctx.set_weights(to_device(G, "bf16"))
    dXK, dXV = to_device(XK[None], "bf16"), to_device(XV[None], "bf16")
    Kc, Vc = dXK[:, :, :c].contiguous(), dXV[:, :, :c].contiguous()
    W = torch.empty(1, heads, M, S, dtype=torch.float32, device="cuda")
    assert ctx.compress_step(Kc, Vc, c, dXK[:, :, c:], dXV[:, :, c:], W_out=W) == M
    torch.cuda.synchronize()
    assert np.allclose(to_host(W), 1.0 / S, rtol=1e-6, atol=0.0), "weights are not uniform"
    for u in range(heads):
        mean_k, mean_v = XK[u].astype(np.float64).mean(axis=0), XV[u].astype(np.float64).mean(axis=0)
        Kr, Vr = orc.compress(XK[u], XV[u], G[0], eps=0.0)
        assert np.allclose(Kr, mean_k, atol=1e-12) and np.allclose(Vr, mean_v, atol=1e-12)
        # every slot equals the mean, up to the bf16 rounding of the stored slot (half an ulp: 2^-8 of the value)
        assert np.abs(to_host(Kc)[0, u] - mean_k).max() <= 2.0 ** -8 * np.abs(mean_k).max() + 1e-6
        assert np.abs(to_host(Vc)[0, u] - mean_v).max() <= 2.0 ** -8 * np.abs(mean_v).max() + 1e-6


@pytest.mark.parametrize("path", [0, 1])
def test_rows_without_a_positive_logit_give_zero_slots(path):
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import api
    rng = np.random.default_rng(6)
    heads, c, S = 2, M, M + B
    XK = wl.round_to_bf16(np.abs(rng.standard_normal((heads, S, D))).astype(np.float32))   # keys >= 0
    XV = wl.round_to_bf16(rng.standard_normal((heads, S, D)).astype(np.float32))
    G = wl.round_to_bf16((rng.standard_normal((1, M, D, K_W)) * 0.02).astype(np.float32))
    G[0, 0::2] = -np.abs(G[0, 0::2])           # even slots: every weight <= 0, so every logit <= 0
    ctx = api.Lococo(1, heads, D, M, K_W, B, dtype=torch.bfloat16, weights_per_head=False, path=path)
    ctx.set_weights(to_device(G, "bf16"))
    dXK, dXV = to_device(XK[None], "bf16"), to_device(XV[None], "bf16")
    Q = torch.zeros(1, heads, B, D, dtype=torch.bfloat16, device="cuda")
    O = torch.empty_like(Q)
    Kc, Vc = dXK[:, :, :c].contiguous(), dXV[:, :, :c].contiguous()
    assert ctx.process_sequence(Q, dXK[:, :, c:].contiguous(), dXV[:, :, c:].contiguous(), B, O, Kc, Vc, c) == M
    torch.cuda.synchronize()
    assert not to_host(Kc)[0, :, 0::2].any() and not to_host(Vc)[0, :, 0::2].any(), "dead rows must give zero slots"
    for u in range(heads):
        Kr, Vr = orc.compress(XK[u], XV[u], G[0])
        assert not Kr[0::2].any() and not Vr[0::2].any()
        assert_close(to_host(Kc)[0, u], Kr, "bf16", "live rows K")
        assert_close(to_host(Vc)[0, u], Vr, "bf16", "live rows V")
