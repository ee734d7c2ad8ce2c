"""Parity of the CUDA path (through the C ABI) with the float64 CPU oracle, element by
element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2406_05317_b200 import workloads as wl
from tests.helpers import assert_close, to_device, to_host, torch_dtype

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2406_05317_b200 import api as _api
    return _api


@pytest.fixture(scope="module")
def orc():
    from oracle import lococo_oracle
    return lococo_oracle


def make_ctx(api, w, path=0, bias=False, norm_eps=1e-6, max_chunk=None):
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, max_chunk or w.B, dtype=torch_dtype(w.dtype), c_in=w.c_in,
                     weights_per_head=w.weights_per_head, norm_eps=norm_eps, path=path)
    G, bvec = wl.make_weights(w, with_bias=bias)
    ctx.set_weights(to_device(G, w.dtype), None if bvec is None else to_device(bvec, w.dtype))
    return ctx, G, bvec


def run_sequence(api, w, path=0, bias=False):
    """GPU process_sequence on workload w; returns numpy O, Kc, Vc, c."""
    ctx, G, bvec = make_ctx(api, w, path, bias)
    Q, K, V = wl.make_qkv(w)
    dQ, dK, dV = (to_device(x, w.dtype) for x in (Q, K, V))
    O = torch.empty_like(dQ)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=dQ.dtype, device="cuda")
    Vc = torch.zeros_like(Kc)
    c = ctx.process_sequence(dQ, dK, dV, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    assert ctx.launch_count() > 0
    return to_host(O), to_host(Kc), to_host(Vc), c


_oracle_cache = {}


def oracle_sequence(orc, w, bias=False):
    """The oracle on workload w (cached: the same workload is checked on several paths)."""
    key = (w, bias)
    if key not in _oracle_cache:
        Q, K, V = wl.make_qkv(w)
        G, bvec = wl.make_weights(w, with_bias=bias)
        _oracle_cache[key] = orc.process_batch(Q, K, V, G, w.B, bias=bvec)[:4]
    return _oracle_cache[key]


def check_sequence(api, orc, w, path=0, bias=False):
    O, Kc, Vc, c = run_sequence(api, w, path, bias)
    Or, Kr, Vr, cr = oracle_sequence(orc, w, bias)
    assert (cr == c).all()
    assert_close(O, Or, w.dtype, f"{w.name} O")
    assert_close(Kc[:, :, :c], Kr[:, :, :c], w.dtype, f"{w.name} K cache")
    assert_close(Vc[:, :, :c], Vr[:, :, :c], w.dtype, f"{w.name} V cache")


# ---------------------------------------------------------------- whole loop
@pytest.mark.parametrize("path", [0, 1])
def test_cfg1_tiny_fp32_full(api, orc, path):
    check_sequence(api, orc, wl.CONFIGS["cfg1"], path)


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("c_mult", [1, 2])
def test_cfg2_slice(api, orc, path, c_mult):
    # Llama-2-7B inference shape, 3 of the 32 heads, all 8 chunks
    check_sequence(api, orc, wl.CONFIGS["cfg2"].slice(heads=3, c_in_mult=c_mult), path)


@pytest.mark.parametrize("path", [0, 1])
def test_cfg3_slice(api, orc, path):
    # streaming shape: 2 sequences x 2 heads, 32 chunks (2 fills + 30 compress steps)
    check_sequence(api, orc, wl.CONFIGS["cfg3"].slice(batch=2, heads=2, L=2048), path)


@pytest.mark.parametrize("path", [0, 1])
def test_cfg4_slice(api, orc, path):
    # fine-tuning shape M=512, shortened chunks so the oracle finishes in seconds:
    # B=1024 keeps S = 1536 spanning several tiles of every kernel
    check_sequence(api, orc, wl.CONFIGS["cfg4"].slice(heads=2, B=1024, L=3072), path)


@pytest.mark.parametrize("B", [256, 320])
def test_two_position_tiles_per_unit(api, orc, B):
    # S = 384 or 448: two compress CTAs per unit, so the one that arrives last merges ONE stored set with its own
    # (the shortest run of the merge's buffer ring); 448 = 2 x 224 has no ragged last tile, 384 has one
    check_sequence(api, orc, wl.CONFIGS["cfg2"].slice(heads=3, B=B, L=4 * B + 96), 0)


def test_tensor_path_ragged_chunks_direct_cache_write(api, orc):
    # tensor-core path with sizes that are multiples of nothing the kernels tile by: B = 100, a short last
    # chunk, a first compress step on a partly filled cache (c = 100), several sequences; with this many
    # units every compress CTA sees all positions of its slots and writes the new cache itself, so the loop
    # alternates between the caller's cache and the workspace's (11 compress steps: the result ends up in
    # the workspace's cache and is copied back)
    w = wl.Workload("tc_ragged", 13, batch=3, heads=2, d=128, M=128, B=100, k=9, L=1177, dtype="bf16",
                    weights_per_head=True, qkv_scale=0.0884, g_std=0.02)
    check_sequence(api, orc, w, 0, bias=True)


@pytest.mark.parametrize("path", [0, 1])
def test_generation_mode_chunk_of_one_token(api, orc, path):
    # B = 1 (the generation stage of Section 3.3 sets the segment length to 1): 128 fill steps, then every step compresses
    # S = M + 1 positions back into M slots
    w = wl.Workload("decode", 12, batch=2, heads=2, d=128, M=128, B=1, k=21, L=160, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02)
    check_sequence(api, orc, w, path)


@pytest.mark.parametrize("batch,heads,B,per_head,c_mult,L", [
    (16, 32, 1, False, 1, 136),     # the generation stage at batch 16: 512 units, 256 two-unit CTAs, 8 steps
    (5, 32, 1, True, 1, 134),       # a set per head, odd batch: the last pair of every head has one unit
    (5, 31, 1, False, 1, 134),      # odd number of units with shared weights
    (5, 32, 4, False, 1, 144),      # chunks of 4 tokens: two-unit compress CTAs, tensor-core attention
    (5, 32, 16, True, 1, 176),      # chunks of 16: S = 144, the widest tile of the two-unit form
    (2, 2, 1, False, 1, 140),       # fewer units than SMs: one unit per compress CTA, warp-per-unit attention
    (5, 32, 1, False, 2, 132),      # keys stacked on values: the one-unit form, warp-per-unit attention
])
def test_generation_stage_two_units_per_cta(api, orc, batch, heads, B, per_head, c_mult, L):
    # Section 3.3: in the generation stage the segment length is 1. Short chunks on a full cache of M = 128 slots run
    # the compress step with two units per CTA (shared weight stages) and, for one query, attention with a warp per unit.
    # With random weights and token-by-token steps the slots soon resemble one another and whole rows of logits sit
    # close to zero, where Eq. 7 is discontinuous (a row with no positive logit is a zero slot, a row with one tiny
    # positive logit is that token): a positive bias keeps the rows away from that edge, so that the comparison
    # measures the arithmetic and not the conditioning of the input.
    w = wl.Workload(f"gen{batch}x{heads}b{B}", 14, batch=batch, heads=heads, d=128, M=128, B=B, k=21, L=L, dtype="bf16",
                    weights_per_head=per_head, qkv_scale=0.0884, g_std=0.02, c_in_mult=c_mult)
    G, _ = wl.make_weights(w)
    bvec = wl.round_to_bf16(np.full((heads if per_head else 1, w.M), 0.05, dtype=np.float32))
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in, weights_per_head=per_head)
    ctx.set_weights(to_device(G, "bf16"), to_device(bvec, "bf16"))
    Qh, Kh, Vh = wl.make_qkv(w)
    Q, K, V = (to_device(x, "bf16") for x in (Qh, Kh, Vh))
    O = torch.empty_like(Q)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
    Vc = torch.zeros_like(Kc)
    assert ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0) == w.M
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK
    Or, Kr, Vr, cr, _ = orc.process_batch(Qh, Kh, Vh, G, w.B, bias=bvec)
    assert_close(to_host(O), Or, "bf16", f"{w.name} O")
    assert_close(to_host(Kc), Kr, "bf16", f"{w.name} K cache")
    assert_close(to_host(Vc), Vr, "bf16", f"{w.name} V cache")


def test_generation_stage_bit_identical_across_unit_pairings(api):
    # a unit's result must not depend on which unit shares its CTA: the same six sequences in another order
    # (units are paired with their neighbours in the batch)
    w = wl.Workload("gen_pairs", 15, batch=6, heads=32, d=128, M=128, B=1, k=21, L=134, dtype="bf16",
                    weights_per_head=False, qkv_scale=0.0884, g_std=0.02)
    Q, K, V = (to_device(x, w.dtype) for x in wl.make_qkv(w))
    ctx, _, _ = make_ctx(api, w)
    outs = []
    for order in ([0, 1, 2, 3, 4, 5], [3, 0, 5, 1, 4, 2]):
        q, k, v = (x[order].contiguous() for x in (Q, K, V))
        O = torch.empty_like(q)
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=q.dtype, device="cuda")
        Vc = torch.zeros_like(Kc)
        assert ctx.process_sequence(q, k, v, w.B, O, Kc, Vc, 0) == w.M
        torch.cuda.synchronize()
        back = torch.argsort(torch.tensor(order))
        outs.append((O[back], Kc[back], Vc[back]))
    assert ctx.device_status() == api.OK
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_everything(api, orc, dtype):
    # sizes that are multiples of nothing: M=40, B=37, L=301 (last chunk short), k=7,
    # bias, per-head weights, c_in = 2d
    w = wl.Workload("ragged", 9, batch=2, heads=3, d=64, M=40, B=37, k=7, L=301, dtype=dtype,
                    weights_per_head=True, qkv_scale=1.0, g_std=0.05, c_in_mult=2)
    check_sequence(api, orc, w, 0, bias=True)


def test_short_sequence_is_full_attention(api, orc):
    # L <= M: only the fill branch runs
    w = wl.Workload("short", 10, batch=1, heads=2, d=128, M=128, B=48, k=21, L=100, dtype="bf16",
                    weights_per_head=False, qkv_scale=1.0)
    check_sequence(api, orc, w, 0)


def test_suspend_resume_bit_identical(api):
    w = wl.CONFIGS["cfg2"].slice(heads=2, L=2048)
    ctx, G, _ = make_ctx(api, w)
    Q, K, V = (to_device(x, w.dtype) for x in wl.make_qkv(w))

    def run(splits):
        O = torch.empty_like(Q)
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
        Vc = torch.zeros_like(Kc)
        c, t0 = 0, 0
        for n in splits:
            sl = slice(t0, t0 + n)
            c = ctx.process_sequence(Q[:, :, sl], K[:, :, sl], V[:, :, sl], w.B, O[:, :, sl], Kc, Vc, c)
            t0 += n
        torch.cuda.synchronize()
        return O, Kc, Vc, c

    a, b = run([2048]), run([1024, 1024])
    assert a[3] == b[3]
    for x, y in zip(a[:3], b[:3]):
        assert torch.equal(x, y)


# ---------------------------------------------------------------- single calls
@pytest.mark.parametrize("dtype,d,M,k,c,b,c_mult,per_head,bias", [
    ("f32", 64, 16, 5, 16, 16, 1, False, False),
    ("f32", 128, 24, 3, 10, 30, 2, True, True),
    ("bf16", 128, 128, 21, 128, 512, 1, True, False),
    ("bf16", 128, 128, 21, 0, 512, 2, False, False),
    ("bf16", 128, 128, 21, 128, 64, 1, False, True),
    ("bf16", 64, 72, 9, 50, 171, 1, False, False),
    ("bf16", 128, 512, 21, 512, 700, 1, False, False),
])
def test_compress_step_and_weights(api, orc, dtype, d, M, k, c, b, c_mult, per_head, bias):
    w = wl.Workload("step", 11, batch=1, heads=2, d=d, M=M, B=b, k=k, L=b, dtype=dtype, weights_per_head=per_head,
                    qkv_scale=1.0, c_in_mult=c_mult)
    ctx, G, bvec = make_ctx(api, w, bias=bias)
    _, Kn, Vn = wl.make_qkv(w)
    wc = w.slice(L=max(c, 1), seed0=77)
    _, Kc, Vc = wl.make_qkv(wc)
    Kc_full = np.zeros((w.batch, w.heads, M, d), np.float32)
    Vc_full = np.zeros_like(Kc_full)
    Kc_full[:, :, :c], Vc_full[:, :, :c] = Kc[:, :, :c], Vc[:, :, :c]
    dKc, dVc, dKn, dVn = (to_device(x, dtype) for x in (Kc_full, Vc_full, Kn, Vn))
    Ko, Vo = torch.zeros_like(dKc), torch.zeros_like(dVc)
    S = c + b
    W = torch.zeros(w.batch, w.heads, M, S, dtype=torch.float32, device="cuda")
    new_len = ctx.compress_step(dKc, dVc, c, dKn, dVn, Ko, Vo, W)
    torch.cuda.synchronize()
    assert new_len == M and ctx.device_status() == api.OK
    Ko_h, Vo_h, W_h = to_host(Ko), to_host(Vo), to_host(W)
    for n in range(w.batch):
        for h in range(w.heads):
            XK = np.vstack([Kc_full[n, h, :c], Kn[n, h]])
            XV = np.vstack([Vc_full[n, h, :c], Vn[n, h]])
            Kr, Vr, wr, _, _ = orc.compress(XK, XV, G[h if per_head else 0],
                                            bias=None if bvec is None else bvec[h if per_head else 0],
                                            want_weights=True)
            assert_close(Ko_h[n, h], Kr, dtype, "K slots")
            assert_close(Vo_h[n, h], Vr, dtype, "V slots")
            assert_close(W_h[n, h], wr, dtype, "mixing weights")
            assert np.abs(W_h[n, h].sum(1) - 1).max() <= 1e-3       # Eq. 7: rows sum to one
    # in-place update gives the same slots
    ctx.compress_step(dKc, dVc, c, dKn, dVn)
    torch.cuda.synchronize()
    assert torch.equal(dKc, Ko) and torch.equal(dVc, Vo)


@pytest.mark.parametrize("dtype,d,c,b", [("f32", 64, 16, 16), ("f32", 128, 0, 45), ("bf16", 128, 128, 512),
                                         ("bf16", 128, 0, 512), ("bf16", 128, 128, 1), ("bf16", 64, 37, 203),
                                         ("bf16", 128, 512, 1100)])
def test_chunk_attention(api, orc, dtype, d, c, b):
    M = max(c, 16)
    w = wl.Workload("attn", 12, batch=2, heads=2, d=d, M=M, B=b, k=3, L=b, dtype=dtype, weights_per_head=False,
                    qkv_scale=1.0)
    ctx = api.Lococo(w.batch, w.heads, d, M, 3, b, dtype=torch_dtype(dtype))
    Q, Kn, Vn = wl.make_qkv(w)
    _, Kc, Vc = wl.make_qkv(w.slice(L=M, seed0=5))
    dQ, dKn, dVn, dKc, dVc = (to_device(x, dtype) for x in (Q, Kn, Vn, Kc, Vc))
    O = torch.empty_like(dQ)
    lse = torch.empty(w.batch, w.heads, b, dtype=torch.float32, device="cuda")
    ctx.chunk_attention(dQ, dKc, dVc, c, dKn, dVn, O, lse)
    torch.cuda.synchronize()
    O_h, lse_h = to_host(O), to_host(lse)
    for n in range(w.batch):
        for h in range(w.heads):
            Or, lr = orc.attention(Q[n, h], np.vstack([Kc[n, h, :c], Kn[n, h]]), np.vstack([Vc[n, h, :c], Vn[n, h]]), c)
            assert_close(O_h[n, h], Or, dtype, "O")
            assert np.abs(lse_h[n, h] - lr).max() <= (2e-2 if dtype == "bf16" else 1e-4 * max(1, np.abs(lr).max()))


def test_strided_views_and_fill_to_other_buffer(api, orc):
    # Q/K/V as slices of one packed [batch, tokens, 3, heads, d] projection output
    w = wl.Workload("strided", 13, batch=2, heads=2, d=64, M=32, B=24, k=5, L=120, dtype="bf16",
                    weights_per_head=False, qkv_scale=1.0)
    ctx, G, _ = make_ctx(api, w)
    Q, K, V = wl.make_qkv(w)
    packed = torch.empty(w.batch, w.L, 3, w.heads, w.d, dtype=torch.bfloat16, device="cuda")
    for i, x in enumerate((Q, K, V)):
        packed[:, :, i] = to_device(x, "bf16").permute(0, 2, 1, 3)
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    assert not q.is_contiguous()
    O = torch.empty(w.batch, w.L, w.heads, w.d, dtype=torch.bfloat16, device="cuda").permute(0, 2, 1, 3)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    ctx.process_sequence(q, k, v, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    Or, Kr, Vr, cr, _ = orc.process_batch(Q, K, V, G, w.B)
    assert_close(to_host(O), Or, "bf16", "O (strided)")
    assert_close(to_host(Kc), Kr, "bf16", "K cache")
    # fill branch into a different output buffer carries the old rows over
    Kc2, Vc2 = torch.zeros_like(Kc), torch.zeros_like(Vc)
    Ko, Vo = torch.full_like(Kc, 7.0), torch.full_like(Vc, 7.0)
    Kc2[:, :, :5], Vc2[:, :, :5] = 1.0, 2.0
    n = ctx.compress_step(Kc2, Vc2, 5, k[:, :, :10], v[:, :, :10], Ko, Vo)
    torch.cuda.synchronize()
    assert n == 15
    assert torch.equal(Ko[:, :, :5], Kc2[:, :, :5]) and torch.equal(Ko[:, :, 5:15], k[:, :, :10])
    assert torch.equal(Vo[:, :, 5:15], v[:, :, :10]) and (Ko[:, :, 15:] == 7.0).all()


def test_host_entry_point_matches_device_entry_point(api):
    w = wl.CONFIGS["cfg2"].slice(heads=2, L=1536)
    ctx, G, _ = make_ctx(api, w)
    Q, K, V = wl.make_qkv(w)
    hq, hk, hv = (to_device(x, w.dtype).cpu().pin_memory() for x in (Q, K, V))
    ho = torch.empty_like(hq).pin_memory()
    hkc = torch.empty(w.batch, w.heads, w.M, w.d, dtype=hq.dtype).pin_memory()
    hvc = torch.empty_like(hkc).pin_memory()
    staging = torch.empty(ctx.host_staging_bytes(w.L), dtype=torch.uint8, device="cuda")
    c = ctx.process_sequence_host(hq, hk, hv, w.B, ho, staging, hkc, hvc)
    dq, dk, dv = hq.cuda(), hk.cuda(), hv.cuda()
    O = torch.empty_like(dq)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=dq.dtype, device="cuda")
    Vc = torch.zeros_like(Kc)
    c2 = ctx.process_sequence(dq, dk, dv, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    assert c == c2 == w.M
    assert torch.equal(ho, O.cpu()) and torch.equal(hkc, Kc.cpu()) and torch.equal(hvc, Vc.cpu())


def test_runtime_argument_errors_launch_nothing(api):
    w = wl.CONFIGS["cfg1"]
    ctx, G, _ = make_ctx(api, w)
    x = torch.zeros(1, 1, 16, 64, device="cuda")
    before = ctx.launch_count()
    with pytest.raises(api.LococoError) as e:
        ctx.compress_step(x, x.clone(), 17, x.clone(), x.clone())
    assert e.value.status == api.ERR_INVALID_ARG
    with pytest.raises(api.LococoError):
        ctx.chunk_attention(x, x.clone(), x.clone(), 0, x.clone(), x.clone(), x)       # O aliases Q
    big = torch.zeros(1, 1, 32, 64, device="cuda")
    with pytest.raises(api.LococoError):
        ctx.chunk_attention(big, x, x.clone(), 0, big.clone(), big.clone(), big.clone())  # b > max_chunk
    with pytest.raises(api.LococoError):
        ctx.compress_step(x[:, :, :, 1:], x.clone(), 0, x.clone(), x.clone())             # misaligned view
    assert ctx.launch_count() == before


def test_repeated_identical_calls_replay_the_same_loop(api):
    # the same argument set called again and again (a serving loop over fixed buffers) is replayed
    # from a cached CUDA graph: results must not change, and new buffer CONTENTS must be seen
    w = wl.CONFIGS["cfg2"].slice(heads=2, L=1536)
    ctx, G, _ = make_ctx(api, w)
    Q, K, V = (to_device(x, w.dtype) for x in wl.make_qkv(w))
    O = torch.empty_like(Q)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
    Vc = torch.zeros_like(Kc)
    outs = []
    side = torch.cuda.Stream()          # graphs need a capturable stream, not the legacy default one
    torch.cuda.synchronize()
    for _ in range(4):
        before = ctx.launch_count()
        with torch.cuda.stream(side):
            c = ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
        torch.cuda.synchronize()
        outs.append((O.clone(), Kc.clone(), Vc.clone(), c, ctx.launch_count() - before))
    for o in outs[1:]:
        assert torch.equal(o[0], outs[0][0]) and torch.equal(o[1], outs[0][1]) and torch.equal(o[2], outs[0][2])
        assert o[3] == outs[0][3] == w.M and o[4] == outs[0][4] > 0
    # same buffers, new contents: a fresh context (eager path) must agree with the replay
    Q2, K2, V2 = (to_device(x, w.dtype) for x in wl.make_qkv(w.slice(seed0=4242)))
    Q.copy_(Q2); K.copy_(K2); V.copy_(V2)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
    torch.cuda.synchronize()
    ctx2, _, _ = make_ctx(api, w)
    O2, Kc2, Vc2 = torch.empty_like(Q), torch.zeros_like(Kc), torch.zeros_like(Vc)
    ctx2.process_sequence(Q2, K2, V2, w.B, O2, Kc2, Vc2, 0)
    torch.cuda.synchronize()
    assert torch.equal(O, O2) and torch.equal(Kc, Kc2) and torch.equal(Vc, Vc2)
    assert ctx.device_status() == api.OK


def test_persistent_loop_equals_stepwise_launches(api):
    # PATH_TENSOR_PERSISTENT runs the compress steps of a call inside one persistent kernel; the
    # default tensor-core path launches every step: same CTA bodies, same bits, fewer launches
    w = wl.CONFIGS["cfg3"].slice(batch=2, heads=4, L=1024)     # 2 fill steps, then 14 compress steps
    Q, K, V = (to_device(x, w.dtype) for x in wl.make_qkv(w))
    res = []
    for path in (api.PATH_TENSOR_PERSISTENT, api.PATH_TENSOR):
        ctx, G, _ = make_ctx(api, w, path=path)
        O = torch.empty_like(Q)
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
        Vc = torch.zeros_like(Kc)
        before = ctx.launch_count()
        c = ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
        torch.cuda.synchronize()
        assert ctx.device_status() == api.OK
        res.append((O, Kc, Vc, c, ctx.launch_count() - before))
    assert res[0][3] == res[1][3] == w.M
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1]) and torch.equal(res[0][2], res[1][2])
    assert res[0][4] < res[1][4]        # one persistent launch instead of two per step


def test_persistent_loop_repeated_calls_survive_other_calls_on_the_handle(api):
    # The persistent kernel's step descriptors travel through a small ring of pinned host slots. Identical
    # calls repeated on a side stream (where the per-chunk path would replay a CUDA graph), with a host-buffer
    # call of more chunks than the ring has slots in between, must keep giving the same bits.
    w = wl.CONFIGS["cfg2"].slice(heads=2, L=3072)      # 6 chunks
    Qh, Kh, Vh = wl.make_qkv(w)
    Q, K, V = (to_device(x, w.dtype) for x in (Qh, Kh, Vh))
    ctx, _, _ = make_ctx(api, w, path=api.PATH_TENSOR_PERSISTENT)
    side = torch.cuda.Stream()

    def call():
        O = torch.empty_like(Q)
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
        Vc = torch.zeros_like(Kc)
        return O, Kc, Vc

    O, Kc, Vc = call()
    outs = []
    torch.cuda.synchronize()
    for rep in range(5):
        if rep == 3:
            pin = lambda x: torch.from_numpy(x).to(torch.bfloat16).pin_memory()
            hO = torch.empty(Q.shape, dtype=torch.bfloat16).pin_memory()
            staging = torch.empty(ctx.host_staging_bytes(w.L) + 256, dtype=torch.uint8, device="cuda")
            off = (-staging.data_ptr()) % 256
            with torch.cuda.stream(side):
                ctx.process_sequence_host(pin(Qh), pin(Kh), pin(Vh), w.B, hO, staging[off:])
            host_O = hO.clone()
        Kc.zero_(); Vc.zero_()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            assert ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0) == w.M
        torch.cuda.synchronize()
        outs.append((O.clone(), Kc.clone(), Vc.clone()))
    assert ctx.device_status() == api.OK
    for o, k, v in outs[1:]:
        assert torch.equal(o, outs[0][0]) and torch.equal(k, outs[0][1]) and torch.equal(v, outs[0][2])
    assert torch.equal(host_O, outs[0][0].cpu())


@pytest.mark.parametrize("heads,L", [(32, 1536), (4, 2048)])
def test_merged_cache_update_has_the_bits_of_the_persistent_kernel(api, heads, L):
    # With several compress CTAs per (unit, slot block) the chunk loop lets the last of them sum the partial
    # blends and write the cache rows (one launch per chunk). The persistent kernel cuts the positions into the
    # same tiles and rebuilds the cache from the same partial sets in its own way: the two must agree bit for bit.
    # (The stand-alone entry points plan their tiles for a launch of their own, so their sums are ordered differently.)
    w = wl.CONFIGS["cfg2"].slice(heads=heads, L=L)
    Q, K, V = (to_device(x, w.dtype) for x in wl.make_qkv(w))
    n_chunks = L // w.B

    def fresh():
        O = torch.empty_like(Q)
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")
        return O, Kc, torch.zeros_like(Kc)

    # the chunk loop (merge inside the step kernel)
    ctx, _, _ = make_ctx(api, w, path=api.PATH_TENSOR)
    O1, Kc1, Vc1 = fresh()
    before = ctx.launch_count()
    c1 = ctx.process_sequence(Q, K, V, w.B, O1, Kc1, Vc1, 0)
    torch.cuda.synchronize()
    assert ctx.device_status() == api.OK and c1 == w.M
    # one launch per chunk, plus the copy back from the second cache after an odd number of steps
    assert ctx.launch_count() - before == n_chunks + (n_chunks % 2)

    # the persistent kernel
    ctx3, _, _ = make_ctx(api, w, path=api.PATH_TENSOR_PERSISTENT)
    O3, Kc3, Vc3 = fresh()
    ctx3.process_sequence(Q, K, V, w.B, O3, Kc3, Vc3, 0)
    torch.cuda.synchronize()
    assert ctx3.device_status() == api.OK
    assert torch.equal(O1, O3) and torch.equal(Kc1, Kc3) and torch.equal(Vc1, Vc3)
