"""Benchmark of the LoCoCo chunk loop (Algorithm 2) on the Llama-2-7B-shaped layer.

One step = one pass of the whole hot path (chunk attention, conv logits, ReLU,
normalisation, both blends, for all 8 chunks) over one 4096-token sequence of a
32-head layer.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "chunk-step tokens/sec per layer (32 heads)"
UNIT = "tokens/s"
WORKLOAD = "cfg2"
WORKLOAD_TEXT = ("cfg2: Llama-2-7B-shaped layer, 32 heads, d=128, M=128, B=512, k=21, L=4096, batch 1 per GPU, "
                 "per-head conv weights, c_in=d")
# The ncu summary of the dominant kernel ends with one machine-readable line: the DRAM bytes of one launch
# (dram__bytes_read.sum + dram__bytes_write.sum) and a digest of the kernel sources at the time of the capture.
STEP_KERNEL_PROFILE = ROOT / "profiles" / "chunk_step_tc_kernel_cfg2.md"
STEP_KERNEL_SOURCES = ("tensor_forward.cu", "tc_common.cuh", "common.cuh")


def kernel_sources_digest():
    import hashlib
    h = hashlib.sha256()
    for name in STEP_KERNEL_SOURCES:
        h.update((ROOT / "paper_2406_05317_b200" / "csrc" / name).read_bytes())
    return h.hexdigest()[:16]


def step_kernel_traffic():
    """DRAM bytes per launch from the committed capture, or None when the kernel sources have changed since."""
    try:
        for line in STEP_KERNEL_PROFILE.read_text().splitlines():
            if line.startswith("traffic_table:"):
                t = json.loads(line[len("traffic_table:"):])
                return float(t["dram_bytes_per_launch"]) if t["sources_sha256_16"] == kernel_sources_digest() else None
    except Exception:
        pass
    return None


# ------------------------------------------------------------------ algorithmic work
def conv_flops(S, M, C, k):
    return 2.0 * S * M * C * k


def blend_flops(S, M, d):
    return 4.0 * M * S * d


def attn_flops(b, c, d):
    return 4.0 * b * (c + (b + 1) / 2.0) * d


def chunk_schedule(L, B, M):
    """(cache_len, b, compress?) for every chunk of Algorithm 2 from an empty cache."""
    out, c = [], 0
    for t0 in range(0, L, B):
        b = min(B, L - t0)
        comp = c + b > M
        out.append((c, b, comp))
        c = M if comp else c + b
    return out


def sequence_flops(w):
    """Algorithmic flops of one (sequence, head) unit: conv, blends, attention."""
    conv = blend = attn = 0.0
    for c, b, comp in chunk_schedule(w.L, w.B, w.M):
        attn += attn_flops(b, c, w.d)
        if comp:
            conv += conv_flops(c + b, w.M, w.c_in, w.k)
            blend += blend_flops(c + b, w.M, w.d)
    return conv, blend, attn


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        j = json.loads(p.read_text())
        return {"bf16_tflops": j["bf16_tflops"], "hbm_gbs": j["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


# ------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.proc, self.path = gpu_index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in open(self.path).read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ the oracle arm
def time_oracle(w, heads_sample, repeats=1):
    """Times the float64 CPU oracle, as it stands, on `heads_sample` heads of the workload.
    Returns (layer tokens/s scaled to all heads, seconds per sample run, threads)."""
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import workloads as wl
    ws = w.slice(heads=heads_sample)
    Q, K, V = wl.make_qkv(ws)
    G, _ = wl.make_weights(ws)
    times = []
    for _ in range(repeats):
        t = time.perf_counter()
        orc.process_batch(Q, K, V, G, ws.B)
        times.append(time.perf_counter() - t)
    dt = sum(times) / len(times)
    layer_seconds = dt * (w.heads / heads_sample)
    return w.batch * w.L / layer_seconds, times, orc.threads()


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, same metric and workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lococo_oracle as orc
    from paper_2406_05317_b200 import workloads as wl
    w = wl.CONFIGS[WORKLOAD]
    threads = orc.threads()
    # a step is the whole workload (all 32 heads, all 8 chunks): a few seconds of CPU work, nothing is scaled
    Q, K, V = wl.make_qkv(w)
    G, _ = wl.make_weights(w)
    for _ in range(args.warmup):
        orc.process_batch(Q, K, V, G, w.B)
    t = time.perf_counter()
    for _ in range(args.steps):
        orc.process_batch(Q, K, V, G, w.B)
    layer_ms = (time.perf_counter() - t) / args.steps * 1e3
    value = w.batch * w.L / (layer_ms / 1e3)
    sample = f"{w.heads} of {w.heads} heads, all {w.n_chunks} chunks (the whole workload), {layer_ms / 1e3:.1f} s per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": layer_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2406_05317_b200 import api, sharding, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    w = wl.CONFIGS[WORKLOAD]
    tdt = torch.bfloat16

    # weak scaling: every rank runs one whole sequence of its own (sequence index = rank)
    seq = list(sharding.weak_scaling_sequences(world, rank))[0]
    Qh, Kh, Vh = (torch.from_numpy(x[None]).to(tdt).pin_memory() for x in wl.make_sequence(w, seq))
    G, _ = wl.make_weights(w)
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=tdt, c_in=w.c_in, weights_per_head=w.weights_per_head)
    ctx.set_weights(torch.from_numpy(G).cuda().to(tdt))
    Q, K, V = Qh.cuda(), Kh.cuda(), Vh.cuda()
    O = torch.empty_like(Q)
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=tdt, device="cuda")
    Vc = torch.zeros_like(Kc)
    Oh = torch.empty_like(Qh).pin_memory()
    Kch = torch.empty(w.batch, w.heads, w.M, w.d, dtype=tdt).pin_memory()
    Vch = torch.empty_like(Kch).pin_memory()
    staging = torch.empty(ctx.host_staging_bytes(w.L), dtype=torch.uint8, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2

    # a side stream: the library replays the chunk loop from a CUDA graph on capturable streams only
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(side)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step_device():
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
        b.record()
        return a, b

    def step_host():
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.process_sequence_host(Qh, Kh, Vh, w.B, Oh, staging, Kch, Vch)
        b.record()
        return a, b

    for _ in range(args.warmup):
        step_device()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = ctx.launch_count()
    events = [step_device() for _ in range(args.steps)]
    barrier()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    local_ms = sum(a.elapsed_time(b) for a, b in events)
    assert ctx.device_status() == api.OK

    # per-kernel timing of the same steps (CUDA events on the launching stream, in the library)
    ctx.profile(True)
    for _ in range(args.steps):
        step_device()
    torch.cuda.synchronize()
    conv_ms, conv_n = ctx.profile_read(0)
    attn_ms, attn_n = ctx.profile_read(1)
    step_ms, step_n = ctx.profile_read(2)
    seq_ms, seq_n = ctx.profile_read(3)
    ctx.profile(False)

    # end to end through the host-buffer entry point
    for _ in range(min(args.warmup, 3)):
        step_host()
    barrier()
    e2e_steps = max(1, min(args.steps, 10))
    ev = [step_host() for _ in range(e2e_steps)]
    barrier()
    e2e_local_ms = sum(a.elapsed_time(b) for a, b in ev) * (args.steps / e2e_steps)

    tokens = float(w.batch * w.L * args.steps)
    total_ms, total_tokens = sharding.aggregate_throughput(dist if world > 1 else None, local_ms, tokens)
    e2e_ms, _ = sharding.aggregate_throughput(dist if world > 1 else None, e2e_local_ms, tokens)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    conv_f, blend_f, attn_f = sequence_flops(w)
    units = w.batch * w.heads
    n_comp = sum(1 for _, _, comp in chunk_schedule(w.L, w.B, w.M) if comp)
    # the dominant kernel: the per-chunk launch that holds attention, conv, normalisation and blends
    # (all chunks of this workload are compress steps); algorithmic flops per launch = the
    # per-unit figures of one chunk x 32 units
    if seq_n:
        kernel = "persistent chunk loop: all 8 steps of Alg. 2 (Eq. 1 attention, Eq. 6 conv, ReLU/Eq. 7, Eq. 4-5 blends) in one launch"
        dom_ms, dom_n, dom_flops_per_seq, n_comp = seq_ms, seq_n, units * (conv_f + blend_f + attn_f), 1
    elif step_n:
        kernel = "chunk step: Eq. 1 attention + Eq. 6 conv + ReLU/Eq. 7 + Eq. 4-5 blends (one launch)"
        dom_ms, dom_n, dom_flops_per_seq = step_ms, step_n, units * (conv_f + blend_f + attn_f)
    else:
        kernel = "Eq. 6 conv + ReLU/Eq. 7 + Eq. 4-5 blends"
        dom_ms, dom_n, dom_flops_per_seq = conv_ms, conv_n, units * (conv_f + blend_f)
    isolated_per_launch_ms = dom_ms / max(dom_n, 1)   # each launch bracketed by events of its own: no overlap with its neighbours
    # The loop's kernels overlap (programmatic dependent launches), so a launch has no duration of its own inside
    # the timed region: the dominant kernel is charged the whole region, finalize passes and hand-overs included.
    dom_per_launch_ms = (total_ms / args.steps) / n_comp if (step_n and not seq_n) else isolated_per_launch_ms
    flops_per_launch = dom_flops_per_seq / n_comp
    achieved = flops_per_launch / (dom_per_launch_ms * 1e-3) / 1e12 if dom_n else None
    step_flops = units * (conv_f + blend_f + attn_f)
    seq_bytes = 4.0 * units * w.L * w.d * 2 + units * 2 * w.M * w.d * 2 + w.heads * w.M * w.c_in * w.k * 2
    roof_ms = max(step_flops / (peaks["bf16_tflops"] * 1e12), seq_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3

    out = {
        "metric": METRIC, "value": total_tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT,
                   "l2": "256 MB flush between timed steps", "chunks_per_step": w.n_chunks,
                   "parallelism": f"sequences x{world} (no collective)"},
        "clocks": clocks,
        "e2e": {"value": total_tokens / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": 3 * Qh.numel() * 2, "d2h_bytes_per_step": (Oh.numel() + 2 * Kch.numel()) * 2},
        "gpu_launches": launches,
        "step_roofline": {"flops_per_step": step_flops, "bytes_per_step": seq_bytes, "roofline_ms": roof_ms,
                          "frac": roof_ms / (total_ms / args.steps), "peak_source": peaks["source"] + " burst"},
        "roofline": {"bound": "tensor", "kernel": kernel, "flops_per_launch": flops_per_launch,
                     "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": (achieved / peaks["bf16_tflops"]) if achieved else None,
                     "traffic": step_kernel_traffic() if (step_n and not seq_n) else None,
                     "peak_source": peaks["source"] + " burst", "launches": dom_n,
                     "us_per_launch": dom_per_launch_ms * 1e3, "us_per_launch_isolated": isolated_per_launch_ms * 1e3,
                     "duration": "timed region / launches of this kernel (its launches overlap their neighbours)"},
    }
    if world == 1:
        from oracle import lococo_oracle as orc
        threads = orc.threads()
        heads_sample = w.heads if threads >= 8 else max(1, min(w.heads, 2 * threads))
        value, times, threads = time_oracle(w, heads_sample)
        out["cpu_baseline"] = {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                               "sample": f"{heads_sample} of {w.heads} heads, all {w.n_chunks} chunks, "
                                         f"{times[0]:.1f} s, scaled by {w.heads}/{heads_sample}"}
        out["eager"] = time_eager(ctx, w, Q, K, V, flush)
        out["configs"] = {name: time_config(name) for name in ("cfg3", "cfg4")}
        out["backward"] = time_backward()
        out["layer_stack"] = time_layer_stack()
        out["generation"] = time_generation()
        out["sweep"] = time_sweep(full=args.sweep)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def time_eager(ctx, w, Q, K, V, flush, runs=10):
    """The headline workload without the CUDA-graph replay: every call gets output and cache tensors that
    differ from the previous call's, so the library launches the chunk loop kernel by kernel each time."""
    import torch
    sets = [(torch.empty_like(Q), torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda"),
             torch.zeros(w.batch, w.heads, w.M, w.d, dtype=Q.dtype, device="cuda")) for _ in range(2)]
    ms = 0.0
    for it in range(3 + runs):
        O, Kc, Vc = sets[it % 2]
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
        b.record()
        b.synchronize()
        if it >= 3:
            ms += a.elapsed_time(b) / runs
    return {"what": "same workload, no CUDA-graph replay (buffers change from call to call)", "ms_per_step": ms,
            "tokens_per_s": w.batch * w.L / (ms * 1e-3)}


def time_config(name, runs=5):
    """Whole lococo_process_sequence at another configuration: seeded inputs of the workload recipe, resident on
    the device, no cache snapshots, repeated identical calls on a side stream (CUDA-graph replay from the third),
    256 MB L2 flush between calls; roofline fraction as for the headline workload."""
    import torch

    from paper_2406_05317_b200 import api, workloads as wl
    w = wl.CONFIGS[name]
    tdt = torch.bfloat16
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=tdt, c_in=w.c_in, weights_per_head=w.weights_per_head)
    G, _ = wl.make_weights(w)
    ctx.set_weights(torch.from_numpy(G).cuda().to(tdt))
    Q = torch.empty(w.batch, w.heads, w.L, w.d, dtype=tdt, device="cuda")
    K, V, O = torch.empty_like(Q), torch.empty_like(Q), torch.empty_like(Q)
    for n in range(w.batch):                       # sequence by sequence: the host never holds the whole batch
        for dst, x in zip((Q, K, V), wl.make_sequence(w, n)):
            dst[n].copy_(torch.from_numpy(x).to(tdt))
    Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=tdt, device="cuda")
    Vc = torch.zeros_like(Kc)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    ms = 0.0
    launches0 = 0
    with torch.cuda.stream(side):
        for it in range(3 + runs):
            if it == 3:
                launches0 = ctx.launch_count()
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
            b.record()
            b.synchronize()
            if it >= 3:
                ms += a.elapsed_time(b) / runs
    assert ctx.device_status() == api.OK
    launches = (ctx.launch_count() - launches0) // runs
    conv_f, blend_f, attn_f = sequence_flops(w)
    units = w.batch * w.heads
    flops = units * (conv_f + blend_f + attn_f)
    sets = w.heads if w.weights_per_head else 1
    nbytes = 4.0 * units * w.L * w.d * 2 + units * 2 * w.M * w.d * 2 + sets * w.M * w.c_in * w.k * 2
    peaks = measured_peaks()
    roof_ms = max(flops / (peaks["bf16_tflops"] * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)) * 1e3
    return {"workload": f"{name}: batch {w.batch}, {w.heads} heads, d={w.d}, M={w.M}, B={w.B}, k={w.k}, L={w.L}, "
                        f"{'per-head' if w.weights_per_head else 'shared'} conv weights, c_in=d, seeded recipe",
            "ms_per_step": ms, "tokens_per_s": w.batch * w.L / (ms * 1e-3), "gpu_launches": launches,
            "flops_per_step": flops, "bytes_per_step": nbytes, "achieved_tflops": flops / (ms * 1e-3) / 1e12,
            "roofline_ms": roof_ms, "frac": roof_ms / ms, "bound": "tensor", "peak_source": peaks["source"] + " burst"}


def time_sweep(full=False, runs=3):
    """Kernel width and cache size (the paper's ablations over k and M, as a performance curve): one layer of 32
    heads, chunks of 512 tokens, weights shared by the heads, 4096 tokens per call; time per chunk step and
    TFLOP/s on algorithmic flops. Default: the corners k in {3, 21, 61} x M in {128, 512}; --sweep: the whole grid."""
    import torch

    from paper_2406_05317_b200 import api, workloads as wl
    base = wl.CONFIGS[WORKLOAD]
    ks = (3, 9, 21, 41, 61) if full else (3, 21, 61)
    Ms = (128, 256, 512, 1024) if full else (128, 512)
    g = torch.Generator(device="cuda").manual_seed(7300)
    shape = (base.batch, base.heads, base.L, base.d)
    Q, K, V = ((torch.randn(shape, device="cuda", generator=g) * base.qkv_scale).to(torch.bfloat16) for _ in range(3))
    O = torch.empty_like(Q)
    rows = []
    side = torch.cuda.Stream()
    for M in Ms:
        for k in ks:
            w = base.slice(M=M, k=k, weights_per_head=False)
            ctx = api.Lococo(w.batch, w.heads, w.d, M, k, w.B, dtype=torch.bfloat16, c_in=w.c_in, weights_per_head=False)
            ctx.set_weights((torch.randn((1, M, w.c_in, k), device="cuda", generator=g) * w.g_std).to(torch.bfloat16))
            Kc = torch.zeros(w.batch, w.heads, M, w.d, dtype=torch.bfloat16, device="cuda")
            Vc = torch.zeros_like(Kc)
            torch.cuda.synchronize()
            ms = 0.0
            with torch.cuda.stream(side):
                for it in range(3 + runs):
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
                    b.record()
                    b.synchronize()
                    if it >= 3:
                        ms += a.elapsed_time(b) / runs
            assert ctx.device_status() == api.OK
            conv_f, blend_f, attn_f = sequence_flops(w)
            flops = w.batch * w.heads * (conv_f + blend_f + attn_f)
            rows.append({"M": M, "k": k, "us_per_chunk_step": ms / w.n_chunks * 1e3,
                         "tflops": flops / (ms * 1e-3) / 1e12})
    return {"workload": f"{base.heads} heads, d={base.d}, B={base.B}, L={base.L}, shared conv weights, c_in=d; "
                        "whole lococo_process_sequence divided by its chunks", "rows": rows}


def time_backward(name="cfg5", runs=2):
    """Secondary figure (not the headline metric): forward with snapshots + backward through all chunk
    steps at the fine-tuning shape (cfg5 = cfg4 shapes), device-resident seeded inputs, CUDA events."""
    import torch

    from paper_2406_05317_b200 import api, workloads as wl
    w = wl.CONFIGS[name]
    ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in,
                     weights_per_head=w.weights_per_head)
    G, _ = wl.make_weights(w)
    ctx.set_weights(torch.from_numpy(G).cuda().to(torch.bfloat16))
    dev = lambda x: torch.from_numpy(x).cuda().to(torch.bfloat16)
    Q, K, V = (dev(x) for x in wl.make_qkv(w))                     # the seeded recipe (heavy-tailed keys)
    PO, PK, PV = (dev(x) for x in wl.make_loss_projections(w))
    cshape = (w.batch, w.heads, w.M, w.d)
    O, gQ, gK, gV = (torch.empty_like(Q) for _ in range(4))
    Kc, Vc = torch.zeros(cshape, dtype=torch.bfloat16, device="cuda"), torch.zeros(cshape, dtype=torch.bfloat16, device="cuda")
    gG = torch.zeros(G.shape, dtype=torch.float32, device="cuda")
    saved = torch.empty(ctx.saved_bytes(w.L, w.B), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(ctx.backward_scratch_bytes(w.L, w.B), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    fwd_ms = bwd_ms = 0.0
    with torch.cuda.stream(side):
        for it in range(1 + runs):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            Kc.zero_(); Vc.zero_()
            e[0].record()
            ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0, saved)
            e[1].record()
            ctx.process_sequence_backward(Q, K, V, O, w.B, saved, PO, PK, PV, gQ, gK, gV, gG, None, scratch)
            e[2].record()
            e[2].synchronize()
            if it:
                fwd_ms += e[0].elapsed_time(e[1]) / runs
                bwd_ms += e[1].elapsed_time(e[2]) / runs
    assert ctx.device_status() == api.OK
    conv_f, blend_f, attn_f = sequence_flops(w)
    fwd_flops = w.batch * w.heads * (conv_f + blend_f + attn_f)
    # recompute of the conv + two conv-sized gradients, two blend-sized pairs, 2.5 x the attention
    bwd_flops = w.batch * w.heads * (3.0 * conv_f + 2.0 * blend_f + 2.5 * attn_f)
    peaks = measured_peaks()
    return {"workload": f"{name}: 32 heads, d=128, M={w.M}, B={w.B}, k={w.k}, L={w.L}, shared conv weights, forward with cache "
                        "snapshots + backward through all chunk steps", "forward_ms": fwd_ms, "backward_ms": bwd_ms,
            "tokens_per_s_fwd_bwd": w.batch * w.L / ((fwd_ms + bwd_ms) * 1e-3),
            "backward_tflops": bwd_flops / (bwd_ms * 1e-3) / 1e12, "backward_frac_of_peak": bwd_flops / (bwd_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "forward_tflops": fwd_flops / (fwd_ms * 1e-3) / 1e12}


def time_layer_stack(layers=32, runs=3):
    """Secondary figure: the paper's own setting (Section 4.1: one conv weight set per layer shared by its heads,
    keys stacked on values as the conv input) for a whole 32-layer prefill of 4096 tokens, one layer after the
    other on one stream; the projections and MLPs around the attention are not part of this library."""
    import torch

    from paper_2406_05317_b200 import api, workloads as wl
    w = wl.CONFIGS[WORKLOAD].slice(c_in_mult=2)
    g = torch.Generator(device="cuda").manual_seed(7000)
    shape = (w.batch, w.heads, w.L, w.d)
    Q, K, V = ((torch.randn(shape, device="cuda", generator=g) * w.qkv_scale).to(torch.bfloat16) for _ in range(3))
    O = torch.empty_like(Q)
    ctxs, caches = [], []
    for _ in range(layers):
        ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, w.B, dtype=torch.bfloat16, c_in=w.c_in, weights_per_head=False)
        ctx.set_weights((torch.randn((1, w.M, w.c_in, w.k), device="cuda", generator=g) * w.g_std).to(torch.bfloat16))
        ctxs.append(ctx)
        caches.append((torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda"),
                       torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda")))
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    ms = 0.0
    with torch.cuda.stream(side):
        for it in range(3 + runs):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for ctx, (Kc, Vc) in zip(ctxs, caches):
                ctx.process_sequence(Q, K, V, w.B, O, Kc, Vc, 0)
            b.record()
            b.synchronize()
            if it >= 3:
                ms += a.elapsed_time(b) / runs
    assert all(c.device_status() == api.OK for c in ctxs)
    return {"workload": f"{layers} layers x ({WORKLOAD} shapes, conv weights shared by the heads of a layer, c_in = 2d), 4096-token prefill",
            "ms": ms, "ms_per_layer": ms / layers, "tokens_per_s_all_layers": w.batch * w.L / (ms * 1e-3)}


def time_generation(batches=(1, 16, 64), steps=256, runs=3):
    """Secondary figure: the generation stage (Section 3.3: chunks of one token on a full cache, every step
    recomputes all M slots from S = M + 1 entries), cfg2's layer shape with the weights shared by the heads,
    `steps` token steps per call after the cache has been filled."""
    import torch

    from paper_2406_05317_b200 import api, workloads as wl
    base = wl.CONFIGS[WORKLOAD]
    res = []
    for batch in batches:
        w = base.slice(batch=batch, B=1, L=base.M + steps)
        g = torch.Generator(device="cuda").manual_seed(7100 + batch)
        shape = (w.batch, w.heads, w.L, w.d)
        Q, K, V = ((torch.randn(shape, device="cuda", generator=g) * w.qkv_scale).to(torch.bfloat16) for _ in range(3))
        O = torch.empty_like(Q)
        ctx = api.Lococo(w.batch, w.heads, w.d, w.M, w.k, 1, dtype=torch.bfloat16, c_in=w.c_in, weights_per_head=False)
        ctx.set_weights((torch.randn((1, w.M, w.c_in, w.k), device="cuda", generator=g) * w.g_std).to(torch.bfloat16))
        Kc = torch.zeros(w.batch, w.heads, w.M, w.d, dtype=torch.bfloat16, device="cuda")
        Vc = torch.zeros_like(Kc)
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        ms = 0.0
        with torch.cuda.stream(side):
            M = w.M
            c = ctx.process_sequence(Q[:, :, :M], K[:, :, :M], V[:, :, :M], 1, O[:, :, :M], Kc, Vc, 0)   # fill steps
            for it in range(2 + runs):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                ctx.process_sequence(Q[:, :, M:], K[:, :, M:], V[:, :, M:], 1, O[:, :, M:], Kc, Vc, c)
                b.record()
                b.synchronize()
                if it >= 2:
                    ms += a.elapsed_time(b) / runs
        assert ctx.device_status() == api.OK
        step_flops = batch * w.heads * (conv_flops(w.M + 1, w.M, w.c_in, w.k) + blend_flops(w.M + 1, w.M, w.d) + attn_flops(1, w.M, w.d))
        res.append({"batch": batch, "us_per_token_step": ms / steps * 1e3, "tokens_per_s": batch * steps / (ms * 1e-3),
                    "tflops": step_flops / (ms / steps * 1e-3) / 1e12})
    return {"workload": f"chunks of one token on a full cache, {base.heads} heads, d={base.d}, M={base.M}, k={base.k}, "
                        f"shared conv weights, {steps} token steps per call", "runs": res}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="time the whole kernel-width x cache-size grid, not its corners")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
