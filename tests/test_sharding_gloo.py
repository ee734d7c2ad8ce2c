"""The multi-GPU host logic on CPU: two gloo ranks shard the (sequence, head) units with no
data-path collective in the forward, sum the shared conv-weight gradient in the backward,
and aggregate timings as max over ranks. The per-rank computation is the CPU oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2406_05317_b200 import sharding, workloads as wl


def test_shard_range_is_a_balanced_partition():
    for n, world in [(32, 2), (32, 8), (7, 3), (3, 4), (512, 8)]:
        parts = [sharding.shard_range(n, world, r) for r in range(world)]
        assert [i for p in parts for i in p] == list(range(n))
        sizes = [len(p) for p in parts]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)
    assert list(sharding.weak_scaling_sequences(4, 2)) == [2]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import lococo_oracle as orc
        w = wl.Workload("shard", 41, batch=1, heads=4, d=16, M=8, B=6, k=3, L=30, dtype="f32",
                        weights_per_head=False, qkv_scale=1.0, g_std=0.3)
        Q, K, V = wl.make_qkv(w)
        G, _ = wl.make_weights(w)
        PO, PK, PV = wl.make_loss_projections(w)
        mine = sharding.shard_range(w.heads, world, rank)
        sl = slice(mine.start, mine.stop)
        # forward: head shard, no collective
        O, Kc, Vc, c, _ = orc.process_batch(Q[:, sl], K[:, sl], V[:, sl], G, w.B)
        # backward: local dG, then the one exchange step
        dQ, dK, dV, dG, _ = orc.grad_batch(Q[:, sl], K[:, sl], V[:, sl], G, w.B, PO[:, sl], PK[:, sl], PV[:, sl])
        dG_t = torch.from_numpy(dG.copy())
        sharding.allreduce_weight_gradient(dist, dG_t)
        ms, units = sharding.aggregate_throughput(dist, 10.0 * (rank + 1), float(len(mine) * w.L))
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), O=O, dQ=dQ, dG=dG_t.numpy(), ms=ms, units=units,
                 start=mine.start, stop=mine.stop)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_heads_and_sum_weight_gradient(tmp_path):
    from oracle import lococo_oracle as orc
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    w = wl.Workload("shard", 41, batch=1, heads=4, d=16, M=8, B=6, k=3, L=30, dtype="f32",
                    weights_per_head=False, qkv_scale=1.0, g_std=0.3)
    Q, K, V = wl.make_qkv(w)
    G, _ = wl.make_weights(w)
    PO, PK, PV = wl.make_loss_projections(w)
    O, *_ = orc.process_batch(Q, K, V, G, w.B)
    dQ, dK, dV, dG, _ = orc.grad_batch(Q, K, V, G, w.B, PO, PK, PV)
    for rank in range(world):
        r = np.load(tmp_path / f"rank{rank}.npz")
        sl = slice(int(r["start"]), int(r["stop"]))
        np.testing.assert_array_equal(r["O"], O[:, sl])           # forward needs no exchange
        np.testing.assert_allclose(r["dQ"], dQ[:, sl], atol=1e-13)
        np.testing.assert_allclose(r["dG"], dG, atol=1e-10)       # every rank holds the full sum
        assert float(r["ms"]) == 20.0                             # max over ranks
        assert float(r["units"]) == w.heads * w.L                 # sum over ranks
