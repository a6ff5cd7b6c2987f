"""The multi-GPU path is row sharding with no collective on the data path.  Two gloo ranks on
CPU: the shards tile the batch, the normaliser is the all-reduced count of valid positions, and
routing a shard with row_offset reproduces the corresponding rows of the unsharded run (shown
with the oracle, whose random streams are keyed by global row exactly like the library's)."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
from paper_2609_36601_b200 import synth
from paper_2609_36601_b200.shard import global_grad_scale, shard_rows


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = synth.Workload("t", 23, 256, "f32", 0.1, 1.5, False, 5, 7, student_scale=1.0)
        d = synth.generate(w, "cpu")                       # every rank generates the same bytes
        mask = (np.arange(w.N) % 5 != 0).astype(np.uint8)
        first, n = shard_rows(w.N, rank, world)
        scale = global_grad_scale(int(mask[first:first + n].sum()))
        s = d["s"].double().numpy()[first:first + n]
        t = d["t"].double().numpy()[first:first + n]
        out = O.route(s, t, d["proposal"].numpy()[first:first + n], w.eps, 1.0, w.seed, row_offset=first,
                      mask=mask[first:first + n], grad_scale=scale, want_grad=True)
        bounds = [None] * world
        dist.all_gather_object(bounds, (first, n))
        loss_sum = torch.tensor([out["loss"].sum() * scale], dtype=torch.float64)
        dist.all_reduce(loss_sum)
        q.put((rank, bounds, scale, out["token"].tolist(), out["corrected"].tolist(), out["grad"].sum(),
               float(loss_sum.item())))
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_matches_single_run():
    world, port = 2, 29731
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = synth.Workload("t", 23, 256, "f32", 0.1, 1.5, False, 5, 7, student_scale=1.0)
    d = synth.generate(w, "cpu")
    mask = (np.arange(w.N) % 5 != 0).astype(np.uint8)
    full = O.route(d["s"].double().numpy(), d["t"].double().numpy(), d["proposal"].numpy(), w.eps, 1.0, w.seed,
                   mask=mask, grad_scale=1.0 / mask.sum(), want_grad=True)
    bounds = res[0][1]
    assert bounds == [(0, 12), (12, 11)] and res[1][1] == bounds          # the shards tile the batch
    assert all(abs(r[2] - 1.0 / mask.sum()) < 1e-15 for r in res)          # global normaliser
    tokens = res[0][3] + res[1][3]
    corrected = res[0][4] + res[1][4]
    assert tokens == full["token"].tolist() and corrected == full["corrected"].tolist()
    assert abs(res[0][6] - full["loss"].sum() / mask.sum()) < 1e-12         # all-reduced objective


def test_shard_rows_properties():
    for n in (0, 1, 7, 16384):
        for world in (1, 2, 3, 8):
            parts = [shard_rows(n, r, world) for r in range(world)]
            assert parts[0][0] == 0 and sum(p[1] for p in parts) == n
            for a, b in zip(parts, parts[1:]):
                assert a[0] + a[1] == b[0]
            assert max(p[1] for p in parts) - min(p[1] for p in parts) <= 1
