"""Vocabulary-sharded routing, the exchange between ranks, without a GPU: gloo ranks each hold a column slice
of the rows; the slice reductions are a numpy stand-in for the GPU kernels (vshard_model.py), the all-gather
is torch.distributed's, and the combine is the library's own (saki_vshard_combine_host), so what is tested
is the protocol: stage order, rank-order summation, the repeat-until-settled loop, the owner of the draw, and
that the answer does not depend on how many ranks hold the row."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle as O
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import binding, synth
from paper_2609_36601_b200.vshard import split_columns, MAX_WAVES
import vshard_model as M
from parity import MARGIN


def _workload():
    w = synth.Workload("vs", 24, 6000, "bf16", 0.1, 1.5, True, 611, 31)
    d = synth.generate(w, "cpu")
    s, t = d["s"].to(torch.float64).numpy().copy(), d["t"].to(torch.float64).numpy().copy()
    x = d["proposal"].numpy().copy()
    mask = np.ones(w.N, dtype=np.uint8)
    mask[5] = 0
    x[7] = w.V + 9                       # a bad id
    s[9, 4000] = np.inf                  # a non-finite row (its slice owner reports it)
    t[11] = s[11] + 1e-3 * np.sin(np.arange(w.V))    # well inside the trust region: lambda = 1
    return w, s, t, x, mask


def _route_ranked(rank, world, w, s, t, x, mask, exchange, eps=None):
    """What one rank does: slice reductions, exchange, the library's host combine.  Returns outputs, the
    gradient slice and the number of stage-1 waves."""
    eps = w.eps if eps is None else eps
    v0, vl = split_columns(w.V, world)[rank]
    sl, tl = s[:, v0:v0 + vl], t[:, v0:v0 + vl]
    xt, mt = torch.as_tensor(x.astype(np.int32)), torch.as_tensor(mask)
    si = binding.vshard_in(None, None, v0, w.V, xt, eps, w.temperature, w.seed, 0, mt, rank, world, dtype=w.dtype,
                           n_rows=w.N)
    si.V_local = vl
    state = torch.zeros((w.N, M.S), dtype=torch.float64)
    out = {k: torch.zeros(w.N, dtype=v.dtype) for k, v in P.alloc_outputs(1, "cpu").items()}
    grad, waves = None, 0

    def wave(stage):
        nonlocal grad
        part, g = M.partial(stage, sl, tl, v0, w.temperature, x, None if stage == 0 else state.numpy(), rank, 1.0, True)
        if g is not None:
            grad = g
        gathered = exchange(torch.as_tensor(part))
        return P.vshard_combine_host(si, stage, gathered, state, out if stage == 3 else None)

    n = wave(0)
    while n > 0 and waves < MAX_WAVES:
        n = wave(1)
        waves += 1
    wave(2)
    wave(3)
    return {k: v.numpy() for k, v in out.items()}, grad, waves


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, s, t, x, mask = _workload()

    def exchange(part):
        gathered = torch.empty((world,) + tuple(part.shape), dtype=torch.float64)
        dist.all_gather_into_tensor(gathered.view(-1), part.contiguous().view(-1))
        return gathered
    out, grad, waves = _route_ranked(rank, world, w, s, t, x, mask, exchange)
    q.put((rank, out, grad, waves))
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def _single_process(world, w, s, t, x, mask, eps=None):
    """The same ranks one after the other in this process (the exchange becomes a stack)."""
    outs = [None] * world
    # run the ranks in lock step: every rank needs every rank's partial of a stage before its combine
    import threading
    barrier = threading.Barrier(world)
    box = {}

    def exchange_for(rank):
        def exchange(part):
            box[rank] = part
            barrier.wait()
            g = torch.stack([box[r] for r in range(world)])
            barrier.wait()
            return g
        return exchange
    th = [threading.Thread(target=lambda r=r: outs.__setitem__(r, _route_ranked(r, world, w, s, t, x, mask, exchange_for(r), eps)))
          for r in range(world)]
    [t_.start() for t_ in th]
    [t_.join() for t_ in th]
    return outs


def _check_against_oracle(w, s, t, x, mask, out, grad_full, eps=None):
    eps = w.eps if eps is None else eps
    ref = O.route(s, t, x, eps, w.temperature, w.seed, 0, mask=mask, grad_scale=1.0, want_grad=True, grad_dtype="f32")
    ok = np.minimum(ref["margin_accept"], ref["margin_draw"]) >= MARGIN
    assert np.array_equal(out["row_status"].astype(np.uint32), ref["status"])
    assert np.array_equal(out["teacher_top1"], ref["teacher_top1"])
    assert np.array_equal(out["corrected"][ok], ref["corrected"][ok]) and np.array_equal(out["token"][ok], ref["token"][ok])
    for name, key in (("lambda", "lam"), ("tv", "tv"), ("kl", "kl"), ("accept_prob", "accept_prob"), ("loss", "loss"),
                      ("logp_x", "logp_x"), ("logq_x", "logq_x"), ("logT_x", "logT_x")):
        assert np.max(np.abs(out[name].astype(np.float64) - ref[key])) <= 2e-6 * (1 + np.max(np.abs(ref[key]))), name
    same = ok & (out["corrected"] == ref["corrected"])
    assert np.max(np.abs(grad_full[same] - ref["grad"][same])) <= 1e-6
    return ref


def test_two_gloo_ranks_route_column_slices_and_agree_with_the_oracle():
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, q)) for r in range(world)]
    [p.start() for p in procs]
    got = sorted([q.get(timeout=300) for _ in range(world)], key=lambda g: g[0])
    [p.join(timeout=60) for p in procs]
    assert all(p.exitcode == 0 for p in procs)
    (_, out0, g0, waves0), (_, out1, g1, waves1) = got
    for k in out0:                                    # every rank ends with the same outputs, bit for bit
        assert np.array_equal(out0[k], out1[k]), k
    assert waves0 == waves1 and 1 <= waves0 <= 4      # a wave moves to the root of a fourth-order model: two as a rule
    w, s, t, x, mask = _workload()
    ref = _check_against_oracle(w, s, t, x, mask, out0, np.concatenate([g0, g1], axis=1))
    st = ref["status"]
    assert st[5] & 4 and st[7] == 16 and st[9] == 8 and st[11] & 1        # masked, bad id, non-finite, saturated
    assert ref["corrected"].sum() >= 2                # some rows needed the draw and its owner rank


@pytest.mark.parametrize("eps", [0.1, 0.0, 3.0])
def test_answer_does_not_depend_on_the_number_of_ranks(eps):
    w, s, t, x, mask = _workload()
    base = None
    for world in (1, 2, 3, 5):
        outs = _single_process(world, w, s, t, x, mask, eps)
        out = outs[0][0]
        for r in range(1, world):
            for k in out:
                assert np.array_equal(out[k], outs[r][0][k]), (world, r, k)
        grad = np.concatenate([o[1] for o in outs], axis=1)
        ref = _check_against_oracle(w, s, t, x, mask, out, grad, eps)
        if base is None:
            base = out
        else:
            ok = np.minimum(ref["margin_accept"], ref["margin_draw"]) >= MARGIN
            for k in ("corrected", "token", "teacher_top1", "row_status"):
                assert np.array_equal(out[k][ok], base[k][ok]), (world, k)
            for k in ("lambda", "tv", "kl", "loss"):
                assert np.max(np.abs(out[k] - base[k])) <= 1e-6, (world, k)
