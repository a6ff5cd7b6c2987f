"""The torch.distributed paths with the NCCL backend on the one GPU a test box has: a process group of one rank.
The exchange of vocabulary-sharded routing (all_gather_into_tensor on device buffers between the stage kernels)
and the normaliser's all-reduce run as they would on eight GPUs; with one rank the slice is the whole row, so
the result must equal the single-process form bit for bit.  Run in a child process: the process group does not
outlive the test."""
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import os, sys, torch
import torch.distributed as dist
sys.path.insert(0, %r)
import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from paper_2609_36601_b200.shard import global_grad_scale, shard_rows
from paper_2609_36601_b200.vshard import route_vocab_sharded, route_vocab_sharded_local
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda:0"))
try:
    w = synth.Workload("t", 96, 32000, "bf16", 0.1, 1.5, True, 41, 17)
    d = synth.generate(w, "cuda:0")
    mask = (torch.arange(w.N, device="cuda:0") %% 7 != 0).to(torch.uint8)
    first, n = shard_rows(w.N, dist.get_rank(), dist.get_world_size())
    assert (first, n) == (0, w.N)
    scale = global_grad_scale(int(mask.sum().item()))
    assert abs(scale - 1.0 / int(mask.sum().item())) < 1e-15
    out, g = route_vocab_sharded(d["s"], d["t"], 0, w.V, d["proposal"], w.eps, w.temperature, w.seed, mask=mask,
                                 grad_scale=scale)
    ref, gs, waves = route_vocab_sharded_local([(d["s"], d["t"], 0)], w.V, d["proposal"], w.eps, w.temperature, w.seed,
                                               mask=mask, grad_scale=scale)
    torch.cuda.synchronize()
    for k in ref:
        assert torch.equal(out[k], ref[k]), k
    assert torch.equal(g, gs[0])
    whole, gw = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, w.temperature, w.seed, mask=mask, grad_scale=scale)
    torch.cuda.synchronize()
    agree = float((out["corrected"] == whole["corrected"]).float().mean().item())
    assert agree >= 0.97, agree                        # the same decisions as the unsharded call (outside the margin)
    assert float((out["lambda"] - whole["lambda"]).abs().max().item()) <= 1e-5
    print("OK waves", waves, "agree", agree)
finally:
    dist.destroy_process_group()
""" % ROOT


def test_vocab_sharded_exchange_and_normaliser_over_nccl():
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), NCCL_NVLS_ENABLE="0")
    r = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert r.returncode == 0, (r.stdout[-1500:], r.stderr[-3000:])
    assert "OK waves" in r.stdout
