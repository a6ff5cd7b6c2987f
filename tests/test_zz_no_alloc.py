"""saki_route_fwd_bwd_noalloc: the entry point for callers that may not allocate device memory (code running
inside another allocator's callback, serving loops with a frozen memory plan).  It must give exactly what
saki_route_fwd_bwd gives, call after call, although its scratch is one fixed device array shared by all
calls.  Collected last on purpose: a run that stops at the first failure has then run every other test."""
import pytest
import torch

import paper_2609_36601_b200 as P
from paper_2609_36601_b200 import synth
from parity import force_second_tier

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_entry_matches_regular_entry_twice_in_a_row():
    prev = P.set_kernel(0)
    try:
        # the V = 32000 workload with some rows that overflow the float32 sums and are handed to the float64
        # kernel, so the fixed scratch really carries a list
        w = synth.shrink(synth.WORKLOADS["cfg2"], 2048)
        d = synth.generate(w, DEV)
        force_second_tier(d, [3, 700, 701, 1999])
        ref_out, ref_g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed, grad_scale=0.5)
        torch.cuda.synchronize()
        n_redo = P.redo_count()
        assert P.last_kernel() == 3 and n_redo > 0, "the workload should exercise the scratch"
        for call in range(2):
            out = P.alloc_outputs(w.N, DEV)
            g = torch.full_like(d["s"], float("nan"))
            P.route_fwd_bwd_noalloc(d["s"], d["t"], d["proposal"], w.eps, out, g, seed=w.seed, grad_scale=0.5)
            torch.cuda.synchronize()
            assert P.redo_count() == n_redo
            for k in ref_out:           # same kernels, same order of operations: identical, not merely close
                assert torch.equal(out[k], ref_out[k]), (call, k)
            assert torch.equal(g, ref_g), call
        # a second workload right after, with different rows on the list: stale list contents must not matter
        w2 = synth.Workload("noalloc2", 300, 8192, "bf16", 0.005, 0.5, True, 99, 18)
        d2 = synth.generate(w2, DEV)
        force_second_tier(d2, [0, 150, 299])
        r2, g2 = P.route_fwd_bwd(d2["s"], d2["t"], d2["proposal"], w2.eps, seed=w2.seed)
        out2 = P.alloc_outputs(w2.N, DEV)
        gg2 = torch.empty_like(d2["s"])
        P.route_fwd_bwd_noalloc(d2["s"], d2["t"], d2["proposal"], w2.eps, out2, gg2, seed=w2.seed)
        torch.cuda.synchronize()
        for k in r2:
            assert torch.equal(out2[k], r2[k]), k
        assert torch.equal(gg2, g2)
    finally:
        P.set_kernel(prev)


def test_noalloc_entry_allocates_nothing_on_a_stream_the_library_has_never_seen():
    """What the entry point is for: on a stream that no regular call has used (the regular entry would now
    allocate that stream's row list) the call leaves the device's free memory exactly as it was, and the
    rows that need the float64 kernel still get there through the fixed array."""
    prev = P.set_kernel(0)
    try:
        w = synth.Workload("noalloc3", 512, 32000, "bf16", 0.05, 1.0, True, 313, 21)
        d = synth.generate(w, DEV)
        force_second_tier(d, [5, 100, 511])
        ref_out, ref_g = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, seed=w.seed)
        torch.cuda.synchronize()
        out = P.alloc_outputs(w.N, DEV)
        g = torch.empty_like(d["s"])
        fresh = torch.cuda.Stream()
        # once on the current stream: the address of the fixed array is looked up on a device's first call
        P.route_fwd_bwd_noalloc(d["s"], d["t"], d["proposal"], w.eps, out, g, seed=w.seed)
        torch.cuda.synchronize()
        g.fill_(float("nan"))
        free_before, _ = torch.cuda.mem_get_info()
        P.route_fwd_bwd_noalloc(d["s"], d["t"], d["proposal"], w.eps, out, g, seed=w.seed, stream=fresh)
        fresh.synchronize()
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, (free_before, free_after)
        assert P.last_kernel() == 3 and P.redo_count(fresh) == 3
        for k in ref_out:
            assert torch.equal(out[k], ref_out[k]), k
        assert torch.equal(g, ref_g)
    finally:
        P.set_kernel(prev)


def test_noalloc_entry_rejects_batches_beyond_its_fixed_scratch():
    s = torch.zeros((1, 2048), dtype=torch.bfloat16, device=DEV)
    big = s.expand((1 << 20) + 1, 2048)          # a view: no memory behind the extra rows, and none is read
    x = torch.zeros((1 << 20) + 1, dtype=torch.int32, device=DEV)
    out = P.alloc_outputs((1 << 20) + 1, DEV)
    with pytest.raises(P.SakiError) as ei:
        P.route_fwd_bwd_noalloc(big, big, x, 0.1, out, s)
    assert ei.value.code == 1 and "fixed scratch" in str(ei.value)
