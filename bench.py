#!/usr/bin/env python
"""Benchmark of the SAKI routing hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg3] [--rows R] [--no-e2e] [--no-cpu] [--no-next] [--no-sweep]

One "step" is one pass of the whole hot path (log-softmax x2, lambda solve,
coupling + TV, routed loss, fused gradient) over one batch of synthetic
positions: one saki_route_fwd_bwd call.  Prints ONE JSON line.

  value     routed positions/s with the logits resident in HBM (whole job)
  e2e       the same through saki_route_host: inputs in pinned host memory,
            host<->device copies inside the timed region
  roofline  algorithmic HBM bytes (read both logit rows once, write the
            gradient row once) / measured kernel time, against the measured
            copy bandwidth of this machine's B200s
  cpu_baseline  the float64 test oracle, as it stands, on a bounded sample:
            on one host core, and on all host cores (a process pool over rows)
  next_step, spec_verify, small_batch  (rank 0, unless --no-next) further calls
            timed the same way beside the headline: saki_route_bwd_from_meta on
            the same logits, saki_spec_verify on its own workload with and
            without early out, and the latency of saki_route_fwd on 8 rows
  lm_head, vocab_sharded  (rank 0, unless --no-sweep) the lm-head GEMM with the row statistics
            in its epilogue, against the measured dense bf16 GEMM rate; vocabulary-sharded
            routing with the ranks run one after the other on this GPU
  sweep     (rank 0, unless --no-sweep) the throughput sweep at its full size
            (65536 positions, three disagreement regimes x three radii) and the
            V = 32000 workload: positions/s, fraction of the copy bandwidth,
            evaluation passes per row, saturated fraction, second-tier rows
  phase_cycles_per_row  where the row-per-SM kernel's cycles go (its phase
            clock, on one extra untimed call)

With N > 1 every rank routes its own batch of the same shape (rows are
independent: no collective on the data path); the time is the maximum over
ranks.  `--gpus N` without a torchrun environment starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed positions/sec (fwd+bwd, V=151936 bf16)"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one rowsm_kernel launch divided by the positions it
# routed, from an ncu capture on 2220 rows of the same workload (the kernel's ncu summary gives the
# command); traffic grows in proportion to the rows, so a full launch is this figure times N
TRAFFIC_BYTES_PER_POSITION = 958376
# rows up to this length are served by the instances of the two streaming kernels that run two CTAs per SM
# (namespace half_sm, meta_stream_kernel<16>); the names below are the ones a profiler shows
TWO_CTA_MAX_V = 98304
FOUR_CTA_MAX_V = 49152      # and the row kernel's instance with four (namespace quarter_sm) up to this length
# warp-instructions the row kernel's one-CTA instance issues per 32 vocabulary elements, from the same capture
ISSUED_PER_32_ELEMENTS = 39.09
# the same for one meta_stream_kernel launch
META_TRAFFIC_BYTES_PER_POSITION = 581046


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


FALLBACK_BF16_TFLOPS = 1590.0


def _tensor_peak():
    """Dense bf16 GEMM throughput of this machine's B200s (a cuBLAS GEMM run back to back for seconds), TFLOP/s."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained)"
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback (burst)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "25", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            busy = [x for x in sm if x > 0.5 * max(sm)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def _bf16_bits(x):
    """Host copy of logits as raw 16-bit words (bf16) or float32 values: small to ship to worker processes."""
    import torch
    return x.cpu().view(torch.int16).numpy() if x.dtype == torch.bfloat16 else x.cpu().numpy()


def _to_f64(a):
    """float64 array of what _bf16_bits shipped (bf16 -> float64 is exact)."""
    import numpy as np
    if a.dtype == np.int16:
        return (a.astype(np.int32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def _oracle_rows(job):
    """Worker of the all-cores baseline: routes a block of rows with the oracle; returns seconds spent."""
    import oracle as O
    sb, tb, x, eps, tau, seed, row0, dtype = job
    t0 = time.perf_counter()
    O.route(_to_f64(sb), _to_f64(tb), x, eps, tau, seed, row0, want_grad=True, grad_dtype=dtype)
    return time.perf_counter() - t0


def _oracle_sample(w, d, rows, grad=True):
    """Times the float64 oracle on `rows` rows of the workload (one host core)."""
    import oracle as O
    s = _to_f64(_bf16_bits(d["s"][:rows]))
    t = _to_f64(_bf16_bits(d["t"][:rows]))
    x = d["proposal"][:rows].to("cpu").numpy()
    t0 = time.perf_counter()
    ref = O.route(s, t, x, w.eps, w.temperature, w.seed, 0, want_grad=grad, grad_dtype=w.dtype)
    dt = time.perf_counter() - t0
    return rows / dt, dt, ref


def _oracle_all_cores(w, d, rows_per_core):
    """The same oracle on every host core at once: a pool of processes, each with its own block of rows
    (the rows that follow the one-core sample).  Returns positions/s over the wall time of the pool."""
    import multiprocessing as mp
    cores = os.cpu_count() or 1
    first = rows_per_core                      # do not reuse the one-core sample's rows
    jobs = []
    for c in range(cores):
        a, b = first + c * rows_per_core, first + (c + 1) * rows_per_core
        if b > w.N:
            break
        jobs.append((_bf16_bits(d["s"][a:b]), _bf16_bits(d["t"][a:b]), d["proposal"][a:b].cpu().numpy(), w.eps,
                     w.temperature, w.seed, a, w.dtype))
    if not jobs:
        return None
    with mp.get_context("spawn").Pool(len(jobs)) as pool:
        pool.map(_oracle_rows, [(j[0][:1], j[1][:1], j[2][:1]) + j[3:] for j in jobs])     # start-up and imports
        t0 = time.perf_counter()
        pool.map(_oracle_rows, jobs, chunksize=1)
        dt = time.perf_counter() - t0
    n = len(jobs) * rows_per_core
    return {"value": n / dt, "unit": UNIT, "cores": len(jobs), "kind": "oracle",
            "sample": f"{n} rows of {w.name} after the one-core sample, {rows_per_core} per process, forward + "
                      f"gradient, {dt:.1f} s wall on {len(jobs)} processes (os.cpu_count() = {cores})"}


def run_reference(args):
    """The reference arm: the float64 oracle on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2609_36601_b200 import synth
    w = synth.WORKLOADS[args.workload]
    rows = args.ref_rows
    d = synth.generate(w, "cpu", rows=rows)
    for _ in range(min(args.warmup, 1)):
        _oracle_sample(w, d, min(rows, 2))
    tot_rows, tot_t = 0, 0.0
    for _ in range(args.steps):
        r, dt, _ = _oracle_sample(w, d, rows)
        tot_rows += rows
        tot_t += dt
    v = tot_rows / tot_t
    line = {"metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": _config(w, args.gpus),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"first {rows} rows of {w.name} per step, forward + gradient, {args.steps} steps"},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def _config(w, world):
    esz = 4 if w.dtype == "f32" else 2
    return {"workload": _describe(w),
            "l2": "inputs (2 x %.1f GB) exceed L2; no flush needed" % (w.N * w.V * esz / 1e9),
            "parallelism": f"rows sharded over {world} GPU(s), no collective"}


def _describe(w):
    return (f"{w.name}: N={w.N} positions, V={w.V}, {w.dtype} logits, eps={w.eps}, temperature={w.temperature}, "
            f"teacher noise sigma={w.sigma}, fused fwd+bwd with {w.dtype} dlogits")


def _lm_head(P, dev, stream, steps, rows=0):
    """saki_lmhead_lse on the teacher's lm-head shape (Qwen3-4B: d_model 2560, V 151936) for cfg3's 16384
    positions: the bf16 GEMM that leaves the logits, row maximum and log-sum-exp from its epilogue."""
    import torch
    N, d, V = (rows or 16384), 2560, 151936
    g = torch.Generator(device=dev).manual_seed(2024)
    h = torch.randn((N, d), generator=g, device=dev).to(torch.bfloat16)
    w = (torch.randn((V, d), generator=g, device=dev) * (2.0 / d ** 0.5)).to(torch.bfloat16)
    logits = torch.empty((N, V), dtype=torch.bfloat16, device=dev)
    scratch = torch.empty(int(P.load_library().saki_lmhead_scratch_bytes(N, V)), dtype=torch.uint8, device=dev)
    for _ in range(3):
        P.lmhead_lse(h, w, 1.0, logits=logits, scratch=scratch, stream=stream)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        _, _, lse = P.lmhead_lse(h, w, 1.0, logits=logits, scratch=scratch, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    flops = 2.0 * N * d * V
    peak, kind = _tensor_peak()
    tf = flops / (ms * 1e-3) / 1e12
    ok = bool(torch.isfinite(lse).all().item())
    return {"call": "saki_lmhead_lse", "workload": f"hidden [{N}, {d}] x weight [{V}, {d}]^T, bf16, fp32 accumulation, bf16 logits "
            "+ row max + log-sum-exp", "ms_per_call": ms, "value": N / (ms * 1e-3), "unit": UNIT, "flops_per_call": flops,
            "kernel": "saki::lmhead_kernel", "results_finite": ok,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                         "peak_kind": f"of {kind} dense bf16 GEMM, MEASURED_PEAKS.json" if kind.startswith("measured") else "of fallback",
                         "traffic": None}}


def _vocab_sharded(P, synth, dev, stream, peak, rows=0):
    """Vocabulary-sharded routing of 4096 rows of the headline workload's shape cut into 8 column slices, the ranks
    run one after the other on this GPU (the calls one rank per GPU would make around its all-gathers): time of
    all ranks' kernels, evaluation waves, bytes a rank sends per row, and the slice kernels' HBM traffic (every
    stage reads the slice again: the rows of a call do not fit in L2) against the copy bandwidth."""
    import torch
    from paper_2609_36601_b200 import binding as B
    from paper_2609_36601_b200.vshard import route_vocab_sharded_local, split_columns
    w = synth.shrink(synth.WORKLOADS["cfg3"], rows or 4096)
    d = synth.generate(w, dev)
    world = 8
    slices = [(d["s"][:, a:a + n], d["t"][:, a:a + n], a) for a, n in split_columns(w.V, world)]
    for _ in range(2):
        out, gs, waves = route_vocab_sharded_local(slices, w.V, d["proposal"], w.eps, w.temperature, w.seed, grad_scale=1.0 / w.N,
                                                   stream=stream)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    out, gs, waves = route_vocab_sharded_local(slices, w.V, d["proposal"], w.eps, w.temperature, w.seed, grad_scale=1.0 / w.N,
                                               stream=stream)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    stages = 3 + waves
    # algorithmic bytes of the staged protocol: the two slices read by stage 0 (its second sweep counted as an L2
    # hit), by the first evaluation wave and by stage 2, the student's slice read and the gradient slice written by
    # stage 3 (later waves touch only the rows still solving: not counted)
    alg = w.N * w.V * 2 * (2 + 2 + 2 + 1 + 1)
    gbs = alg / dt / 1e9
    return {"call": "saki_vshard_partial / saki_vshard_combine", "rows": w.N, "V": w.V, "ranks_emulated_on_one_gpu": world,
            "ms_all_ranks": dt * 1e3, "ms_per_rank": dt * 1e3 / world, "value": w.N / dt, "unit": UNIT,
            "evaluation_waves": waves, "stages": stages,
            "bytes_sent_per_row_and_rank": stages * B.VSHARD_PARTIALS * 8, "arithmetic": "f32 per element, f64 sums and scalars",
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "algorithmic_bytes": alg},
            "note": "value = rows / wall time of all 8 ranks' kernels run one after the other on this GPU, host-side "
                    "sequencing included (a rank's own share is ms_per_rank, the exchanges not included)"}


def _sweep(P, synth, dev, stream, peak, args):
    """positions/s of saki_route_fwd_bwd on every cell of the throughput sweep at its full size (one input set
    per disagreement regime, three radii each) and on the V = 32000 workload; timed like the headline."""
    import torch
    cells = []
    groups = [[n for n in synth.WORKLOADS if n.startswith("cfg4_" + r + "_")] for r in ("s05", "s20", "ind")]
    groups.append(["cfg2"])
    for names in groups:
        w0 = synth.WORKLOADS[names[0]]
        d = synth.generate(w0, dev)
        g = torch.empty_like(d["s"])
        out = None
        for name in names:
            w = synth.WORKLOADS[name]
            n_steps = 3 if w.N * w.V > (1 << 32) else 20

            def call():
                nonlocal out
                out, _ = P.route_fwd_bwd(d["s"], d["t"], d["proposal"], w.eps, w.temperature, w.seed, 0,
                                         grad_scale=1.0 / w.N, out=out, dlogits=g, stream=stream)
            for _ in range(3):
                call()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n_steps):
                call()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / n_steps
            gbs = synth.bytes_per_position(w, True) * w.N / (ms * 1e-3) / 1e9
            st = out["row_status"]
            cells.append({"workload": name, "N": w.N, "V": w.V, "eps": w.eps,
                          "teacher": "independent" if w.sigma < 0 else f"sigma={w.sigma:g}",
                          "value": w.N / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "achieved_gbs": gbs,
                          "frac": gbs / peak, "kernel": P.last_kernel(),
                          "evaluation_passes_per_row": P.solve_evaluations(stream) / w.N,
                          "frac_saturated": float(((st & 1) != 0).float().mean().item()),
                          "second_tier_rows": int(P.redo_count(stream)),
                          "correction_rate": float(out["corrected"].float().mean().item()),
                          "mean_lambda": float(out["lambda"].mean().item()),
                          "rows_flagged": int(P.check())})
        del d, g, out
        torch.cuda.empty_cache()
    return {"call": "saki_route_fwd_bwd", "timing": "3 warm-up calls, then 3 timed calls per cell (20 for the short "
            "workload), CUDA events; inputs exceed L2", "frac": "of the same copy bandwidth as roofline.peak",
            "cells": cells}


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2609_36601_b200 as P
    from paper_2609_36601_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    if args.kernel:
        P.set_kernel(args.kernel)
    dev = f"cuda:{local}"
    P.load_library()

    w = synth.WORKLOADS[args.workload]
    if args.rows:
        w = synth.shrink(w, args.rows)
    d = synth.generate(w, dev)
    s, t, x = d["s"], d["t"], d["proposal"]
    row_offset = rank * w.N                      # ranks route disjoint global rows
    g = torch.empty_like(s)
    out = None
    stream = torch.cuda.current_stream()

    def step():
        nonlocal out
        out, _ = P.route_fwd_bwd(s, t, x, w.eps, w.temperature, w.seed, row_offset, grad_scale=1.0 / w.N,
                                 out=out, dlogits=g, stream=stream)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    l0 = P.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    ev[0].record(stream)
    for k in range(args.steps):
        step()
        ev[k + 1].record(stream)
    torch.cuda.synchronize()
    launches = P.launch_count() - l0
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    per_step = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    total_ms = ev[0].elapsed_time(ev[-1])
    if world > 1:
        tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())
    ms_per_step = total_ms / args.steps
    value = world * w.N / (ms_per_step * 1e-3)
    n_flagged = P.check()
    kernel_used = P.last_kernel()
    evals_last_step = P.solve_evaluations(stream) if kernel_used == 3 else 0   # of the last timed launch
    redo_last_step = P.redo_count(stream)
    phases = None
    if kernel_used == 3 and rank == 0:        # one more call, untimed, with the kernel's phase clock on
        P.set_phase_clock(True)
        step()
        ph = P.phase_cycles(stream)
        P.set_phase_clock(False)
        rows_ph = max(1, ph.pop("rows"))
        ph.pop("spare", None)
        phases = {k: round(v / rows_ph, 1) for k, v in ph.items()}
        phases["total"] = round(sum(ph.values()) / rows_ph, 1)

    # ---- the step that follows the path: the trainer's loss and gradient from this call's metadata
    # (saki_route_bwd_from_meta), on the same logits; reported beside the headline, not in it
    nxt = None
    if not args.no_next and rank == 0:
        adv = out["logT_x"] - out["logp_x"]
        mf = lambda: P.route_bwd_from_meta(s, out["corrected"], x, out["teacher_top1"], adv, w.temperature,
                                           rollout_status=out["row_status"], grad_scale=1.0 / w.N, dlogits=g,
                                           stream=stream)
        for _ in range(3):
            mf()
        torch.cuda.synchronize()
        l1 = P.launch_count()
        m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        m0.record(stream)
        for _ in range(args.steps):
            mf()
        m1.record(stream)
        torch.cuda.synchronize()
        mms = m0.elapsed_time(m1) / args.steps
        mbytes = 2 * w.V * s.element_size() * w.N
        nxt = {"call": "saki_route_bwd_from_meta", "value": w.N / (mms * 1e-3), "unit": UNIT, "ms_per_step": mms,
               "gpu_launches": int(P.launch_count() - l1), "kernel": {4: "saki::meta_stream_kernel<%d>" % (16 if w.V <= TWO_CTA_MAX_V else 32)}.get(P.last_kernel(), "saki::meta_general_kernel"),
               "algorithmic_bytes_per_launch": mbytes, "achieved_gbs": mbytes / (mms * 1e-3) / 1e9,
               "traffic": META_TRAFFIC_BYTES_PER_POSITION * w.N if META_TRAFFIC_BYTES_PER_POSITION else None}

    # ---- block verification (saki_spec_verify) on its own workload, with and without early out; beside the
    # headline like the step above
    spec = None
    if not args.no_next and rank == 0 and "cfg5" in synth.WORKLOADS:
        w5 = synth.WORKLOADS["cfg5"]
        d5 = synth.generate(w5, dev)
        s5, t5 = d5["s"].view(w5.B, w5.K + 1, w5.V), d5["t"].view(w5.B, w5.K + 1, w5.V)
        draft = d5["proposal"].view(w5.B, w5.K + 1)[:, :w5.K].contiguous()
        spec = {"call": "saki_spec_verify", "workload": "cfg5: B=%d sequences, K=%d draft tokens, V=%d, bf16, eps=%g" %
                (w5.B, w5.K, w5.V, w5.eps), "positions": w5.N}
        prev = P.set_spec_early_out(True)
        for on in (False, True):
            P.set_spec_early_out(on)
            for _ in range(3):
                r5 = P.spec_verify(s5, t5, draft, w5.eps, seed=w5.seed, stream=stream)
            torch.cuda.synchronize()
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record(stream)
            for _ in range(args.steps):
                r5 = P.spec_verify(s5, t5, draft, w5.eps, seed=w5.seed, stream=stream)
            c1.record(stream)
            torch.cuda.synchronize()
            ms5 = c0.elapsed_time(c1) / args.steps
            if on:
                spec.update({"ms_per_call": ms5, "value": w5.B / (ms5 * 1e-3), "unit": "sequences/s",
                             "positions_routed": P.spec_positions_routed(stream),
                             "mean_accepted": float(r5["n_accept"].float().mean().item())})
            else:
                spec["ms_per_call_all_positions"] = ms5
        P.set_spec_early_out(prev)
        del d5, s5, t5

    # ---- latency of a decoding step of a small batch: saki_route_fwd on the first 8 rows (forward only, as
    # at rollout time); automatic dispatch sends so few long rows to the cluster kernel
    small = None
    if not args.no_next and rank == 0 and w.N >= 8:
        s8, t8, x8 = s[:8], t[:8], x[:8]
        o8 = None
        for _ in range(5):
            o8 = P.route_fwd(s8, t8, x8, w.eps, w.temperature, w.seed, row_offset, out=o8, stream=stream)
        torch.cuda.synchronize()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record(stream)
        for _ in range(50):
            P.route_fwd(s8, t8, x8, w.eps, w.temperature, w.seed, row_offset, out=o8, stream=stream)
        q1.record(stream)
        torch.cuda.synchronize()
        small = {"call": "saki_route_fwd", "rows": 8, "us_per_call": q0.elapsed_time(q1) / 50 * 1e3,
                 "kernel": {2: "saki::cluster_kernel", 3: "saki::rowsm_kernel"}.get(P.last_kernel(), "saki::general_kernel")}

    # ---- end to end: host buffers through saki_route_host
    e2e = None
    if not args.no_e2e:
        hs, ht = s.to("cpu").pin_memory(), t.to("cpu").pin_memory()
        hx = x.to("cpu").pin_memory()
        hg = torch.empty(s.shape, dtype=s.dtype, pin_memory=True)
        hout = None
        esz = s.element_size()
        h2d = 2 * s.numel() * esz + hx.numel() * 4
        d2h = s.numel() * esz + w.N * (1 + 4 * 14)
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        hout, _ = P.route_host(hs, ht, hx, w.eps, w.temperature, w.seed, row_offset, grad_scale=1.0 / w.N,
                               out=hout, dlogits=hg)      # warm-up: staging buffers get allocated
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            hout, _ = P.route_host(hs, ht, hx, w.eps, w.temperature, w.seed, row_offset, grad_scale=1.0 / w.N,
                                   out=hout, dlogits=hg)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if world > 1:
            tt = torch.tensor([dt], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            dt = float(tt.item())
        e2e = {"value": world * w.N * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": n_e2e, "host_memory": "pinned"}
        same = all(torch.equal(hout[k], out[k].cpu()) for k in ("corrected", "token", "lambda"))
        e2e["matches_device_path"] = bool(same)
        del hs, ht, hg

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = _peaks()
    bpp = synth.bytes_per_position(w, backward=True)
    kern_ms = statistics.mean(per_step)          # one kernel launch per step
    achieved = bpp * w.N / (kern_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": f"of {peak_kind} (device-to-device copy, MEASURED_PEAKS.json)"
                if peak_kind == "measured" else "of fallback",
                "traffic": (TRAFFIC_BYTES_PER_POSITION * w.N) if TRAFFIC_BYTES_PER_POSITION else None,
                "algorithmic_bytes_per_launch": bpp * w.N, "kernel": {3: "saki::%s::rowsm_kernel<false>" % ("quarter_sm" if w.V <= FOUR_CTA_MAX_V else "half_sm" if w.V <= TWO_CTA_MAX_V else "full_sm"),
                           2: "saki::cluster_kernel"}.get(kernel_used, "saki::general_kernel"),
                "kernel_ms": kern_ms,
                "frac_of_nominal_8TBs": achieved / 8000.0}
    if kernel_used == 3:
        # What the kernel is actually bound by: exponentials on the special-function pipe.  Per vocabulary
        # element 2 in pass lse (student, teacher), 2 in pass final (p, q; a quarter of the p's are computed on
        # the FMA pipe instead: 1.75 on this pipe) and 1 per evaluation pass, the
        # evaluation passes counted by the kernel itself; peak = 16 ex2 per clock per SM (the throughput of
        # base-2 exponentials on this architecture) x SMs x the SM clock sampled during the timed region.
        evals = evals_last_step / max(1, w.N)
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        xu_peak = 16.0 * sm_count * mhz * 1e6 / 1e9
        xu_ach = (3.75 + evals) * w.V * w.N / (kern_ms * 1e-3) / 1e9
        roofline["special_function_pipe"] = {"achieved": xu_ach, "peak": xu_peak, "unit": "G ex2/s",
                                             "frac": xu_ach / xu_peak, "evaluation_passes_per_row": evals,
                                             "ex2_per_element": 3.75 + evals, "exponentials_per_element": 4.0 + evals}
        # and its other near-binding bound: issue slots (4 warp-instructions per clock per SM); the instruction
        # count per 32 elements is the profiler's (smsp__inst_executed.sum of the capture the kernel's ncu
        # summary describes, divided by the elements of that launch), not counted live
        if w.V > TWO_CTA_MAX_V:
            iss_peak = 4.0 * sm_count * mhz * 1e6 / 1e9
            iss_ach = ISSUED_PER_32_ELEMENTS * w.V * w.N / 32.0 / (kern_ms * 1e-3) / 1e9
            roofline["issue_slots"] = {"achieved": iss_ach, "peak": iss_peak, "unit": "G warp-instructions/s",
                                       "frac": iss_ach / iss_peak, "issued_per_32_elements": ISSUED_PER_32_ELEMENTS,
                                       "source": "ncu capture on 2220 rows of this workload"}

    stats = {"correction_rate": float(out["corrected"].float().mean().item()),
             "median_tv": float(out["tv"].median().item()), "mean_lambda": float(out["lambda"].mean().item()),
             "frac_saturated": float(((out["row_status"] & 1) != 0).float().mean().item()),
             "rows_flagged": n_flagged, "second_tier_rows": int(redo_last_step)}

    cpu = None
    if not args.no_cpu:
        import numpy as np
        n1 = min(args.cpu_rows, w.N)
        v, dt, ref = _oracle_sample(w, d, n1)
        got = {k: out[k][:n1].cpu().numpy() for k in ("corrected", "token", "teacher_top1", "lambda", "tv", "loss")}
        margin = np.minimum(ref["margin_accept"], ref["margin_draw"])
        exempt = margin < 1e-6            # decisions too close to call: counted, not compared
        ok = ~exempt
        flags_agree = int(np.sum(got["corrected"][ok] == ref["corrected"][ok]))
        tokens_agree = int(np.sum(got["token"][ok] == ref["token"][ok]))
        loss_err = np.abs(got["loss"] - ref["loss"])
        stats["oracle_sample"] = {
            "rows": int(n1), "margin_exempt": int(exempt.sum()),
            "margin_exempt_accept": int(np.sum(ref["margin_accept"] < 1e-6)),
            "margin_exempt_draw": int(np.sum(ref["margin_draw"] < 1e-6)),
            "flags_agree": f"{flags_agree}/{int(ok.sum())}", "tokens_agree": f"{tokens_agree}/{int(ok.sum())}",
            "teacher_top1_agree": f"{int(np.sum(got['teacher_top1'] == ref['teacher_top1']))}/{int(n1)}",
            "max_abs_dlambda": float(np.max(np.abs(got["lambda"] - ref["lam"]))),
            "max_abs_dtv": float(np.max(np.abs(got["tv"] - ref["tv"]))),
            "loss_beyond_1e-4_relative": int(np.sum(loss_err[ok] > 1e-4 * np.abs(ref["loss"][ok])))}
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {n1} rows of {w.name}, forward + gradient, {dt:.1f} s on one host core "
                         f"(of {os.cpu_count()})"}
        if w.N >= 2 * n1:
            allc = _oracle_all_cores(w, d, max(8, n1 // 4))
            if allc:
                cpu["all_cores"] = allc

    # ---- the throughput sweep at its full size and the V = 32000 workload, the step in front of the path (the
    # lm-head GEMM with the first row statistics in its epilogue) and vocabulary-sharded rows: beside the headline
    sweep = lm_head = vocab_sharded = None
    if not args.no_sweep and not args.rows and rank == 0:
        del s, t, g, x, d
        out = None
        torch.cuda.empty_cache()
        sweep = _sweep(P, synth, dev, stream, peak, args)
        torch.cuda.empty_cache()
        vocab_sharded = _vocab_sharded(P, synth, dev, stream, peak)
        torch.cuda.empty_cache()
        lm_head = _lm_head(P, dev, stream, 5)      # last: a dense GEMM at the power limit would colour what follows it

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": _config(w, world),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "stats": stats, "achieved_gbs": achieved}
    if phases is not None:
        line["phase_cycles_per_row"] = phases
    if lm_head is not None:
        line["lm_head"] = lm_head
    if vocab_sharded is not None:
        line["vocab_sharded"] = vocab_sharded
    if sweep is not None:
        line["sweep"] = sweep
    if nxt is not None:
        nxt["roofline"] = {"bound": "hbm", "achieved": nxt["achieved_gbs"], "peak": peak, "unit": "GB/s",
                           "frac": nxt["achieved_gbs"] / peak}
        line["next_step"] = nxt
    if spec is not None:
        line["spec_verify"] = spec
    if small is not None:
        line["small_batch"] = small
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def _spawn_ranks(n):
    """`--gpus N` outside a torchrun environment: start N ranks of this command, one GPU each, on this node."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")                       # NCCL's own log stays on, in a file per rank:
    env.setdefault("NCCL_DEBUG_FILE", os.path.join(tempfile.gettempdir(), "saki_bench_nccl.%h.%p.log"))   # stdout carries the JSON line
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--rows", type=int, default=0, help="cut the workload to its first R rows (profiling)")
    ap.add_argument("--kernel", type=int, default=0, choices=[0, 1, 2, 3],
                    help="row kernel (saki_set_kernel): 0 automatic, 1 general, 2 cluster, 3 row-per-SM (profiling)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-next", action="store_true", help="skip the metadata-driven backward measurement")
    ap.add_argument("--no-sweep", action="store_true", help="skip the throughput sweep and the V = 32000 workload")
    ap.add_argument("--section", default="all", choices=["all", "lm_head", "vocab_sharded"],
                    help="lm_head / vocab_sharded: time only that section (on --rows positions if given) and print its object (profiling)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-rows", type=int, default=384)
    ap.add_argument("--ref-rows", type=int, default=32)
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        sys.exit(_spawn_ranks(args.gpus))
    if args.section == "vocab_sharded":
        import torch
        import paper_2609_36601_b200 as P
        from paper_2609_36601_b200 import synth
        torch.cuda.set_device(0)
        peak, _ = _peaks()
        print(json.dumps(_vocab_sharded(P, synth, "cuda:0", torch.cuda.current_stream(), peak, args.rows)))
        return
    if args.section == "lm_head":
        import torch
        import paper_2609_36601_b200 as P
        torch.cuda.set_device(0)
        print(json.dumps(_lm_head(P, "cuda:0", torch.cuda.current_stream(), args.steps, args.rows)))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
