#!/usr/bin/env python
"""Benchmark of the SAKI routing hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg3] [--rows R] [--no-e2e] [--no-cpu]

One "step" is one pass of the whole hot path (log-softmax x2, lambda solve,
coupling + TV, routed loss, fused gradient) over one batch of synthetic
positions: one saki_route_fwd_bwd call.  Prints ONE JSON line.

  value     routed positions/s with the logits resident in HBM (whole job)
  e2e       the same through saki_route_host: inputs in pinned host memory,
            host<->device copies inside the timed region
  roofline  algorithmic HBM bytes (read both logit rows once, write the
            gradient row once) / measured kernel time, against the measured
            copy bandwidth of this machine's B200s
  cpu_baseline  the float64 test oracle, as it stands, on a bounded sample
  next_step, spec_verify, small_batch  (rank 0, unless --no-next) further calls
            timed the same way beside the headline: saki_route_bwd_from_meta on
            the same logits, saki_spec_verify on its own workload with and
            without early out, and the latency of saki_route_fwd on 8 rows

With N > 1 (under torchrun) every rank routes its own batch of the same
shape (rows are independent: no collective on the data path); the time is
the maximum over ranks.
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
# routed: ncu capture on 2220 rows of the same workload (profiles/rowsm_kernel_cfg3.md); traffic grows
# in proportion to the rows, so a full launch is this figure times N
TRAFFIC_BYTES_PER_POSITION = 945005
# rows up to this length are served by the instances of the two streaming kernels that run two CTAs per SM
# (namespace half_sm, meta_stream_kernel<16>); the names below are the ones a profiler shows
TWO_CTA_MAX_V = 98304
# the same for one meta_stream_kernel launch (profiles/meta_stream_kernel_cfg3.md)
META_TRAFFIC_BYTES_PER_POSITION = 581046


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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


def _oracle_sample(w, d, rows, grad=True):
    """Times the float64 oracle on `rows` rows of the workload (host cores)."""
    import numpy as np
    import torch
    import oracle as O
    idx = torch.arange(rows)
    s = d["s"][idx.to(d["s"].device)].to("cpu").to(torch.float64).numpy()
    t = d["t"][idx.to(d["t"].device)].to("cpu").to(torch.float64).numpy()
    x = d["proposal"][:rows].to("cpu").numpy()
    t0 = time.perf_counter()
    ref = O.route(s, t, x, w.eps, w.temperature, w.seed, 0, want_grad=grad, grad_dtype=w.dtype)
    dt = time.perf_counter() - t0
    return rows / dt, dt, ref


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
            "config": {"workload": _describe(w), "sample": f"{rows} rows per step"},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"first {rows} rows of {w.name}, forward + gradient, {args.steps} steps"},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def _describe(w):
    return (f"{w.name}: N={w.N} positions, V={w.V}, {w.dtype} logits, eps={w.eps}, temperature={w.temperature}, "
            f"teacher noise sigma={w.sigma}, fused fwd+bwd with {w.dtype} dlogits")


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
                "algorithmic_bytes_per_launch": bpp * w.N, "kernel": {3: "saki::%s::rowsm_kernel" % ("half_sm" if w.V <= TWO_CTA_MAX_V else "full_sm"),
                           2: "saki::cluster_kernel"}.get(kernel_used, "saki::general_kernel"),
                "kernel_ms": kern_ms,
                "frac_of_nominal_8TBs": achieved / 8000.0}
    if kernel_used == 3:
        # What the kernel is actually bound by: exponentials on the special-function pipe.  Per vocabulary
        # element 2 in pass lse (student, teacher), 2 in pass final (p, q) and 1 per evaluation pass, the
        # evaluation passes counted by the kernel itself; peak = 16 ex2 per clock per SM (the throughput of
        # base-2 exponentials on this architecture) x SMs x the SM clock sampled during the timed region.
        evals = evals_last_step / max(1, w.N)
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        xu_peak = 16.0 * sm_count * mhz * 1e6 / 1e9
        xu_ach = (4.0 + evals) * w.V * w.N / (kern_ms * 1e-3) / 1e9
        roofline["special_function_pipe"] = {"achieved": xu_ach, "peak": xu_peak, "unit": "G ex2/s",
                                             "frac": xu_ach / xu_peak, "evaluation_passes_per_row": evals,
                                             "ex2_per_element": 4.0 + evals}

    stats = {"correction_rate": float(out["corrected"].float().mean().item()),
             "median_tv": float(out["tv"].median().item()), "mean_lambda": float(out["lambda"].mean().item()),
             "frac_saturated": float(((out["row_status"] & 1) != 0).float().mean().item()),
             "rows_flagged": n_flagged}

    cpu = None
    if not args.no_cpu:
        v, dt, ref = _oracle_sample(w, d, args.cpu_rows)
        import numpy as np
        agree = int(np.sum(out["corrected"][:args.cpu_rows].cpu().numpy() == ref["corrected"]))
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {args.cpu_rows} rows of {w.name}, forward + gradient, {dt:.1f} s on one host core "
                         f"(of {os.cpu_count()}); accept/correct flags agree with the GPU on {agree}/{args.cpu_rows}"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": _describe(w), "l2": "inputs (2 x %.1f GB) exceed L2; no flush needed" %
                       (s.numel() * s.element_size() / 1e9), "parallelism": f"rows sharded over {world} GPU(s), no collective"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu,
            "stats": stats, "achieved_gbs": achieved}
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
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-rows", type=int, default=384)
    ap.add_argument("--ref-rows", type=int, default=32)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
