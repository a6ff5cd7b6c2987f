"""The float64 oracle over many rows at once: a pool of processes, one block of rows each.  The oracle itself
is untouched (every worker calls oracle.route_row / oracle.spec_verify row by row); this module only ships the
rows to the workers, as the raw 16-bit words the GPU sees, and brings the per-row scalars back.  Gradient rows
are too large to bring back for thousands of rows, so a worker checks them where they are: it is handed the
GPU's gradient rows (raw words too) and runs the same grad_check the in-process tests use."""
import multiprocessing as mp
import os

import numpy as np
import torch

_POOL = None


def _pool():
    global _POOL
    if _POOL is None:
        _POOL = mp.get_context("spawn").Pool(min(os.cpu_count() or 1, 32))
    return _POOL


def bits(x: torch.Tensor) -> np.ndarray:
    """Host copy as raw words: int16 for bf16 (widened exactly in the worker), float32 as is."""
    x = x.detach().cpu().contiguous()
    return x.view(torch.int16).numpy() if x.dtype == torch.bfloat16 else x.numpy()


def widen(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.int16:
        return (a.astype(np.int32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def _route_block(job):
    import oracle as O
    from parity import grad_check
    sb, tb, x, ids, eps, tau, seed, grad_scale, dtype, gb = job
    s64, t64 = widen(sb), widen(tb)
    g64 = None if gb is None else widen(gb)
    rows = []
    for i in range(len(ids)):
        r = O.route_row(s64[i], t64[i], int(x[i]), eps, tau, seed, int(ids[i]), 1, grad_scale, g64 is not None, dtype)
        grad = r.pop("grad", None)
        r["grad_stats"] = None
        r["grad_error"] = None
        if g64 is not None:
            r["grad_ref_nonzero"] = bool(np.any(grad != 0))
            r["_grad"] = grad
        rows.append(r)
    return rows, g64


def _route_block_checked(job):
    """Routes the block; where the GPU's flags agree with the oracle's (the caller passes them), checks the GPU's
    gradient row against the oracle's and returns the statistics instead of the row."""
    from parity import grad_check
    rows, g64 = _route_block(job[:-1])
    corrected_gpu = job[-1]
    dtype = job[8]
    for i, r in enumerate(rows):
        grad = r.pop("_grad", None)
        if grad is None or corrected_gpu is None or int(corrected_gpu[i]) != int(r["corrected"]):
            continue
        tok = r["teacher_top1"] if r["corrected"] == 1 else r["token"]
        try:
            r["grad_stats"] = grad_check(g64[i:i + 1], grad[None, :], dtype, np.array([tok]) if tok >= 0 else None)
        except AssertionError as e:           # reported to the caller, which fails the test with the row number
            r["grad_error"] = str(e)
    return rows


def route_rows(d, rows, eps, tau, seed, grad_scale=1.0, dtype="bf16", g=None, corrected_gpu=None, row_offset=0):
    """Oracle results for the rows `rows` of the generated workload d (dict of device tensors), as a dict of
    arrays indexed like `rows`, plus "grad_stats" / "grad_error" per row when the GPU's gradient `g` (device
    tensor, all rows) and its flags are given."""
    rows = np.asarray(list(rows), dtype=np.int64)
    idx = torch.as_tensor(rows, device=d["s"].device)
    sb, tb = bits(d["s"][idx]), bits(d["t"][idx])
    x = d["proposal"][idx].cpu().numpy()
    gb = None if g is None else bits(g[idx])
    cg = None if corrected_gpu is None else corrected_gpu[idx].cpu().numpy()
    n_blocks = max(1, min(len(rows), 4 * (os.cpu_count() or 1)))
    cuts = np.linspace(0, len(rows), n_blocks + 1).astype(int)
    jobs = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        if b > a:
            jobs.append((sb[a:b], tb[a:b], x[a:b], rows[a:b] + row_offset, eps, tau, seed, grad_scale, dtype,
                         None if gb is None else gb[a:b], None if cg is None else cg[a:b]))
    res = [r for block in _pool().map(_route_block_checked, jobs, chunksize=1) for r in block]
    out = {}
    for k in res[0]:
        if k in ("grad_stats", "grad_error"):
            out[k] = [r[k] for r in res]
        elif k not in ("grad_ref_nonzero",):
            out[k] = np.array([r[k] for r in res])
    return out


def _spec_block(job):
    import oracle as O
    sb, tb, draft, eps, tau, seed, seq_ids = job
    s64, t64 = widen(sb), widen(tb)
    return [O.spec_verify(s64[i:i + 1], t64[i:i + 1], draft[i:i + 1], eps, tau, seed=seed, seq_offset=int(b))
            for i, b in enumerate(seq_ids)]


def spec_verify_seqs(s3, t3, draft, seqs, eps, tau, seed):
    """oracle.spec_verify for each sequence of `seqs` (global sequence ids key the random streams)."""
    seqs = np.asarray(list(seqs), dtype=np.int64)
    idx = torch.as_tensor(seqs, device=s3.device)
    sb, tb = bits(s3[idx]), bits(t3[idx])
    dr = draft[idx].cpu().numpy()
    n_blocks = max(1, min(len(seqs), 4 * (os.cpu_count() or 1)))
    cuts = np.linspace(0, len(seqs), n_blocks + 1).astype(int)
    jobs = [(sb[a:b], tb[a:b], dr[a:b], eps, tau, seed, seqs[a:b]) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
    return [r for block in _pool().map(_spec_block, jobs, chunksize=1) for r in block]
