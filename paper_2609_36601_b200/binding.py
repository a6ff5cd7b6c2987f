"""Thin ctypes binding of the C-ABI library: argument marshalling only.

Every function takes torch tensors (device memory and streams are torch's),
passes raw pointers, sizes and strides to the library, and returns torch
tensors.  There is no CPU fallback: if the library is missing or cannot be
loaded the first call raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsaki.so")
_lib = None

SAKI_F32, SAKI_BF16 = 0, 1
ROW_SATURATED, ROW_EPS_ZERO, ROW_MASKED, ROW_NONFINITE, ROW_BAD_ID, ROW_TIMEOUT, ROW_NOT_COMPUTED = 1, 2, 4, 8, 16, 32, 64

_FLOAT_FIELDS = ("lambda", "kl", "tv", "accept_prob", "logp_x", "logq_x", "logT_x", "logp_y", "logq_y", "logT_y", "loss")
EXPORTS = ("saki_route_fwd", "saki_route_fwd_bwd", "saki_route_fwd_bwd_noalloc", "saki_route_host",
           "saki_route_bwd_from_meta", "saki_select_tm", "saki_spec_verify",
           "saki_vshard_partial", "saki_vshard_combine", "saki_vshard_combine_host",
           "saki_lmhead_scratch_bytes", "saki_lmhead_lse",
           "saki_sample_proposal", "saki_check", "saki_set_kernel", "saki_last_kernel", "saki_redo_count",
           "saki_set_spec_early_out", "saki_spec_positions_routed", "saki_solve_evaluations", "saki_set_wait_limit", "saki_set_phase_clock", "saki_phase_cycles",
           "saki_launch_count",
           "saki_last_error", "saki_version")


class SakiError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"saki error {code}: {text}")
        self.code = code


class SakiIn(C.Structure):
    _fields_ = [("student_logits", C.c_void_p), ("teacher_logits", C.c_void_p),
                ("ld_s", C.c_int64), ("ld_t", C.c_int64), ("N", C.c_int64),
                ("V", C.c_int32), ("dtype", C.c_int32),
                ("proposal", C.c_void_p), ("mask", C.c_void_p),
                ("eps", C.c_float), ("temperature", C.c_float),
                ("seed", C.c_uint64), ("row_offset", C.c_uint64)]


class SakiOut(C.Structure):
    _fields_ = [("corrected", C.c_void_p), ("token", C.c_void_p), ("teacher_top1", C.c_void_p)] + \
               [(f, C.c_void_p) for f in _FLOAT_FIELDS] + [("row_status", C.c_void_p)]


class SakiMetaIn(C.Structure):
    _fields_ = [("student_logits", C.c_void_p), ("ld_s", C.c_int64), ("N", C.c_int64),
                ("V", C.c_int32), ("dtype", C.c_int32),
                ("corrected", C.c_void_p), ("proposal", C.c_void_p), ("teacher_top1", C.c_void_p),
                ("advantage", C.c_void_p), ("mask", C.c_void_p), ("rollout_status", C.c_void_p),
                ("temperature", C.c_float)]


class SakiMetaOut(C.Structure):
    _fields_ = [("loss", C.c_void_p), ("logp_tok", C.c_void_p), ("row_status", C.c_void_p)]


class SakiSelectIn(C.Structure):
    _fields_ = [("N", C.c_int64), ("B", C.c_int64), ("seq_start", C.c_void_p), ("corrected", C.c_void_p),
                ("tv", C.c_void_p), ("mask", C.c_void_p), ("rollout_status", C.c_void_p), ("mode", C.c_int32),
                ("seed", C.c_uint64), ("row_offset", C.c_uint64)]


class SakiVshardIn(C.Structure):
    _fields_ = [("student_logits", C.c_void_p), ("teacher_logits", C.c_void_p),
                ("ld_s", C.c_int64), ("ld_t", C.c_int64), ("N", C.c_int64),
                ("V", C.c_int32), ("V_local", C.c_int32), ("v0", C.c_int32), ("dtype", C.c_int32),
                ("proposal", C.c_void_p), ("mask", C.c_void_p),
                ("eps", C.c_float), ("temperature", C.c_float),
                ("seed", C.c_uint64), ("row_offset", C.c_uint64),
                ("rank", C.c_int32), ("world", C.c_int32)]


VSHARD_PARTIALS, VSHARD_STATE = 16, 32


class SakiLmheadIn(C.Structure):
    _fields_ = [("hidden", C.c_void_p), ("ld_h", C.c_int64), ("weight", C.c_void_p), ("ld_w", C.c_int64),
                ("N", C.c_int64), ("d", C.c_int32), ("V", C.c_int32), ("temperature", C.c_float)]


class SakiSpecIn(C.Structure):
    _fields_ = [("student_logits", C.c_void_p), ("teacher_logits", C.c_void_p),
                ("ss_seq", C.c_int64), ("ss_pos", C.c_int64), ("ts_seq", C.c_int64), ("ts_pos", C.c_int64),
                ("B", C.c_int64), ("K", C.c_int32), ("V", C.c_int32), ("dtype", C.c_int32),
                ("draft", C.c_void_p), ("draft_ld", C.c_int64),
                ("eps", C.c_float), ("temperature", C.c_float),
                ("seed", C.c_uint64), ("seq_offset", C.c_uint64)]


class SakiSpecOut(C.Structure):
    _fields_ = [("n_accept", C.c_void_p), ("next_token", C.c_void_p), ("next_is_correction", C.c_void_p),
                ("per_pos", SakiOut)]


def load_library(path: str | None = None):
    """Loads libsaki.so (built in-tree by `python -m paper_2609_36601_b200.build`)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise SakiError(-1, f"{p} not found: build it with `python -m paper_2609_36601_b200.build`; "
                            "there is no CPU fallback")
    lib = C.CDLL(p)
    lib.saki_route_fwd.argtypes = [C.POINTER(SakiIn), C.POINTER(SakiOut), C.c_void_p]
    lib.saki_route_fwd_bwd.argtypes = [C.POINTER(SakiIn), C.POINTER(SakiOut), C.c_void_p, C.c_int64, C.c_float, C.c_void_p]
    lib.saki_route_fwd_bwd_noalloc.argtypes = lib.saki_route_fwd_bwd.argtypes
    lib.saki_route_fwd_bwd_noalloc.restype = C.c_int
    lib.saki_route_host.argtypes = [C.POINTER(SakiIn), C.POINTER(SakiOut), C.c_void_p, C.c_int64, C.c_float]
    lib.saki_route_bwd_from_meta.argtypes = [C.POINTER(SakiMetaIn), C.POINTER(SakiMetaOut), C.c_void_p, C.c_int64,
                                             C.c_float, C.c_void_p]
    lib.saki_route_bwd_from_meta.restype = C.c_int
    lib.saki_select_tm.argtypes = [C.POINTER(SakiSelectIn), C.c_void_p, C.c_void_p, C.c_void_p]
    lib.saki_select_tm.restype = C.c_int
    lib.saki_spec_verify.argtypes = [C.POINTER(SakiSpecIn), C.POINTER(SakiSpecOut), C.c_void_p]
    lib.saki_sample_proposal.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_float,
                                         C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
    lib.saki_check.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.saki_set_kernel.argtypes = [C.c_int]
    lib.saki_redo_count.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.saki_set_spec_early_out.argtypes = [C.c_int]
    lib.saki_set_spec_early_out.restype = C.c_int
    lib.saki_spec_positions_routed.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.saki_spec_positions_routed.restype = C.c_int
    lib.saki_solve_evaluations.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.saki_solve_evaluations.restype = C.c_int
    lib.saki_vshard_partial.argtypes = [C.POINTER(SakiVshardIn), C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_float, C.c_void_p]
    lib.saki_vshard_partial.restype = C.c_int
    lib.saki_vshard_combine.argtypes = [C.POINTER(SakiVshardIn), C.c_int, C.c_void_p, C.c_void_p, C.POINTER(SakiOut),
                                        C.c_void_p, C.c_void_p]
    lib.saki_vshard_combine.restype = C.c_int
    lib.saki_vshard_combine_host.argtypes = [C.POINTER(SakiVshardIn), C.c_int, C.c_void_p, C.c_void_p, C.POINTER(SakiOut),
                                             C.POINTER(C.c_int32)]
    lib.saki_vshard_combine_host.restype = C.c_int
    lib.saki_lmhead_scratch_bytes.argtypes = [C.c_int64, C.c_int32]
    lib.saki_lmhead_scratch_bytes.restype = C.c_int64
    lib.saki_lmhead_lse.argtypes = [C.POINTER(SakiLmheadIn), C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.c_int64, C.c_void_p]
    lib.saki_lmhead_lse.restype = C.c_int
    lib.saki_set_wait_limit.argtypes = [C.c_int64]
    lib.saki_set_wait_limit.restype = C.c_int64
    lib.saki_set_phase_clock.argtypes = [C.c_int]
    lib.saki_set_phase_clock.restype = C.c_int
    lib.saki_phase_cycles.argtypes = [C.c_void_p, C.POINTER(C.c_uint64)]
    lib.saki_phase_cycles.restype = C.c_int
    lib.saki_launch_count.restype = C.c_uint64
    lib.saki_last_error.restype = C.c_char_p
    for f in ("saki_route_fwd", "saki_route_fwd_bwd", "saki_route_host", "saki_spec_verify",
              "saki_sample_proposal", "saki_check", "saki_set_kernel", "saki_last_kernel", "saki_redo_count",
              "saki_version"):
        getattr(lib, f).restype = C.c_int
    _lib = lib
    return lib


def _raise(lib, rc):
    if rc != 0:
        raise SakiError(rc, lib.saki_last_error().decode())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SAKI_F32
    if t.dtype == torch.bfloat16:
        return SAKI_BF16
    raise SakiError(1, f"unsupported logits dtype {t.dtype}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def alloc_outputs(n: int, device):
    """Preallocated per-position output tensors for the calls that take `out=`."""
    return _alloc_out(n, device)


def _alloc_out(n: int, device, pinned=False):
    kw = dict(device=device)
    if pinned:
        kw = dict(device="cpu", pin_memory=True)
    out = {"corrected": torch.empty(n, dtype=torch.uint8, **kw),
           "token": torch.empty(n, dtype=torch.int32, **kw),
           "teacher_top1": torch.empty(n, dtype=torch.int32, **kw),
           "row_status": torch.empty(n, dtype=torch.int32, **kw)}
    for f in _FLOAT_FIELDS:
        out[f] = torch.empty(n, dtype=torch.float32, **kw)
    return out


def _out_struct(out: dict) -> SakiOut:
    so = SakiOut()
    for name, _ in SakiOut._fields_:
        t = out.get(name)
        setattr(so, name, t.data_ptr() if t is not None else None)
    return so


def _vec_check(v, dtype, n, dev, name):
    if v.dtype != dtype or v.shape != (n,) or v.device != dev or not v.is_contiguous():
        raise ValueError(f"{name} must be a contiguous {dtype} tensor of length N on the logits' device")
    return v


def _check_rows(s, t):
    if s.dim() != 2 or t.shape != s.shape or t.dtype != s.dtype or s.stride(1) != 1 or t.stride(1) != 1:
        raise SakiError(1, "student/teacher logits must be [N,V] of the same dtype with unit stride along V")


def _in_struct(s, t, proposal, mask, eps, temperature, seed, row_offset) -> SakiIn:
    si = SakiIn()
    si.student_logits, si.teacher_logits = s.data_ptr(), t.data_ptr()
    si.ld_s, si.ld_t = (s.stride(0) if s.shape[0] > 1 else s.shape[1]), (t.stride(0) if t.shape[0] > 1 else t.shape[1])
    si.N, si.V, si.dtype = s.shape[0], s.shape[1], _dtype_code(s)
    si.proposal = proposal.data_ptr()
    si.mask = mask.data_ptr() if mask is not None else None
    si.eps, si.temperature, si.seed, si.row_offset = eps, temperature, seed, row_offset
    return si


def route_fwd(s, t, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None, out=None, stream=None):
    """saki_route_fwd on device tensors; returns the dict of per-position output tensors."""
    lib = load_library()
    _check_rows(s, t)
    out = out if out is not None else _alloc_out(s.shape[0], s.device)
    si, so = _in_struct(s, t, proposal, mask, eps, temperature, seed, row_offset), _out_struct(out)
    _raise(lib, lib.saki_route_fwd(C.byref(si), C.byref(so), _stream_ptr(stream)))
    return out


def route_fwd_bwd(s, t, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None, grad_scale=1.0,
                  out=None, dlogits=None, stream=None):
    """saki_route_fwd_bwd on device tensors; returns (outputs dict, dlogits)."""
    lib = load_library()
    _check_rows(s, t)
    out = out if out is not None else _alloc_out(s.shape[0], s.device)
    if dlogits is None:
        dlogits = torch.empty_like(s)
    ld_g = dlogits.stride(0) if dlogits.shape[0] > 1 else dlogits.shape[1]
    si, so = _in_struct(s, t, proposal, mask, eps, temperature, seed, row_offset), _out_struct(out)
    _raise(lib, lib.saki_route_fwd_bwd(C.byref(si), C.byref(so), dlogits.data_ptr(), ld_g, grad_scale,
                                       _stream_ptr(stream)))
    return out, dlogits


def route_bwd_from_meta(s, corrected, proposal, teacher_top1, advantage, temperature=1.0, mask=None,
                        rollout_status=None, grad_scale=1.0, dlogits=None, stream=None):
    """saki_route_bwd_from_meta on device tensors: loss and gradient of the routed objective for the
    current student logits `s`, from the rollout's metadata.  Returns (outputs dict, dlogits)."""
    lib = load_library()
    if s.dim() != 2 or s.stride(1) != 1:
        raise ValueError("logits must be [N,V] with unit stride along V")
    n, dev = s.shape[0], s.device
    if dlogits is None:
        dlogits = torch.empty_like(s)
    ld_g = dlogits.stride(0) if dlogits.shape[0] > 1 else dlogits.shape[1]
    out = {"loss": torch.empty(n, dtype=torch.float32, device=dev),
           "logp_tok": torch.empty(n, dtype=torch.float32, device=dev),
           "row_status": torch.empty(n, dtype=torch.int32, device=dev)}
    keep = [_vec_check(corrected, torch.uint8, n, dev, "corrected"),
            _vec_check(proposal, torch.int32, n, dev, "proposal"),
            _vec_check(teacher_top1, torch.int32, n, dev, "teacher_top1"),
            _vec_check(advantage, torch.float32, n, dev, "advantage")]
    mi = SakiMetaIn()
    mi.student_logits = s.data_ptr()
    mi.ld_s = s.stride(0) if n > 1 else s.shape[1]
    mi.N, mi.V, mi.dtype = n, s.shape[1], _dtype_code(s)
    mi.corrected, mi.proposal, mi.teacher_top1, mi.advantage = (t.data_ptr() for t in keep)
    if mask is not None:
        keep.append(_vec_check(mask, torch.uint8, n, dev, "mask"))
        mi.mask = keep[-1].data_ptr()
    if rollout_status is not None:
        keep.append(_vec_check(rollout_status, torch.int32, n, dev, "rollout_status"))
        mi.rollout_status = keep[-1].data_ptr()
    mi.temperature = temperature
    mo = SakiMetaOut(out["loss"].data_ptr(), out["logp_tok"].data_ptr(), out["row_status"].data_ptr())
    _raise(lib, lib.saki_route_bwd_from_meta(C.byref(mi), C.byref(mo), dlogits.data_ptr(), ld_g, grad_scale,
                                             _stream_ptr(stream)))
    return out, dlogits


SELECT_RANDOM, SELECT_TV_WEIGHTED = 0, 1


def select_tm(seq_start, corrected, tv, mode, seed=0, row_offset=0, mask=None, rollout_status=None, stream=None):
    """saki_select_tm on device tensors: the placement controls (Random-TM, TV-Weighted-TM).  `seq_start`
    is the int64 [B+1] tensor of trajectory boundaries.  Returns (selected uint8 [N], m int32 [B])."""
    lib = load_library()
    dev = corrected.device
    n, nb = corrected.shape[0], seq_start.shape[0] - 1
    if seq_start.dtype != torch.int64 or seq_start.device != dev or not seq_start.is_contiguous():
        raise ValueError("seq_start must be a contiguous int64 tensor on the same device")
    keep = [_vec_check(corrected, torch.uint8, n, dev, "corrected")]
    si = SakiSelectIn()
    si.N, si.B, si.seq_start, si.corrected = n, nb, seq_start.data_ptr(), corrected.data_ptr()
    if tv is not None:
        keep.append(_vec_check(tv, torch.float32, n, dev, "tv"))
        si.tv = tv.data_ptr()
    if mask is not None:
        keep.append(_vec_check(mask, torch.uint8, n, dev, "mask"))
        si.mask = mask.data_ptr()
    if rollout_status is not None:
        keep.append(_vec_check(rollout_status, torch.int32, n, dev, "rollout_status"))
        si.rollout_status = rollout_status.data_ptr()
    si.mode, si.seed, si.row_offset = mode, seed, row_offset
    selected = torch.empty(n, dtype=torch.uint8, device=dev)
    m = torch.empty(max(nb, 0), dtype=torch.int32, device=dev)
    _raise(lib, lib.saki_select_tm(C.byref(si), selected.data_ptr(), m.data_ptr(), _stream_ptr(stream)))
    return selected, m


def route_fwd_bwd_noalloc(s, t, proposal, eps, out, dlogits, temperature=1.0, seed=0, row_offset=0, mask=None,
                          grad_scale=1.0, stream=None):
    """saki_route_fwd_bwd_noalloc: the variant for callers that cannot allocate device memory.  The caller
    passes every buffer (`out`: dict of preallocated output tensors, `dlogits`); the library's own scratch
    is a fixed device array, so nothing is allocated on the way (at most 1,048,576 rows per call)."""
    lib = load_library()
    _check_rows(s, t)
    ld_g = dlogits.stride(0) if dlogits.shape[0] > 1 else dlogits.shape[1]
    si, so = _in_struct(s, t, proposal, mask, eps, temperature, seed, row_offset), _out_struct(out)
    _raise(lib, lib.saki_route_fwd_bwd_noalloc(C.byref(si), C.byref(so), dlogits.data_ptr(), ld_g, grad_scale,
                                               _stream_ptr(stream)))
    return out, dlogits


def vshard_in(s_loc, t_loc, v0, V, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None, rank=0, world=1,
              dtype=None, n_rows=None) -> SakiVshardIn:
    """The argument record of the vocabulary-sharded calls: this rank's columns [v0, v0 + V_local) of both logit
    tensors.  `s_loc` / `t_loc` may be None for the host-side combine (which reads no logits); then `dtype`
    ("bf16" / "f32") and `n_rows` say what the slices hold."""
    si = SakiVshardIn()
    if s_loc is not None:
        si.student_logits, si.teacher_logits = s_loc.data_ptr(), t_loc.data_ptr()
        si.ld_s = s_loc.stride(0) if s_loc.shape[0] > 1 else max(1, s_loc.shape[1])
        si.ld_t = t_loc.stride(0) if t_loc.shape[0] > 1 else max(1, t_loc.shape[1])
        si.N, si.V_local, si.dtype = s_loc.shape[0], s_loc.shape[1], _dtype_code(s_loc)
    else:
        si.N, si.V_local, si.dtype = n_rows, 0, (SAKI_BF16 if dtype == "bf16" else SAKI_F32)
    si.V, si.v0 = V, v0
    si.proposal = proposal.data_ptr()
    si.mask = mask.data_ptr() if mask is not None else None
    si.eps, si.temperature, si.seed, si.row_offset = eps, temperature, seed, row_offset
    si.rank, si.world = rank, world
    return si


def vshard_partial(si: SakiVshardIn, stage: int, state, partial, dlogits=None, grad_scale=1.0, stream=None):
    """saki_vshard_partial: this rank's partial vectors of one stage (device tensors, float64)."""
    lib = load_library()
    ld_g = 0
    if dlogits is not None:
        ld_g = dlogits.stride(0) if dlogits.shape[0] > 1 else max(1, dlogits.shape[1])
    _raise(lib, lib.saki_vshard_partial(C.byref(si), stage, state.data_ptr() if state is not None else None,
                                        partial.data_ptr(), dlogits.data_ptr() if dlogits is not None else None, ld_g,
                                        grad_scale, _stream_ptr(stream)))


def vshard_combine(si: SakiVshardIn, stage: int, gathered, state, out=None, n_solving=None, stream=None):
    """saki_vshard_combine: folds the gathered partials [world, N, 16] into the per-row state (device tensors)."""
    lib = load_library()
    so = _out_struct(out) if out is not None else None
    _raise(lib, lib.saki_vshard_combine(C.byref(si), stage, gathered.data_ptr(), state.data_ptr(),
                                        C.byref(so) if so is not None else None,
                                        n_solving.data_ptr() if n_solving is not None else None, _stream_ptr(stream)))


def vshard_combine_host(si: SakiVshardIn, stage: int, gathered, state, out=None) -> int:
    """saki_vshard_combine_host: the same combine on host tensors; returns the number of rows still solving."""
    lib = load_library()
    so = _out_struct(out) if out is not None else None
    n = C.c_int32(0)
    _raise(lib, lib.saki_vshard_combine_host(C.byref(si), stage, gathered.data_ptr(), state.data_ptr(),
                                             C.byref(so) if so is not None else None, C.byref(n)))
    return int(n.value)


def lmhead_lse(hidden, weight, temperature=1.0, logits=None, scratch=None, stream=None):
    """saki_lmhead_lse: logits = hidden @ weight.T (bf16 in, fp32 accumulation, bf16 out) with each row's maximum and
    log-sum-exp (of the stored bf16 values / temperature) from the GEMM's epilogue.  hidden [N, d], weight [V, d] on
    the GPU.  Returns (logits, row_max, lse)."""
    lib = load_library()
    if hidden.dtype != torch.bfloat16 or weight.dtype != torch.bfloat16 or hidden.shape[1] != weight.shape[1]:
        raise ValueError("hidden [N, d] and weight [V, d] must be bf16 with the same d")
    if hidden.stride(1) != 1 or weight.stride(1) != 1:
        raise ValueError("hidden and weight need unit stride along d")
    N, d = hidden.shape
    V = weight.shape[0]
    dev = hidden.device
    logits = logits if logits is not None else torch.empty((N, V), dtype=torch.bfloat16, device=dev)
    need = int(lib.saki_lmhead_scratch_bytes(N, V))
    if scratch is None or scratch.numel() * scratch.element_size() < need:
        scratch = torch.empty(need, dtype=torch.uint8, device=dev)
    row_max = torch.empty(N, dtype=torch.float32, device=dev)
    lse = torch.empty(N, dtype=torch.float32, device=dev)
    li = SakiLmheadIn()
    li.hidden, li.ld_h = hidden.data_ptr(), (hidden.stride(0) if N > 1 else d)
    li.weight, li.ld_w = weight.data_ptr(), (weight.stride(0) if V > 1 else d)
    li.N, li.d, li.V, li.temperature = N, d, V, temperature
    ld_l = logits.stride(0) if N > 1 else V
    _raise(lib, lib.saki_lmhead_lse(C.byref(li), logits.data_ptr(), ld_l, row_max.data_ptr(), lse.data_ptr(),
                                    scratch.data_ptr(), scratch.numel() * scratch.element_size(), _stream_ptr(stream)))
    return logits, row_max, lse


def route_host(s, t, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None, grad_scale=1.0,
               backward=True, out=None, dlogits=None):
    """saki_route_host: every tensor lives in HOST memory (pinned for full copy speed); the library
    stages the rows through the GPU and returns when the host outputs are complete."""
    lib = load_library()
    _check_rows(s, t)
    if s.is_cuda:
        raise SakiError(1, "route_host takes host tensors")
    out = out if out is not None else _alloc_out(s.shape[0], "cpu", pinned=True)
    if backward and dlogits is None:
        dlogits = torch.empty(s.shape, dtype=s.dtype, pin_memory=True)
    ld_g = (dlogits.stride(0) if dlogits.shape[0] > 1 else dlogits.shape[1]) if backward else 0
    si, so = _in_struct(s, t, proposal, mask, eps, temperature, seed, row_offset), _out_struct(out)
    _raise(lib, lib.saki_route_host(C.byref(si), C.byref(so), dlogits.data_ptr() if backward else None, ld_g,
                                    grad_scale))
    return out, dlogits


def spec_verify(s, t, draft, eps, temperature=1.0, seed=0, seq_offset=0, stream=None):
    """saki_spec_verify on device tensors s, t: [B,K+1,V], draft: [B,K] int32."""
    lib = load_library()
    if s.dim() != 3 or t.shape != s.shape or t.dtype != s.dtype or s.stride(2) != 1 or t.stride(2) != 1:
        raise SakiError(1, "logits must be [B,K+1,V] with unit stride along V")
    B, K1, V = s.shape
    per = _alloc_out(B * K1, s.device)
    res = {"n_accept": torch.empty(B, dtype=torch.int32, device=s.device),
           "next_token": torch.empty(B, dtype=torch.int32, device=s.device),
           "next_is_correction": torch.empty(B, dtype=torch.uint8, device=s.device), "per_pos": per}
    si = SakiSpecIn()
    si.student_logits, si.teacher_logits = s.data_ptr(), t.data_ptr()
    si.ss_seq, si.ss_pos, si.ts_seq, si.ts_pos = s.stride(0), s.stride(1), t.stride(0), t.stride(1)
    si.B, si.K, si.V, si.dtype = B, K1 - 1, V, _dtype_code(s)
    si.draft, si.draft_ld = draft.data_ptr(), (draft.stride(0) if B > 1 else draft.shape[1])
    si.eps, si.temperature, si.seed, si.seq_offset = eps, temperature, seed, seq_offset
    so = SakiSpecOut()
    so.n_accept, so.next_token, so.next_is_correction = (res["n_accept"].data_ptr(), res["next_token"].data_ptr(),
                                                        res["next_is_correction"].data_ptr())
    so.per_pos = _out_struct(per)
    _raise(lib, lib.saki_spec_verify(C.byref(si), C.byref(so), _stream_ptr(stream)))
    return res


def sample_proposal(s, temperature=1.0, seed=0, row_offset=0, stream=None):
    """saki_sample_proposal: x_i ~ softmax(s_i / temperature) by Philox-keyed Gumbel-max."""
    lib = load_library()
    out = torch.empty(s.shape[0], dtype=torch.int32, device=s.device)
    ld = s.stride(0) if s.shape[0] > 1 else s.shape[1]
    _raise(lib, lib.saki_sample_proposal(s.data_ptr(), ld, s.shape[0], s.shape[1], _dtype_code(s), temperature,
                                         seed, row_offset, out.data_ptr(), _stream_ptr(stream)))
    return out


def check(stream=None) -> int:
    """saki_check: synchronises the stream and returns the number of rows flagged since the last check."""
    lib = load_library()
    n = C.c_uint64(0)
    rc = lib.saki_check(_stream_ptr(stream), C.byref(n))
    if rc not in (0, 4):
        _raise(lib, rc)
    return int(n.value)


def set_kernel(which: int) -> int:
    """saki_set_kernel: 0 automatic, 1 general (float64), 2 cluster, 3 row-per-SM; returns the previous choice."""
    return load_library().saki_set_kernel(which)


def last_kernel() -> int:
    """The kernel that served the calling thread's last routing call: 1 general (float64), 2 cluster, 3 row-per-SM,
    4 the streaming kernel of route_bwd_from_meta."""
    return load_library().saki_last_kernel()


def redo_count(stream=None) -> int:
    """Rows of the last routing call that the float32 kernel handed to the float64 kernel (synchronises)."""
    lib = load_library()
    n = C.c_uint64(0)
    _raise(lib, lib.saki_redo_count(_stream_ptr(stream), C.byref(n)))
    return int(n.value)


def solve_evaluations(stream=None) -> int:
    """Evaluation passes of the row-per-SM kernel in the last routing call, over all rows (synchronises)."""
    lib = load_library()
    n = C.c_uint64(0)
    _raise(lib, lib.saki_solve_evaluations(_stream_ptr(stream), C.byref(n)))
    return int(n.value)


PHASES = ("row_top", "copy_wait", "lse", "lse_reduce", "lse_gather", "lse_scalar", "solve_top", "solve",
          "solve_combine", "solve_scalar", "final_top", "final", "row_end", "tail", "spare", "rows")


def set_wait_limit(cycles: int) -> int:
    """SM cycles a block of the row-per-SM kernel waits for a row's bulk copy before it flags its rows TIMEOUT
    (0: the default of about two seconds); returns the previous setting."""
    return int(load_library().saki_set_wait_limit(int(cycles)))


def set_phase_clock(on: bool) -> bool:
    """Phase clock of the row-per-SM kernel for the calls that follow (default off); returns the previous setting."""
    return bool(load_library().saki_set_phase_clock(1 if on else 0))


def phase_cycles(stream=None) -> dict:
    """SM cycles per phase of the row-per-SM kernel's row loop in the last routing call, summed over thread
    blocks, and the number of rows behind them (synchronises)."""
    lib = load_library()
    buf = (C.c_uint64 * len(PHASES))()
    _raise(lib, lib.saki_phase_cycles(_stream_ptr(stream), buf))
    return {k: int(v) for k, v in zip(PHASES, buf)}


def set_spec_early_out(on: bool) -> bool:
    """Early out of block verification on the row-per-SM kernel (default on); returns the previous setting."""
    return bool(load_library().saki_set_spec_early_out(1 if on else 0))


def spec_positions_routed(stream=None) -> int:
    """Positions the last spec_verify actually routed under early out (synchronises); 0 without early out."""
    lib = load_library()
    n = C.c_uint64(0)
    _raise(lib, lib.saki_spec_positions_routed(_stream_ptr(stream), C.byref(n)))
    return int(n.value)


def launch_count() -> int:
    return int(load_library().saki_launch_count())


def last_error() -> str:
    return load_library().saki_last_error().decode()


def version() -> int:
    return load_library().saki_version()
