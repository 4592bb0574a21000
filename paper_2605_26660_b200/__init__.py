"""Python binding of the windq CUDA library (argument marshalling only).

Every function below has the name of the C-ABI entry point it calls
(``include/windq.h``) and does nothing but check tensor types, allocate output
tensors with torch, pass raw device pointers and the current CUDA stream, and
turn a non-zero status into ``WindqError``.  All arithmetic happens in the CUDA
kernels.  There is no CPU fallback: if the shared library is missing and cannot
be built, importing this package raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

N_BITWIDTHS = 6     # columns of per-bit-width tables: 8, 4, 3, 2, 1.58, 1
N_FEATURES = 8
ACTION_BITS = (16.0, 8.0, 4.0, 3.0, 2.0, 1.58, 1.0)   # action code -> nominal bits (Eq. 3)

STATUS_NAMES = {0: "OK", 1: "ERR_NULL", 2: "ERR_SHAPE", 3: "ERR_ALIGN", 4: "ERR_ARG", 5: "ERR_SCRATCH",
                6: "ERR_CUDA", 7: "ERR_UNSUPPORTED"}


class WindqError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("windq status %d (%s): %s" % (status, STATUS_NAMES.get(status, "?"), message))
        self.status = status


def _load() -> ctypes.CDLL:
    try:
        path = _build.build()
    except Exception as exc:  # no nvcc, or a compile error
        if os.path.exists(_build.LIB):
            path = _build.LIB   # a library built elsewhere travelled with the tree
        else:
            raise ImportError("the windq CUDA library is not built and cannot be built here: %s" % exc) from exc
    lib = ctypes.CDLL(path)
    i64, i32, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
    lib.windq_create.argtypes = [ctypes.POINTER(vp), i32]
    lib.windq_destroy.argtypes = [vp]
    lib.windq_destroy.restype = None
    lib.windq_last_error.argtypes = [vp]
    lib.windq_last_error.restype = ctypes.c_char_p
    lib.windq_reserve.argtypes = [vp, i64]
    lib.windq_selfcheck.argtypes = [vp, vp, vp]
    lib.windq_fit_work.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), i32]
    for name in ("windq_scratch_bytes_act_stats",):
        getattr(lib, name).argtypes = [i64, i64]
        getattr(lib, name).restype = i64
    for name in ("windq_scratch_bytes_unit_features", "windq_scratch_bytes_fit_eval", "windq_scratch_bytes_salient_select"):
        getattr(lib, name).argtypes = [i64, i64, i32]
        getattr(lib, name).restype = i64
    lib.windq_act_stats.argtypes = [vp, vp, i64, i64, i64, vp, vp]
    lib.windq_act_stats_noalloc.argtypes = [vp, vp, i64, i64, i64, vp, vp]
    lib.windq_act_stats_batch.argtypes = [vp, vp, i32, vp]
    lib.windq_scratch_bytes_act_stats_batch.restype = i64
    lib.windq_scratch_bytes_act_stats_batch.argtypes = [vp, i32]
    lib.windq_unit_features.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp]
    lib.windq_fit_eval.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.windq_apply_plan_batch.argtypes = [vp, vp, i32, i32, vp, i32, vp]
    lib.windq_effective_bits_batch.argtypes = [vp, vp, i32, i32, i32, i32, vp]
    lib.windq_unit_features_batch.argtypes = [vp, vp, i32, i32, vp]
    lib.windq_unit_features_batch2.argtypes = [vp, vp, vp, i32, i32, vp]
    lib.windq_scratch_bytes_unit_features_batch.restype = i64
    lib.windq_scratch_bytes_unit_features_batch.argtypes = [vp, i32, i32]
    lib.windq_fit_eval_batch.argtypes = [vp, vp, i32, i32, vp, i32, vp]
    lib.windq_features_fit_batch.argtypes = [vp, vp, i32, i32, vp, i32, vp]
    lib.windq_scratch_bytes_features_fit_batch.restype = i64
    lib.windq_scratch_bytes_features_fit_batch.argtypes = [vp, i32, i32]
    lib.windq_scratch_bytes_fit_eval_batch.restype = i64
    lib.windq_scratch_bytes_fit_eval_batch.argtypes = [vp, i32, i32]
    lib.windq_fit_eval_protected.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.windq_scratch_bytes_fit_eval_protected.argtypes = [i64, i64, i32]
    lib.windq_scratch_bytes_fit_eval_protected.restype = i64
    lib.windq_effective_bits.argtypes = [vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.windq_salient_select.argtypes = [vp, vp, i64, i64, i64, i32, vp, i64, vp, vp, vp, vp]
    lib.windq_effective_bits_protected.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp, vp]
    lib.windq_apply_plan_protected.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp]
    lib.windq_scratch_bytes_apply_plan_protected.argtypes = [i64, i64, i32]
    lib.windq_scratch_bytes_apply_plan_protected.restype = i64
    lib.windq_unit_saliency.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp]
    lib.windq_fallback.argtypes = [vp, vp, vp, vp, i64, ctypes.c_float, vp, vp, vp]
    lib.windq_apply_plan_refined.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.windq_apply_plan_protected_refined.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp]
    lib.windq_fit_refine_protected.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, i32, ctypes.c_float, vp, vp, vp, vp]
    lib.windq_fit_refine.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, i32, ctypes.c_float, vp, vp, vp, vp]
    lib.windq_scratch_bytes_fit_refine.restype = i64
    lib.windq_scratch_bytes_fit_refine.argtypes = [i64, i64, i32]
    lib.windq_greedy_allocate.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, vp, vp, vp]
    lib.windq_scratch_bytes_greedy_allocate.restype = i64
    lib.windq_scratch_bytes_greedy_allocate.argtypes = [i64]
    lib.windq_apply_plan.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.windq_apply_plan_multi.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, i32, vp]
    lib.windq_apply_plan_searched.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.windq_fit_ternary_search.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.windq_scratch_bytes_fit_ternary_search.argtypes = [i64, i64, i32]
    lib.windq_scratch_bytes_fit_ternary_search.restype = i64
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _need(t: torch.Tensor, dtype, name: str, dims=None):
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (name, dtype, t.dtype))
    if dims is not None and t.dim() != dims:
        raise ValueError("%s must have %d dimensions" % (name, dims))
    return t


def _matrix(t: torch.Tensor, name: str):
    _need(t, torch.float16, name, 2)
    if t.stride(1) != 1:
        raise ValueError("%s must be row-major (unit stride along columns)" % name)
    return t.shape[0], t.shape[1], t.stride(0)


class Context:
    """Owns a ``windq_ctx`` on one CUDA device."""

    def __init__(self, device: int | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.device = int(device)
        self._h = ctypes.c_void_p()
        st = _lib.windq_create(ctypes.byref(self._h), self.device)
        if st:
            raise WindqError(st, _lib.windq_last_error(None).decode())

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            _lib.windq_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st:
            raise WindqError(st, _lib.windq_last_error(self._h).decode())

    def reserve(self, nbytes: int):
        self._check(_lib.windq_reserve(self._h, int(nbytes)))


def windq_create(device: int | None = None) -> Context:
    return Context(device)


def windq_destroy(ctx: Context) -> None:
    ctx.close()


def windq_selfcheck(ctx: Context, stream=None) -> int:
    """Number of fp16 scale values for which the fits' fast reciprocal differs from IEEE division (0 is expected)."""
    out = torch.zeros(1, dtype=torch.int64, device=torch.device("cuda", ctx.device))
    ctx._check(_lib.windq_selfcheck(ctx._h, _ptr(out), _stream(stream)))
    return int(out.item())


def windq_reserve(ctx: Context, nbytes: int) -> None:
    ctx.reserve(nbytes)


def windq_fit_work(ctx: Context, reset: bool = False):
    """(clip candidates evaluated in full, clip candidates searched) by the fits of this context since the counters
    were last reset, counted once per warp pass.  Synchronises the device."""
    a, b = ctypes.c_int64(0), ctypes.c_int64(0)
    ctx._check(_lib.windq_fit_work(ctx._h, ctypes.byref(a), ctypes.byref(b), 1 if reset else 0))
    return int(a.value), int(b.value)


def windq_scratch_bytes_act_stats(T: int, C: int) -> int:
    return int(_lib.windq_scratch_bytes_act_stats(T, C))


def windq_scratch_bytes_unit_features(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_unit_features(R, C, G))


def windq_scratch_bytes_fit_eval(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_fit_eval(R, C, G))


def windq_act_stats(ctx: Context, X: torch.Tensor, s_out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """s[j] = mean_t X[t, j]^2.  X: fp16 [T, C]; returns fp32 [C]."""
    T, C, ldx = _matrix(X, "X")
    if s_out is None:
        s_out = torch.empty(C, dtype=torch.float32, device=X.device)
    _need(s_out, torch.float32, "s_out", 1)
    ctx._check(_lib.windq_act_stats(ctx._h, _ptr(X), T, C, ldx, _ptr(s_out), _stream(stream)))
    return s_out


MAX_ACT_JOBS = 16   # WINDQ_MAX_ACT_JOBS of the header


class _ActJob(ctypes.Structure):
    _fields_ = [("X", ctypes.c_void_p), ("T", ctypes.c_int64), ("C", ctypes.c_int64), ("ldx", ctypes.c_int64),
                ("s_out", ctypes.c_void_p)]


def windq_act_stats_batch(ctx: Context, Xs, s_outs=None, stream=None):
    """windq_act_stats of up to 16 inputs in one launch.  ``s_outs`` may hold one preallocated fp32 [C] tensor
    per input.  Returns the list of statistics."""
    if not Xs:
        raise ValueError("Xs must be non-empty")
    if s_outs is not None and len(s_outs) != len(Xs):
        raise ValueError("s_outs must have one entry per input")
    jobs = (_ActJob * len(Xs))()
    outs = []
    for j, X in enumerate(Xs):
        T, C, ldx = _matrix(X, "X")
        s = s_outs[j] if s_outs is not None else torch.empty(C, dtype=torch.float32, device=X.device)
        _need(s, torch.float32, "s_out", 1)
        if s.numel() < C:
            raise ValueError("s_out must have at least C entries")
        jobs[j] = _ActJob(X.data_ptr(), T, C, ldx, s.data_ptr())
        outs.append(s)
    ctx._check(_lib.windq_act_stats_batch(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), len(Xs), _stream(stream)))
    return outs


def windq_scratch_bytes_act_stats_batch(shapes) -> int:
    """Scratch of a windq_act_stats_batch call over inputs of the given (T, C) shapes."""
    jobs = (_ActJob * len(shapes))()
    for j, (T, C) in enumerate(shapes):
        jobs[j] = _ActJob(None, int(T), int(C), int(C), None)
    return int(_lib.windq_scratch_bytes_act_stats_batch(ctypes.cast(jobs, ctypes.c_void_p), len(shapes)))


NOALLOC_SCRATCH_BYTES = 4 * 1024 * 1024   # WINDQ_NOALLOC_SCRATCH_BYTES of the header


def windq_act_stats_noalloc(ctx: Context, X: torch.Tensor, s_out: torch.Tensor, stream=None) -> torch.Tensor:
    """windq_act_stats for callers that must not allocate device memory: the partial sums live in
    an array built into the library, so neither the library nor this wrapper allocates anything.
    ``s_out`` (fp32 [C]) is therefore required.  Shapes that need more than NOALLOC_SCRATCH_BYTES
    (4 * C * ceil(T / 64) bytes) raise WindqError with status ERR_SCRATCH.  Calls that can overlap
    on the GPU share that array and must be ordered by the caller."""
    T, C, ldx = _matrix(X, "X")
    _need(s_out, torch.float32, "s_out", 1)
    if s_out.numel() < C:
        raise ValueError("s_out must have at least C entries")
    ctx._check(_lib.windq_act_stats_noalloc(ctx._h, _ptr(X), T, C, ldx, _ptr(s_out), _stream(stream)))
    return s_out


def windq_unit_features(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, feat_out: torch.Tensor | None = None,
                        stream=None) -> torch.Tensor:
    """Table 1 features per unit.  Returns fp32 [U, 8]."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    if feat_out is None:
        feat_out = torch.empty((max(C // max(G, 1), 0), N_FEATURES), dtype=torch.float32, device=W.device)
    _need(feat_out, torch.float32, "feat_out", 2)
    ctx._check(_lib.windq_unit_features(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(feat_out), _stream(stream)))
    return feat_out


def windq_fit_eval(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor, *,
                   want_energy: bool = True, want_clip_idx: bool = True, want_group_err: bool = False,
                   out: dict | None = None, stream=None, thresh: torch.Tensor | None = None) -> dict:
    """Fits every group under all six bit-widths.  With ``thresh`` (fp32 [U], from windq_salient_select) the
    call is windq_fit_eval_protected: the salient weights are left out of the fits.

    Returns dict(err [U,6] f32, energy [U] f32 | None, clip_idx [4,U,R] u8 | None,
    group_err [6,U,R] f32 | None).  ``out`` may hold preallocated tensors under the same keys.
    """
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(clip_grid, torch.float32, "clip_grid", 1)
    U = C // G if G > 0 else 0
    out = dict(out) if out else {}
    dev = W.device
    if out.get("err") is None:
        out["err"] = torch.empty((U, N_BITWIDTHS), dtype=torch.float32, device=dev)
    if want_energy and out.get("energy") is None:
        out["energy"] = torch.empty(U, dtype=torch.float32, device=dev)
    if want_clip_idx and out.get("clip_idx") is None:
        out["clip_idx"] = torch.empty((4, U, R), dtype=torch.uint8, device=dev)
    if want_group_err and out.get("group_err") is None:
        out["group_err"] = torch.empty((N_BITWIDTHS, U, R), dtype=torch.float32, device=dev)
    for key in ("energy", "clip_idx", "group_err"):
        out.setdefault(key, None)
    if thresh is None:
        ctx._check(_lib.windq_fit_eval(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                       _ptr(out["err"]), _ptr(out["energy"]), _ptr(out["clip_idx"]), _ptr(out["group_err"]),
                                       _stream(stream)))
    else:
        _need(thresh, torch.float32, "thresh", 1)
        if thresh.numel() != U:
            raise ValueError("thresh must have one entry per unit")
        ctx._check(_lib.windq_fit_eval_protected(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid),
                                                 clip_grid.numel(), _ptr(thresh), _ptr(out["err"]), _ptr(out["energy"]),
                                                 _ptr(out["clip_idx"]), _ptr(out["group_err"]), _stream(stream)))
    return out


class _ApplyJob(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("R", ctypes.c_int64), ("C", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("s", ctypes.c_void_p), ("actions", ctypes.c_void_p), ("clip_idx", ctypes.c_void_p),
                ("code_offsets", ctypes.c_void_p), ("codes_out", ctypes.c_void_p), ("scales_out", ctypes.c_void_p),
                ("zeros_out", ctypes.c_void_p), ("Wq_out", ctypes.c_void_p)]


def windq_apply_plan_batch(ctx: Context, jobs, G: int, clip_grid: torch.Tensor, *, stream=None) -> list:
    """windq_apply_plan of up to 24 (matrix, plan) pairs in one launch.  ``jobs``: a sequence of dicts with the keys
    W, s, actions, clip_idx, code_offsets, codes (uint8 output, sized by the caller) and optionally scales, zeros
    ([U, R] fp16) and wq ([R, C] fp16 with the row stride of W, or None for no fake-quantised output; absent = allocated).
    Returns one dict(codes, scales, zeros, wq) per job."""
    if not jobs:
        raise ValueError("jobs must not be empty")
    _need(clip_grid, torch.float32, "clip_grid", 1)
    arr = (_ApplyJob * len(jobs))()
    results = []
    for j, job in enumerate(jobs):
        W, s, actions, clip_idx = job["W"], job["s"], job["actions"], job["clip_idx"]
        R, C, ldw = _matrix(W, "W")
        _need(s, torch.float32, "s", 1)
        _need(actions, torch.uint8, "actions", 1)
        _need(clip_idx, torch.uint8, "clip_idx", 3)
        _need(job["code_offsets"], torch.int64, "code_offsets", 1)
        _need(job["codes"], torch.uint8, "codes", 1)
        U = C // G if G > 0 else 0
        if actions.numel() != U or job["code_offsets"].numel() != U + 1 or tuple(clip_idx.shape) != (4, U, R) \
                or not clip_idx.is_contiguous():
            raise ValueError("job %d: actions [U], code_offsets [U + 1] and a contiguous clip_idx [4, U, R] are needed" % j)
        dev = W.device
        scales = job.get("scales")
        zeros = job.get("zeros")
        if scales is None:
            scales = torch.empty((U, R), dtype=torch.float16, device=dev)
        if zeros is None:
            zeros = torch.empty((U, R), dtype=torch.float16, device=dev)
        wq_out = job["wq"] if "wq" in job else torch.empty_strided((R, C), (ldw, 1), dtype=torch.float16, device=dev)
        if wq_out is not None and (_matrix(wq_out, "wq")[2] != ldw or wq_out.shape != W.shape):
            raise ValueError("job %d: wq must have the shape and row stride of W" % j)
        arr[j] = _ApplyJob(W.data_ptr(), R, C, ldw, s.data_ptr(), actions.data_ptr(), clip_idx.data_ptr(),
                           job["code_offsets"].data_ptr(), job["codes"].data_ptr(), scales.data_ptr(), zeros.data_ptr(),
                           None if wq_out is None else wq_out.data_ptr())
        results.append(dict(codes=job["codes"], scales=scales, zeros=zeros, wq=wq_out))
    ctx._check(_lib.windq_apply_plan_batch(ctx._h, ctypes.cast(arr, ctypes.c_void_p), len(jobs), int(G), _ptr(clip_grid),
                                           clip_grid.numel(), _stream(stream)))
    return results


class _BitsJob(ctypes.Structure):
    _fields_ = [("actions", ctypes.c_void_p), ("U", ctypes.c_int64), ("R", ctypes.c_int64),
                ("unit_centibits_out", ctypes.c_void_p), ("code_offsets_out", ctypes.c_void_p),
                ("total_centibits_out", ctypes.c_void_p), ("total_packed_bytes_out", ctypes.c_void_p)]


def windq_effective_bits_batch(ctx: Context, actions_list, Rs, G: int, scale_bits: int = 16, zero_bits: int = 16,
                               outs=None, stream=None) -> list:
    """windq_effective_bits of up to 32 plans in one launch.  ``actions_list``: one u8 tensor per plan; ``Rs``: the
    row count of each plan's matrix.  ``outs`` may hold one dict of preallocated outputs per plan (keys as
    windq_effective_bits; a key that is present with value None is not computed).  Returns the list of dicts."""
    if len(actions_list) != len(Rs) or not actions_list:
        raise ValueError("actions_list and Rs must be non-empty and equally long")
    jobs = (_BitsJob * len(actions_list))()
    results = []
    for j, (acts, R) in enumerate(zip(actions_list, Rs)):
        _need(acts, torch.uint8, "actions", 1)
        U = acts.numel()
        out = dict(outs[j]) if outs else {}
        dev = acts.device
        if "unit_centibits" not in out:
            out["unit_centibits"] = torch.empty(U, dtype=torch.int64, device=dev)
        if "code_offsets" not in out:
            out["code_offsets"] = torch.empty(U + 1, dtype=torch.int64, device=dev)
        if out.get("total_centibits") is None:
            out["total_centibits"] = torch.empty(1, dtype=torch.int64, device=dev)
        if "total_packed_bytes" not in out:
            out["total_packed_bytes"] = torch.empty(1, dtype=torch.int64, device=dev)
        ptr = lambda x: None if x is None else x.data_ptr()
        jobs[j] = _BitsJob(acts.data_ptr(), U, int(R), ptr(out["unit_centibits"]), ptr(out["code_offsets"]),
                           ptr(out["total_centibits"]), ptr(out["total_packed_bytes"]))
        results.append(out)
    ctx._check(_lib.windq_effective_bits_batch(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), len(actions_list), int(G),
                                               int(scale_bits), int(zero_bits), _stream(stream)))
    return results


class _FeatJob(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("R", ctypes.c_int64), ("C", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("s", ctypes.c_void_p), ("feat_out", ctypes.c_void_p)]


def windq_unit_features_batch(ctx: Context, Ws, G: int, ss, feats=None, stream=None, feats_2G=None):
    """windq_unit_features of up to 16 matrices in one pass.  ``feats`` may hold one preallocated [U, 8] fp32
    tensor per matrix.  Returns the list of feature tensors.

    With ``feats_2G`` (True, or a list with one preallocated [U / 2, 8] tensor or None per matrix) the call is
    windq_unit_features_batch2: the features at chunk width 2 G come out of the same pass, and the result is
    (features at G, features at 2 G)."""
    if len(Ws) != len(ss) or not Ws:
        raise ValueError("Ws and ss must be non-empty and equally long")
    jobs = (_FeatJob * len(Ws))()
    outs, outs2 = [], []
    wide = (ctypes.c_void_p * len(Ws))()
    for j, (W, s) in enumerate(zip(Ws, ss)):
        R, C, ldw = _matrix(W, "W")
        _need(s, torch.float32, "s", 1)
        U = C // G if G > 0 else 0
        f = feats[j] if feats is not None else torch.empty((U, N_FEATURES), dtype=torch.float32, device=W.device)
        _need(f, torch.float32, "feat_out", 2)
        if tuple(f.shape) != (U, N_FEATURES) or not f.is_contiguous():
            raise ValueError("feat_out must be a contiguous [U, 8] tensor")
        jobs[j] = _FeatJob(W.data_ptr(), R, C, ldw, s.data_ptr(), f.data_ptr())
        outs.append(f)
        if feats_2G is not None:
            f2 = torch.empty((U // 2, N_FEATURES), dtype=torch.float32, device=W.device) if feats_2G is True else feats_2G[j]
            if f2 is not None:
                _need(f2, torch.float32, "feat_out_2G", 2)
                if tuple(f2.shape) != (U // 2, N_FEATURES) or not f2.is_contiguous():
                    raise ValueError("feat_out_2G must be a contiguous [U / 2, 8] tensor")
            wide[j] = None if f2 is None else f2.data_ptr()
            outs2.append(f2)
    if feats_2G is None:
        ctx._check(_lib.windq_unit_features_batch(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), len(Ws), int(G), _stream(stream)))
        return outs
    ctx._check(_lib.windq_unit_features_batch2(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), ctypes.cast(wide, ctypes.c_void_p),
                                               len(Ws), int(G), _stream(stream)))
    return outs, outs2


class _FitJob(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("R", ctypes.c_int64), ("C", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("s", ctypes.c_void_p), ("err_out", ctypes.c_void_p), ("energy_out", ctypes.c_void_p),
                ("clip_idx_out", ctypes.c_void_p), ("group_err_out", ctypes.c_void_p), ("lowbit_out", ctypes.c_void_p)]


def windq_fit_eval_batch(ctx: Context, Ws, G: int, ss, clip_grid: torch.Tensor, *, want_energy: bool = True,
                         want_clip_idx: bool = True, want_group_err: bool = False, want_lowbit: bool = False, outs=None,
                         stream=None) -> list:
    """windq_fit_eval of up to 16 matrices in one launch.  ``Ws`` and ``ss`` are equally long sequences of weight
    matrices and their statistics; ``outs`` may hold one dict of preallocated outputs per matrix (keys as
    windq_fit_eval, and ``lowbit``: fp16 [3, U, R], the parameters of the two low-bit fits that
    windq_apply_plan_multi can take).  Returns the list of output dicts."""
    if len(Ws) != len(ss) or not Ws:
        raise ValueError("Ws and ss must be non-empty and equally long")
    _need(clip_grid, torch.float32, "clip_grid", 1)
    jobs = (_FitJob * len(Ws))()
    results = []
    for j, (W, s) in enumerate(zip(Ws, ss)):
        R, C, ldw = _matrix(W, "W")
        _need(s, torch.float32, "s", 1)
        U = C // G if G > 0 else 0
        out = dict(outs[j]) if outs else {}
        dev = W.device
        if out.get("err") is None:
            out["err"] = torch.empty((U, N_BITWIDTHS), dtype=torch.float32, device=dev)
        if want_energy and out.get("energy") is None:
            out["energy"] = torch.empty(U, dtype=torch.float32, device=dev)
        if want_clip_idx and out.get("clip_idx") is None:
            out["clip_idx"] = torch.empty((4, U, R), dtype=torch.uint8, device=dev)
        if want_group_err and out.get("group_err") is None:
            out["group_err"] = torch.empty((N_BITWIDTHS, U, R), dtype=torch.float32, device=dev)
        if want_lowbit and out.get("lowbit") is None:
            out["lowbit"] = torch.empty((3, U, R), dtype=torch.float16, device=dev)
        for key in ("energy", "clip_idx", "group_err", "lowbit"):
            out.setdefault(key, None)
        if out["lowbit"] is not None and (tuple(out["lowbit"].shape) != (3, U, R) or not out["lowbit"].is_contiguous()
                                          or out["lowbit"].dtype != torch.float16):
            raise ValueError("lowbit must be a contiguous fp16 [3, U, R] tensor")
        ptr = lambda x: None if x is None else x.data_ptr()
        jobs[j] = _FitJob(W.data_ptr(), R, C, ldw, s.data_ptr(), ptr(out["err"]), ptr(out["energy"]), ptr(out["clip_idx"]),
                          ptr(out["group_err"]), ptr(out["lowbit"]))
        results.append(out)
    ctx._check(_lib.windq_fit_eval_batch(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), len(Ws), int(G), _ptr(clip_grid),
                                         clip_grid.numel(), _stream(stream)))
    return results


def windq_fit_refine(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor,
                     clip_idx: torch.Tensor, n_steps: int = 10, lr: float = 0.01, *, want_group_err: bool = False,
                     stream=None, thresh: torch.Tensor | None = None) -> dict:
    """Refines the step sizes of the four uniform fits by ``n_steps`` Adam steps, warm-started from ``clip_idx``
    ([4, U, R] u8 of windq_fit_eval).  With ``thresh`` (fp32 [U]) the salient weights are left out of the groups
    (windq_fit_refine_protected; clip_idx then comes from the protected fit).  Returns dict(err [U,4] f32, scale [4,U,R] f16, group_err [4,U,R] f32 | None)."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(clip_grid, torch.float32, "clip_grid", 1)
    _need(clip_idx, torch.uint8, "clip_idx", 3)
    U = C // G if G > 0 else 0
    if tuple(clip_idx.shape) != (4, U, R) or not clip_idx.is_contiguous():
        raise ValueError("clip_idx must be a contiguous [4, U, R] tensor")
    dev = W.device
    out = dict(err=torch.empty((U, 4), dtype=torch.float32, device=dev),
               scale=torch.empty((4, U, R), dtype=torch.float16, device=dev),
               group_err=torch.empty((4, U, R), dtype=torch.float32, device=dev) if want_group_err else None)
    if thresh is not None:
        _need(thresh, torch.float32, "thresh", 1)
        if thresh.numel() != U:
            raise ValueError("thresh must have one entry per unit")
        ctx._check(_lib.windq_fit_refine_protected(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid),
                                                   clip_grid.numel(), _ptr(clip_idx), _ptr(thresh), int(n_steps), float(lr),
                                                   _ptr(out["err"]), _ptr(out["scale"]), _ptr(out["group_err"]),
                                                   _stream(stream)))
        return out
    ctx._check(_lib.windq_fit_refine(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                     _ptr(clip_idx), int(n_steps), float(lr), _ptr(out["err"]), _ptr(out["scale"]),
                                     _ptr(out["group_err"]), _stream(stream)))
    return out


def windq_effective_bits(ctx: Context, actions: torch.Tensor, R: int, G: int, scale_bits: int = 16, zero_bits: int = 16,
                         out: dict | None = None, stream=None) -> dict:
    """Returns dict(unit_centibits [U] i64, code_offsets [U+1] i64, total_centibits [1] i64,
    total_packed_bytes [1] i64), all on the device."""
    _need(actions, torch.uint8, "actions", 1)
    U = actions.numel()
    dev = actions.device
    out = dict(out) if out else {}
    if out.get("unit_centibits") is None:
        out["unit_centibits"] = torch.empty(U, dtype=torch.int64, device=dev)
    if out.get("code_offsets") is None:
        out["code_offsets"] = torch.empty(U + 1, dtype=torch.int64, device=dev)
    if out.get("total_centibits") is None:
        out["total_centibits"] = torch.empty(1, dtype=torch.int64, device=dev)
    if out.get("total_packed_bytes") is None:
        out["total_packed_bytes"] = torch.empty(1, dtype=torch.int64, device=dev)
    ctx._check(_lib.windq_effective_bits(ctx._h, _ptr(actions), U, int(R), int(G), int(scale_bits), int(zero_bits),
                                         _ptr(out["unit_centibits"]), _ptr(out["code_offsets"]),
                                         _ptr(out["total_centibits"]), _ptr(out["total_packed_bytes"]), _stream(stream)))
    return out


def windq_apply_plan(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor,
                     actions: torch.Tensor, code_offsets: torch.Tensor, codes_out: torch.Tensor,
                     clip_idx: torch.Tensor | None = None, *, want_wq: bool = True, out: dict | None = None,
                     stream=None, scale_in: torch.Tensor | None = None) -> dict:
    """Applies a plan.  ``code_offsets`` comes from windq_effective_bits for the same actions;
    ``codes_out`` is a uint8 tensor of at least code_offsets[U] bytes (the caller sizes it, e.g.
    from the worst case 2*R*C + 16*U, to avoid a device-to-host read).  With ``scale_in`` (fp16 [4, U, R] from
    windq_fit_refine; needs ``clip_idx``) the call is windq_apply_plan_refined.

    Returns dict(codes, scales [U,R] f16, zeros [U,R] f16, wq [R,C] f16 | None).
    """
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(clip_grid, torch.float32, "clip_grid", 1)
    _need(actions, torch.uint8, "actions", 1)
    _need(code_offsets, torch.int64, "code_offsets", 1)
    _need(codes_out, torch.uint8, "codes_out", 1)
    if clip_idx is not None:
        _need(clip_idx, torch.uint8, "clip_idx", 3)
        if not clip_idx.is_contiguous():
            raise ValueError("clip_idx must be contiguous")
    U = C // G if G > 0 else 0
    if actions.numel() != U or code_offsets.numel() != U + 1:
        raise ValueError("actions must have U and code_offsets U + 1 entries")
    out = dict(out) if out else {}
    dev = W.device
    if out.get("scales") is None:
        out["scales"] = torch.empty((U, R), dtype=torch.float16, device=dev)
    if out.get("zeros") is None:
        out["zeros"] = torch.empty((U, R), dtype=torch.float16, device=dev)
    if want_wq and out.get("wq") is None:
        out["wq"] = torch.empty_strided((R, C), (ldw, 1), dtype=torch.float16, device=dev)
    out.setdefault("wq", None)
    if out["wq"] is not None and (_matrix(out["wq"], "wq")[2] != ldw or out["wq"].shape != W.shape):
        raise ValueError("wq must have the shape and row stride of W")
    out["codes"] = codes_out
    if scale_in is not None:
        _need(scale_in, torch.float16, "scale_in", 3)
        if clip_idx is None or tuple(scale_in.shape) != (4, U, R) or not scale_in.is_contiguous():
            raise ValueError("scale_in must be a contiguous [4, U, R] tensor and needs clip_idx")
        ctx._check(_lib.windq_apply_plan_refined(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid),
                                                 clip_grid.numel(), _ptr(actions), _ptr(clip_idx), _ptr(scale_in),
                                                 _ptr(code_offsets), _ptr(codes_out), _ptr(out["scales"]),
                                                 _ptr(out["zeros"]), _ptr(out["wq"]), _stream(stream)))
        return out
    ctx._check(_lib.windq_apply_plan(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                     _ptr(actions), _ptr(clip_idx), _ptr(code_offsets), _ptr(codes_out), _ptr(out["scales"]),
                                     _ptr(out["zeros"]), _ptr(out["wq"]), _stream(stream)))
    return out


def windq_scratch_bytes_fit_eval_protected(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_fit_eval_protected(R, C, G))


def windq_scratch_bytes_apply_plan_protected(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_apply_plan_protected(R, C, G))


def windq_scratch_bytes_fit_refine(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_fit_refine(R, C, G))


def windq_scratch_bytes_greedy_allocate(U: int) -> int:
    return int(_lib.windq_scratch_bytes_greedy_allocate(U))


def windq_scratch_bytes_salient_select(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_salient_select(R, C, G))


def windq_salient_select(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, rate_ppm: int, *,
                         want_mask: bool = True, out: dict | None = None, stream=None) -> dict:
    """Top-r salient weights per unit (key |w| * sqrt(s_j), rate in parts per million).

    Returns dict(thresh [U] f32, count [U] i64, mask [R, C/8] u8 | None)."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    U = C // G if G > 0 else 0
    out = dict(out) if out else {}
    dev = W.device
    if out.get("thresh") is None:
        out["thresh"] = torch.empty(U, dtype=torch.float32, device=dev)
    if out.get("count") is None:
        out["count"] = torch.empty(U, dtype=torch.int64, device=dev)
    if want_mask and out.get("mask") is None:
        out["mask"] = torch.empty((R, C // 8), dtype=torch.uint8, device=dev)
    out.setdefault("mask", None)
    ctx._check(_lib.windq_salient_select(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), int(rate_ppm), _ptr(out["thresh"]),
                                         _ptr(out["count"]), _ptr(out["mask"]), _stream(stream)))
    return out


def windq_effective_bits_protected(ctx: Context, actions: torch.Tensor, n_protected: torch.Tensor, R: int, G: int,
                                   scale_bits: int = 16, zero_bits: int = 16, stream=None) -> dict:
    """Eq. 6 with INT8-protected weights.  Returns dict(unit_centibits [U] i64, total_centibits [1] i64)."""
    _need(actions, torch.uint8, "actions", 1)
    _need(n_protected, torch.int64, "n_protected", 1)
    U = actions.numel()
    if n_protected.numel() != U:
        raise ValueError("n_protected must have one entry per unit")
    unit = torch.empty(U, dtype=torch.int64, device=actions.device)
    total = torch.empty(1, dtype=torch.int64, device=actions.device)
    ctx._check(_lib.windq_effective_bits_protected(ctx._h, _ptr(actions), _ptr(n_protected), U, int(R), int(G),
                                                   int(scale_bits), int(zero_bits), _ptr(unit), _ptr(total), _stream(stream)))
    return dict(unit_centibits=unit, total_centibits=total)


def windq_unit_saliency(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, sal_out: torch.Tensor | None = None,
                        stream=None) -> torch.Tensor:
    """Mean of sqrt(s_j) * |w| over every unit: fp32 [U]."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    if sal_out is None:
        sal_out = torch.empty(max(C // max(G, 1), 0), dtype=torch.float32, device=W.device)
    _need(sal_out, torch.float32, "sal_out", 1)
    ctx._check(_lib.windq_unit_saliency(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(sal_out), _stream(stream)))
    return sal_out


def windq_fallback(ctx: Context, err: torch.Tensor, energy: torch.Tensor, actions: torch.Tensor, theta: float,
                   stream=None) -> dict:
    """Moves units whose relative error exceeds theta to higher precision.
    Returns dict(actions [U] u8, n_changed [1] i64)."""
    _need(err, torch.float32, "err", 2)
    _need(energy, torch.float32, "energy", 1)
    _need(actions, torch.uint8, "actions", 1)
    U = actions.numel()
    if err.shape != (U, N_BITWIDTHS) or energy.numel() != U or not err.is_contiguous():
        raise ValueError("err must be a contiguous [U, 6] table and energy [U]")
    out = torch.empty_like(actions)
    n = torch.empty(1, dtype=torch.int64, device=actions.device)
    ctx._check(_lib.windq_fallback(ctx._h, _ptr(err), _ptr(energy), _ptr(actions), U, float(theta), _ptr(out), _ptr(n),
                                   _stream(stream)))
    return dict(actions=out, n_changed=n)


def windq_greedy_allocate(ctx: Context, saliency: torch.Tensor, n_weights: torch.Tensor, n_groups: torch.Tensor,
                          target_cb: int, headroom_cb: int, n_protected: torch.Tensor | None = None, *,
                          scale_bits: int = 0, zero_bits: int = 0, stream=None) -> dict:
    """The heuristic allocator's rule over U units: rank by saliency, free budget from the bottom, promote from the top.
    Returns dict(actions [U] u8, order [U] i64 (most sensitive first), total_centibits [1] i64)."""
    _need(saliency, torch.float32, "saliency", 1)
    _need(n_weights, torch.int64, "n_weights", 1)
    _need(n_groups, torch.int64, "n_groups", 1)
    U = saliency.numel()
    if n_weights.numel() != U or n_groups.numel() != U:
        raise ValueError("n_weights and n_groups must have one entry per unit")
    if not (saliency.is_contiguous() and n_weights.is_contiguous() and n_groups.is_contiguous()):
        raise ValueError("saliency, n_weights and n_groups must be contiguous")
    if n_protected is not None:
        _need(n_protected, torch.int64, "n_protected", 1)
        if n_protected.numel() != U or not n_protected.is_contiguous():
            raise ValueError("n_protected must be contiguous with one entry per unit")
    actions = torch.empty(U, dtype=torch.uint8, device=saliency.device)
    order = torch.empty(U, dtype=torch.int64, device=saliency.device)
    total = torch.empty(1, dtype=torch.int64, device=saliency.device)
    ctx._check(_lib.windq_greedy_allocate(ctx._h, _ptr(saliency), _ptr(n_weights), _ptr(n_protected), _ptr(n_groups), U,
                                          int(target_cb), int(headroom_cb), int(scale_bits), int(zero_bits), _ptr(actions),
                                          _ptr(order), _ptr(total), _stream(stream)))
    return dict(actions=actions, order=order, total_centibits=total)


def windq_apply_plan_protected(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor,
                               actions: torch.Tensor, code_offsets: torch.Tensor, codes_out: torch.Tensor,
                               thresh: torch.Tensor, prot_q_out: torch.Tensor, clip_idx: torch.Tensor | None = None, *,
                               want_wq: bool = True, stream=None, scale_in: torch.Tensor | None = None) -> dict:
    """windq_apply_plan with the salient weights (key >= thresh[u]) kept on an INT8 grid per unit.
    ``prot_q_out`` is an int8 tensor sized by the caller (sum of the counts of windq_salient_select is enough).

    Returns dict(codes, scales, zeros, wq | None, prot_scale [U] f16, prot_offsets [U+1] i64, prot_q)."""
    R, C, ldw = _matrix(W, "W")
    for t_, dt, nm in ((s, torch.float32, "s"), (clip_grid, torch.float32, "clip_grid"), (actions, torch.uint8, "actions"),
                       (code_offsets, torch.int64, "code_offsets"), (codes_out, torch.uint8, "codes_out"),
                       (thresh, torch.float32, "thresh"), (prot_q_out, torch.int8, "prot_q_out")):
        _need(t_, dt, nm, 1)
    if clip_idx is not None:
        _need(clip_idx, torch.uint8, "clip_idx", 3)
    U = C // G if G > 0 else 0
    if actions.numel() != U or code_offsets.numel() != U + 1 or thresh.numel() != U:
        raise ValueError("actions and thresh must have U entries and code_offsets U + 1")
    dev = W.device
    out = dict(codes=codes_out, scales=torch.empty((U, R), dtype=torch.float16, device=dev),
               zeros=torch.empty((U, R), dtype=torch.float16, device=dev),
               wq=torch.empty_strided((R, C), (ldw, 1), dtype=torch.float16, device=dev) if want_wq else None,
               prot_scale=torch.empty(U, dtype=torch.float16, device=dev),
               prot_offsets=torch.empty(U + 1, dtype=torch.int64, device=dev), prot_q=prot_q_out)
    if scale_in is not None:
        _need(scale_in, torch.float16, "scale_in", 3)
        if clip_idx is None or tuple(scale_in.shape) != (4, U, R) or not scale_in.is_contiguous():
            raise ValueError("scale_in must be a contiguous [4, U, R] tensor and needs clip_idx")
        ctx._check(_lib.windq_apply_plan_protected_refined(
            ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(), _ptr(actions), _ptr(clip_idx),
            _ptr(scale_in), _ptr(code_offsets), _ptr(thresh), _ptr(codes_out), _ptr(out["scales"]), _ptr(out["zeros"]),
            _ptr(out["wq"]), _ptr(out["prot_scale"]), _ptr(out["prot_offsets"]), _ptr(prot_q_out), prot_q_out.numel(),
            _stream(stream)))
        return out
    ctx._check(_lib.windq_apply_plan_protected(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                               _ptr(actions), _ptr(clip_idx), _ptr(code_offsets), _ptr(thresh), _ptr(codes_out),
                                               _ptr(out["scales"]), _ptr(out["zeros"]), _ptr(out["wq"]), _ptr(out["prot_scale"]),
                                               _ptr(out["prot_offsets"]), _ptr(prot_q_out), prot_q_out.numel(), _stream(stream)))
    return out


class _PlanOut(ctypes.Structure):
    _fields_ = [("actions", ctypes.c_void_p), ("code_offsets", ctypes.c_void_p), ("codes_out", ctypes.c_void_p),
                ("scales_out", ctypes.c_void_p), ("zeros_out", ctypes.c_void_p), ("Wq_out", ctypes.c_void_p)]


def windq_apply_plan_multi(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor,
                           clip_idx: torch.Tensor, plans, *, lowbit: torch.Tensor | None = None, stream=None) -> list:
    """Up to four plans of one matrix in one pass over its weights.  ``plans``: a sequence of dicts with the keys
    actions, code_offsets, codes (uint8 output, sized by the caller) and optionally scales, zeros ([U, R] fp16) and
    wq ([R, C] fp16 with the row stride of W, or None for no fake-quantised output; absent = allocated).
    ``lowbit`` (fp16 [3, U, R] from windq_fit_eval_batch(want_lowbit=True)) spares the low-bit units their sums.
    Returns one dict(codes, scales, zeros, wq) per plan."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(clip_grid, torch.float32, "clip_grid", 1)
    _need(clip_idx, torch.uint8, "clip_idx", 3)
    U = C // G if G > 0 else 0
    if tuple(clip_idx.shape) != (4, U, R) or not clip_idx.is_contiguous():
        raise ValueError("clip_idx must be a contiguous [4, U, R] tensor")
    if lowbit is not None:
        _need(lowbit, torch.float16, "lowbit", 3)
        if tuple(lowbit.shape) != (3, U, R) or not lowbit.is_contiguous():
            raise ValueError("lowbit must be a contiguous [3, U, R] tensor")
    if not plans:
        raise ValueError("plans must not be empty")
    arr = (_PlanOut * len(plans))()
    results = []
    dev = W.device
    for j, pl in enumerate(plans):
        actions, offs, codes = pl["actions"], pl["code_offsets"], pl["codes"]
        _need(actions, torch.uint8, "actions", 1)
        _need(offs, torch.int64, "code_offsets", 1)
        _need(codes, torch.uint8, "codes", 1)
        if actions.numel() != U or offs.numel() != U + 1:
            raise ValueError("plan %d: actions must have U and code_offsets U + 1 entries" % j)
        scales = pl.get("scales")
        zeros = pl.get("zeros")
        if scales is None:
            scales = torch.empty((U, R), dtype=torch.float16, device=dev)
        if zeros is None:
            zeros = torch.empty((U, R), dtype=torch.float16, device=dev)
        wq_out = pl["wq"] if "wq" in pl else torch.empty_strided((R, C), (ldw, 1), dtype=torch.float16, device=dev)
        if wq_out is not None and (_matrix(wq_out, "wq")[2] != ldw or wq_out.shape != W.shape):
            raise ValueError("plan %d: wq must have the shape and row stride of W" % j)
        arr[j] = _PlanOut(actions.data_ptr(), offs.data_ptr(), codes.data_ptr(), scales.data_ptr(), zeros.data_ptr(),
                          None if wq_out is None else wq_out.data_ptr())
        results.append(dict(codes=codes, scales=scales, zeros=zeros, wq=wq_out))
    ctx._check(_lib.windq_apply_plan_multi(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                           _ptr(clip_idx), _ptr(lowbit), ctypes.cast(arr, ctypes.c_void_p), len(plans),
                                           _stream(stream)))
    return results


def windq_scratch_bytes_fit_ternary_search(R: int, C: int, G: int) -> int:
    return int(_lib.windq_scratch_bytes_fit_ternary_search(R, C, G))


def windq_fit_ternary_search(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, thr_grid: torch.Tensor, *,
                             thresh: torch.Tensor | None = None, want_group_err: bool = False, out: dict | None = None,
                             stream=None) -> dict:
    """Search over the ternary threshold ratio.  Returns dict(err [U] f32, thr_idx [U, R] u8, alpha [U, R] f16,
    group_err [U, R] f32 | None)."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(thr_grid, torch.float32, "thr_grid", 1)
    U = C // G if G > 0 else 0
    if thresh is not None:
        _need(thresh, torch.float32, "thresh", 1)
        if thresh.numel() != U:
            raise ValueError("thresh must have U entries")
    out = dict(out) if out else {}
    dev = W.device
    if out.get("err") is None:
        out["err"] = torch.empty(U, dtype=torch.float32, device=dev)
    if out.get("thr_idx") is None:
        out["thr_idx"] = torch.empty((U, R), dtype=torch.uint8, device=dev)
    if out.get("alpha") is None:
        out["alpha"] = torch.empty((U, R), dtype=torch.float16, device=dev)
    if want_group_err and out.get("group_err") is None:
        out["group_err"] = torch.empty((U, R), dtype=torch.float32, device=dev)
    out.setdefault("group_err", None)
    ctx._check(_lib.windq_fit_ternary_search(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(thr_grid), thr_grid.numel(),
                                             _ptr(thresh), _ptr(out["err"]), _ptr(out["thr_idx"]), _ptr(out["alpha"]),
                                             _ptr(out["group_err"]), _stream(stream)))
    return out


def windq_apply_plan_searched(ctx: Context, W: torch.Tensor, G: int, s: torch.Tensor, clip_grid: torch.Tensor,
                              actions: torch.Tensor, code_offsets: torch.Tensor, codes_out: torch.Tensor,
                              clip_idx: torch.Tensor, thr_grid: torch.Tensor, thr_idx: torch.Tensor, *,
                              want_wq: bool = True, out: dict | None = None, stream=None) -> dict:
    """windq_apply_plan with the ternary thresholds chosen by windq_fit_ternary_search (thr_idx u8 [U, R])."""
    R, C, ldw = _matrix(W, "W")
    _need(s, torch.float32, "s", 1)
    _need(clip_grid, torch.float32, "clip_grid", 1)
    _need(thr_grid, torch.float32, "thr_grid", 1)
    _need(actions, torch.uint8, "actions", 1)
    _need(code_offsets, torch.int64, "code_offsets", 1)
    _need(codes_out, torch.uint8, "codes_out", 1)
    _need(clip_idx, torch.uint8, "clip_idx", 3)
    _need(thr_idx, torch.uint8, "thr_idx", 2)
    U = C // G if G > 0 else 0
    if actions.numel() != U or code_offsets.numel() != U + 1:
        raise ValueError("actions must have U and code_offsets U + 1 entries")
    if tuple(clip_idx.shape) != (4, U, R) or tuple(thr_idx.shape) != (U, R) or not clip_idx.is_contiguous() \
            or not thr_idx.is_contiguous():
        raise ValueError("clip_idx must be a contiguous [4, U, R] and thr_idx a contiguous [U, R] tensor")
    out = dict(out) if out else {}
    dev = W.device
    if out.get("scales") is None:
        out["scales"] = torch.empty((U, R), dtype=torch.float16, device=dev)
    if out.get("zeros") is None:
        out["zeros"] = torch.empty((U, R), dtype=torch.float16, device=dev)
    if want_wq and out.get("wq") is None:
        out["wq"] = torch.empty_strided((R, C), (ldw, 1), dtype=torch.float16, device=dev)
    out.setdefault("wq", None)
    out["codes"] = codes_out
    ctx._check(_lib.windq_apply_plan_searched(ctx._h, _ptr(W), R, C, ldw, int(G), _ptr(s), _ptr(clip_grid), clip_grid.numel(),
                                              _ptr(actions), _ptr(clip_idx), _ptr(thr_grid), thr_grid.numel(), _ptr(thr_idx),
                                              _ptr(code_offsets), _ptr(codes_out), _ptr(out["scales"]), _ptr(out["zeros"]),
                                              _ptr(out["wq"]), _stream(stream)))
    return out


class _FeatFitJob(ctypes.Structure):
    _fields_ = [("W", ctypes.c_void_p), ("R", ctypes.c_int64), ("C", ctypes.c_int64), ("ldw", ctypes.c_int64),
                ("s", ctypes.c_void_p), ("feat_out", ctypes.c_void_p), ("err_out", ctypes.c_void_p),
                ("energy_out", ctypes.c_void_p), ("clip_idx_out", ctypes.c_void_p), ("group_err_out", ctypes.c_void_p),
                ("lowbit_out", ctypes.c_void_p)]


def _featfit_jobs(Ws, G, ss, feats, outs, want_energy, want_clip_idx, want_group_err):
    jobs = (_FeatFitJob * len(Ws))()
    results, feat_list = [], []
    for j, (W, s) in enumerate(zip(Ws, ss)):
        R, C, ldw = _matrix(W, "W")
        _need(s, torch.float32, "s", 1)
        U = C // G if G > 0 else 0
        out = dict(outs[j]) if outs else {}
        dev = W.device
        f = feats[j] if feats is not None else torch.empty((U, N_FEATURES), dtype=torch.float32, device=dev)
        _need(f, torch.float32, "feat_out", 2)
        if tuple(f.shape) != (U, N_FEATURES) or not f.is_contiguous():
            raise ValueError("feat_out must be a contiguous [U, 8] tensor")
        if out.get("err") is None:
            out["err"] = torch.empty((U, N_BITWIDTHS), dtype=torch.float32, device=dev)
        if want_energy and out.get("energy") is None:
            out["energy"] = torch.empty(U, dtype=torch.float32, device=dev)
        if want_clip_idx and out.get("clip_idx") is None:
            out["clip_idx"] = torch.empty((4, U, R), dtype=torch.uint8, device=dev)
        if want_group_err and out.get("group_err") is None:
            out["group_err"] = torch.empty((N_BITWIDTHS, U, R), dtype=torch.float32, device=dev)
        for key in ("energy", "clip_idx", "group_err"):
            out.setdefault(key, None)
        ptr = lambda x: None if x is None else x.data_ptr()
        jobs[j] = _FeatFitJob(W.data_ptr(), R, C, ldw, s.data_ptr(), f.data_ptr(), ptr(out["err"]), ptr(out["energy"]),
                              ptr(out["clip_idx"]), ptr(out["group_err"]), ptr(out.get("lowbit")))
        results.append(out)
        feat_list.append(f)
    return jobs, feat_list, results


def windq_scratch_bytes_features_fit_batch(Ws, G: int) -> int:
    jobs = (_FeatFitJob * len(Ws))()
    for j, W in enumerate(Ws):
        R, C, ldw = _matrix(W, "W")
        jobs[j] = _FeatFitJob(W.data_ptr(), R, C, ldw, None, None, None, None, None, None, None)
    return int(_lib.windq_scratch_bytes_features_fit_batch(ctypes.cast(jobs, ctypes.c_void_p), len(Ws), int(G)))


def windq_features_fit_batch(ctx: Context, Ws, G: int, ss, clip_grid: torch.Tensor, *, feats=None, want_energy: bool = True,
                             want_clip_idx: bool = True, want_group_err: bool = False, outs=None, stream=None):
    """windq_unit_features_batch and windq_fit_eval_batch of up to 16 matrices in one pass over the weights.
    Returns (list of feature tensors, list of fit output dicts)."""
    if len(Ws) != len(ss) or not Ws:
        raise ValueError("Ws and ss must be non-empty and equally long")
    _need(clip_grid, torch.float32, "clip_grid", 1)
    jobs, feat_list, results = _featfit_jobs(Ws, G, ss, feats, outs, want_energy, want_clip_idx, want_group_err)
    ctx._check(_lib.windq_features_fit_batch(ctx._h, ctypes.cast(jobs, ctypes.c_void_p), len(Ws), int(G), _ptr(clip_grid),
                                             clip_grid.numel(), _stream(stream)))
    return feat_list, results
