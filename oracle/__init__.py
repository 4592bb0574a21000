"""ctypes front end of the CPU oracle (test infrastructure, not the product).

The oracle is the C++ file next to this module, built as ``libwindq_oracle.so``
with ``g++ -O2 -ffp-contract=off``.  Nothing here touches CUDA or imports the
GPU package; inputs and outputs are numpy arrays (fp16 data as ``uint16`` bit
patterns or ``float16`` arrays).  Only tests, the smoke check and the
benchmark's CPU-baseline leg may import this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "windq_oracle.cpp")
_LIB = os.path.join(_HERE, "libwindq_oracle.so")

CXX_FLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-Wall"]

N_BITWIDTHS = 6          # table columns: 8, 4, 3, 2, 1.58, 1
N_FEATURES = 8


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(["g++", *CXX_FLAGS, "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_half_to_float.restype = ctypes.c_float
        _lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        _lib.oracle_float_to_half.restype = ctypes.c_uint16
        _lib.oracle_float_to_half.argtypes = [ctypes.c_float]
        _lib.oracle_psum8.restype = ctypes.c_float
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _as_u16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    assert a.dtype == np.uint16, a.dtype
    return a


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def half_to_float(h: int) -> float:
    return float(lib().oracle_half_to_float(int(h)))


def float_to_half(f: float) -> int:
    return int(lib().oracle_float_to_half(ctypes.c_float(f)))


def psum8(x) -> float:
    x = _f32(x)
    return float(lib().oracle_psum8(_p(x), ctypes.c_int(x.size)))


def uniform_candidate(w, s, bits: int, p: float, want_codes: bool = True):
    """One clip candidate on one row-group: (scale, zero, error, codes)."""
    w, s = _f32(w), _f32(s)
    G = w.size
    scale, zero, err = ctypes.c_float(), ctypes.c_float(), ctypes.c_float()
    codes = np.zeros(G, np.uint8) if want_codes else None
    rc = lib().oracle_uniform_candidate(_p(w), _p(s), ctypes.c_int(G), ctypes.c_int(bits), ctypes.c_float(p),
                                        ctypes.byref(scale), ctypes.byref(zero), ctypes.byref(err), _p(codes))
    if rc:
        raise ValueError("oracle_uniform_candidate: bad arguments")
    return scale.value, zero.value, err.value, codes


def act_stats(X) -> np.ndarray:
    X = _as_u16(X)
    T, C = X.shape
    s = np.zeros(C, np.float32)
    rc = lib().oracle_act_stats(_p(X), ctypes.c_int64(T), ctypes.c_int64(C), ctypes.c_int64(C), _p(s))
    if rc:
        raise ValueError("oracle_act_stats: bad arguments")
    return s


def unit_features(W, G: int, s) -> np.ndarray:
    W, s = _as_u16(W), _f32(s)
    R, C = W.shape
    feat = np.zeros((C // G, N_FEATURES), np.float32)
    rc = lib().oracle_unit_features(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C),
                                    ctypes.c_int(G), _p(s), _p(feat))
    if rc:
        raise ValueError("oracle_unit_features: bad arguments")
    return feat


def fit_eval(W, G: int, s, clip_grid, units=None, threads: int = 1, want_group_err: bool = True, thresh=None):
    """Returns dict(err[U,6], energy[U], clip_idx[4,U,R], group_err[6,U,R]).

    ``thresh`` (fp32 [U], from salient_select) takes the protected weights out of the fits.

    ``units`` = (begin, end) restricts the work to a unit range (other rows of
    the outputs stay zero).  ``threads`` > 1 runs the same single-threaded
    routine over disjoint unit ranges concurrently (units are independent).
    """
    W, s, clip_grid = _as_u16(W), _f32(s), _f32(clip_grid)
    R, C = W.shape
    U = C // G
    K = clip_grid.size
    u0, u1 = (0, U) if units is None else units
    err = np.zeros((U, N_BITWIDTHS), np.float32)
    energy = np.zeros(U, np.float32)
    clip_idx = np.zeros((4, U, R), np.uint8)
    group_err = np.zeros((N_BITWIDTHS, U, R), np.float32) if want_group_err else None

    if thresh is not None:
        thresh = _f32(thresh)
        assert thresh.size == U

    def run(a, b):
        if thresh is None:
            rc = lib().oracle_fit_eval(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                       _p(s), _p(clip_grid), ctypes.c_int(K), ctypes.c_int64(a), ctypes.c_int64(b),
                                       _p(err), _p(energy), _p(clip_idx), _p(group_err))
        else:
            rc = lib().oracle_fit_eval_protected(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C),
                                                 ctypes.c_int(G), _p(s), _p(clip_grid), ctypes.c_int(K), ctypes.c_int64(a),
                                                 ctypes.c_int64(b), _p(thresh), _p(err), _p(energy), _p(clip_idx),
                                                 _p(group_err))
        if rc:
            raise ValueError("oracle_fit_eval: bad arguments")

    if threads <= 1 or u1 - u0 <= 1:
        run(u0, u1)
    else:
        bounds = np.linspace(u0, u1, min(threads, u1 - u0) + 1).astype(np.int64)
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda ab: run(int(ab[0]), int(ab[1])), zip(bounds[:-1], bounds[1:])))
    return dict(err=err, energy=energy, clip_idx=clip_idx, group_err=group_err)


def effective_bits(actions, R: int, G: int, scale_bits: int = 16, zero_bits: int = 16):
    """Returns dict(unit_centibits[U], code_offsets[U+1], total_centibits, total_packed_bytes)."""
    actions = np.ascontiguousarray(actions, dtype=np.uint8)
    U = actions.size
    unit_cb = np.zeros(U, np.int64)
    offs = np.zeros(U + 1, np.int64)
    total = ctypes.c_int64()
    packed = ctypes.c_int64()
    rc = lib().oracle_effective_bits(_p(actions), ctypes.c_int64(U), ctypes.c_int64(R), ctypes.c_int(G),
                                     ctypes.c_int(scale_bits), ctypes.c_int(zero_bits), _p(unit_cb), _p(offs),
                                     ctypes.byref(total), ctypes.byref(packed))
    if rc:
        raise ValueError("oracle_effective_bits: bad arguments")
    return dict(unit_centibits=unit_cb, code_offsets=offs, total_centibits=total.value,
                total_packed_bytes=packed.value)


def apply_plan(W, G: int, s, clip_grid, actions, clip_idx=None, want_wq: bool = True, thresh=None, scale_in=None):
    """Returns dict(codes[bytes], scales[U,R] u16, zeros[U,R] u16, wq[R,C] u16, code_offsets).

    With ``thresh`` (fp32 [U], from salient_select) the salient weights are protected; the result then
    also holds prot_scale[U] u16, prot_offsets[U+1] i64 and prot_q (int8 codes, row-major per unit).
    With ``scale_in`` (fp16 [4][U][R], from fit_refine; needs clip_idx) the uniform groups use those scales."""
    W, s, clip_grid = _as_u16(W), _f32(s), _f32(clip_grid)
    actions = np.ascontiguousarray(actions, dtype=np.uint8)
    R, C = W.shape
    U = C // G
    offs = effective_bits(actions, R, G)["code_offsets"]
    codes = np.zeros(int(offs[U]), np.uint8)
    scales = np.zeros((U, R), np.uint16)
    zeros = np.zeros((U, R), np.uint16)
    wq = np.zeros((R, C), np.uint16) if want_wq else None
    if clip_idx is not None:
        clip_idx = np.ascontiguousarray(clip_idx, dtype=np.uint8)
        assert clip_idx.shape == (4, U, R)
    if thresh is not None:
        thresh = _f32(thresh)
        assert thresh.size == U
        prot_scale = np.zeros(U, np.uint16)
        prot_offsets = np.zeros(U + 1, np.int64)
        prot_q = np.zeros(R * C, np.int8)
        if scale_in is not None:
            assert clip_idx is not None
            scale_in = _as_u16(scale_in)
            assert scale_in.shape == (4, U, R)
            rc = lib().oracle_apply_plan_protected_refined(
                _p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G), _p(s), _p(clip_grid),
                ctypes.c_int(clip_grid.size), _p(actions), _p(clip_idx), _p(scale_in), _p(offs), _p(thresh), _p(codes),
                _p(scales), _p(zeros), _p(wq), _p(prot_scale), _p(prot_offsets), _p(prot_q))
        else:
            rc = lib().oracle_apply_plan_protected(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                                   _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size), _p(actions), _p(clip_idx),
                                                   _p(offs), _p(thresh), _p(codes), _p(scales), _p(zeros), _p(wq),
                                                   _p(prot_scale), _p(prot_offsets), _p(prot_q))
        if rc:
            raise ValueError("oracle_apply_plan_protected: bad arguments")
        return dict(codes=codes, scales=scales, zeros=zeros, wq=wq, code_offsets=offs, prot_scale=prot_scale,
                    prot_offsets=prot_offsets, prot_q=prot_q[:int(prot_offsets[U])].copy())
    if scale_in is not None:
        assert clip_idx is not None
        scale_in = _as_u16(scale_in)
        assert scale_in.shape == (4, U, R)
        rc = lib().oracle_apply_plan_refined(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                             _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size), _p(actions), _p(clip_idx),
                                             _p(scale_in), _p(offs), _p(codes), _p(scales), _p(zeros), _p(wq))
        if rc:
            raise ValueError("oracle_apply_plan_refined: bad arguments")
        return dict(codes=codes, scales=scales, zeros=zeros, wq=wq, code_offsets=offs)
    rc = lib().oracle_apply_plan(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                 _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size), _p(actions), _p(clip_idx),
                                 _p(offs), _p(codes), _p(scales), _p(zeros), _p(wq))
    if rc:
        raise ValueError("oracle_apply_plan: bad arguments")
    return dict(codes=codes, scales=scales, zeros=zeros, wq=wq, code_offsets=offs)


def salient_select(W, G: int, s, rate_ppm: int, want_mask: bool = True):
    """Top-r selection of salient weights per unit.  Returns dict(thresh[U] f32, count[U] i64,
    mask[R, C/8] u8 | None) -- bit (col % 8) of mask[r, col // 8] is set for a protected weight."""
    W, s = _as_u16(W), _f32(s)
    R, C = W.shape
    U = C // G
    thresh = np.zeros(U, np.float32)
    count = np.zeros(U, np.int64)
    mask = np.zeros((R, C // 8), np.uint8) if want_mask else None
    rc = lib().oracle_salient_select(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                     _p(s), ctypes.c_int64(rate_ppm), _p(thresh), _p(count), _p(mask))
    if rc:
        raise ValueError("oracle_salient_select: bad arguments")
    return dict(thresh=thresh, count=count, mask=mask)


def effective_bits_protected(actions, n_protected, R: int, G: int, scale_bits: int = 16, zero_bits: int = 16):
    """Eq. 6 with INT8-protected weights.  Returns dict(unit_centibits[U], total_centibits)."""
    actions = np.ascontiguousarray(actions, dtype=np.uint8)
    n_protected = np.ascontiguousarray(n_protected, dtype=np.int64)
    U = actions.size
    unit_cb = np.zeros(U, np.int64)
    total = ctypes.c_int64()
    rc = lib().oracle_effective_bits_protected(_p(actions), _p(n_protected), ctypes.c_int64(U), ctypes.c_int64(R),
                                               ctypes.c_int(G), ctypes.c_int(scale_bits), ctypes.c_int(zero_bits),
                                               _p(unit_cb), ctypes.byref(total))
    if rc:
        raise ValueError("oracle_effective_bits_protected: bad arguments")
    return dict(unit_centibits=unit_cb, total_centibits=total.value)


def unit_saliency(W, G: int, s):
    """Mean of sqrt(s_j) * |w| over every unit.  Returns fp32 [U]."""
    W, s = _as_u16(W), _f32(s)
    R, C = W.shape
    out = np.zeros(C // G, np.float32)
    rc = lib().oracle_unit_saliency(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G), _p(s), _p(out))
    if rc:
        raise ValueError("oracle_unit_saliency: bad arguments")
    return out


def fallback(err, energy, actions, theta: float):
    """Moves every unit whose relative error exceeds theta to higher precision.  Returns (actions, n_changed)."""
    err, energy = _f32(err), _f32(energy)
    actions = np.ascontiguousarray(actions, dtype=np.uint8)
    U = actions.size
    assert err.shape == (U, N_BITWIDTHS) and energy.size == U
    out = np.zeros(U, np.uint8)
    n = ctypes.c_int64()
    rc = lib().oracle_fallback(_p(err), _p(energy), _p(actions), ctypes.c_int64(U), ctypes.c_float(theta), _p(out), ctypes.byref(n))
    if rc:
        raise ValueError("oracle_fallback: bad arguments")
    return out, n.value


def greedy_allocate(saliency, n_weights, n_groups, target_cb: int, headroom_cb: int, n_protected=None,
                    scale_bits: int = 0, zero_bits: int = 0):
    """The heuristic allocator's deterministic rule.  Returns (actions u8 [U], order i64 [U], total centibits)."""
    sal = _f32(saliency)
    U = sal.size
    n = np.ascontiguousarray(n_weights, dtype=np.int64)
    g = np.ascontiguousarray(n_groups, dtype=np.int64)
    p = None if n_protected is None else np.ascontiguousarray(n_protected, dtype=np.int64)
    assert n.size == U and g.size == U and (p is None or p.size == U)
    actions = np.zeros(U, np.uint8)
    order = np.zeros(U, np.int64)
    total = ctypes.c_int64()
    rc = lib().oracle_greedy_allocate(_p(sal), _p(n), _p(p), _p(g), ctypes.c_int64(U), ctypes.c_int64(target_cb),
                                      ctypes.c_int64(headroom_cb), ctypes.c_int(scale_bits), ctypes.c_int(zero_bits),
                                      _p(actions), _p(order), ctypes.byref(total))
    if rc:
        raise ValueError("oracle_greedy_allocate: bad arguments")
    return actions, order, total.value


def refine_trace(w, s, bits: int, scale0: float, zf: float, T: int, lr: float):
    """The refinement iteration on one group.  Returns (scales, losses, grads) of the iterates evaluated."""
    w, s = _f32(w), _f32(s)
    G = w.size
    assert s.size == G
    sc, lo, gr = (np.zeros(T + 1, np.float32) for _ in range(3))
    fn = lib().oracle_refine_trace
    fn.restype = ctypes.c_int
    n = fn(_p(w), _p(s), ctypes.c_int(G), ctypes.c_int(bits), ctypes.c_float(scale0), ctypes.c_float(zf), ctypes.c_int(T),
           ctypes.c_float(lr), _p(sc), _p(lo), _p(gr))
    if n < 0:
        raise ValueError("oracle_refine_trace: bad arguments")
    return sc[:n], lo[:n], gr[:n]


def fit_refine(W, G: int, s, clip_grid, clip_idx, T: int = 10, lr: float = 0.01, thresh=None):
    """Step-size refinement of the four uniform fits, warm-started from clip_idx [4][U][R] of fit_eval.
    With ``thresh`` (fp32 [U]) the salient weights are left out of the groups as in the protected fit.
    Returns dict(err [U][4] f32, scale [4][U][R] f16, group_err [4][U][R] f32)."""
    W, s, clip_grid = _as_u16(W), _f32(s), _f32(clip_grid)
    R, C = W.shape
    U = C // G
    clip_idx = np.ascontiguousarray(clip_idx, dtype=np.uint8)
    assert clip_idx.shape == (4, U, R)
    err = np.zeros((U, 4), np.float32)
    scale = np.zeros((4, U, R), np.uint16)
    gerr = np.zeros((4, U, R), np.float32)
    if thresh is not None:
        thresh = _f32(thresh)
        assert thresh.size == U
        rc = lib().oracle_fit_refine_protected(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(W.strides[0] // 2),
                                               ctypes.c_int(G), _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size),
                                               _p(clip_idx), _p(thresh), ctypes.c_int(T), ctypes.c_float(lr), _p(err),
                                               _p(scale), _p(gerr))
    else:
        rc = lib().oracle_fit_refine(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(W.strides[0] // 2),
                                     ctypes.c_int(G), _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size), _p(clip_idx),
                                     ctypes.c_int(T), ctypes.c_float(lr), _p(err), _p(scale), _p(gerr))
    if rc:
        raise ValueError("oracle_fit_refine: bad arguments (%d)" % rc)
    return dict(err=err, scale=scale.view(np.float16), group_err=gerr)


def ternary_candidate(w, s, rho: float, want_trits: bool = True):
    """One threshold ratio on one row-group: (alpha, error, trits)."""
    w, s = _f32(w), _f32(s)
    G = w.size
    alpha, err = ctypes.c_float(), ctypes.c_float()
    trits = np.zeros(G, np.uint8) if want_trits else None
    rc = lib().oracle_ternary_candidate(_p(w), _p(s), ctypes.c_int(G), ctypes.c_float(rho), ctypes.byref(alpha),
                                        ctypes.byref(err), _p(trits))
    if rc:
        raise ValueError("oracle_ternary_candidate: bad arguments")
    return alpha.value, err.value, trits


def binary_candidate(w, s, want_bits: bool = True):
    """The 1-bit fit of one row-group: (alpha, error, bits)."""
    w, s = _f32(w), _f32(s)
    G = w.size
    alpha, err = ctypes.c_float(), ctypes.c_float()
    bits = np.zeros(G, np.uint8) if want_bits else None
    rc = lib().oracle_binary_candidate(_p(w), _p(s), ctypes.c_int(G), ctypes.byref(alpha), ctypes.byref(err), _p(bits))
    if rc:
        raise ValueError("oracle_binary_candidate: bad arguments")
    return alpha.value, err.value, bits


def fit_ternary_search(W, G: int, s, thr_grid, units=None, threads: int = 1, thresh=None, want_group_err: bool = True):
    """Search over the ternary threshold ratio.  Returns dict(err [U] f32, thr_idx [U][R] u8, alpha [U][R] f16,
    group_err [U][R] f32 | None).  ``units``, ``threads`` and ``thresh`` as in fit_eval."""
    W, s, thr_grid = _as_u16(W), _f32(s), _f32(thr_grid)
    R, C = W.shape
    U = C // G
    u0, u1 = (0, U) if units is None else units
    err = np.zeros(U, np.float32)
    thr_idx = np.zeros((U, R), np.uint8)
    alpha = np.zeros((U, R), np.uint16)
    gerr = np.zeros((U, R), np.float32) if want_group_err else None
    if thresh is not None:
        thresh = _f32(thresh)
        assert thresh.size == U

    def run(a, b):
        rc = lib().oracle_fit_ternary_search(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                             _p(s), _p(thr_grid), ctypes.c_int(thr_grid.size), ctypes.c_int64(a),
                                             ctypes.c_int64(b), _p(thresh), _p(err), _p(thr_idx), _p(alpha), _p(gerr))
        if rc:
            raise ValueError("oracle_fit_ternary_search: bad arguments")

    if threads <= 1 or u1 - u0 <= 1:
        run(u0, u1)
    else:
        bounds = np.linspace(u0, u1, min(threads, u1 - u0) + 1).astype(np.int64)
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda ab: run(int(ab[0]), int(ab[1])), zip(bounds[:-1], bounds[1:])))
    return dict(err=err, thr_idx=thr_idx, alpha=alpha.view(np.float16), group_err=gerr)


def apply_plan_searched(W, G: int, s, clip_grid, actions, clip_idx, thr_grid, thr_idx, want_wq: bool = True):
    """apply_plan with the ternary thresholds chosen by fit_ternary_search (thr_idx u8 [U][R])."""
    W, s, clip_grid, thr_grid = _as_u16(W), _f32(s), _f32(clip_grid), _f32(thr_grid)
    actions = np.ascontiguousarray(actions, dtype=np.uint8)
    R, C = W.shape
    U = C // G
    offs = effective_bits(actions, R, G)["code_offsets"]
    codes = np.zeros(int(offs[U]), np.uint8)
    scales = np.zeros((U, R), np.uint16)
    zeros = np.zeros((U, R), np.uint16)
    wq = np.zeros((R, C), np.uint16) if want_wq else None
    if clip_idx is not None:
        clip_idx = np.ascontiguousarray(clip_idx, dtype=np.uint8)
        assert clip_idx.shape == (4, U, R)
    thr_idx = np.ascontiguousarray(thr_idx, dtype=np.uint8)
    assert thr_idx.shape == (U, R)
    rc = lib().oracle_apply_plan_searched(_p(W), ctypes.c_int64(R), ctypes.c_int64(C), ctypes.c_int64(C), ctypes.c_int(G),
                                          _p(s), _p(clip_grid), ctypes.c_int(clip_grid.size), _p(actions), _p(clip_idx),
                                          _p(thr_grid), ctypes.c_int(thr_grid.size), _p(thr_idx), _p(offs), _p(codes),
                                          _p(scales), _p(zeros), _p(wq))
    if rc:
        raise ValueError("oracle_apply_plan_searched: bad arguments")
    return dict(codes=codes, scales=scales, zeros=zeros, wq=wq, code_offsets=offs)
