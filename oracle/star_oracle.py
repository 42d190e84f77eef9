"""numpy front end of the C oracle in ``star_oracle.c``.

TEST INFRASTRUCTURE ONLY (see the header of ``star_oracle.c``).  This module
compiles the C file with gcc on first use and marshals numpy arrays into it.
It holds no arithmetic of its own.

bf16 gradients travel as ``numpy.uint16`` arrays holding the raw bit patterns;
fp32 gradients as ``numpy.float32`` arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "star_oracle.c")
_LIB = os.path.join(_HERE, "libstar_oracle.so")
_lock = threading.Lock()
_lib = None

DTYPE_F32 = 0
DTYPE_BF16 = 1

# IEEE sequence must survive the compiler: no contraction, no fast-math.
CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall", "-Wextra",
          "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile ``star_oracle.c`` into ``libstar_oracle.so`` beside it."""
    with _lock:
        stale = (not os.path.exists(_LIB)
                 or os.path.getmtime(_LIB) < os.path.getmtime(_SRC))
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        common = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                  ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p,
                  ctypes.c_int, ctypes.c_void_p]
        lib.oracle_group_update_f32.argtypes = common + [
            ctypes.c_float, ctypes.c_float, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        lib.oracle_group_update_f32.restype = ctypes.c_int
        lib.oracle_group_update_f64.argtypes = common + [
            ctypes.c_double, ctypes.c_double, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_group_update_f64.restype = ctypes.c_int
        lib.oracle_group_reduce_f32.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int,
                                                ctypes.c_int]
        lib.oracle_group_reduce_f32.restype = ctypes.c_int
        lib.oracle_update_from_sums_f32.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                    ctypes.c_int, ctypes.c_int64, ctypes.c_int,
                                                    ctypes.c_float, ctypes.c_float, ctypes.c_float]
        lib.oracle_update_from_sums_f32.restype = ctypes.c_int
        _lib = lib
    return _lib


def _grad_dtype(grads: Sequence[Optional[np.ndarray]]) -> int:
    kinds = {g.dtype for g in grads if g is not None}
    if kinds == {np.dtype(np.float32)}:
        return DTYPE_F32
    if kinds == {np.dtype(np.uint16)}:
        return DTYPE_BF16
    raise TypeError("gradients must all be float32, or all uint16 (bf16 bits): %r" % kinds)


SUM_ORDERS = {"linear": 0, "tree": 1}


def _call(fn, real, params, momentum, grads, group_offsets, group_members, lrs, mu, wd,
          snapshots, sum_order="linear"):
    n = params.shape[0]
    if params.dtype != real or momentum.dtype != real:
        raise TypeError("params/momentum must be %s" % real)
    if momentum.shape != (n,) or params.ndim != 1:
        raise ValueError("params and momentum must be 1-D of equal length")
    for a in (params, momentum):
        if not a.flags.c_contiguous or not a.flags.writeable:
            raise ValueError("params/momentum must be contiguous and writeable")
    W = len(grads)
    dt = _grad_dtype(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    keep = []
    for w, g in enumerate(grads):
        if g is None:
            ptrs[w] = None
            continue
        if g.shape != (n,) or not g.flags.c_contiguous:
            raise ValueError("gradient %d must be contiguous with %d elements" % (w, n))
        keep.append(g)
        ptrs[w] = g.ctypes.data
    off = np.ascontiguousarray(group_offsets, dtype=np.int32)
    mem = np.ascontiguousarray(group_members, dtype=np.int32)
    K = off.shape[0] - 1 if off.shape[0] > 0 else 0
    lr_arr = np.ascontiguousarray(np.broadcast_to(np.asarray(lrs, dtype=real), (max(K, 0),)))
    for w in mem[: off[K] if K > 0 else 0]:
        if 0 <= w < W and grads[w] is None:
            raise ValueError("scheduled worker %d has no gradient buffer" % w)
    snap_ptrs = None
    snap_kinds = set()
    if snapshots is not None:
        if len(snapshots) != K:
            raise ValueError("snapshots needs one entry (array or None) per group")
        snap_ptrs = (ctypes.c_void_p * max(K, 1))()
        for k, s in enumerate(snapshots):
            if s is None:
                snap_ptrs[k] = None
                continue
            if s.dtype == np.uint16 and real == np.float32:
                snap_kinds.add(DTYPE_BF16)
            elif s.dtype == real:
                snap_kinds.add(DTYPE_F32)
            else:
                raise ValueError("snapshot %d has the wrong dtype" % k)
            if s.shape != (n,) or not s.flags.c_contiguous:
                raise ValueError("snapshot %d has the wrong shape" % k)
            snap_ptrs[k] = s.ctypes.data
    if len(snap_kinds) > 1:
        raise ValueError("snapshots must all have one dtype")
    extra = [snap_kinds.pop() if snap_kinds else DTYPE_F32] if real == np.float32 else []
    rc = fn(params.ctypes.data, momentum.ctypes.data, ptrs, W, dt, n,
            off.ctypes.data, mem.ctypes.data, K, lr_arr.ctypes.data,
            mu, wd, snap_ptrs, *extra, SUM_ORDERS[sum_order])
    if rc != 0:
        raise ValueError("schedule outside the definition (empty group, duplicate or "
                         "out-of-range member)")


def group_update_f32(params, momentum, grads, group_offsets, group_members, lrs, mu, wd,
                     snapshots=None, sum_order="linear"):
    """Canonical binary32 grouped update, in place on ``params`` / ``momentum``.

    ``lrs`` is a scalar or one learning rate per group.  ``mu`` and ``wd`` are
    rounded to binary32 on the way in, as the C signature takes floats.
    ``sum_order`` is "linear" (left to right) or "tree" (pairwise).  Snapshot
    arrays are float32, or uint16 to receive the parameters rounded to bf16.
    """
    _call(_load().oracle_group_update_f32, np.float32, params, momentum, grads,
          group_offsets, group_members, lrs, float(np.float32(mu)), float(np.float32(wd)),
          snapshots, sum_order)


def group_update_f64(params, momentum, grads, group_offsets, group_members, lrs, mu, wd,
                     snapshots=None, sum_order="linear"):
    """Binary64 shadow of the same loop, in place on float64 arrays."""
    _call(_load().oracle_group_update_f64, np.float64, params, momentum, grads,
          group_offsets, group_members, lrs, float(mu), float(wd), snapshots, sum_order)


def group_reduce_f32(grads, members, out_dtype="f32", sum_order="linear") -> np.ndarray:
    """Binary32 sum of ``grads[m]`` for m in ``members`` (listed order or
    pairwise): what a parent of the all-reduce architecture forwards.  Returns
    a float32 array, or uint16 bf16 bit patterns for ``out_dtype="bf16"``."""
    W = len(grads)
    dt = _grad_dtype(grads)
    n = next(g for g in grads if g is not None).shape[0]
    ptrs = (ctypes.c_void_p * max(W, 1))()
    for w, g in enumerate(grads):
        if g is None:
            continue
        if g.shape != (n,) or not g.flags.c_contiguous:
            raise ValueError("gradient %d must be contiguous with %d elements" % (w, n))
        ptrs[w] = g.ctypes.data
    mem = np.ascontiguousarray(members, dtype=np.int32)
    for w in mem:
        if 0 <= w < W and grads[w] is None:
            raise ValueError("listed worker %d has no gradient buffer" % w)
    out = np.empty(n, np.uint16 if out_dtype == "bf16" else np.float32)
    rc = _load().oracle_group_reduce_f32(out.ctypes.data, DTYPE_BF16 if out_dtype == "bf16" else DTYPE_F32,
                                         ptrs, W, dt, n, mem.ctypes.data, mem.shape[0],
                                         SUM_ORDERS[sum_order])
    if rc != 0:
        raise ValueError("member list outside the definition (empty, duplicate or out-of-range member)")
    return out


def update_from_sums_f32(params, momentum, sums, n_reports, lr, mu, wd) -> None:
    """One update from partial sums (float32 arrays, added left to right), the
    mean taken over ``n_reports`` gradient reports; in place."""
    n = params.shape[0]
    for a in (params, momentum):
        if a.dtype != np.float32 or a.shape != (n,) or not a.flags.c_contiguous or not a.flags.writeable:
            raise ValueError("params/momentum must be contiguous writeable float32 of equal length")
    R = len(sums)
    ptrs = (ctypes.c_void_p * max(R, 1))()
    for r, s in enumerate(sums):
        if s.dtype != np.float32 or s.shape != (n,) or not s.flags.c_contiguous:
            raise ValueError("partial sum %d must be contiguous float32 with %d elements" % (r, n))
        ptrs[r] = s.ctypes.data
    rc = _load().oracle_update_from_sums_f32(params.ctypes.data, momentum.ctypes.data, ptrs, R, n,
                                             int(n_reports), float(np.float32(lr)), float(np.float32(mu)),
                                             float(np.float32(wd)))
    if rc != 0:
        raise ValueError("need at least one partial sum and n_reports >= their number")
