"""ctypes binding of ``libstar.so`` (declared in ``include/star.h``).

Argument marshalling only: every function here has the name of the C entry
point it forwards to, turns torch tensors into device pointers and Python lists
into host arrays, and raises :class:`StarError` on a non-zero status.  PyTorch
supplies device memory and the current stream; nothing is computed in Python
and there is no fallback: if the library is missing, importing this module
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

from .workloads import ModeDecision

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libstar.so")

STAR_OK = 0
STAR_ERR_NULL_POINTER = 1
STAR_ERR_INVALID_ARG = 2
STAR_ERR_BAD_SCHEDULE = 3
STAR_ERR_UNSUPPORTED = 4
STAR_ERR_WORKSPACE_TOO_SMALL = 5
STAR_ERR_CUDA = 6

STAR_DTYPE_F32 = 0
STAR_DTYPE_BF16 = 1
STAR_MAX_WORKERS = 64
STAR_SUM_LINEAR = 0
STAR_SUM_TREE = 1


class StarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = _lib.star_status_string(status).decode()
        extra = ""
        if status == STAR_ERR_CUDA:
            extra = " (cudaError %d)" % _lib.star_last_cuda_error()
        super().__init__("%s failed: %s%s" % (where, name, extra))


class star_multi_plan_t(ctypes.Structure):
    _fields_ = [
        ("magic", ctypes.c_uint64),
        ("d_workspace", ctypes.c_void_p),
        ("total_elements", ctypes.c_int64),
        ("n_tiles", ctypes.c_int64),
        ("complete_workers", ctypes.c_uint64),
        ("n_tensors", ctypes.c_int32),
        ("W", ctypes.c_int32),
        ("grad_dtype", ctypes.c_int32),
        ("tile_elements", ctypes.c_int32),
        ("n_snapshot_sets", ctypes.c_int32),
        ("snapshot_dtype", ctypes.c_int32),
    ]


def _load() -> ctypes.CDLL:
    # (Re)build in-tree when the library is missing or older than its sources and
    # nvcc is at hand; otherwise fail loudly: there is no CPU fallback.
    try:
        from . import build as _build
        if _build.is_stale():
            _build.build()
    except Exception as exc:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "%s is missing and could not be built (%s): run "
                "`python -m paper_2512_09685_b200.build`; there is no CPU fallback" % (LIB_PATH, exc))
    lib = ctypes.CDLL(LIB_PATH)
    c_int, c_i64, c_vp, c_f = ctypes.c_int, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float
    lib.star_status_string.argtypes = [c_int]
    lib.star_status_string.restype = ctypes.c_char_p
    lib.star_last_cuda_error.argtypes = []
    lib.star_last_cuda_error.restype = c_int
    lib.star_launch_count.argtypes = []
    lib.star_launch_count.restype = c_i64
    lib.star_schedule_validate.argtypes = [c_vp, c_vp, c_int, c_int]
    lib.star_schedule_static_x.argtypes = [c_vp, c_int, c_int, c_int, c_int, c_vp, c_vp, c_vp]
    lib.star_schedule_from_labels.argtypes = [c_vp, c_int, c_vp, c_vp, c_vp]
    lib.star_schedule_dynamic_x.argtypes = [c_vp, c_vp, c_int, c_vp, c_vp, c_vp]
    lib.star_group_update.argtypes = [c_vp, c_vp, c_vp, c_int, c_int, c_i64, c_vp, c_vp, c_int,
                                      c_f, c_f, c_f, c_vp]
    lib.star_multi_workspace_bytes.argtypes = [c_int, c_vp, c_int, c_vp]
    lib.star_multi_prepare.argtypes = [c_int, c_vp, c_vp, c_vp, c_vp, c_int, c_int, c_vp,
                                       ctypes.c_size_t, c_vp, c_vp]
    lib.star_group_update_multi.argtypes = [c_vp, c_vp, c_vp, c_int, c_f, c_f, c_f, c_vp]
    lib.star_group_update_multi_lrs.argtypes = [c_vp, c_vp, c_vp, c_int, c_vp, c_f, c_f, c_vp]
    lib.star_group_update_multi_lrs.restype = c_int
    lib.star_group_update_ex.argtypes = [c_vp, c_vp, c_vp, c_int, c_int, c_i64, c_vp, c_vp, c_int,
                                         c_vp, c_f, c_f, c_vp, c_int, c_int, c_vp]
    lib.star_group_update_ex.restype = c_int
    lib.star_cluster_iteration_times.argtypes = [c_vp, c_int, c_int, ctypes.c_double, c_vp, c_vp]
    lib.star_cluster_iteration_times.restype = c_int
    lib.star_mode_times.argtypes = [c_vp, c_vp, c_int, ctypes.c_double, ctypes.c_double, c_vp, c_vp]
    lib.star_mode_times.restype = c_int
    lib.star_choose_mode.argtypes = [c_vp, c_vp, c_int, ctypes.c_double, ctypes.c_double, c_vp, c_vp,
                                     c_vp, c_vp, c_vp]
    lib.star_choose_mode.restype = c_int
    lib.star_choose_all_reduce_mode.argtypes = [c_vp, c_vp, c_int] + [ctypes.c_double] * 4 + [c_vp] * 7
    lib.star_choose_all_reduce_mode.restype = c_int
    lib.star_assign_parents.argtypes = [c_vp, c_int, c_int, c_vp]
    lib.star_assign_parents.restype = c_int
    lib.star_build_tree.argtypes = [c_vp, c_int, c_int, c_vp]
    lib.star_build_tree.restype = c_int
    lib.star_shard_range.argtypes = [c_i64, c_int, c_int, c_i64, c_vp, c_vp]
    lib.star_shard_range.restype = c_int
    lib.star_host_workspace_bytes.argtypes = [c_int, c_int, c_i64, c_vp]
    lib.star_host_workspace_bytes.restype = c_int
    lib.star_group_update_host.argtypes = [c_vp, c_vp, c_vp, c_int, c_int, c_i64, c_vp, c_vp, c_int,
                                           c_f, c_f, c_f, c_vp, ctypes.c_size_t, c_vp]
    lib.star_group_update_host.restype = c_int
    lib.star_host_workspace_bytes_ex.argtypes = [c_int, c_int, c_int, c_int, c_i64, c_vp]
    lib.star_host_workspace_bytes_ex.restype = c_int
    lib.star_group_update_host_ex.argtypes = [c_vp, c_vp, c_vp, c_int, c_int, c_i64, c_vp, c_vp, c_int,
                                              c_vp, c_f, c_f, c_vp, c_int, c_int, c_vp, ctypes.c_size_t, c_vp]
    lib.star_group_update_host_ex.restype = c_int
    lib.star_group_update_multi_noalloc.argtypes = [c_int, c_vp, c_vp, c_vp, c_vp, c_int, c_int, c_vp, c_vp,
                                                    c_int, c_f, c_f, c_f, c_vp]
    lib.star_group_update_multi_noalloc.restype = c_int
    lib.star_group_reduce.argtypes = [c_vp, c_int, c_vp, c_int, c_int, c_i64, c_vp, c_int, c_int, c_vp]
    lib.star_group_reduce.restype = c_int
    lib.star_group_update_from_sums.argtypes = [c_vp, c_vp, c_vp, c_int, c_i64, c_int, c_f, c_f, c_f, c_vp]
    lib.star_group_update_from_sums.restype = c_int
    lib.star_multi_workspace_bytes_ex.argtypes = [c_int, c_vp, c_int, c_int, c_vp]
    lib.star_multi_workspace_bytes_ex.restype = c_int
    lib.star_multi_prepare_ex.argtypes = [c_int, c_vp, c_vp, c_vp, c_vp, c_int, c_int, c_int, c_vp, c_int, c_vp,
                                          ctypes.c_size_t, c_vp, c_vp]
    lib.star_multi_prepare_ex.restype = c_int
    lib.star_group_update_multi_ex.argtypes = [c_vp, c_vp, c_vp, c_int, c_vp, c_f, c_f, c_vp, c_int, c_vp]
    lib.star_group_update_multi_ex.restype = c_int
    for name in ("star_schedule_validate", "star_schedule_static_x", "star_schedule_from_labels",
                 "star_schedule_dynamic_x", "star_group_update", "star_multi_workspace_bytes",
                 "star_multi_prepare", "star_group_update_multi"):
        getattr(lib, name).restype = c_int
    return lib


_lib = _load()


def _check(status: int, where: str) -> None:
    if status != STAR_OK:
        raise StarError(status, where)


def _i32(values: Sequence[int]):
    return (ctypes.c_int32 * max(len(values), 1))(*values)


def star_status_string(status: int) -> str:
    return _lib.star_status_string(status).decode()


def star_last_cuda_error() -> int:
    return _lib.star_last_cuda_error()


def star_launch_count() -> int:
    return _lib.star_launch_count()


# ---------------------------------------------------------------------------
# schedule encoding (host only)
# ---------------------------------------------------------------------------
Schedule = Tuple[List[int], List[int]]


def _unpack(offsets, members, n_groups) -> Schedule:
    K = n_groups.value
    off = list(offsets[: K + 1])
    return off, list(members[: off[K]])


def star_schedule_validate(group_offsets: Sequence[int], group_members: Sequence[int],
                           n_groups: int, W: int) -> int:
    """Returns the status code (does not raise)."""
    return _lib.star_schedule_validate(_i32(group_offsets), _i32(group_members), n_groups, W)


def star_schedule_static_x(arrival_order: Optional[Sequence[int]], W: int, x: int,
                           sort_members: bool = False) -> Schedule:
    offsets, members, K = _i32([0] * (W + 1)), _i32([0] * W), ctypes.c_int(0)
    if arrival_order is None:
        order, n_arrived = None, W
    else:
        if len(arrival_order) > W:
            raise StarError(STAR_ERR_INVALID_ARG, "star_schedule_static_x")
        order, n_arrived = _i32(arrival_order), len(arrival_order)
    _check(_lib.star_schedule_static_x(order, n_arrived, W, x, int(sort_members), offsets, members,
                                       ctypes.byref(K)), "star_schedule_static_x")
    return _unpack(offsets, members, K)


def star_schedule_from_labels(group_of_worker: Sequence[int]) -> Schedule:
    W = len(group_of_worker)
    offsets, members, K = _i32([0] * (W + 1)), _i32([0] * W), ctypes.c_int(0)
    _check(_lib.star_schedule_from_labels(_i32(group_of_worker), W, offsets, members,
                                          ctypes.byref(K)), "star_schedule_from_labels")
    return _unpack(offsets, members, K)


def star_schedule_dynamic_x(iter_time: Sequence[float], cluster_of_worker: Sequence[int]) -> Schedule:
    W = len(cluster_of_worker)
    if len(iter_time) != W:
        raise StarError(STAR_ERR_INVALID_ARG, "star_schedule_dynamic_x")
    offsets, members, K = _i32([0] * (W + 1)), _i32([0] * W), ctypes.c_int(0)
    times = (ctypes.c_double * max(W, 1))(*iter_time)
    _check(_lib.star_schedule_dynamic_x(times, _i32(cluster_of_worker), W, offsets, members,
                                        ctypes.byref(K)), "star_schedule_dynamic_x")
    return _unpack(offsets, members, K)


def _f64(values: Sequence[float]):
    return (ctypes.c_double * max(len(values), 1))(*values)


def star_cluster_iteration_times(iter_time: Sequence[float], n_clusters: int = 0,
                                 max_distance: float = -1.0) -> List[int]:
    """Cluster label per worker (average-linkage agglomerative clustering)."""
    W = len(iter_time)
    labels, K = _i32([0] * W), ctypes.c_int(0)
    _check(_lib.star_cluster_iteration_times(_f64(iter_time), W, n_clusters, max_distance, labels,
                                             ctypes.byref(K)), "star_cluster_iteration_times")
    return list(labels[:W])


def star_mode_times(iter_time: Sequence[float], cluster_of_worker: Optional[Sequence[int]], phi: float,
                    M: float) -> Tuple[List[float], Optional[float]]:
    """(T_x for x = 1..W by Eq. 1, T_d by Eq. 2 or None without clusters)."""
    W = len(iter_time)
    T_static, T_dynamic = _f64([0.0] * W), ctypes.c_double(0.0)
    clusters = None if cluster_of_worker is None else _i32(cluster_of_worker)
    _check(_lib.star_mode_times(_f64(iter_time), clusters, W, phi, M, T_static, ctypes.byref(T_dynamic)),
           "star_mode_times")
    return list(T_static[:W]), (None if clusters is None else T_dynamic.value)


def star_choose_mode(iter_time: Sequence[float], cluster_of_worker: Optional[Sequence[int]], phi: float,
                     M: float) -> Tuple[int, float, Schedule]:
    """(x, T, schedule): x = 0 means the dynamic mode."""
    W = len(iter_time)
    x, T, K = ctypes.c_int(0), ctypes.c_double(0.0), ctypes.c_int(0)
    offsets, members = _i32([0] * (W + 1)), _i32([0] * W)
    clusters = None if cluster_of_worker is None else _i32(cluster_of_worker)
    _check(_lib.star_choose_mode(_f64(iter_time), clusters, W, phi, M, ctypes.byref(x), ctypes.byref(T),
                                 offsets, members, ctypes.byref(K)), "star_choose_mode")
    return x.value, T.value, _unpack(offsets, members, K)


def star_choose_all_reduce_mode(iter_time: Sequence[float], child_time: Sequence[float], phi: float,
                                M: float, t_w_max: float, straggler_threshold: float = 0.2):
    """(x, t_w, T_a, removed workers, schedule of the one contributing group)."""
    W = len(iter_time)
    if len(child_time) != W:
        raise StarError(STAR_ERR_INVALID_ARG, "star_choose_all_reduce_mode")
    x, t_w, T, K = ctypes.c_int(0), ctypes.c_double(0.0), ctypes.c_double(0.0), ctypes.c_int(0)
    removed, offsets, members = _i32([0] * W), _i32([0] * (W + 1)), _i32([0] * W)
    _check(_lib.star_choose_all_reduce_mode(_f64(iter_time), _f64(child_time), W, phi, M, t_w_max,
                                            straggler_threshold, ctypes.byref(x), ctypes.byref(t_w),
                                            ctypes.byref(T), removed, offsets, members, ctypes.byref(K)),
           "star_choose_all_reduce_mode")
    return x.value, t_w.value, T.value, list(removed[: x.value]), _unpack(offsets, members, K)


def star_assign_parents(removed: Sequence[int], W: int) -> List[int]:
    """Parent of every worker (-1 for ring members) when ``removed`` leave the ring."""
    out = _i32([0] * W)
    _check(_lib.star_assign_parents(_i32(removed), len(removed), W, out), "star_assign_parents")
    return list(out[:W])


def star_build_tree(latency: Sequence[float], fanout: int) -> List[int]:
    """Parent of every worker (-1 = child of the root) in the latency-ordered tree."""
    W = len(latency)
    out = _i32([0] * W)
    _check(_lib.star_build_tree(_f64(latency), W, fanout, out), "star_build_tree")
    return list(out[:W])


def star_shard_range(n: int, world: int, rank: int, align: int = 16) -> Tuple[int, int]:
    """(first, count) of the element range rank ``rank`` of ``world`` owns."""
    first, count = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(_lib.star_shard_range(n, world, rank, align, ctypes.byref(first), ctypes.byref(count)),
           "star_shard_range")
    return first.value, count.value


def encode(decision: ModeDecision) -> Schedule:
    """Dispatch a mode decision to the matching C encoder."""
    if decision.kind == "labels":
        return star_schedule_from_labels(decision.labels)
    if decision.kind == "static_x":
        return star_schedule_static_x(decision.arrival_order, decision.W, decision.x,
                                      decision.sort_members)
    if decision.kind == "dynamic_x":
        return star_schedule_dynamic_x(decision.iter_time, decision.labels)
    raise ValueError(decision.kind)


# ---------------------------------------------------------------------------
# fused grouped update
# ---------------------------------------------------------------------------
def _grad_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return STAR_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return STAR_DTYPE_BF16
    raise TypeError("gradients must be float32 or bfloat16, got %s" % t.dtype)


def _state(t: torch.Tensor, what: str) -> int:
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous():
        raise TypeError("%s must be a contiguous float32 CUDA tensor" % what)
    return t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def star_group_update(params: torch.Tensor, momentum: torch.Tensor,
                      grads: Sequence[Optional[torch.Tensor]], group_offsets: Sequence[int],
                      group_members: Sequence[int], lr: float, mu: float, wd: float,
                      stream=None) -> None:
    """In-place fused grouped update of one flat tensor on the current device."""
    n = params.numel()
    p, v = _state(params, "params"), _state(momentum, "momentum")
    if momentum.numel() != n:
        raise ValueError("params and momentum differ in size")
    W = len(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    dt = None
    for w, g in enumerate(grads):
        if g is None:
            continue
        if not g.is_cuda or not g.is_contiguous() or g.numel() != n:
            raise ValueError("gradient %d must be a contiguous CUDA tensor of %d elements" % (w, n))
        d = _grad_dtype(g)
        if dt is not None and d != dt:
            raise TypeError("gradients differ in dtype")
        dt = d
        ptrs[w] = g.data_ptr()
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    _check(_lib.star_group_update(p, v, ptrs, W, STAR_DTYPE_F32 if dt is None else dt, n,
                                  _i32(group_offsets), _i32(group_members), K, lr, mu, wd,
                                  _stream(stream)), "star_group_update")


class FlatRoundBuffers:
    """The buffers of a flat round marshalled once: for callers that run many
    rounds on the same tensors (only the schedule and the scalars change per
    round), which saves building the pointer array and re-checking the tensors
    on every call -- on launch-bound sizes that is most of the host time.  Holds
    references to the tensors; computes nothing."""

    def __init__(self, params: torch.Tensor, momentum: torch.Tensor, grads: Sequence[Optional[torch.Tensor]]):
        self.n = params.numel()
        self.p, self.v = _state(params, "params"), _state(momentum, "momentum")
        if momentum.numel() != self.n:
            raise ValueError("params and momentum differ in size")
        self.W = len(grads)
        self.ptrs, self.dtype = _grad_pointers(grads, self.n)
        self._keep = (params, momentum, list(grads))

    def star_group_update(self, group_offsets: Sequence[int], group_members: Sequence[int], lr: float, mu: float,
                          wd: float, stream=None) -> None:
        K = len(group_offsets) - 1 if len(group_offsets) else 0
        _check(_lib.star_group_update(self.p, self.v, self.ptrs, self.W, self.dtype, self.n, _i32(group_offsets),
                                      _i32(group_members), K, lr, mu, wd, _stream(stream)), "star_group_update")


def star_group_update_ex(params: torch.Tensor, momentum: torch.Tensor,
                         grads: Sequence[Optional[torch.Tensor]], group_offsets: Sequence[int],
                         group_members: Sequence[int], lrs: Sequence[float], mu: float, wd: float,
                         snapshots: Optional[Sequence[Optional[torch.Tensor]]] = None,
                         sum_order: int = STAR_SUM_LINEAR, stream=None) -> None:
    """The round with one learning rate per group; ``snapshots[k]`` (CUDA tensor,
    all float32 or all bfloat16, or None) receives the parameters right after
    group k's update; ``sum_order`` is STAR_SUM_LINEAR or STAR_SUM_TREE."""
    n = params.numel()
    p, v = _state(params, "params"), _state(momentum, "momentum")
    if momentum.numel() != n:
        raise ValueError("params and momentum differ in size")
    W = len(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    dt = None
    for w, g in enumerate(grads):
        if g is None:
            continue
        if not g.is_cuda or not g.is_contiguous() or g.numel() != n:
            raise ValueError("gradient %d must be a contiguous CUDA tensor of %d elements" % (w, n))
        d = _grad_dtype(g)
        if dt is not None and d != dt:
            raise TypeError("gradients differ in dtype")
        dt = d
        ptrs[w] = g.data_ptr()
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    if len(lrs) != K:
        raise ValueError("need one learning rate per group")
    lr_arr = (ctypes.c_float * max(K, 1))(*lrs)
    snap_arr, snap_dt = None, STAR_DTYPE_F32
    if snapshots is not None:
        if len(snapshots) != K:
            raise ValueError("snapshots needs one entry (tensor or None) per group")
        snap_arr = (ctypes.c_void_p * max(K, 1))()
        kinds = set()
        for k, s in enumerate(snapshots):
            if s is None:
                continue
            if s.numel() != n or not s.is_cuda or not s.is_contiguous():
                raise ValueError("snapshot %d must be a contiguous CUDA tensor of %d elements" % (k, n))
            kinds.add(_grad_dtype(s))
            snap_arr[k] = s.data_ptr()
        if len(kinds) > 1:
            raise TypeError("snapshots differ in dtype")
        snap_dt = kinds.pop() if kinds else STAR_DTYPE_F32
    _check(_lib.star_group_update_ex(p, v, ptrs, W, STAR_DTYPE_F32 if dt is None else dt, n,
                                     _i32(group_offsets), _i32(group_members), K, lr_arr, mu, wd,
                                     snap_arr, snap_dt, sum_order, _stream(stream)), "star_group_update_ex")


def _grad_pointers(grads: Sequence[Optional[torch.Tensor]], n: int):
    """(ctypes array of W device pointers, dtype code) of a list of flat gradient tensors."""
    W = len(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    dt = None
    for w, g in enumerate(grads):
        if g is None:
            continue
        if not g.is_cuda or not g.is_contiguous() or g.numel() != n:
            raise ValueError("gradient %d must be a contiguous CUDA tensor of %d elements" % (w, n))
        d = _grad_dtype(g)
        if dt is not None and d != dt:
            raise TypeError("gradients differ in dtype")
        dt = d
        ptrs[w] = g.data_ptr()
    return ptrs, STAR_DTYPE_F32 if dt is None else dt


def star_group_reduce(out: torch.Tensor, grads: Sequence[Optional[torch.Tensor]], members: Sequence[int],
                      sum_order: int = STAR_SUM_LINEAR, stream=None) -> None:
    """``out[i] = grads[members[0]][i] + grads[members[1]][i] + ...`` (what a parent
    of the all-reduce architecture forwards to the ring); ``out`` is a float32
    or bfloat16 CUDA tensor."""
    n = out.numel()
    if not out.is_cuda or not out.is_contiguous():
        raise TypeError("out must be a contiguous CUDA tensor")
    ptrs, dt = _grad_pointers(grads, n)
    _check(_lib.star_group_reduce(out.data_ptr(), _grad_dtype(out), ptrs, len(grads), dt, n, _i32(members),
                                  len(members), sum_order, _stream(stream)), "star_group_reduce")


def star_group_update_from_sums(params: torch.Tensor, momentum: torch.Tensor, sums: Sequence[torch.Tensor],
                                n_reports: int, lr: float, mu: float, wd: float, stream=None) -> None:
    """One update from the ring members' aggregates ``sums`` (float32 CUDA tensors,
    added in the listed order), the mean taken over ``n_reports`` gradient reports."""
    n = params.numel()
    p, v = _state(params, "params"), _state(momentum, "momentum")
    if momentum.numel() != n:
        raise ValueError("params and momentum differ in size")
    for r, t in enumerate(sums):
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or t.numel() != n:
            raise ValueError("sum %d must be a contiguous float32 CUDA tensor of %d elements" % (r, n))
    ptrs = (ctypes.c_void_p * max(len(sums), 1))(*[t.data_ptr() for t in sums])
    _check(_lib.star_group_update_from_sums(p, v, ptrs, len(sums), n, n_reports, lr, mu, wd, _stream(stream)),
           "star_group_update_from_sums")


def star_multi_workspace_bytes(sizes: Sequence[int], W: int) -> int:
    out = ctypes.c_size_t(0)
    arr = (ctypes.c_int64 * max(len(sizes), 1))(*sizes)
    _check(_lib.star_multi_workspace_bytes(len(sizes), arr, W, ctypes.byref(out)),
           "star_multi_workspace_bytes")
    return out.value


def star_multi_prepare(params: Sequence[torch.Tensor], momentum: Sequence[torch.Tensor],
                       grads: Sequence[Sequence[Optional[torch.Tensor]]], workspace: torch.Tensor,
                       stream=None) -> star_multi_plan_t:
    """``grads[w][t]`` = worker w's gradient for tensor t.  ``workspace`` is a
    uint8 CUDA tensor of at least :func:`star_multi_workspace_bytes` bytes; the
    returned plan refers to it (keep the tensor alive)."""
    T, W = len(params), len(grads)
    if len(momentum) != T or any(len(g) != T for g in grads):
        raise ValueError("params, momentum and every worker's gradient list need one entry per tensor")
    sizes = [p.numel() for p in params]
    P = (ctypes.c_void_p * max(T, 1))(*[_state(p, "params") if p.numel() else None for p in params])
    V = (ctypes.c_void_p * max(T, 1))(*[_state(v, "momentum") if v.numel() else None for v in momentum])
    G = (ctypes.c_void_p * max(T * W, 1))()
    dt = None
    for w in range(W):
        for t in range(T):
            g = grads[w][t]
            if g is None:
                continue
            if not g.is_cuda or not g.is_contiguous() or g.numel() != sizes[t]:
                raise ValueError("gradient [%d][%d] must be a contiguous CUDA tensor of %d elements"
                                 % (w, t, sizes[t]))
            d = _grad_dtype(g)
            if dt is not None and d != dt:
                raise TypeError("gradients differ in dtype")
            dt = d
            G[t * W + w] = g.data_ptr() if sizes[t] else None
    if momentum and any(v.numel() != s for v, s in zip(momentum, sizes)):
        raise ValueError("params and momentum differ in size")
    if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous uint8 CUDA tensor")
    plan = star_multi_plan_t()
    S = (ctypes.c_int64 * max(T, 1))(*sizes)
    _check(_lib.star_multi_prepare(T, P, V, G, S, W, STAR_DTYPE_F32 if dt is None else dt,
                                   workspace.data_ptr(), workspace.numel(), _stream(stream),
                                   ctypes.byref(plan)), "star_multi_prepare")
    return plan


def star_group_update_multi(plan: star_multi_plan_t, group_offsets: Sequence[int],
                            group_members: Sequence[int], lr: float, mu: float, wd: float,
                            stream=None) -> None:
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    _check(_lib.star_group_update_multi(ctypes.byref(plan), _i32(group_offsets), _i32(group_members),
                                        K, lr, mu, wd, _stream(stream)), "star_group_update_multi")


def star_group_update_multi_lrs(plan: star_multi_plan_t, group_offsets: Sequence[int],
                                group_members: Sequence[int], lrs: Sequence[float], mu: float, wd: float,
                                stream=None) -> None:
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    if len(lrs) != K:
        raise ValueError("need one learning rate per group")
    _check(_lib.star_group_update_multi_lrs(ctypes.byref(plan), _i32(group_offsets), _i32(group_members), K,
                                            (ctypes.c_float * max(K, 1))(*lrs), mu, wd, _stream(stream)),
           "star_group_update_multi_lrs")


def star_multi_workspace_bytes_ex(sizes: Sequence[int], W: int, n_snapshot_sets: int) -> int:
    out = ctypes.c_size_t(0)
    arr = (ctypes.c_int64 * max(len(sizes), 1))(*sizes)
    _check(_lib.star_multi_workspace_bytes_ex(len(sizes), arr, W, n_snapshot_sets, ctypes.byref(out)),
           "star_multi_workspace_bytes_ex")
    return out.value


def _list_pointers(params, momentum, grads):
    """Pointer arrays (P, V, G, sizes array, dtype code) of a tensor list;
    ``grads[w][t]`` = worker w's gradient for tensor t."""
    T, W = len(params), len(grads)
    if len(momentum) != T or any(len(g) != T for g in grads):
        raise ValueError("params, momentum and every worker's gradient list need one entry per tensor")
    sizes = [p.numel() for p in params]
    if any(v.numel() != s for v, s in zip(momentum, sizes)):
        raise ValueError("params and momentum differ in size")
    P = (ctypes.c_void_p * max(T, 1))(*[_state(p, "params") if p.numel() else None for p in params])
    V = (ctypes.c_void_p * max(T, 1))(*[_state(v, "momentum") if v.numel() else None for v in momentum])
    G = (ctypes.c_void_p * max(T * W, 1))()
    dt = None
    for w in range(W):
        for t in range(T):
            g = grads[w][t]
            if g is None or sizes[t] == 0:
                continue
            if not g.is_cuda or not g.is_contiguous() or g.numel() != sizes[t]:
                raise ValueError("gradient [%d][%d] must be a contiguous CUDA tensor of %d elements"
                                 % (w, t, sizes[t]))
            d = _grad_dtype(g)
            if dt is not None and d != dt:
                raise TypeError("gradients differ in dtype")
            dt = d
            G[t * W + w] = g.data_ptr()
    S = (ctypes.c_int64 * max(T, 1))(*sizes)
    return P, V, G, S, sizes, STAR_DTYPE_F32 if dt is None else dt


def star_multi_prepare_ex(params: Sequence[torch.Tensor], momentum: Sequence[torch.Tensor],
                          grads: Sequence[Sequence[Optional[torch.Tensor]]],
                          snapshot_sets: Sequence[Sequence[Optional[torch.Tensor]]], workspace: torch.Tensor,
                          stream=None) -> star_multi_plan_t:
    """As :func:`star_multi_prepare`, registering ``snapshot_sets[s][t]`` (tensor
    t's buffer of snapshot set s, all float32 or all bfloat16, or None)."""
    T, W, S_sets = len(params), len(grads), len(snapshot_sets)
    P, V, G, S, sizes, dt = _list_pointers(params, momentum, grads)
    if any(len(one) != T for one in snapshot_sets):
        raise ValueError("every snapshot set needs one entry (tensor or None) per tensor")
    snaps = (ctypes.c_void_p * max(T * S_sets, 1))()
    kinds = set()
    for s_index, one in enumerate(snapshot_sets):
        for t, buf in enumerate(one):
            if buf is None or sizes[t] == 0:
                continue
            if not buf.is_cuda or not buf.is_contiguous() or buf.numel() != sizes[t]:
                raise ValueError("snapshot [%d][%d] must be a contiguous CUDA tensor of %d elements"
                                 % (s_index, t, sizes[t]))
            kinds.add(_grad_dtype(buf))
            snaps[t * S_sets + s_index] = buf.data_ptr()
    if len(kinds) > 1:
        raise TypeError("snapshots differ in dtype")
    if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous uint8 CUDA tensor")
    plan = star_multi_plan_t()
    _check(_lib.star_multi_prepare_ex(T, P, V, G, S, W, dt, S_sets, snaps, kinds.pop() if kinds else STAR_DTYPE_F32,
                                      workspace.data_ptr(), workspace.numel(), _stream(stream),
                                      ctypes.byref(plan)), "star_multi_prepare_ex")
    return plan


def star_group_update_multi_ex(plan: star_multi_plan_t, group_offsets: Sequence[int],
                               group_members: Sequence[int], lrs: Sequence[float], mu: float, wd: float,
                               snapshot_set_of_group: Optional[Sequence[int]] = None,
                               sum_order: int = STAR_SUM_LINEAR, stream=None) -> None:
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    if len(lrs) != K or (snapshot_set_of_group is not None and len(snapshot_set_of_group) != K):
        raise ValueError("need one learning rate (and one snapshot set index) per group")
    sets = None if snapshot_set_of_group is None else _i32(snapshot_set_of_group)
    _check(_lib.star_group_update_multi_ex(ctypes.byref(plan), _i32(group_offsets), _i32(group_members), K,
                                           (ctypes.c_float * max(K, 1))(*lrs), mu, wd, sets, sum_order,
                                           _stream(stream)), "star_group_update_multi_ex")


def star_host_workspace_bytes(max_scheduled: int, grad_dtype: torch.dtype, chunk_elements: int) -> int:
    out = ctypes.c_size_t(0)
    dt = STAR_DTYPE_BF16 if grad_dtype == torch.bfloat16 else STAR_DTYPE_F32
    _check(_lib.star_host_workspace_bytes(max_scheduled, dt, chunk_elements, ctypes.byref(out)),
           "star_host_workspace_bytes")
    return out.value


def star_group_update_host(params: torch.Tensor, momentum: torch.Tensor,
                           grads: Sequence[Optional[torch.Tensor]], group_offsets: Sequence[int],
                           group_members: Sequence[int], lr: float, mu: float, wd: float,
                           workspace: torch.Tensor, stream=None) -> None:
    """Fused grouped update of HOST tensors (ideally pinned), streamed through the
    device workspace in chunks.  Results are in ``params`` / ``momentum`` once the
    stream has been synchronized."""
    n = params.numel()
    for t, what in ((params, "params"), (momentum, "momentum")):
        if t.dtype != torch.float32 or t.is_cuda or not t.is_contiguous():
            raise TypeError("%s must be a contiguous float32 host tensor" % what)
    if momentum.numel() != n:
        raise ValueError("params and momentum differ in size")
    W = len(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    dt = None
    for w, g in enumerate(grads):
        if g is None:
            continue
        if g.is_cuda or not g.is_contiguous() or g.numel() != n:
            raise ValueError("gradient %d must be a contiguous host tensor of %d elements" % (w, n))
        d = _grad_dtype(g)
        if dt is not None and d != dt:
            raise TypeError("gradients differ in dtype")
        dt = d
        ptrs[w] = g.data_ptr()
    if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous uint8 CUDA tensor")
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    _check(_lib.star_group_update_host(params.data_ptr(), momentum.data_ptr(), ptrs, W,
                                       STAR_DTYPE_F32 if dt is None else dt, n, _i32(group_offsets),
                                       _i32(group_members), K, lr, mu, wd, workspace.data_ptr(),
                                       workspace.numel(), _stream(stream)), "star_group_update_host")


def star_host_workspace_bytes_ex(max_scheduled: int, grad_dtype: torch.dtype, max_snapshots: int,
                                 snapshot_dtype: torch.dtype, chunk_elements: int) -> int:
    out = ctypes.c_size_t(0)
    code = lambda dt: STAR_DTYPE_BF16 if dt == torch.bfloat16 else STAR_DTYPE_F32       # noqa: E731
    _check(_lib.star_host_workspace_bytes_ex(max_scheduled, code(grad_dtype), max_snapshots, code(snapshot_dtype),
                                             chunk_elements, ctypes.byref(out)), "star_host_workspace_bytes_ex")
    return out.value


def star_group_update_host_ex(params: torch.Tensor, momentum: torch.Tensor,
                              grads: Sequence[Optional[torch.Tensor]], group_offsets: Sequence[int],
                              group_members: Sequence[int], lrs: Sequence[float], mu: float, wd: float,
                              workspace: torch.Tensor, snapshots: Optional[Sequence[Optional[torch.Tensor]]] = None,
                              sum_order: int = STAR_SUM_LINEAR, stream=None) -> None:
    """The host-buffer round with per-group rates, host snapshot tensors
    (``snapshots[k]``: float32 or bfloat16 host tensor or None) and the summation order."""
    n = params.numel()
    for t, what in ((params, "params"), (momentum, "momentum")):
        if t.dtype != torch.float32 or t.is_cuda or not t.is_contiguous():
            raise TypeError("%s must be a contiguous float32 host tensor" % what)
    if momentum.numel() != n:
        raise ValueError("params and momentum differ in size")
    W = len(grads)
    ptrs = (ctypes.c_void_p * max(W, 1))()
    dt = None
    for w, g in enumerate(grads):
        if g is None:
            continue
        if g.is_cuda or not g.is_contiguous() or g.numel() != n:
            raise ValueError("gradient %d must be a contiguous host tensor of %d elements" % (w, n))
        d = _grad_dtype(g)
        if dt is not None and d != dt:
            raise TypeError("gradients differ in dtype")
        dt = d
        ptrs[w] = g.data_ptr()
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    if len(lrs) != K:
        raise ValueError("need one learning rate per group")
    snap_arr, snap_dt = None, STAR_DTYPE_F32
    if snapshots is not None:
        if len(snapshots) != K:
            raise ValueError("snapshots needs one entry (tensor or None) per group")
        snap_arr = (ctypes.c_void_p * max(K, 1))()
        kinds = set()
        for k, s in enumerate(snapshots):
            if s is None:
                continue
            if s.is_cuda or not s.is_contiguous() or s.numel() != n:
                raise ValueError("snapshot %d must be a contiguous host tensor of %d elements" % (k, n))
            kinds.add(_grad_dtype(s))
            snap_arr[k] = s.data_ptr()
        if len(kinds) > 1:
            raise TypeError("snapshots differ in dtype")
        snap_dt = kinds.pop() if kinds else STAR_DTYPE_F32
    if workspace.dtype != torch.uint8 or not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous uint8 CUDA tensor")
    _check(_lib.star_group_update_host_ex(params.data_ptr(), momentum.data_ptr(), ptrs, W,
                                          STAR_DTYPE_F32 if dt is None else dt, n, _i32(group_offsets),
                                          _i32(group_members), K, (ctypes.c_float * max(K, 1))(*lrs), mu, wd,
                                          snap_arr, snap_dt, sum_order, workspace.data_ptr(), workspace.numel(),
                                          _stream(stream)), "star_group_update_host_ex")


STAR_STATIC_SCRATCH_BYTES = 1 << 20


def star_group_update_multi_noalloc(params: Sequence[torch.Tensor], momentum: Sequence[torch.Tensor],
                                    grads: Sequence[Sequence[Optional[torch.Tensor]]],
                                    group_offsets: Sequence[int], group_members: Sequence[int],
                                    lr: float, mu: float, wd: float, stream=None) -> None:
    """One round over a tensor list for callers that have no way to obtain a
    device workspace (``grads[w][t]`` = worker w's gradient for tensor t).

    The pointer table goes into a fixed array inside the library
    (``STAR_STATIC_SCRATCH_BYTES``) that every call on the device shares; lists
    whose table is larger are rejected with ``STAR_ERR_WORKSPACE_TOO_SMALL``.
    Results equal :func:`star_multi_prepare` + :func:`star_group_update_multi`.
    The caller must serialize calls that could overlap on the GPU, and should
    make the first call on each device outside stream capture."""
    T, W = len(params), len(grads)
    if len(momentum) != T or any(len(g) != T for g in grads):
        raise ValueError("params, momentum and every worker's gradient list need one entry per tensor")
    sizes = [p.numel() for p in params]
    if any(v.numel() != s for v, s in zip(momentum, sizes)):
        raise ValueError("params and momentum differ in size")
    P = (ctypes.c_void_p * max(T, 1))(*[_state(p, "params") if p.numel() else None for p in params])
    V = (ctypes.c_void_p * max(T, 1))(*[_state(v, "momentum") if v.numel() else None for v in momentum])
    G = (ctypes.c_void_p * max(T * W, 1))()
    dt = None
    for w in range(W):
        for t in range(T):
            g = grads[w][t]
            if g is None or sizes[t] == 0:
                continue
            if not g.is_cuda or not g.is_contiguous() or g.numel() != sizes[t]:
                raise ValueError("gradient [%d][%d] must be a contiguous CUDA tensor of %d elements"
                                 % (w, t, sizes[t]))
            d = _grad_dtype(g)
            if dt is not None and d != dt:
                raise TypeError("gradients differ in dtype")
            dt = d
            G[t * W + w] = g.data_ptr()
    S = (ctypes.c_int64 * max(T, 1))(*sizes)
    K = len(group_offsets) - 1 if len(group_offsets) else 0
    _check(_lib.star_group_update_multi_noalloc(T, P, V, G, S, W, STAR_DTYPE_F32 if dt is None else dt,
                                                _i32(group_offsets), _i32(group_members), K, lr, mu, wd,
                                                _stream(stream)), "star_group_update_multi_noalloc")
