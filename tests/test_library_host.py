"""Host-side checks of the CUDA library that need no GPU: it loads, exports
every symbol the header declares, its schedule encoders agree with the
schedule oracle, and argument errors are reported before any CUDA call."""
import ctypes
import itertools
import os
import random
import re

import pytest

from oracle import schedule as S
from paper_2512_09685_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "star.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(star_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert "star_group_update" in names and "star_group_update_multi" in names
    assert len(names) >= 11
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_mirrors_every_entry_point():
    for name in declared_symbols():
        assert callable(getattr(B, name)), name


def test_status_strings():
    assert B.star_status_string(0) == "STAR_OK"
    assert B.star_status_string(3) == "STAR_ERR_BAD_SCHEDULE"
    assert B.star_status_string(6) == "STAR_ERR_CUDA"
    assert B.star_status_string(99) == "STAR_ERR_UNKNOWN"


def test_static_x_matches_oracle_on_every_small_case():
    rng = random.Random(0)
    for W in range(0, 9):
        for x in range(1, W + 2):
            for sort_members in (False, True):
                assert B.star_schedule_static_x(None, W, x, sort_members) == \
                    tuple(S.static_x(None, W, x, sort_members))
                for _ in range(4):
                    k = rng.randint(0, W)
                    order = rng.sample(range(W), k)
                    assert B.star_schedule_static_x(order, W, x, sort_members) == \
                        tuple(S.static_x(order, W, x, sort_members))


def test_static_x_modes_of_the_paper():
    assert B.star_schedule_static_x(None, 8, 8) == ([0, 8], list(range(8)))           # SSGD
    assert B.star_schedule_static_x([2, 0, 1], 3, 1) == ([0, 1, 2, 3], [2, 0, 1])     # ASGD
    for x in (1, 2, 4, 8):                                                            # Section IV-B, N = 8
        off, mem = B.star_schedule_static_x(None, 8, x)
        assert len(off) - 1 == 8 // x


def test_static_x_rejects_bad_input():
    for order, W, x in (([0, 0], 4, 1), ([4], 4, 1), ([-1], 4, 1), ([0], 4, 0)):
        with pytest.raises(B.StarError):
            B.star_schedule_static_x(order, W, x)
    with pytest.raises(B.StarError) as e:
        B.star_schedule_static_x(None, 65, 1)
    assert e.value.status == B.STAR_ERR_UNSUPPORTED


def test_from_labels_matches_oracle_exhaustively():
    for W in range(0, 6):
        for labels in itertools.product([-1, 0, 1, 5], repeat=W):
            assert B.star_schedule_from_labels(labels) == tuple(S.from_labels(labels))
    with pytest.raises(B.StarError):
        B.star_schedule_from_labels([0, -2])


def test_dynamic_x_matches_oracle():
    rng = random.Random(1)
    for _ in range(300):
        W = rng.randint(1, 12)
        times = [rng.choice([0.1, 0.2, 0.35, 0.5, 0.8]) + rng.random() * rng.choice([0, 0.01])
                 for _ in range(W)]
        clusters = [rng.randint(-1, 3) for _ in range(W)]
        got = B.star_schedule_dynamic_x(times, clusters)
        assert got == tuple(S.dynamic_x(times, clusters))
        assert B.star_schedule_validate(got[0], got[1], len(got[0]) - 1, W) == B.STAR_OK
    with pytest.raises(B.StarError):
        B.star_schedule_dynamic_x([float("nan")], [0])


def test_validate_matches_oracle():
    rng = random.Random(2)
    cases = [([0, 2, 4], [0, 1, 2, 3], 2, 4), ([0], [], 0, 4), ([0, 1], [2], 1, 4),
             ([0, 0, 2], [0, 1], 2, 4), ([0, 2], [1, 1], 1, 4), ([0, 1, 2], [1, 1], 2, 4),
             ([0, 1], [4], 1, 4), ([1, 2], [0, 1], 1, 4), ([0, 2, 1], [0, 1], 2, 4),
             ([0, 1], [-1], 1, 4)]
    for _ in range(500):
        W = rng.randint(1, 6)
        K = rng.randint(1, 4)
        off = [0]
        for _ in range(K):
            off.append(off[-1] + rng.randint(0, 3))
        mem = [rng.randint(-1, W) for _ in range(max(off[-1], 1))]
        cases.append((off, mem, K, W))
    n_ok = 0
    for off, mem, K, W in cases:
        ok = B.star_schedule_validate(off, mem, K, W) == B.STAR_OK
        assert ok == S.is_valid(off, mem, K, W), (off, mem, K, W)
        n_ok += ok
    assert n_ok >= 3
    assert B.star_schedule_validate([0, 1], [0], 1, 65) == B.STAR_ERR_UNSUPPORTED
    assert B.star_schedule_validate([0, 1], [0], -1, 4) == B.STAR_ERR_INVALID_ARG


def test_compute_entry_points_reject_bad_arguments_before_any_cuda_call():
    lib = B._lib
    off = (ctypes.c_int32 * 3)(0, 0, 2)          # empty first group
    mem = (ctypes.c_int32 * 2)(0, 1)
    ptrs = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    fake = ctypes.c_void_p(0x10000)
    assert lib.star_group_update(fake, fake, ptrs, 2, 1, 16, off, mem, 2, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_BAD_SCHEDULE
    good = (ctypes.c_int32 * 2)(0, 2)
    assert lib.star_group_update(fake, fake, ptrs, 2, 1, -1, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_INVALID_ARG
    assert lib.star_group_update(fake, fake, ptrs, 2, 7, 16, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_INVALID_ARG
    assert lib.star_group_update(fake, fake, ptrs, 65, 1, 16, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_UNSUPPORTED
    assert lib.star_group_update(None, fake, ptrs, 2, 1, 16, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_NULL_POINTER
    # params and momentum overlap
    assert lib.star_group_update(fake, fake, ptrs, 2, 1, 16, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_INVALID_ARG
    # a scheduled worker without a buffer
    holes = (ctypes.c_void_p * 2)(0x1000, None)
    other = ctypes.c_void_p(0x20000)
    assert lib.star_group_update(fake, other, holes, 2, 1, 16, good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_NULL_POINTER
    # no-ops succeed without touching anything
    assert lib.star_group_update(None, None, None, 2, 1, 0, good, mem, 1, 0.1, 0.9, 0.0, None) == 0
    assert lib.star_group_update(None, None, None, 2, 1, 16, good, mem, 0, 0.1, 0.9, 0.0, None) == 0
    plan = B.star_multi_plan_t()
    assert lib.star_group_update_multi(ctypes.byref(plan), good, mem, 1, 0.1, 0.9, 0.0, None) \
        == B.STAR_ERR_INVALID_ARG
    out = ctypes.c_size_t(0)
    sizes = (ctypes.c_int64 * 2)(5, -1)
    assert lib.star_multi_workspace_bytes(2, sizes, 4, ctypes.byref(out)) == B.STAR_ERR_INVALID_ARG
    sizes = (ctypes.c_int64 * 2)(5, 5000)
    assert lib.star_multi_workspace_bytes(2, sizes, 4, ctypes.byref(out)) == 0 and out.value >= 256


def test_without_a_gpu_the_compute_path_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    lib = B._lib
    good = (ctypes.c_int32 * 2)(0, 1)
    mem = (ctypes.c_int32 * 1)(0)
    ptrs = (ctypes.c_void_p * 1)(0x100000)
    rc = lib.star_group_update(ctypes.c_void_p(0x200000), ctypes.c_void_p(0x300000), ptrs, 1, 1, 64,
                               good, mem, 1, 0.1, 0.9, 0.0, None)
    assert rc == B.STAR_ERR_CUDA and B.star_last_cuda_error() != 0
