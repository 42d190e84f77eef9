"""Do the pins have teeth?  Plant one plausible mistake at a time in a COPY of
the oracle's C source (on the CPU, in a temporary directory), build it, and
require that the pins reject it: the hand-worked example, the exact-rational
brute force, or the comparison with PyTorch's SGD."""
import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import star_oracle as O
from tests import exact_arith as X
from tests.test_oracle_pins import (_read_golden, all_schedules, bf16_bits, bf16_snapshot_probe_values,
                                    bf16_values, csr)

SRC = os.path.join(os.path.dirname(O.__file__), "star_oracle.c")

MUTANTS = {
    "sum_instead_of_mean": ("const float gbar = s / (float)(last - first);", "const float gbar = s;"),
    "reciprocal_multiply": ("const float gbar = s / (float)(last - first);",
                            "const float gbar = s * (1.0f / (float)(last - first));"),
    "weight_decay_dropped": ("const float d = fmaf(wd, p, gbar);", "const float d = gbar;"),
    "weight_decay_on_momentum": ("const float d = fmaf(wd, p, gbar);", "const float d = fmaf(wd, v, gbar);"),
    "ascent_instead_of_descent": ("p = fmaf(-lrs[k], v, p);", "p = fmaf(lrs[k], v, p);"),
    "step_uses_gradient_not_momentum": ("p = fmaf(-lrs[k], v, p);", "p = fmaf(-lrs[k], d, p);"),
    "momentum_operands_swapped": ("v = fmaf(mu, v, d);", "v = fmaf(mu, d, v);"),
    "momentum_not_fused": ("v = fmaf(mu, v, d);", "v = mu * v + d;"),
    "update_not_fused": ("p = fmaf(-lrs[k], v, p);", "p = p - lrs[k] * v;"),
    "first_group_learning_rate_everywhere": ("p = fmaf(-lrs[k], v, p);", "p = fmaf(-lrs[0], v, p);"),
    "groups_in_reverse_order": ("for (int k = 0; k < n_groups; ++k) {\n            const int first",
                                "for (int k = n_groups - 1; k >= 0; --k) {\n            const int first"),
    "member_index_instead_of_member": ("s = s + grad_at(grads[group_members[j]], grad_dtype, i);",
                                       "s = s + grad_at(grads[j], grad_dtype, i);"),
    "last_member_skipped": ("for (int j = first + 1; j < last; ++j)\n                    s = s + grad_at",
                            "for (int j = first + 1; j < last - 1; ++j)\n                    s = s + grad_at"),
    "tree_split_not_a_power_of_two": ("while (2 * h < count)\n        h *= 2;", "h = count / 2;"),
    "tree_drops_the_right_half": ("tree_sum_f32(grads, dtype, members + h, count - h, i);",
                                  "tree_sum_f32(grads, dtype, members + h, 1, i);"),
    "bf16_widened_wrongly": ("uint32_t u = (uint32_t)h << 16;", "uint32_t u = (uint32_t)h << 15;"),
    "snapshot_of_the_old_state": ("((float *)snapshots[k])[i] = p;", "((float *)snapshots[k])[i] = params[i];"),
    "bf16_snapshot_truncated_not_rounded": ("u += 0x7fffu + ((u >> 16) & 1u);", "u += 0u;"),
    "bf16_snapshot_ties_away": ("u += 0x7fffu + ((u >> 16) & 1u);", "u += 0x8000u;"),
    "dampened_momentum": ("v = fmaf(mu, v, d);", "v = fmaf(mu, v, (1.0f - mu) * d);"),
}


def build_mutant(tmp_path, name):
    text = open(SRC).read()
    old, new = MUTANTS[name]
    assert text.count(old) >= 1, "mutation site not found: " + name
    path = tmp_path / (name + ".c")
    path.write_text(text.replace(old, new, 1))        # first occurrence = the f32 function
    lib_path = str(tmp_path / (name + ".so"))
    subprocess.check_call(["gcc", *[f for f in O.CFLAGS if f not in ("-Wall", "-Wextra")], "-o", lib_path,
                           str(path), "-lm"])
    lib = ctypes.CDLL(lib_path)
    common = [ctypes.c_void_p] * 3 + [ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
    lib.oracle_group_update_f32.argtypes = common + [ctypes.c_float, ctypes.c_float, ctypes.c_void_p, ctypes.c_int,
                                                     ctypes.c_int]
    lib.oracle_group_update_f32.restype = ctypes.c_int

    def update(p, v, grads, off, mem, lrs, mu, wd, snapshots=None, sum_order="linear"):
        O._call(lib.oracle_group_update_f32, np.float32, p, v, grads, off, mem, lrs,
                float(np.float32(mu)), float(np.float32(wd)), snapshots, sum_order)
    return update


def pins_accept(update) -> bool:
    """A reduced set of the pins of test_oracle_pins.py, as one predicate."""
    # hand-worked example (fp32 and bf16 inputs), with the trail of intermediate p
    scal, cases = _read_golden()
    for as_bf16 in (False, True):
        for _, groups, p_want, v_want, trail in cases:
            p = np.full(3, scal["p0"][0], np.float32)
            v = np.full(3, scal["v0"][0], np.float32)
            gs = [np.full(3, g, np.float32) for g in scal["g"]]
            if as_bf16:
                gs = [bf16_bits(g) for g in gs]
            off, mem = csr(groups)
            snaps = [np.zeros(3, np.float32) for _ in groups]
            update(p, v, gs, off, mem, scal["lr"][0], scal["mu"][0], scal["wd"][0], snapshots=snaps)
            if not (np.all(p == p_want) and np.all(v == v_want)):
                return False
            if any(not np.all(s == t) for s, t in zip(snaps, trail)):
                return False
    # exact-rational brute force on every 5th schedule, per-group learning rates
    rng = np.random.default_rng(3)
    W, n = 4, 5
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    v0 = rng.normal(0, 0.02, n).astype(np.float32)
    g32 = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(W)]
    bits = [bf16_bits(g) for g in g32]
    for grads, vals in ((g32, g32), (bits, [bf16_values(b) for b in bits])):
        for index, groups in enumerate(all_schedules(W)):
            if index % 5:
                continue
            lrs = [np.float32(0.1 * (1 + 0.5 * k)) for k in range(len(groups))]
            p, v = p0.copy(), v0.copy()
            off, mem = csr(groups)
            update(p, v, grads, off, mem, lrs, np.float32(0.9), np.float32(1e-3))
            for i in range(n):
                pe, ve, _ = X.grouped_update_exact32(
                    X.to_fraction(p0[i]), X.to_fraction(v0[i]), [X.to_fraction(g[i]) for g in vals],
                    groups, [X.to_fraction(l) for l in lrs], X.to_fraction(np.float32(0.9)),
                    X.to_fraction(np.float32(1e-3)))
                if X.to_fraction(p[i]) != pe or X.to_fraction(v[i]) != ve:
                    return False
    # tree order: exact pairwise sums for group sizes 3, 5, 6, 7
    for size in (3, 5, 6, 7):
        gs = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(size)]
        p, v = p0.copy(), v0.copy()
        update(p, v, gs, [0, size], list(range(size)), np.float32(0.1), np.float32(0.9), np.float32(1e-3),
               sum_order="tree")
        for i in range(n):
            pe, ve, _ = X.grouped_update_exact32(
                X.to_fraction(p0[i]), X.to_fraction(v0[i]), [X.to_fraction(g[i]) for g in gs],
                [list(range(size))], [X.to_fraction(np.float32(0.1))], X.to_fraction(np.float32(0.9)),
                X.to_fraction(np.float32(1e-3)), tree=True)
            if X.to_fraction(p[i]) != pe or X.to_fraction(v[i]) != ve:
                return False
    # bf16 snapshots against PyTorch's cast (parameters held still by zero gradients)
    x = bf16_snapshot_probe_values()
    snap = np.zeros(x.size, np.uint16)
    update(x.copy(), np.zeros(x.size, np.float32), [np.zeros(x.size, np.float32)], [0, 1], [0], 0.1, 0.9, 0.0,
           snapshots=[snap])
    if not np.array_equal(snap, torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)):
        return False
    # PyTorch's SGD, two rounds of three groups (fp32 state: agreement to rounding)
    n = 64
    p0 = rng.normal(0, 0.05, n).astype(np.float32)
    gs = [rng.normal(0, 0.01, n).astype(np.float32) for _ in range(6)]
    groups = [[0, 1, 2], [3], [4, 5]]
    param = torch.nn.Parameter(torch.from_numpy(p0.astype(np.float64)))
    opt = torch.optim.SGD([param], lr=0.1, momentum=0.9, weight_decay=1e-2)
    p, v = p0.copy(), np.zeros(n, np.float32)
    off, mem = csr(groups)
    for _ in range(2):
        for grp in groups:
            param.grad = torch.from_numpy(sum(gs[w].astype(np.float64) for w in grp) / len(grp))
            opt.step()
        update(p, v, gs, off, mem, 0.1, 0.9, 1e-2)
    return bool(np.allclose(p, param.detach().numpy(), rtol=1e-5, atol=1e-7))


def test_the_unmutated_oracle_passes_the_reduced_pins():
    assert pins_accept(O.group_update_f32)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_reject_mutant(tmp_path, name):
    assert not pins_accept(build_mutant(tmp_path, name)), "the pins did not notice: " + name
