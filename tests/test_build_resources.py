"""Register and spill budget of the hot kernels, read from ptxas at build time.
The bandwidth result depends on four resident blocks per SM (<= 64 registers)
without spills; a change that breaks that shows up here, on the CPU."""
import os
import re
import subprocess

from paper_2512_09685_b200 import build as lib_build


def ptxas_report():
    cmd = [lib_build.nvcc(), *lib_build.NVCC_FLAGS, "-I", os.path.join(lib_build.ROOT, "include"), "-I",
           lib_build.CSRC, "-Xptxas", "-v", os.path.join(lib_build.CSRC, "api.cu"), "-o", os.devnull]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    report, current = {}, None
    for line in out.stderr.splitlines():
        m = re.search(r"Compiling entry function '(\S+)'", line)
        if m:
            current = m.group(1)
            report[current] = {"spill": 0, "regs": None}
            continue
        if current is None:
            continue
        m = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", line)
        if m and report[current]["regs"] is None:        # the entry function's own line comes first
            report[current]["spill"] = max(report[current]["spill"], int(m.group(2)) + int(m.group(3)))
        m = re.search(r"Used (\d+) registers", line)
        if m:
            report[current]["regs"] = int(m.group(1))
    return report


def test_hot_kernels_fit_four_blocks_per_sm_without_spills():
    report = ptxas_report()
    hot = [name for name in report
           if re.search(r"star_update_flat_kernelINS_(8GradBF16ELi8|7GradF32ELi4)ELi4E", name)
           or re.search(r"star_update_multi_kernelINS_(8GradBF16ELi8|7GradF32ELi4)ELi4E", name)
           or re.search(r"star_update_flat_snapshot_kernelINS_(8GradBF16ELi8|7GradF32ELi4)ELi4ELi0E", name)]
    assert len(hot) == 6, sorted(report)
    for name in hot:
        assert report[name]["regs"] <= 64, (name, report[name])
        assert report[name]["spill"] == 0, (name, report[name])


def test_extended_and_reduce_kernels_do_not_spill():
    """The snapshot / tree-order kernels of the flat entry point and the group
    reduce kernels, every instantiation: no spills; the variants for groups of up
    to 4 members keep the 64-register budget of the linear kernels, the larger
    tree variants are compiled for two blocks per SM (<= 128 registers).  The
    tensor-list variants may save a few registers around their out-of-line
    element path, nothing more."""
    report = ptxas_report()
    flat = {n: r for n, r in report.items()
            if "star_update_flat_snapshot_kernel" in n or "star_group_reduce_kernel" in n}
    assert len(flat) == 2 * 2 * 4 + 2 * 2 * 4, sorted(flat)      # dtype x (vector, element) x tree span, two kernels
    for name, r in flat.items():
        tree = int(re.search(r"ELi(\d+)EEEv", name).group(1))
        assert r["spill"] == 0, (name, r)
        assert r["regs"] <= (64 if tree <= 4 else 128), (name, r)
    lists = {n: r for n, r in report.items() if "star_update_multi_ex_kernel" in n}
    assert len(lists) == 8, sorted(lists)
    for name, r in lists.items():
        assert r["spill"] <= 128, (name, r)
