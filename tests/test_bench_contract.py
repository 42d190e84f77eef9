"""The benchmark's reference arm runs on the CPU: check the JSON line it prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "3", "--warmup", "1"], capture_output=True, text=True, timeout=600,
                         cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True
    assert d["steps"] == 3 and d["warmup"] == 1 and d["value"] > 0 and d["ms_per_step"] > 0
    assert d["config"]["workload"] == "cfg4_gpt2_medium" and d["vs_baseline"] is None
    sys.path.insert(0, ROOT)
    import bench
    from paper_2512_09685_b200 import workloads as WL
    assert d["config"] == bench.config_for(WL.BY_NAME["cfg4_gpt2_medium"], 1)     # what the GPU arm prints too
    assert d["config"]["bytes_per_step"] == 354_823_168 * (16 * 2 + 16)
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_other_ranks_of_the_reference_arm_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "3", "--warmup", "1"], capture_output=True, text=True, timeout=120,
                         cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_product_code_never_touches_the_oracle():
    """Only tests, the smoke check and the benchmark's CPU legs may use oracle/."""
    pkg = os.path.join(ROOT, "paper_2512_09685_b200")
    for folder, _, files in os.walk(pkg):
        for name in files:
            if name.endswith((".py", ".cu", ".cc", ".cuh", ".h")):
                text = open(os.path.join(folder, name)).read()
                for needle in ("import oracle", "from oracle", "oracle/", "star_oracle", "oracle."):
                    assert needle not in text, (os.path.join(folder, name), needle)
    for name in os.listdir(os.path.join(ROOT, "oracle")):
        if name.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", name)).read()
            assert "paper_2512_09685_b200" not in text and "star.h" not in text, name
