"""Host-side checks of bench.py's output contract (no GPU): the reference arm prints one JSON line with the keys the
harness reads, and the arithmetic helpers agree with figures worked out by hand."""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, cwd=ROOT,
                         env={**os.environ, "RANK": "0", "WORLD_SIZE": "1"})
    assert out.returncode == 0, out.stderr[-2000:]
    line = out.stdout.strip().splitlines()[-1]
    d = json.loads(line)
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 1 and d["n_gpus"] == 1 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "cfg1" and d["gpu_launches"] == 0
    # both arms describe the workload with the same object
    import bench
    from paper_2608_01662_b200.configs import CONFIGS
    assert d["config"] == bench.config_dict(CONFIGS["cfg1"], CONFIGS["cfg1"].L)


def test_reference_arm_is_silent_on_other_ranks():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "cfg1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, cwd=ROOT,
                         env={**os.environ, "RANK": "1", "WORLD_SIZE": "2"})
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_algorithmic_work_of_the_attention_launch():
    import bench
    from paper_2608_01662_b200.configs import CONFIGS
    cfg = CONFIGS["cfg3"]
    # a late query attends S + Ksp + W = 4 + 2048 + 1024 rows; each costs 2 * H * (d_qk + d_v) flop
    pos = np.array([100000], dtype=np.int64)
    assert bench.attn_flops_per_launch(cfg, pos) == 3076 * 2 * 64 * (576 + 512)
    # an early query sees only [0, t]
    assert bench.attn_flops_per_launch(cfg, np.array([9], dtype=np.int64)) == 10 * 2 * 64 * (576 + 512)
    dec = CONFIGS["cfg4"]
    one = bench.attn_bytes_per_launch(dec, np.array([50000], dtype=np.int64))
    assert one == (4 + 2048 + 256) * 576 * 2 + 64 * 576 * 2 + 64 * 512 * 2   # rows + q + out of one sequence
