"""The benchmark's CPU-checker arm runs without a GPU and prints one well-formed JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-500:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "weights_quantized_per_s" and d["unit"] == "weights/s"
    assert d["value"] > 0 and d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True
    assert d["config"]["workload"] == "large_layer"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--gpus", "2"], capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_algorithmic_bytes_of_the_bench_workload():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2202_07471_b200 import workloads as W
    wl = W.WORKLOADS[bench.WORKLOAD]
    # 3x3 layers: 4 B read + 1 B code + 4/9 B kernel sum per weight + 8 B per channel
    assert bench.algorithmic_bytes(wl.shapes) == 8 * (2048 * 2048 * 9 * 5 + 2048 * 2048 * 4 + 2048 * 8)


def test_parity_checker_of_the_bench_counts_corrupted_channels():
    """bench.py compares the timed outputs with the checker slab by slab on several threads; a
    corrupted code, scale or error sum must be counted once per channel, clean outputs not at all."""
    sys.path.insert(0, ROOT)
    import numpy as np
    import bench
    import oracle
    from paper_2202_07471_b200 import workloads as W
    ws = [W.random_layer((70, 12, 3, 3), seed=1), W.random_layer((9, 40, 1, 1), seed=2)]
    good = []
    for w in ws:
        r = oracle.quantize_layer(w, bits=4)
        good.append((r.codes.copy(), r.scales.copy(), r.kernel_err.copy(), r.channel_err.copy()))
    bad = [tuple(a.copy() for a in o) for o in good]
    bad[0][0][3, 2, 1, 1] += 1          # one code of channel 3
    bad[0][2][65, 7] = 0.25             # one kernel sum of channel 65 (second slab)
    bad[1][1][8] *= 2.0                 # one scale
    bad[1][3][8] = 0.125                # and the channel sum of the same channel: still one channel
    ch, mism, dt = bench.oracle_check_all(ws, [good, bad], 4, oracle.MODE_EKC, threads=3, slab=64)
    assert ch == 79 and mism == [0, 3] and dt > 0
