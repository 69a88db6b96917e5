"""The benchmark's contract that can be checked without a GPU: the reference arm (the CPU
oracle on a bounded sample) prints one JSON line with the agreed keys, and a plain
`--gpus N` start would re-execute itself under torch.distributed.run."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--config", "config0", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "packed_attn_fwd_bwd_useful_tflops"
    assert d["unit"] == "TFLOP/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["steps"] == 2 and d["warmup"] == 1 and d["value"] > 0 and d["ms_per_step"] > 0
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and d["gpu_launches"] == 0
    assert set(d["config"]) == {"workload", "step", "l2", "per_gpu_batch"}     # the GPU arm's keys
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] and d["e2e"]["value"] == d["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0


def test_headline_and_target_workloads_are_the_nine_full_size_ones():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.TARGET_CONFIGS == ["config1", "config2", "config3"] + [f"config4:{i}" for i in range(6)]
    assert bench.HEADLINE in bench.TARGET_CONFIGS
    flops = {n: sum(bench.get_workload(n).useful_flops()) for n in bench.TARGET_CONFIGS}
    assert max(flops, key=flops.get) == bench.HEADLINE          # the largest workload is the headline
    # every workload has a tracked DRAM-traffic figure for the roofline
    for n in bench.TARGET_CONFIGS:
        b, how = bench.dram_traffic(n)
        assert b and b > 1e8 and "ncu" in how
