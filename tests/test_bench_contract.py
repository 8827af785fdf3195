"""bench.py contract checks that need no GPU: the reference arm (the CPU oracle timed on the
host cores) prints one JSON line with the agreed keys, and ranks other than 0 stay silent."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra_env=None, *args):
    env = dict(os.environ)
    env.update(extra_env or {})
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", *args],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr
    return out.stdout.strip()


def test_reference_arm_prints_one_json_line():
    text = _run(None, "--steps", "2", "--warmup", "1", "--workload", "resnet20")
    lines = [l for l in text.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "gossip_rounds_per_s" and d["unit"] == "rounds/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["dtype"] == "f32"
    assert d["steps"] == 2 and d["warmup"] == 1 and d["value"] > 0 and d["ms_per_step"] > 0
    assert "workload" in d["config"] and "model" not in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == 1 and cb["value"] == d["value"] and cb["sample"]
    e = d["e2e"]
    assert e["value"] == d["value"] and e["unit"] == d["unit"]
    assert e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0


def test_reference_arm_other_ranks_print_nothing():
    assert _run({"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"}, "--steps", "1", "--warmup", "1") == ""


def test_reference_arm_runs_the_whole_default_workload():
    # the default workload is timed at full width by the oracle (no scaling), larger ones on a
    # stated column sample
    sys.path.insert(0, ROOT)
    import bench
    from paper_2002_09692_b200 import synth
    cols, frac, sample = bench.oracle_sample(synth.WORKLOADS["vgg16"])
    assert cols == synth.WORKLOADS["vgg16"].N and frac == 1.0 and "nothing scaled" in sample
    cols, frac, sample = bench.oracle_sample(synth.WORKLOADS["gpt2s"])
    assert cols == bench.ORACLE_MAX_COLUMNS < synth.WORKLOADS["gpt2s"].N and "scaled by" in sample
    assert frac == cols / synth.WORKLOADS["gpt2s"].N
    # at N ranks the job is N column shards; the oracle runs one and says what fraction that is
    cols, frac, sample = bench.oracle_sample(synth.WORKLOADS["vgg16"], 4)
    assert cols == synth.WORKLOADS["vgg16"].N and frac == 0.25 and "4 shard(s)" in sample
    assert bench.workload_config(synth.WORKLOADS["vgg16"], 0.01, 4)["sharding"].startswith("column shards")
    small = bench.workload_config(synth.WORKLOADS["resnet20"], 0.01, 1)
    assert "L2-resident" in small["l2"]
    big = bench.workload_config(synth.WORKLOADS["vgg16"], 0.01, 1)
    assert "far larger" in big["l2"]


def test_recorded_dram_traffic_is_tied_to_the_kernel_sources():
    # the ncu figure is reported only for the workload it was captured on and only while the
    # kernel's sources are the ones that were captured
    sys.path.insert(0, ROOT)
    import bench
    assert bench.ncu_traffic("resnet20", 0.01) is None
    assert bench.ncu_traffic("vgg16", 0.001) is None
    got = bench.ncu_traffic("vgg16", 0.01)
    if bench.NCU_TRAFFIC["kernel_sources_sha256"] == bench.kernel_sources_hash():
        assert got == bench.NCU_TRAFFIC["bytes_per_launch"]
        algorithmic = 12 * 32 * 14_728_266
        assert 0.9 * algorithmic < got < 1.1 * algorithmic
    else:
        assert got is None
