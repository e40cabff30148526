"""Host-side pieces of bench.py that need no GPU: the DRAM-traffic figures tied to the kernel sources, the config
shared by both arms, the reference arm's line."""
import hashlib
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_traffic_is_read_from_profiles_and_dropped_when_the_kernel_source_changes(tmp_path, monkeypatch):
    (tmp_path / "profiles").mkdir()
    (tmp_path / "k.cu").write_text("__global__ void k() {}\n")
    sha = hashlib.sha256((tmp_path / "k.cu").read_bytes()).hexdigest()
    (tmp_path / "profiles" / "k_w.txt").write_text(
        "some kernel on some workload\n"
        f"# bench-traffic: workload=w kernel=main source=k.cu sha256={sha} dram_bytes_per_launch=123000000\n"
        f"# bench-traffic: workload=w kernel=second source=k.cu sha256={sha} dram_bytes_per_launch=5\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.profiled_traffic("w") == 123e6 and bench.profiled_traffic("w", "second") == 5.0
    assert bench.profiled_traffic("other") is None
    (tmp_path / "k.cu").write_text("__global__ void k() { /* changed */ }\n")
    assert bench.profiled_traffic("w") is None               # the counters describe another program now


def test_committed_traffic_lines_name_existing_sources():
    for fn in os.listdir(os.path.join(ROOT, "profiles")):
        for line in open(os.path.join(ROOT, "profiles", fn)):
            if line.startswith("# bench-traffic:"):
                kv = dict(t.split("=", 1) for t in line.split()[2:])
                assert os.path.isfile(os.path.join(ROOT, kv["source"])), (fn, kv["source"])
                assert float(kv["dram_bytes_per_launch"]) > 0 and kv["workload"] in bench.FACTORIES


def test_both_arms_describe_the_workload_with_the_same_config():
    from paper_2406_07368_b200 import workloads as wl
    for name in bench.FACTORIES:
        W = wl.WORKLOADS[name]()
        a, b = bench.base_config(W), bench.base_config(W)
        assert a == b and a["workload"] == name and "l2" in a and a["parallelism"] == "single GPU"
    assert bench.base_config(wl.llama7b_prefill(), world=8)["parallelism"] == "replicas only"


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "tree_verify", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-500:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "config", "cpu_baseline", "e2e"):
        assert key in line
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
