"""The benchmark's modes stay runnable: host-side helpers on CPU, one short run of every mode
on the GPU (small workloads, a few steps), each checked for the keys the contract names."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_algorithmic_bytes_and_traffic_record():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2504_04704_b200 import synth
    w = synth.WORKLOADS["llama8b_128k"]
    assert bench.algorithmic_bytes(w, 19968) == 256 * ((131072 + 19968) * 512 + 4 * 19968)      # the headline's 19.82 GB
    assert bench.algorithmic_bytes(w, 19968, elem_bytes=1) == 256 * ((131072 + 19968) * 256 + 4 * 19968)
    assert bench.append_alg_bytes(1792, 512, 128, 0, 128) == 1792 * (1024 * 512 + 640 * 512 + 512)
    # a record is honoured only while the kernel's source files hash to what it names
    rec = json.load(open(bench.TRAFFIC_JSON))
    for key, r in rec.items():
        want = r["traffic_bytes_per_launch"] if r["kernel_source_hash"] == bench.kernel_source_hash(r["source_files"]) else None
        assert bench.captured_traffic(key) == want
    assert bench.captured_traffic("no such workload") is None


def test_gpus_flag_starts_its_own_ranks(monkeypatch):
    """``--gpus N`` outside a torchrun environment re-launches the benchmark under
    ``torch.distributed.run`` with N local ranks on 127.0.0.1 and the same arguments."""
    sys.path.insert(0, ROOT)
    import bench
    seen = {}
    monkeypatch.setattr(bench.subprocess, "call", lambda cmd: seen.setdefault("cmd", cmd) and 0)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7"])
    assert bench.respawn_under_torchrun(4) == 0
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "4", "--steps", "7"]
    assert os.path.basename(cmd[cmd.index("--master-port") + 2]) == "bench.py"


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert lines, out.stdout[-500:]
    return lines


@pytest.mark.gpu
def test_bench_modes_run():
    common = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "roofline", "clocks", "gpu_launches"}
    (line,) = run_bench("--workload", "tiny", "--steps", "3", "--warmup", "3", "--e2e-steps", "1", "--sustained", "0.2",
                       "--cpu-seconds", "1.5")
    assert common <= set(line) and {"e2e", "cpu_baseline", "parity", "single_steps_ms"} <= set(line)
    assert line["parity"]["unexplained_tight"] == 0 and line["parity"]["rows_bit_exact"]
    assert line["e2e"]["h2d_bytes_per_step"] > 0 and line["cpu_baseline"]["single_thread_value"] > 0
    assert {"bound", "achieved", "peak", "unit", "frac", "traffic"} <= set(line["roofline"])
    (line,) = run_bench("--workload", "tiny", "--steps", "3", "--paged", "64", "--storage", "fp16")
    assert line["config"]["paged"] and line["value"] > 0
    (line,) = run_bench("--workload", "tiny", "--steps", "3", "--storage", "fp8", "--variant", "l2norm")
    assert line["value"] > 0
    (line,) = run_bench("--workload", "decode_append", "--append", "--layers", "1", "--steps", "3")
    assert common <= set(line) and line["skip_call_ms"] > 0
    for extra in ([], ["--ragged"]):
        (line,) = run_bench("--workload", "decode_append", "--append", "--loop", "--layers", "1", "--tokens", "600", *extra)
        assert line["calls"]["total"] == 600 and line["calls"]["compressions"] > 0
    cells = run_bench("--workload", "sweep", "--sweep", "--sweep-B", "1", "--steps", "2")
    assert len(cells) == 24 and all(c["config"]["cell"]["B"] == 1 for c in cells)
    (ref,) = run_bench("--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0", "--cpu-seconds", "1")
    assert ref["impl"] == "reference" and ref["cpu_baseline"]["kind"] == "oracle"
