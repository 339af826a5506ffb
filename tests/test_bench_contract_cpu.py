"""bench.py's reference arm (the CPU oracle) prints the agreed JSON line; the CUDA arm refuses to run without a GPU."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True, text=True,
                          timeout=600)


def test_reference_arm_prints_the_contract_line():
    p = _run(["--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0"])
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in line, key
    assert line["impl"] == "reference" and line["n_gpus"] == 1 and line["steps"] == 1
    assert line["unit"] == "tokens/s" and line["higher_is_better"] is True and line["vs_baseline"] is None
    assert line["config"]["workload"] == "tiny"
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == line["value"]
    e2e = line["e2e"]
    assert e2e["value"] == line["value"] and e2e["h2d_bytes_per_step"] == 0 and e2e["d2h_bytes_per_step"] == 0
    assert line["value"] > 0 and line["ms_per_step"] > 0


@pytest.mark.skipif(torch.cuda.is_available(), reason="needs a machine without a GPU")
def test_cuda_arm_fails_loudly_without_a_gpu():
    p = _run(["--workload", "tiny", "--steps", "1"])
    assert p.returncode != 0
    assert "CUDA" in (p.stderr + p.stdout)


@pytest.mark.skipif(torch.cuda.is_available(), reason="needs a machine without a GPU")
def test_gpus_flag_starts_ranks_itself_and_refuses_without_enough_devices():
    """`--gpus 2` outside a torchrun environment takes the self-spawn path; with fewer than 2 devices it exits non-zero
    with a message instead of running one rank and calling it two."""
    p = _run(["--gpus", "2", "--workload", "tiny", "--steps", "1"])
    assert p.returncode != 0
    assert "needs 2 CUDA devices" in p.stderr


def test_reference_arm_under_two_ranks_prints_one_line_from_rank_zero():
    """Launched the way the scaling run launches it (torch.distributed.run, 2 processes, 127.0.0.1): rank 0 alone runs
    the oracle and prints the line with n_gpus = 2; rank 1 exits 0 without output."""
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "tiny",
           "--steps", "1", "--warmup", "0"]
    p = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["cpu_baseline"]["cores"] == len(os.sched_getaffinity(0))


def test_world_size_must_match_the_gpus_flag():
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "4", "--workload", "tiny"],
                       cwd=ROOT, capture_output=True, text=True, timeout=120, env=env)
    assert p.returncode != 0 and "WORLD_SIZE" in (p.stderr + p.stdout)


def test_recorded_traffic_counts_only_for_the_recorded_kernel_source(tmp_path, monkeypatch):
    """The roofline's `traffic` figure comes from a record keyed on the hash of the kernel's source file: a record made
    for other source text is ignored (null) rather than reported stale."""
    import hashlib
    sys.path.insert(0, ROOT)
    import bench
    digest = bench.attention_source_digest()
    rec = tmp_path / "traffic.txt"
    rec.write_text(f"# comment\nllama8b_32k {'0' * 64} 111\nllama8b_32k {digest} 4318434000\n")
    monkeypatch.setattr(bench, "TRAFFIC_RECORD", str(rec))
    assert bench.recorded_traffic("llama8b_32k") == 4318434000
    assert bench.recorded_traffic("qwen_vl_16k") is None
    rec.write_text(f"llama8b_32k {'0' * 64} 111\n")
    assert bench.recorded_traffic("llama8b_32k") is None
