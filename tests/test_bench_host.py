"""Host logic of bench.py that needs no GPU: how the CPU oracle's phase times become tokens/s/layer, what the
config of a line says, and that `--gpus N` outside a launcher starts N ranks itself of which rank 0 alone prints
the one JSON line (checked with the reference arm, which runs on the host cores)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2404_01365_b200 import synth  # noqa: E402


def test_phase_times_of_a_sample_scale_to_the_whole_path():
    w = synth.WORKLOADS["llama2_13b"]                      # S = 2048, T = 256
    ph = {"prefill": 1.0, "select": 0.01, "compact": 0.09, "decode": 0.8, "S": 1024, "T": 16}
    # whole prompt = 2 s, all decode steps = 12.8 s: 256 tokens in 14.9 s
    assert bench.compose_tokens_per_s(w, ph) == pytest.approx(256 / (2.0 + 0.01 + 0.09 + 12.8))
    full = dict(ph, S=2048, T=256)
    assert bench.compose_tokens_per_s(w, full) == pytest.approx(256 / 1.9)


def test_config_names_the_workload_and_its_footprint():
    w = synth.WORKLOADS["llama2_13b"]
    cfg = bench.workload_config(w, w.L, w.B, 0.5, 1, False, True)
    assert cfg["workload"].startswith("llama2_13b") and cfg["B"] == 8 and cfg["k"] == 6912 and cfg["L"] == 40
    assert "17.0 GB dense" in cfg["l2"] and "67.9 GB compact" in cfg["l2"]
    assert "model" not in cfg
    assert bench.HEADLINE == "llama2_13b"                   # the largest single-GPU configuration is the default


def test_gpus_n_starts_n_ranks_and_rank_zero_prints_one_line():
    env = dict(os.environ, OMP_NUM_THREADS="1")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_swiglu_f32",
                        "--gpus", "2", "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["steps"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
