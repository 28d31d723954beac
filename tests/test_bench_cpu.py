"""Host-side checks of bench.py that need no GPU: the reference arm (the fp64 oracle timed on the host cores)
prints one JSON line with the keys the benchmark contract names, the flop count of a layer matches the formula
counted by hand, and the comparison layers count fewer flops than L4Q."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2402_04902_b200 import synth  # noqa: E402


def test_layer_flops_formula():
    cfg = synth.CONFIG2                                  # 4096 x 4096, 4096 tokens, rank 16
    M, o, i, r = 4096, 4096, 4096, 16
    assert bench.layer_flops(cfg) == 6.0 * M * o * i + 8.0 * o * i * r
    assert bench.layer_flops(cfg, layer="lora") == 4.0 * M * o * i + 6.0 * M * r * (i + o)
    assert bench.layer_flops(cfg, layer="lora") < bench.layer_flops(cfg, layer="qat_lora") < bench.layer_flops(cfg) * 1.01
    assert set(bench.workloads()) >= {"llama7b_mlp", "llama7b_attn_proj", "llama7b_mlp_3bit_r64", "mistral7b_block"}


@pytest.mark.timeout(600)
def test_reference_arm_prints_one_contract_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "llama7b_attn_proj", "--steps", "1", "--warmup", "0"], capture_output=True, text=True,
                         env=env, timeout=580)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == bench.METRIC and j["unit"] == bench.UNIT
    assert j["higher_is_better"] is True and j["value"] > 0 and j["dtype"] == "f64"
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["cores"] >= 1
    assert j["e2e"]["value"] == j["value"] and j["e2e"]["h2d_bytes_per_step"] == 0
    assert j["config"]["workload"] == "llama7b_attn_proj"


def test_other_ranks_of_the_reference_arm_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, env=env, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
