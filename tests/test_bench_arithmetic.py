"""The benchmark's algorithmic-work figures against hand-computed values (the roofline fractions rest on them)."""
import importlib.util
import os

import pytest

from paper_2505_24791_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_sweep_flops_per_sample_match_the_closed_form(bench):
    """F = N (24 d^2 L + 2 d L^2) + 2 L D d + 4 L d D per sample and sweep of one block."""
    want = {"cfg1": 53e6, "cfg2": 6.72e9, "cfg3": 52.7e9, "cfg4": 224.5e9}
    for name, f in want.items():
        cfg = synth.config(name)
        L, D = synth.seq_len(cfg), synth.token_dim(cfg)
        got = bench.sweep_flops_per_row(cfg, L, D) * L
        d, n = cfg["width"], cfg["n_layers"]
        assert got == n * (24 * d * d * L + 2 * d * L * L) + 2 * L * D * d + 4 * L * d * D
        assert abs(got - f) / f < 0.02, (name, got)


def test_sequential_block_bytes(bench):
    # cfg3: 201.5 MB of weights per step (more than L2, so streamed 255 times) and 68.5 GB of K/V reads
    cfg = synth.config("cfg3")
    total, w_blk = bench.seq_block_bytes(cfg, 256, 48, 64)
    assert abs(w_blk - (8 * 12 * 1024 * 1024 + 2 * 48 * 1024) * 2) < 1
    kv = 8 * 64 * (2 * 1024 * 256 * 255 + 4 * 1024 * 255)
    assert abs(total - (w_blk * 255 + kv)) < 1 and 119e9 < total < 121e9
    # cfg2: 25.2 MB of weights stay in L2 (counted once), 17.1 GB of K/V reads
    cfg = synth.config("cfg2")
    total, w_blk = bench.seq_block_bytes(cfg, 256, 12, 64)
    assert 25.1e6 < w_blk < 25.3e6 and 17.0e9 < total - w_blk < 17.3e9
    # cfg4: 1023 steps of 203 MB and 274 GB of K/V reads at batch 16
    cfg = synth.config("cfg4")
    total, w_blk = bench.seq_block_bytes(cfg, 1024, 192, 16)
    assert 480e9 < total < 486e9


def test_class_work_gemm_flops_and_bounds(bench):
    cfg = synth.config("cfg3")
    w = bench.class_work(cfg, 256, 48, 64)
    assert w["gemm_qkv"] == ("tensor", 2.0 * 3 * 1024 * 1024, 0.0)
    assert w["gemm_mlp_up"][1] == w["gemm_mlp_down"][1] == 2.0 * 4096 * 1024
    assert w["attention"][1] == 2.0 * 1024 * 256
    assert w["seq_block"][0] == "hbm" and w["seq_block"][2] == bench.seq_block_bytes(cfg, 256, 48, 64)[0]
    assert bench.class_work(synth.config("cfg1"), 64, 12, 4)["gemm_qkv"][0] == "alu"


def test_reference_arm_prints_the_contract_line_on_cpu():
    """`bench.py --impl reference` needs no GPU: it times the oracle on the host cores and prints one JSON line."""
    import json
    import subprocess
    import sys
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "samples/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["higher_is_better"] is True and line["gpu_launches"] == 0 and "workload" in line["config"]
