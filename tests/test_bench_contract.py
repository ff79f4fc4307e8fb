"""The bench program's contract, as far as it can be checked without a GPU: the reference arm (the oracle on the
host cores) prints one JSON line with the agreed keys for a forward workload and for the quantizer workload, and the
accounting helpers agree with hand-evaluated byte and FLOP counts."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KEYS = {"impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
        "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"}


def run_reference(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0", *args],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


@pytest.mark.parametrize("workload,metric,unit", [("decode_qproj", "decode_algorithmic_GBps", "GB/s"),
                                                  ("msvid_512x384_l4", "msvid_algorithmic_GBps", "GB/s"),
                                                  ("admm_300x260_r64_l4", "admm_update_TFLOPs", "TFLOP/s")])
def test_reference_arm_line(workload, metric, unit):
    d = run_reference("--workload", workload)
    assert KEYS <= set(d)
    assert d["impl"] == "reference" and d["metric"] == metric and d["unit"] == unit
    assert d["value"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["config"]["workload"] == workload
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_admm_flop_count_by_hand():
    sys.path.insert(0, ROOT)
    import bench
    # N = 4, M = 3, R = 2, one inner iteration: W V 2*4*3*2 = 48, V^T V (a triangle) 3*2*2 = 12, Cholesky 8/3, solves 2*4*2*2 = 32
    assert abs(bench.admm_flops(4, 3, 2, 1) - (48 + 12 + 8 / 3 + 32)) < 1e-9
    assert abs(bench.admm_flops(4, 3, 2, 3) - (48 + 12 + 8 / 3 + 96)) < 1e-9
    assert bench.admm_shape("admm_8192x4096_r1664_l16_in3") == (8192, 4096, 1664, 16, 3)


def test_accounting_against_hand_counts():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2512_24545_b200 import inputs
    spec = inputs.qproj(1664)                     # 4096 x 4096, k = 1664, l = 16, fp16 envelopes, bf16 activations
    signs = 1664 * (4096 + 4096) // 8
    env = 2 * 16 * (4096 + 4096 + 2 * 1664)
    assert bench.algorithmic_bytes(spec, 1) == signs + env + 2 * (4096 + 4096)
    assert bench.expanded_flops(spec, 3) == 2.0 * 16 * 3 * 1664 * (4096 + 4096)
    assert bench.materialised_flops(spec, 3) == (2.0 * 3 + 2.0 * 16) * 1664 * (4096 + 4096)
