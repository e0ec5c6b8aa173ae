"""Byte accounting of the paper's two CNN experiments (host logic only: no GPU work is launched)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_memory_table_shapes_and_ratios():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--memory-table"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    t = json.loads(out.stdout.strip().splitlines()[-1])
    # 1-D net: per layer Moonwalk keeps fragments (2/block of an fp32 cotangent), sign bits and one
    # cotangent per 4 layers; Backprop keeps the activation as three bf16 term planes and sign bits
    act = 4 * 128 * 2048 * 256                       # one fp32 activation
    for blk in (4, 16):
        rows = {r["depth"]: r for r in t["fragmental_cnn1d"][f"block_{blk}"]["rows"]}
        per_layer = (rows[32]["moonwalk_residual"] - rows[16]["moonwalk_residual"]) / 16
        expect = act * 2 / blk + act / 32 + act / 4
        assert abs(per_layer - expect) <= 0.02 * expect
        per_layer_bp = (rows[32]["backprop_residual"] - rows[16]["backprop_residual"]) / 16
        assert abs(per_layer_bp - (1.5 * act + act / 32)) <= 0.02 * 1.5 * act
        # workspaces outside the residual part do not grow with depth (weights aside)
        fixed16 = rows[16]["moonwalk_workspace"] - rows[16]["moonwalk_residual"]
        fixed32 = rows[32]["moonwalk_workspace"] - rows[32]["moonwalk_residual"]
        assert fixed32 - fixed16 <= 16 * 40e6
    b4, b16 = t["fragmental_cnn1d"]["block_4"], t["fragmental_cnn1d"]["block_16"]
    assert b16["moonwalk_max_depth"] > b4["moonwalk_max_depth"] > 1.5 * b4["backprop_max_depth"]
    # 2-D net: what survives between the phases stops growing after the first layers
    s = {r["depth"]: r for r in t["strided_cnn"]}
    assert s[8]["moonwalk_residual"] - s[2]["moonwalk_residual"] < 0.03e9
    assert s[8]["backprop_residual"] > 1.3 * s[8]["moonwalk_residual"]
