"""The benchmark's algorithmic bytes and FLOPs per step against figures worked out by hand from the
3.5B shape: per layer 4 h^2 + 3 h I parameters, adapter 2 h^2, tied head V h."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import rd_inputs  # noqa: E402

H, I, V = 5280, 17920, 65536
PER_LAYER = 4 * H * H + 3 * H * I            # 395,366,400 parameters


def test_weight_bytes_of_one_df_step():
    assert PER_LAYER == 395_366_400
    b, f = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, batch=1, rows=0, ctx_sum=0, inner=1, esz=2)
    assert b == 2 * ((2 + 2) * PER_LAYER + V * H + 4 * PER_LAYER + 2 * H * H) == 7_129_436_160
    b4, _ = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, batch=1, rows=0, ctx_sum=0, inner=4, esz=2)
    assert b4 - b == 3 * 3_274_444_800       # every further inner iteration streams core + adapter again


def test_kv_bytes_and_flops():
    rows, ctx = 32, 640
    b0, f0 = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, 1, 0, 0, 1, 2)
    b, f = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, 1, rows, ctx, 1, 2)
    layers = 2 + 4 + 2
    assert b - b0 == (ctx + rows) * 2 * H * 2 * layers          # K and V read once per layer, rows written
    dense = 2 * rows * (b0 // 2)
    attn = 4 * H * layers * rows * ctx
    assert f == dense + attn


def test_ar_token_is_about_fifteen_df_steps_of_weights():
    df, _ = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, 1, 0, 0, 1, 2)
    ar, _ = bench.step_bytes_flops(rd_inputs.SHAPE_3P5B, 1, 0, 0, 32, 2)
    assert abs(ar / 1e9 - 108.6) < 0.1 and 15.0 < ar / df < 15.5
