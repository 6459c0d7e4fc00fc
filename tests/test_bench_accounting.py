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


# ---- the timed region: K steps at a full window, whatever K is -------------------------------------
def _commits_by_simulation(segments, batch, gen, window):
    """Fixed exit, counted the slow way: step t of a generation (1-based) commits one token per
    sequence when window <= t <= gen + window - 1."""
    tok = 0
    for ramp, n in segments:
        for t in range(ramp + 1, ramp + n + 1):
            if window <= t <= gen + window - 1:
                tok += batch
    return tok


def test_fewer_steps_than_the_window_still_commit():
    # the case that once measured an empty wavefront: 20 timed steps, window 32
    segs = bench.plan_timed_region(20, gen=256, window=32)
    assert segs == [(31, 20)]
    assert bench.expected_fixed_exit_tokens(segs, 1, 256, 32) == 20 == _commits_by_simulation(segs, 1, 256, 32)


def test_steps_equal_to_the_window():
    segs = bench.plan_timed_region(32, gen=256, window=32)
    assert segs == [(31, 32)] and _commits_by_simulation(segs, 4, 256, 32) == 128
    assert bench.expected_fixed_exit_tokens(segs, 4, 256, 32) == 128


def test_more_steps_than_one_generation_holds_restart_it():
    K = 256 + 32 - 1 + 10                     # more than a whole generation's steps
    segs = bench.plan_timed_region(K, gen=256, window=32)
    assert bench.full_window_steps(256, 32) == 225
    assert segs == [(31, 225), (31, 297 - 225)] and sum(n for _, n in segs) == K
    assert bench.expected_fixed_exit_tokens(segs, 1, 256, 32) == K == _commits_by_simulation(segs, 1, 256, 32)


def test_every_timed_step_has_a_full_window():
    for K, gen, W in ((1, 64, 4), (61, 64, 4), (200, 64, 4), (20, 1024, 32)):
        for ramp, n in bench.plan_timed_region(K, gen, W):
            assert ramp == W - 1
            # rows in flight during step t: positions appended so far and not yet committed
            for t in range(ramp + 1, ramp + n + 1):
                assert min(t, gen) - max(0, t - W) == W


def test_generation_shorter_than_its_window():
    segs = bench.plan_timed_region(10, gen=4, window=8)
    assert segs == [(0, 10)] or sum(n for _, n in segs) == 10
    assert bench.expected_fixed_exit_tokens(segs, 1, 4, 8) == _commits_by_simulation(segs, 1, 4, 8)


def test_prefill_flops_of_a_512_token_prompt():
    # 511 rows: dense 2 * rows * parameters streamed, attention 4 h per (row, key, layer)
    f = bench.prefill_flops(rd_inputs.SHAPE_3P5B, [512], 32)
    dense = 2 * 511 * (4 * PER_LAYER + 32 * (4 * PER_LAYER + 2 * H * H))
    attn = 4 * H * (2 + 2 + 32 * 4) * (511 * 512 // 2)
    assert f == dense + attn and 54e12 < f < 57e12
