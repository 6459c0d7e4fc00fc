"""GPU test of rd_debug_read_kv_noalloc, the K/V read-out that allocates nothing.

Some users of this library cannot allocate device memory at the moment they want to look at the
cache: a serving process that gave every remaining byte of the device to its KV caches, or one
whose other sessions keep stepping on other streams and must not be stalled by cudaMalloc /
cudaFree.  For them the library stages the read through a fixed array inside its own image.  The
test calls it through the C ABI twice in a row and compares each result with rd_debug_read_kv,
which allocates its staging buffer: the values must be identical, bit for bit (the comparison the
cache tests of this suite use).  The second call asks for fewer rows than the first, so that
leftovers of the first call in the shared array would be noticed.  This file sorts last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from gpu_harness import gpu_model

pytestmark = pytest.mark.gpu


def _session(max_ctx):
    shape = rd_inputs.TWIN
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=3, bf16=True)
    gm = gpu_model(shape, w, bf16=True)
    sess = rd.Session(gm, batch=2, max_context=max_ctx, max_window=4, max_new_tokens=8, seed=11)
    for b, L in enumerate((37, 21)):
        sess.prefill(b, rd_inputs.make_prompt(L, shape["vocab"], seed=40 + b), 2)
    for _ in range(5):
        sess.df_step(4, 1, 0.0)
    return gm, sess


def test_noalloc_read_equals_allocating_read_twice_in_a_row():
    gm, sess = _session(128)
    # (block, layer, which, seq, pos0, n): a large read first, then a smaller one elsewhere
    for block, layer, which, seq, pos0, n in ((1, 3, 0, 0, 0, 41), (2, 1, 1, 1, 5, 9)):
        want = sess.read_kv(block, layer, which, seq, pos0, n)
        got = sess.read_kv_noalloc(block, layer, which, seq, pos0, n)
        assert got.shape == want.shape == (n, rd_inputs.TWIN["hidden"])
        assert np.abs(want).max() > 0, "the cache rows under test are empty"
        assert np.array_equal(got, want)
    assert sess.read_kv_noalloc(0, 0, 0, 0, 3, 0).shape == (0, rd_inputs.TWIN["hidden"])
    sess.close()
    gm.close()


def test_noalloc_read_refuses_more_than_the_fixed_array_holds():
    gm, sess = _session(2400)
    n = 2300                                   # 2300 * 480 values > 1,048,576
    assert n * rd_inputs.TWIN["hidden"] > 1 << 20
    with pytest.raises(rd.RdError) as err:
        sess.read_kv_noalloc(1, 0, 0, 0, 0, n)
    assert err.value.code == rd.RD_E_CAPACITY
    assert b"staging array" in rd.lib().rd_last_cuda_error()
    ok = sess.read_kv_noalloc(1, 0, 0, 0, 0, 2000)      # still usable afterwards, and within the limit
    assert np.array_equal(ok, sess.read_kv(1, 0, 0, 0, 0, 2000))
    sess.close()
    gm.close()
