"""GPU tests of the boundary's behaviour that is not arithmetic of the method: the analytic work
counters of rd_stats, prefill as an enqueue-only call, and the RD_E_TIMEOUT path of the bounded
pipeline waits."""
import os
import sys

import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from gpu_harness import gpu_model

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402

pytestmark = pytest.mark.gpu


def _twin(seed=0):
    shape = rd_inputs.TWIN
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=seed, bf16=True)
    return shape, gpu_model(shape, w, bf16=True)


def test_work_counters_follow_the_cost_remark():
    """Fixed exit, W = 4, one sequence, prompt 20, 10 tokens: rows in flight per step are
    1, 2, 3, 4, 4, ..., 3, 2, 1; the counters must equal the per-step figures the benchmark's formula
    gives for those rows and contexts, and the histogram one commit per step once the ramp is over."""
    shape, gm = _twin()
    L, N, W = 20, 10, 4
    sess = rd.Session(gm, batch=1, max_context=64, max_window=W, max_new_tokens=N, seed=1)
    sess.prefill(0, rd_inputs.make_prompt(L, shape["vocab"], seed=3), 2)
    want_b = want_f = 0
    steps = N + W - 1
    for t in range(1, steps + 1):
        sess.df_step(W, 1, 0.0)
        first = max(0, t - W)                       # rows first .. last of the generation are in flight
        last = min(t - 1, N - 1)
        rows = last - first + 1
        ctx = (L - 1) + last + 1                    # cache rows 0 .. position of the newest row
        b, f = bench.step_bytes_flops(shape, 1, rows, ctx, 1, 2)
        # the formula takes every row to attend the whole context; the library counts p + 1 keys for the row at p
        layers = shape["n_prelude"] + shape["n_core"] + shape["n_coda"]
        f -= 4 * shape["hidden"] * layers * (rows * ctx - sum(L - 1 + j + 1 for j in range(first, last + 1)))
        want_b += b
        want_f += f
    st = sess.stats()
    assert st["weight_bytes"] + st["kv_bytes"] == want_b
    assert st["flops"] == want_f
    assert st["tokens_committed"] == N and st["df_steps"] == steps
    hist = st["commit_hist"]
    assert hist[0] == W - 1 and hist[1] == N and sum(hist) == steps
    sess.close()
    gm.close()


def test_prefill_only_enqueues_and_leaves_other_sequences_alone():
    """rd_prefill returns without waiting for the device, keeps nothing of the caller's buffer, and a
    prefill of one sequence between two steps does not disturb the other sequence's wavefront: the
    other sequence's tokens equal those of a session in which it runs alone."""
    shape, gm = _twin(seed=5)
    W, N = 4, 12
    p0 = rd_inputs.make_prompt(31, shape["vocab"], seed=1)
    p1 = rd_inputs.make_prompt(45, shape["vocab"], seed=2)
    alone = rd.Session(gm, batch=2, max_context=128, max_window=W, max_new_tokens=N, seed=8)
    alone.prefill(0, p0, 3)
    for _ in range(N + W):
        alone.df_step(W, 1, 0.0)
    want0 = alone.tokens(0).copy()
    alone.close()
    sess = rd.Session(gm, batch=2, max_context=128, max_window=W, max_new_tokens=N, seed=8)
    buf = p0.copy()
    sess.prefill(0, buf, 3)
    buf[:] = 0                                      # the prompt was copied before the call returned
    for _ in range(5):
        sess.df_step(W, 1, 0.0)
    sess.prefill(1, p1, 3)                          # arrives while sequence 0 is mid-wavefront
    for _ in range(N + W):
        sess.df_step(W, 1, 0.0)
    assert np.array_equal(sess.tokens(0), want0)
    n1, done1 = sess.committed(1)
    assert done1 and n1 == len(p1) + N
    sess.close()
    gm.close()


def test_a_wait_that_runs_out_is_reported_and_the_library_stays_usable():
    """The bounded waits of the GEMM pipeline: one CTA of one launch never gets its first operand tile
    (rd_debug_expire_next_wait), its waits give up, the kernel raises the status word and returns, and
    rd_sync reports RD_E_TIMEOUT.  The session can be destroyed and a new session gives the same
    tokens as one that never saw the failure."""
    shape, gm = _twin(seed=7)
    prompt = rd_inputs.make_prompt(25, shape["vocab"], seed=4)

    def run(expire):
        sess = rd.Session(gm, batch=1, max_context=96, max_window=4, max_new_tokens=8, seed=2)
        sess.prefill(0, prompt, 2)
        sess.df_step(4, 1, 0.0)
        sess.sync()
        if expire:
            sess.expire_next_wait()
            sess.df_step(4, 1, 0.0)
            with pytest.raises(rd.RdError) as err:
                sess.sync()
            assert err.value.code == rd.RD_E_TIMEOUT
            with pytest.raises(rd.RdError) as err:      # the report is sticky for this session
                sess.committed(0)
            assert err.value.code == rd.RD_E_TIMEOUT
            sess.close()
            return None
        for _ in range(12):
            sess.df_step(4, 1, 0.0)
        out = sess.tokens(0).copy()
        sess.close()
        return out

    before = run(False)
    run(True)
    after = run(False)
    assert np.array_equal(before, after)
    gm.close()


def test_session_needs_the_models_device_current_and_read_ranges_do_not_wrap():
    shape, gm = _twin(seed=9)
    sess = rd.Session(gm, batch=1, max_context=64, max_window=2, max_new_tokens=4)
    sess.prefill(0, rd_inputs.make_prompt(9, shape["vocab"], seed=1), 1)
    big = 2 ** 31 - 1
    out = np.empty((2, shape["hidden"]), dtype=np.float32)
    for fn in (rd.lib().rd_debug_read_kv, rd.lib().rd_debug_read_kv_noalloc):
        # pos0 + n would wrap a 32-bit sum: refused on the host, no kernel is launched
        assert fn(sess.handle, 1, 0, 0, 0, big, 2, out.ctypes.data) == rd.RD_E_INVALID_ARG
        assert fn(sess.handle, 1, 0, 0, 0, 63, 2, out.ctypes.data) == rd.RD_E_INVALID_ARG
        assert fn(sess.handle, 1, 0, 0, 0, 62, 2, out.ctypes.data) == rd.RD_OK
    sess.close()
    gm.close()


def test_pipelined_poll_reports_each_step_one_step_late():
    """rd_poll_begin / rd_poll_end: the copy of the commit counters rides behind its step while the next
    step is already enqueued; what it reports is that step's state, and a third open ticket is refused."""
    shape, gm = _twin(seed=11)
    W, N, L = 4, 6, 14
    sess = rd.Session(gm, batch=1, max_context=64, max_window=W, max_new_tokens=N, seed=3)
    sess.prefill(0, rd_inputs.make_prompt(L, shape["vocab"], seed=8), 2)
    seen, pending = [], None
    for t in range(1, N + W + 2):
        sess.df_step(W, 1, 0.0)
        ticket = sess.poll_begin()
        if pending is not None:
            seen.append(sess.poll_end(pending, 0))
        pending = ticket
    with pytest.raises(rd.RdError) as err:
        a = sess.poll_begin()
        sess.poll_begin()                                # both tickets out
    assert err.value.code == rd.RD_E_STATE
    sess.poll_end(a)
    seen.append(sess.poll_end(pending, -1))
    want = [(L + max(0, min(t, N + W - 1) - (W - 1)), t >= N + W - 1) for t in range(1, N + W + 2)]
    assert seen == want
    sess.close()
    gm.close()
