"""GPU parity of the slot engine (Appendix, "Larger Batch Sizes"): hidden-state slots drawn from a pool
smaller than batch x window, sequences of different ages stepping together, requests arriving while
others are mid-wavefront (prefill only enqueues), a finished sequence's slot index reused by a new
request.  The oracle side is per-sequence: every sequence runs its own single-sequence sampler, told by
a host model of the pool (tests/helpers.py) in which steps it may extend its wavefront; the GPU's
rows, latents, logits, delta, drafts and commit counts are compared every step."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model
from helpers import SMALL, SlotPoolModel, make_oracle

pytestmark = pytest.mark.gpu


class SlicedJobs:
    """Host model of the sliced prefills: every step works off one unit (one pass over one chunk of at
    most max(512, decode rows) prompt rows) of the oldest job; the step whose unit finishes a job is the first
    step its sequence takes part in."""

    def __init__(self, chunk_rows):
        self.chunk_rows = chunk_rows
        self.queue = []

    def add(self, b, prompt, r, old=None):
        n = len(prompt) - 1
        self.queue.append([b, prompt, r, (r + 2) * -(-n // self.chunk_rows), old])

    def before_step(self, start, units=1):
        while units > 0 and self.queue:
            job = self.queue[0]
            if job[3] > 0:
                job[3] -= 1
                units -= 1
            if job[3] == 0:
                start(*job[:3], job[4])
                self.queue.pop(0)


def _run_staggered(shape, bf16, tol, tie_gap, W, n_slots, eps, temperature, max_new, wkw, sliced=False):
    model, w = make_oracle(shape, seed=3, bf16=bf16, contract=bf16, max_ctx=160, gain_jitter=0.0 if bf16 else 0.1, **wkw)
    gm = gpu_model(shape, w, bf16=bf16)
    B = 4
    sess = rd.Session(gm, batch=B, max_context=160, max_window=W, max_iters_per_pos=8, max_new_tokens=max_new,
                      keep_logits=True, temperature=temperature, seed=21, latent_slots=n_slots)
    sm = orc.Sampler(model, seed=21, temperature=temperature, max_iters_per_pos=8)
    cap = n_slots or B * W                           # 0: the plain batch x window table
    pool = SlotPoolModel(cap)
    prompts = {b: rd_inputs.make_prompt(L, shape["vocab"], seed=50 + b) for b, L in enumerate((23, 9, 41, 15))}
    arrivals = {0: [0, 1], 3: [2], 7: [3]}          # step -> sequences that arrive before it
    seqs = [None] * B

    ls = LockStep(sm, sess, seqs, tol, tie_gap=tie_gap)
    restarted, widest, stalled = False, 0, False
    jobs = SlicedJobs(-(-max(512, cap) // 16) * 16)

    def start(b, prompt, r, old):
        seqs[b] = pool.start(sm, b, prompt, r, max_new, old=old)

    for step in range(400):
        for b in arrivals.get(step, []):
            if sliced and b != 0:
                # admitted between the steps of the running sequences; the oracle's sequence starts
                # at the step that works off the job's last unit
                jobs.add(b, prompts[b], 2)
                sess.prefill_sliced(b, prompts[b], 2)
                continue
            seqs[b] = pool.start(sm, b, prompts[b], 2, max_new)
            sess.prefill(b, prompts[b], 2)
        if not restarted and seqs[1] is not None and seqs[1].done:
            # the finished sequence's entry takes a new request while the others are in flight
            old = seqs[1]
            p = rd_inputs.make_prompt(12, shape["vocab"], seed=77)
            if sliced:
                jobs.add(1, p, 3, old)
                sess.prefill_sliced(1, p, 3)
                with pytest.raises(rd.RdError) as err:            # one job per sequence
                    sess.prefill_sliced(1, p, 3)
                assert err.value.code == rd.RD_E_STATE
                with pytest.raises(rd.RdError) as err:            # the workspace is the jobs'
                    sess.prefill(1, p, 3)
                assert err.value.code == rd.RD_E_STATE
            else:
                seqs[1] = pool.start(sm, 1, p, 3, max_new, old=old)
                sess.prefill(1, p, 3)
            restarted = True
        assert sess.prefill_pending() == len(jobs.queue)
        jobs.before_step(start)
        live = [sq for sq in seqs if sq is not None]
        ls.seqs = live
        if restarted and not jobs.queue and all(sq.done for sq in live) and step > 8:
            break
        wants_more = sum(1 for sq in live if not sq.done and len(sq.window) < W)
        ls.df_pooled(pool, W, 1, eps)
        in_flight = sum(len(sq.window) for sq in live)
        widest = max(widest, in_flight)
        assert in_flight <= cap
        stalled |= pool.free == 0 and wants_more > 0
    assert restarted and all(sq.done for sq in live)
    ls.final_tokens_equal()
    assert sliced or (widest == n_slots and stalled)  # the pool was the limit at some point
    print(f"steps {ls.steps}, near-ties {ls.near_ties} of {ls.n_drafts}, max err {ls.max_err}")
    sess.close()
    gm.close()
    return ls


def test_fp32_pool_smaller_than_batch_times_window_fixed_exit():
    ls = _run_staggered(SMALL, False, Tolerance(1e-4), 0.0, W=4, n_slots=10, eps=0.0, temperature=0.0, max_new=9, wkw=dict(std=0.08))
    assert ls.near_ties == 0


def test_fp32_sliced_prefill_admission_fixed_table():
    """Requests admitted by rd_prefill_sliced while sequence 0 decodes: one prefill unit per step."""
    ls = _run_staggered(SMALL, False, Tolerance(1e-4), 0.0, W=4, n_slots=0, eps=0.0, temperature=0.0, max_new=30, wkw=dict(std=0.08),
                        sliced=True)
    assert ls.near_ties == 0


def test_fp32_sliced_prefill_admission_pool_adaptive():
    ls = _run_staggered(SMALL, False, Tolerance(1e-4), 0.0, W=4, n_slots=7, eps=0.05, temperature=0.8, max_new=30, wkw=dict(std=0.08),
                        sliced=True)
    assert ls.near_ties == 0


def test_bf16_twin_sliced_prefill_admission():
    ls = _run_staggered(rd_inputs.TWIN, True, Tolerance(5e-2, 2e-2), 3e-2, W=8, n_slots=20, eps=0.0, temperature=0.0, max_new=12,
                        wkw=dict(adapter_s_scale=0.25), sliced=True)
    assert ls.near_ties <= max(2, int(0.08 * ls.n_drafts))


def test_sliced_prefill_equals_whole_prefill_bit_for_bit():
    """The same prompt through rd_prefill and through rd_prefill_sliced + rd_prefill_advance: the caches
    and the tokens of the decode that follows are the same bits."""
    model, w = make_oracle(SMALL, seed=5, max_ctx=704, std=0.08)
    gm = gpu_model(SMALL, w)
    L = 600                                          # two chunks of prompt rows per pass
    prompt = rd_inputs.make_prompt(L, SMALL["vocab"], seed=9)
    out = []
    for mode in ("whole", "sliced"):
        sess = rd.Session(gm, batch=2, max_context=704, max_window=4, max_new_tokens=12, seed=4)
        if mode == "whole":
            sess.prefill(1, prompt, 3)
        else:
            sess.set_prefill_units(0)
            sess.prefill_sliced(1, prompt, 3)
            assert sess.prefill_pending() == 1 and sess.committed(1) == (L, False)
            sess.prefill_advance(3)
            assert sess.prefill_pending() == 1
            sess.prefill_advance(1000)
            assert sess.prefill_pending() == 0 and sess.committed(1) == (L, False)
        kv = [sess.read_kv(blk, 0, which, 1, 0, L - 1) for blk in range(3) for which in range(2)]
        for _ in range(20):
            sess.df_step(4, 1, 0.0)
        out.append((kv, sess.tokens(1).copy()))
        sess.close()
    for a, b in zip(out[0][0], out[1][0]):
        assert np.array_equal(a, b)
    assert np.array_equal(out[0][1], out[1][1]) and len(out[0][1]) == L + 12
    gm.close()


def test_sliced_prefill_of_a_one_token_prompt():
    """A one-token prompt has no rows to prefill: the job finishes, without a unit, at the next step."""
    model, w = make_oracle(SMALL, seed=5, max_ctx=64, std=0.08)
    gm = gpu_model(SMALL, w)
    out = []
    for sliced in (False, True):
        sess = rd.Session(gm, batch=1, max_context=64, max_window=4, max_new_tokens=8, seed=4)
        (sess.prefill_sliced if sliced else sess.prefill)(0, np.array([7], dtype=np.int32), 2)
        assert sess.prefill_pending() == (1 if sliced else 0)
        for _ in range(14):
            sess.df_step(4, 1, 0.0)
        assert sess.prefill_pending() == 0 and sess.committed(0) == (9, True)
        out.append(sess.tokens(0).copy())
        sess.close()
    assert np.array_equal(out[0], out[1])
    gm.close()


def test_sliced_prefill_under_ar_steps():
    """rd_ar_step works the jobs off as rd_df_step does: a sequence admitted in slices while another
    decodes sequentially produces the tokens it produces alone, and does not change the other's."""
    model, w = make_oracle(SMALL, seed=6, max_ctx=128, std=0.08)
    gm = gpu_model(SMALL, w)
    pa = rd_inputs.make_prompt(20, SMALL["vocab"], seed=1)
    pb = rd_inputs.make_prompt(33, SMALL["vocab"], seed=2)

    def run(admit_b, alone_b=False):
        sess = rd.Session(gm, batch=2, max_context=128, max_window=4, max_new_tokens=10, seed=8)
        if not alone_b:
            sess.prefill(0, pa, 3)
        for step in range(30):
            if step == 2 and admit_b:
                (sess.prefill if alone_b else sess.prefill_sliced)(1, pb, 3)
            if alone_b and step < 2:
                continue                                   # nothing prefilled yet: a step would be out of order
            sess.ar_step(3)
        out = sess.tokens(0).copy(), sess.tokens(1).copy(), sess.committed(1)
        sess.close()
        return out

    a_alone, _, _ = run(False)
    a_both, b_both, (nb, done_b) = run(True)
    _, b_alone, _ = run(True, alone_b=True)
    assert np.array_equal(a_alone, a_both) and len(a_both) == 20 + 10
    assert done_b and nb == 33 + 10 and np.array_equal(b_both, b_alone)
    gm.close()


def test_fp32_pool_adaptive_exit_sampling():
    ls = _run_staggered(SMALL, False, Tolerance(1e-4), 0.0, W=4, n_slots=7, eps=0.05, temperature=0.8, max_new=9, wkw=dict(std=0.08))
    assert ls.near_ties == 0


def test_bf16_twin_pool_tensor_core_path():
    ls = _run_staggered(rd_inputs.TWIN, True, Tolerance(5e-2, 2e-2), 3e-2, W=8, n_slots=20, eps=0.0, temperature=0.0, max_new=12,
                        wkw=dict(adapter_s_scale=0.25))
    assert ls.near_ties <= max(2, int(0.08 * ls.n_drafts))


def test_pool_arguments():
    model, w = make_oracle(SMALL, seed=0)
    gm = gpu_model(SMALL, w)
    for bad in (-1, 2 * 4 + 1):
        with pytest.raises(rd.RdError) as err:
            rd.Session(gm, batch=2, max_context=64, max_window=4, max_new_tokens=4, latent_slots=bad)
        assert err.value.code == rd.RD_E_INVALID_ARG
    rd.Session(gm, batch=2, max_context=64, max_window=4, max_new_tokens=4, latent_slots=8).close()   # = batch x window: plain table
    gm.close()
