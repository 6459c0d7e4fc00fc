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


def _run_staggered(shape, bf16, tol, tie_gap, W, n_slots, eps, temperature, max_new, wkw):
    model, w = make_oracle(shape, seed=3, bf16=bf16, contract=bf16, max_ctx=160, gain_jitter=0.0 if bf16 else 0.1, **wkw)
    gm = gpu_model(shape, w, bf16=bf16)
    B = 4
    sess = rd.Session(gm, batch=B, max_context=160, max_window=W, max_iters_per_pos=8, max_new_tokens=max_new,
                      keep_logits=True, temperature=temperature, seed=21, latent_slots=n_slots)
    sm = orc.Sampler(model, seed=21, temperature=temperature, max_iters_per_pos=8)
    pool = SlotPoolModel(n_slots)
    prompts = {b: rd_inputs.make_prompt(L, shape["vocab"], seed=50 + b) for b, L in enumerate((23, 9, 41, 15))}
    arrivals = {0: [0, 1], 3: [2], 7: [3]}          # step -> sequences that arrive before it
    seqs = [None] * B

    ls = LockStep(sm, sess, seqs, tol, tie_gap=tie_gap)
    restarted, widest, stalled = False, 0, False
    for step in range(400):
        for b in arrivals.get(step, []):
            seqs[b] = pool.start(sm, b, prompts[b], 2, max_new)
            sess.prefill(b, prompts[b], 2)
        if not restarted and seqs[1] is not None and seqs[1].done:
            # the finished sequence's entry takes a new request while the others are in flight
            old = seqs[1]
            p = rd_inputs.make_prompt(12, shape["vocab"], seed=77)
            seqs[1] = pool.start(sm, 1, p, 3, max_new, old=old)
            sess.prefill(1, p, 3)
            restarted = True
        live = [sq for sq in seqs if sq is not None]
        ls.seqs = live
        if restarted and all(sq.done for sq in live) and step > 8:
            break
        wants_more = sum(1 for sq in live if not sq.done and len(sq.window) < W)
        ls.df_pooled(pool, W, 1, eps)
        in_flight = sum(len(sq.window) for sq in live)
        widest = max(widest, in_flight)
        assert in_flight <= n_slots
        stalled |= pool.free == 0 and wants_more > 0
    assert restarted and all(sq.done for sq in live)
    ls.final_tokens_equal()
    assert widest == n_slots and stalled              # the pool was the limit at some point
    print(f"steps {ls.steps}, near-ties {ls.near_ties} of {ls.n_drafts}, max err {ls.max_err}")
    sess.close()
    gm.close()
    return ls


def test_fp32_pool_smaller_than_batch_times_window_fixed_exit():
    ls = _run_staggered(SMALL, False, Tolerance(1e-4), 0.0, W=4, n_slots=10, eps=0.0, temperature=0.0, max_new=9, wkw=dict(std=0.08))
    assert ls.near_ties == 0


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
