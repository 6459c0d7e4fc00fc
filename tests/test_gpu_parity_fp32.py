"""GPU parity, float32 configuration: the tiny model of the first benchmark configuration in full,
plus edge cases, against the oracle in float64.  Tolerance (stated by the benchmark spec): max-abs 1e-4 on
latents and logits; committed tokens identical."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model
from helpers import MICRO, SMALL, make_oracle

pytestmark = pytest.mark.gpu
TOL = Tolerance(1e-4)


def _setup(shape, prompt_len, max_new, W, seed=0, temperature=0.0, batch=1, std=0.02, cap=64, gain_jitter=0.0,
           max_ctx=None, prompt_lens=None, **wkw):
    model, w = make_oracle(shape, seed=seed, std=std, gain_jitter=gain_jitter, max_ctx=max_ctx or 256, **wkw)
    gm = gpu_model(shape, w)
    sess = rd.Session(gm, batch=batch, max_context=max_ctx or 256, max_window=W, max_iters_per_pos=cap,
                      max_new_tokens=max_new, keep_logits=True, temperature=temperature, seed=seed + 100)
    sm = orc.Sampler(model, seed=seed + 100, temperature=temperature, max_iters_per_pos=cap)
    return model, gm, sess, sm


def _prefill_both(sm, sess, shape, lens, r, max_new, seed=0):
    seqs = []
    for b, L in enumerate(lens):
        prompt = rd_inputs.make_prompt(L, shape["vocab"], seed=seed + b)
        seqs.append(sm.prefill(b, prompt, r, max_new))
        sess.prefill(b, prompt, r)
    return seqs


def test_config1_df_w4_full_run():
    """Tiny model, prompt 32, 64 new tokens, greedy, DF sampler W=4, one inner iteration."""
    model, gm, sess, sm = _setup(rd_inputs.TINY, 32, 64, 4)
    seqs = _prefill_both(sm, sess, rd_inputs.TINY, [32], 8, 64)
    ls = LockStep(sm, sess, seqs, TOL)
    while not ls.all_done():
        ls.df(4, 1, 0.0)
    assert ls.steps == 64 + 4 - 1 and ls.near_ties == 0
    ls.final_tokens_equal()
    st = sess.stats()
    assert st["rows_core"] == 64 * 4 and st["rows_prelude"] == 64 * 4 and st["tokens_committed"] == 64


def test_config1_ar_r8_full_run_and_df_window1_identity():
    model, gm, sess, sm = _setup(rd_inputs.TINY, 32, 64, 1)
    seqs = _prefill_both(sm, sess, rd_inputs.TINY, [32], 8, 64)
    ls = LockStep(sm, sess, seqs, TOL)
    while not ls.all_done():
        ls.ar(8)
    ls.final_tokens_equal()
    ar_tokens = sess.tokens(0).copy()
    ar_z = sess.debug_read(rd.RD_DBG_LATENTS, 0).copy()
    # rd_df_step(1, r, 0) computes exactly what rd_ar_step(r) computes: bit-identical on the GPU
    sess2 = rd.Session(gm, batch=1, max_context=256, max_window=1, max_new_tokens=64, keep_logits=True, seed=100)
    sess2.prefill(0, rd_inputs.make_prompt(32, 512, seed=0), 8)
    for _ in range(64):
        sess2.df_step(1, 8, 0.0)
    assert np.array_equal(sess2.tokens(0), ar_tokens)
    assert np.array_equal(sess2.debug_read(rd.RD_DBG_LATENTS, 0), ar_z)


@pytest.mark.parametrize("W,inner,eps,temperature", [(3, 2, 0.0, 0.0), (5, 1, 0.05, 0.0), (4, 1, 0.0, 1.0),
                                                     (4, 2, 0.02, 0.7), (1, 1, 1e-3, 0.0)])
def test_small_models_modes(W, inner, eps, temperature):
    """Fixed and adaptive exit, greedy and sampled, gains != 1, on a small model."""
    model, gm, sess, sm = _setup(SMALL, 9, 14, W, std=0.08, gain_jitter=0.1, temperature=temperature, cap=12)
    seqs = _prefill_both(sm, sess, SMALL, [9], 3, 14)
    ls = LockStep(sm, sess, seqs, TOL)
    for _ in range(400):
        if ls.all_done():
            break
        ls.df(W, inner, eps)
    assert ls.all_done() and ls.near_ties == 0
    ls.final_tokens_equal()


def test_batch_ragged_prompts_and_single_token_prompt():
    """Several sequences with different prompt lengths (one of length 1) step together."""
    lens = [1, 7, 12, 4]
    model, gm, sess, sm = _setup(SMALL, 0, 10, 3, std=0.08, gain_jitter=0.1, batch=4, cap=9)
    seqs = _prefill_both(sm, sess, SMALL, lens, 2, 10)
    ls = LockStep(sm, sess, seqs, TOL)
    for _ in range(200):
        if ls.all_done():
            break
        ls.df(3, 1, 0.03)
    assert ls.all_done()
    ls.final_tokens_equal()


def test_prefill_longer_than_one_chunk_and_kv_cache_contents():
    """A prompt longer than the 512-row prefill chunk (two chunks: 512 + 87 rows); cache rows compared
    directly, across the chunk boundary too."""
    model, gm, sess, sm = _setup(SMALL, 0, 4, 2, std=0.08, gain_jitter=0.1, max_ctx=640)
    seqs = _prefill_both(sm, sess, SMALL, [600], 2, 4)
    for blk, name in enumerate(("prelude", "core", "coda")):
        for which, arr in ((0, seqs[0].caches[name].K), (1, seqs[0].caches[name].V)):
            got = sess.read_kv(blk, 0, which, 0, 0, 599)
            want = arr[0, :599].reshape(599, -1)
            assert np.abs(got - want).max() < 1e-4
    ls = LockStep(sm, sess, seqs, TOL)
    while not ls.all_done():
        ls.df(2, 1, 0.0)
    ls.final_tokens_equal()


def test_micro_shape_head_dim_8():
    model, gm, sess, sm = _setup(MICRO, 0, 6, 2, std=0.3, gain_jitter=0.1)
    seqs = _prefill_both(sm, sess, MICRO, [5], 2, 6)
    ls = LockStep(sm, sess, seqs, TOL)
    while not ls.all_done():
        ls.df(2, 2, 0.0)
    ls.final_tokens_equal()


def test_argument_and_state_errors():
    model, gm, sess, sm = _setup(SMALL, 0, 4, 2, max_ctx=32)
    with pytest.raises(rd.RdError) as e:
        sess.df_step(2, 1, 0.0)                       # nothing prefilled
    assert e.value.code == rd.RD_E_STATE
    with pytest.raises(rd.RdError) as e:
        sess.prefill(0, np.zeros(40, dtype=np.int32), 1)   # prompt + budget > max_context
    assert e.value.code == rd.RD_E_CAPACITY
    with pytest.raises(rd.RdError) as e:
        sess.prefill(0, np.array([0, 128], dtype=np.int32), 1)   # token id out of range
    assert e.value.code == rd.RD_E_INVALID_ARG
    sess.prefill(0, np.array([1, 2, 3], dtype=np.int32), 1)
    with pytest.raises(rd.RdError) as e:
        sess.df_step(3, 1, 0.0)                       # window > max_window
    assert e.value.code == rd.RD_E_CAPACITY
    sess.df_step(2, 1, 0.0)
    with pytest.raises(rd.RdError) as e:
        sess.ar_step(2)                               # AR inside an open wavefront
    assert e.value.code == rd.RD_E_STATE
    # steps after the budget are no-ops
    for _ in range(10):
        sess.df_step(2, 1, 0.0)
    n, done = sess.committed(0)
    assert done and n == 3 + 4


def test_slot_reuse_while_another_sequence_is_in_flight():
    """Continuous batching in its minimal form: a finished sequence's slot is prefilled again with a
    new prompt while the other sequence of the batch is in the middle of its wavefront; both go on in
    lock step with the oracle (sequences are independent)."""
    W = 3
    model, gm, sess, sm = _setup(SMALL, 0, 6, W, batch=2, gain_jitter=0.1)
    seqs = _prefill_both(sm, sess, SMALL, [7, 12], 2, 6)
    ls = LockStep(sm, sess, seqs, TOL)
    while not ls.all_done():                        # first generation of both sequences
        ls.df(W, 1, 0.0)
    # sequence 1 starts a new request and gets two steps ahead ...
    prompt1 = rd_inputs.make_prompt(9, SMALL["vocab"], seed=77)
    seqs[1] = sm.prefill(1, prompt1, 2, 6)
    sess.prefill(1, prompt1, 2)
    ls.df(W, 1, 0.0)
    ls.df(W, 1, 0.0)
    assert len(seqs[1].window) > 1                  # sequence 1 has an open wavefront
    # ... then slot 0 is reused for another request while slot 1 is in flight
    prompt0 = rd_inputs.make_prompt(5, SMALL["vocab"], seed=78)
    seqs[0] = sm.prefill(0, prompt0, 3, 6)
    sess.prefill(0, prompt0, 3)
    while not ls.all_done():
        ls.df(W, 1, 0.0)
    ls.final_tokens_equal()
    assert ls.near_ties == 0
