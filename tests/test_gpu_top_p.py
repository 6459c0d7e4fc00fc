"""GPU parity of Sample with top-p (the paper's evaluation samples with temperature 0.2 and top-p
0.95) against the oracle, in lock-step, through the C ABI."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model
from helpers import SMALL, make_oracle

pytestmark = pytest.mark.gpu


def _pair(shape, W, max_new, temperature, top_p, batch=1, bf16=False, seed=0, cap=16, std=0.05, **okw):
    model, w = make_oracle(shape, seed=seed, std=std, gain_jitter=0.0, bf16=bf16, contract=bf16, **okw)
    gm = gpu_model(shape, w, bf16=bf16)
    sess = rd.Session(gm, batch=batch, max_context=256, max_window=W, max_iters_per_pos=cap, max_new_tokens=max_new,
                      keep_logits=True, temperature=temperature, seed=seed + 31, top_p=top_p)
    sm = orc.Sampler(model, seed=seed + 31, temperature=temperature, max_iters_per_pos=cap, top_p=top_p)
    return sess, sm


def _prefill(sm, sess, shape, lens, r, max_new):
    seqs = []
    for b, L in enumerate(lens):
        prompt = rd_inputs.make_prompt(L, shape["vocab"], seed=b)
        seqs.append(sm.prefill(b, prompt, r, max_new))
        sess.prefill(b, prompt, r)
    return seqs


@pytest.mark.parametrize("temperature,top_p", [(1.0, 0.9), (0.2, 0.95), (1.5, 0.5), (1.0, 0.05)])
def test_fp32_lock_step_with_top_p(temperature, top_p):
    """float32 configuration: logits agree to 1e-4, so the kept sets agree except for tokens whose
    cumulative mass is within 1e-3 of the cut; tokens must be identical otherwise."""
    sess, sm = _pair(SMALL, 4, 24, temperature, top_p, batch=2, std=0.1)
    seqs = _prefill(sm, sess, SMALL, [9, 17], 2, 24)
    ls = LockStep(sm, sess, seqs, Tolerance(1e-4), nucleus_band=1e-3)
    while not ls.all_done():
        ls.df(4, 1, 0.0)
    ls.final_tokens_equal()
    assert ls.boundary_cases <= 2
    # the cut really removes tokens: some drafts differ from what plain sampling would have drawn
    plain = orc.Sampler(sm.m, seed=sm.seed, temperature=temperature)
    differs = 0
    for sq in seqs:
        q = plain.prefill(sq.seq_id, rd_inputs.make_prompt([9, 17][sq.seq_id], SMALL["vocab"], seed=sq.seq_id), 2, 24)
        while not q.done:
            plain.df_step(q, 4, 1, 0.0)
        differs += int(not np.array_equal(q.committed(), sq.committed()))
    assert differs > 0


@pytest.mark.parametrize("vocab", [65536, 50001])
def test_full_vocabulary_and_ragged_vocabulary(vocab):
    """The largest vocabulary the top-p kernel takes (every thread of the row's cluster holds its full
    32 logits) and one that is not a multiple of 4 (scalar loads, a partly filled last group)."""
    shape = dict(SMALL, vocab=vocab, n_core=1)
    sess, sm = _pair(shape, 3, 6, 1.0, 0.9, batch=2, std=0.1)
    seqs = _prefill(sm, sess, shape, [4, 7], 1, 6)
    ls = LockStep(sm, sess, seqs, Tolerance(1e-4), nucleus_band=1e-3)
    while not ls.all_done():
        ls.df(3, 1, 0.0)
    ls.final_tokens_equal()
    assert ls.boundary_cases <= 1
    # and with a cut so low that most rows go through the search for tau
    sess, sm = _pair(shape, 3, 6, 1.0, 0.002, batch=2, std=0.1)
    seqs = _prefill(sm, sess, shape, [4, 7], 1, 6)
    ls = LockStep(sm, sess, seqs, Tolerance(1e-4), nucleus_band=1e-5)
    while not ls.all_done():
        ls.df(3, 1, 0.0)
    ls.final_tokens_equal()


def test_vocabulary_beyond_the_kernel_limit_is_refused():
    shape = dict(SMALL, vocab=65540, n_core=1)
    model, w = make_oracle(shape, seed=0, std=0.1)
    gm = gpu_model(shape, w)
    with pytest.raises(rd.RdError):
        rd.Session(gm, batch=1, max_context=64, max_window=2, max_new_tokens=4, temperature=1.0, top_p=0.9)
    rd.Session(gm, batch=1, max_context=64, max_window=2, max_new_tokens=4, temperature=1.0).close()   # fine without top-p


def test_bf16_twin_ragged_batch_top_p():
    """bf16 configuration (tensor-core GEMMs), ragged batch, adaptive exit, T = 1, top-p 0.9.  The
    logit tolerance moves the cumulative masses near the cut by a few percent: band 0.1."""
    shape = rd_inputs.TWIN
    # (the contractive adapter of the other bf16 tests: a row takes up to 16 recurrences here, along which
    # rounding differences between two bf16 evaluations grow with the plain init)
    sess, sm = _pair(shape, 8, 16, 1.0, 0.9, batch=4, bf16=True, std=0.02, adapter_s_scale=0.25)
    seqs = _prefill(sm, sess, shape, [5, 33, 12, 40], 4, 16)
    ls = LockStep(sm, sess, seqs, Tolerance(5e-2, 2e-2), tie_gap=3e-2, nucleus_band=0.1)
    for _ in range(40):
        if ls.all_done():
            break
        ls.df(8, 1, 1e-3)
    assert ls.all_done()
    assert ls.near_ties <= max(2, int(0.08 * ls.n_drafts))


def test_tiny_top_p_is_greedy_and_one_is_plain_sampling_on_the_gpu():
    """A nucleus of one token reproduces greedy decoding; top_p = 1 and top_p = 0 leave temperature
    sampling as it was (same tokens as a session created without the field)."""
    model, w = make_oracle(SMALL, seed=2, std=0.1)
    gm = gpu_model(SMALL, w)
    prompt = rd_inputs.make_prompt(11, SMALL["vocab"], seed=4)

    def run(temperature, top_p):
        s = rd.Session(gm, batch=1, max_context=128, max_window=4, max_new_tokens=20, temperature=temperature,
                       seed=9, top_p=top_p)
        s.prefill(0, prompt, 2)
        while not s.committed(0)[1]:
            s.df_step(4, 1, 0.0)
        return s.tokens(0)

    greedy = run(0.0, 0.0)
    assert np.array_equal(run(1.0, 1e-7), greedy)
    plain = run(1.0, 0.0)
    assert np.array_equal(run(1.0, 1.0), plain)
    assert not np.array_equal(plain, greedy)
    assert np.array_equal(run(1.0, 0.9), run(1.0, 0.9))          # run-to-run identical


def test_bad_top_p_is_refused():
    model, w = make_oracle(SMALL, seed=2)
    gm = gpu_model(SMALL, w)
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(rd.RdError):
            rd.Session(gm, batch=1, max_context=64, max_window=2, max_new_tokens=4, temperature=1.0, top_p=bad)
