"""GPU parity of the stabilisers of Section 3.4 (momentum on the input conditioning, linearly
scheduled latent noise) in lock step with the oracle: float32 on a small model at 1e-4, bf16 on the
reduced-width twin at the bf16 tolerance; the conditioning e itself is compared too."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model
from helpers import SMALL, make_oracle

pytestmark = pytest.mark.gpu


def _pair(shape, bf16, W, N, eta, beta, cap=12, temperature=0.0, seed=0):
    model, w = make_oracle(shape, seed=seed, gain_jitter=0.0 if bf16 else 0.1, bf16=bf16, contract=bf16, max_ctx=128)
    gm = gpu_model(shape, w, bf16=bf16)
    sess = rd.Session(gm, batch=1, max_context=128, max_window=W, max_iters_per_pos=cap, max_new_tokens=N,
                      keep_logits=True, temperature=temperature, seed=seed + 5, eta=eta, beta=beta)
    sm = orc.Sampler(model, seed=seed + 5, temperature=temperature, max_iters_per_pos=cap, eta=eta, beta=beta)
    prompt = rd_inputs.make_prompt(21, shape["vocab"], seed=seed)
    seqs = [sm.prefill(0, prompt, 3, N)]
    sess.prefill(0, prompt, 3)
    return gm, sess, sm, seqs


@pytest.mark.parametrize("W,inner,eps,eta,beta", [(4, 1, 0.0, 0.1, 0.0), (4, 1, 0.0, 0.0, 0.5), (5, 2, 0.0, 0.3, 0.8),
                                                  (4, 1, 0.02, 0.1, 0.5)])
def test_fp32_stabilisers_lock_step(W, inner, eps, eta, beta):
    gm, sess, sm, seqs = _pair(SMALL, False, W, 14, eta, beta)
    ls = LockStep(sm, sess, seqs, Tolerance(1e-4))
    while not ls.all_done():
        rows = list(seqs[0].window)
        ls.df(W, inner, eps)
        e_gpu = sess.debug_read(rd.RD_DBG_EMBED, 0)
        for i, r in enumerate(rows):                       # the conditioning after momentum
            assert np.abs(e_gpu[i] - r.e_prev).max() <= 1e-4 if eta > 0 else True
    assert ls.near_ties == 0
    ls.final_tokens_equal()
    sess.close()
    gm.close()


def test_bf16_twin_stabilisers_lock_step():
    gm, sess, sm, seqs = _pair(rd_inputs.TWIN, True, 8, 20, 0.1, 0.5, temperature=1.0)
    ls = LockStep(sm, sess, seqs, Tolerance(5e-2, 2e-2), tie_gap=3e-2)
    while not ls.all_done():
        ls.df(8, 1, 1e-3)
    ls.final_tokens_equal()
    assert ls.near_ties <= max(2, int(0.08 * ls.n_drafts))
    sess.close()
    gm.close()


def test_ar_step_ignores_the_stabilisers():
    """rd_ar_step is the plain sequential recurrence whatever eta and beta the session carries."""
    outs = []
    for eta, beta in ((0.0, 0.0), (0.2, 0.7)):
        gm, sess, sm, seqs = _pair(SMALL, False, 1, 6, eta, beta)
        for _ in range(6):
            sess.ar_step(5)
        outs.append((sess.tokens(0).copy(), sess.debug_read(rd.RD_DBG_LATENTS, 0).copy()))
        sess.close()
        gm.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_bad_strengths_are_refused():
    model, w = make_oracle(SMALL, seed=0)
    gm = gpu_model(SMALL, w)
    for eta, beta in ((1.0, 0.0), (-0.1, 0.0), (0.0, 1.5)):
        with pytest.raises(rd.RdError) as err:
            rd.Session(gm, batch=1, max_context=64, max_window=2, max_new_tokens=4, eta=eta, beta=beta)
        assert err.value.code == rd.RD_E_INVALID_ARG
    gm.close()
