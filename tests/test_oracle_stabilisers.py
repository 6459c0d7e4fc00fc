"""Pins for the oracle's stabilisers (Section 3.4): momentum on the input conditioning and scheduled
latent noise."""
import numpy as np

import rd_inputs
from oracle import rd_oracle as orc
from helpers import SMALL, make_oracle


def _run(eta, beta, W=4, inner=1, eps=0.0, steps=6, cap=64, seed=3):
    model, _ = make_oracle(SMALL, seed=1)
    sm = orc.Sampler(model, seed=seed, eta=eta, beta=beta, max_iters_per_pos=cap)
    sq = sm.prefill(0, rd_inputs.make_prompt(9, SMALL["vocab"], seed=2), 2, 12)
    infos = [sm.df_step(sq, W, inner, eps) for _ in range(steps)]
    return model, sm, sq, infos


def test_zero_strength_changes_nothing():
    _, _, sq0, i0 = _run(0.0, 0.0)
    model, _ = make_oracle(SMALL, seed=1)
    sm = orc.Sampler(model, seed=3)                       # the sampler without the two arguments
    sq = sm.prefill(0, rd_inputs.make_prompt(9, SMALL["vocab"], seed=2), 2, 12)
    for a in i0:
        b = sm.df_step(sq, 4, 1, 0.0)
        assert np.array_equal(a["z"], b["z"]) and np.array_equal(a["logits"], b["logits"])


def test_momentum_is_the_stated_recursion_per_position():
    """e_t = eta e_{t-1} + (1 - eta) P_t for a position's later steps, e_0 = P_0: unrolled by hand
    from the conditioning the same model computes without momentum on the same tokens."""
    eta = 0.3
    model, _ = make_oracle(SMALL, seed=1)
    prompt = rd_inputs.make_prompt(9, SMALL["vocab"], seed=2)
    sm = orc.Sampler(model, seed=3, eta=eta)
    sq = sm.prefill(0, prompt, 2, 12)
    # reference: a second sampler without momentum, forced to see the same input tokens, gives P_t
    model2, _ = make_oracle(SMALL, seed=1)
    sm2 = orc.Sampler(model2, seed=3)
    sq2 = sm2.prefill(0, prompt, 2, 12)
    e_hist = {}
    for step in range(5):
        pos = np.array([r.pos for r in sq.window])
        sq2.tokens[:] = sq.tokens                          # same y_current
        p_t = model2.prelude(sq2.tokens[pos], pos, sq2.caches)
        sm.df_step(sq, 4, 1, 0.0)
        # (sq2's own window is not advanced: only its prelude is used)
        for i, p in enumerate(pos):
            want = p_t[i] if p not in e_hist else np.float32(eta) * e_hist[p] + np.float32(1 - eta) * p_t[i]
            e_hist[p] = want
        got = {r.pos: r.e_prev for r in sq.window}
        for p in got:
            if p in e_hist and got[p] is not None:
                assert np.allclose(got[p], e_hist[p], rtol=0, atol=1e-12)


def test_noise_schedule_is_linear_and_ends_at_zero():
    """With beta = 1 a position's first step starts from pure noise (its initial state is wiped out),
    and at step t the mix is beta (1 - t / T)."""
    model, _ = make_oracle(SMALL, seed=1)
    W = 4
    sm = orc.Sampler(model, seed=3, beta=1.0)
    sq = sm.prefill(0, rd_inputs.make_prompt(9, SMALL["vocab"], seed=2), 2, 12)
    row = sq.window[0]
    z0 = row.z.copy()
    noise0 = orc.latent_noise(3, 0, row.pos, 0, SMALL["hidden"], 1.0, model.dtype)
    pos = np.array([row.pos])
    e = model.prelude(sq.tokens[pos], pos, sq.caches)
    want = model.core(e, noise0[None, :], pos, sq.caches)   # beta_0 = 1: z' = noise
    info = sm.df_step(sq, W, 1, 0.0)
    assert np.allclose(info["z"][0], want[0], atol=1e-12)
    assert not np.allclose(noise0, z0)
    # schedule values through the public behaviour: beta_t for t = 0..T
    betas = [0.8 * max(0.0, 1.0 - t / W) for t in range(W + 1)]
    assert betas[0] == 0.8 and betas[-1] == 0.0 and np.allclose(np.diff(betas), -0.2)


def test_noise_draws_are_fresh_per_step_and_standard_normal():
    a = orc.latent_noise(7, 1, 40, 0, 4096, 1.0, np.float64)
    b = orc.latent_noise(7, 1, 40, 1, 4096, 1.0, np.float64)
    c = orc.init_state(7, 1, 40, 4096, 1.0, np.float64)
    assert abs(np.corrcoef(a, b)[0, 1]) < 0.06 and abs(np.corrcoef(a, c)[0, 1]) < 0.06
    assert abs(a.mean()) < 0.06 and abs(a.std() - 1.0) < 0.04
    assert np.array_equal(a, orc.latent_noise(7, 1, 40, 0, 4096, 1.0, np.float64))


def test_noise_and_momentum_keep_the_sampler_invariants():
    _, _, sq, infos = _run(0.1, 0.5, W=4, steps=15)
    assert sq.done and sq.n_committed == 9 + 12
    for info in infos:
        if info is not None:
            assert len(info["pos"]) <= 4
