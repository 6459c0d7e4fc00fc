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


def _check_noise_mix_against_hand_schedule(W, inner, eps, cap, schedule, n_steps):
    """Every step: recompute z = R^inner(e, (1 - b) z + b z_noise) from each row's stored z and the
    number of steps it has taken, with b read from `schedule` (numbers, not the formula), on a copy
    of the caches, and compare with what the sampler produced."""
    import copy
    beta = 0.8
    model, _ = make_oracle(SMALL, seed=1)
    sm = orc.Sampler(model, seed=3, beta=beta, max_iters_per_pos=cap)
    sq = sm.prefill(0, rd_inputs.make_prompt(9, SMALL["vocab"], seed=2), 2, 12)
    seen = set()
    for _ in range(n_steps):
        rows = sq.window
        pos = np.array([r.pos for r in rows])
        caches = copy.deepcopy(sq.caches)
        e = model.prelude(sq.tokens[pos], pos, caches)
        z = np.stack([r.z for r in rows]).copy()
        for i, r in enumerate(rows):
            b = schedule[r.steps]
            seen.add(r.steps)
            noise = orc.latent_noise(3, 0, r.pos, r.steps, SMALL["hidden"], 1.0, model.dtype)
            z[i] = (1.0 - b) * z[i] + b * noise
        for _ in range(inner):
            z = model.core(e, z, pos, caches)
        info = sm.df_step(sq, W, inner, eps)
        assert np.allclose(info["z"], z, rtol=0, atol=1e-6), f"rows at steps {[r.steps - 1 for r in rows]}"
    return seen


def test_noise_schedule_fixed_exit_is_the_hand_written_one():
    """Fixed exit, window 4, beta 0.8: a position's steps 0, 1, 2, 3 mix in 0.8, 0.6, 0.4, 0.2 of noise
    (linear in the steps taken, the later steps less noisy; zero would come at step 4, which no
    position takes)."""
    seen = _check_noise_mix_against_hand_schedule(4, 1, 0.0, 64, {0: 0.8, 1: 0.6, 2: 0.4, 3: 0.2}, 8)
    assert seen == {0, 1, 2, 3}


def test_noise_schedule_adaptive_exit_runs_over_cap_by_inner_steps():
    """Adaptive exit, cap 12 core iterations, 2 per step: a position gets 6 steps and its mix falls
    from 0.8 by 0.8 / 6 per step."""
    sched = {0: 0.8, 1: 0.6666666666666667, 2: 0.5333333333333333, 3: 0.4, 4: 0.26666666666666666, 5: 0.13333333333333333}
    seen = _check_noise_mix_against_hand_schedule(8, 2, 1e-12, 12, sched, 9)
    assert seen == {0, 1, 2, 3, 4, 5}


def test_a_shifted_or_shortened_schedule_is_told_apart():
    """The check above has teeth: schedules off by one step, or stretched over one step fewer, miss
    by far more than its tolerance."""
    import pytest
    for wrong in ({0: 0.6, 1: 0.4, 2: 0.2, 3: 0.0}, {0: 0.8, 1: 0.8 * 2 / 3, 2: 0.8 / 3, 3: 0.0}):
        with pytest.raises(AssertionError):
            _check_noise_mix_against_hand_schedule(4, 1, 0.0, 64, wrong, 8)


def test_full_strength_noise_wipes_out_the_initial_state():
    """With beta = 1 a position's first step starts from pure noise."""
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
