"""Pins for the oracle's top-p (nucleus) sampling: the sampling settings of the paper's evaluation
(Appendix: temperature 0.2, top-p 0.95)."""
import itertools

import numpy as np
import pytest

from oracle import rd_oracle as orc


def test_hand_worked_distribution():
    """Probabilities 0.5, 0.3, 0.15, 0.05 (in shuffled order): the kept set is read off the running
    sums 0.5, 0.8, 0.95, 1.0."""
    probs = np.array([0.15, 0.5, 0.05, 0.3])
    logits = np.log(probs) + 3.0                      # any shift: softmax is shift-invariant
    keep = lambda p: set(np.nonzero(orc.nucleus(logits, 1.0, p))[0].tolist())
    assert keep(0.3) == {1}
    assert keep(0.49) == {1}
    assert keep(0.51) == {1, 3}
    assert keep(0.79) == {1, 3}
    assert keep(0.81) == {1, 3, 0}
    assert keep(0.94) == {1, 3, 0}
    assert keep(0.96) == {0, 1, 2, 3}
    assert keep(1.0) == {0, 1, 2, 3}


def test_temperature_enters_before_the_cut():
    """At temperature T the distribution is softmax(l / T): with T = 0.5 the probabilities above
    become proportional to their squares (0.25, 0.09, 0.0225, 0.0025) / 0.365."""
    probs = np.array([0.5, 0.3, 0.15, 0.05])
    logits = np.log(probs)
    sq = probs ** 2 / np.sum(probs ** 2)              # 0.685, 0.247, 0.0616, 0.0068
    assert sq[0] < 0.7 < sq[0] + sq[1]
    assert orc.nucleus(logits, 0.5, 0.7).tolist() == [True, True, False, False]
    assert orc.nucleus(logits, 1.0, 0.7).tolist() == [True, True, False, False]
    assert orc.nucleus(logits, 0.5, 0.6).tolist() == [True, False, False, False]
    assert orc.nucleus(logits, 1.0, 0.6).tolist() == [True, True, False, False]


@pytest.mark.parametrize("seed", range(6))
def test_smallest_set_of_most_probable_tokens_by_search_over_all_subsets(seed):
    """Definition check without sorting: among all subsets whose mass reaches top_p take the smallest
    size; the nucleus is the subset of that size with the largest mass."""
    rng = np.random.default_rng(seed)
    V = 7
    logits = rng.normal(0, 2.0, V).astype(np.float32)
    q = np.exp(logits.astype(np.float64) - logits.max())
    q /= q.sum()
    for top_p in (0.2, 0.5, 0.77, 0.9, 0.99):
        best = None
        for k in range(1, V + 1):
            cands = [(sum(q[list(c)]), c) for c in itertools.combinations(range(V), k)]
            mass, c = max(cands)
            if mass >= top_p:
                best = set(c)
                break
        assert set(np.nonzero(orc.nucleus(logits, 1.0, top_p))[0].tolist()) == best


def test_equal_logits_at_the_cut_stay_together_and_limits():
    logits = np.array([2.0, 1.0, 1.0, 1.0, -3.0], dtype=np.float32)
    q = np.exp(logits - logits.max()); q /= q.sum()
    p_cut = float(q[0] + 0.5 * q[1])                  # the cut falls on the first of the three equal tokens
    assert orc.nucleus(logits, 1.0, p_cut).tolist() == [True, True, True, True, False]
    assert orc.nucleus(logits, 1.0, 1e-9).tolist() == [True, False, False, False, False]
    assert orc.nucleus(logits, 1.0, 1.0).all()


def test_tiny_top_p_is_greedy_and_one_is_plain_sampling():
    rng = np.random.default_rng(3)
    for t in range(20):
        logits = rng.normal(0, 1.5, 50).astype(np.float32)
        assert orc.sample_token(logits, 0.7, 5, 0, t, top_p=1e-6) == int(np.argmax(logits))
        assert orc.sample_token(logits, 0.7, 5, 0, t, top_p=1.0) == orc.sample_token(logits, 0.7, 5, 0, t)


def test_sampled_frequencies_follow_the_renormalised_nucleus():
    """Gumbel-max over the kept tokens samples softmax(l / T) renormalised over them: compare the
    frequencies over many token positions (fresh noise each) with that distribution."""
    rng = np.random.default_rng(0)
    V, T, top_p, n = 12, 0.8, 0.85, 6000
    logits = rng.normal(0, 1.2, V).astype(np.float32)
    keep = orc.nucleus(logits, T, top_p)
    q = np.exp((logits.astype(np.float64) - logits.max()) / T) * keep
    q /= q.sum()
    assert 1 < keep.sum() < V
    counts = np.zeros(V)
    for pos in range(n):
        counts[orc.sample_token(logits, T, 17, 0, pos, top_p=top_p)] += 1
    assert counts[~keep].sum() == 0
    chi2 = float(np.sum((counts[keep] - n * q[keep]) ** 2 / (n * q[keep])))
    assert chi2 < 30.0                                # 99.9 % point of chi-square with <= 10 degrees of freedom


def test_sampler_passes_top_p_through():
    from helpers import SMALL, make_oracle
    import rd_inputs
    model, _ = make_oracle(SMALL, std=0.08)
    prompt = rd_inputs.make_prompt(6, SMALL["vocab"], 1)
    a = orc.Sampler(model, seed=2, temperature=1.0, top_p=1e-6)
    g = orc.Sampler(model, seed=2, temperature=0.0)
    s = orc.Sampler(model, seed=2, temperature=1.0)
    sa, sg, ss = a.prefill(0, prompt, 2, 6), g.prefill(0, prompt, 2, 6), s.prefill(0, prompt, 2, 6)
    a.generate_ar(sa, 2)
    g.generate_ar(sg, 2)
    s.generate_ar(ss, 2)
    assert np.array_equal(sa.committed(), sg.committed())     # a nucleus of one token is greedy decoding
    assert not np.array_equal(ss.committed(), sg.committed()) # while plain sampling at T = 1 is not
