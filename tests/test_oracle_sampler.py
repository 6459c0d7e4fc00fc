"""Pins for the oracle's samplers: the identities and behaviours the paper states."""
import hashlib
import math

import numpy as np
import pytest

import rd_inputs
from oracle import rd_oracle as orc
from helpers import MICRO, SMALL, make_oracle


def _prompt(n, vocab, seed=0):
    return rd_inputs.make_prompt(n, vocab, seed)


# ---- Section 3.3: "with this simplified exit rule, r' = r exactly recovers the AR sampler" ----
@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_df_window1_equals_ar(temperature):
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=11, temperature=temperature)
    prompt = _prompt(7, 128)
    a = sm.prefill(0, prompt, r=3, max_new=10)
    d = sm.prefill(0, prompt, r=3, max_new=10)
    for _ in range(10):
        ia = sm.ar_step(a, r=5)
        idf = sm.df_step(d, window=1, inner_iters=5, exit_threshold=0.0)
        assert np.array_equal(ia["z"], idf["z"]) and np.array_equal(ia["logits"], idf["logits"])
        assert idf["n_commit"] == 1
    assert a.done and d.done
    assert np.array_equal(a.committed(), d.committed())
    for b in ("prelude", "core", "coda"):
        assert np.array_equal(a.caches[b].K, d.caches[b].K)
    if temperature > 0:       # sampling really is in play: differs from greedy
        g = orc.Sampler(model, seed=11).prefill(0, prompt, 3, 10)
        orc.Sampler(model, seed=11).generate_ar(g, 5)
        assert not np.array_equal(g.committed(), a.committed())


# ---- derived from the same identity plus causality: the first committed token ----
@pytest.mark.parametrize("W,ri", [(4, 1), (3, 2), (2, 4)])
def test_first_committed_token_equals_ar(W, ri):
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=5)
    prompt = _prompt(9, 128, seed=1)
    a = sm.prefill(0, prompt, r=4, max_new=6)
    ia = sm.ar_step(a, r=W * ri)
    d = sm.prefill(0, prompt, r=4, max_new=6)
    for t in range(W):
        idf = sm.df_step(d, W, ri, 0.0)
        assert idf["n_commit"] == (1 if t == W - 1 else 0)
    # position L-1 saw a committed prefix and a fixed input for all W steps
    # (equal up to summation order: the BLAS call sees 1 row in AR and several in DF)
    assert np.abs(idf["z"][0] - ia["z"][0]).max() < 1e-12
    assert d.committed()[-1] == a.committed()[-1]


def test_adaptive_zero_threshold_commits_at_cap():
    """delta < 0 never holds, so every commit is a cap commit: first token = AR(r = cap)."""
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=5, max_iters_per_pos=6)
    prompt = _prompt(5, 128, seed=2)
    a = sm.prefill(0, prompt, 2, 4)
    ia = sm.ar_step(a, r=6)
    d = sm.prefill(0, prompt, 2, 4)
    commits = [sm.df_step(d, 8, 2, 1e-30)["n_commit"] for _ in range(3)]
    assert commits == [0, 0, 1]
    assert d.committed()[-1] == a.committed()[-1]


# ---- Section 3.3: frozen tokens leave the state, their KV entries are final ----
def _frozen_digest(sq):
    f = sq.n_committed - 1          # oldest in-flight position
    hsh = hashlib.sha256()
    hsh.update(sq.tokens[: sq.n_committed].tobytes())
    for b in ("prelude", "core", "coda"):
        hsh.update(sq.caches[b].K[:, :f].tobytes())
        hsh.update(sq.caches[b].V[:, :f].tobytes())
    return f, hsh.hexdigest()


@pytest.mark.parametrize("eps", [0.0, 0.05])
def test_frozen_positions_stop_changing(eps):
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=9, max_iters_per_pos=12)
    sq = sm.prefill(0, _prompt(6, 128, seed=3), 3, 12)
    snaps = []
    while not sq.done:
        sm.df_step(sq, 4, 1, eps)
        if not sq.done:
            snaps.append((sq.n_committed, sq.tokens[: sq.n_committed].copy(),
                          {b: (sq.caches[b].K[:, : sq.n_committed - 1].copy(),
                               sq.caches[b].V[:, : sq.n_committed - 1].copy()) for b in sq.caches}))
    for n, toks, kv in snaps:
        assert np.array_equal(sq.tokens[:n], toks)
        for b in kv:
            assert np.array_equal(sq.caches[b].K[:, : n - 1], kv[b][0])
            assert np.array_equal(sq.caches[b].V[:, : n - 1], kv[b][1])


# ---- "advances by at least one token per step"; the wavefront limiter ----
@pytest.mark.parametrize("W,ri,N", [(4, 1, 9), (1, 3, 4), (5, 2, 3)])
def test_fixed_mode_progress_window_bound_and_pass_counts(W, ri, N):
    model, _ = make_oracle(MICRO, std=0.3)
    sm = orc.Sampler(model, seed=1)
    prompt = _prompt(4, 32)
    sq = sm.prefill(0, prompt, 2, N)
    base = dict(model.row_passes)
    steps, commits = 0, []
    while not sq.done:
        assert 1 <= len(sq.window) <= W
        info = sm.df_step(sq, W, ri, 0.0)
        commits.append(info["n_commit"])
        steps += 1
    assert steps == N + W - 1                      # one token per step after a W-1 step ramp
    assert commits[: W - 1] == [0] * (W - 1) and commits[W - 1:] == [1] * N
    assert sq.n_committed == len(prompt) + N
    # cost remark: w tokens cost (r + r/r') f w with r = W r': W r' passes of R and W passes of
    # P and C per token
    assert model.row_passes["core"] - base["core"] == N * W * ri
    assert model.row_passes["prelude"] - base["prelude"] == N * W
    assert model.row_passes["coda"] - base["coda"] == N * W


def test_ar_pass_counts():
    model, _ = make_oracle(MICRO, std=0.3)
    sm = orc.Sampler(model, seed=1)
    sq = sm.prefill(0, _prompt(4, 32), 2, 5)
    base = dict(model.row_passes)
    sm.generate_ar(sq, 7)
    assert model.row_passes["core"] - base["core"] == 5 * 7        # (r + 1) f w
    assert model.row_passes["prelude"] - base["prelude"] == 5
    assert model.row_passes["coda"] - base["coda"] == 5


def test_prefill_pass_counts_and_single_token_prompt():
    model, _ = make_oracle(MICRO, std=0.3)
    sm = orc.Sampler(model, seed=1)
    sq = sm.prefill(0, _prompt(6, 32), 3, 2)
    assert model.row_passes == {"prelude": 5, "core": 15, "coda": 5}
    assert len(sq.window) == 1 and sq.window[0].pos == 5 and sq.window[0].steps == 0
    one = sm.prefill(1, _prompt(1, 32), 3, 2)
    assert model.row_passes == {"prelude": 5, "core": 15, "coda": 5}   # nothing to prefill
    sm.generate_ar(one, 2)
    assert one.n_committed == 3


def test_adaptive_stalls_when_window_full_then_cap_releases():
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=2, max_iters_per_pos=7)
    sq = sm.prefill(0, _prompt(5, 128), 2, 20)
    sizes, commits = [], []
    for _ in range(9):
        sizes.append(len(sq.window))
        commits.append(sm.df_step(sq, 3, 1, 1e-30)["n_commit"])
    # grows to the cap of 3 rows, stalls with no append, first row leaves at 7 iterations
    assert sizes == [1, 2, 3, 3, 3, 3, 3, 3, 3]
    assert commits == [0, 0, 0, 0, 0, 0, 1, 1, 1]


def test_adaptive_prefix_rule():
    """k* is the longest prefix with delta < eps (Eq. 3): a converged row behind an unconverged
    one must wait.  Built by hand: make row 1 converged by giving row 0 a large threshold miss."""
    model, _ = make_oracle(SMALL, std=0.08)
    sm = orc.Sampler(model, seed=2, max_iters_per_pos=1000)
    sq = sm.prefill(0, _prompt(5, 128), 2, 20)
    for _ in range(40):
        if sq.done:
            break
        info = sm.df_step(sq, 4, 1, 0.02)
        fr = info["delta"] < np.float32(0.02)
        k = 0
        while k < len(fr) and fr[k]:
            k += 1
        assert info["n_commit"] == k
        if k < len(fr):
            assert not fr[k]


# ---- convergence remark: R a contraction => adaptive DF reaches the AR solution ----
def test_contractive_model_adaptive_df_equals_ar():
    # The RMSNorm closing R makes the map scale-free in s, so a small weight scale alone does not
    # contract; shrinking the adapter's s-half until the e-half dominates its output does.
    model, _ = make_oracle(SMALL, std=0.05, adapter_s_scale=2e-3)
    prompt = _prompt(8, 128, seed=4)
    sm = orc.Sampler(model, seed=3, max_iters_per_pos=10_000)
    a = sm.prefill(0, prompt, 30, 12)
    sm.generate_ar(a, 60)
    d = sm.prefill(0, prompt, 30, 12)
    steps = sm.generate_df(d, window=4, inner_iters=1, exit_threshold=1e-9, max_steps=5000)
    assert d.done and steps < 5000
    assert np.array_equal(a.committed(), d.committed())


# ---- Section 3.5: wavefront 1 = the token-per-token adaptive-compute sampler ----
def test_wavefront1_adaptive_equals_iterate_until_converged():
    model, _ = make_oracle(SMALL, std=0.04)
    eps, cap = 1e-3, 50
    prompt = _prompt(6, 128, seed=6)
    sm = orc.Sampler(model, seed=4, max_iters_per_pos=cap)
    d = sm.prefill(0, prompt, 8, 5)
    sm.generate_df(d, 1, 1, eps)
    # independent loop: per token iterate s = R(e, s) until ||s - s_prev|| / ||s|| < eps
    ref = sm.prefill(0, prompt, 8, 5)
    toks = list(prompt)
    for t in range(5):
        pos = np.array([len(toks) - 1])
        e = model.prelude(np.array([toks[-1]]), pos, ref.caches)
        s = orc.init_state(4, 0, int(pos[0]), 64, 1.0, np.float64)[None]
        for it in range(cap):
            s_new = model.core(e, s, pos, ref.caches)
            dl = np.linalg.norm((s_new - s).astype(np.float32)) / np.linalg.norm(s_new.astype(np.float32))
            s = s_new
            if dl < eps:
                break
        toks.append(int(np.argmax(model.coda(s, pos, ref.caches)[0])))
    assert list(d.committed()) == toks


# ---- causality: information flows left to right only ----
def test_causality_later_rows_do_not_touch_earlier_results():
    model, _ = make_oracle(SMALL, std=0.08)
    rng = np.random.default_rng(0)
    tokens = rng.integers(0, 128, size=8)
    s0 = rng.standard_normal((8, 64))
    pos = np.arange(8)
    outs = []
    for variant in range(2):
        t, s = tokens.copy(), s0.copy()
        if variant:
            t[5] = (t[5] + 1) % 128
            s[6] += 1.0
        c = model.new_caches()
        outs.append(model.coda(model.core(model.prelude(t, pos, c), s, pos, c), pos, c))
    assert np.array_equal(outs[0][:5], outs[1][:5])
    assert not np.array_equal(outs[0][5], outs[1][5])


def test_budget_truncation_and_multi_commit():
    """Several rows can freeze in one step; commits stop at the budget."""
    model, _ = make_oracle(SMALL, std=0.02)
    sm = orc.Sampler(model, seed=3, max_iters_per_pos=4)
    sq = sm.prefill(0, _prompt(5, 128), 4, 3)
    total = 0
    while not sq.done:
        total += sm.df_step(sq, 4, 2, 0.5)["n_commit"]      # loose threshold: everything freezes
    assert total == 3 and sq.n_committed == 8 and sq.window == []


# ---- the cache against a no-cache recomputation ----
class NoCacheModel:
    """Keeps, per (block, layer, position), the normed layer input of the position's most recent
    pass, and recomputes every K and V (with rotation) at each attention call."""

    def __init__(self, model):
        self.m, self.cfg, self.dtype, self.max_ctx = model, model.cfg, model.dtype, model.max_ctx
        self.row_passes = {"prelude": 0, "core": 0, "coda": 0}

    def new_caches(self):
        return {b: {} for b in ("prelude", "core", "coda")}

    def _layer(self, blk, l, x, pos, store):
        c, w, p = self.cfg, self.m.w, f"{blk}.{l}."
        H, d = c.n_heads, c.head_dim
        a = orc.rmsnorm(x, w[p + "g1"], c.norm_eps)
        for i, ps in enumerate(pos):
            store[(l, int(ps))] = a[i].copy()
        out = np.empty_like(x)
        for i, ps in enumerate(pos):
            ctx = np.arange(int(ps) + 1)
            A = np.stack([store[(l, int(j))] for j in ctx])
            K = orc.rope((A @ w[p + "wk"].T).reshape(-1, H, d), ctx, self.m.cos, self.m.sin)
            V = (A @ w[p + "wv"].T).reshape(-1, H, d)
            q = orc.rope((a[i:i + 1] @ w[p + "wq"].T).reshape(1, H, d), pos[i:i + 1], self.m.cos, self.m.sin)[0]
            o = np.empty((H, d))
            for hh in range(H):
                sc = K[:, hh] @ q[hh] / math.sqrt(d)
                pr = np.exp(sc - sc.max()); pr /= pr.sum()
                o[hh] = pr @ V[:, hh]
            y = x[i] + o.reshape(-1) @ w[p + "wo"].T
            m2 = orc.rmsnorm(y, w[p + "g2"], c.norm_eps)
            g, u = m2 @ w[p + "wg"].T, m2 @ w[p + "wu"].T
            out[i] = y + (g / (1 + np.exp(-g)) * u) @ w[p + "wd"].T
        return out

    def prelude(self, tokens, pos, caches):
        x = self.m.w["emb"][np.asarray(tokens)]
        for l in range(self.cfg.n_prelude):
            x = self._layer("prelude", l, x, pos, caches["prelude"])
        return x

    def core(self, e, s, pos, caches):
        x = np.concatenate([e, s], axis=1) @ self.m.w["adapter"].T
        for l in range(self.cfg.n_core):
            x = self._layer("core", l, x, pos, caches["core"])
        return orc.rmsnorm(x, self.m.w["g_core"], self.cfg.norm_eps)

    def coda(self, s, pos, caches, head=True):
        x = s
        for l in range(self.cfg.n_coda):
            x = self._layer("coda", l, x, pos, caches["coda"])
        if not head:
            return None
        return orc.rmsnorm(x, self.m.w["g_final"], self.cfg.norm_eps) @ self.m.w["head"].T


@pytest.mark.parametrize("eps", [0.0, 0.05])
def test_cached_sampler_equals_no_cache_recomputation(eps):
    model, _ = make_oracle(MICRO, std=0.3, max_ctx=40)
    prompt = _prompt(5, 32, seed=8)
    sm = orc.Sampler(model, seed=6, max_iters_per_pos=9)
    sb = orc.Sampler(NoCacheModel(model), seed=6, max_iters_per_pos=9)
    a, b = sm.prefill(0, prompt, 3, 8), sb.prefill(0, prompt, 3, 8)
    while not a.done:
        ia, ib = sm.df_step(a, 3, 2, eps), sb.df_step(b, 3, 2, eps)
        assert np.abs(ia["logits"] - ib["logits"]).max() < 1e-9
        assert np.array_equal(ia["drafts"], ib["drafts"]) and ia["n_commit"] == ib["n_commit"]
    assert b.done and np.array_equal(a.committed(), b.committed())


def test_one_latent_slot_turns_the_sampler_into_the_sequential_decoder():
    """A pool with a single slot for hidden states (Appendix, "Larger Batch Sizes") leaves one position
    in flight at a time; with the fixed exit it gets `window` steps of r' iterations on its own and is
    then committed, which is the sequential decoder with r = window * r' (Section 3.3's identity),
    token for token, in window steps per token."""
    from helpers import SlotPoolModel
    model, _ = make_oracle(SMALL, seed=4)
    prompt = rd_inputs.make_prompt(7, SMALL["vocab"], seed=9)
    sm = orc.Sampler(model, seed=5)
    pool = SlotPoolModel(1)
    sq = pool.start(sm, 0, prompt, 3, 6)
    steps = 0
    while not sq.done:
        pool.drive(sm, [sq], 4, 2, 0.0)
        assert len(sq.window) <= 1
        steps += 1
    model2, _ = make_oracle(SMALL, seed=4)
    sm2 = orc.Sampler(model2, seed=5)
    sq2 = sm2.prefill(0, prompt, 3, 6)
    sm2.generate_ar(sq2, 8)
    assert np.array_equal(sq.committed(), sq2.committed()) and steps == 6 * 4


def test_a_large_enough_pool_changes_nothing_and_a_small_one_only_delays():
    """With as many slots as batch x window the pooled schedule is the plain sampler; with fewer, every
    sequence still finishes with its full budget and never holds more rows than the window."""
    from helpers import SlotPoolModel
    prompts = [rd_inputs.make_prompt(5 + 2 * b, SMALL["vocab"], seed=b) for b in range(3)]

    def run(n_slots):
        model, _ = make_oracle(SMALL, seed=2)
        sm = orc.Sampler(model, seed=1)
        pool = SlotPoolModel(n_slots)
        seqs = [pool.start(sm, b, prompts[b], 2, 8) for b in range(3)]
        steps = 0
        while not all(sq.done for sq in seqs):
            pool.drive(sm, seqs, 4, 1, 0.0)
            assert sum(len(sq.window) for sq in seqs) <= n_slots and all(len(sq.window) <= 4 for sq in seqs)
            steps += 1
            assert steps < 500
        return [sq.committed() for sq in seqs], steps

    model, _ = make_oracle(SMALL, seed=2)
    sm = orc.Sampler(model, seed=1)
    plain = []
    for b in range(3):
        sq = sm.prefill(b, prompts[b], 2, 8)
        sm.generate_df(sq, 4, 1, 0.0)
        plain.append(sq.committed())
    full, steps_full = run(12)
    assert all(np.array_equal(a, b) for a, b in zip(full, plain)) and steps_full == 8 + 4 - 1
    small, steps_small = run(5)
    assert all(len(t) == len(p) for t, p in zip(small, plain)) and steps_small > steps_full
