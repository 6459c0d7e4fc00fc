"""CPU oracle for the recurrent-depth model and its samplers.  TEST INFRASTRUCTURE.

This file is the slow, plain statement of what the CUDA library must compute.
Only the test-suite, the smoke check and the benchmark's `cpu_baseline` /
`--impl reference` legs may import it; the product path never does, and this
file imports nothing from the product package.

What follows the paper and where:

* model  e = P(x), s_0 ~ N(0, sigma^2 I), s_i = R(e, s_{i-1}), p = C(s_r)
  -- Section 3.1 (unnumbered display).  R is conditioned on e at every
  iteration (input injection, Section 3.2) through an adapter over
  concat(e, s).
* KV-cache sharing: one K/V entry per (layer, position), holding the most
  recent recurrence -- Section 3.2, "KV Cache Sharing".
* prefill: all prompt positions iterate the recurrence simultaneously --
  Section 3.3, second remark.
* autoregressive sampler -- Section 3.1 display applied token by token.
* diffusion-forcing sampler, fixed exit -- Algorithm 1; adaptive exit --
  Eq. 3 (delta_i and k*) and Algorithm 2; wavefront limiter -- Section 3.5.
* stabilisers: momentum on the conditioning and scheduled latent noise --
  Section 3.4 (both displays) and the two stabiliser steps of Algorithm 1.
* Sample: greedy, temperature, top-p -- Algorithms 1-2 name it; the Appendix
  gives the settings of the evaluation (temperature 0.2, top-p 0.95).

The paper does not print the layer internals; the reading used here (pre-norm
residual layers, RMSNorm, rotary embedding on adjacent pairs, SwiGLU, one
RMSNorm closing the recurrent block, one before the head) is listed with the
other readings in the repository's design notes.

Arithmetic: numpy, in `dtype` (float64 for the small configurations, float32
at the 3.5B shape where float64 weights do not fit).  `contract=True` rounds
to bfloat16 at the points where the bf16 configuration stores or feeds bf16
(GEMM inputs, q, K/V cache); the residual stream, latents, softmax and logits
stay in `dtype`.

Pins (tests/test_oracle_*.py): Philox known-answer vectors; layer math against
an independent per-element loop and against torch's attention on a full causal
sequence; cache against a no-cache recomputation; causality; AR == DF(W=1,
r'=r); first-token identity DF(W, r') vs AR(r = W r'); progress and window
bounds; pass counters of the cost remark; contraction => adaptive DF == AR;
top-p against a hand-worked distribution, a search over all subsets, and the
sampled frequencies.
Parity unpinned: quality of the sampler's text (needs trained weights).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

# --------------------------------------------------------------------------
# Counter-based random numbers (Philox4x32-10, Salmon et al. 2011)
# --------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)

STREAM_INIT_STATE = 0
STREAM_GUMBEL = 1
STREAM_NOISE = 2


def philox4x32_10(ctr, key):
    """Philox4x32 with 10 rounds.  ctr: [...,4] uint32, key: (k0, k1) -> [...,4] uint32."""
    ctr = np.asarray(ctr, dtype=np.uint32)
    c0, c1, c2, c3 = (ctr[..., i].astype(np.uint64) for i in range(4))
    k0 = np.uint64(int(key[0]) & 0xFFFFFFFF)
    k1 = np.uint64(int(key[1]) & 0xFFFFFFFF)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def _draw_blocks(seed, stream, seq, pos, n_blocks):
    """Raw 32-bit words of blocks 0..n_blocks-1 for (stream, seq, pos): [n_blocks, 4]."""
    ctr = np.empty((n_blocks, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(n_blocks, dtype=np.uint32)
    ctr[:, 1] = np.uint32(pos)
    ctr[:, 2] = np.uint32(seq)
    ctr[:, 3] = np.uint32(stream)
    return philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))


def _unit_interval(words):
    """Map 32-bit words to (0,1): u = ((x >> 9) + 1/2) * 2^-23, exact in float32."""
    return ((words >> np.uint32(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def init_state(seed, seq, pos, hidden, sigma, dtype):
    """s_0 ~ N(0, sigma^2 I) for one position (Section 3.1; InitState in Algorithms 1-2).

    Keyed by (seed, sequence, position) only, so that every sampler sees the
    same s_0 at a position.  Element j is output j%4 of block j//4; a block's
    four words (x0..x3) give two Box-Muller pairs: r(u0) cos/sin(2 pi u1) and
    r(u2) cos/sin(2 pi u3), r(u) = sqrt(-2 ln u).
    """
    nb = (hidden + 3) // 4
    u = _unit_interval(_draw_blocks(seed, STREAM_INIT_STATE, seq, pos, nb))
    out = np.empty((nb, 4), dtype=np.float64)
    for a in (0, 2):
        r = np.sqrt(-2.0 * np.log(u[:, a]))
        th = 2.0 * math.pi * u[:, a + 1]
        out[:, a] = r * np.cos(th)
        out[:, a + 1] = r * np.sin(th)
    return (sigma * out.reshape(-1)[:hidden]).astype(dtype)


def latent_noise(seed, seq, pos, step, hidden, sigma, dtype):
    """z_noise of the noise-injection stabiliser (Section 3.4, second display): a fresh N(0, sigma^2 I)
    draw for position `pos` at its `step`-th sampler step.  Same construction as init_state on the
    noise stream; the step index sits in bits 8.. of the counter's stream word."""
    nb = (hidden + 3) // 4
    u = _unit_interval(_draw_blocks(seed, STREAM_NOISE | (int(step) << 8), seq, pos, nb))
    out = np.empty((nb, 4), dtype=np.float64)
    for a in (0, 2):
        r = np.sqrt(-2.0 * np.log(u[:, a]))
        th = 2.0 * math.pi * u[:, a + 1]
        out[:, a] = r * np.cos(th)
        out[:, a + 1] = r * np.sin(th)
    return (sigma * out.reshape(-1)[:hidden]).astype(dtype)


def gumbel_noise(seed, seq, token_pos, vocab):
    """-log(-log u_v), v < vocab, float32; u_v keyed by (seed, sequence, token position, v)."""
    nb = (vocab + 3) // 4
    u = _unit_interval(_draw_blocks(seed, STREAM_GUMBEL, seq, token_pos, nb)).reshape(-1)[:vocab]
    u = u.astype(np.float32)
    return -np.log(-np.log(u))


def nucleus(logits, temperature, top_p):
    """Boolean mask of the tokens top-p sampling keeps (Appendix, sampling settings of the
    evaluation: temperature 0.2, top-p 0.95): tokens in descending order of probability under
    softmax(logits / T) up to and including the first at which the cumulative probability reaches
    top_p; tokens whose logit equals that of the last one kept are kept with it."""
    l = np.asarray(logits).astype(np.float32).astype(np.float64)
    if top_p >= 1.0:
        return np.ones(l.shape[0], dtype=bool)
    q = np.exp((l - l.max()) / float(temperature))
    q /= q.sum()
    order = np.argsort(-l, kind="stable")
    cum = np.cumsum(q[order])
    k = int(np.searchsorted(cum, top_p, side="left"))      # first rank whose cumulative mass >= top_p
    k = min(k, l.shape[0] - 1)
    return l >= l[order[k]]


def sample_token(logits, temperature, seed, seq, token_pos, top_p=1.0):
    """Sample(p) of Algorithms 1-2.  Greedy (temperature 0): arg max, lowest index on ties.
    Otherwise the Gumbel-max form of sampling from softmax(logits / T), decided in float32; with
    top_p < 1 the arg max runs over the tokens of `nucleus` only, which samples from the
    distribution renormalised over them."""
    l32 = np.asarray(logits).astype(np.float32)
    if temperature <= 0.0:
        return int(np.argmax(l32))
    score = l32 / np.float32(temperature) + gumbel_noise(seed, seq, token_pos, l32.shape[0])
    if top_p < 1.0:
        score = np.where(nucleus(l32, temperature, top_p), score, -np.inf)
    return int(np.argmax(score))


# --------------------------------------------------------------------------
# Model
# --------------------------------------------------------------------------
@dataclass
class RDConfig:
    hidden: int
    n_heads: int
    head_dim: int
    mlp_inner: int
    n_prelude: int
    n_core: int
    n_coda: int
    vocab: int
    rope_base: float = 10000.0
    norm_eps: float = 1e-6
    init_sigma: float = 1.0
    tie_embeddings: bool = True


def bf16_round(x):
    """Round to the nearest bfloat16 (ties to even), result in x's dtype."""
    x = np.asarray(x)
    u = x.astype(np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(x.dtype)


def rmsnorm(x, g, eps):
    """g * x / sqrt(mean(x^2) + eps), row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return g * (x / np.sqrt(ms + eps))


def rope_tables(max_pos, head_dim, base):
    """cos/sin of pos * base^(-2i/d), i < d/2: computed in double, stored as float32."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv = base ** (-2.0 * i / head_dim)
    ang = np.arange(max_pos, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def rope(x, pos, cos, sin):
    """Rotate adjacent pairs (2i, 2i+1) of every head by the position's angle.  x: [n,H,d]."""
    c = cos[pos][:, None, :].astype(x.dtype)
    s = sin[pos][:, None, :].astype(x.dtype)
    x0, x1 = x[..., 0::2], x[..., 1::2]
    out = np.empty_like(x)
    out[..., 0::2] = x0 * c - x1 * s
    out[..., 1::2] = x0 * s + x1 * c
    return out


class KVCache:
    """K and V of one block: [layer, position, head, dim]; a position's entry is overwritten by
    its most recent pass (KV-cache sharing, Section 3.2)."""

    def __init__(self, n_layers, max_ctx, n_heads, head_dim, dtype):
        self.K = np.zeros((n_layers, max_ctx, n_heads, head_dim), dtype=dtype)
        self.V = np.zeros((n_layers, max_ctx, n_heads, head_dim), dtype=dtype)


class RDModel:
    def __init__(self, cfg: RDConfig, weights: dict, dtype=np.float64, contract=False,
                 max_ctx=4096):
        self.cfg = cfg
        self.dtype = np.dtype(dtype)
        self.contract = contract
        self.w = {k: np.asarray(v).astype(dtype, copy=False) for k, v in weights.items()}
        if cfg.tie_embeddings:
            self.w["head"] = self.w["emb"]
        self.cos, self.sin = rope_tables(max_ctx, cfg.head_dim, cfg.rope_base)
        self.max_ctx = max_ctx
        self.row_passes = {"prelude": 0, "core": 0, "coda": 0}

    def _q(self, x):
        return bf16_round(x) if self.contract else x

    def new_caches(self):
        c = self.cfg
        return {b: KVCache(n, self.max_ctx, c.n_heads, c.head_dim, self.dtype)
                for b, n in (("prelude", c.n_prelude), ("core", c.n_core), ("coda", c.n_coda))}

    def layer(self, blk, l, x, pos, cache: KVCache):
        """One pre-norm transformer layer over rows `x` [n,h] of ONE sequence at positions `pos`.

        Every row first overwrites its own K/V entry, then row at position p attends entries
        0..p (causal: information flows left to right only)."""
        c, w, p = self.cfg, self.w, f"{blk}.{l}."
        n, H, d = x.shape[0], c.n_heads, c.head_dim
        a = self._q(rmsnorm(x, w[p + "g1"], c.norm_eps))
        q = (a @ w[p + "wq"].T).reshape(n, H, d)
        k = (a @ w[p + "wk"].T).reshape(n, H, d)
        v = (a @ w[p + "wv"].T).reshape(n, H, d)
        q = self._q(rope(q, pos, self.cos, self.sin))
        k = self._q(rope(k, pos, self.cos, self.sin))
        v = self._q(v)
        cache.K[l, pos] = k
        cache.V[l, pos] = v
        o = np.empty((n, H, d), dtype=self.dtype)
        scale = 1.0 / math.sqrt(d)
        for i in range(n):
            m = int(pos[i]) + 1
            s = np.einsum("hd,mhd->hm", q[i], cache.K[l, :m]) * scale
            s = s - s.max(axis=1, keepdims=True)
            pr = np.exp(s)
            pr = pr / pr.sum(axis=1, keepdims=True)
            o[i] = np.einsum("hm,mhd->hd", pr, cache.V[l, :m])
        x = x + self._q(o.reshape(n, H * d)) @ w[p + "wo"].T
        m2 = self._q(rmsnorm(x, w[p + "g2"], c.norm_eps))
        g = m2 @ w[p + "wg"].T
        u = m2 @ w[p + "wu"].T
        act = self._q((g / (1.0 + np.exp(-g))) * u)
        return x + act @ w[p + "wd"].T

    def prelude(self, tokens, pos, caches):
        """e = P(x)."""
        x = self.w["emb"][np.asarray(tokens)]
        for l in range(self.cfg.n_prelude):
            x = self.layer("prelude", l, x, pos, caches["prelude"])
        self.row_passes["prelude"] += len(pos)
        return x

    def core(self, e, s, pos, caches):
        """s' = R(e, s): adapter over concat(e, s), the core layers, one closing RMSNorm."""
        x = self._q(np.concatenate([e, s], axis=1)) @ self.w["adapter"].T
        for l in range(self.cfg.n_core):
            x = self.layer("core", l, x, pos, caches["core"])
        self.row_passes["core"] += len(pos)
        return rmsnorm(x, self.w["g_core"], self.cfg.norm_eps)

    def coda(self, s, pos, caches, head=True):
        """logits of p = C(s) (softmax left to the sampler)."""
        x = s
        for l in range(self.cfg.n_coda):
            x = self.layer("coda", l, x, pos, caches["coda"])
        self.row_passes["coda"] += len(pos)
        if not head:
            return None
        return self._q(rmsnorm(x, self.w["g_final"], self.cfg.norm_eps)) @ self.w["head"].T


# --------------------------------------------------------------------------
# Samplers
# --------------------------------------------------------------------------
@dataclass
class Row:
    """One in-flight position of the wavefront."""
    pos: int
    z: np.ndarray
    steps: int = 0      # sampler steps this position has taken
    iters: int = 0      # core iterations this position has taken (steps * r')
    e_prev: object = None   # input conditioning e this position used in the previous step (momentum)


@dataclass
class Sequence:
    """Generation state of one sequence: y_current (committed tokens followed by drafts), the
    number of frozen tokens |y_frozen|, the wavefront, and the three caches."""
    seq_id: int
    tokens: np.ndarray
    n_prompt: int
    n_committed: int
    max_new: int
    caches: dict
    window: list = field(default_factory=list)
    done: bool = False

    def committed(self):
        return self.tokens[: self.n_committed].copy()


class Sampler:
    def __init__(self, model: RDModel, seed=0, temperature=0.0, max_iters_per_pos=64, eta=0.0, beta=0.0, top_p=1.0):
        """eta: momentum on the input conditioning, e = eta e_prev + (1 - eta) P(y_current)
        (Section 3.4, first display); a position's first step has no e_prev and takes P(.) as is.
        beta: latent noise, z' = (1 - beta_t) z + beta_t z_noise (second display), beta_t falling
        linearly with the steps t a position has taken: beta_t = beta max(0, 1 - t / T), T the
        number of steps a position gets (the window when the exit is fixed, cap / r' otherwise)."""
        self.m = model
        self.seed = seed
        self.temperature = temperature
        self.cap = max_iters_per_pos
        self.eta = eta
        self.beta = beta
        self.top_p = top_p

    def _init(self, seq_id, pos):
        c = self.m.cfg
        return init_state(self.seed, seq_id, pos, c.hidden, c.init_sigma, self.m.dtype)

    def _sample(self, logits, seq_id, token_pos):
        return sample_token(logits, self.temperature, self.seed, seq_id, token_pos, self.top_p)

    def prefill(self, seq_id, prompt, r, max_new, first_row=True):
        """Section 3.3: the prompt's positions 0..L-2 run P, r simultaneous passes of R and the
        coda layers (to fill its cache).  Position L-1 becomes the first in-flight position with
        a fresh state (the initialisation steps of Algorithm 1); first_row=False leaves the
        wavefront empty (no slot free for its hidden state yet, see df_step's may_append)."""
        prompt = np.asarray(prompt, dtype=np.int64)
        L = len(prompt)
        assert L >= 1 and L + max_new <= self.m.max_ctx
        tokens = np.zeros(L + max_new + 1, dtype=np.int64)
        tokens[:L] = prompt
        sq = Sequence(seq_id, tokens, L, L, max_new, self.m.new_caches())
        if L > 1:
            pos = np.arange(L - 1)
            e = self.m.prelude(prompt[:-1], pos, sq.caches)
            s = np.stack([self._init(seq_id, p) for p in pos])
            for _ in range(r):
                s = self.m.core(e, s, pos, sq.caches)
            self.m.coda(s, pos, sq.caches, head=False)
        sq.window = [Row(L - 1, self._init(seq_id, L - 1))] if first_row else []
        sq.done = max_new <= 0
        if sq.done:
            sq.window = []
        return sq

    def ar_step(self, sq: Sequence, r):
        """One token of the sequential sampler: e = P(x), s_0, r times s = R(e, s), p = C(s_r)."""
        if sq.done:
            return None
        assert len(sq.window) == 1 and sq.window[0].steps == 0, "AR step inside an open wavefront"
        row = sq.window[0]
        pos = np.array([row.pos])
        e = self.m.prelude(sq.tokens[pos], pos, sq.caches)
        s = row.z[None, :]
        for _ in range(r):
            s = self.m.core(e, s, pos, sq.caches)
        logits = self.m.coda(s, pos, sq.caches)
        tok = self._sample(logits[0], sq.seq_id, row.pos + 1)
        sq.tokens[row.pos + 1] = tok
        sq.n_committed += 1
        info = {"pos": pos, "z": s.copy(), "logits": logits, "drafts": np.array([tok]), "n_commit": 1}
        if sq.n_committed - sq.n_prompt >= sq.max_new:
            sq.done, sq.window = True, []
        else:
            sq.window = [Row(row.pos + 1, self._init(sq.seq_id, row.pos + 1))]
        return info

    def df_step(self, sq: Sequence, window, inner_iters, exit_threshold, may_append=True):
        """One step of the diffusion-forcing sampler (Algorithm 1 when exit_threshold <= 0,
        Algorithm 2 otherwise).  Returns what the step computed, for inspection.

        may_append=False: the engine has no slot for a further hidden state this step (Appendix,
        "Larger Batch Sizes": a bounded number of slots shared by the sequences), so the wavefront is
        not extended, exactly as when it is full (Section 3.5); nothing else changes.  A sequence may
        then hold no in-flight position at all: the step computes nothing for it and only appends."""
        if sq.done:
            return None
        rows = sq.window
        assert len(rows) <= window
        if not rows:
            info = {"pos": np.zeros(0, dtype=np.int64), "z": np.zeros((0, self.m.cfg.hidden), dtype=self.m.dtype),
                    "logits": np.zeros((0, self.m.cfg.vocab), dtype=self.m.dtype), "drafts": np.zeros(0, dtype=np.int64),
                    "delta": np.zeros(0, dtype=np.float32), "n_commit": 0}
            if may_append:
                nxt = sq.n_committed - 1
                sq.window.append(Row(nxt, self._init(sq.seq_id, nxt)))
            return info
        pos = np.array([r_.pos for r_ in rows])
        # e <- P(y_current): the oldest row reads the last committed token, the others the
        # drafts of the previous step.
        e = self.m.prelude(sq.tokens[pos], pos, sq.caches)
        if self.eta > 0.0:                                # momentum on the conditioning
            e = e.copy()
            for i, r_ in enumerate(rows):
                if r_.e_prev is not None:
                    e[i] = np.float32(self.eta) * r_.e_prev + np.float32(1.0 - self.eta) * e[i]
                r_.e_prev = e[i].copy()
        z_prev = np.stack([r_.z for r_ in rows])
        z = z_prev
        if self.beta > 0.0:                               # noise injection, less of it at later steps
            c = self.m.cfg
            T = window if exit_threshold <= 0 else -(-self.cap // inner_iters)
            z = z.copy()
            for i, r_ in enumerate(rows):
                bt = np.float32(self.beta * max(0.0, 1.0 - r_.steps / T))
                noise = latent_noise(self.seed, sq.seq_id, r_.pos, r_.steps, c.hidden, c.init_sigma, self.m.dtype)
                z[i] = (np.float32(1.0) - bt) * z[i] + bt * noise
        for _ in range(inner_iters):                      # inner recurrence
            z = self.m.core(e, z, pos, sq.caches)
        logits = self.m.coda(z, pos, sq.caches)           # every in-flight row yields a draft
        drafts = np.array([self._sample(logits[i], sq.seq_id, int(pos[i]) + 1)
                           for i in range(len(rows))])
        sq.tokens[pos + 1] = drafts                        # y_current <- [y_frozen, y_hat]
        # Eq. 3, decided in float32 like the kernel.
        z32, zp32 = z.astype(np.float32), z_prev.astype(np.float32)
        num = np.sqrt(np.sum((z32 - zp32) ** 2, axis=1, dtype=np.float32))
        den = np.sqrt(np.sum(z32 ** 2, axis=1, dtype=np.float32))
        delta = np.where(den > 0, num / np.where(den > 0, den, 1), np.inf).astype(np.float32)
        freezable = []
        for i, r_ in enumerate(rows):
            r_.z = z[i]
            r_.steps += 1
            r_.iters += inner_iters
            if exit_threshold <= 0:
                freezable.append(r_.steps >= window)
            else:
                freezable.append(bool(delta[i] < np.float32(exit_threshold)) or r_.iters >= self.cap)
        k = 0                                              # k*: longest all-freezable prefix
        while k < len(rows) and freezable[k]:
            k += 1
        k = min(k, sq.max_new - (sq.n_committed - sq.n_prompt))
        sq.n_committed += k
        sq.window = rows[k:]
        info = {"pos": pos, "z": z.copy(), "logits": logits, "drafts": drafts, "delta": delta,
                "n_commit": k}
        last_row_pos = sq.n_prompt + sq.max_new - 2       # its draft is the last token wanted
        if sq.n_committed - sq.n_prompt >= sq.max_new:
            sq.done, sq.window = True, []
        elif len(sq.window) < window and may_append:
            nxt = sq.n_committed - 1 + len(sq.window)
            if nxt <= last_row_pos:
                sq.window.append(Row(nxt, self._init(sq.seq_id, nxt)))
        return info

    def force_draft(self, sq: Sequence, token_pos, token):
        """Overwrite the draft (or the just-committed token) at `token_pos`; used by lock-step
        tests to follow the other side through an admissible near-tie."""
        sq.tokens[token_pos] = token

    def generate_ar(self, sq, r):
        n = 0
        while not sq.done:
            self.ar_step(sq, r)
            n += 1
        return n

    def generate_df(self, sq, window, inner_iters, exit_threshold, max_steps=1 << 30):
        n = 0
        while not sq.done and n < max_steps:
            self.df_step(sq, window, inner_iters, exit_threshold)
            n += 1
        return n
