"""Pins for the oracle's layer math: textbook routines, an independent per-element loop, torch's
causal attention on a full sequence, and a no-cache recomputation of the KV cache."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import rd_oracle as orc
from helpers import MICRO, SMALL, make_oracle


def test_rmsnorm_unit_rms_and_gain():
    x = np.random.default_rng(0).standard_normal((5, 64)) * 7
    y = orc.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt((y ** 2).mean(axis=1)), 1.0)
    g = np.linspace(0.5, 2, 64)
    assert np.allclose(orc.rmsnorm(x, g, 0.0), y * g)
    # eps sits inside the square root, added to the mean square
    assert np.allclose(orc.rmsnorm(np.zeros((1, 4)) + 2.0, np.ones(4), 5.0), 2.0 / 3.0)


def test_rope_is_a_rotation_and_relative():
    cos, sin = orc.rope_tables(64, 8, 10000.0)
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal((1, 1, 8)), rng.standard_normal((1, 1, 8))
    for p in (0, 3, 17):
        rq = orc.rope(q, np.array([p]), cos, sin)
        assert np.allclose(np.linalg.norm(rq), np.linalg.norm(q), atol=1e-6)
    assert np.allclose(orc.rope(q, np.array([0]), cos, sin), q)
    d1 = (orc.rope(q, np.array([9]), cos, sin) * orc.rope(k, np.array([4]), cos, sin)).sum()
    d2 = (orc.rope(q, np.array([25]), cos, sin) * orc.rope(k, np.array([20]), cos, sin)).sum()
    assert abs(d1 - d2) < 1e-5
    # pair (0,1) turns by pos radians (frequency base^0 = 1), counter-clockwise
    e0 = np.zeros((1, 1, 8)); e0[0, 0, 0] = 1
    r = orc.rope(e0, np.array([2]), cos, sin)[0, 0]
    assert np.allclose(r[:2], [math.cos(2), math.sin(2)], atol=1e-6) and np.allclose(r[2:], 0)
    # pair i uses base^(-2i/d)
    e2 = np.zeros((1, 1, 8)); e2[0, 0, 4] = 1
    r = orc.rope(e2, np.array([3]), cos, sin)[0, 0]
    ang = 3 * 10000.0 ** (-4 / 8)
    assert np.allclose(r[4:6], [math.cos(ang), math.sin(ang)], atol=1e-6)


def test_bf16_round_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -9, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -9, -3.14159], dtype=np.float32)
    y = orc.bf16_round(x)
    # bf16 has 8 significant bits: spacing 2^-7 at 1.0; 1+2^-8 is a tie -> even (1.0);
    # 1+3*2^-9 rounds up to 1+2^-7
    assert y[0] == 1.0 and y[1] == 1.0 and y[2] == 1.0 and y[3] == 1.0 + 2 ** -7
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(y, t)
    big = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    assert np.array_equal(orc.bf16_round(big),
                          torch.from_numpy(big).to(torch.bfloat16).to(torch.float32).numpy())


def _loop_layer(model, blk, l, x, pos, K, V):
    """Per-element restatement of one layer in pure Python floats.  K, V: dict pos -> [H][d]."""
    c, w, p = model.cfg, model.w, f"{blk}.{l}."
    h, H, d, I = c.hidden, c.n_heads, c.head_dim, c.mlp_inner
    n = len(pos)

    def norm(vec, g):
        ms = sum(t * t for t in vec) / len(vec)
        return [g[j] * vec[j] / math.sqrt(ms + c.norm_eps) for j in range(len(vec))]

    def matvec(W, vec):
        return [sum(W[o][j] * vec[j] for j in range(len(vec))) for o in range(len(W))]

    def rot(vec, ps):
        out = list(vec)
        for hh in range(H):
            for i in range(d // 2):
                ang = ps * c.rope_base ** (-2.0 * i / d)
                a, b = vec[hh * d + 2 * i], vec[hh * d + 2 * i + 1]
                out[hh * d + 2 * i] = a * math.cos(ang) - b * math.sin(ang)
                out[hh * d + 2 * i + 1] = a * math.sin(ang) + b * math.cos(ang)
        return out

    xs = [list(map(float, x[i])) for i in range(n)]
    qs = []
    for i in range(n):
        a = norm(xs[i], w[p + "g1"])
        qs.append(rot(matvec(w[p + "wq"], a), int(pos[i])))
        K[int(pos[i])] = rot(matvec(w[p + "wk"], a), int(pos[i]))
        V[int(pos[i])] = matvec(w[p + "wv"], a)
    out = []
    for i in range(n):
        o = [0.0] * h
        for hh in range(H):
            sc = [sum(qs[i][hh * d + t] * K[j][hh * d + t] for t in range(d)) / math.sqrt(d)
                  for j in range(int(pos[i]) + 1)]
            mx = max(sc)
            ex = [math.exp(s - mx) for s in sc]
            tot = sum(ex)
            for t in range(d):
                o[hh * d + t] = sum(ex[j] / tot * V[j][hh * d + t] for j in range(len(sc)))
        y = [xs[i][j] + v for j, v in enumerate(matvec(w[p + "wo"], o))]
        m2 = norm(y, w[p + "g2"])
        g, u = matvec(w[p + "wg"], m2), matvec(w[p + "wu"], m2)
        act = [g[j] / (1 + math.exp(-g[j])) * u[j] for j in range(I)]
        out.append([y[j] + v for j, v in enumerate(matvec(w[p + "wd"], act))])
    return np.array(out)


def test_layer_against_per_element_loop():
    model, _ = make_oracle(MICRO, std=0.3, max_ctx=16)
    rng = np.random.default_rng(2)
    caches = model.new_caches()
    K, V = {}, {}
    # first call fills positions 0..3, second refines 2..4 (overwrite + append), as a wavefront does
    for pos in (np.arange(4), np.array([2, 3, 4])):
        x = rng.standard_normal((len(pos), 16))
        got = model.layer("core", 1, x, pos, caches["core"])
        want = _loop_layer(model, "core", 1, x, pos, K, V)
        # the oracle's rotary tables are rounded to float32 (6e-8); nothing else differs
        assert np.abs(got - want).max() < 5e-7


def _torch_forward(model, tokens, r, s0):
    """Full-sequence forward with torch building blocks: every position at once, causal mask."""
    c = model.cfg
    w = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in model.w.items()}
    n, H, d = len(tokens), c.n_heads, c.head_dim
    inv = torch.tensor([c.rope_base ** (-2.0 * i / d) for i in range(d // 2)], dtype=torch.float64)
    ang = torch.arange(n, dtype=torch.float64)[:, None] * inv[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)          # e^{i pos theta}

    def rope(t):                                         # complex multiplication of adjacent pairs
        tc = torch.view_as_complex(t.reshape(n, H, d // 2, 2).contiguous())
        return torch.view_as_real(tc * rot[:, None, :]).reshape(n, H, d)

    def layer(blk, l, x):
        p = f"{blk}.{l}."
        a = F.rms_norm(x, (c.hidden,), w[p + "g1"], c.norm_eps)
        q = rope(F.linear(a, w[p + "wq"]).reshape(n, H, d)).transpose(0, 1)
        k = rope(F.linear(a, w[p + "wk"]).reshape(n, H, d)).transpose(0, 1)
        v = F.linear(a, w[p + "wv"]).reshape(n, H, d).transpose(0, 1)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(0, 1).reshape(n, H * d)
        x = x + F.linear(o, w[p + "wo"])
        m = F.rms_norm(x, (c.hidden,), w[p + "g2"], c.norm_eps)
        return x + F.linear(F.silu(F.linear(m, w[p + "wg"])) * F.linear(m, w[p + "wu"]), w[p + "wd"])

    x = F.embedding(torch.as_tensor(tokens), w["emb"])
    for l in range(c.n_prelude):
        x = layer("prelude", l, x)
    e, s = x, torch.from_numpy(s0)
    for _ in range(r):
        x = F.linear(torch.cat([e, s], dim=1), w["adapter"])
        for l in range(c.n_core):
            x = layer("core", l, x)
        s = F.rms_norm(x, (c.hidden,), w["g_core"], c.norm_eps)
    x = s
    for l in range(c.n_coda):
        x = layer("coda", l, x)
    return s.numpy(), F.linear(F.rms_norm(x, (c.hidden,), w["g_final"], c.norm_eps), w["head"]).numpy()


def test_model_against_torch_full_sequence():
    model, _ = make_oracle(SMALL, std=0.08, max_ctx=32)
    tokens = np.random.default_rng(3).integers(0, 128, size=12)
    pos = np.arange(12)
    s0 = np.random.default_rng(4).standard_normal((12, 64))
    caches = model.new_caches()
    e = model.prelude(tokens, pos, caches)
    s = s0
    for _ in range(3):
        s = model.core(e, s, pos, caches)
    logits = model.coda(s, pos, caches)
    s_t, logits_t = _torch_forward(model, tokens, 3, s0)
    assert np.abs(s - s_t).max() < 5e-7
    assert np.abs(logits - logits_t).max() < 5e-7


def test_incremental_cache_equals_full_sequence():
    """Feeding positions one at a time through the cache gives what the full causal pass gives
    (one pass per block, so each position's K/V is final when later positions read it)."""
    model, _ = make_oracle(SMALL, std=0.08, max_ctx=32)
    tokens = np.random.default_rng(5).integers(0, 128, size=9)
    s0 = np.random.default_rng(6).standard_normal((9, 64))
    full = model.new_caches()
    pos = np.arange(9)
    lf = model.coda(model.core(model.prelude(tokens, pos, full), s0, pos, full), pos, full)
    inc = model.new_caches()
    for p in range(9):
        pp = np.array([p])
        li = model.coda(model.core(model.prelude(tokens[pp], pp, inc), s0[pp], pp, inc), pp, inc)
        assert np.abs(li[0] - lf[p]).max() < 1e-10
    # chunks of rows (a wavefront) behave the same
    ch = model.new_caches()
    for lo, hi in ((0, 4), (4, 9)):
        pp = np.arange(lo, hi)
        lc = model.coda(model.core(model.prelude(tokens[pp], pp, ch), s0[pp], pp, ch), pp, ch)
        assert np.abs(lc - lf[lo:hi]).max() < 1e-10


def test_contract_mode_rounds_only_where_stated():
    """With bf16-valued weights, contract mode stays within bf16 resolution of the plain mode and
    its cache holds exactly representable bf16 values."""
    plain, w = make_oracle(SMALL, std=0.08, bf16=True, max_ctx=32)
    contr = orc.RDModel(plain.cfg, w, dtype=np.float64, contract=True, max_ctx=32)
    tokens = np.random.default_rng(7).integers(0, 128, size=6)
    pos = np.arange(6)
    s0 = np.random.default_rng(8).standard_normal((6, 64))
    c1, c2 = plain.new_caches(), contr.new_caches()
    l1 = plain.coda(plain.core(plain.prelude(tokens, pos, c1), s0, pos, c1), pos, c1)
    l2 = contr.coda(contr.core(contr.prelude(tokens, pos, c2), s0, pos, c2), pos, c2)
    assert 0 < np.abs(l1 - l2).max() < 0.05
    k = c2["core"].K[:, :6]
    assert np.array_equal(k, orc.bf16_round(k))
    assert not np.array_equal(c1["core"].K[:, :6], orc.bf16_round(c1["core"].K[:, :6]))
