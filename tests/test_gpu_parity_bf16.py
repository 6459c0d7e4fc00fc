"""GPU parity, bf16 configurations: reduced-width twin of the 3.5B shape (head_dim 96, 2/4/2 layers)
in lock step with the oracle's bf16-contract mode, and truncated runs at the full 3.5B shape.
Tolerance (stated by the benchmark spec): |err| <= 5e-2 + 2e-2 |want| on latents and logits; tokens identical
except at near-ties of the deciding scores, which are counted and bounded."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model
from helpers import make_oracle

pytestmark = pytest.mark.gpu
TOL = Tolerance(5e-2, 2e-2)
# Two bf16 pipelines that sum in different orders round differently at every bf16 store; the
# resulting noise floor on logits is ~1.5e-2 here (inside the stated tolerance).  A GPU/oracle token
# mismatch is admissible only if the oracle's own score gap between the two tokens is below
# TIE_GAP; top-2 gaps average ~0.3, so a few percent of the arg-max decisions are such near-ties.
TIE_GAP = 3e-2
MAX_TIE_FRACTION = 0.08


def _ties_ok(ls):
    return ls.near_ties <= max(2, int(MAX_TIE_FRACTION * ls.n_drafts))


def _setup(shape, W, max_new, batch=1, temperature=0.0, cap=64, max_ctx=256, seed=0, gemm_path=None,
           dtype=np.float64, std=0.02, **wkw):
    model, w = make_oracle(shape, seed=seed, std=std, gain_jitter=0.0, bf16=True, contract=True, max_ctx=max_ctx,
                           dtype=dtype, **wkw)
    gm = gpu_model(shape, w, bf16=True)
    sess = rd.Session(gm, batch=batch, max_context=max_ctx, max_window=W, max_iters_per_pos=cap,
                      max_new_tokens=max_new, keep_logits=True, temperature=temperature, seed=seed + 7)
    if gemm_path is not None:
        sess.set_gemm_path(gemm_path)      # raises if the tensor-core path is unavailable
    sm = orc.Sampler(model, seed=seed + 7, temperature=temperature, max_iters_per_pos=cap)
    return model, gm, sess, sm


def _prefill_both(sm, sess, shape, lens, r, max_new, seed=0):
    seqs = []
    for b, L in enumerate(lens):
        prompt = rd_inputs.make_prompt(int(L), shape["vocab"], seed=seed + b)
        seqs.append(sm.prefill(b, prompt, r, max_new))
        sess.prefill(b, prompt, r)
    return seqs


def _run(ls, W, inner, eps, max_steps=2000):
    for _ in range(max_steps):
        if ls.all_done():
            break
        ls.df(W, inner, eps)
    assert ls.all_done()
    ls.final_tokens_equal()


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("W,inner,eps,temperature", [(4, 1, 0.0, 0.0), (16, 2, 0.0, 0.0), (8, 1, 1e-3, 0.0),
                                                     (16, 1, 1e-3, 1.0)])
def test_twin_df_modes(path, W, inner, eps, temperature):
    model, gm, sess, sm = _setup(rd_inputs.TWIN, W, 24, temperature=temperature, cap=16, gemm_path=path)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [40], 4, 24)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    _run(ls, W, inner, eps)
    print(f"path {path} W {W}: steps {ls.steps}, near-ties {ls.near_ties}, max err {ls.max_err}")
    assert _ties_ok(ls)
    assert (sess.stats()["tc_gemm_launches"] > 0) == (path == 1)


@pytest.mark.parametrize("path", [0, 1])
def test_twin_ar_and_window1_identity(path):
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 1, 8, gemm_path=path)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [20], 4, 8)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    while not ls.all_done():
        ls.ar(6)
    ls.final_tokens_equal()
    ar_tokens, ar_z = sess.tokens(0).copy(), sess.debug_read(rd.RD_DBG_LATENTS, 0).copy()
    sess2 = rd.Session(gm, batch=1, max_context=256, max_window=1, max_new_tokens=8, keep_logits=True, seed=7)
    sess2.set_gemm_path(path)
    sess2.prefill(0, rd_inputs.make_prompt(20, 4096, seed=0), 4)
    for _ in range(8):
        sess2.df_step(1, 6, 0.0)
    assert np.array_equal(sess2.tokens(0), ar_tokens)
    assert np.array_equal(sess2.debug_read(rd.RD_DBG_LATENTS, 0), ar_z)


@pytest.mark.parametrize("path", [0, 1])
def test_twin_batched_ragged_sampling(path):
    """Batched serving shape: ragged prompts, temperature sampling on the shared counter stream,
    adaptive exit."""
    lens = rd_inputs.make_prompt_lengths(4, 3, 60, seed=3)
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 8, 16, batch=4, temperature=1.0, cap=12, gemm_path=path)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, lens, 3, 16)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    _run(ls, 8, 1, 1e-3)
    assert _ties_ok(ls)


def test_twin_long_prefix_attention():
    """A prompt spanning many attention tiles (long-context shape, reduced width)."""
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 8, 10, max_ctx=1200)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [1100], 1, 10)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    _run(ls, 8, 1, 0.0)
    assert _ties_ok(ls)


def test_gpu_run_to_run_bit_identical():
    """Fixed-order reductions everywhere: two runs give the same bits."""
    outs = []
    for _ in range(2):
        model, gm, sess, sm = _setup(rd_inputs.TWIN, 8, 12)
        sess.prefill(0, rd_inputs.make_prompt(30, 4096, seed=1), 3)
        for _ in range(19):
            sess.df_step(8, 1, 0.0)
        outs.append((sess.tokens(0).copy(), sess.debug_read(rd.RD_DBG_LATENTS, 0).copy(),
                     sess.debug_read(rd.RD_DBG_LOGITS, 0).copy()))
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)


def test_twin_window_64_rows():
    """A 64-row wavefront: the 64-row GEMM tile and the four-query-block attention path in decode.
    A row stays in flight for 64 recurrences here; with the plain random init the recurrence is not
    contractive and bf16 rounding differences between the two sides grow with every pass, so the
    latent's share of the adapter is scaled down (contractive recurrence, as for the convergence pin)."""
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 64, 70, max_ctx=256, adapter_s_scale=0.25)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [50], 2, 70)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    widest = 0
    for _ in range(80):                       # ramp to the full window and a few steps beyond
        if ls.all_done():
            break
        widest = max(widest, len(seqs[0].window))
        ls.df(64, 1, 0.0)
    assert widest == 64
    assert _ties_ok(ls)


@pytest.mark.parametrize("path", [1, 2])
def test_twin_batch_8_window_16_is_128_rows(path):
    """128 rows in flight: the 128-row GEMM tile (path 1: on CTA pairs, 64 rows per CTA; path 2: single
    CTAs), ragged prompts of up to 100 tokens (prefill chunks of 128 rows too), greedy, fixed exit."""
    lens = rd_inputs.make_prompt_lengths(8, 3, 100, seed=4)
    # (a row lives 16 steps here: the weaker feedback keeps rounding noise from growing along the recurrence)
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 16, 20, batch=8, cap=8, max_ctx=160, gemm_path=path, adapter_s_scale=0.25)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, lens, 2, 20)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    for _ in range(22):
        if ls.all_done():
            break
        ls.df(16, 1, 0.0)
    assert _ties_ok(ls)
    assert sess.stats()["tc_gemm_launches"] > 0


@pytest.mark.parametrize("path", [1, 2])
def test_twin_batch_16_window_16_is_256_rows(path):
    """The batched-serving row count: 16 sequences x 16 in-flight rows = the 256-row GEMM tile (path 1:
    on CTA pairs, one MMA of 256 features over two SMs; path 2: on single CTAs), ragged prompts,
    temperature sampling, adaptive exit."""
    lens = rd_inputs.make_prompt_lengths(16, 2, 40, seed=9)
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 16, 20, batch=16, temperature=1.0, cap=8, max_ctx=128, gemm_path=path)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, lens, 2, 20)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    for _ in range(24):
        if ls.all_done():
            break
        ls.df(16, 1, 1e-3)
    assert _ties_ok(ls)
    assert sess.stats()["tc_gemm_launches"] > 0      # no silent fall-back to the plain kernels


def test_twin_window_64_rows_plain_init_first_steps():
    """The 64-row window with the plain random init (no scaling of the adapter): the first 16 steps,
    before rounding differences have had many recurrences to grow."""
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 64, 70, max_ctx=256)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [50], 2, 70)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    for _ in range(16):
        ls.df(64, 1, 0.0)
    assert len(seqs[0].window) == 17 and _ties_ok(ls)


@pytest.mark.parametrize("scale,steps", [(0.25, 140), (1.0, 16)])
def test_twin_window_128_rows(scale, steps):
    """The paper's default maximum wavefront, 128 rows of one sequence: the eight-warp attention
    groups and the 128-row GEMM tile.  The full ramp runs with the contractive adapter (a row stays in
    flight for 128 recurrences), the plain init for the first 16 steps."""
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 128, 140, max_ctx=256, adapter_s_scale=scale)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, [40], 2, 140)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    widest = 0
    for _ in range(steps):
        if ls.all_done():
            break
        ls.df(128, 1, 0.0)
        widest = max(widest, len(seqs[0].window))
    assert widest == min(128, steps + 1)
    assert _ties_ok(ls)
    assert sess.stats()["tc_gemm_launches"] > 0


def test_twin_long_context_batch_4_window_32():
    """The long-context regime: four sequences with prompts of about 4,100 tokens (ragged), a wavefront
    of up to 32 rows each, greedy.  Every head's keys span 65 tiles, cut into 8 splits per (sequence,
    head), and the prefill runs in nine 512-row chunks per sequence.
    Behind a prefix this long the random-init recurrence amplifies rounding differences with every
    step a row stays in flight: the oracle's own float32 and float64 bf16-contract modes drift apart
    by 1.3e-2 per step on the oldest row's latent (6e-2 after six steps) with the plain init.  With the layers'
    matrices halved (exact in bf16) and the contractive adapter of the other wide-window tests that
    drift stays near 3e-2 over 16 steps, so the stated bound can be asked of the first 20 steps
    (21 rows per sequence in flight at the end)."""
    lens = [4096, 4033, 4127, 3970]
    model, gm, sess, sm = _setup(rd_inputs.TWIN, 32, 36, batch=4, max_ctx=4200, adapter_s_scale=0.25, layer_scale=0.5)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, lens, 1, 36)
    # cache rows of the prefill, deep inside the prefix and at its end
    for b, L in ((0, 4096), (3, 3970)):
        for blk, name in enumerate(("prelude", "core", "coda")):
            got = sess.read_kv(blk, 1, 0, b, L - 70, 69)
            want = seqs[b].caches[name].K[1, L - 70:L - 1].reshape(69, -1)
            assert TOL.excess(got, want) <= 0, f"sequence {b} {name} keys off by {np.abs(got - want).max():.3e}"
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    for _ in range(20):
        ls.df(32, 1, 0.0)
    assert all(len(sq.window) == 21 for sq in seqs)
    print(f"near-ties {ls.near_ties} of {ls.n_drafts}, max err {ls.max_err}")
    assert _ties_ok(ls)


@pytest.mark.parametrize("rows", [(1, 4), (4, 8), (8, 16), (16, 16)])
def test_twin_unfused_swiglu_path_and_fused_agree(rows):
    """The gate/up projection with the SwiGLU in its epilogue (default) and with partial sums plus a
    separate kernel: the second is run in lock step with the oracle here (the first everywhere else),
    and the two give the same tokens and latents within the rounding of the different summation order.
    Row counts cover the 16-, 32-, 128- and 256-row tiles."""
    B, W = rows
    lens = rd_inputs.make_prompt_lengths(B, 5, 40, seed=6)
    model, gm, sess, sm = _setup(rd_inputs.TWIN, W, 12, batch=B, cap=8, max_ctx=96, adapter_s_scale=0.25)
    sess.set_fused_swiglu(False)
    seqs = _prefill_both(sm, sess, rd_inputs.TWIN, lens, 2, 12)
    ls = LockStep(sm, sess, seqs, TOL, tie_gap=TIE_GAP)
    for _ in range(10):
        ls.df(W, 1, 0.0)
    assert _ties_ok(ls)
    z_unfused = sess.debug_read(rd.RD_DBG_LATENTS, 0).copy()
    sess2 = rd.Session(gm, batch=B, max_context=96, max_window=W, max_iters_per_pos=8, max_new_tokens=12,
                       keep_logits=True, seed=7)
    for b, L in enumerate(lens):
        sess2.prefill(b, rd_inputs.make_prompt(int(L), rd_inputs.TWIN["vocab"], seed=b), 2)
    for _ in range(10):
        sess2.df_step(W, 1, 0.0)
    z_fused = sess2.debug_read(rd.RD_DBG_LATENTS, 0)
    assert z_fused.shape == z_unfused.shape and np.abs(z_fused - z_unfused).max() < 5e-2


@pytest.mark.parametrize("W,batch,L", [(16, 2, 700), (64, 1, 300), (128, 1, 90)])
def test_attention_paths_agree_bit_for_bit(W, batch, L):
    """K and V through the TMA ring (default, run in lock step with the oracle everywhere else) and
    through cp.async feed the same tensor-core arithmetic in the same order: tokens, latents and cache
    rows must be identical.  Covers the half-tile warps (groups of up to 32 rows), the four-warp and the
    eight-warp groups, several key tiles and splits."""
    shape = rd_inputs.TWIN
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=21, bf16=True, adapter_s_scale=0.25)
    gm = gpu_model(shape, w, bf16=True)
    outs = []
    for path in (2, 1):
        sess = rd.Session(gm, batch=batch, max_context=L + 160, max_window=W, max_new_tokens=W + 12, seed=13, temperature=0.7)
        sess.set_attention_path(path)
        for b in range(batch):
            sess.prefill(b, rd_inputs.make_prompt(L - 37 * b, shape["vocab"], seed=30 + b), 2)
        for _ in range(W + 6):
            sess.df_step(W, 1, 0.0)
        outs.append([sess.tokens(b).copy() for b in range(batch)] + [sess.debug_read(rd.RD_DBG_LATENTS, 0).copy(),
                    sess.read_kv(1, 3, 0, 0, 0, L + 4), sess.read_kv(2, 1, 1, batch - 1, 0, L - 37 * (batch - 1) + 4)])
        sess.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
    gm.close()


@pytest.mark.parametrize("L", [100, 300, 700])
def test_prefill_attention_on_tcgen05_agrees_with_the_mma_sync_kernel(L):
    """Prefill attends 128-row groups with both products on tcgen05 (default; in lock step with the oracle
    wherever a test prefills a bf16 model) or with the windowed mma.sync kernel (path 2).  Same inputs,
    same bf16 rounding of P, different summation order: cache rows agree to bf16 rounding and the tokens
    of a short generation are the same.  Prompts of one, three and six groups, the last one ragged."""
    shape = rd_inputs.TWIN
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=21, bf16=True, adapter_s_scale=0.25)
    gm = gpu_model(shape, w, bf16=True)
    outs = []
    for path in (2, 3):
        sess = rd.Session(gm, batch=1, max_context=L + 64, max_window=4, max_new_tokens=8, seed=13)
        sess.set_attention_path(path)
        sess.prefill(0, rd_inputs.make_prompt(L, shape["vocab"], seed=30), 2)
        kv = [sess.read_kv(blk, l, which, 0, 0, L - 1) for blk, l in ((0, 1), (1, 0), (1, 3), (2, 1)) for which in (0, 1)]
        for _ in range(6):
            sess.df_step(4, 1, 0.0)
        outs.append((kv, sess.tokens(0).copy()))
        sess.close()
    for a, b in zip(outs[0][0], outs[1][0]):
        assert np.abs(a).max() > 0 and TOL.excess(b, a) <= 0 and np.sqrt(np.mean((a - b) ** 2)) < 5e-3
    assert np.array_equal(outs[0][1], outs[1][1])
    gm.close()
