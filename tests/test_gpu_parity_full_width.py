"""GPU parity at the full widths of the 3.5B shape (hidden 5280 = 55 x 96, MLP 17920, vocabulary
65536; one layer per block so that the oracle finishes in seconds), bf16, with the 32-row wavefront
the benchmark times: every GEMM shape, the 32-row tile of the tensor-core kernel and its partial-sum
consumers run as they do in the benchmark, in lock step with the oracle's bf16-contract mode.

Tolerances.  Latents: the stated bound |err| <= 5e-2 + 2e-2 |want| on every element.  Logits: at
these widths the bound cannot hold element by element for ANY bf16 evaluation: the oracle's own
bf16-contract and float32 modes differ by rms 3.0e-2 on the logits (rms 1.46) with 3 % of the 65536
entries outside the bound, because the random-init MLP (output rms 2.1 on a residual of rms 1)
amplifies rounding noise about 2.5 x per layer.  So the logits are bounded statistically: rms error
<= 3.5e-2, at most 3 % of the entries outside the element-wise bound, largest error <= 0.2 (measured:
rms 2.4e-2, 1 %, 0.12).  Tokens: a mismatch is admissible when the oracle's own gap between the two
tokens is below 0.08 (the difference of two logits that each carry the measured rms noise of 2.4e-2
has a standard deviation of 3.4e-2; 0.08 is 2.4 of those); top-2 gaps of 65536 random logits are
~0.3, so such near-ties are frequent here (bounded at 12 % of the drafts).  The element-wise bound
itself is checked at these widths by the one-layer test below.
Also: launching a step as a programmatic-dependent-launch chain or as ordinary launches gives the
same bits."""
import numpy as np
import pytest

import paper_2510_14961_b200 as rd
import rd_inputs
from oracle import rd_oracle as orc
from gpu_harness import LockStep, Tolerance, gpu_model

pytestmark = pytest.mark.gpu

FULL_WIDTH = dict(rd_inputs.SHAPE_3P5B, n_prelude=1, n_core=1, n_coda=1)


def test_full_width_df_window_32_lock_step():
    shape = FULL_WIDTH
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=11, bf16=True)
    W, N, L = 32, 36, 24
    om = orc.RDModel(orc.RDConfig(**shape), w, dtype=np.float32, contract=True, max_ctx=L + N + 8)
    gm = gpu_model(shape, w, bf16=True)
    sess = rd.Session(gm, batch=1, max_context=L + N + 8, max_window=W, max_new_tokens=N, keep_logits=True, seed=3)
    sm = orc.Sampler(om, seed=3)
    prompt = rd_inputs.make_prompt(L, shape["vocab"], seed=5)
    seqs = [sm.prefill(0, prompt, 2, N)]
    sess.prefill(0, prompt, 2)
    ls = LockStep(sm, sess, seqs, Tolerance(5e-2, 2e-2), tie_gap=0.08, logit_noise=(3.5e-2, 0.03, 0.2))
    while not ls.all_done():
        ls.df(W, 1, 0.0)
    ls.final_tokens_equal()
    print(f"steps {ls.steps}, drafts {ls.n_drafts}, near-ties {ls.near_ties}, max err {ls.max_err}")
    assert ls.near_ties <= max(2, int(0.12 * ls.n_drafts))
    st = sess.stats()
    assert st["tc_gemm_launches"] > 0
    sess.close()
    gm.close()


@pytest.mark.parametrize("eps,cap", [(0.0, 64), (1e-3, 3)])
def test_full_width_one_layer_every_logit_within_the_stated_bound(eps, cap):
    """The stated bf16 tolerance, |err| <= 5e-2 + 2e-2 |want|, on EVERY latent and EVERY logit at the
    full widths (reductions over 5280, 10560 and 17920, vocabulary 65536) with the 32-row GEMM tile:
    8 sequences x a 4-row window, one core layer, no prelude or coda layers.  Rounding noise between
    two bf16 evaluations grows with every layer and every recurrence a row goes through (the
    oracle's own float32 and float64 contract modes drift apart by rms 3e-3 .. 8e-3 on the logits over
    a row's first eight recurrences at these widths), so the element-wise bound can only be asked of
    a short path: here a row sees one layer and at most four recurrences, and the layer's matrices
    are halved (exact in bf16) so that the layer adds less noise to its residual stream.  A wrong
    head, adapter or projection at these shapes shows up element-wise here.
    Second case: the adaptive exit (Eq. 3) in lock step at these widths: delta over 5280 features is
    compared every step, and since a random-init recurrence does not converge to 1e-3, every position
    is committed by the iteration cap (3) under the prefix rule."""
    shape = dict(rd_inputs.SHAPE_3P5B, n_prelude=0, n_core=1, n_coda=0)
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=12, bf16=True, layer_scale=0.5)
    B, W, N = 8, 4, 6
    lens = [int(x) for x in rd_inputs.make_prompt_lengths(B, 3, 14, seed=2)]
    max_ctx = max(lens) + N + 8
    om = orc.RDModel(orc.RDConfig(**shape), w, dtype=np.float32, contract=True, max_ctx=max_ctx)
    gm = gpu_model(shape, w, bf16=True)
    sess = rd.Session(gm, batch=B, max_context=max_ctx, max_window=W, max_new_tokens=N, keep_logits=True, seed=4,
                      max_iters_per_pos=cap)
    sm = orc.Sampler(om, seed=4, max_iters_per_pos=cap)
    seqs = []
    for b in range(B):
        prompt = rd_inputs.make_prompt(lens[b], shape["vocab"], seed=6 + b)
        seqs.append(sm.prefill(b, prompt, 2, N))
        sess.prefill(b, prompt, 2)
    ls = LockStep(sm, sess, seqs, Tolerance(5e-2, 2e-2), tie_gap=3e-2)
    while not ls.all_done():
        ls.df(W, 1, eps)
    ls.final_tokens_equal()
    print(f"steps {ls.steps}, drafts {ls.n_drafts}, near-ties {ls.near_ties}, max err {ls.max_err}")
    assert ls.steps == N + (W if eps <= 0 else cap) - 1
    assert ls.near_ties <= max(2, int(0.08 * ls.n_drafts))
    assert sess.stats()["tc_gemm_launches"] > 0
    sess.close()
    gm.close()


def test_chained_and_plain_launches_give_the_same_bits():
    shape = rd_inputs.TWIN
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=2, bf16=True)
    gm = gpu_model(shape, w, bf16=True)
    outs = []
    for chained in (True, False):
        sess = rd.Session(gm, batch=2, max_context=128, max_window=8, max_new_tokens=20, keep_logits=True,
                          temperature=1.0, seed=9)
        sess.set_launch_chaining(chained)
        for b, L in enumerate((33, 17)):
            sess.prefill(b, rd_inputs.make_prompt(L, shape["vocab"], seed=b), 3)
        for _ in range(30):
            sess.df_step(8, 2, 1e-3)
        outs.append([sess.tokens(b).copy() for b in range(2)] + [sess.debug_read(rd.RD_DBG_LATENTS, 0).copy()]
                    + [sess.read_kv(1, 2, 0, 1, 0, 30)])
        sess.close()
    for a, b in zip(*outs):
        assert np.array_equal(a, b)
    gm.close()
