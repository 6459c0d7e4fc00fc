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
tokens is below 0.12 = 5 x the measured rms noise; top-2 gaps of 65536 random logits are ~0.3, so
such near-ties are frequent here (bounded at 20 % of the drafts).
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
    ls = LockStep(sm, sess, seqs, Tolerance(5e-2, 2e-2), tie_gap=0.12, logit_noise=(3.5e-2, 0.03, 0.2))
    while not ls.all_done():
        ls.df(W, 1, 0.0)
    ls.final_tokens_equal()
    print(f"steps {ls.steps}, drafts {ls.n_drafts}, near-ties {ls.near_ties}, max err {ls.max_err}")
    assert ls.near_ties <= max(2, int(0.20 * ls.n_drafts))
    st = sess.stats()
    assert st["tc_gemm_launches"] > 0
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
