"""Shared test helpers: small model shapes and oracle construction."""
import numpy as np

import rd_inputs
from oracle import rd_oracle as orc

MICRO = dict(hidden=16, n_heads=2, head_dim=8, mlp_inner=24, n_prelude=1, n_core=2, n_coda=1, vocab=32)
SMALL = dict(hidden=64, n_heads=2, head_dim=32, mlp_inner=96, n_prelude=1, n_core=2, n_coda=1, vocab=128)


def oracle_config(shape, **kw):
    return orc.RDConfig(**shape, **kw)


def make_oracle(shape, seed=0, std=0.02, gain_jitter=0.1, dtype=np.float64, contract=False,
                bf16=False, max_ctx=256, adapter_s_scale=1.0, layer_scale=1.0, **cfg_kw):
    w = rd_inputs.make_weights(**rd_inputs.shape_args(shape), seed=seed, std=std,
                               gain_jitter=gain_jitter, bf16=bf16, adapter_s_scale=adapter_s_scale,
                               layer_scale=layer_scale)
    model = orc.RDModel(oracle_config(shape, **cfg_kw), w, dtype=dtype, contract=contract,
                        max_ctx=max_ctx)
    return model, w


class SlotPoolModel:
    """Host-side model of the engine's pool of latent slots (counts only): after every step the rows
    that left return their slots (all sequences first), then the sequences that want to extend their
    wavefront take free slots in index order.  drive() runs one oracle step of every sequence under
    that policy and returns the per-sequence infos."""

    def __init__(self, n_slots):
        self.free = n_slots

    def start(self, sampler, seq_id, prompt, r, max_new, old=None):
        if old is not None:
            self.free += len(old.window)              # a restarted sequence returns what it held
        first = self.free > 0 and max_new > 0
        if first:
            self.free -= 1
        return sampler.prefill(seq_id, prompt, r, max_new, first_row=first)

    def drive(self, sampler, seqs, window, inner, eps):
        before = [None if sq.done else len(sq.window) for sq in seqs]
        # first pass: every sequence steps without extending; count what it returns and whether it wants a slot
        infos, wants = [], []
        for sq in seqs:
            if sq.done:
                infos.append(None)
                wants.append(False)
                continue
            infos.append(sampler.df_step(sq, window, inner, eps, may_append=False))
            wants.append(not sq.done and len(sq.window) < window and
                         sq.n_committed - 1 + len(sq.window) <= sq.n_prompt + sq.max_new - 2)
        for sq, b4 in zip(seqs, before):
            if b4 is not None:
                self.free += b4 - len(sq.window)      # rows that left (all of them when the sequence finished)
        from oracle import rd_oracle as _orc
        for sq, want in zip(seqs, wants):
            if want and self.free > 0:
                nxt = sq.n_committed - 1 + len(sq.window)
                sq.window.append(_orc.Row(nxt, sampler._init(sq.seq_id, nxt)))
                self.free -= 1
        return infos
