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
