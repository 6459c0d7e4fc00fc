"""Seeded synthetic inputs for the recurrent-depth sampler: weights and prompts.

This module only *generates inputs*.  It holds none of the method's arithmetic
(no layer math, no sampler logic, no counter-based generator the method draws
from), so that both the CPU checker and the CUDA library can be fed from it
without sharing any computation.

Tensor order (the order in which the C-ABI `rd_load` expects its pointer
array, and the key order of the dict returned by `make_weights`):

    emb [V,h]
    for block in (prelude, core, coda): for layer l:
        g1 [h], wq [h,h], wk [h,h], wv [h,h], wo [h,h], g2 [h],
        wg [I,h], wu [I,h], wd [h,I]
    adapter [h,2h], g_core [h], g_final [h]
    head [V,h]            (only when embeddings are not tied)

All matrices are stored [out_features, in_features] row-major.
"""
from __future__ import annotations

import numpy as np

BLOCKS = ("prelude", "core", "coda")


def tensor_specs(hidden, mlp_inner, n_prelude, n_core, n_coda, vocab, tie_embeddings=True):
    """Ordered list of (name, shape, is_gain) for a model of the given shape."""
    h, I, V = hidden, mlp_inner, vocab
    specs = [("emb", (V, h), False)]
    for blk, n in zip(BLOCKS, (n_prelude, n_core, n_coda)):
        for l in range(n):
            p = f"{blk}.{l}."
            specs += [
                (p + "g1", (h,), True),
                (p + "wq", (h, h), False),
                (p + "wk", (h, h), False),
                (p + "wv", (h, h), False),
                (p + "wo", (h, h), False),
                (p + "g2", (h,), True),
                (p + "wg", (I, h), False),
                (p + "wu", (I, h), False),
                (p + "wd", (h, I), False),
            ]
    specs += [("adapter", (h, 2 * h), False), ("g_core", (h,), True), ("g_final", (h,), True)]
    if not tie_embeddings:
        specs.append(("head", (V, h), False))
    return specs


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 holding the same values."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_weights(hidden, mlp_inner, n_prelude, n_core, n_coda, vocab, tie_embeddings=True,
                 seed=0, std=0.02, gain_jitter=0.0, bf16=False, adapter_s_scale=1.0, layer_scale=1.0):
    """Random-init weights: matrices N(0, std), gains 1 + gain_jitter * N(0,1).

    Returns a dict name -> float32 array in `tensor_specs` order.  With
    `bf16=True` every matrix value is rounded to the nearest bfloat16 (gains
    stay float32), so both consumers see exactly the values the bf16
    configuration stores.  `adapter_s_scale` scales the half of the adapter
    that multiplies the latent state (columns h..2h-1); tests use it to make
    the recurrence more or less contractive.  `layer_scale` scales every
    matrix inside the layers (wq .. wd; not the embedding, adapter or head):
    below 1 a layer adds less to its residual stream, so it amplifies
    perturbations of its input less.
    """
    rng = np.random.default_rng(seed)
    out = {}
    for name, shape, is_gain in tensor_specs(hidden, mlp_inner, n_prelude, n_core, n_coda,
                                             vocab, tie_embeddings):
        if is_gain:
            g = np.ones(shape, dtype=np.float32)
            if gain_jitter:
                g += gain_jitter * rng.standard_normal(shape, dtype=np.float32)
            out[name] = g
            continue
        w = rng.standard_normal(shape, dtype=np.float32)
        w *= np.float32(std)
        if name == "adapter" and adapter_s_scale != 1.0:
            w[:, hidden:] *= np.float32(adapter_s_scale)
        if layer_scale != 1.0 and "." in name:
            w *= np.float32(layer_scale)
        if bf16:
            w = from_bf16_bits(to_bf16_bits(w))
        out[name] = w
    return out


def make_prompt(n, vocab, seed=0):
    """`n` token ids uniform in [0, vocab)."""
    rng = np.random.default_rng(seed + 0x5EED)
    return rng.integers(0, vocab, size=n, dtype=np.int32)


def make_prompt_lengths(batch, lo, hi, seed=0):
    """`batch` prompt lengths uniform in [lo, hi]."""
    rng = np.random.default_rng(seed + 0x1E46)
    return rng.integers(lo, hi + 1, size=batch, dtype=np.int32)


# Workload shapes named by the benchmark configurations.
TINY = dict(hidden=256, n_heads=4, head_dim=64, mlp_inner=688, n_prelude=1, n_core=2, n_coda=1,
            vocab=512)
SHAPE_3P5B = dict(hidden=5280, n_heads=55, head_dim=96, mlp_inner=17920, n_prelude=2, n_core=4,
                  n_coda=2, vocab=65536)
# Reduced-width twin of the 3.5B shape (same structure: head_dim 96, 2/4/2 layers).
TWIN = dict(hidden=480, n_heads=5, head_dim=96, mlp_inner=1664, n_prelude=2, n_core=4, n_coda=2,
            vocab=4096)


def shape_args(shape: dict) -> dict:
    """The subset of a shape dict that `tensor_specs` / `make_weights` take."""
    return {k: shape[k] for k in ("hidden", "mlp_inner", "n_prelude", "n_core", "n_coda", "vocab")}
