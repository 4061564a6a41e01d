"""Shared set-up for the parity tests: same seeded inputs for the oracle and the CUDA path."""
from dataclasses import replace

import numpy as np
import torch

from oracle import tidar_oracle as O
from tidar_synth import CONFIGS, gen_model_weights, gen_token_ids, tensor_id

# Max-abs tolerance for bf16 hidden states / logits against the float64 oracle (the
# figure the build target states; fp32 accumulation, bf16 operands and activations).
TOL_LOGITS = 3e-2


def depth_tol(ref):
    """Max-abs tolerance for activations of a deep model: 3e-2 of the reference's scale.

    Every activation stored in bf16 carries 2^-9 relative rounding error; about six of them
    feed each layer's residual update, and the errors add up like a random walk, so after L
    layers the relative error is about 2^-9 * sqrt(6 L) (2.5 % at L = 28, measured 1.8 % rms
    for both the tensor-core and the plain fp32-accumulate kernels).  For activations of
    scale <= 1 (the 2-layer model, logits) this is the absolute 3e-2.
    """
    return TOL_LOGITS * max(1.0, float(np.abs(ref).max()))


# Token ids must agree wherever the oracle's top-1 margin exceeds this.
MARGIN = 0.1


def oracle_cfg(sh, n_layers=None):
    return O.OracleConfig(n_layers or sh.n_layers, sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn,
                          sh.vocab, sh.rope_theta, sh.rms_eps, sh.mask_token_id, 1.0)


def make_model(name, n_layers=None, vocab=None, tied=None):
    sh = CONFIGS[name]
    if n_layers is not None or vocab is not None:
        sh = sh.reduced(n_layers or sh.n_layers, vocab)
    if tied is not None:
        sh = replace(sh, tie_lm_head=tied)
    wt = gen_model_weights(sh)                     # host bf16, the single source of values
    return sh, wt


def prompt_ids(sh, n=None, seed=None):
    return gen_token_ids(sh.seed if seed is None else seed, tensor_id("prompt"), n or sh.prompt_len, sh.vocab - 1).numpy().astype(np.int64)


def top1_margin(logits):
    part = np.partition(logits, -2, axis=-1)
    return part[..., -1] - part[..., -2]
