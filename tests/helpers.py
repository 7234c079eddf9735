"""Shared by the tests: tiny model shapes and oracle construction."""
import numpy as np

from paper_2505_18164_b200 import inputs as I
from oracle import mdi_oracle as O


def tiny_shape(arch="gpt", dtype=I.DT_F32, L=2, d=32, H=2, V=17, C=16, F=None, n_kv=None):
    hd = d // H
    if arch == "gpt":
        return I.ModelShape(I.ARCH_GPT, L, d, H, hd, n_kv or H, F or 4 * d, V, C, dtype, 1, 1, I.ACT_GELU_TANH)
    return I.ModelShape(I.ARCH_LLAMA, L, d, H, hd, n_kv or H, F or 3 * d - 8, V, C, dtype, 0, 0, I.ACT_SWIGLU)


def make_oracle(shape, seed=0, std=0.02):
    w = I.make_weights(shape, seed, std)
    return O.Oracle(shape, w), w


def parity_tolerance(shape):
    """Absolute logit tolerance: 1e-4 for fp32 weights, 3e-2 for bf16 weights."""
    return 1e-4 if shape.weight_dtype == I.DT_F32 else 3e-2


def oracle_reference(orc, prompts, n_new):
    """Per sample: the oracle's greedy tokens, logits [n_new][V] and top-1/top-2 margins."""
    toks, lgs, margins = [], [], []
    for p in prompts:
        t, l = orc.generate_sequential([int(v) for v in p], n_new)
        toks.append(t)
        lgs.append(l)
        top2 = np.sort(l, axis=1)[:, -2:]
        margins.append(top2[:, 1] - top2[:, 0])
    return toks, lgs, margins
