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
