"""Seeded synthetic workloads: model shapes, weight tensors and prompts.

Holds no model arithmetic.  It names the five workloads (shape, partition
boundaries, samples in flight, prompt and generation lengths), lists the
parameter tensors of a shape, and fills them from the counter-based generator
in ``csrc/synth_inputs.c`` (every element a pure function of seed, tensor
ordinal and element index).  The same host buffers feed both the CUDA library
(through ``mdi_load_weights``) and the CPU checker used by the tests.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field, replace
from typing import Dict, List, Tuple

import numpy as np

ARCH_GPT = 0
ARCH_LLAMA = 1
DT_F32 = 0
DT_BF16 = 1
ACT_GELU_TANH = 0
ACT_GELU_ERF = 1
ACT_SWIGLU = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmdi_inputs.so")
_lib = None


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` first")
        lib = ctypes.CDLL(_LIB_PATH)
        lib.synth_normal.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_double, ctypes.c_int,
                                     ctypes.c_uint64, ctypes.c_uint64, ctypes.c_void_p]
        lib.synth_normal.restype = None
        lib.synth_const.argtypes = [ctypes.c_double, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p]
        lib.synth_const.restype = None
        lib.synth_tokens.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int32, ctypes.c_uint64,
                                     ctypes.c_void_p]
        lib.synth_tokens.restype = None
        _lib = lib
    return _lib


@dataclass(frozen=True)
class ModelShape:
    arch: int
    n_layer: int
    d_model: int
    n_head: int
    head_dim: int
    n_kv_head: int
    d_ff: int
    vocab: int
    n_ctx: int
    weight_dtype: int
    tied_lm_head: int
    has_bias: int
    act: int
    norm_eps: float = 1e-5
    rope_theta: float = 1e4


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    part_bounds: Tuple[int, ...]   # K+1 ascending layer indices, half-open ranges
    n_samples: int
    n_prompt: int
    n_new: int
    weight_seed: int = 0
    prompt_seed: int = 1

    @property
    def n_partitions(self) -> int:
        return len(self.part_bounds) - 1


def _gpt(L, d, H, V, C, dt):
    return ModelShape(ARCH_GPT, L, d, H, d // H, H, 4 * d, V, C, dt, 1, 1, ACT_GELU_TANH)


def _even_bounds(L, K):
    return tuple(range(0, L + 1, L // K))


WORKLOADS: Dict[str, Workload] = {
    "tiny_gpt_fp32": Workload("tiny_gpt_fp32", _gpt(6, 384, 6, 65, 256, DT_F32), (0, 2, 4, 6), 3, 16, 64),
    "gpt2_small": Workload("gpt2_small", _gpt(12, 768, 12, 50257, 1024, DT_BF16), _even_bounds(12, 3), 3, 64, 512),
    "gpt2_medium": Workload("gpt2_medium", _gpt(24, 1024, 16, 50257, 1024, DT_BF16), _even_bounds(24, 4), 8, 128, 768),
    "gpt2_xl": Workload("gpt2_xl", _gpt(48, 1600, 25, 50257, 1024, DT_BF16), _even_bounds(48, 6), 16, 256, 768),
    "llama_7b": Workload(
        "llama_7b",
        ModelShape(ARCH_LLAMA, 32, 4096, 32, 128, 32, 11008, 32000, 2048, DT_BF16, 0, 0, ACT_SWIGLU),
        _even_bounds(32, 8), 64, 128, 512),
}
WORKLOAD_ORDER = ["tiny_gpt_fp32", "gpt2_small", "gpt2_medium", "gpt2_xl", "llama_7b"]

# The paper's own two models as synthetic shapes (Section IV-A): what it states - blocks, embedding width, heads,
# vocabulary, context, blocks per node, three samples, fp32 (its boards had no 16-bit arithmetic), a
# one-token prompt and 800 generated tokens - is kept; what it does not state is chosen here: the MLP width
# (5120 gives the quoted 304 M parameters; 5632 is the width of the public 1.1 B model), the number of
# key/value heads (16 = plain multi-head attention for the small model, 4 for the large one), untied output layer.
PAPER_SHAPES: Dict[str, Workload] = {
    "nanollama_3nodes": Workload(
        "nanollama_3nodes",
        ModelShape(ARCH_LLAMA, 12, 1024, 16, 64, 16, 5120, 32000, 2048, DT_F32, 0, 0, ACT_SWIGLU),
        (0, 2, 7, 12), 3, 1, 800),
    "nanollama_2nodes": Workload(
        "nanollama_2nodes",
        ModelShape(ARCH_LLAMA, 12, 1024, 16, 64, 16, 5120, 32000, 2048, DT_F32, 0, 0, ACT_SWIGLU),
        (0, 5, 12), 3, 1, 800),
    "tinyllama_3nodes": Workload(
        "tinyllama_3nodes",
        ModelShape(ARCH_LLAMA, 22, 2048, 32, 64, 4, 5632, 32000, 2048, DT_F32, 0, 0, ACT_SWIGLU),
        (0, 6, 14, 22), 3, 1, 800),
}
ALL_WORKLOADS: Dict[str, Workload] = {**WORKLOADS, **PAPER_SHAPES}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (shape fields go to the shape)."""
    shape_kw = {k: v for k, v in kw.items() if k in ModelShape.__dataclass_fields__}
    rest = {k: v for k, v in kw.items() if k not in shape_kw}
    return replace(w, shape=replace(w.shape, **shape_kw), **rest)


def tensor_specs(s: ModelShape) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, kind) of every parameter tensor, in ordinal order.

    kind: "normal" (N(0, 0.02)), "ones", "zeros".  Linear weights are row-major
    [out_features, in_features].  The fused attention projection stacks q rows,
    then k rows, then v rows.
    """
    d, F, V = s.d_model, s.d_ff, s.vocab
    q_rows = s.n_head * s.head_dim
    kv_rows = s.n_kv_head * s.head_dim
    out: List[Tuple[str, Tuple[int, ...], str]] = [("wte", (V, d), "normal")]
    if s.arch == ARCH_GPT:
        out.append(("wpe", (s.n_ctx, d), "normal"))
    for i in range(s.n_layer):
        p = f"h.{i}."
        out.append((p + "ln1.g", (d,), "ones"))
        if s.arch == ARCH_GPT:
            out.append((p + "ln1.b", (d,), "zeros"))
        out.append((p + "attn.wqkv", (q_rows + 2 * kv_rows, d), "normal"))
        if s.has_bias:
            out.append((p + "attn.bqkv", (q_rows + 2 * kv_rows,), "normal"))
        out.append((p + "attn.wo", (d, q_rows), "normal"))
        if s.has_bias:
            out.append((p + "attn.bo", (d,), "normal"))
        out.append((p + "ln2.g", (d,), "ones"))
        if s.arch == ARCH_GPT:
            out.append((p + "ln2.b", (d,), "zeros"))
        if s.act == ACT_SWIGLU:
            out.append((p + "mlp.wgate", (F, d), "normal"))
            out.append((p + "mlp.wup", (F, d), "normal"))
            out.append((p + "mlp.wdown", (d, F), "normal"))
        else:
            out.append((p + "mlp.w1", (F, d), "normal"))
            if s.has_bias:
                out.append((p + "mlp.b1", (F,), "normal"))
            out.append((p + "mlp.w2", (d, F), "normal"))
            if s.has_bias:
                out.append((p + "mlp.b2", (d,), "normal"))
    out.append(("lnf.g", (d,), "ones"))
    if s.arch == ARCH_GPT:
        out.append(("lnf.b", (d,), "zeros"))
    if not s.tied_lm_head:
        out.append(("lm_head", (V, d), "normal"))
    return out


def np_dtype(weight_dtype: int):
    """Host container dtype: float32, or uint16 holding bfloat16 bit patterns."""
    return np.float32 if weight_dtype == DT_F32 else np.uint16


def make_tensor(seed: int, ordinal: int, shape: Tuple[int, ...], kind: str, weight_dtype: int,
                std: float = 0.02) -> np.ndarray:
    lib = _load()
    n = int(np.prod(shape))
    a = np.empty(shape, dtype=np_dtype(weight_dtype))
    if kind == "normal":
        lib.synth_normal(seed, ordinal, std, weight_dtype, 0, n, a.ctypes.data)
    else:
        lib.synth_const(1.0 if kind == "ones" else 0.0, weight_dtype, n, a.ctypes.data)
    return a


def make_weights(s: ModelShape, seed: int = 0, std: float = 0.02) -> Dict[str, np.ndarray]:
    """All parameter tensors of a shape, as host arrays keyed by name."""
    return {name: make_tensor(seed, k, shp, kind, s.weight_dtype, std)
            for k, (name, shp, kind) in enumerate(tensor_specs(s))}


def iter_weights(s: ModelShape, seed: int = 0, std: float = 0.02):
    """Yield (name, array) one tensor at a time (bounded host memory for large shapes)."""
    for k, (name, shp, kind) in enumerate(tensor_specs(s)):
        yield name, make_tensor(seed, k, shp, kind, s.weight_dtype, std)


def make_prompts(vocab: int, n_samples: int, n_prompt: int, seed: int = 1) -> np.ndarray:
    """[n_samples, n_prompt] int32 token ids, uniform over the vocabulary; sample s uses stream s."""
    lib = _load()
    out = np.empty((n_samples, n_prompt), dtype=np.int32)
    for smp in range(n_samples):
        row = np.empty(n_prompt, dtype=np.int32)
        lib.synth_tokens(seed, smp, vocab, n_prompt, row.ctypes.data)
        out[smp] = row
    return out


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float32 (container conversion only)."""
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_f32(a: np.ndarray) -> np.ndarray:
    return a if a.dtype == np.float32 else bf16_bits_to_f32(a)


def param_bytes(s: ModelShape) -> int:
    bpe = 4 if s.weight_dtype == DT_F32 else 2
    return sum(int(np.prod(shp)) for _, shp, _ in tensor_specs(s)) * bpe
