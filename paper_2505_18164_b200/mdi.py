"""Python binding of the C-ABI library ``libmdi.so`` (see ``include/mdi.h``).

Argument marshalling only: every step of the decoding path runs in the CUDA
library.  There is no CPU fallback: loading fails loudly if the library has not
been built, and creating a context fails if there is no CUDA device.
"""
from __future__ import annotations

import ctypes
import os
from typing import Iterable, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmdi.so")

MDI_OK = 0
TRACE_WORDS = 128
KV_DEFAULT, KV_BF16, KV_F16, KV_F32 = 0, 1, 2, 3
ERR_ARG, ERR_SHAPE, ERR_OOM, ERR_CONTEXT, ERR_STATE, ERR_TIMEOUT, ERR_CUDA = -1, -2, -3, -4, -5, -6, -7
_ERR_NAMES = {ERR_ARG: "MDI_ERR_ARG", ERR_SHAPE: "MDI_ERR_SHAPE", ERR_OOM: "MDI_ERR_OOM", ERR_CONTEXT: "MDI_ERR_CONTEXT",
              ERR_STATE: "MDI_ERR_STATE", ERR_TIMEOUT: "MDI_ERR_TIMEOUT", ERR_CUDA: "MDI_ERR_CUDA"}

EXPORTS = ["mdi_create", "mdi_destroy", "mdi_load_weights", "mdi_prefill", "mdi_prefill_dev", "mdi_step",
           "mdi_generate", "mdi_generate_dev", "mdi_get_logits", "mdi_set_sampling", "mdi_set_teacher_tokens", "mdi_reset_sample",
           "mdi_get_stats", "mdi_get_partition_times", "mdi_get_trace", "mdi_memory_bytes", "mdi_sync", "mdi_last_error", "mdi_greedy_argmax_static"]


class MdiError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"{_ERR_NAMES.get(code, code)}: {text}")
        self.code = code


class ModelShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("arch", "n_layer", "d_model", "n_head", "head_dim", "n_kv_head", "d_ff", "vocab", "n_ctx",
                 "weight_dtype", "tied_lm_head", "has_bias", "act")] + \
               [("norm_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


class Options(ctypes.Structure):
    _fields_ = [("page_tokens", ctypes.c_int), ("kv_pool_tokens", ctypes.c_int), ("attn_splits", ctypes.c_int),
                ("rounds_per_graph", ctypes.c_int), ("kv_cache_dtype", ctypes.c_int), ("prefill_mode", ctypes.c_int), ("tc_min_group", ctypes.c_int), ("wait_limit_ms", ctypes.c_int), ("debug_withhold_handoff", ctypes.c_int),
                ("scheduler", ctypes.c_int), ("in_kernel_timing", ctypes.c_int), ("fused_blocks_per_head", ctypes.c_int),
                ("reserved0", ctypes.c_int), ("trace_slot", ctypes.c_int), ("td_b_kblocks", ctypes.c_int)]


class Stats(ctypes.Structure):
    _fields_ = [("n_partitions", ctypes.c_int), ("n_samples", ctypes.c_int), ("n_groups", ctypes.c_int),
                ("weight_bytes", ctypes.c_int64 * 16), ("kv_pool_bytes", ctypes.c_int64 * 16),
                ("kv_pages_in_use", ctypes.c_int64 * 16), ("tokens_generated", ctypes.c_int64),
                ("stage_steps", ctypes.c_int64), ("kernel_launches", ctypes.c_int64),
                ("last_prefill_ms", ctypes.c_float), ("last_generate_ms", ctypes.c_float),
                ("last_run_ms", ctypes.c_float), ("kv_element_bytes", ctypes.c_int)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} has not been built (python -m paper_2505_18164_b200.build); "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.mdi_create.argtypes = [ctypes.POINTER(ModelShape), ctypes.POINTER(ci), ci, ci, ctypes.POINTER(Options),
                                 ctypes.POINTER(vp)]
        L.mdi_destroy.argtypes = [vp]
        L.mdi_destroy.restype = None
        L.mdi_load_weights.argtypes = [vp, ctypes.c_char_p, vp, ctypes.c_size_t]
        L.mdi_prefill.argtypes = [vp, ci, vp, ci]
        L.mdi_prefill_dev.argtypes = [vp, ci, vp, ci]
        L.mdi_step.argtypes = [vp, ci, ci, vp, vp]
        L.mdi_generate.argtypes = [vp, ci, ci, vp]
        L.mdi_generate_dev.argtypes = [vp, ci, ci, vp]
        L.mdi_get_logits.argtypes = [vp, ci, vp]
        L.mdi_set_sampling.argtypes = [vp, ctypes.c_float, ci, ctypes.c_uint64]
        L.mdi_set_teacher_tokens.argtypes = [vp, ci, vp, ci]
        L.mdi_reset_sample.argtypes = [vp, ci]
        L.mdi_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
        L.mdi_get_partition_times.argtypes = [vp, ci, ctypes.POINTER(ctypes.c_double), ci]
        L.mdi_get_trace.argtypes = [vp, vp, ci]
        L.mdi_memory_bytes.argtypes = [vp, ci]
        L.mdi_memory_bytes.restype = ctypes.c_int64
        L.mdi_sync.argtypes = [vp]
        L.mdi_greedy_argmax_static.argtypes = [vp, ci, ci, vp, vp]
        L.mdi_last_error.argtypes = [vp]
        L.mdi_last_error.restype = ctypes.c_char_p
        _lib = L
    return _lib


def _ptr(x) -> int:
    """Address of a numpy array (host) or torch tensor (host or device), or a raw integer address."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def greedy_argmax_static(logits_dev, n_rows: int, n_cols: int, out_dev, stream: int = 0):
    """mdi_greedy_argmax_static: per-row argmax of device logits without any allocation (see mdi.h).
    ``logits_dev`` / ``out_dev``: device tensors or raw addresses; ``stream``: a cudaStream_t value."""
    rc = lib().mdi_greedy_argmax_static(_ptr(logits_dev), n_rows, n_cols, _ptr(out_dev), stream)
    if rc != MDI_OK:
        raise MdiError(rc, (lib().mdi_last_error(None) or b"").decode())


class Context:
    """One model on one GPU: mdi_create ... mdi_destroy."""

    def __init__(self, shape, part_bounds: Sequence[int], n_samples: int, page_tokens: int = 0,
                 kv_pool_tokens: int = 0, attn_splits: int = 0, rounds_per_graph: int = 0, scheduler: int = 0,
                 kv_cache_dtype: int = 0, prefill_mode: int = 0, tc_min_group: int = 0,
                 wait_limit_ms: int = 0, debug_withhold_handoff: int = 0, in_kernel_timing: int = 0,
                 fused_blocks_per_head: int = 0, trace_slot: int = 0, td_b_kblocks: int = 0):
        self._h = None
        self.shape = shape
        self.K = len(part_bounds) - 1
        self.n_samples = n_samples
        cs = ModelShape(**{n: getattr(shape, n) for n, _ in ModelShape._fields_})
        bounds = (ctypes.c_int * len(part_bounds))(*part_bounds)
        opts = Options(page_tokens, kv_pool_tokens, attn_splits, rounds_per_graph, kv_cache_dtype, prefill_mode, tc_min_group,
                       wait_limit_ms, debug_withhold_handoff, scheduler, in_kernel_timing, fused_blocks_per_head,
                       0, trace_slot, td_b_kblocks)
        h = ctypes.c_void_p()
        rc = lib().mdi_create(ctypes.byref(cs), bounds, self.K, n_samples, ctypes.byref(opts), ctypes.byref(h))
        if rc != MDI_OK:
            raise MdiError(rc, (lib().mdi_last_error(None) or b"").decode())
        self._h = h

    def _check(self, rc: int):
        if rc != MDI_OK:
            raise MdiError(rc, (lib().mdi_last_error(self._h) or b"").decode())

    def close(self):
        if self._h and _lib is not None:
            _lib.mdi_destroy(self._h)
        self._h = None

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def load_weights(self, name: str, host: np.ndarray):
        host = np.ascontiguousarray(host)
        self._check(lib().mdi_load_weights(self._h, name.encode(), host.ctypes.data, host.nbytes))

    def load_all(self, named: Iterable):
        for name, a in (named.items() if hasattr(named, "items") else named):
            self.load_weights(name, a)

    def prefill(self, sample: int, prompt_host: np.ndarray):
        p = np.ascontiguousarray(prompt_host, np.int32)
        self._check(lib().mdi_prefill(self._h, sample, p.ctypes.data, p.size))

    def prefill_dev(self, sample: int, prompt_dev, n_prompt: int):
        self._check(lib().mdi_prefill_dev(self._h, sample, _ptr(prompt_dev), n_prompt))

    def step(self, partition: int, slot: int, act_in_dev, act_out_dev):
        self._check(lib().mdi_step(self._h, partition, slot, _ptr(act_in_dev), _ptr(act_out_dev)))

    def generate(self, n_samples: int, n_new_tokens: int, out_host: Optional[np.ndarray] = None) -> np.ndarray:
        if out_host is None:
            out_host = np.empty((n_samples, n_new_tokens), np.int32)
        assert out_host.dtype == np.int32 and out_host.size >= n_samples * n_new_tokens and out_host.flags.c_contiguous
        self._check(lib().mdi_generate(self._h, n_samples, n_new_tokens, out_host.ctypes.data))
        return out_host

    def generate_dev(self, n_samples: int, n_new_tokens: int, out_dev):
        self._check(lib().mdi_generate_dev(self._h, n_samples, n_new_tokens, _ptr(out_dev)))

    def get_logits(self, sample: int) -> np.ndarray:
        out = np.empty(self.shape.vocab, np.float32)
        self._check(lib().mdi_get_logits(self._h, sample, out.ctypes.data))
        return out

    def set_sampling(self, temperature: float, top_k: int, seed: int):
        self._check(lib().mdi_set_sampling(self._h, temperature, top_k, seed))

    def set_teacher_tokens(self, sample: int, tokens: Sequence[int]):
        t = np.ascontiguousarray(tokens, np.int32)
        self._check(lib().mdi_set_teacher_tokens(self._h, sample, t.ctypes.data, t.size))

    def reset_sample(self, sample: int):
        self._check(lib().mdi_reset_sample(self._h, sample))

    def stats(self) -> Stats:
        st = Stats()
        self._check(lib().mdi_get_stats(self._h, ctypes.byref(st)))
        return st

    def partition_times(self, partition: int):
        """(blocks in the partition's team, [12] mean milliseconds per category) of the last generate."""
        out = (ctypes.c_double * 12)()
        rc = lib().mdi_get_partition_times(self._h, partition, out, 12)
        if rc < 0:
            self._check(rc)
        return rc, list(out)

    def trace(self) -> np.ndarray:
        """[blocks][TRACE_WORDS] uint64 time stamps of the traced schedule slot ((ns << 4) | category, 0 = unused)."""
        buf = np.zeros(1024 * TRACE_WORDS, np.uint64)
        rc = lib().mdi_get_trace(self._h, buf.ctypes.data, buf.size)
        if rc < 0:
            self._check(rc)
        return buf[: rc * TRACE_WORDS].reshape(rc, TRACE_WORDS)

    def memory_bytes(self, partition: int) -> int:
        return lib().mdi_memory_bytes(self._h, partition)

    def sync(self):
        self._check(lib().mdi_sync(self._h))
