"""CPU checker: Python face of ``mdi_oracle.c`` plus the schedulers.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never imports it, and it never
imports the product.

``Oracle`` wraps one model.  On top of the C primitives it offers
  * ``generate_sequential``: each sample alone, cached greedy decoding (the
    plain definition the method must reproduce);
  * ``generate_full_recompute``: each sample alone, the whole decoder re-run on
    the whole sequence for every new token (no cache at all);
  * ``generate_pipeline``: a literal simulation of the starter-node loop
    (Algorithm 1) and the secondary-node loop (Algorithm 2) with FIFO queues
    between nodes, per-sample caches per node (Section III-D) and messages that
    carry the sample id.  It also returns the (tick, node, sample) trace that
    the worked example of Section III-C fixes.

Readings of the paper used here (its pseudocode is off by one in two places):
iterations are counted from 0, sample n = k mod n_samples, the first visit of a
sample is k < n_samples; a call that asks for n_new tokens yields exactly n_new
tokens per sample, i.e. one prompt visit plus n_new output-layer evaluations at
the starter, the last of which is not fed back.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from collections import deque
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mdi_oracle.c")
_LIB = os.path.join(_HERE, "libmdi_oracle.so")


def build(force: bool = False) -> str:
    """Compile the C checker with gcc (fp64 arithmetic as written: no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-fno-fast-math", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"])
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("arch", "n_layer", "d_model", "n_head", "head_dim", "n_kv_head", "d_ff", "vocab", "n_ctx",
                 "weight_dtype", "tied_lm_head", "has_bias", "act")] + \
               [("norm_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


_lib = None
_fp = ctypes.POINTER(ctypes.c_float)


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, ci, cd = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        L.orc_model_new.restype = vp
        L.orc_model_new.argtypes = [ctypes.POINTER(_Shape)]
        L.orc_model_free.argtypes = [vp]
        L.orc_model_set.argtypes = [vp, ctypes.c_char_p, vp]
        L.orc_cache_new.restype = vp
        L.orc_cache_new.argtypes = [vp, ci, ci]
        L.orc_cache_free.argtypes = [vp]
        L.orc_cache_len.argtypes = [vp]
        L.orc_layernorm.argtypes = [vp, vp, vp, ci, ci, cd, vp]
        L.orc_rmsnorm.argtypes = [vp, vp, ci, ci, cd, vp]
        L.orc_linear.argtypes = [vp, vp, ci, ci, ci, vp, ci, vp]
        for f in (L.orc_gelu_tanh, L.orc_gelu_erf, L.orc_silu):
            f.restype = cd
            f.argtypes = [cd]
        L.orc_rope.argtypes = [vp, ci, ci, cd]
        L.orc_attend.argtypes = [vp, vp, vp, ci, ci, ctypes.c_size_t, vp]
        L.orc_argmax.argtypes = [vp, ci]
        L.orc_embed.argtypes = [vp, vp, ci, ci, vp]
        L.orc_head.argtypes = [vp, vp, vp]
        L.orc_blocks_cached.argtypes = [vp, vp, vp, ci]
        L.orc_full_forward.argtypes = [vp, vp, ci, vp]
        L.orc_num_threads.restype = ci
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def num_threads() -> int:
    return lib().orc_num_threads()


# ---- elementary operations, exposed for the pin tests --------------------------------------

def _dt(a: np.ndarray) -> int:
    assert a.dtype in (np.float32, np.uint16)
    return 0 if a.dtype == np.float32 else 1


def layernorm(x, g, b, eps):
    x = np.ascontiguousarray(x, np.float32)
    y = np.empty_like(x)
    lib().orc_layernorm(_p(x), _p(g), _p(b), _dt(g), x.size, eps, _p(y))
    return y


def rmsnorm(x, g, eps):
    x = np.ascontiguousarray(x, np.float32)
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(g), _dt(g), x.size, eps, _p(y))
    return y


def linear(W, b, X):
    X = np.ascontiguousarray(np.atleast_2d(X), np.float32)
    T, n_in = X.shape
    n_out = W.shape[0]
    assert W.shape[1] == n_in and W.flags.c_contiguous
    Y = np.empty((T, n_out), np.float32)
    lib().orc_linear(_p(W), _p(b), _dt(W), n_out, n_in, _p(X), T, _p(Y))
    return Y


def gelu_tanh(x: float) -> float:
    return lib().orc_gelu_tanh(float(x))


def gelu_erf(x: float) -> float:
    return lib().orc_gelu_erf(float(x))


def silu(x: float) -> float:
    return lib().orc_silu(float(x))


def rope(v, pos, theta):
    v = np.array(v, np.float32, copy=True)
    lib().orc_rope(_p(v), v.size, int(pos), float(theta))
    return v


def attend(q, K, V):
    """One head: q [hd], K and V [n_keys][hd] -> [hd]."""
    q = np.ascontiguousarray(q, np.float32)
    K = np.ascontiguousarray(K, np.float32)
    V = np.ascontiguousarray(V, np.float32)
    out = np.empty_like(q)
    lib().orc_attend(_p(q), _p(K), _p(V), K.shape[0], q.size, K.shape[1], _p(out))
    return out


def argmax(x) -> int:
    x = np.ascontiguousarray(x, np.float32)
    return lib().orc_argmax(_p(x), x.size)


# ---- sampling from the pmf (Section III-B: "a probability mass function that is then sampled") ----------

_M64 = (1 << 64) - 1


def splitmix64_mix(z: int) -> int:
    """Output function of the splitmix64 generator (Steele, Lea, Flood 2014), on a 64-bit state z."""
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def sample_uniform(seed: int, sample: int, index: int) -> float:
    """Counter-based uniform in [0, 1) for (seed, sample, index of the output-layer evaluation)."""
    h = splitmix64_mix((splitmix64_mix((seed ^ (sample << 32)) & _M64) + index) & _M64)
    return (h >> 11) / 9007199254740992.0


def sample_top_k(logits, top_k: int, temperature: float, u: float) -> int:
    """Keep the top_k largest logits (larger first, lower index first on ties), p_j = exp((l_j - l_0) / T) in
    fp64, and return the first token whose running sum exceeds u * sum(p)."""
    lg = np.asarray(logits, np.float32)
    order = sorted(range(lg.size), key=lambda i: (-float(lg[i]), i))[:top_k]
    p = [math.exp((float(lg[i]) - float(lg[order[0]])) / float(temperature)) for i in order]
    z = 0.0
    for v in p:
        z += v
    target, c = u * z, 0.0
    for i, v in zip(order, p):
        c += v
        if c > target:
            return i
    return order[-1]


# ---- model ----------------------------------------------------------------------------------

class Cache:
    """Keys and values of one sample for the blocks [lo, hi) of one node."""

    def __init__(self, model: "Oracle", lo: int, hi: int):
        self._h = lib().orc_cache_new(model._h, lo, hi)

    def __len__(self):
        return lib().orc_cache_len(self._h)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_cache_free(self._h)
            self._h = None


class Oracle:
    def __init__(self, shape, weights: Dict[str, np.ndarray]):
        """shape: any object with the fields of ``_Shape``; weights: name -> host array
        (float32, or uint16 bfloat16 bit patterns), kept alive by this object."""
        self.shape = shape
        cs = _Shape(**{n: getattr(shape, n) for n, _ in _Shape._fields_})
        self._h = lib().orc_model_new(ctypes.byref(cs))
        self._w = {}
        for name, a in weights.items():
            a = np.ascontiguousarray(a)
            assert _dt(a) == shape.weight_dtype, name
            self._w[name] = a
            if lib().orc_model_set(self._h, name.encode(), _p(a)) != 0:
                raise KeyError(name)
        self.d = shape.d_model
        self.V = shape.vocab

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_model_free(self._h)
            self._h = None

    # starter input layers / output layers / a chunk of blocks
    def embed(self, tokens: Sequence[int], pos0: int) -> np.ndarray:
        t = np.ascontiguousarray(tokens, np.int32)
        X = np.empty((t.size, self.d), np.float32)
        lib().orc_embed(self._h, _p(t), t.size, pos0, _p(X))
        return X

    def head(self, x: np.ndarray) -> np.ndarray:
        x = np.ascontiguousarray(x, np.float32).reshape(self.d)
        out = np.empty(self.V, np.float32)
        lib().orc_head(self._h, _p(x), _p(out))
        return out

    def blocks(self, cache: Cache, X: np.ndarray) -> np.ndarray:
        X = np.array(X, np.float32, copy=True).reshape(-1, self.d)
        if lib().orc_blocks_cached(self._h, cache._h, _p(X), X.shape[0]) != 0:
            raise ValueError("context overflow")
        return X

    def full_logits(self, tokens: Sequence[int]) -> np.ndarray:
        t = np.ascontiguousarray(tokens, np.int32)
        out = np.empty((t.size, self.V), np.float32)
        if lib().orc_full_forward(self._h, _p(t), t.size, _p(out)) != 0:
            raise ValueError("context overflow")
        return out

    # ---- plain definitions -------------------------------------------------------------
    def generate_full_recompute(self, prompt: Sequence[int], n_new: int):
        """No cache: rerun the decoder on the whole sequence for each new token."""
        seq = list(prompt)
        logits = []
        for _ in range(n_new):
            lg = self.full_logits(seq)[-1]
            logits.append(lg)
            seq.append(argmax(lg))
        return seq[len(prompt):], np.stack(logits)

    def generate_sequential(self, prompt: Sequence[int], n_new: int, bounds: Sequence[int] = None,
                            forced: Sequence[int] = None, sampler=None):
        """One sample, cached greedy decoding through the chunks given by ``bounds``.

        ``forced``: tokens fed back in place of the argmax (the argmax is still
        returned), so that a second implementation can be compared step by step.
        ``sampler``: None for greedy, or (temperature, top_k, seed, sample index): the i-th token is then drawn
        with sample_top_k and the uniform sample_uniform(seed, sample index, i).
        Returns (tokens [n_new], logits [n_new][V])."""
        L = self.shape.n_layer
        bounds = list(bounds) if bounds is not None else [0, L]
        caches = [Cache(self, lo, hi) for lo, hi in zip(bounds[:-1], bounds[1:])]
        toks, logits = [], []
        feed = list(prompt)
        pos = 0
        for i in range(n_new):
            X = self.embed(feed, pos)
            for c in caches:
                X = self.blocks(c, X)
            pos += len(feed)
            lg = self.head(X[-1])
            logits.append(lg)
            if sampler is None:
                toks.append(argmax(lg))
            else:
                temperature, top_k, seed, smp = sampler
                toks.append(sample_top_k(lg, top_k, temperature, sample_uniform(seed, smp, i)))
            feed = [toks[-1] if forced is None else int(forced[i])]
        return toks, np.stack(logits)

    # ---- Algorithms 1 and 2, literally ---------------------------------------------------
    def generate_pipeline(self, prompts: Sequence[Sequence[int]], n_new: int, bounds: Sequence[int],
                          head_on_starter: bool = True):
        """Recurrent pipeline over len(bounds)-1 nodes and len(prompts) samples.

        Node 0 is the starter (input layers, its blocks and - as in the paper - the
        output layers); nodes 1.. are secondaries.  Each node owns an input FIFO; a
        message is (sample id, payload).  Nodes are stepped in lock-step ticks: in a
        tick every node whose input queue is non-empty handles one message, and what
        it sends becomes visible to the receiver at the next tick (equal processing
        times, as the paper's example assumes).

        ``head_on_starter=False`` moves the output layers to the last node, which then
        sends the starter a token instead of an activation; the results must not change.

        Returns (tokens [S][n_new], logits [S][n_new][V], trace) with trace a list of
        (tick, node, sample, kind), kind in {"prefill", "decode", "head"}.
        """
        S, K = len(prompts), len(bounds) - 1
        queues = [deque() for _ in range(K)]
        caches: List[List[Optional[Cache]]] = [[None] * S for _ in range(K)]
        seqs = [list(p) for p in prompts]
        n_fed = [0] * S                      # tokens of the sample already pushed through the pipeline
        out_tok = [[] for _ in range(S)]
        out_lg = [[] for _ in range(S)]
        visits = [0] * S                     # starter visits per sample
        trace = []
        for n in range(S):                   # every sample starts in the starter's input queue (Algorithm 1, initialisation)
            queues[0].append((n, None))
        tick = 0
        total_visits = S * (n_new + 1)
        done_visits = 0

        def emit(n, x_last):
            lg = self.head(x_last)
            out_lg[n].append(lg)
            t = argmax(lg)
            out_tok[n].append(t)
            seqs[n].append(t)

        while done_visits < total_visits:
            sends = []
            for p in range(K):
                if not queues[p]:
                    continue
                n, payload = queues[p].popleft()
                if p == 0:
                    first = visits[n] == 0
                    visits[n] += 1
                    done_visits += 1
                    if not first:
                        if head_on_starter:
                            emit(n, payload[-1])
                            trace.append((tick, 0, n, "head"))
                        else:                # payload is the token chosen by the last node
                            pass
                    if visits[n] <= n_new:   # not the last visit: feed back through the input layers
                        if caches[0][n] is None:
                            caches[0][n] = Cache(self, bounds[0], bounds[1])
                        new = seqs[n][n_fed[n]:]
                        X = self.embed(new, n_fed[n])
                        n_fed[n] += len(new)
                        X = self.blocks(caches[0][n], X)
                        trace.append((tick, 0, n, "prefill" if first else "decode"))
                        if K == 1:
                            if head_on_starter:
                                sends.append((0, (n, X)))
                            else:
                                emit(n, X[-1])
                                trace.append((tick, 0, n, "head"))
                                sends.append((0, (n, None)))
                        else:
                            sends.append((1, (n, X)))
                else:
                    first = caches[p][n] is None
                    if first:
                        caches[p][n] = Cache(self, bounds[p], bounds[p + 1])
                    X = self.blocks(caches[p][n], payload)
                    trace.append((tick, p, n, "prefill" if first else "decode"))
                    if p == K - 1 and not head_on_starter:
                        emit(n, X[-1])
                        trace.append((tick, p, n, "head"))
                        sends.append((0, (n, None)))
                    else:
                        sends.append(((p + 1) % K, (n, X)))
            for dst, msg in sends:
                queues[dst].append(msg)
            tick += 1
            if tick > 10 * (total_visits + K) * max(1, K):
                raise RuntimeError("pipeline simulation did not terminate")
        return out_tok, [np.stack(l) for l in out_lg], trace
