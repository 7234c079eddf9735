"""The tensor-core persistent kernel (scheduler 4: one cooperative launch, a team of thread blocks per partition, every
linear layer a tcgen05 contraction fed by a TMA weight ring, partial sums completed by the consuming phase) against the
CPU oracle, through the C ABI.

Same protocol as test_gpu_parity.py.  Shapes cover: the GPT and the Llama block, grouped-query heads, head_dim 32 / 64 /
128, groups of 1 to 8 samples (and groups of unequal size), fewer samples than partitions, one partition, a hidden width
of more k-blocks than the resident B operand holds (several k ranges per matrix), matrices of several 128-row tiles and
a vocabulary that is no multiple of 128, cache pages crossed during the call, the three cache element types, resumed
calls, the bounded-wait time-out, and agreement with the stream scheduler.
"""
import time

import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, oracle_reference, parity_tolerance, tiny_shape
from test_gpu_parity import _ctx, _check_teacher_forced_stepwise, _check_free_running

pytestmark = pytest.mark.gpu

TD_CASES = [
    # arch, L, d, H, n_kv, F, V, C, bounds, S, P, N, opts
    ("llama", 4, 128, 2, 2, 384, 211, 96, [0, 2, 4], 6, 9, 16, {}),                              # groups of 3, head_dim 64
    ("llama", 4, 128, 2, 1, 384, 211, 96, [0, 2, 4], 16, 5, 10, dict(kv_cache_dtype=2)),          # groups of 8, one kv head, fp16 cache
    ("llama", 2, 256, 2, 2, 2304, 300, 64, [0, 1, 2], 5, 7, 12, dict(page_tokens=8)),             # head_dim 128, 36 k-blocks of hidden units, groups of 3 and 2
    ("gpt", 3, 128, 4, None, 512, 523, 64, [0, 1, 2, 3], 5, 6, 14, {}),                          # GPT block, head_dim 32, K = 3
    ("gpt", 3, 128, 4, None, 512, 523, 64, [0, 1, 2, 3], 2, 6, 14, dict(kv_cache_dtype=1)),       # fewer samples than partitions, bf16 cache
    ("gpt", 4, 256, 4, None, 1024, 1000, 160, [0, 4], 8, 40, 50, dict(page_tokens=16)),           # one partition, long cache over several pages
    ("llama", 3, 192, 3, 3, 448, 131, 48, [0, 1, 3], 1, 3, 20, {}),                              # one sample, unequal partitions
]


def _shape(arch, L, d, H, n_kv, F, V, C):
    return tiny_shape(arch, I.DT_BF16, L=L, d=d, H=H, V=V, C=C, F=F, n_kv=n_kv)


@pytest.mark.parametrize("arch,L,d,H,n_kv,F,V,C,bounds,S,P,N,opts", TD_CASES)
def test_tc_persistent_kernel_matches_oracle(arch, L, d, H, n_kv, F, V, C, bounds, S, P, N, opts):
    shape = _shape(arch, L, d, H, n_kv, F, V, C)
    orc, w = make_oracle(shape, seed=3, std=0.04)
    prompts = I.make_prompts(V, S, P, seed=5)
    toks, lgs, margins = oracle_reference(orc, prompts, N)
    ctx = _ctx(shape, bounds, S, w, scheduler=4, **opts)
    _check_teacher_forced_stepwise(ctx, shape, prompts, toks, lgs, margins, N)
    _check_free_running(ctx, shape, prompts, toks, margins, N)
    assert ctx.stats().kernel_launches > 0
    ctx.close()


def test_tc_persistent_kernel_agrees_with_the_stream_scheduler():
    """A long free-running call and a resumed one: tokens equal those of the stream scheduler wherever the oracle's
    margin is clear, final logits agree to rounding, and one generate call is one launch."""
    shape = _shape("llama", 4, 128, 2, 1, 384, 211, 160)
    orc, w = make_oracle(shape, seed=11, std=0.05)
    prompts = I.make_prompts(211, 6, 6, seed=2)
    toks, lgs, margins = oracle_reference(orc, prompts, 90)
    outs, logits = [], []
    for sched in (1, 4):
        ctx = _ctx(shape, [0, 1, 4], 6, w, scheduler=sched)
        for s in range(6):
            ctx.set_teacher_tokens(s, toks[s])
            ctx.prefill(s, prompts[s])
        l0 = ctx.stats().kernel_launches
        a = ctx.generate(6, 50).copy()
        l1 = ctx.stats().kernel_launches
        b = ctx.generate(6, 40).copy()          # resumed call: feeds the last token first
        if sched == 4:
            assert l1 - l0 == 1
        outs.append(np.concatenate([a, b], axis=1))
        logits.append(np.stack([ctx.get_logits(s) for s in range(6)]))
        ctx.close()
    tol = parity_tolerance(shape)
    for s in range(6):
        ok = margins[s] > 2 * tol
        assert np.array_equal(outs[0][s][ok], outs[1][s][ok]) and np.array_equal(outs[1][s][ok], np.asarray(toks[s])[ok])
        assert np.abs(logits[1][s] - lgs[s][-1]).max() <= tol
    assert np.abs(logits[0] - logits[1]).max() < 1e-3


def test_tc_persistent_kernel_is_deterministic():
    shape = _shape("gpt", 3, 128, 4, None, 512, 523, 64)
    _, w = make_oracle(shape, seed=4, std=0.05)
    prompts = I.make_prompts(523, 7, 5, seed=3)
    runs = []
    for _ in range(2):
        ctx = _ctx(shape, [0, 1, 3], 7, w, scheduler=4)
        for s in range(7):
            ctx.prefill(s, prompts[s])
        out = ctx.generate(7, 30).copy()
        runs.append((out, np.stack([ctx.get_logits(s) for s in range(7)])))
        ctx.close()
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])


def test_tc_persistent_kernel_times_out_cleanly():
    """A partition withholds its output flag once: the next partition's bounded wait runs out, the call reports
    MDI_ERR_TIMEOUT within the limit, every sample is reset, and the same context then generates correctly."""
    from paper_2505_18164_b200 import mdi
    shape = _shape("llama", 3, 128, 2, 2, 384, 97, 48)
    orc, w = make_oracle(shape, seed=9, std=0.06)
    ctx = mdi.Context(shape, [0, 1, 2, 3], 3, scheduler=4, wait_limit_ms=50, debug_withhold_handoff=1)
    ctx.load_all(w)
    prompts = I.make_prompts(97, 3, 5, seed=12)
    for s in range(3):
        ctx.prefill(s, prompts[s])
    t0 = time.time()
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(3, 8)
    assert e.value.code == mdi.ERR_TIMEOUT and "gave up waiting" in str(e.value)
    assert time.time() - t0 < 20.0
    assert ctx.stats().kv_pages_in_use[0] == 0
    toks, _, margins = oracle_reference(orc, prompts, 8)
    for s in range(3):
        ctx.prefill(s, prompts[s])
    out = ctx.generate(3, 8)
    tol = parity_tolerance(shape)
    for s in range(3):
        ok = margins[s] > 2 * tol
        assert np.array_equal(out[s][ok], np.asarray(toks[s])[ok])
    ctx.close()


def test_tc_persistent_kernel_refuses_what_it_cannot_run():
    from paper_2505_18164_b200 import mdi
    with pytest.raises(mdi.MdiError) as e:                                 # fp32 weights
        mdi.Context(tiny_shape("gpt", I.DT_F32, L=2, d=128, H=2, V=97, C=32), [0, 2], 2, scheduler=4)
    assert e.value.code == mdi.ERR_SHAPE
    with pytest.raises(mdi.MdiError) as e:                                 # width not a multiple of 64
        mdi.Context(tiny_shape("gpt", I.DT_BF16, L=2, d=96, H=3, V=97, C=32), [0, 2], 2, scheduler=4)
    assert e.value.code == mdi.ERR_SHAPE
    with pytest.raises(mdi.MdiError) as e:                                 # groups of more than 8 samples
        mdi.Context(_shape("gpt", 2, 128, 4, None, 512, 97, 32), [0, 2], 9, scheduler=4)
    assert e.value.code == mdi.ERR_SHAPE
