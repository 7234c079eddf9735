"""The fused-phase persistent kernel (scheduler 3: two team barriers per block of the model, weights repacked
per thread block into tensor-core fragment order) against the CPU oracle, through the C ABI.

Same protocol as test_gpu_parity.py.  Shapes cover: one and several samples per group (1, 2 and 3-4 columns
pairs of the B operand), fewer samples than partitions, head_dim 16/32/64, a vocabulary that is not a multiple
of the 16-row tile, a hidden width that gives blocks unequal numbers of hidden units, resumed generate calls,
and agreement with the other schedulers.
"""
import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, oracle_reference, parity_tolerance, tiny_shape
from test_gpu_parity import _ctx, _check_teacher_forced_stepwise, _check_free_running

pytestmark = pytest.mark.gpu

FUSED_CASES = [
    # L, d, H, V, C, bounds, S, P, N, opts
    (4, 64, 4, 97, 64, [0, 2, 4], 2, 9, 16, dict(page_tokens=8)),
    (4, 64, 4, 97, 64, [0, 2, 4], 5, 9, 16, dict(page_tokens=8)),            # groups of 3 and 2
    (3, 128, 2, 131, 96, [0, 1, 2, 3], 2, 17, 30, {}),                        # fewer samples than partitions, head_dim 64
    (3, 128, 2, 131, 96, [0, 1, 2, 3], 3, 17, 40, dict(prefill_mode=1)),
    (4, 64, 2, 97, 64, [0, 1, 2, 3, 4], 1, 4, 9, {}),                         # one sample, four partitions
    (2, 256, 4, 2100, 48, [0, 1, 2], 4, 5, 8, {}),                            # 2 per group, 132 vocabulary tiles
    (2, 256, 16, 333, 160, [0, 2], 4, 100, 50, dict(page_tokens=4)),          # one partition, 4 per group, head_dim 16, long cache
    (5, 192, 3, 1000, 64, [0, 1, 5], 2, 3, 20, {}),                           # unequal partitions, d_ff 768 = 48 hidden units
]


@pytest.mark.parametrize("L,d,H,V,C,bounds,S,P,N,opts", FUSED_CASES)
def test_fused_kernel_matches_oracle(L, d, H, V, C, bounds, S, P, N, opts):
    shape = tiny_shape("gpt", I.DT_BF16, L=L, d=d, H=H, V=V, C=C)
    orc, w = make_oracle(shape, seed=3, std=0.04)
    prompts = I.make_prompts(V, S, P, seed=5)
    toks, lgs, margins = oracle_reference(orc, prompts, N)
    ctx = _ctx(shape, bounds, S, w, scheduler=3, **opts)
    _check_teacher_forced_stepwise(ctx, shape, prompts, toks, lgs, margins, N)
    _check_free_running(ctx, shape, prompts, toks, margins, N)
    ctx.close()


def test_fused_kernel_agrees_with_the_other_schedulers():
    """Tokens of a long free-running call (and of a resumed one) equal those of the stream scheduler and of the
    phase-per-matrix kernel wherever the oracle's margin is clear; final logits agree to rounding."""
    shape = tiny_shape("gpt", I.DT_BF16, L=3, d=128, H=4, V=211, C=160)
    orc, w = make_oracle(shape, seed=11, std=0.05)
    prompts = I.make_prompts(211, 3, 6, seed=2)
    toks, lgs, margins = oracle_reference(orc, prompts, 90)
    outs, logits = [], []
    for sched in (1, 2, 3):
        ctx = _ctx(shape, [0, 1, 2, 3], 3, w, scheduler=sched)
        for s in range(3):
            ctx.set_teacher_tokens(s, toks[s])
            ctx.prefill(s, prompts[s])
        a = ctx.generate(3, 50)
        b = ctx.generate(3, 40)          # resumed call: feeds the last token first
        outs.append(np.concatenate([a, b], axis=1))
        logits.append(np.stack([ctx.get_logits(s) for s in range(3)]))
        ctx.close()
    tol = parity_tolerance(shape)
    for s in range(3):
        ok = margins[s] > 2 * tol
        for o in outs:
            assert np.array_equal(o[s][ok], np.asarray(toks[s])[ok])
    assert np.abs(logits[2] - logits[0]).max() < 1e-3 and np.abs(logits[2] - logits[1]).max() < 1e-3


def test_fused_kernel_is_deterministic():
    """Partial sums meet in integer accumulators, so two runs give bit-identical logits."""
    shape = tiny_shape("gpt", I.DT_BF16, L=2, d=128, H=2, V=300, C=64)
    _, w = make_oracle(shape, seed=4, std=0.05)
    prompts = I.make_prompts(300, 2, 5, seed=9)
    res = []
    for _ in range(2):
        ctx = _ctx(shape, [0, 1, 2], 2, w, scheduler=3)
        for s in range(2):
            ctx.prefill(s, prompts[s])
        out = ctx.generate(2, 30)
        res.append((out.copy(), ctx.get_logits(0).copy(), ctx.get_logits(1).copy()))
        ctx.close()
    assert np.array_equal(res[0][0], res[1][0])
    assert np.array_equal(res[0][1], res[1][1]) and np.array_equal(res[0][2], res[1][2])


def test_fused_scheduler_refuses_shapes_it_does_not_cover():
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("llama", I.DT_BF16, L=2, d=64, H=4, V=50, C=32)
    with pytest.raises(mdi.MdiError):
        mdi.Context(shape, [0, 1, 2], 2, scheduler=3)


def test_fused_kernel_withheld_handoff_times_out_and_the_context_survives():
    """Failure detection without faulting anything (as for the other persistent kernel): partition 0 withholds its
    output handoff once, waits are given 50 ms, the call returns MDI_ERR_TIMEOUT, the samples are reset, and the
    same context then generates correctly."""
    import time
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", I.DT_BF16, L=3, d=64, H=4, V=97, C=48)
    orc, w = make_oracle(shape, seed=9, std=0.06)
    ctx = mdi.Context(shape, [0, 1, 2, 3], 3, scheduler=3, wait_limit_ms=50, debug_withhold_handoff=1)
    ctx.load_all(w)
    prompts = I.make_prompts(97, 3, 5, seed=12)
    for s in range(3):
        ctx.prefill(s, prompts[s])
    t0 = time.time()
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(3, 8)
    assert e.value.code == mdi.ERR_TIMEOUT and "gave up waiting" in str(e.value)
    assert time.time() - t0 < 20.0
    assert ctx.stats().kv_pages_in_use[0] == 0                      # every sample was reset
    toks, _, margins = oracle_reference(orc, prompts, 8)
    for s in range(3):
        ctx.prefill(s, prompts[s])
    out = ctx.generate(3, 8)                                        # the hook was one-shot: this run is normal
    tol = parity_tolerance(shape)
    for s in range(3):
        ok = margins[s] > 2 * tol
        assert np.array_equal(out[s][ok], np.asarray(toks[s])[ok])
    ctx.close()


def test_fused_kernel_one_or_two_blocks_per_head_agree():
    """A head served by one thread block, or shared by the two blocks of a cluster (halves of the q/k/v rows, of each
    cache page's rows and of the output rows, exchanged through distributed shared memory): same tokens where the
    oracle's margin is clear, logits equal to rounding, both within tolerance of the oracle."""
    shape = tiny_shape("gpt", I.DT_BF16, L=4, d=256, H=4, V=523, C=192)
    orc, w = make_oracle(shape, seed=21, std=0.04)
    prompts = I.make_prompts(523, 5, 70, seed=8)
    toks, lgs, margins = oracle_reference(orc, prompts, 60)
    tol = parity_tolerance(shape)
    res = []
    for blocks_per_head in (0, 1):
        ctx = _ctx(shape, [0, 2, 4], 5, w, scheduler=3, page_tokens=32, fused_blocks_per_head=blocks_per_head)
        for s in range(5):
            ctx.set_teacher_tokens(s, toks[s])
            ctx.prefill(s, prompts[s])
        out = ctx.generate(5, 60)
        lg = np.stack([ctx.get_logits(s) for s in range(5)])
        for s in range(5):
            ok = margins[s] > 2 * tol
            assert np.array_equal(out[s][ok], np.asarray(toks[s])[ok])
            assert np.abs(lg[s] - lgs[s][-1]).max() <= tol
        res.append(lg)
        ctx.close()
    assert np.abs(res[0] - res[1]).max() < 1e-3

