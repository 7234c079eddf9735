"""CUDA library against the CPU oracle, through the C ABI (python binding = marshalling only).

Protocol.  Random N(0, 0.02) weights give flat logits, so free-running greedy sequences of two
correct implementations fork at the first near-tie.  The main comparison is therefore
teacher-forced: the library is fed the oracle's tokens, which makes every step's logits
comparable: max |delta| <= tol (1e-4 fp32 weights, 3e-2 bf16 weights).  The library's own argmax
must equal the oracle's wherever the oracle's top-1/top-2 margin exceeds 2*tol (both logits
may move by tol).  A free-running run must equal the oracle up to each sample's first
low-margin step.
"""
import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, oracle_reference, parity_tolerance, tiny_shape

pytestmark = pytest.mark.gpu


def _ctx(shape, bounds, S, weights, **kw):
    from paper_2505_18164_b200 import mdi
    ctx = mdi.Context(shape, bounds, S, **kw)
    ctx.load_all(weights)
    return ctx


def _check_teacher_forced_stepwise(ctx, shape, prompts, toks, lgs, margins, n_new):
    tol = parity_tolerance(shape)
    S = len(prompts)
    for s in range(S):
        ctx.set_teacher_tokens(s, toks[s])
        ctx.prefill(s, prompts[s])
    worst, gated = 0.0, 0
    for i in range(n_new):
        out = ctx.generate(S, 1)
        for s in range(S):
            lg = ctx.get_logits(s)
            worst = max(worst, float(np.abs(lg - lgs[s][i]).max()))
            if margins[s][i] > 2 * tol:
                assert out[s, 0] == toks[s][i], (s, i)
            else:
                gated += 1
    print(f"teacher-forced: worst |dlogit| {worst:.3e} (tol {tol:g}), margin-gated steps {gated}/{n_new * S}")
    assert worst <= tol, worst
    return worst, gated


def _check_free_running(ctx, shape, prompts, toks, margins, n_new):
    tol = parity_tolerance(shape)
    S = len(prompts)
    for s in range(S):
        ctx.reset_sample(s)
        ctx.prefill(s, prompts[s])
    out = ctx.generate(S, n_new)
    for s in range(S):
        low = np.nonzero(margins[s] <= 2 * tol)[0]
        upto = int(low[0]) if low.size else n_new
        assert list(out[s, :upto]) == toks[s][:upto], s
    return out


CASES = [
    # arch, dtype, L, d, H, n_kv, V, C, bounds, S, P, N, opts
    ("gpt", I.DT_F32, 4, 64, 4, None, 97, 64, [0, 4], 1, 5, 12, {}),
    ("gpt", I.DT_F32, 4, 64, 4, None, 97, 64, [0, 1, 2, 4], 3, 7, 20, dict(page_tokens=4, attn_splits=3)),
    ("gpt", I.DT_BF16, 4, 64, 4, None, 97, 64, [0, 2, 4], 5, 9, 16, dict(page_tokens=8, attn_splits=2)),
    ("gpt", I.DT_BF16, 4, 64, 4, None, 97, 64, [0, 2, 4], 5, 9, 16, dict(page_tokens=8, attn_splits=2, kv_cache_dtype=1)),
    ("gpt", I.DT_BF16, 3, 128, 2, None, 131, 96, [0, 1, 2, 3], 2, 17, 30, dict(attn_splits=4)),
    ("gpt", I.DT_BF16, 3, 128, 2, None, 131, 96, [0, 1, 2, 3], 2, 17, 30, dict(attn_splits=4, prefill_mode=1)),
    ("llama", I.DT_BF16, 4, 64, 4, None, 101, 64, [0, 2, 3, 4], 3, 6, 20, dict(page_tokens=4, attn_splits=2)),
    ("llama", I.DT_BF16, 4, 64, 4, None, 101, 64, [0, 2, 3, 4], 3, 6, 20, dict(page_tokens=4, attn_splits=2, kv_cache_dtype=1)),
    ("gpt", I.DT_BF16, 4, 64, 4, None, 97, 64, [0, 2, 4], 5, 9, 16, dict(page_tokens=8, attn_splits=2, kv_cache_dtype=2)),   # fp16 cache
    ("llama", I.DT_BF16, 4, 64, 4, 2, 101, 64, [0, 2, 3, 4], 3, 6, 20, dict(page_tokens=4, attn_splits=2, kv_cache_dtype=2)),
    ("llama", I.DT_BF16, 2, 256, 2, 1, 300, 40, [0, 2], 11, 3, 10, dict(kv_cache_dtype=2)),   # fp16 cache, tensor-core steps
    ("llama", I.DT_F32, 2, 128, 4, 2, 67, 48, [0, 1, 2], 4, 11, 14, dict(attn_splits=3)),
    ("llama", I.DT_BF16, 2, 256, 2, 1, 300, 40, [0, 2], 11, 3, 10, {}),         # one partition, group > 8 items
    ("llama", I.DT_BF16, 2, 256, 2, 1, 300, 40, [0, 2], 11, 3, 10, dict(prefill_mode=1)),   # the same on the CUDA-core kernels
    ("llama", I.DT_BF16, 2, 256, 2, 1, 300, 200, [0, 1, 2], 2, 150, 6, {}),     # prompt longer than one prefill chunk
    ("llama", I.DT_BF16, 2, 256, 2, 1, 300, 40, [0, 2], 3, 9, 6, dict(prefill_mode=1)),
    ("gpt", I.DT_F32, 2, 64, 4, None, 50, 32, [0, 1, 2], 3, 10, 22, {}),        # prompt + new == n_ctx exactly
    ("gpt", I.DT_BF16, 4, 64, 2, None, 97, 64, [0, 1, 2, 3, 4], 1, 4, 9, {}),   # one sample, four partitions
    ("gpt", I.DT_BF16, 3, 128, 2, None, 131, 96, [0, 1, 2, 3], 5, 6, 12, dict(tc_min_group=1, attn_splits=2)),  # small groups on tensor cores
    ("gpt", I.DT_BF16, 2, 256, 4, None, 2100, 48, [0, 1, 2], 4, 5, 8, {}),      # d_ff 1024+: several tiles per warp, 2 per group
    ("gpt", I.DT_BF16, 4, 64, 2, None, 97, 64, [0, 1, 2, 3, 4], 1, 4, 9, {}),   # one sample, four partitions
    ("gpt", I.DT_BF16, 3, 128, 2, None, 131, 96, [0, 1, 2, 3], 5, 6, 12, dict(tc_min_group=1, attn_splits=2)),  # small groups on tensor cores
]


@pytest.mark.parametrize("scheduler", [0, 1], ids=["persistent", "streams"])
@pytest.mark.parametrize("arch,dtype,L,d,H,n_kv,V,C,bounds,S,P,N,opts", CASES)
def test_small_shapes_match_oracle(arch, dtype, L, d, H, n_kv, V, C, bounds, S, P, N, opts, scheduler):
    shape = tiny_shape(arch, dtype, L=L, d=d, H=H, V=V, C=C, n_kv=n_kv)
    orc, w = make_oracle(shape, seed=3, std=0.08 if dtype == I.DT_F32 else 0.04)
    prompts = I.make_prompts(V, S, P, seed=5)
    toks, lgs, margins = oracle_reference(orc, prompts, N)
    ctx = _ctx(shape, bounds, S, w, scheduler=scheduler, **opts)
    _check_teacher_forced_stepwise(ctx, shape, prompts, toks, lgs, margins, N)
    _check_free_running(ctx, shape, prompts, toks, margins, N)
    ctx.close()


def test_results_do_not_depend_on_partitioning_or_grouping():
    """Same model cut three ways and run with different numbers of samples in flight:
    the tokens and final logits of sample 0 stay the same to rounding."""
    shape = tiny_shape("gpt", I.DT_F32, L=4, d=64, H=4, V=97, C=64)
    orc, w = make_oracle(shape, seed=7, std=0.08)
    prompts = I.make_prompts(97, 6, 6, seed=2)
    ref = None
    for bounds, S in (([0, 4], 1), ([0, 2, 4], 2), ([0, 1, 2, 3, 4], 6), ([0, 1, 4], 5)):
        ctx = _ctx(shape, bounds, S, w)
        for s in range(S):
            ctx.prefill(s, prompts[s])
        out = ctx.generate(S, 10)
        lg = ctx.get_logits(0)
        if ref is None:
            ref = (out[0].copy(), lg)
        else:
            assert np.array_equal(out[0], ref[0])
            assert np.abs(lg - ref[1]).max() < 1e-5
        ctx.close()


def test_schedulers_agree():
    """Eager stream scheduler, captured steady-state windows and the persistent kernel give the same tokens."""
    shape = tiny_shape("gpt", I.DT_F32, L=3, d=64, H=4, V=97, C=128)
    orc, w = make_oracle(shape, seed=11, std=0.08)
    prompts = I.make_prompts(97, 3, 4, seed=2)
    outs = []
    for rpg, sched in ((-1, 1), (2, 1), (5, 1), (0, 2)):
        ctx = _ctx(shape, [0, 1, 2, 3], 3, w, rounds_per_graph=rpg, scheduler=sched)
        for s in range(3):
            ctx.prefill(s, prompts[s])
        a = ctx.generate(3, 50)
        b = ctx.generate(3, 40)          # resumed call: feeds the last token first
        outs.append(np.concatenate([a, b], axis=1))
        st = ctx.stats()
        assert st.kernel_launches > 0 and st.stage_steps > 0
        ctx.close()
    assert all(np.array_equal(outs[0], o) for o in outs[1:])
    toks, _, margins = oracle_reference(orc, prompts, 90)
    for s in range(3):
        low = np.nonzero(margins[s] <= 2e-4)[0]
        upto = int(low[0]) if low.size else 90
        assert list(outs[0][s, :upto]) == toks[s][:upto]


def test_step_entry_point_matches_oracle_chunks():
    """mdi_step: one sample, one partition, one position - against the oracle's chunk forward."""
    import torch
    from oracle import mdi_oracle as O
    shape = tiny_shape("llama", I.DT_BF16, L=4, d=64, H=4, V=101, C=32)
    orc, w = make_oracle(shape, seed=4, std=0.04)
    bounds = [0, 1, 3, 4]
    ctx = _ctx(shape, bounds, 2, w, page_tokens=4)
    caches = [[O.Cache(orc, lo, hi) for lo, hi in zip(bounds[:-1], bounds[1:])] for _ in range(2)]
    seq = {0: [5, 9, 2, 77, 13, 40], 1: [1, 1, 8]}
    tok_in = torch.zeros(1, dtype=torch.int32, device="cuda")
    tok_out = torch.zeros(1, dtype=torch.int32, device="cuda")
    acts = [torch.zeros(64, dtype=torch.float32, device="cuda") for _ in range(2)]
    for slot in (0, 1):
        for pos, t in enumerate(seq[slot]):
            tok_in.fill_(t)
            x = orc.embed([t], pos)
            ctx.step(0, slot, tok_in, acts[0])
            x = orc.blocks(caches[slot][0], x)
            ctx.sync()
            assert np.abs(acts[0].cpu().numpy() - x[0]).max() < 5e-3
            ctx.step(1, slot, acts[0], acts[1])
            x1 = orc.blocks(caches[slot][1], acts[0].cpu().numpy()[None])
            ctx.sync()
            assert np.abs(acts[1].cpu().numpy() - x1[0]).max() < 5e-3
            ctx.step(2, slot, acts[1], tok_out)
            x2 = orc.blocks(caches[slot][2], acts[1].cpu().numpy()[None])
            lg = orc.head(x2[0])
            got = ctx.get_logits(slot)
            assert np.abs(got - lg).max() < 3e-2
            top2 = np.sort(lg)[-2:]
            if top2[1] - top2[0] > 6e-2:
                assert int(tok_out.item()) == O.argmax(lg)
    ctx.close()


def test_errors_leave_the_context_usable():
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", I.DT_F32, L=2, d=64, H=4, V=50, C=32)
    orc, w = make_oracle(shape, seed=1)
    with pytest.raises(mdi.MdiError) as e:
        mdi.Context(shape, [0, 2, 1], 2)
    assert e.value.code == mdi.ERR_ARG
    ctx = mdi.Context(shape, [0, 1, 2], 2, page_tokens=4, kv_pool_tokens=24)
    with pytest.raises(mdi.MdiError) as e:
        ctx.prefill(0, [1, 2, 3])
    assert e.value.code == mdi.ERR_STATE                       # weights missing
    with pytest.raises(mdi.MdiError) as e:
        ctx.load_weights("no.such", np.zeros(4, np.float32))
    assert e.value.code == mdi.ERR_ARG
    with pytest.raises(mdi.MdiError) as e:
        ctx.load_weights("wte", np.zeros(4, np.float32))
    assert e.value.code == mdi.ERR_SHAPE
    ctx.load_all(w)
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(2, 4)
    assert e.value.code == mdi.ERR_STATE                       # not prefilled
    with pytest.raises(mdi.MdiError) as e:
        ctx.prefill(0, list(range(33)))
    assert e.value.code == mdi.ERR_CONTEXT
    ctx.prefill(0, [1, 2, 3, 4, 5])
    with pytest.raises(mdi.MdiError) as e:
        ctx.prefill(0, [1, 2, 3])
    assert e.value.code == mdi.ERR_STATE                       # slot already holds tokens
    with pytest.raises(mdi.MdiError) as e:
        ctx.prefill(1, list(range(1, 22)))                     # 5 + 21 rows > pool of 24 tokens
    assert e.value.code == mdi.ERR_OOM
    ctx.prefill(1, [7, 8])
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(2, 40)
    assert e.value.code == mdi.ERR_CONTEXT
    out = ctx.generate(2, 6)                                   # still works after the failures
    toks, _, margins = oracle_reference(orc, [[1, 2, 3, 4, 5], [7, 8]], 6)
    for s in range(2):
        low = np.nonzero(margins[s] <= 2e-4)[0]
        upto = int(low[0]) if low.size else 6
        assert list(out[s, :upto]) == toks[s][:upto]
    st = ctx.stats()
    assert st.kv_pages_in_use[0] > 0
    ctx.reset_sample(0)
    ctx.reset_sample(1)
    assert ctx.stats().kv_pages_in_use[0] == 0
    ctx.close()
