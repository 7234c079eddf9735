"""Edge cases of the C-ABI calls on the GPU: degenerate sizes, slot reuse, context boundary."""
import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, oracle_reference, tiny_shape

pytestmark = pytest.mark.gpu


def _safe_prefix(toks, margins, tol):
    low = np.nonzero(margins <= 2 * tol)[0]
    return int(low[0]) if low.size else len(toks)


@pytest.mark.parametrize("dtype,scheduler", [(I.DT_F32, 0), (I.DT_F32, 1), (I.DT_BF16, 0), (I.DT_BF16, 1)])
def test_degenerate_sizes_and_slot_reuse(dtype, scheduler):
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", dtype, L=3, d=64, H=4, V=97, C=48)
    orc, w = make_oracle(shape, seed=9, std=0.06)
    tol = 1e-4 if dtype == I.DT_F32 else 3e-2
    ctx = mdi.Context(shape, [0, 1, 2, 3], 4, page_tokens=4, scheduler=scheduler)
    ctx.load_all(w)
    prompts = [[5], [7, 8, 9, 10, 11, 12, 13], [1, 2]]              # a one-token prompt among them
    toks, _, margins = oracle_reference(orc, prompts, 10)
    for s, p in enumerate(prompts):
        ctx.prefill(s, p)
    # fewer samples than slots; zero new tokens is a no-op that leaves the pending token pending
    assert ctx.generate(3, 0).shape == (3, 0)
    first = ctx.generate(3, 1)                                      # only the pending tokens: no pipeline pass at all
    rest = ctx.generate(3, 9)
    out = np.concatenate([first, rest], axis=1)
    for s in range(3):
        n = _safe_prefix(toks[s], margins[s], tol)
        assert list(out[s, :n]) == toks[s][:n]
    # reuse slot 1 for another prompt while the others keep their state; then a call over a subset of the samples
    pages_before = ctx.stats().kv_pages_in_use[0]
    ctx.reset_sample(1)
    assert ctx.stats().kv_pages_in_use[0] < pages_before
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(3, 2)                                          # sample 1 has no prompt now
    assert e.value.code == mdi.ERR_STATE
    ctx.reset_sample(0)
    ctx.reset_sample(2)
    p2 = [33, 34, 35, 36]
    t2, _, m2 = oracle_reference(orc, [p2], 8)
    ctx.prefill(0, p2)
    out2 = ctx.generate(1, 8)
    n = _safe_prefix(t2[0], m2[0], tol)
    assert list(out2[0, :n]) == t2[0][:n]
    ctx.close()


def test_context_boundary():
    """prompt + new == n_ctx + 1 is legal (the last token is never fed); one more is refused."""
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("llama", I.DT_BF16, L=2, d=64, H=4, V=101, C=24)
    orc, w = make_oracle(shape, seed=2, std=0.06)
    ctx = mdi.Context(shape, [0, 1, 2], 2, page_tokens=8)
    ctx.load_all(w)
    prompts = I.make_prompts(101, 2, 10, seed=6)
    toks, _, margins = oracle_reference(orc, prompts, 15)          # 10 + 15 == 24 + 1
    for s in range(2):
        ctx.prefill(s, prompts[s])
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(2, 16)
    assert e.value.code == mdi.ERR_CONTEXT
    out = ctx.generate(2, 15)
    for s in range(2):
        n = _safe_prefix(toks[s], margins[s], 3e-2)
        assert list(out[s, :n]) == toks[s][:n]
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(2, 1)                                          # would have to feed a 25th position
    assert e.value.code == mdi.ERR_CONTEXT
    ctx.close()


def test_generate_dev_and_prefill_dev_match_host_forms():
    import torch
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", I.DT_BF16, L=2, d=64, H=4, V=97, C=32)
    _, w = make_oracle(shape, seed=5, std=0.06)
    prompts = I.make_prompts(97, 3, 6, seed=3)
    res = []
    for dev in (False, True):
        ctx = mdi.Context(shape, [0, 1, 2], 3)
        ctx.load_all(w)
        if dev:
            pd = torch.from_numpy(prompts).cuda()
            out = torch.zeros((3, 12), dtype=torch.int32, device="cuda")
            for s in range(3):
                ctx.prefill_dev(s, pd[s], 6)
            ctx.generate_dev(3, 12, out)
            res.append(out.cpu().numpy())
        else:
            for s in range(3):
                ctx.prefill(s, prompts[s])
            res.append(ctx.generate(3, 12))
        ctx.close()
    assert np.array_equal(res[0], res[1])


def test_a_withheld_handoff_times_out_and_the_context_survives():
    """Failure detection without faulting anything: partition 0 is told to withhold its output handoff once, the
    waits are given 50 ms, the call must come back with MDI_ERR_TIMEOUT (not hang), the samples are reset, and
    the same context then generates correctly."""
    import time
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", I.DT_F32, L=3, d=64, H=4, V=97, C=48)
    orc, w = make_oracle(shape, seed=9, std=0.06)
    ctx = mdi.Context(shape, [0, 1, 2, 3], 3, scheduler=2, wait_limit_ms=50, debug_withhold_handoff=1)
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
    with pytest.raises(mdi.MdiError) as e:
        ctx.generate(3, 2)
    assert e.value.code == mdi.ERR_STATE                            # nothing is prefilled any more
    toks, _, margins = oracle_reference(orc, prompts, 8)
    for s in range(3):
        ctx.prefill(s, prompts[s])
    out = ctx.generate(3, 8)                                        # the hook was one-shot: this run is normal
    for s in range(3):
        n = _safe_prefix(toks[s], margins[s], 1e-4)
        assert list(out[s, :n]) == toks[s][:n]
    ctx.close()


def test_weights_loaded_again_replace_the_tiled_copies():
    """The tensor-core linear layers read tiled copies of the matrices: loading other weights into the same context
    must rebuild them (first visits and decode steps both on the tensor-core path)."""
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("llama", I.DT_BF16, L=2, d=256, H=2, V=300, C=40, n_kv=1)
    prompts = I.make_prompts(300, 3, 9, seed=4)
    ctx = mdi.Context(shape, [0, 1, 2], 3, scheduler=1, tc_min_group=1)
    for seed in (3, 11):
        orc, w = make_oracle(shape, seed=seed, std=0.04)
        toks, lgs, margins = oracle_reference(orc, prompts, 6)
        ctx.load_all(w)
        for s in range(3):
            ctx.reset_sample(s)
            ctx.prefill(s, prompts[s])
        out = ctx.generate(3, 6)
        for s in range(3):
            n = _safe_prefix(toks[s], margins[s], 3e-2)
            assert list(out[s, :n]) == toks[s][:n], (seed, s)
            if n == 6:
                assert np.abs(ctx.get_logits(s) - lgs[s][5]).max() < 3e-2
    ctx.close()
