"""The five named workloads against the CPU oracle, through the C ABI.

Every workload runs at its full model shape, partitioning, number of samples in flight and prompt length, in the
launch configuration bench.py times; the generation length is the workload's own (the Llama-7B shape: 256 of its
512 new tokens unless pytest is given --full-lengths).  For the three large shapes the oracle follows a stated
subset of the samples (first and last slot), so that the CPU side finishes in a few minutes.

Protocol as in test_gpu_parity.py: checked samples are teacher-forced with the oracle's tokens; every
token must equal the oracle's where its top-1/top-2 margin exceeds twice the logit tolerance; logits are
compared (max |delta| <= tolerance) at the end of every chunk of steps.
"""
import numpy as np
import pytest

from oracle import mdi_oracle as O
from paper_2505_18164_b200 import inputs as I
from helpers import parity_tolerance

pytestmark = pytest.mark.gpu


def _run(name, n_prompt=None, n_new=None, check=None, chunk=8, scheduler=0, **ctx_opts):
    from paper_2505_18164_b200 import mdi
    w = I.ALL_WORKLOADS[name]
    w = I.scaled(w, n_prompt=n_prompt or w.n_prompt, n_new=n_new or w.n_new)
    s, S, P, N = w.shape, w.n_samples, w.n_prompt, w.n_new
    check = list(range(S)) if check is None else check
    tol = parity_tolerance(s)
    ctx = mdi.Context(s, list(w.part_bounds), S, kv_pool_tokens=S * ((P + N + 15) // 16 * 16), scheduler=scheduler, **ctx_opts)
    weights = {}
    for nm, a in I.iter_weights(s, w.weight_seed):
        ctx.load_weights(nm, a)
        weights[nm] = a
    orc = O.Oracle(s, weights)
    prompts = I.make_prompts(s.vocab, S, P, w.prompt_seed)
    ref = {smp: orc.generate_sequential([int(t) for t in prompts[smp]], N, list(w.part_bounds)) for smp in check}
    for smp in range(S):
        if smp in ref:
            ctx.set_teacher_tokens(smp, ref[smp][0])
        ctx.prefill(smp, prompts[smp])
    got = np.zeros((S, N), np.int32)
    worst, done = 0.0, 0
    while done < N:
        n = min(chunk, N - done)
        got[:, done:done + n] = ctx.generate(S, n)
        done += n
        for smp in check:
            worst = max(worst, float(np.abs(ctx.get_logits(smp) - ref[smp][1][done - 1]).max()))
    gated = 0
    for smp in check:
        toks, lg = ref[smp]
        top2 = np.sort(lg, axis=1)[:, -2:]
        ok = (top2[:, 1] - top2[:, 0]) > 2 * tol
        gated += int((~ok).sum())
        assert np.array_equal(got[smp][ok], np.asarray(toks)[ok]), f"{name}: sample {smp} tokens differ from the oracle"
    print(f"{name}: worst |dlogit| {worst:.3e} (tol {tol:g}), margin-gated {gated}/{len(check) * N} steps, "
          f"{ctx.stats().kernel_launches} launches")
    assert worst <= tol, worst
    ctx.close()
    return worst


@pytest.mark.parametrize("scheduler", [0, 1], ids=["persistent", "streams"])
def test_tiny_gpt_fp32_full(scheduler):
    _run("tiny_gpt_fp32", scheduler=scheduler)


def test_gpt2_small_full_size_as_benchmarked():
    _run("gpt2_small", chunk=64)


def test_gpt2_small_stream_scheduler_short():
    _run("gpt2_small", n_new=40, chunk=20, scheduler=1)


def test_gpt2_medium_full_size():
    """Full prompts and generation length (128 + 768): caches grow over seven 128-row pages with two samples per
    group; first and last slot follow the oracle."""
    _run("gpt2_medium", check=[0, 7], chunk=64)


def test_gpt2_xl_full_size_ends_at_the_context_limit():
    """256-token prompts + 768 new tokens = n_ctx: the last token is produced from position 1022 and never fed, so
    1023 rows are cached; groups of 3,3,3,3,2,2 samples; every attention split holds rows."""
    w = I.ALL_WORKLOADS["gpt2_xl"]
    assert w.n_prompt + w.n_new == w.shape.n_ctx
    _run("gpt2_xl", check=[0, 15], chunk=64)


def test_llama_7b_long(full_lengths):
    """Full 128-token prompts, groups of eight on the tensor cores, slots 0 and 63 against the oracle; 256 new tokens
    by default, all 512 with --full-lengths."""
    _run("llama_7b", n_new=None if full_lengths else 256, check=[0, 63], chunk=32)


@pytest.mark.parametrize("name", ["nanollama_3nodes", "nanollama_2nodes", "tinyllama_3nodes"])
def test_paper_model_shapes(name):
    """The paper's own models as synthetic fp32 shapes: unequal partitions, one-token prompts (Section IV-A)."""
    _run(name, n_new=10, check=[0, 2], chunk=5)
