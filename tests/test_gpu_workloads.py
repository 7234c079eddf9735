"""The five named workloads against the CPU oracle, through the C ABI.

gpt2_small runs at its full size (3 samples, 64-token prompts, 512 new tokens) in the launch
configuration bench.py times; the larger shapes keep their full model shape, partitioning and number of
samples in flight but shorter prompts and generations, and the oracle follows a stated subset of the
samples (first and last slot), so that the CPU side finishes in seconds to a few minutes.

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


def _run(name, n_prompt=None, n_new=None, check=None, chunk=8, scheduler=0):
    from paper_2505_18164_b200 import mdi
    w = I.ALL_WORKLOADS[name]
    w = I.scaled(w, n_prompt=n_prompt or w.n_prompt, n_new=n_new or w.n_new)
    s, S, P, N = w.shape, w.n_samples, w.n_prompt, w.n_new
    check = list(range(S)) if check is None else check
    tol = parity_tolerance(s)
    ctx = mdi.Context(s, list(w.part_bounds), S, kv_pool_tokens=S * ((P + N + 15) // 16 * 16), scheduler=scheduler)
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


@pytest.mark.parametrize("scheduler", [0, 1], ids=["persistent", "streams"])
def test_tiny_gpt_fp32_full(scheduler):
    _run("tiny_gpt_fp32", scheduler=scheduler)


def test_gpt2_small_full_size_as_benchmarked():
    _run("gpt2_small", chunk=64)


def test_gpt2_small_stream_scheduler_short():
    _run("gpt2_small", n_new=40, chunk=20, scheduler=1)


def test_gpt2_medium_shape():
    _run("gpt2_medium", n_prompt=32, n_new=24, check=[0, 7])


def test_gpt2_xl_shape_uneven_groups():
    _run("gpt2_xl", n_prompt=16, n_new=12, check=[0, 15], chunk=6)


def test_llama_7b_shape_groups_of_eight():
    _run("llama_7b", n_prompt=8, n_new=6, check=[0, 63], chunk=3)


@pytest.mark.parametrize("name", ["nanollama_3nodes", "nanollama_2nodes", "tinyllama_3nodes"])
def test_paper_model_shapes(name):
    """The paper's own models as synthetic fp32 shapes: unequal partitions, one-token prompts (Section IV-A)."""
    _run(name, n_new=10, check=[0, 2], chunk=5)
