"""Sampling from the pmf (temperature, top-k) on the GPU against the CPU oracle.

Two checks per step, both through the C ABI: (1) teacher-forced with the oracle's sampled tokens, the logits
agree within the usual tolerance; (2) the token the library drew equals the oracle's sampler applied to the
library's own logits with the same counter-based uniform - integer work decided in fp64 on both sides, so the
comparison is exact."""
import numpy as np
import pytest

from oracle import mdi_oracle as O
from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, parity_tolerance, tiny_shape

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("arch,dtype,V,top_k,temperature", [("gpt", I.DT_F32, 97, 5, 1.0), ("llama", I.DT_BF16, 2100, 40, 0.7),
                                                          ("gpt", I.DT_BF16, 300, 64, 1.6), ("gpt", I.DT_F32, 50, 1, 0.5)])
def test_sampled_tokens_reproduce_from_the_logits(arch, dtype, V, top_k, temperature):
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape(arch, dtype, L=3, d=64, H=4, V=V, C=48)
    orc, w = make_oracle(shape, seed=13, std=0.08 if dtype == I.DT_F32 else 0.04)
    S, P, N, seed = 4, 6, 14, 2025
    prompts = I.make_prompts(V, S, P, seed=9)
    ref = [orc.generate_sequential([int(t) for t in prompts[s]], N, sampler=(temperature, top_k, seed, s)) for s in range(S)]
    ctx = mdi.Context(shape, [0, 1, 2, 3], S)
    ctx.load_all(w)
    ctx.set_sampling(temperature, top_k, seed)
    for s in range(S):
        ctx.set_teacher_tokens(s, ref[s][0])
        ctx.prefill(s, prompts[s])
    tol, worst, same_as_oracle = parity_tolerance(shape), 0.0, 0
    for i in range(N):
        out = ctx.generate(S, 1)
        for s in range(S):
            lg = ctx.get_logits(s)
            worst = max(worst, float(np.abs(lg - ref[s][1][i]).max()))
            assert out[s, 0] == O.sample_top_k(lg, top_k, temperature, O.sample_uniform(seed, s, i)), (s, i)
            same_as_oracle += int(out[s, 0] == ref[s][0][i])
    assert worst <= tol, worst
    assert same_as_oracle >= 0.9 * S * N                # logits differ by rounding only, so nearly every draw agrees
    if top_k == 1:                                        # top-1 sampling is the greedy argmax
        assert same_as_oracle == S * N or dtype != I.DT_F32
    # back to greedy on the same context
    ctx.set_sampling(0.0, 0, 0)
    for s in range(S):
        ctx.reset_sample(s)
        ctx.prefill(s, prompts[s])
    g = ctx.generate(S, 4)
    for s in range(S):
        assert g[s, -1] == int(np.argmax(ctx.get_logits(s)))
    with pytest.raises(mdi.MdiError) as e:
        ctx.set_sampling(1.0, 65, 1)
    assert e.value.code == mdi.ERR_ARG
    ctx.close()


def test_sampling_parameters_reach_replayed_graph_windows():
    """The stream scheduler replays captured windows of the schedule; the token-choice parameters travel in kernel
    arguments, so a change of them must not be answered from a window captured before it.  Sample with seed A over
    several windows, then switch to seed B, then to greedy, and check every token against the oracle's sampler
    (or the argmax) applied to the library's own logits."""
    from paper_2505_18164_b200 import mdi
    shape = tiny_shape("gpt", I.DT_F32, L=2, d=64, H=4, V=97, C=64)
    _, w = make_oracle(shape, seed=13, std=0.08)
    S, P, n = 3, 4, 6
    prompts = I.make_prompts(97, S, P, seed=9)
    ctx = mdi.Context(shape, [0, 1, 2], S, scheduler=1, rounds_per_graph=2)
    ctx.load_all(w)
    launches_before = None
    for temperature, top_k, seed in ((1.3, 20, 111), (1.3, 20, 222), (0.0, 0, 0), (0.9, 7, 222)):
        ctx.set_sampling(temperature, top_k, seed)
        for s in range(S):
            ctx.reset_sample(s)
            ctx.prefill(s, prompts[s])
        # one call over several windows, then token by token so that every step's logits can be read back
        block = ctx.generate(S, n).copy()
        for s in range(S):
            ctx.reset_sample(s)
            ctx.set_teacher_tokens(s, block[s])
            ctx.prefill(s, prompts[s])
        for i in range(n):
            out = ctx.generate(S, 1)
            for s in range(S):
                lg = ctx.get_logits(s)
                want = (O.sample_top_k(lg, top_k, temperature, O.sample_uniform(seed, s, i)) if temperature > 0
                        else int(np.argmax(lg)))
                assert out[s, 0] == want == block[s, i], (temperature, seed, s, i)
    ctx.close()
