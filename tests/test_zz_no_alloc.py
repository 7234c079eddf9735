"""The allocation-free greedy argmax entry point (mdi_greedy_argmax_static) against the library's own
output layer.

Some callers cannot allocate device memory where they choose tokens (their own pool owns the device, or an
allocation's implicit synchronisation is not acceptable there), so this entry point keeps its working memory
in a fixed array inside the library.  The check: run the normal path (mdi_generate), fetch the logits of
each sample's last output-layer evaluation, hand them to the new entry point through the C ABI and require
the same token ids - integer work, so bit-exact - on two calls in a row (the fixed array is reused and keeps
the first call's contents).  This file sorts last so that a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I
from helpers import make_oracle, tiny_shape

pytestmark = pytest.mark.gpu


def test_static_argmax_matches_generate_twice_in_a_row():
    import torch
    from paper_2505_18164_b200 import mdi
    V = 2100                                     # three blocks of columns, the last one ragged
    shape = tiny_shape("gpt", I.DT_F32, L=2, d=64, H=4, V=V, C=32)
    _, w = make_oracle(shape, seed=21, std=0.08)
    S = 3
    prompts = I.make_prompts(V, S, 5, seed=8)
    ctx = mdi.Context(shape, [0, 1, 2], S)
    ctx.load_all(w)
    for s in range(S):
        ctx.prefill(s, prompts[s])
    out = torch.full((S,), -1, dtype=torch.int32, device="cuda")
    for call in range(2):
        toks = ctx.generate(S, 3)                # existing entry point: last column = argmax of the last logits
        logits = np.stack([ctx.get_logits(s) for s in range(S)])
        dev = torch.from_numpy(logits).cuda()
        out.fill_(-1)
        mdi.greedy_argmax_static(dev, S, V, out, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.array_equal(got, toks[:, -1]), (call, got, toks[:, -1])
        assert np.array_equal(got, logits.argmax(axis=1))
    # ties go to the lowest index, also across blocks of columns
    tie = torch.zeros((2, V), dtype=torch.float32, device="cuda")
    tie[0, 1500] = 1.0
    tie[0, 700] = 1.0
    tie[1, 2099] = 3.0
    mdi.greedy_argmax_static(tie, 2, V, out, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert out.cpu().numpy()[:2].tolist() == [700, 2099]
    ctx.close()


def test_static_argmax_rejects_sizes_beyond_its_fixed_scratch():
    import torch
    from paper_2505_18164_b200 import mdi
    x = torch.zeros(8, dtype=torch.float32, device="cuda")
    out = torch.zeros(8, dtype=torch.int32, device="cuda")
    for rows, cols in ((65, 8), (1, 262145)):
        with pytest.raises(mdi.MdiError) as e:
            mdi.greedy_argmax_static(x, rows, cols, out)
        assert e.value.code == mdi.ERR_SHAPE and "exceeds the fixed scratch" in str(e.value)
    with pytest.raises(mdi.MdiError) as e:
        mdi.greedy_argmax_static(None, 1, 8, out)
    assert e.value.code == mdi.ERR_ARG
