"""CPU-only checks of the product side: the C-ABI library loads and exports what include/mdi.h declares,
the workload tables are consistent, and the multi-process aggregation of bench.py works (gloo, 2 ranks)."""
import ctypes
import os
import re
import subprocess
import sys
import textwrap

import numpy as np
import pytest

from paper_2505_18164_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "mdi.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(mdi_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2505_18164_b200 import mdi
    L = ctypes.CDLL(mdi.LIB_PATH)
    names = _declared()
    assert "mdi_create" in names and "mdi_generate" in names and "mdi_step" in names and len(names) >= 17
    for n in names:
        assert hasattr(L, n), n
    assert sorted(mdi.EXPORTS) == names            # the binding covers the same set


def test_create_without_gpu_fails_cleanly_or_gives_a_context():
    """No compute here: either there is no CUDA device (error code, message, no crash) or creation works."""
    from paper_2505_18164_b200 import mdi
    shape = I.WORKLOADS["tiny_gpt_fp32"].shape
    try:
        ctx = mdi.Context(shape, [0, 2, 4, 6], 3)
    except mdi.MdiError as e:
        assert e.code in (mdi.ERR_CUDA, mdi.ERR_OOM) and str(e)
    else:
        assert ctx.memory_bytes(0) > 0
        ctx.close()
    with pytest.raises(mdi.MdiError) as e:
        mdi.Context(shape, [0, 6, 4], 3)
    assert e.value.code == mdi.ERR_ARG             # argument checks come before any device work


def test_workload_tables():
    assert I.WORKLOAD_ORDER == ["tiny_gpt_fp32", "gpt2_small", "gpt2_medium", "gpt2_xl", "llama_7b"]
    for name in I.WORKLOAD_ORDER:
        w = I.WORKLOADS[name]
        s = w.shape
        assert w.part_bounds[0] == 0 and w.part_bounds[-1] == s.n_layer
        assert all(b > a for a, b in zip(w.part_bounds[:-1], w.part_bounds[1:]))
        assert w.n_prompt + w.n_new <= s.n_ctx + 1
        assert s.n_head * s.head_dim == s.d_model
    # the paper's small model: 304 million parameters (Section IV-A)
    nano = I.param_bytes(I.PAPER_SHAPES["nanollama_3nodes"].shape) / 4
    assert abs(nano - 304e6) < 3e6
    assert abs(I.param_bytes(I.PAPER_SHAPES["tinyllama_3nodes"].shape) / 4 - 1.1e9) < 0.02e9
    # sizes quoted for the shapes: whole-model parameter bytes
    mb = {n: I.param_bytes(I.WORKLOADS[n].shape) / 1e6 for n in I.WORKLOAD_ORDER}
    assert abs(mb["gpt2_small"] - 248.9) < 1.0     # 247.3 MB of matrices + wpe
    assert abs(mb["llama_7b"] - 13476.8) < 5.0
    specs = dict((n, shp) for n, shp, _ in I.tensor_specs(I.WORKLOADS["llama_7b"].shape))
    assert specs["h.0.attn.wqkv"] == (3 * 4096, 4096) and specs["h.31.mlp.wdown"] == (4096, 11008) and "wpe" not in specs


def test_generator_is_deterministic_and_sliceable():
    a = I.make_tensor(0, 5, (7, 9), "normal", I.DT_F32)
    b = I.make_tensor(0, 5, (7, 9), "normal", I.DT_F32)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, I.make_tensor(0, 6, (7, 9), "normal", I.DT_F32))
    h = I.make_tensor(0, 5, (7, 9), "normal", I.DT_BF16)
    f = I.bf16_bits_to_f32(h)
    assert np.abs(f - a).max() <= np.abs(a).max() * 2.0 ** -8     # round-to-nearest bfloat16 of the same values
    big = I.as_f32(I.make_tensor(3, 1, (400, 500), "normal", I.DT_F32))
    assert abs(float(big.mean())) < 3e-4 and abs(float(big.std()) - 0.02) < 3e-4
    p = I.make_prompts(65, 3, 16)
    assert p.shape == (3, 16) and p.min() >= 0 and p.max() < 65 and not np.array_equal(p[0], p[1])


def test_bench_aggregation_two_ranks_gloo(tmp_path):
    """bench.py --gpus N runs N independent replicas; its numbers combine as the max over ranks of the time
    and the sum of the tokens.  Two gloo ranks on CPU exercise exactly that code."""
    script = tmp_path / "agg.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        run_ms, e2e_ms = bench.max_over_ranks([100.0 + 50.0 * rank, 200.0 - 10.0 * rank], world, "cpu")
        v = bench.aggregate_tokens_per_s(world, 3, 512, 2, run_ms)
        if rank == 0:
            print(json.dumps(dict(run_ms=run_ms, e2e_ms=e2e_ms, value=v)))
        dist.destroy_process_group()
    """))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1]
    d = json.loads(line)
    assert d["run_ms"] == 150.0 and d["e2e_ms"] == 200.0
    assert abs(d["value"] - 2 * 3 * 512 * 2 / 0.150) < 1e-6


def test_reference_arm_prints_its_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
                          "--workload", "tiny_gpt_fp32"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    d = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_bench_byte_counts_and_cpu_sample_plans():
    """Bytes a round of the schedule must move (every group streams the model once, every sample reads its cache at
    the weights' width), against figures worked out by hand from the shapes: 12 d^2 + 13 d parameters per GPT block,
    4 d^2 + 3 d F + 2 d per Llama block, V d + norm vectors for the output layers, cache rows of 2 d elements."""
    import bench
    for name, kv_bpe, gb in (("tiny_gpt_fp32", 4, 0.1308), ("gpt2_small", 2, 0.7774), ("gpt2_medium", 2, 3.234), ("llama_7b", 2, 118.64)):
        w = I.WORKLOADS[name]
        s = w.shape
        bpe = 4 if s.weight_dtype == I.DT_F32 else 2
        block = (12 * s.d_model ** 2 + 13 * s.d_model) if s.arch == I.ARCH_GPT else (4 * s.d_model ** 2 + 3 * s.d_model * s.d_ff + 2 * s.d_model)
        head = s.vocab * s.d_model + (2 if s.arch == I.ARCH_GPT else 1) * s.d_model
        G = min(w.n_samples, w.n_partitions)
        n_pass = w.n_new - 1
        mean_rows = w.n_prompt + (n_pass - 1) / 2 + 1                      # rows read per pass, averaged, plus the one written
        want = G * (s.n_layer * block + head) * bpe + w.n_samples * s.n_layer * 2 * s.d_model * (mean_rows + 1) * kv_bpe
        got = bench.decode_bytes(w, w.n_samples, kv_bpe)
        assert got["passes"] == n_pass and abs(got["total"] / n_pass - want) < 1e-6 * want
        assert abs(got["total"] / n_pass / 1e9 - gb) < 2e-3 * gb
    assert bench.oracle_sample_plan(I.WORKLOADS["tiny_gpt_fp32"], 16) == ("full",)
    kind, p_s, n_s = bench.oracle_sample_plan(I.WORKLOADS["llama_7b"], 16)
    assert kind == "slot0" and 8 <= p_s <= 128 and 8 <= n_s <= 511
    for name in I.WORKLOAD_ORDER:                                         # the two arms describe the workload alike
        w = I.WORKLOADS[name]
        assert bench.workload_config(w, 1)["workload"] == name and bench.workload_config(w, 1) == bench.workload_config(w, 1)
